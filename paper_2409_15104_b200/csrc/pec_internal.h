// Internal declarations shared by the translation units of libpec.so (not part of the ABI).
#pragma once
#include <cstdint>
#include <cstddef>
#include <cuda_runtime.h>
#include "pec.h"

namespace pec {

constexpr int kHeadDim = 128;

// Host-resolved description of one attention launch, passed to kernels by value.
struct AttnParams {
    const void *q, *k, *v;
    void *o;
    float *lse;
    int64_t q_stride_t, q_stride_h, k_stride_t, k_stride_h, v_stride_t, v_stride_h;  // elements
    int32_t Hq, Hkv, group;          // group = Hq / Hkv
    const int32_t *cu_seqlens;       // device or nullptr
    int32_t B;
    int64_t chunk_start, chunk_len;  // single request: query rows handled by this call
    int64_t total_rows;              // rows of o / lse (chunk_len, or packed total)
    // Key subset of a single request: up to two half-open intervals, already cut to the K/V
    // prefix.  Packed batches use [0, request length) per request instead.
    int64_t iv_lo[2], iv_hi[2];
    int32_t n_iv;
    int32_t causal;
    float scale;                     // softmax scale
    float scale_log2;                // scale * log2(e)
    int32_t o_is_bf16;
    int32_t *status;
    // Split-KV launches (decode): grid.z CTAs each take `split_keys` keys of interval 0 and write
    // their partial to slice blockIdx.z of o / lse ([splits][total_rows][Hq][D] / [splits][total_rows][Hq]).
    int32_t splits;                  // 1 = ordinary launch
    int64_t split_keys;              // multiple of 128
};

void set_error(const char *fmt, ...);

// Fills lo/hi with the two zigzag intervals of partition part_id (planner rule, see pec.h).
void zigzag_intervals(int64_t seq_len, int32_t num_parts, int32_t part_id, int32_t align,
                      int64_t lo[2], int64_t hi[2]);

// Kernel launchers (each returns a pec_status).
int launch_attn_f32(const AttnParams &p, cudaStream_t stream);
int launch_attn_prefill_bf16(const AttnParams &p, cudaStream_t stream);   // every launch that is not split over the keys
int launch_attn_split_bf16(const AttnParams &p, cudaStream_t stream);     // split-KV launches (decode)
int launch_merge(const float *o_a, const float *lse_a, const float *o_b, const float *lse_b,
                 void *o_out, float *lse_out, int64_t items, int out_is_bf16, int inplace,
                 cudaStream_t stream);

// Split-KV decode (pec_decode.cu): sizes of the scratch one call needs.
struct DecodeShape {
    int32_t splits;
    int64_t split_keys;
    size_t scratch_bytes;            // partial O + partial LSE of every split
};

struct MergeParts {
    const float *o[PEC_MERGE_MAX_PARTS];
    const float *lse[PEC_MERGE_MAX_PARTS];
    int32_t n;
};
int launch_merge_n(const MergeParts &parts, void *o_out, float *lse_out, int64_t items, int out_is_bf16,
                   cudaStream_t stream);

}  // namespace pec
