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
    // Packed batch: tiles listed heaviest first by pec_plan_worklist (device, 4 x int32 per tile:
    // first row of the request, position of the tile's first row, rows, request length), or nullptr
    // to let every CTA search cu_seqlens.
    const int32_t *worklist;
    int32_t n_items;
    // Single request: the query rows of the call as up to two ascending segments of positions
    // (a chunk is one segment, the rows of a zigzag partition are two), each cut into tiles from its
    // own first row.  Row r of o / lse belongs to position out_pos0 + r.
    int64_t q_lo[2], q_hi[2];
    int32_t n_qseg;
    int64_t out_pos0;
    int64_t total_rows;              // rows of o / lse (chunk_len, or packed total)
    // Incoming partial state of the same rows ([total_rows, Hq, D] fp32 / [total_rows, Hq]) that the
    // epilogue merges its own result into (online softmax across launches), or nullptr.  May alias o / lse.
    const float *acc_o;
    const float *acc_lse;
    // Key subset of a single request: up to two half-open intervals, already cut to the K/V
    // prefix.  Packed batches use [0, request length) per request instead.
    int64_t iv_lo[2], iv_hi[2];
    int32_t n_iv;
    int32_t causal;
    float scale;                     // softmax scale
    float scale_log2;                // scale * log2(e)
    int32_t o_is_bf16;
    int32_t overlap_previous;        // launch as a programmatic dependent of the preceding kernel on the stream
    int32_t *status;
    int64_t wait_cycles;             // limit of every device-side barrier wait, in SM clock cycles
    int32_t test_skip_last_load;     // test hook: the loader leaves out its last item (a wait must then run out)
    // Split-KV launches (decode): grid.z CTAs each take `split_keys` keys of interval 0 and write
    // their partial to slice blockIdx.z of o / lse ([splits][total_rows][Hq][D] / [splits][total_rows][Hq]).
    int32_t splits;                  // 1 = ordinary launch
    int64_t split_keys;              // multiple of 128
};

void set_error(const char *fmt, ...);

// Process-wide settings behind pec_control (pec_api.cpp).
int64_t wait_limit_cycles();
int32_t test_skip_last_load();

// Fills lo/hi with the two zigzag intervals of partition part_id (planner rule, see pec.h).
void zigzag_intervals(int64_t seq_len, int32_t num_parts, int32_t part_id, int32_t align,
                      int64_t lo[2], int64_t hi[2]);

// Kernel launchers (each returns a pec_status).
int launch_attn_f32(const AttnParams &p, cudaStream_t stream);
int launch_attn_prefill_bf16(const AttnParams &p, cudaStream_t stream);   // every launch that is not split over the keys
int launch_attn_split_bf16(const AttnParams &p, cudaStream_t stream);     // split-KV launches (decode)
// Rows [row_lo, row_hi) of o / lse that no CTA of an attention launch covers: zero / -inf, or a copy
// of the incoming state (rounded to the output type).
int launch_fill_rows(const AttnParams &p, int64_t row_lo, int64_t row_hi, cudaStream_t stream);
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
