// LSE merge of two partial attention results (online-softmax combination, Section 2.2):
//   lse = ln(e^{lse_a} + e^{lse_b});  o = e^{lse_a-lse} o_a + e^{lse_b-lse} o_b   per (row, head).
// HBM-bound: 2 reads + 1 write of 128 fp32 plus one LSE each = 1548 B per (row, head).
//
// A warp owns 32 consecutive (row, head) items.  Lane i loads the two LSE values of item i
// (one coalesced 128-byte request per side), computes that item's weights and writes its merged
// LSE; the weights are then broadcast with warp shuffles while all 32 lanes stream each item's
// 128 channels as one float4 per lane (512 contiguous bytes per item and side).  Sides whose
// weight is zero are not read, and an in-place merge whose side b is empty writes nothing.
#include <cuda_bf16.h>
#include "pec_internal.h"

namespace pec {

constexpr int kMergeThreads = 256;
constexpr int kItemsPerWarp = 32;
constexpr int kUnroll = 4;

// Streaming (evict-first) load; coherent, so the in-place form may read what it later overwrites.
__device__ __forceinline__ float4 ld_stream(const float4 *p) { return __ldcs(p); }

template <bool kOutBf16, bool kInplace>
__global__ void __launch_bounds__(kMergeThreads)
merge_kernel(const float *o_a, const float *lse_a, const float *__restrict__ o_b,
             const float *__restrict__ lse_b, void *o_out, float *lse_out, int64_t items)
{
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * kMergeThreads + threadIdx.x) >> 5;
    const int64_t n_warps = ((int64_t)gridDim.x * kMergeThreads) >> 5;
    const int64_t n_groups = (items + kItemsPerWarp - 1) / kItemsPerWarp;

    for (int64_t g = warp; g < n_groups; g += n_warps) {
        const int64_t base = g * kItemsPerWarp;
        const int64_t mine = base + lane;
        float wa = 0.f, wb = 0.f;
        if (mine < items) {
            const float la = lse_a[mine], lb = lse_b[mine];
            const float m = fmaxf(la, lb);
            float lse = -INFINITY;
            if (m != -INFINITY) {
                const float ea = expf(la - m), eb = expf(lb - m);   // the larger one is exactly 1
                const float tot = ea + eb;
                const float inv = 1.f / tot;
                wa = ea * inv;
                wb = eb * inv;
                lse = m + logf(tot);
            }
            if (!kInplace || lb != -INFINITY) lse_out[mine] = lse;
        }
        const int n_here = (items - base) < kItemsPerWarp ? (int)(items - base) : kItemsPerWarp;
#pragma unroll 1
        for (int i0 = 0; i0 < n_here; i0 += kUnroll) {
            float4 a[kUnroll], b[kUnroll];
            float fa[kUnroll], fb[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const int i = i0 + u;                       // warp-uniform
                fa[u] = __shfl_sync(0xffffffffu, wa, i & 31);
                fb[u] = __shfl_sync(0xffffffffu, wb, i & 31);
                a[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                b[u] = a[u];
                if (i < n_here) {
                    const int64_t off = (base + i) * (kHeadDim / 4) + lane;
                    if (fa[u] != 0.f && !(kInplace && fb[u] == 0.f)) a[u] = ld_stream(reinterpret_cast<const float4 *>(o_a) + off);   // in place with an empty b: a stays, unread
                    if (fb[u] != 0.f) b[u] = ld_stream(reinterpret_cast<const float4 *>(o_b) + off);
                }
            }
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const int i = i0 + u;
                if (i >= n_here) continue;
                if (kInplace && fb[u] == 0.f) continue;     // result is side a, already in place
                float4 r;
                r.x = fa[u] * a[u].x + fb[u] * b[u].x;
                r.y = fa[u] * a[u].y + fb[u] * b[u].y;
                r.z = fa[u] * a[u].z + fb[u] * b[u].z;
                r.w = fa[u] * a[u].w + fb[u] * b[u].w;
                const int64_t off = (base + i) * (kHeadDim / 4) + lane;
                if (kOutBf16) {
                    __nv_bfloat162 lo = __floats2bfloat162_rn(r.x, r.y);
                    __nv_bfloat162 hi = __floats2bfloat162_rn(r.z, r.w);
                    uint2 pk;
                    pk.x = *reinterpret_cast<uint32_t *>(&lo);
                    pk.y = *reinterpret_cast<uint32_t *>(&hi);
                    reinterpret_cast<uint2 *>(o_out)[off] = pk;
                } else {
                    reinterpret_cast<float4 *>(o_out)[off] = r;
                }
            }
        }
    }
}

// n-way form: lane i takes the n LSE values of item i, turns them into n weights (registers), and
// the weights of each item are again broadcast by shuffles while the lanes stream that item's
// channels from every part with a non-zero weight.  Bytes per item: at most (n + 1) * 516.
// The output may alias part 0: each item is read before it is written, by the same warp.
template <bool kOutBf16>
__global__ void __launch_bounds__(kMergeThreads)
merge_n_kernel(const MergeParts parts, void *o_out, float *lse_out, int64_t items)
{
    const int lane = threadIdx.x & 31;
    const int n = parts.n;
    const int64_t warp = ((int64_t)blockIdx.x * kMergeThreads + threadIdx.x) >> 5;
    const int64_t n_warps = ((int64_t)gridDim.x * kMergeThreads) >> 5;
    const int64_t n_groups = (items + kItemsPerWarp - 1) / kItemsPerWarp;

    for (int64_t g = warp; g < n_groups; g += n_warps) {
        const int64_t base = g * kItemsPerWarp;
        const int64_t mine = base + lane;
        float w[PEC_MERGE_MAX_PARTS];
#pragma unroll
        for (int k = 0; k < PEC_MERGE_MAX_PARTS; ++k) w[k] = 0.f;
        if (mine < items) {
            float m = -INFINITY;
#pragma unroll
            for (int k = 0; k < PEC_MERGE_MAX_PARTS; ++k)
                if (k < n) { w[k] = parts.lse[k][mine]; m = fmaxf(m, w[k]); }
            float lse = -INFINITY;
            if (m != -INFINITY) {
                float tot = 0.f;
#pragma unroll
                for (int k = 0; k < PEC_MERGE_MAX_PARTS; ++k)
                    if (k < n) { w[k] = expf(w[k] - m); tot += w[k]; }     // the largest one is exactly 1
                const float inv = 1.f / tot;
#pragma unroll
                for (int k = 0; k < PEC_MERGE_MAX_PARTS; ++k) w[k] *= inv;
                lse = m + logf(tot);
            } else {
#pragma unroll
                for (int k = 0; k < PEC_MERGE_MAX_PARTS; ++k) w[k] = 0.f;
            }
            lse_out[mine] = lse;
        }
        const int n_here = (items - base) < kItemsPerWarp ? (int)(items - base) : kItemsPerWarp;
#pragma unroll 2
        for (int i = 0; i < n_here; ++i) {
            const int64_t off = (base + i) * (kHeadDim / 4) + lane;
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            // four parts at a time: all their loads are issued before the first is used
#pragma unroll
            for (int k0 = 0; k0 < PEC_MERGE_MAX_PARTS; k0 += 4) {
                if (k0 < n) {                                  // warp-uniform
                    float f[4];
                    float4 v[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        f[u] = (k0 + u < n) ? __shfl_sync(0xffffffffu, w[k0 + u], i) : 0.f;
                        v[u] = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (f[u] != 0.f) v[u] = ld_stream(reinterpret_cast<const float4 *>(parts.o[k0 + u]) + off);
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        acc.x = fmaf(f[u], v[u].x, acc.x); acc.y = fmaf(f[u], v[u].y, acc.y);
                        acc.z = fmaf(f[u], v[u].z, acc.z); acc.w = fmaf(f[u], v[u].w, acc.w);
                    }
                }
            }
            if (kOutBf16) {
                __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y);
                __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z, acc.w);
                uint2 pk;
                pk.x = *reinterpret_cast<uint32_t *>(&lo);
                pk.y = *reinterpret_cast<uint32_t *>(&hi);
                reinterpret_cast<uint2 *>(o_out)[off] = pk;
            } else {
                reinterpret_cast<float4 *>(o_out)[off] = acc;
            }
        }
    }
}

// Rows of an attention call that no CTA covers because they see no key of the call's subset: the
// partial of such a row is the merge identity (o = 0, lse = -inf), or - with an incoming state - that
// state unchanged, rounded to the output type.  One float4 of a row per thread.
template <bool kOutBf16>
__global__ void __launch_bounds__(kMergeThreads)
fill_rows_kernel(void *o, float *lse, const float *__restrict__ acc_o, const float *__restrict__ acc_lse,
                 int64_t item_lo, int64_t item_hi)
{
    const int64_t n4 = (item_hi - item_lo) * (kHeadDim / 4);
    const int64_t stride = (int64_t)gridDim.x * kMergeThreads;
    for (int64_t i = (int64_t)blockIdx.x * kMergeThreads + threadIdx.x; i < n4; i += stride) {
        const int64_t off = item_lo * (kHeadDim / 4) + i;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (acc_o) v = ld_stream(reinterpret_cast<const float4 *>(acc_o) + off);
        if (kOutBf16) {
            __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y);
            __nv_bfloat162 hi = __floats2bfloat162_rn(v.z, v.w);
            uint2 pk;
            pk.x = *reinterpret_cast<uint32_t *>(&lo);
            pk.y = *reinterpret_cast<uint32_t *>(&hi);
            reinterpret_cast<uint2 *>(o)[off] = pk;
        } else {
            reinterpret_cast<float4 *>(o)[off] = v;
        }
        if ((i & (kHeadDim / 4 - 1)) == 0) {
            const int64_t item = item_lo + i / (kHeadDim / 4);
            lse[item] = acc_lse ? acc_lse[item] : -INFINITY;
        }
    }
}

static int merge_grid(int64_t items, const char *who, int64_t *ctas_out)
{
    static int sm_count = 0;
    if (sm_count == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sm_count <= 0) {
            sm_count = 0;
            set_error("%s: cannot query the device: %s", who, cudaGetErrorString(cudaGetLastError()));
            return PEC_ERR_CUDA;
        }
    }
    const int64_t n_groups = (items + kItemsPerWarp - 1) / kItemsPerWarp;
    const int64_t warps_per_cta = kMergeThreads / 32;
    int64_t ctas = (n_groups + warps_per_cta - 1) / warps_per_cta;
    const int64_t cap = (int64_t)sm_count * 8;
    *ctas_out = ctas > cap ? cap : ctas;
    return PEC_OK;
}

int launch_fill_rows(const AttnParams &p, int64_t row_lo, int64_t row_hi, cudaStream_t stream)
{
    if (row_hi <= row_lo) return PEC_OK;
    const int64_t item_lo = row_lo * p.Hq, item_hi = row_hi * p.Hq;
    int64_t ctas = 0;
    const int rc = merge_grid(item_hi - item_lo, "pec_prefill_attn", &ctas);
    if (rc != PEC_OK) return rc;
    if (p.o_is_bf16) fill_rows_kernel<true><<<(unsigned)ctas, kMergeThreads, 0, stream>>>(p.o, p.lse, p.acc_o, p.acc_lse, item_lo, item_hi);
    else             fill_rows_kernel<false><<<(unsigned)ctas, kMergeThreads, 0, stream>>>(p.o, p.lse, p.acc_o, p.acc_lse, item_lo, item_hi);
    const cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) { set_error("pec_prefill_attn: fill launch failed: %s", cudaGetErrorString(err)); return PEC_ERR_CUDA; }
    return PEC_OK;
}

int launch_merge_n(const MergeParts &parts, void *o_out, float *lse_out, int64_t items, int out_is_bf16,
                   cudaStream_t stream)
{
    int64_t ctas = 0;
    const int rc = merge_grid(items, "pec_attn_merge_n", &ctas);
    if (rc != PEC_OK) return rc;
    if (out_is_bf16) merge_n_kernel<true><<<(unsigned)ctas, kMergeThreads, 0, stream>>>(parts, o_out, lse_out, items);
    else             merge_n_kernel<false><<<(unsigned)ctas, kMergeThreads, 0, stream>>>(parts, o_out, lse_out, items);
    const cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) { set_error("pec_attn_merge_n: launch failed: %s", cudaGetErrorString(err)); return PEC_ERR_CUDA; }
    return PEC_OK;
}

int launch_merge(const float *o_a, const float *lse_a, const float *o_b, const float *lse_b,
                 void *o_out, float *lse_out, int64_t items, int out_is_bf16, int inplace,
                 cudaStream_t stream)
{
    int64_t ctas = 0;
    const int rc = merge_grid(items, "pec_attn_merge", &ctas);
    if (rc != PEC_OK) return rc;
    if (out_is_bf16)  merge_kernel<true, false><<<(unsigned)ctas, kMergeThreads, 0, stream>>>(o_a, lse_a, o_b, lse_b, o_out, lse_out, items);
    else if (inplace) merge_kernel<false, true><<<(unsigned)ctas, kMergeThreads, 0, stream>>>(o_a, lse_a, o_b, lse_b, o_out, lse_out, items);
    else              merge_kernel<false, false><<<(unsigned)ctas, kMergeThreads, 0, stream>>>(o_a, lse_a, o_b, lse_b, o_out, lse_out, items);
    const cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) { set_error("pec_attn_merge: launch failed: %s", cudaGetErrorString(err)); return PEC_ERR_CUDA; }
    return PEC_OK;
}

}  // namespace pec
