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
                    if (fa[u] != 0.f) a[u] = ld_stream(reinterpret_cast<const float4 *>(o_a) + off);
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

int launch_merge(const float *o_a, const float *lse_a, const float *o_b, const float *lse_b,
                 void *o_out, float *lse_out, int64_t items, int out_is_bf16, int inplace,
                 cudaStream_t stream)
{
    static int sm_count = 0;
    if (sm_count == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sm_count <= 0) {
            sm_count = 0;
            set_error("pec_attn_merge: cannot query the device: %s", cudaGetErrorString(cudaGetLastError()));
            return PEC_ERR_CUDA;
        }
    }
    const int64_t n_groups = (items + kItemsPerWarp - 1) / kItemsPerWarp;
    const int64_t warps_per_cta = kMergeThreads / 32;
    int64_t ctas = (n_groups + warps_per_cta - 1) / warps_per_cta;
    const int64_t cap = (int64_t)sm_count * 8;          // 8 resident CTAs of 256 threads per SM
    if (ctas > cap) ctas = cap;
    if (out_is_bf16)  merge_kernel<true, false><<<(unsigned)ctas, kMergeThreads, 0, stream>>>(o_a, lse_a, o_b, lse_b, o_out, lse_out, items);
    else if (inplace) merge_kernel<false, true><<<(unsigned)ctas, kMergeThreads, 0, stream>>>(o_a, lse_a, o_b, lse_b, o_out, lse_out, items);
    else              merge_kernel<false, false><<<(unsigned)ctas, kMergeThreads, 0, stream>>>(o_a, lse_a, o_b, lse_b, o_out, lse_out, items);
    const cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) { set_error("pec_attn_merge: launch failed: %s", cudaGetErrorString(err)); return PEC_ERR_CUDA; }
    return PEC_OK;
}

}  // namespace pec
