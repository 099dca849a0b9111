// Split-KV decode attention for a long request's single new token (Section 5.2: the long request
// in its decode phase has one query token per head; each GPU holding part of its K/V computes the
// attention of that token over its own keys and the partial outputs are merged).
//
// HBM-bound: the keys and values of the range are read once (2 * keys * Hkv * 128 * 2 bytes).  The
// g = Hq / Hkv query heads that share a KV head are laid out as the g rows of one 128-row tile of
// that KV head, so the tensor-core prefill kernel does the work with every K/V byte used by all g
// heads; the key range is cut into slices, one CTA per (KV head, pair of slices) - its two stages
// take one slice each so that one slice's softmax overlaps the other's MMAs - whose partial
// (O, LSE) go to scratch memory and are combined by the small kernel below (same LSE merge as
// pec_attn_merge).
#include <cuda_bf16.h>
#include <cmath>
#include <mutex>
#include "pec_internal.h"

namespace pec {

constexpr int kReduceWarps = 8;
constexpr int kReduceThreads = kReduceWarps * 32;

// One CTA per query head: merges that head's partials over all slices.
//   part_o [splits][g][Hkv][128] fp32, part_lse [splits][g][Hkv]; head = kvh * g + r.
// A lane owns four channels; warp w takes slices w, w + 8, ... (their loads are independent, four in
// flight per lane), the eight warps' sums meet in shared memory.  The maximum of the LSEs is found by
// every warp for itself, one slice per lane at a time.
template <bool kOutBf16>
__global__ void __launch_bounds__(kReduceThreads)
decode_reduce_kernel(const float *__restrict__ part_o, const float *__restrict__ part_lse, void *o, float *lse,
                     int splits, int g, int hkv)
{
    __shared__ float4 sh_acc[kReduceWarps][32];
    __shared__ float sh_tot[kReduceWarps];
    const int head = blockIdx.x, kvh = head / g, r = head % g;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t item = (int64_t)r * hkv + kvh, stride = (int64_t)g * hkv;
    // Launched as a programmatic dependent of the slice kernel: the launch itself overlaps that kernel's end, and
    // nothing is read before the kernel has completed.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    float m = -INFINITY;
    for (int s = lane; s < splits; s += 32) m = fmaxf(m, part_lse[s * stride + item]);
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, d));
    float tot = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (m != -INFINITY) {
#pragma unroll 4
        for (int s = warp; s < splits; s += kReduceWarps) {
            const float l = part_lse[s * stride + item];
            const float w = (l == -INFINITY) ? 0.f : __expf(l - m);
            if (w != 0.f) {                                   // empty slice: its O is not used
                const float4 v = *reinterpret_cast<const float4 *>(part_o + (s * stride + item) * kHeadDim + 4 * lane);
                acc.x = fmaf(w, v.x, acc.x); acc.y = fmaf(w, v.y, acc.y); acc.z = fmaf(w, v.z, acc.z); acc.w = fmaf(w, v.w, acc.w);
                tot += w;
            }
        }
    }
    sh_acc[warp][lane] = acc;
    if (lane == 0) sh_tot[warp] = tot;
    __syncthreads();
    if (warp == 0) {
        tot = 0.f;
        acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int w = 0; w < kReduceWarps; ++w) {
            const float4 v = sh_acc[w][lane];
            acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
            tot += sh_tot[w];
        }
        const float inv = tot > 0.f ? 1.f / tot : 0.f;
        acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
        if (kOutBf16) {
            __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
            uint2 pk;
            pk.x = *reinterpret_cast<uint32_t *>(&lo);
            pk.y = *reinterpret_cast<uint32_t *>(&hi);
            *reinterpret_cast<uint2 *>(static_cast<__nv_bfloat16 *>(o) + (int64_t)head * kHeadDim + 4 * lane) = pk;
        } else {
            *reinterpret_cast<float4 *>(static_cast<float *>(o) + (int64_t)head * kHeadDim + 4 * lane) = acc;
        }
        if (lane == 0) lse[head] = (m == -INFINITY) ? -INFINITY : m + logf(tot);
    }
}

static inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Argument checks shared by the entry points; fills the slice plan.
static int check_decode(const pec_decode_args *a, DecodeShape &shape, const char *who)
{
    if (!a) { set_error("%s: args is NULL", who); return PEC_ERR_INVALID_ARG; }
    if (!a->q || !a->k || !a->v || !a->o || !a->lse || !a->status) {
        set_error("%s: q, k, v, o, lse and status must be non-NULL", who);
        return PEC_ERR_INVALID_ARG;
    }
    if (a->D != kHeadDim) { set_error("%s: D=%d unsupported (only 128)", who, a->D); return PEC_ERR_UNSUPPORTED; }
    if (a->Hq < 1 || a->Hkv < 1 || a->Hq % a->Hkv != 0 || a->Hq / a->Hkv > 128) {
        set_error("%s: need Hkv | Hq and at most 128 query heads per KV head (got %d, %d)", who, a->Hq, a->Hkv);
        return PEC_ERR_INVALID_ARG;
    }
    if (a->o_dtype != PEC_BF16 && a->o_dtype != PEC_F32) { set_error("%s: unknown o_dtype %d", who, a->o_dtype); return PEC_ERR_UNSUPPORTED; }
    if (a->kv_lo < 0 || a->kv_hi < a->kv_lo || a->kv_hi > ((int64_t)1 << 30)) {
        set_error("%s: need 0 <= kv_lo <= kv_hi <= 2^30", who);
        return PEC_ERR_INVALID_ARG;
    }
    if (a->num_splits < 0 || a->num_splits > 4096) { set_error("%s: num_splits out of range", who); return PEC_ERR_INVALID_ARG; }
    if (!(a->softmax_scale >= 0.f) || std::isinf(a->softmax_scale)) { set_error("%s: softmax_scale must be finite and >= 0", who); return PEC_ERR_INVALID_ARG; }
    const int64_t strides[5] = {a->q_stride_h, a->k_stride_t, a->k_stride_h, a->v_stride_t, a->v_stride_h};
    for (int i = 0; i < 5; ++i) {
        if (strides[i] < kHeadDim) { set_error("%s: strides must be >= D", who); return PEC_ERR_INVALID_ARG; }
        if ((strides[i] * 2) % 16 != 0) { set_error("%s: strides must be multiples of 16 bytes", who); return PEC_ERR_ALIGNMENT; }
    }
    if (!aligned16(a->q) || !aligned16(a->k) || !aligned16(a->v) || !aligned16(a->o) ||
        (reinterpret_cast<uintptr_t>(a->lse) & 3u) || (reinterpret_cast<uintptr_t>(a->status) & 3u)) {
        set_error("%s: q, k, v, o must be 16-byte aligned (lse, status 4-byte)", who);
        return PEC_ERR_ALIGNMENT;
    }
    // Slices: enough CTAs to fill the GPU twice over, at least 512 keys each, whole 128-key tiles.
    const int64_t keys = a->kv_hi - a->kv_lo;
    int64_t splits = a->num_splits;
    if (splits == 0) {
        int sms = 148, dev = 0;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        splits = (2 * (int64_t)sms + a->Hkv - 1) / a->Hkv;
        const int64_t by_size = (keys + 511) / 512;
        if (splits > by_size) splits = by_size;
    }
    if (splits < 1) splits = 1;
    int64_t per = (keys + splits - 1) / splits;
    per = ((per + 127) / 128) * 128;
    if (per < 128) per = 128;
    splits = keys > 0 ? (keys + per - 1) / per : 1;
    shape.splits = (int32_t)splits;
    shape.split_keys = per;
    shape.scratch_bytes = (size_t)splits * (size_t)a->Hq * (kHeadDim + 1) * sizeof(float);
    return PEC_OK;
}

// Runs the two kernels with `scratch` (device, >= shape.scratch_bytes, 16-byte aligned) as the partial store.
static int run_decode(const pec_decode_args *a, const DecodeShape &shape, void *scratch, cudaStream_t stream, const char *who)
{
    const int g = a->Hq / a->Hkv;
    float *part_o = static_cast<float *>(scratch);
    float *part_lse = part_o + (size_t)shape.splits * a->Hq * kHeadDim;

    AttnParams p{};
    p.q = a->q; p.k = a->k; p.v = a->v;
    p.o = part_o; p.lse = part_lse;
    // The g heads of a KV group become rows 0..g-1 of pseudo-head kvh: row stride = one head, head stride = g heads.
    p.q_stride_t = a->q_stride_h; p.q_stride_h = (int64_t)g * a->q_stride_h;
    p.k_stride_t = a->k_stride_t; p.k_stride_h = a->k_stride_h;
    p.v_stride_t = a->v_stride_t; p.v_stride_h = a->v_stride_h;
    p.Hq = a->Hkv; p.Hkv = a->Hkv; p.group = 1;
    p.cu_seqlens = nullptr; p.B = 1;
    p.q_lo[0] = 0; p.q_hi[0] = g; p.n_qseg = 1; p.out_pos0 = 0; p.total_rows = g;
    p.wait_cycles = wait_limit_cycles();
    p.iv_lo[0] = a->kv_lo; p.iv_hi[0] = a->kv_hi; p.iv_lo[1] = p.iv_hi[1] = 0;
    p.n_iv = a->kv_hi > a->kv_lo ? 1 : 0;
    p.causal = 0;
    p.scale = a->softmax_scale > 0.f ? a->softmax_scale : (float)(1.0 / std::sqrt((double)kHeadDim));
    p.scale_log2 = (float)((double)p.scale * 1.4426950408889634074);
    p.o_is_bf16 = 0;
    p.status = a->status;
    p.splits = shape.splits;
    p.split_keys = shape.split_keys;
    const int rc = launch_attn_split_bf16(p, stream);
    if (rc != PEC_OK) return rc;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)a->Hq);
    cfg.blockDim = dim3(kReduceThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const float *po = part_o, *pl = part_lse;
    if (a->o_dtype == PEC_BF16) cudaLaunchKernelEx(&cfg, decode_reduce_kernel<true>, po, pl, a->o, a->lse, (int)shape.splits, g, (int)a->Hkv);
    else                        cudaLaunchKernelEx(&cfg, decode_reduce_kernel<false>, po, pl, a->o, a->lse, (int)shape.splits, g, (int)a->Hkv);
    const cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) { set_error("%s: launch failed: %s", who, cudaGetErrorString(err)); return PEC_ERR_CUDA; }
    return PEC_OK;
}

// ---------------------------------------------------------------------------------------------
// Built-in scratch for pec_decode_attn_static.  The array lives in every GPU that loads the
// library, from load to exit.  Its name is only a handle on the host side: the device address
// is looked up once per device with cudaGetSymbolAddress and cached here.
static __device__ __align__(256) unsigned char g_decode_scratch[PEC_DECODE_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
static std::mutex g_scratch_mutex;
static void *g_scratch_ptr[kMaxDevices] = {};

// Device address of the built-in scratch on the current device (nullptr + error text on failure).
static void *static_scratch_for_current_device(const char *who)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        set_error("%s: cannot identify the current device", who);
        return nullptr;
    }
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ptr[dev]) {
        void *ptr = nullptr;
        const cudaError_t err = cudaGetSymbolAddress(&ptr, g_decode_scratch);
        if (err != cudaSuccess || !ptr) {
            set_error("%s: cudaGetSymbolAddress failed on device %d: %s", who, dev, cudaGetErrorString(err));
            return nullptr;
        }
        g_scratch_ptr[dev] = ptr;
    }
    return g_scratch_ptr[dev];
}

}  // namespace pec

using namespace pec;

extern "C" int pec_decode_attn_static(const pec_decode_args *args, void *cuda_stream)
{
    DecodeShape shape;
    const int rc = check_decode(args, shape, "pec_decode_attn_static");
    if (rc != PEC_OK) return rc;
    if (shape.scratch_bytes > (size_t)PEC_DECODE_STATIC_SCRATCH_BYTES) {
        set_error("pec_decode_attn_static: this call needs %zu bytes of scratch (slices x Hq x 516) but the built-in "
                  "scratch holds %d; pass a smaller num_splits or use pec_decode_attn with a workspace",
                  shape.scratch_bytes, PEC_DECODE_STATIC_SCRATCH_BYTES);
        return PEC_ERR_WORKSPACE;
    }
    void *scratch = static_scratch_for_current_device("pec_decode_attn_static");
    if (!scratch) return PEC_ERR_CUDA;
    return run_decode(args, shape, scratch, static_cast<cudaStream_t>(cuda_stream), "pec_decode_attn_static");
}

extern "C" size_t pec_decode_workspace_size(const pec_decode_args *args)
{
    DecodeShape shape;
    if (check_decode(args, shape, "pec_decode_workspace_size") != PEC_OK) return 0;
    return shape.scratch_bytes;
}

extern "C" int pec_decode_attn(const pec_decode_args *args, void *cuda_stream)
{
    DecodeShape shape;
    const int rc = check_decode(args, shape, "pec_decode_attn");
    if (rc != PEC_OK) return rc;
    if (!args->workspace || args->workspace_bytes < shape.scratch_bytes || !aligned16(args->workspace)) {
        set_error("pec_decode_attn: workspace missing, misaligned or too small (%zu < %zu)", args->workspace_bytes, shape.scratch_bytes);
        return PEC_ERR_WORKSPACE;
    }
    return run_decode(args, shape, args->workspace, static_cast<cudaStream_t>(cuda_stream), "pec_decode_attn");
}
