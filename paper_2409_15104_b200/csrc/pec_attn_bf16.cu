// bf16 partial causal attention on the sm_100a tensor cores (Eq. 3-4 as KV-tile partial attention
// with online-softmax state: running max, running sum, fp32 accumulator).
//
// One CTA = one (128-row query tile, head).  Q, K and V tiles arrive by TMA into 128-byte-swizzled
// shared memory; S = Q K^T and O += P V run as tcgen05.mma with fp32 accumulators in tensor
// memory (TMEM); the four warps own the 128 TMEM lanes (one query row per thread) for the softmax.
// P is written back to TMEM as packed bf16 and consumed as the A operand of the second MMA.
//
// TMEM columns: [0,128) S (fp32), reused as P (bf16 pairs, columns [0,64)); [128,256) O (fp32).
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "pec_internal.h"
#include "pec_sm100.cuh"
#include "pec_tile.cuh"

namespace pec {
using namespace sm100;

constexpr int kTileM = 128, kTileN = 128;
constexpr int kThreads = 128;
constexpr uint32_t kHalfTileBytes = 128 * 64 * 2;          // one TMA box: 128 rows x 64 bf16
constexpr uint32_t kTileBytes = 2 * kHalfTileBytes;        // 128 x 128 bf16
constexpr uint32_t kTmemCols = 256;
constexpr uint32_t kColS = 0, kColP = 0, kColO = 128;
constexpr size_t kSmemBytes = 3 * kTileBytes + 1024 /*alignment slack*/ + 64 /*barriers*/;
constexpr long long kWaitCycles = 2000000000LL;            // bounded waits give up after ~1 s

struct Shared {
    uint64_t bar_q, bar_kv, bar_mma;
    uint32_t tmem_base;
    volatile int abort_flag;
};

// Bounded mbarrier wait.  Returns false (and raises the abort flag / status word) on expiry.
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, Shared *sh, int32_t *status)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (!mbar_try_wait(bar, parity)) {
        if (sh->abort_flag) return false;
        if (clock64() - t0 > kWaitCycles) {
            sh->abort_flag = 1;
            if (status) atomicExch(status, (int)PEC_ERR_TIMEOUT);
            return false;
        }
    }
    return true;
}

__global__ void __launch_bounds__(kThreads, 1)
attn_bf16_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_v, const AttnParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;           // swizzled tiles need 1024-byte alignment
    const uint32_t sQ = tiles, sK = tiles + kTileBytes, sV = tiles + 2 * kTileBytes;
    Shared *sh = reinterpret_cast<Shared *>(smem_raw + (tiles - raw) + 3 * kTileBytes);
    const uint32_t bar_q = smem_u32(&sh->bar_q), bar_kv = smem_u32(&sh->bar_kv), bar_mma = smem_u32(&sh->bar_mma);

    // Heaviest (latest) causal tiles first.
    const int64_t tile = (int64_t)gridDim.x - 1 - blockIdx.x;
    TileJob job;
    if (!locate_tile(p, tile, kTileM, job)) return;

    const int tid = threadIdx.x, warp = tid >> 5;
    const int h = blockIdx.y, kvh = h / p.group;

    // An earlier CTA's wait expired: the launch is already lost, leave at once (uniform decision).
    if (tid == 0) sh->abort_flag = (p.status && *reinterpret_cast<volatile int32_t *>(p.status) != 0) ? 1 : 0;
    __syncthreads();
    if (sh->abort_flag) return;

    if (tid == 0) {
        mbar_init(bar_q, 1);
        mbar_init(bar_kv, 1);
        mbar_init(bar_mma, 1);
        mbar_init_fence();
        prefetch_tmap(&tm_q); prefetch_tmap(&tm_k); prefetch_tmap(&tm_v);
    }
    if (warp == 0) {
        __syncwarp();
        tmem_alloc(smem_u32(&sh->tmem_base), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh->tmem_base;
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;  // this warp's TMEM lanes

    if (tid == 0) {
        mbar_arrive_expect_tx(bar_q, kTileBytes);
        tma_load_3d(sQ, &tm_q, bar_q, 0, h, (int)job.q_row0);
        tma_load_3d(sQ + kHalfTileBytes, &tm_q, bar_q, 64, h, (int)job.q_row0);
    }

    constexpr uint32_t idesc_qk = idesc_bf16_f32(kTileM, kTileN, 0, 0);
    constexpr uint32_t idesc_pv = idesc_bf16_f32(kTileM, kHeadDim, 0, 1);

    float m_run = -INFINITY, l_run = 0.f;
    const int64_t my_pos = job.q_pos0 + tid;
    const int64_t last_pos = job.q_pos0 + job.n_rows - 1;
    uint32_t kv_phase = 0, mma_phase = 0;
    bool first = true, ok = true;

    for (int t = 0; t < job.n_iv && ok; ++t) {
        const int64_t lo = job.iv_lo[t];
        const int64_t hi = job.iv_hi[t];
        int64_t end = hi;                                     // keys at or after `end` are invisible to the whole tile
        if (p.causal && end > last_pos + 1) end = last_pos + 1;
        for (int64_t k0 = lo; k0 < end && ok; k0 += kTileN) {
            if (tid == 0) {
                const int krow = (int)(job.kv_row0 + k0);
                mbar_arrive_expect_tx(bar_kv, 2 * kTileBytes);
                tma_load_3d(sK, &tm_k, bar_kv, 0, kvh, krow);
                tma_load_3d(sK + kHalfTileBytes, &tm_k, bar_kv, 64, kvh, krow);
                tma_load_3d(sV, &tm_v, bar_kv, 0, kvh, krow);
                tma_load_3d(sV + kHalfTileBytes, &tm_v, bar_kv, 64, kvh, krow);
                if (first) ok = wait_bar(bar_q, 0, sh, p.status);
                ok = ok && wait_bar(bar_kv, kv_phase, sh, p.status);
                if (ok) {
                    // S = Q K^T: both operands K-major; 8 steps of 16 channels, 4 per 64-channel half tile
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks) {
                        const uint32_t off = (uint32_t)(ks >> 2) * kHalfTileBytes + (uint32_t)(ks & 3) * 32u;
                        mma_ss(tmem + kColS, smem_desc_sw128(sQ + off, 16, 1024), smem_desc_sw128(sK + off, 16, 1024),
                               idesc_qk, ks > 0 ? 1u : 0u);
                    }
                    tc_commit(bar_mma);
                }
            }
            kv_phase ^= 1;
            ok = __all_sync(0xffffffffu, wait_bar(bar_mma, mma_phase, sh, p.status));   // warp-uniform
            mma_phase ^= 1;
            if (!ok) break;
            tc_fence_after();

            // visible columns of this row inside the tile
            int64_t lim = hi;
            if (p.causal && my_pos + 1 < lim) lim = my_pos + 1;
            int n_vis = (int)(lim - k0);
            n_vis = n_vis < 0 ? 0 : (n_vis > kTileN ? kTileN : n_vis);

            float s[kTileN];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t r[32];
                tmem_ld32(tmem + lane_base + kColS + c * 32, r);
#pragma unroll
                for (int j = 0; j < 32; ++j) s[c * 32 + j] = __uint_as_float(r[j]);
            }
            float mx = -INFINITY;
#pragma unroll
            for (int j = 0; j < kTileN; ++j) {
                s[j] = (j < n_vis) ? s[j] * p.scale_log2 : -INFINITY;
                mx = fmaxf(mx, s[j]);
            }
            const float m_new = fmaxf(m_run, mx);
            const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
            const float alpha = ex2(m_run - m_use);           // 0 while the row has seen no key
            float rs = 0.f;
#pragma unroll
            for (int j = 0; j < kTileN; ++j) { s[j] = ex2(s[j] - m_use); rs += s[j]; }
            l_run = l_run * alpha + rs;
            m_run = m_new;

            if (!first) {                                     // rescale the accumulator rows
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t r[32];
                    tmem_ld32(tmem + lane_base + kColO + c * 32, r);
#pragma unroll
                    for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * alpha);
                    tmem_st32(tmem + lane_base + kColO + c * 32, r);
                }
            }
            // P as packed bf16: column c of the A operand holds keys 2c (low half) and 2c+1 (high half)
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t r[32];
#pragma unroll
                for (int j = 0; j < 32; ++j) r[j] = pack_bf16(s[c * 64 + 2 * j], s[c * 64 + 2 * j + 1]);
                tmem_st32(tmem + lane_base + kColP + c * 32, r);
            }
            tmem_st_wait();
            tc_fence_before();
            __syncthreads();

            if (tid == 0) {
                tc_fence_after();
                // O (+)= P V: A = P from TMEM (8 columns per 16 keys), B = V tile stored [key][channel]
                // (N-contiguous): 16 keys = 2048 bytes per step, channel halves 16 KiB apart.
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    mma_ts(tmem + kColO, tmem + kColP + ks * 8, smem_desc_sw128(sV + ks * 2048u, kHalfTileBytes, 1024),
                           idesc_pv, (!first || ks > 0) ? 1u : 0u);
                }
                tc_commit(bar_mma);
            }
            ok = __all_sync(0xffffffffu, wait_bar(bar_mma, mma_phase, sh, p.status));
            mma_phase ^= 1;
            tc_fence_after();
            first = false;
        }
    }

    // A tile without any key tile never consumed its Q copy: let it land before the CTA retires.
    if (first && tid == 0) wait_bar(bar_q, 0, sh, p.status);
    __syncwarp();

    // Epilogue: O / l and LSE = ln2 * m + ln l; rows without any visible key give 0 and -inf.
    // (TMEM loads are warp-wide; only the global stores are predicated on the row being valid.)
    if (ok) {
        const bool valid = tid < job.n_rows;
        const bool empty = (l_run == 0.f);
        const float inv = empty ? 0.f : 1.f / l_run;
        const int64_t row = job.out_row0 + tid;
        const int64_t obase = (row * p.Hq + h) * kHeadDim;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            uint32_t r[32];
            if (first) {
#pragma unroll
                for (int j = 0; j < 32; ++j) r[j] = 0u;
            } else {
                tmem_ld32(tmem + lane_base + kColO + c * 32, r);
            }
            if (!valid) continue;
            if (p.o_is_bf16) {
                __nv_bfloat16 *o = static_cast<__nv_bfloat16 *>(p.o) + obase + c * 32;
#pragma unroll
                for (int j = 0; j < 32; j += 8) {
                    uint4 pk;
                    pk.x = pack_bf16(__uint_as_float(r[j + 0]) * inv, __uint_as_float(r[j + 1]) * inv);
                    pk.y = pack_bf16(__uint_as_float(r[j + 2]) * inv, __uint_as_float(r[j + 3]) * inv);
                    pk.z = pack_bf16(__uint_as_float(r[j + 4]) * inv, __uint_as_float(r[j + 5]) * inv);
                    pk.w = pack_bf16(__uint_as_float(r[j + 6]) * inv, __uint_as_float(r[j + 7]) * inv);
                    *reinterpret_cast<uint4 *>(o + j) = pk;
                }
            } else {
                float *o = static_cast<float *>(p.o) + obase + c * 32;
#pragma unroll
                for (int j = 0; j < 32; j += 4)
                    *reinterpret_cast<float4 *>(o + j) = make_float4(__uint_as_float(r[j]) * inv, __uint_as_float(r[j + 1]) * inv,
                                                                     __uint_as_float(r[j + 2]) * inv, __uint_as_float(r[j + 3]) * inv);
            }
        }
        if (valid) p.lse[row * p.Hq + h] = empty ? -INFINITY : m_run * 0.6931471805599453f + logf(l_run);
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

// ------------------------------------------------------------------------------------------ host
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *sym = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(sym);
    }
    return fn;
}

// [rows, heads, 128] bf16 tensor with element strides (stride_t, stride_h); box = 64 channels x 1 head x 128 rows.
static bool make_map(CUtensorMap *map, const void *base, int64_t rows, int32_t heads, int64_t stride_t, int64_t stride_h)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[3] = {(cuuint64_t)kHeadDim, (cuuint64_t)heads, (cuuint64_t)(rows > 0 ? rows : 1)};
    cuuint64_t strides[2] = {(cuuint64_t)stride_h * 2, (cuuint64_t)stride_t * 2};
    cuuint32_t box[3] = {64, 1, 128};
    cuuint32_t estr[3] = {1, 1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int launch_attn_bf16(const AttnParams &p, cudaStream_t stream)
{
    if (!p.status) { set_error("pec_prefill_attn: the bf16 path needs a status word"); return PEC_ERR_INVALID_ARG; }
    // Rows the maps may touch: queries up to the chunk end, keys up to the end of the visible subset.
    int64_t q_rows, kv_rows;
    if (p.cu_seqlens) { q_rows = p.total_rows; kv_rows = p.total_rows; }
    else {
        q_rows = p.chunk_start + p.chunk_len;
        kv_rows = 0;
        for (int t = 0; t < p.n_iv; ++t) kv_rows = p.iv_hi[t] > kv_rows ? p.iv_hi[t] : kv_rows;
    }
    CUtensorMap tm_q, tm_k, tm_v;
    if (!make_map(&tm_q, p.q, q_rows, p.Hq, p.q_stride_t, p.q_stride_h) ||
        !make_map(&tm_k, p.k, kv_rows, p.Hkv, p.k_stride_t, p.k_stride_h) ||
        !make_map(&tm_v, p.v, kv_rows, p.Hkv, p.v_stride_t, p.v_stride_h)) {
        set_error("pec_prefill_attn: cuTensorMapEncodeTiled failed (driver too old, or strides/addresses not encodable)");
        return PEC_ERR_CUDA;
    }
    if (cudaFuncSetAttribute(attn_bf16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes) != cudaSuccess) {
        set_error("pec_prefill_attn: cannot raise the shared-memory limit: %s", cudaGetErrorString(cudaGetLastError()));
        return PEC_ERR_CUDA;
    }
    int64_t tiles = (p.total_rows + kTileM - 1) / kTileM;
    if (p.cu_seqlens) tiles += p.B;
    if (tiles > 0x7fffffff || p.Hq > 65535) { set_error("pec_prefill_attn: grid too large"); return PEC_ERR_UNSUPPORTED; }
    dim3 grid((unsigned)tiles, (unsigned)p.Hq);
    attn_bf16_kernel<<<grid, kThreads, kSmemBytes, stream>>>(tm_q, tm_k, tm_v, p);
    const cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) { set_error("pec_prefill_attn: launch failed: %s", cudaGetErrorString(err)); return PEC_ERR_CUDA; }
    return PEC_OK;
}

}  // namespace pec
