// y = merge(o_1 .. o_n) w^T: the post-self-attention linear layer (Eq. 5) taking the partial
// attention results of one request - the outputs O_1, O_2 of the GPUs that share a long request in
// Section 5.2's colocation example, or the partials of n key partitions (Section 2.2) - as they
// are, fp32 [T, Hq, 128] with their per-(row, head) LSEs.  The LSE-weighted combination is the
// GEMM's A-operand producer, so the merged O never goes to memory.
//
// A cluster of two CTAs computes one 256 x 512 tile of y with 256-row MMAs (cta_group::2), two per
// 16-channel slice (N = 256 each); each CTA keeps its 128 rows x 512 columns of the fp32
// accumulator in its own tensor memory (all 512 columns: one CTA per SM).  Per K step of 64
// channels (half a head) a CTA
//   * loads by TMA its half of the two 256-row groups of w (2 x 16 KB), and
//   * builds its own 128 x 64 A tile in shared memory: sixteen producer warps in two groups that
//     take alternate K steps read the n partials' rows from global memory (4 channels = one
//     16-byte load per partial and thread, eight rows per thread), weight them by
//     exp(lse_i - lse), round to bf16 and store the 8 bytes where the 128-byte swizzle of a
//     K-major tile puts them; a proxy fence, then one arrive per warp on the pair leader's barrier.
// The leader's barrier of a slot therefore counts the loader's expect-tx arrive plus 2 x 8 producer
// warps; its wait acquires at cluster scope because half of the producers are in the other CTA.
// A tile is reused across the 512 columns only, so every column tile re-reads the partials through
// the L2: n x 32 bytes per clock and SM at the full MMA rate, against 32 for w.  That is what binds
// the kernel: an SM takes in about 40-48 bytes per clock here, so for n = 2 (96 wanted) the MMAs run
// at about 40 % of their rate, and a merge pass followed by pec_linear is faster.  The call exists
// for callers that cannot spare the merged copy's memory or its pass.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "pec_host.h"
#include "pec_internal.h"
#include "pec_sm100.cuh"
#include "pec_tma_store.cuh"

namespace pec {
using namespace sm100;

namespace lmg {
constexpr int kBM = 128, kBN = 512, kBK = 64;
constexpr int kSlots = 4;
constexpr int kProducerWarps = 16, kGroupWarps = 8;         // two groups on alternate K steps
constexpr int kMmaWarp = kProducerWarps, kLoadWarp = kProducerWarps + 1;
constexpr int kThreads = (kProducerWarps + 2) * 32;         // 576
constexpr uint32_t kABytes = kBM * kBK * 2;                 // this CTA's 128 rows of merged O
constexpr uint32_t kWGroupBytes = 128 * kBK * 2;            // this CTA's half of one 256-row group of w
constexpr uint32_t kSlotBytes = kABytes + 2 * kWGroupBytes; // 48 KB
constexpr uint32_t kTmemCols = 512;
constexpr int kMaxParts = PEC_LINEAR_MERGED_MAX_PARTS;

struct Shared {
    uint64_t full[kSlots], empty[kSlots], acc_full;
    uint32_t tmem_base;
    volatile int abort_flag;
};
constexpr size_t kSmemBytes = kSlots * kSlotBytes + 1024 + sizeof(Shared);

struct Params {
    const float *o[kMaxParts];
    const float *lse[kMaxParts];
    int64_t M;
    int32_t N, Hq, band, by_cols, test_skip_last_load;
    int32_t *status;
    long long wait_cycles;
};

// Cluster-scope forms for a barrier that threads of the partner CTA arrive on after writing their own
// shared memory with ordinary stores: the arrive releases, the wait acquires, both at cluster scope.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_suspend_cluster(uint32_t bar, uint32_t parity, uint32_t ns)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(ns) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_bounded_cluster(uint32_t bar, uint32_t parity, volatile int *abort_flag, int32_t *status,
                                                          long long limit_cycles, int timeout_code)
{
    const long long t0 = clock64();
    while (!mbar_try_wait_suspend_cluster(bar, parity, 2000u)) {
        if (*abort_flag) return false;
        if (clock64() - t0 > limit_cycles) {
            *abort_flag = 1;
            if (status) atomicExch(status, timeout_code);
            return false;
        }
    }
    return true;
}
// Orders this thread's ordinary shared-memory stores before later reads of the same memory by the async
// proxy (TMA, tcgen05.mma operands).
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

struct WaitCtx { volatile int *abort_flag; int32_t *status; long long limit; };
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, const WaitCtx &w)
{
    return mbar_wait_bounded(bar, parity, w.abort_flag, w.status, w.limit, (int)PEC_ERR_TIMEOUT);
}
__device__ __forceinline__ bool wait_bar_cluster(uint32_t bar, uint32_t parity, const WaitCtx &w)
{
    return mbar_wait_bounded_cluster(bar, parity, w.abort_flag, w.status, w.limit, (int)PEC_ERR_TIMEOUT);
}

template <int kParts>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
linear_merged_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_y, const __grid_constant__ Params p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring = (raw + 1023u) & ~1023u;
    uint8_t *ring_ptr = smem_raw + (ring - raw);
    Shared *sh = reinterpret_cast<Shared *>(ring_ptr + kSlots * kSlotBytes);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();                  // 0 = leader
    // Tile order in bands, as in linear_kernel: by_cols == 0: bands of `band` row pairs (the partials' rows of a
    // band stay in L2 while every column tile is visited); by_cols == 1: bands of `band` column tiles (their rows of w stay).
    const int pairs = (int)(gridDim.x >> 1), gn = (int)gridDim.y;
    const int64_t seq = (int64_t)blockIdx.y * pairs + (blockIdx.x >> 1);
    int pair_i, col_i;
    if (!p.by_cols) {
        const int band_i = (int)(seq / ((int64_t)p.band * gn));
        const int band_pairs = (pairs - band_i * p.band) < p.band ? (pairs - band_i * p.band) : p.band;
        const int within = (int)(seq - (int64_t)band_i * p.band * gn);
        pair_i = band_i * p.band + within % band_pairs;
        col_i = within / band_pairs;
    } else {
        const int band_i = (int)(seq / ((int64_t)p.band * pairs));
        const int band_cols = (gn - band_i * p.band) < p.band ? (gn - band_i * p.band) : p.band;
        const int within = (int)(seq - (int64_t)band_i * p.band * pairs);
        col_i = band_i * p.band + within % band_cols;
        pair_i = within / band_cols;
    }
    const int64_t m0 = (int64_t)pair_i * (2 * kBM) + rank * kBM;
    const int n0 = col_i * kBN;
    const int n_kb = 2 * p.Hq;                                // 64 channels per step, 128 per head
    const WaitCtx wctx = {&sh->abort_flag, p.status, p.wait_cycles};

    if (tid == 0) {
        sh->abort_flag = (p.status && *reinterpret_cast<volatile int32_t *>(p.status) != 0) ? 1 : 0;
        for (int s = 0; s < kSlots; ++s) {
            mbar_init(smem_u32(&sh->full[s]), 1 + 2 * kGroupWarps);   // loader + both CTAs' producer warps of the step
            mbar_init(smem_u32(&sh->empty[s]), 1);
        }
        mbar_init(smem_u32(&sh->acc_full), 1);
        mbar_init_fence();
        prefetch_tmap(&tm_w); prefetch_tmap(&tm_y);
    }
    __syncthreads();
    cluster_sync();                                           // both CTAs' barriers exist before anyone signals them
    if (warp == 0) {
        tmem_alloc_pair(smem_u32(&sh->tmem_base), kTmemCols);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh->tmem_base;

    if (warp == kLoadWarp) {
        if (lane == 0) {
            for (int kb = 0; kb < n_kb; ++kb) {
                const int slot = kb % kSlots, fill = kb / kSlots;
                if (p.test_skip_last_load && rank == 1 && kb == n_kb - 1) break;   // test hook: the pair's waits for this step run out
                if (fill > 0 && !wait_bar(smem_u32(&sh->empty[slot]), (fill - 1) & 1, wctx)) break;
                const uint32_t b = ring + slot * kSlotBytes + kABytes;
                const uint32_t bar = leader_addr(smem_u32(&sh->full[slot]));
                if (rank == 0) mbar_arrive_expect_tx(smem_u32(&sh->full[slot]), 4 * kWGroupBytes);   // both CTAs' bytes
                tma_load_2d_pair(b, &tm_w, bar, kb * kBK, n0 + (int)rank * 128);
                tma_load_2d_pair(b + kWGroupBytes, &tm_w, bar, kb * kBK, n0 + 256 + (int)rank * 128);
            }
        }
        __syncwarp();
    } else if (warp == kMmaWarp) {
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = idesc_bf16_f32(2 * kBM, 256, 0, 0);
            bool ok = true;
            for (int kb = 0; kb < n_kb && ok; ++kb) {
                const int slot = kb % kSlots;
                ok = wait_bar_cluster(smem_u32(&sh->full[slot]), (kb / kSlots) & 1, wctx);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a = ring + slot * kSlotBytes, b = a + kABytes;
#pragma unroll
                for (int ks = 0; ks < kBK / 16; ++ks) {
                    const uint64_t da = smem_desc_sw128(a + ks * 32u, 16, 1024);
                    const uint32_t acc = (kb > 0 || ks > 0) ? 1u : 0u;
                    mma_ss_pair(tmem, da, smem_desc_sw128(b + ks * 32u, 16, 1024), idesc, acc);
                    mma_ss_pair(tmem + 256, da, smem_desc_sw128(b + kWGroupBytes + ks * 32u, 16, 1024), idesc, acc);
                }
                tc_commit_pair(smem_u32(&sh->empty[slot]));
            }
            if (ok) tc_commit_pair(smem_u32(&sh->acc_full));
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ A-tile producers, then epilogue
        const int group = warp / kGroupWarps;                 // takes K steps kb = 2 * head + group
        const int gt = tid & (kGroupWarps * 32 - 1);
        // A thread takes 4 channels (one 16-byte load per part) of rows rsub + 16 i, i = 0..7: a warp's load covers two
        // rows' 256 contiguous bytes.  The weights of a warp's 16 rows are worked out one row per lane (lanes 16-31
        // repeat lanes 0-15) and fetched by shuffle where they are used.
        const int c4 = gt & 15, rsub = gt >> 4;
        const int w_row = 2 * (gt >> 5) + (lane & 1) + 16 * ((lane & 15) >> 1);   // the row whose weights this lane works out
        const int w_src = lane >> 4;                                              // + 2 i: the lane that owns row rsub + 16 i
        const int64_t row_elems = (int64_t)p.Hq * 128;
        const int64_t wr = m0 + w_row, last_row = p.M - 1;
        bool ok = true;
        // The LSEs of the next head are asked for one step ahead, so that a step's loads of O do not wait for them.
        float l_next[kParts];
        auto load_lse = [&](int head) {
#pragma unroll
            for (int q = 0; q < kParts; ++q)
                l_next[q] = (wr < p.M && head < p.Hq) ? __ldg(p.lse[q] + wr * p.Hq + head) : -INFINITY;
        };
        load_lse(0);
        // Rows per batch of loads in flight: what the registers hold.
        constexpr int kRowBatch = kParts <= 2 ? 8 : (kParts <= 4 ? 4 : 2);
        for (int head = 0; head < p.Hq && ok; ++head) {
            const int kb = 2 * head + group, slot = kb % kSlots, fill = kb / kSlots;
            // Weights of this head: exp(lse_i - lse), all zero where no part saw a key (and for rows past the end).
            float wgt[kParts];
            {
                float mx = -INFINITY, tot = 0.f;
#pragma unroll
                for (int q = 0; q < kParts; ++q) mx = fmaxf(mx, l_next[q]);
#pragma unroll
                for (int q = 0; q < kParts; ++q) {
                    wgt[q] = (l_next[q] == -INFINITY) ? 0.f : __expf(l_next[q] - mx);
                    tot += wgt[q];
                }
                const float inv = (tot > 0.f) ? 1.f / tot : 0.f;
#pragma unroll
                for (int q = 0; q < kParts; ++q) wgt[q] *= inv;
            }
            load_lse(head + 1);
            // The merged chunks are formed in registers before the slot is waited for, so the loads of a step run
            // under the previous steps' MMAs.  What a part holds where its weight is zero is never used.
            uint2 packed[8];
            const int64_t col = head * 128 + group * 64 + c4 * 4;
#pragma unroll
            for (int i0 = 0; i0 < 8; i0 += kRowBatch) {
                float4 v[kRowBatch][kParts];
#pragma unroll
                for (int i = 0; i < kRowBatch; ++i) {
                    int64_t r = m0 + rsub + 16 * (i0 + i);
                    r = r < last_row ? r : last_row;           // rows past the end: a valid address, weight zero
                    const int64_t off = r * row_elems + col;
#pragma unroll
                    for (int q = 0; q < kParts; ++q) v[i][q] = __ldg(reinterpret_cast<const float4 *>(p.o[q] + off));
                }
#pragma unroll
                for (int i = 0; i < kRowBatch; ++i) {
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int q = 0; q < kParts; ++q) {
                        const float wq = __shfl_sync(0xffffffffu, wgt[q], 2 * (i0 + i) + w_src);
                        if (wq != 0.f) {
                            acc.x = fmaf(wq, v[i][q].x, acc.x); acc.y = fmaf(wq, v[i][q].y, acc.y);
                            acc.z = fmaf(wq, v[i][q].z, acc.z); acc.w = fmaf(wq, v[i][q].w, acc.w);
                        }
                    }
                    packed[i0 + i] = make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
                }
            }
            if (fill > 0) ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->empty[slot]), (fill - 1) & 1, wctx));
            if (!ok) break;
            uint8_t *a_tile = ring_ptr + slot * kSlotBytes;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int rr = rsub + 16 * i;
                *reinterpret_cast<uint2 *>(a_tile + rr * 128 + (((c4 >> 1) ^ (rr & 7)) << 4) + (c4 & 1) * 8) = packed[i];
            }
            fence_proxy_async_smem();                         // generic-proxy stores -> visible to the MMA's reads
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(leader_addr(smem_u32(&sh->full[slot])));
        }
        // Epilogue: warp w reads lane quarter w % 4 of column group w / 4 (128 columns), rounds to bf16, lays its 32 rows
        // out in the operand ring (free once every MMA has completed) as two boxes of 64 columns and hands them to the TMA.
        ok = __all_sync(0xffffffffu, ok && wait_bar(smem_u32(&sh->acc_full), 0, wctx));
        if (ok) {
            tc_fence_after();
            const int quarter = warp & 3, cgroup = warp >> 2;
            const int row0 = (int)m0 + quarter * 32;
            const uint32_t taddr = tmem + ((uint32_t)(quarter * 32) << 16) + cgroup * 128;
            const uint32_t boxes = ring + (uint32_t)warp * (2 * kStoreBoxBytes);
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
                uint32_t r[32];
                tmem_ld32(taddr + c * 32, r);
                const uint32_t box = boxes + (c >> 1) * kStoreBoxBytes;
#pragma unroll
                for (int i = 0; i < 32; i += 8)
                    box_put(box, lane, (c & 1) * 4 + (i >> 3),
                            pack_bf16(__uint_as_float(r[i + 0]), __uint_as_float(r[i + 1])), pack_bf16(__uint_as_float(r[i + 2]), __uint_as_float(r[i + 3])),
                            pack_bf16(__uint_as_float(r[i + 4]), __uint_as_float(r[i + 5])), pack_bf16(__uint_as_float(r[i + 6]), __uint_as_float(r[i + 7])));
                if (c & 1) {
                    const int col0 = n0 + cgroup * 128 + (c >> 1) * 64;
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0 && row0 < p.M && col0 < p.N) box_store(&tm_y, box, col0, row0);
                }
            }
            if (lane == 0) { bulk_commit(); bulk_wait_read(); }     // the boxes must outlive the TMA's reads of them
            __syncwarp();
        }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();                                           // the partner is done with this CTA's memory too
    if (warp == 0) tmem_dealloc_pair(tmem, kTmemCols);
}

template <int kParts>
static bool prepare()
{
    static unsigned char ready[host::kMaxDevices] = {};
    static std::mutex ready_mutex;
    return host::once_per_device(ready, ready_mutex, [] {
        return cudaFuncSetAttribute(linear_merged_kernel<kParts>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes) == cudaSuccess; });
}

template <int kParts>
static cudaError_t launch(dim3 grid, cudaStream_t stream, const CUtensorMap &tm_w, const CUtensorMap &tm_y, const Params &p)
{
    if (!prepare<kParts>()) return cudaErrorUnknown;
    linear_merged_kernel<kParts><<<grid, kThreads, kSmemBytes, stream>>>(tm_w, tm_y, p);
    return cudaGetLastError();
}

}  // namespace lmg
}  // namespace pec

using namespace pec;

extern "C" int pec_linear_merged(const void *const *o_parts, const float *const *lse_parts, int32_t n, int64_t rows, int32_t Hq,
                                 int32_t D, const void *w, int64_t w_stride, void *y, int64_t y_stride, int32_t N,
                                 int32_t *status, void *cuda_stream)
{
    if (!o_parts || !lse_parts || !w || !y || !status) { set_error("pec_linear_merged: NULL argument"); return PEC_ERR_INVALID_ARG; }
    if (n < 1 || n > lmg::kMaxParts) { set_error("pec_linear_merged: need 1 <= n <= %d parts", lmg::kMaxParts); return PEC_ERR_INVALID_ARG; }
    if (D != 128) { set_error("pec_linear_merged: D must be 128"); return PEC_ERR_UNSUPPORTED; }
    if (rows < 0 || Hq < 1 || N < 1 || rows >= ((int64_t)1 << 31)) { set_error("pec_linear_merged: need 0 <= rows < 2^31, Hq >= 1, N >= 1"); return PEC_ERR_INVALID_ARG; }
    if (N % 8 != 0) { set_error("pec_linear_merged: N must be a multiple of 8"); return PEC_ERR_UNSUPPORTED; }
    const int64_t K = (int64_t)Hq * 128;
    if (w_stride < K || y_stride < N) { set_error("pec_linear_merged: a row stride is smaller than the row"); return PEC_ERR_INVALID_ARG; }
    bool aligned = !(w_stride % 8) && !(y_stride % 8) && !(reinterpret_cast<uintptr_t>(w) & 15u) && !(reinterpret_cast<uintptr_t>(y) & 15u) &&
                   !(reinterpret_cast<uintptr_t>(status) & 3u);
    for (int i = 0; i < n; ++i) {
        if (!o_parts[i] || !lse_parts[i]) { set_error("pec_linear_merged: part %d is NULL", i); return PEC_ERR_INVALID_ARG; }
        aligned = aligned && !(reinterpret_cast<uintptr_t>(o_parts[i]) & 15u) && !(reinterpret_cast<uintptr_t>(lse_parts[i]) & 3u);
    }
    if (!aligned) { set_error("pec_linear_merged: w, y and the parts must be 16-byte aligned, w and y with row strides that are multiples of 8"); return PEC_ERR_ALIGNMENT; }
    if (rows == 0) return PEC_OK;
    CUtensorMap tm_w, tm_y;
    if (!host::make_matrix_map(&tm_w, w, N, K, w_stride, 128) || !host::make_matrix_map(&tm_y, y, rows, N, y_stride, (int)sm100::kStoreBoxRows)) {
        set_error("pec_linear_merged: cuTensorMapEncodeTiled failed");
        return PEC_ERR_CUDA;
    }
    lmg::Params p = {};
    for (int i = 0; i < n; ++i) { p.o[i] = static_cast<const float *>(o_parts[i]); p.lse[i] = lse_parts[i]; }
    p.M = rows; p.N = N; p.Hq = Hq;
    p.status = status; p.wait_cycles = (long long)wait_limit_cycles(); p.test_skip_last_load = test_skip_last_load();
    const int64_t pairs = (rows + 2 * lmg::kBM - 1) / (2 * lmg::kBM), gn = (N + lmg::kBN - 1) / lmg::kBN;
    if (gn > 65535) { set_error("pec_linear_merged: N too large"); return PEC_ERR_UNSUPPORTED; }
    // Bands of one operand that stay in L2 while the other streams, the cheaper orientation by modelled traffic (the
    // partials weigh n fp32 values per element of the merged operand).  Measured on 32768 rows, Hq = 32, N = 4096:
    // bands of 32 MB against 24 MB: n = 2 1.43 against 1.49 ms, n = 4 3.08 against 2.55 ms.
    const int64_t a_tile = (int64_t)2 * lmg::kBM * K * 4 * n, w_tile = (int64_t)lmg::kBN * K * 2;
    const int64_t a_bytes = pairs * a_tile, w_bytes = gn * w_tile;
    const int64_t band_bytes = (int64_t)(n <= 2 ? 32 : 24) << 20;
    auto clamp_band = [](int64_t b) { return b < 1 ? (int64_t)1 : (b > 32 ? (int64_t)32 : b); };
    const int64_t band_rows = clamp_band(band_bytes / a_tile), band_cols = clamp_band(band_bytes / w_tile);
    const int64_t by_rows_traffic = a_bytes + w_bytes * ((pairs + band_rows - 1) / band_rows);
    const int64_t by_cols_traffic = w_bytes + a_bytes * ((gn + band_cols - 1) / band_cols);
    p.by_cols = by_cols_traffic < by_rows_traffic ? 1 : 0;
    p.band = (int32_t)(p.by_cols ? band_cols : band_rows);
    dim3 grid((unsigned)(2 * pairs), (unsigned)gn);           // clusters of two CTAs along x
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t err = cudaErrorUnknown;
    switch (n) {
    case 1: err = lmg::launch<1>(grid, stream, tm_w, tm_y, p); break;
    case 2: err = lmg::launch<2>(grid, stream, tm_w, tm_y, p); break;
    case 3: err = lmg::launch<3>(grid, stream, tm_w, tm_y, p); break;
    case 4: err = lmg::launch<4>(grid, stream, tm_w, tm_y, p); break;
    case 5: err = lmg::launch<5>(grid, stream, tm_w, tm_y, p); break;
    case 6: err = lmg::launch<6>(grid, stream, tm_w, tm_y, p); break;
    case 7: err = lmg::launch<7>(grid, stream, tm_w, tm_y, p); break;
    case 8: err = lmg::launch<8>(grid, stream, tm_w, tm_y, p); break;
    }
    if (err != cudaSuccess) { set_error("pec_linear_merged: launch failed: %s", cudaGetErrorString(err)); return PEC_ERR_CUDA; }
    return PEC_OK;
}
