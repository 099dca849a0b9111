// y = x w^T in bf16 with fp32 accumulation: the dense steps either side of the attention - QKV
// generation (Eq. 2, with W_Q, W_K, W_V of all heads stacked row-wise in w so that y is the fused
// [T, (Hq + 2 Hkv) * 128] tensor whose slices pec_prefill_attn reads through strides) and the
// post-self-attention linear layer (Eq. 5).
//
// A cluster of two CTAs computes 256 x 256 tiles of y with 256-row MMAs (cta_group::2).  Per K
// step of 64 each CTA loads, by TMA into a 6-slot ring (128-byte swizzle, both operands K-major),
// its own 128 rows of x and 128 of the 256 rows of w - half the shared-memory operand traffic per
// operation of a single-CTA 128 x 256 tile - and keeps its 128 rows of the fp32 accumulator in its
// own tensor memory.  The even-ranked CTA (the leader) issues every tcgen05.mma; both CTAs' loads
// count on the leader's "full" barrier and the leader's commits arrive on both CTAs' barriers.
// The kernel is persistent: one pair per two SMs walks every (number of pairs)-th tile of a banded
// tile order, the operand ring runs on through the tile boundaries and the accumulator is double-
// buffered (2 x 256 tensor-memory columns), so the MMAs of the next tile run while warps 0-3 of each
// CTA read the finished one out (a lane = a row), round to bf16, lay their rows out in staging
// boxes of 32 rows x 64 columns and hand those to the TMA; the pair's barriers, tensor memory and
// first loads' latency are paid once per CTA, not per tile.  "Accumulator free" is signalled to
// the leader by all eight reading warps of the pair (cluster-scope release / acquire).
// Tensor-bound: 2 * M * N * K operations.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "pec_host.h"
#include "pec_internal.h"
#include "pec_sm100.cuh"
#include "pec_tma_store.cuh"

namespace pec {
using namespace sm100;

namespace lin {
constexpr int kBM = 128, kBN = 256, kBK = 64;
constexpr int kMaxSlots = 6;
// Operand ring and staging boxes per warp: 6 slots (192 KB) + 2 boxes; with the rotary encoding 5 slots + 4 boxes, so that
// both heads of a tile are staged side by side and a row's cosines and sines are worked out once per tile.  224 KB either way.
template <bool kRope> struct Cfg { static constexpr int kSlots = kRope ? 5 : 6, kBoxes = kRope ? 4 : 2; };
constexpr int kThreads = 192;                               // 4 epilogue warps, MMA warp, loader warp
constexpr uint32_t kABytes = kBM * kBK * 2;                 // this CTA's 128 rows of x
constexpr uint32_t kWBytes = 128 * kBK * 2;                 // this CTA's half of the 256 rows of w
constexpr uint32_t kSlotBytes = kABytes + kWBytes;          // 32 KB
// What the waits of a CTA need: its abort flag, the caller's status word and the wait limit.
struct WaitCtx { volatile int *abort_flag; int32_t *status; long long limit; };
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, const WaitCtx &w)
{
    return mbar_wait_bounded(bar, parity, w.abort_flag, w.status, w.limit, (int)PEC_ERR_TIMEOUT);
}

// Rotary position encoding applied to the accumulator before it is rounded (kRope): the leading rot_cols
// columns of y are heads of 128 channels; channel i < 64 of a head pairs with channel i + 64 and the pair of
// the row at position p is turned by the angle p * f_i.  The angle's cosine and sine come from two small tables
// by the addition theorem, p = 64 a + b:  cos(p f) = C[a][i] F[i][b] - S[a][i] G[i][b], sin likewise, with
// C, S = cos, sin(64 a f_i) ("coarse", one row of 64 per 64 positions) and F, G = cos, sin(b f_i) ("fine",
// 64 x 64, stored channel-major so that a warp's 32 consecutive positions read 128 contiguous bytes).
// A table of every position's angles read row by row costs 32 memory wavefronts per load instruction (each
// lane its own line) and made the epilogue 6 % of the GEMM; these reads are one or two wavefronts each.
// Table layout (floats): F [64][64] | G [64][64] | C [na][64] | S [na][64], na = ceil(n_pos / 64).
struct Rope {
    const float *table;
    const int32_t *positions;                                 // [M] or NULL: row r is at position pos0 + r
    int64_t pos0;
    int32_t n_pos, rot_cols;
};
constexpr int kRopeFine = 64 * 64;

// 16 accumulator columns of row `lane` -> bf16 -> chunks `chunk`, `chunk` + 1 of a box (see pec_tma_store.cuh).
__device__ __forceinline__ void box_put16(uint32_t box, int lane, int chunk, const uint32_t *r)
{
#pragma unroll
    for (int i = 0; i < 16; i += 8)
        box_put(box, lane, chunk + (i >> 3),
                pack_bf16(__uint_as_float(r[i + 0]), __uint_as_float(r[i + 1])), pack_bf16(__uint_as_float(r[i + 2]), __uint_as_float(r[i + 3])),
                pack_bf16(__uint_as_float(r[i + 4]), __uint_as_float(r[i + 5])), pack_bf16(__uint_as_float(r[i + 6]), __uint_as_float(r[i + 7])));
}
// Cosines and sines of sixteen channels i0 .. i0 + 15 for the row at position 64 a + b (see Rope).
__device__ __forceinline__ void rope_angles(const float *table, int na, int a, int b, int i0, float (&c)[16], float (&s)[16])
{
    const float *cc = table + 2 * kRopeFine + (int64_t)a * 64 + i0, *cs = cc + (int64_t)na * 64;
    float4 c4[4], s4[4];
#pragma unroll
    for (int v = 0; v < 4; ++v) { c4[v] = __ldg(reinterpret_cast<const float4 *>(cc) + v); s4[v] = __ldg(reinterpret_cast<const float4 *>(cs) + v); }
    const float *ccf = reinterpret_cast<const float *>(c4), *csf = reinterpret_cast<const float *>(s4);
    const float *f = table + i0 * 64 + b, *g = f + kRopeFine;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const float fc = __ldg(f + j * 64), fs = __ldg(g + j * 64);
        c[j] = ccf[j] * fc - csf[j] * fs;
        s[j] = csf[j] * fc + ccf[j] * fs;
    }
}
// Two 16-column accumulator loads in flight, then one wait.
__device__ __forceinline__ void tmem_ld16x2(uint32_t ta, uint32_t (&a)[16], uint32_t tb, uint32_t (&b)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%32];\n\t"
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%33];\n\t"
        "tcgen05.wait::ld.sync.aligned;"
        : "=r"(a[0]), "=r"(a[1]), "=r"(a[2]), "=r"(a[3]), "=r"(a[4]), "=r"(a[5]), "=r"(a[6]), "=r"(a[7]),
          "=r"(a[8]), "=r"(a[9]), "=r"(a[10]), "=r"(a[11]), "=r"(a[12]), "=r"(a[13]), "=r"(a[14]), "=r"(a[15]),
          "=r"(b[0]), "=r"(b[1]), "=r"(b[2]), "=r"(b[3]), "=r"(b[4]), "=r"(b[5]), "=r"(b[6]), "=r"(b[7]),
          "=r"(b[8]), "=r"(b[9]), "=r"(b[10]), "=r"(b[11]), "=r"(b[12]), "=r"(b[13]), "=r"(b[14]), "=r"(b[15])
        : "r"(ta), "r"(tb) : "memory");
}

// ---------------------------------------------------------------------------------------------
// The kernel: one CTA pair per two SMs walks its share of the tiles (see the head of the file).
struct Shared {
    uint64_t full[kMaxSlots], empty[kMaxSlots], acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    volatile int abort_flag;
};
template <bool kRope> constexpr size_t smem_bytes() { return Cfg<kRope>::kSlots * kSlotBytes + 4 * Cfg<kRope>::kBoxes * kStoreBoxBytes + 1024 + sizeof(Shared); }

__device__ __forceinline__ void arrive_cluster(uint32_t cluster_bar)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ bool wait_cluster(uint32_t bar, uint32_t parity, const WaitCtx &w)
{
    const long long t0 = clock64();
    for (;;) {
        uint32_t ok;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(ok) : "r"(bar), "r"(parity), "r"(2000u) : "memory");
        if (ok) return true;
        if (*w.abort_flag) return false;
        if (clock64() - t0 > w.limit) {
            *w.abort_flag = 1;
            if (w.status) atomicExch(w.status, (int)PEC_ERR_TIMEOUT);
            return false;
        }
    }
}
__device__ __forceinline__ void bulk_wait_read_1() { asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory"); }

struct Tiles { int32_t pairs, gn, band, by_cols, n_clusters; int64_t total; };
__device__ __forceinline__ void tile_of(const Tiles &t, int64_t seq, int &pair_i, int &col_i)
{
    if (!t.by_cols) {
        const int band_i = (int)(seq / ((int64_t)t.band * t.gn));
        const int band_pairs = (t.pairs - band_i * t.band) < t.band ? (t.pairs - band_i * t.band) : t.band;
        const int within = (int)(seq - (int64_t)band_i * t.band * t.gn);
        pair_i = band_i * t.band + within % band_pairs;
        col_i = within / band_pairs;
    } else {
        const int band_i = (int)(seq / ((int64_t)t.band * t.pairs));
        const int band_cols = (t.gn - band_i * t.band) < t.band ? (t.gn - band_i * t.band) : t.band;
        const int within = (int)(seq - (int64_t)band_i * t.band * t.pairs);
        col_i = band_i * t.band + within % band_cols;
        pair_i = within / band_cols;
    }
}

template <bool kRope>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
linear_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_y,
                         int64_t M, int32_t N, int32_t K, const Tiles tiles, int32_t *status,
                         long long wait_cycles, int32_t test_skip_last_load, const Rope rope)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t ring = (raw + 1023u) & ~1023u;
    constexpr int kSlots = Cfg<kRope>::kSlots, kBoxes = Cfg<kRope>::kBoxes;
    const uint32_t stage = ring + kSlots * kSlotBytes;
    Shared *sh = reinterpret_cast<Shared *>(smem_raw + (ring - raw) + kSlots * kSlotBytes + 4 * kBoxes * kStoreBoxBytes);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = cluster_ctarank();                  // 0 = leader
    const int cid = (int)(blockIdx.x >> 1);
    const int n_kb = (K + kBK - 1) / kBK;
    const WaitCtx wctx = {&sh->abort_flag, status, wait_cycles};

    if (tid == 0) {
        sh->abort_flag = (status && *reinterpret_cast<volatile int32_t *>(status) != 0) ? 1 : 0;
        for (int s = 0; s < kSlots; ++s) { mbar_init(smem_u32(&sh->full[s]), 1); mbar_init(smem_u32(&sh->empty[s]), 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(smem_u32(&sh->acc_full[b]), 1); mbar_init(smem_u32(&sh->acc_empty[b]), 8); }
        mbar_init_fence();
        prefetch_tmap(&tm_x); prefetch_tmap(&tm_w); prefetch_tmap(&tm_y);
    }
    __syncthreads();
    cluster_sync();                                           // both CTAs' barriers exist before anyone signals them
    if (warp == 0) {
        tmem_alloc_pair(smem_u32(&sh->tmem_base), 512);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh->tmem_base;

    if (warp == 5) {
        if (lane == 0) {
            int it = 0;
            bool ok = true;
            for (int64_t seq = cid; seq < tiles.total && ok; seq += tiles.n_clusters) {
                int pair_i, col_i;
                tile_of(tiles, seq, pair_i, col_i);
                const int m0 = pair_i * (2 * kBM) + (int)rank * kBM, n0 = col_i * kBN;
                const bool last_tile = seq + tiles.n_clusters >= tiles.total;
                for (int kb = 0; kb < n_kb; ++kb, ++it) {
                    const int slot = it % kSlots, fill = it / kSlots;
                    if (test_skip_last_load && rank == 1 && last_tile && kb == n_kb - 1) { ok = false; break; }   // test hook
                    if (fill > 0 && !wait_bar(smem_u32(&sh->empty[slot]), (fill - 1) & 1, wctx)) { ok = false; break; }
                    const uint32_t a = ring + slot * kSlotBytes;
                    const uint32_t bar = leader_addr(smem_u32(&sh->full[slot]));
                    if (rank == 0) mbar_arrive_expect_tx(smem_u32(&sh->full[slot]), 2 * kSlotBytes);   // both CTAs' bytes
                    tma_load_2d_pair(a, &tm_x, bar, kb * kBK, m0);
                    tma_load_2d_pair(a + kABytes, &tm_w, bar, kb * kBK, n0 + (int)rank * 128);
                }
            }
        }
        __syncwarp();
    } else if (warp == 4) {
        if (lane == 0 && rank == 0) {
            constexpr uint32_t idesc = idesc_bf16_f32(2 * kBM, kBN, 0, 0);
            bool ok = true;
            int it = 0, ti = 0;
            for (int64_t seq = cid; seq < tiles.total && ok; seq += tiles.n_clusters, ++ti) {
                const int b = ti & 1;
                if (ti >= 2) {                                // both CTAs have read this accumulator's previous tile out
                    ok = wait_cluster(smem_u32(&sh->acc_empty[b]), ((ti >> 1) - 1) & 1, wctx);
                    if (!ok) break;
                    tc_fence_after();
                }
                const uint32_t acc = tmem + b * 256;
                for (int kb = 0; kb < n_kb && ok; ++kb, ++it) {
                    const int slot = it % kSlots;
                    ok = wait_bar(smem_u32(&sh->full[slot]), (it / kSlots) & 1, wctx);
                    if (!ok) break;
                    const uint32_t a = ring + slot * kSlotBytes, bb = a + kABytes;
#pragma unroll
                    for (int ks = 0; ks < kBK / 16; ++ks)
                        mma_ss_pair(acc, smem_desc_sw128(a + ks * 32u, 16, 1024), smem_desc_sw128(bb + ks * 32u, 16, 1024), idesc,
                                    (kb > 0 || ks > 0) ? 1u : 0u);
                    tc_commit_pair(smem_u32(&sh->empty[slot]));
                }
                if (ok) tc_commit_pair(smem_u32(&sh->acc_full[b]));
            }
        }
        __syncwarp();
    } else {
        const uint32_t boxes = stage + (uint32_t)warp * (kBoxes * kStoreBoxBytes);
        int ti = 0, n_sent = 0;
        bool ok = true;
        for (int64_t seq = cid; seq < tiles.total && ok; seq += tiles.n_clusters, ++ti) {
            int pair_i, col_i;
            tile_of(tiles, seq, pair_i, col_i);
            const int m0 = pair_i * (2 * kBM) + (int)rank * kBM, n0 = col_i * kBN;
            const int b = ti & 1;
            const int row0 = m0 + warp * 32;
            const int64_t row = (int64_t)row0 + lane;
            [[maybe_unused]] int rope_a = 0, rope_b = 0, rope_na = 0;
            if constexpr (kRope) {
                int64_t pos = 0;
                if (row < M) pos = rope.positions ? (int64_t)rope.positions[row] : rope.pos0 + row;
                pos = pos < 0 ? 0 : (pos >= rope.n_pos ? rope.n_pos - 1 : pos);
                rope_a = (int)(pos >> 6); rope_b = (int)(pos & 63); rope_na = (rope.n_pos + 63) >> 6;
            }
            ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->acc_full[b]), (ti >> 1) & 1, wctx));
            if (!ok) break;
            tc_fence_after();
            const uint32_t taddr = tmem + ((uint32_t)(warp * 32) << 16) + b * 256;
            // A staging box may be written again once the TMA has read what was sent from it two boxes ago.
            auto box_for = [&]() {
                if (n_sent >= 2) { if (lane == 0) bulk_wait_read_1(); __syncwarp(); }
                return boxes + (uint32_t)(n_sent & 1) * kStoreBoxBytes;
            };
            auto send = [&](uint32_t box, int j) {            // columns n0 + 64 j .. + 63
                fence_async_smem();
                __syncwarp();
                if (lane == 0) {
                    if (row0 < M && n0 + 64 * j < N) box_store(&tm_y, box, n0 + 64 * j, row0);
                    bulk_commit();
                }
                ++n_sent;
            };
            if constexpr (!kRope) {
#pragma unroll 1
                for (int j = 0; j < 4; ++j) {
                    uint32_t r[32];
                    const uint32_t box = box_for();
                    tmem_ld32(taddr + j * 64, r);
                    box_put16(box, lane, 0, r);
                    box_put16(box, lane, 2, r + 16);
                    tmem_ld32(taddr + j * 64 + 32, r);
                    box_put16(box, lane, 4, r);
                    box_put16(box, lane, 6, r + 16);
                    if (j == 3) {                             // the accumulator is in registers / shared memory: hand it back
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) arrive_cluster(leader_addr(smem_u32(&sh->acc_empty[b])));
                    }
                    send(box, j);
                }
            } else {
                // Two heads per tile, two boxes per head (channels 0-63 and their partners 64-127), all four staged side by
                // side; sixteen pairs of both heads per step, so a row's cosines and sines are worked out once per tile.
                if (n_sent > 0) { if (lane == 0) bulk_wait_read(); __syncwarp(); }
                const bool turn0 = n0 < rope.rot_cols, turn1 = n0 + 128 < rope.rot_cols;    // rot_cols: whole heads
#pragma unroll 1
                for (int it = 0; it < 4; ++it) {
                    float cf[16], sf[16];
                    if (turn0) rope_angles(rope.table, rope_na, rope_a, rope_b, it * 16, cf, sf);   // a tile of value heads needs none
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        uint32_t a[16], bq[16];
                        tmem_ld16x2(taddr + hh * 128 + it * 16, a, taddr + hh * 128 + 64 + it * 16, bq);
                        if (hh == 0 ? turn0 : turn1) {
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                const float xa = __uint_as_float(a[j]), xb = __uint_as_float(bq[j]);
                                a[j] = __float_as_uint(xa * cf[j] - xb * sf[j]);
                                bq[j] = __float_as_uint(xb * cf[j] + xa * sf[j]);
                            }
                        }
                        box_put16(boxes + (2 * hh) * kStoreBoxBytes, lane, it * 2, a);
                        box_put16(boxes + (2 * hh + 1) * kStoreBoxBytes, lane, it * 2, bq);
                    }
                }
                tc_fence_before();                            // the accumulator is in shared memory: hand it back
                __syncwarp();
                if (lane == 0) arrive_cluster(leader_addr(smem_u32(&sh->acc_empty[b])));
#pragma unroll
                for (int j = 0; j < 4; ++j) send(boxes + j * kStoreBoxBytes, j);
            }
        }
        if (lane == 0) bulk_wait_read();                      // the boxes must outlive the TMA's reads of them
        __syncwarp();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();                                           // the partner is done with this CTA's memory too
    if (warp == 0) tmem_dealloc_pair(tmem, 512);
}
}  // namespace lin
}  // namespace pec

// The two-level tables of Rope, worked out in fp64 and stored as fp32: one thread per (fine or coarse) entry.
namespace pec {
namespace lin {
__global__ void rope_table_kernel(double log2_theta, int64_t na, float *table)
{
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= kRopeFine + na * 64) return;
    int i;
    double p;
    float *c_out, *s_out;
    if (idx < kRopeFine) {                                    // fine: channel-major, F[i][b]
        i = (int)(idx >> 6); p = (double)(idx & 63);
        c_out = table + idx; s_out = c_out + kRopeFine;
    } else {                                                  // coarse: C[a][i]
        const int64_t j = idx - kRopeFine;
        i = (int)(j & 63); p = (double)((j >> 6) * 64);
        c_out = table + 2 * kRopeFine + j; s_out = c_out + na * 64;
    }
    double s, c;
    sincos(p * exp2(-(double)(2 * i) / 128.0 * log2_theta), &s, &c);
    *c_out = (float)c;
    *s_out = (float)s;
}
}  // namespace lin
}  // namespace pec

using namespace pec;

static int linear_common(const char *who, const void *x, int64_t x_stride, const void *w, int64_t w_stride, void *y, int64_t y_stride,
                         int64_t M, int32_t N, int32_t K, int32_t *status, void *cuda_stream, const lin::Rope *rope)
{
    if (!x || !w || !y || !status) { set_error("%s: x, w, y and status must be non-NULL", who); return PEC_ERR_INVALID_ARG; }
    if (M < 0 || N < 1 || K < 1 || M >= ((int64_t)1 << 31)) { set_error("%s: need 0 <= M < 2^31, N >= 1, K >= 1", who); return PEC_ERR_INVALID_ARG; }
    if (N % 8 != 0 || K % 8 != 0) { set_error("%s: N and K must be multiples of 8", who); return PEC_ERR_UNSUPPORTED; }
    if (x_stride < K || w_stride < K || y_stride < N) { set_error("%s: a row stride is smaller than the row", who); return PEC_ERR_INVALID_ARG; }
    if (x_stride % 8 != 0 || w_stride % 8 != 0 || y_stride % 8 != 0 || (reinterpret_cast<uintptr_t>(x) & 15u) ||
        (reinterpret_cast<uintptr_t>(w) & 15u) || (reinterpret_cast<uintptr_t>(y) & 15u) || (reinterpret_cast<uintptr_t>(status) & 3u)) {
        set_error("%s: x, w, y must be 16-byte aligned with row strides that are multiples of 8 elements", who);
        return PEC_ERR_ALIGNMENT;
    }
    if (rope) {
        if (!rope->table || rope->n_pos < 1) { set_error("%s: the table must be non-NULL with n_pos >= 1", who); return PEC_ERR_INVALID_ARG; }
        if (rope->rot_cols < 0 || rope->rot_cols > N) { set_error("%s: rot_cols must lie in [0, N]", who); return PEC_ERR_INVALID_ARG; }
        if (rope->rot_cols % 128 != 0) { set_error("%s: rot_cols must be a multiple of 128 (whole heads)", who); return PEC_ERR_UNSUPPORTED; }
        if (!rope->positions && (rope->pos0 < 0 || rope->pos0 + M > rope->n_pos)) {
            set_error("%s: positions pos0 .. pos0 + M - 1 must lie inside the tables", who);
            return PEC_ERR_INVALID_ARG;
        }
        if ((reinterpret_cast<uintptr_t>(rope->table) & 15u) || (reinterpret_cast<uintptr_t>(rope->positions) & 3u)) {
            set_error("%s: the table must be 16-byte aligned", who);
            return PEC_ERR_ALIGNMENT;
        }
    }
    if (M == 0) return PEC_OK;
    CUtensorMap tm_x, tm_w, tm_y;
    if (!host::make_matrix_map(&tm_x, x, M, K, x_stride, lin::kBM) || !host::make_matrix_map(&tm_w, w, N, K, w_stride, 128) ||
        !host::make_matrix_map(&tm_y, y, M, N, y_stride, (int)sm100::kStoreBoxRows)) {
        set_error("%s: cuTensorMapEncodeTiled failed", who);
        return PEC_ERR_CUDA;
    }
    static unsigned char ready[host::kMaxDevices] = {};
    static int sm_count[host::kMaxDevices] = {};
    static std::mutex ready_mutex;
    if (!host::once_per_device(ready, ready_mutex, [] {
            int dev = 0, sms = 0;
            if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return false;
            sm_count[dev] = sms;
            return cudaFuncSetAttribute(lin::linear_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lin::smem_bytes<false>()) == cudaSuccess &&
                   cudaFuncSetAttribute(lin::linear_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)lin::smem_bytes<true>()) == cudaSuccess; })) {
        set_error("%s: cannot raise the shared-memory limit: %s", who, cudaGetErrorString(cudaGetLastError()));
        return PEC_ERR_CUDA;
    }
    int dev = 0;
    cudaGetDevice(&dev);
    const int64_t pairs = (M + 2 * lin::kBM - 1) / (2 * lin::kBM), gn = (N + lin::kBN - 1) / lin::kBN;
    const int64_t tile_bytes = (int64_t)2 * lin::kBM * K * 2;           // 256 rows of either operand
    int64_t band = ((int64_t)24 << 20) / tile_bytes;
    band = band < 4 ? 4 : (band > 32 ? 32 : band);
    const int64_t x_bytes = (int64_t)M * K * 2, w_bytes = (int64_t)N * K * 2;
    const int64_t by_rows_traffic = x_bytes + w_bytes * ((pairs + band - 1) / band);
    const int64_t by_cols_traffic = w_bytes + x_bytes * ((gn + band - 1) / band);
    lin::Tiles tiles;
    tiles.pairs = (int32_t)pairs; tiles.gn = (int32_t)gn; tiles.band = (int32_t)band;
    tiles.by_cols = by_cols_traffic < by_rows_traffic ? 1 : 0;
    tiles.total = pairs * gn;
    const int64_t max_clusters = sm_count[dev] / 2 > 0 ? sm_count[dev] / 2 : 1;
    tiles.n_clusters = (int32_t)(tiles.total < max_clusters ? tiles.total : max_clusters);
    dim3 grid((unsigned)(2 * tiles.n_clusters));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (rope)
        lin::linear_kernel<true><<<grid, lin::kThreads, lin::smem_bytes<true>(), stream>>>(
            tm_x, tm_w, tm_y, M, N, K, tiles, status, (long long)wait_limit_cycles(), test_skip_last_load(), *rope);
    else
        lin::linear_kernel<false><<<grid, lin::kThreads, lin::smem_bytes<false>(), stream>>>(
            tm_x, tm_w, tm_y, M, N, K, tiles, status, (long long)wait_limit_cycles(), test_skip_last_load(), lin::Rope{});
    const cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) { set_error("%s: launch failed: %s", who, cudaGetErrorString(err)); return PEC_ERR_CUDA; }
    return PEC_OK;
}

extern "C" int pec_linear(const void *x, int64_t x_stride, const void *w, int64_t w_stride, void *y, int64_t y_stride,
                          int64_t M, int32_t N, int32_t K, int32_t *status, void *cuda_stream)
{
    return linear_common("pec_linear", x, x_stride, w, w_stride, y, y_stride, M, N, K, status, cuda_stream, nullptr);
}

extern "C" int pec_linear_rope(const void *x, int64_t x_stride, const void *w, int64_t w_stride, void *y, int64_t y_stride,
                               int64_t M, int32_t N, int32_t K, const float *rope_table, int64_t n_pos,
                               const int32_t *positions, int64_t pos0, int32_t rot_cols, int32_t *status, void *cuda_stream)
{
    if (n_pos >= ((int64_t)1 << 31)) { set_error("pec_linear_rope: n_pos must be below 2^31"); return PEC_ERR_INVALID_ARG; }
    lin::Rope rope = {rope_table, positions, pos0, (int32_t)n_pos, rot_cols};
    return linear_common("pec_linear_rope", x, x_stride, w, w_stride, y, y_stride, M, N, K, status, cuda_stream, &rope);
}

extern "C" size_t pec_rope_table_floats(int64_t n_pos)
{
    if (n_pos < 0 || n_pos >= ((int64_t)1 << 31)) return 0;
    return (size_t)(2 * lin::kRopeFine) + (size_t)((n_pos + 63) / 64) * 128;
}

extern "C" int pec_rope_table(double theta, int64_t n_pos, int32_t D, float *table, void *cuda_stream)
{
    if (!table || n_pos < 0 || !(theta > 0.0)) { set_error("pec_rope_table: need a table, n_pos >= 0 and theta > 0"); return PEC_ERR_INVALID_ARG; }
    if (D != 128) { set_error("pec_rope_table: D must be 128"); return PEC_ERR_UNSUPPORTED; }
    if (n_pos >= ((int64_t)1 << 31)) { set_error("pec_rope_table: n_pos must be below 2^31"); return PEC_ERR_INVALID_ARG; }
    if (reinterpret_cast<uintptr_t>(table) & 15u) { set_error("pec_rope_table: the table must be 16-byte aligned"); return PEC_ERR_ALIGNMENT; }
    const int64_t na = (n_pos + 63) / 64, n = lin::kRopeFine + na * 64;
    lin::rope_table_kernel<<<(unsigned)((n + 255) / 256), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(std::log2(theta), na, table);
    const cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) { set_error("pec_rope_table: launch failed: %s", cudaGetErrorString(err)); return PEC_ERR_CUDA; }
    return PEC_OK;
}
