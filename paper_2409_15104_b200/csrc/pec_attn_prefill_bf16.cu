// bf16 partial causal attention on the sm_100a tensor cores (Eq. 3-4 as KV-tile partial attention
// with online-softmax state: running max, running sum, fp32 accumulator) - the kernel behind
// pec_prefill_attn for every launch that is not split over the keys.
//
// One CTA = one head x 256 query rows, handled as two 128-row tiles ("stages").  Warp roles (three
// warpgroups):
//   warps 0-3   softmax of stage 0 (one query row per thread = one TMEM lane)
//   warps 4-7   softmax of stage 1
//   warp  8, 10 MMA issuers of stage 0 and stage 1 (one elected lane issues the stage's tcgen05.mma)
//   warp  9     TMA loader (Q once, then K and V tiles through a ring of shared-memory slots)
//   warp  11    idle; it completes the third warpgroup so that it can hand its registers to the
//               softmax warpgroups (setmaxnreg acts on whole warpgroups)
// K and V arrive as 128-key tiles and a tile's scores are one 128 x 128 product (N = 128 halves the
// shared-memory traffic of the Q operand per FLOP against 64-key products, and shared-memory
// bandwidth is what the tensor pipe waits for here).  Tensor memory has room for one such score
// buffer beside the two accumulators, so BOTH stages share it, in turns: S_0(j) lands in it, the
// softmax warps of stage 0 pull their rows into registers (128 per thread) and hand the buffer back
// at once; S_1(j) follows while stage 0 is still at its exponentials, then S_0(j+1), and so on.
// P (bf16) goes to a region of its own per stage, so a product O += P(j) V_j never holds the score
// buffer.  Per stage the issue order is S(j+1), PV(j): the next scores wait in the buffer (or are on
// their way) when the stage's softmax comes back for them, and the tensor pipe always has the other
// stage's work queued.  The accumulator is rescaled lazily: the reference maximum of a row only moves
// when the new maximum exceeds it by 2^8, and a warp that has to rescale first waits for the PV
// product still in flight on its O.
//
// TMEM columns: scores [0, 128); P_s [128 + 64 s, +64); O_s [256 + 128 s, +128).
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "pec_host.h"
#include "pec_internal.h"
#include "pec_sm100.cuh"
#include "pec_tile.cuh"

namespace pec {
using namespace sm100;
namespace pf {

constexpr int kTile = 128;                                 // rows per stage, keys per K/V tile
constexpr int kHalf = 64;                                  // keys per call of the four-step PV helper
constexpr int kBlockM = 2 * kTile;                         // query rows per CTA
constexpr int kStages = 4;                                 // K/V ring slots
constexpr int kThreads = 384;                              // three full warpgroups
constexpr int kSoftmaxWarps = 8, kMmaWarp0 = 8, kLoadWarp = 9, kMmaWarp1 = 10;
constexpr int kLightRegs = 56, kSoftmaxRegs = 224;          // 256 * 224 + 128 * 56 = 384 * 168 (the launch allocation)
constexpr uint32_t kHalfTileBytes = 128 * 64 * 2;          // one TMA box: 128 rows x 64 channels
constexpr uint32_t kTileBytes = 2 * kHalfTileBytes;        // 128 x 128 bf16
constexpr uint32_t kKeyHalfBytes = kHalf * 128;            // 64 rows of a box (128 bytes per row)
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0, kColP = 128, kColO = 256;    // P: + 64 * stage; O: + 128 * stage
constexpr float kRescaleThreshold = 8.0f;                  // log2 units

// What a CTA works on, worked out once by thread 0 and shared through shared memory.  All rows and
// positions fit in 32 bits (the host rejects larger problems).
struct Geom {
    int32_t found;               // 0: tile index past the end
    int32_t q_row0, out_row0, kv_row0;
    int32_t rows[2];             // valid query rows per stage
    int32_t pos0[2];             // position of each stage's first row in its request
    int32_t n[2];                // key tiles each stage takes part in (a prefix of the CTA's walk)
    int32_t lo[2], hi[2];        // visible-key intervals (positions)
    int32_t cnt[2];              // key tiles per interval walked by the CTA (union over both stages)
    int32_t n_max;               // cnt[0] + cnt[1]
};

struct Shared {
    uint64_t bar_q[2];                       // one per stage's Q tile
    uint64_t kv_full[kStages], kv_empty[kStages];
    uint64_t s_full[2], s_taken[2], p_ready[2];   // [stage], one phase per key tile
    uint64_t pv_done[2];                     // one phase per PV product of the stage
    uint64_t o_final[2];                     // the stage's last PV product is done
    Geom g;
    uint32_t tmem_base;
    volatile int abort_flag;
};
constexpr size_t kSmemBytes = (2 + kStages) * kTileBytes + 1024 /*alignment slack*/ + sizeof(Shared);

// Bounded mbarrier wait (the limit is a launch parameter).  Returns false (and raises the abort flag /
// status word) on expiry.
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, Shared *sh, const AttnParams &p)
{
    return mbar_wait_bounded(bar, parity, &sh->abort_flag, p.status, p.wait_cycles, (int)PEC_ERR_TIMEOUT);
}

__global__ void __launch_bounds__(kThreads, 1)
attn_prefill_bf16_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                         const __grid_constant__ CUtensorMap tm_v, const AttnParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;           // swizzled tiles need 1024-byte alignment
    const uint32_t sQ = tiles, sRing = tiles + 2 * kTileBytes;
    Shared *sh = reinterpret_cast<Shared *>(smem_raw + (tiles - raw) + (2 + kStages) * kTileBytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int h = blockIdx.y, kvh = h / p.group;

    // The loader warp finds the CTA's tile and its first lane works out the geometry: heaviest (latest) causal tiles first; per stage
    // the rows, positions and number of key tiles it takes part in.  Key tiles are walked interval 0
    // first, then interval 1, in ascending position, so each stage's tiles are a prefix of the walk.
    // It then initialises the barriers its loads complete on and starts the first loads (Q of stage 0,
    // K(0), Q of stage 1, V(0)) before the CTA-wide sync: their latency is the longest part of a CTA's
    // start-up.  Meanwhile warp 1 initialises the other barriers and warp 2 allocates tensor memory.
    // (Loops over the two intervals and stages are unrolled with constant indices, so the geometry
    // stays in registers.)
    TileJob job;
    bool job_found = false;
    if (warp == kLoadWarp)                                    // whole warp; a work-list is sorted already
        job_found = locate_tile_warp(p, p.worklist ? (int64_t)blockIdx.x : (int64_t)gridDim.x - 1 - blockIdx.x, kBlockM, job);
    if (tid == kLoadWarp * 32) {
        Geom g = {};
        g.found = job_found ? 1 : 0;
        sh->abort_flag = 0;
        if (g.found) {
            g.q_row0 = (int32_t)job.q_row0; g.out_row0 = (int32_t)job.out_row0; g.kv_row0 = (int32_t)job.kv_row0;
            g.cnt[0] = g.cnt[1] = 0;
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                const bool used = t < job.n_iv;
                g.lo[t] = used ? (int32_t)job.iv_lo[t] : 0;
                g.hi[t] = used ? (int32_t)job.iv_hi[t] : 0;
            }
#pragma unroll
            for (int st = 0; st < 2; ++st) {
                int32_t rows = job.n_rows - st * kTile;
                rows = rows < 0 ? 0 : (rows > kTile ? kTile : rows);
                g.rows[st] = rows;
                g.pos0[st] = (int32_t)job.q_pos0 + st * kTile;
                g.n[st] = 0;
                if (rows > 0) {
                    const int32_t last = g.pos0[st] + rows - 1;
#pragma unroll
                    for (int t = 0; t < 2; ++t) {
                        int32_t end = g.hi[t];
                        if (p.causal && end > last + 1) end = last + 1;
                        const int32_t c = end > g.lo[t] ? (end - g.lo[t] + kTile - 1) / kTile : 0;
                        g.n[st] += c;
                        g.cnt[t] = c > g.cnt[t] ? c : g.cnt[t];
                    }
                }
            }
            g.n_max = g.cnt[0] + g.cnt[1];
        }
        sh->g = g;                                            // a CTA past the last tile has no rows and no keys
        mbar_init(smem_u32(&sh->bar_q[0]), 1);
        mbar_init(smem_u32(&sh->bar_q[1]), 1);
#pragma unroll
        for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&sh->kv_full[s]), 1); mbar_init(smem_u32(&sh->kv_empty[s]), 2); }
        mbar_init_fence();
        if (g.n_max > 0) {
            const int krow = g.kv_row0 + (g.cnt[0] > 0 ? g.lo[0] : g.lo[1]);
#pragma unroll
            for (int st = 0; st < 2; ++st) {
                const uint32_t bar_q = smem_u32(&sh->bar_q[st]);
                mbar_arrive_expect_tx(bar_q, kTileBytes);
                tma_load_3d(sQ + st * kTileBytes, &tm_q, bar_q, 0, h, g.q_row0 + st * kTile);
                tma_load_3d(sQ + st * kTileBytes + kHalfTileBytes, &tm_q, bar_q, 64, h, g.q_row0 + st * kTile);
                // ring items 0 and 1: K(0) and V(0)
                const void *map = st ? (const void *)&tm_v : (const void *)&tm_k;
                const uint32_t dst = sRing + st * kTileBytes, bar = smem_u32(&sh->kv_full[st]);
                mbar_arrive_expect_tx(bar, kTileBytes);
                tma_load_3d(dst, map, bar, 0, kvh, krow);
                tma_load_3d(dst + kHalfTileBytes, map, bar, 64, kvh, krow);
            }
        }
    } else if (tid == 32) {
        // Every CTA of the grid has started once the last one has said so: from then on a following launch that
        // may overlap this one (overlap_previous) takes the SMs this grid leaves.
        griddep_launch_dependents();
        prefetch_tmap(&tm_q); prefetch_tmap(&tm_k); prefetch_tmap(&tm_v);
        for (int st = 0; st < 2; ++st) {
            mbar_init(smem_u32(&sh->s_full[st]), 1);
            mbar_init(smem_u32(&sh->s_taken[st]), 4);         // one arrival per softmax warp
            mbar_init(smem_u32(&sh->p_ready[st]), 4);
            mbar_init(smem_u32(&sh->pv_done[st]), 1);
            mbar_init(smem_u32(&sh->o_final[st]), 1);
        }
        mbar_init_fence();
    } else if (warp == 2) {
        tmem_alloc(smem_u32(&sh->tmem_base), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const int n_max = sh->g.n_max;
    const uint32_t tmem = sh->tmem_base;

    // Warps 8-11 (the whole third warpgroup) give registers up, warps 0-7 take them.
    if (warp == kLoadWarp) {
        // ------------------------------------------------------------------ TMA loader
        reg_dealloc<kLightRegs>();
        if (lane == 0 && n_max > 0) {
            for (int i = 2; i < 2 * n_max; ++i) {              // items: K(0), V(0) (loaded above), K(1), V(1), ...
                const int slot = i % kStages, fill = i / kStages;
                if (sh->abort_flag) break;
                if (p.test_skip_last_load && i == 2 * n_max - 1) break;   // test hook: the issuers' wait for V(last) runs out
                if (fill > 0 && !wait_bar(smem_u32(&sh->kv_empty[slot]), (fill - 1) & 1, sh, p)) break;
                const int jt = i >> 1, c0 = sh->g.cnt[0];
                const int krow = sh->g.kv_row0 + (jt < c0 ? sh->g.lo[0] + jt * kTile : sh->g.lo[1] + (jt - c0) * kTile);
                const void *map = (i & 1) ? (const void *)&tm_v : (const void *)&tm_k;
                const uint32_t dst = sRing + slot * kTileBytes, bar = smem_u32(&sh->kv_full[slot]);
                mbar_arrive_expect_tx(bar, kTileBytes);
                tma_load_3d(dst, map, bar, 0, kvh, krow);
                tma_load_3d(dst + kHalfTileBytes, map, bar, 64, kvh, krow);
            }
        }
        __syncwarp();
    } else if (warp == kMmaWarp0 || warp == kMmaWarp1) {
        // ------------------------------------------------------------------ MMA issuers, one warp per stage
        // The whole warp walks the loop and one elected lane issues: addresses, descriptors and loop
        // state stay warp-uniform, which keeps the instruction count per MMA low.  An issuer shares its
        // scheduler with two softmax warps, and one warp issuing for both stages was the kernel's
        // bottleneck.  The stages' accumulators and P regions are disjoint; the score buffer they share is
        // handed from one to the other through the "taken" barriers.  Each issuer waits for and releases
        // every ring item, used by its stage or not, so the "empty" barriers always see two arrivals per item.
        reg_dealloc<kLightRegs>();
        if (n_max > 0) {
            const int st = (warp == kMmaWarp0) ? 0 : 1;
            const bool leader = elect_one();
            constexpr uint32_t idesc_qk = idesc_bf16_f32(kTile, kTile, 0, 0);
            constexpr uint32_t idesc_pv = idesc_bf16_f32(kTile, kHeadDim, 0, 1);
            auto wait_u = [&](uint64_t *bar, uint32_t parity) {
                return __all_sync(0xffffffffu, wait_bar(smem_u32(bar), parity, sh, p));
            };
            auto kv_wait = [&](int item) { return wait_u(&sh->kv_full[item % kStages], (item / kStages) & 1); };
            auto kv_release = [&](int item) { if (leader) tc_commit(smem_u32(&sh->kv_empty[item % kStages])); };
            const uint32_t tS = tmem + kColS, tP = tmem + kColP + st * 64, tO = tmem + kColO + st * kTile;
            // Descriptors: the stage's Q tile gives eight fixed A descriptors (16 channels per K step, four steps
            // per 64-channel box); a K or V tile is the ring's first descriptor plus the slot offset.
            constexpr uint32_t kBox16 = kHalfTileBytes >> 4;
            uint64_t a_desc[8];
#pragma unroll
            for (int ks = 0; ks < 8; ++ks)
                a_desc[ks] = smem_desc_sw128(sQ + st * kTileBytes + (uint32_t)(ks >> 2) * kHalfTileBytes + (uint32_t)(ks & 3) * 32u, 16, 1024);
            const uint64_t k_ring = smem_desc_sw128(sRing, 16, 1024), v_ring = smem_desc_sw128(sRing, kHalfTileBytes, 1024);
            const int n_st = sh->g.n[st], n_ot = sh->g.n[st ^ 1];
            // S(j) = Q K_j^T for the 128 keys of tile j, both operands K-major, into the shared score buffer.
            auto issue_qk = [&](int j) {
                const uint64_t k0 = k_ring + (uint32_t)((((2 * j) % kStages) * kTileBytes) >> 4);
                if (leader) mma_ss_k128_commit<kBox16>(tS, a_desc, k0, idesc_qk, smem_u32(&sh->s_full[st]));
            };
            // O (+)= P(j) V_j: A = P from TMEM (8 columns per 16 keys), B = the V tile stored [key][channel]
            // (N-contiguous): 16 keys = 2048 bytes per step, channel halves 16 KiB apart.
            auto issue_pv = [&](int j, bool last) {
                const uint64_t v0 = v_ring + (uint32_t)((((2 * j + 1) % kStages) * kTileBytes) >> 4);
                if (leader) {
                    mma_ts_k64(tO, tP, v0, idesc_pv, j > 0 ? 1u : 0u);
                    mma_ts_k64(tO, tP + 32, v0 + (kKeyHalfBytes >> 4), idesc_pv, 1u);
                    tc_commit(smem_u32(&sh->pv_done[st]));
                    if (last) tc_commit(smem_u32(&sh->o_final[st]));
                }
            };
            // The score buffer is used in the order (0,0), (1,0), (0,1), (1,1), ... (stage, tile), a stage that has
            // run out of tiles dropping out; S(j) may be issued once the previous user's softmax warps hold
            // their scores in registers.
            auto wait_buffer = [&](int j) {
                int pst, pj;
                if (st == 0) {
                    if (j == 0) return true;
                    pst = (j - 1 < n_ot) ? 1 : 0; pj = j - 1;
                } else {
                    if (j < n_ot) { pst = 0; pj = j; }
                    else if (j > 0) { pst = 1; pj = j - 1; }
                    else return true;
                }
                const bool got = wait_u(&sh->s_taken[pst], pj & 1);
                if (got) tc_fence_after();
                return got;
            };

            bool ok = wait_u(&sh->bar_q[st], 0) && kv_wait(0);
            if (ok) {
                if (n_st > 0) { ok = wait_buffer(0); if (ok) issue_qk(0); }
                kv_release(0);
            }
            for (int j = 0; j < n_max && ok; ++j) {
                if (j + 1 < n_max) {
                    ok = kv_wait(2 * j + 2);                       // K(j+1)
                    if (!ok) break;
                    if (j + 1 < n_st) {
                        ok = wait_buffer(j + 1);
                        if (!ok) break;
                        issue_qk(j + 1);
                    }
                    kv_release(2 * j + 2);
                }
                ok = kv_wait(2 * j + 1);                           // V(j)
                if (!ok) break;
                if (j < n_st) {
                    ok = wait_u(&sh->p_ready[st], j & 1);
                    if (!ok) break;
                    tc_fence_after();
                    issue_pv(j, j == n_st - 1);
                }
                kv_release(2 * j + 1);
            }
        }
        __syncwarp();
    } else if (warp >= kSoftmaxWarps) {
        // The spare warp looks at the caller's status word: if an earlier CTA's wait expired the launch is
        // lost, and raising the abort flag stops the loader, after which every wait of this CTA fails fast.
        // (Kept off the start-up path: the word is a global-memory read.)
        reg_dealloc<kLightRegs>();
        if (lane == 0 && p.status && *reinterpret_cast<volatile int32_t *>(p.status) != 0) sh->abort_flag = 1;
    } else {
        // ------------------------------------------------------------------ softmax + epilogue
        reg_alloc<kSoftmaxRegs>();
        const int st = warp >> 2, quarter = warp & 3;
        const int row_in_tile = quarter * 32 + lane;
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        const uint32_t tS = tmem + lane_base + kColS;
        const uint32_t tP = tmem + lane_base + kColP + st * 64;
        const uint32_t tO = tmem + lane_base + kColO + st * kTile;
        const int n_t = sh->g.n[st], n_hf = 2 * n_t;
        const uint32_t bar_pv = smem_u32(&sh->pv_done[st]);
        // Per interval: where it ends, and the first key position that some row of this stage cannot
        // see (tiles reaching past it need the mask).
        const int pos0 = sh->g.pos0[st], my_pos = pos0 + row_in_tile, t0 = sh->g.cnt[0];
        int iv_full[2], iv_mine[2];
#pragma unroll
        for (int t = 0; t < 2; ++t) {
            const int hi_t = sh->g.hi[t];
            iv_full[t] = (p.causal && pos0 + 1 < hi_t) ? pos0 + 1 : hi_t;
            iv_mine[t] = (p.causal && my_pos + 1 < hi_t) ? my_pos + 1 : hi_t;
        }
        int k0 = sh->g.lo[0], cur = 0;
        const int rows_valid = sh->g.rows[st] - quarter * 32;                   // of this warp's 32 rows
        const int64_t row0 = (int64_t)sh->g.out_row0 + st * kTile + quarter * 32;

        float m_ref = -INFINITY, l_run = 0.f;                // m_ref in log2 units of the scaled scores
        bool ok = true;
        for (int j = 0; j < n_t && ok; ++j, k0 += kTile) {
            if (j == t0) { cur = 1; k0 = sh->g.lo[1]; }
            uint32_t r[kTile];
            ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->s_full[st]), j & 1, sh, p));   // warp-uniform
            if (!ok) break;
            tc_fence_after();
            tmem_ld128(tS, r);
            // The scores are in registers: the buffer may take the other stage's next tile.
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->s_taken[st]));
            // Last tile: start pulling this row of the incoming state towards the L2 (4 x 128 bytes).
            if (p.acc_o != nullptr && j == n_t - 1 && lane < rows_valid) {
                const float *src = p.acc_o + ((row0 + lane) * p.Hq + h) * kHeadDim;
#pragma unroll
                for (int c = 0; c < 4; ++c) prefetch_l2(src + 32 * c);
            }
            // Mask only when some row of this stage cannot see the whole tile.
            const bool masked = k0 + kTile > (cur ? iv_full[1] : iv_full[0]);
            if (masked) {
                int n_vis = (cur ? iv_mine[1] : iv_mine[0]) - k0;
                n_vis = n_vis < 0 ? 0 : (n_vis > kTile ? kTile : n_vis);
#pragma unroll
                for (int c = 0; c < kTile; ++c) r[c] = (c < n_vis) ? r[c] : 0xff800000u;   // -inf
            }
            float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
            for (int c = 0; c < kTile; c += 8) {
                mx0 = fmax3(mx0, __uint_as_float(r[c + 0]), __uint_as_float(r[c + 1]));
                mx1 = fmax3(mx1, __uint_as_float(r[c + 2]), __uint_as_float(r[c + 3]));
                mx2 = fmax3(mx2, __uint_as_float(r[c + 4]), __uint_as_float(r[c + 5]));
                mx3 = fmax3(mx3, __uint_as_float(r[c + 6]), __uint_as_float(r[c + 7]));
            }
            const float m_new = fmax3(mx0, mx1, fmaxf(mx2, mx3)) * p.scale_log2;   // -inf stays -inf (scale > 0)

            // Lazy rescale: move the reference maximum only when it is outgrown by 2^8.
            float alpha = 1.f;
            const bool grow = m_new > m_ref + kRescaleThreshold;
            if (grow) {
                alpha = ex2(m_ref - m_new);                   // 0 when the row had no key so far
                m_ref = m_new;
                l_run *= alpha;
            }
            bool pv_waited = (j == 0);
            if (j > 0 && __any_sync(0xffffffffu, grow)) {
                // O still receives P(j-1) V: wait for that product (phase j-1 of the stage's PV barrier; PV(j)
                // cannot be issued before this warp hands P(j) over, so the phase is unambiguous).
                ok = __all_sync(0xffffffffu, wait_bar(bar_pv, (j - 1) & 1, sh, p));
                if (!ok) break;
                pv_waited = true;
                tc_fence_after();
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint32_t o[32];
                    tmem_ld32(tO + c * 32, o);
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                    tmem_st32(tO + c * 32, o);
                }
            }
            const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
            const float2 sc2 = make_float2(p.scale_log2, p.scale_log2), nm2 = make_float2(neg_m, neg_m);
            float2 sum[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) sum[i] = make_float2(0.f, 0.f);
            // p = 2^(s * scale - m): packed FMA for the argument, the special-function unit for 2^x, packed
            // adds for the row sum.  P is packed to bf16 pairs: column c of the A operand holds keys 2c (low
            // half) and 2c+1 (high half); r[i] is reused for pair i.
#pragma unroll
            for (int i = 0; i < kTile / 2; ++i) {
                const float2 x = __ffma2_rn(make_float2(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1])), sc2, nm2);
                const float2 e = make_float2(ex2(x.x), ex2(x.y));
                sum[i & 3] = __fadd2_rn(sum[i & 3], e);
                r[i] = pack_bf16(e.x, e.y);
            }
            const float2 s01 = __fadd2_rn(__fadd2_rn(sum[0], sum[1]), __fadd2_rn(sum[2], sum[3]));
            l_run += s01.x + s01.y;
            // P(j-1) is read by its product until that is done.
            if (!pv_waited) {
                ok = __all_sync(0xffffffffu, wait_bar(bar_pv, (j - 1) & 1, sh, p));
                if (!ok) break;
                tc_fence_after();
            }
            tmem_st32(tP, r);
            tmem_st32(tP + 32, r + 32);
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh->p_ready[st]));
        }

        // Epilogue: O / l and LSE = ln2 * m + ln l; rows without any visible key give 0 and -inf.  With an
        // incoming state (acc_o, acc_lse) the stage's own result is merged into it by the LSE rule first
        // (online softmax across launches): out = c_own * O_raw + c_acc * acc.
        // A thread holds one whole row, so storing from registers would touch 32 rows per instruction.
        // Each warp instead stages 32 rows x 256 bytes in its quarter of the stage's Q tile (no longer
        // read once the stage's last product is done; 16-byte chunks XOR-swizzled by row against bank
        // conflicts) and writes it out two rows per instruction, 256 contiguous bytes each.
        // A launch that overlaps its predecessor has walked its key tiles beside that kernel's last CTAs; the incoming
        // state and the output buffers are the predecessor's (or an earlier kernel's) until it has completed.
        griddep_wait();
        const bool has_acc = p.acc_o != nullptr;
        const int sub = lane >> 4, chunk = lane & 15;                            // read-back: row parity and 16-byte chunk
        // The incoming state's LSE and its first 64 channels are asked for before the wait for the last product,
        // so that their latency runs under it (the lines were prefetched towards the L2 one tile ago).
        const float *acc_base = has_acc ? p.acc_o + ((row0 + sub) * p.Hq + h) * kHeadDim + chunk * 4 : nullptr;
        float la = -INFINITY;
        float4 inc[16];
        if (has_acc && sh->g.rows[st] > 0) {
            if (lane < rows_valid) la = p.acc_lse[(row0 + lane) * p.Hq + h];
            const float *src = acc_base;
#pragma unroll
            for (int rr = 0; rr < 16; ++rr, src += 2 * (int64_t)p.Hq * kHeadDim) {
                inc[rr] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (2 * rr + sub < rows_valid) inc[rr] = *reinterpret_cast<const float4 *>(src);
            }
        }
        if (ok && n_hf > 0) ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->o_final[st]), 0, sh, p));
        // A stage without keys never waited for its Q tile: the load must have landed before the tile is reused.
        if (ok && n_hf == 0 && n_max > 0) ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->bar_q[st]), 0, sh, p));
        if (ok && sh->g.rows[st] > 0) {
            tc_fence_after();
            const bool empty = (l_run == 0.f);
            float c_own = empty ? 0.f : 1.f / l_run, c_acc = 0.f;
            float lse_row = empty ? -INFINITY : m_ref * 0.6931471805599453f + logf(l_run);
            if (has_acc) {
                const float mx = fmaxf(lse_row, la);
                if (mx != -INFINITY) {
                    const float e_own = empty ? 0.f : expf(lse_row - mx), e_acc = (la == -INFINITY) ? 0.f : expf(la - mx);
                    const float inv_tot = 1.f / (e_own + e_acc);           // the larger of the two terms is exactly 1
                    c_own *= e_own * inv_tot;
                    c_acc = e_acc * inv_tot;
                    lse_row = mx + logf(e_own + e_acc);
                }
            }
            // An in-place merge has nothing to write where no row of the warp gained a key.
            const bool in_place = has_acc && static_cast<const void *>(p.acc_o) == p.o;
            const bool skip = in_place && __all_sync(0xffffffffu, empty || lane >= rows_valid);
            uint8_t *stage_buf = smem_raw + (tiles - raw) + st * kTileBytes + quarter * 8192;
            uint8_t *my_row = stage_buf + lane * 256;
            const int o_esz = p.o_is_bf16 ? 2 : 4;
            const int64_t row_bytes = (int64_t)p.Hq * kHeadDim * o_esz;
            uint8_t *out = static_cast<uint8_t *>(p.o) + (row0 + sub) * row_bytes + (int64_t)h * kHeadDim * o_esz;
            if (skip) {
                // nothing
            } else if (!has_acc && p.o_is_bf16) {
                // One pass: a row is 256 bytes of bf16.
#pragma unroll
                for (int half = 0; half < 2; ++half) {                        // 64 channels = 8 chunks of 16 bytes
                    uint32_t r[64];
                    if (n_hf == 0) {
#pragma unroll
                        for (int i = 0; i < 64; ++i) r[i] = 0u;
                    } else {
                        tmem_ld64(tO + half * 64, r);
                    }
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        uint4 pk;
                        pk.x = pack_bf16(__uint_as_float(r[8 * i + 0]) * c_own, __uint_as_float(r[8 * i + 1]) * c_own);
                        pk.y = pack_bf16(__uint_as_float(r[8 * i + 2]) * c_own, __uint_as_float(r[8 * i + 3]) * c_own);
                        pk.z = pack_bf16(__uint_as_float(r[8 * i + 4]) * c_own, __uint_as_float(r[8 * i + 5]) * c_own);
                        pk.w = pack_bf16(__uint_as_float(r[8 * i + 6]) * c_own, __uint_as_float(r[8 * i + 7]) * c_own);
                        *reinterpret_cast<uint4 *>(my_row + (((half * 8 + i) ^ (lane & 15)) << 4)) = pk;
                    }
                }
                __syncwarp();
                // All sixteen loads first, then the stores: two rows (2 x 256 contiguous bytes) per instruction.
                uint4 val[16];
#pragma unroll
                for (int rr = 0; rr < 16; ++rr) {
                    const int row = 2 * rr + sub;
                    val[rr] = *reinterpret_cast<const uint4 *>(stage_buf + row * 256 + ((chunk ^ (row & 15)) << 4));
                }
                uint8_t *dst = out + chunk * 16;
#pragma unroll
                for (int rr = 0; rr < 16; ++rr, dst += 2 * row_bytes)
                    if (2 * rr + sub < rows_valid) *reinterpret_cast<uint4 *>(dst) = val[rr];
            } else {
                // Two passes of 64 channels staged as fp32 (256 bytes of a row each).
#pragma unroll 1
                for (int pass = 0; pass < 2; ++pass) {
                    // The second half of the incoming state: its latency runs under the TMEM read and the staging.
                    if (has_acc && pass == 1) {
                        const float *src = acc_base + 64;
#pragma unroll
                        for (int rr = 0; rr < 16; ++rr, src += 2 * (int64_t)p.Hq * kHeadDim) {
                            inc[rr] = make_float4(0.f, 0.f, 0.f, 0.f);
                            if (2 * rr + sub < rows_valid) inc[rr] = *reinterpret_cast<const float4 *>(src);
                        }
                    }
                    uint32_t r[64];                                               // 64 channels = 16 chunks of 16 bytes
                    if (n_hf == 0) {
#pragma unroll
                        for (int i = 0; i < 64; ++i) r[i] = 0u;
                    } else {
                        tmem_ld64(tO + pass * 64, r);
                    }
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float4 f = make_float4(__uint_as_float(r[4 * i]) * c_own, __uint_as_float(r[4 * i + 1]) * c_own,
                                                     __uint_as_float(r[4 * i + 2]) * c_own, __uint_as_float(r[4 * i + 3]) * c_own);
                        *reinterpret_cast<float4 *>(my_row + ((i ^ (lane & 15)) << 4)) = f;
                    }
                    __syncwarp();
                    float4 val[16];
#pragma unroll
                    for (int rr = 0; rr < 16; ++rr) {
                        const int row = 2 * rr + sub;
                        val[rr] = *reinterpret_cast<const float4 *>(stage_buf + row * 256 + ((chunk ^ (row & 15)) << 4));
                    }
                    if (has_acc) {
#pragma unroll
                        for (int rr = 0; rr < 16; ++rr) {
                            const float w = __shfl_sync(0xffffffffu, c_acc, 2 * rr + sub);   // the row's weight sits with its owner
                            val[rr].x = fmaf(w, inc[rr].x, val[rr].x); val[rr].y = fmaf(w, inc[rr].y, val[rr].y);
                            val[rr].z = fmaf(w, inc[rr].z, val[rr].z); val[rr].w = fmaf(w, inc[rr].w, val[rr].w);
                        }
                    }
                    if (p.o_is_bf16) {
                        uint8_t *dst = out + pass * 128 + chunk * 8;
#pragma unroll
                        for (int rr = 0; rr < 16; ++rr, dst += 2 * row_bytes)
                            if (2 * rr + sub < rows_valid)
                                *reinterpret_cast<uint2 *>(dst) = make_uint2(pack_bf16(val[rr].x, val[rr].y), pack_bf16(val[rr].z, val[rr].w));
                    } else {
                        uint8_t *dst = out + pass * 256 + chunk * 16;
#pragma unroll
                        for (int rr = 0; rr < 16; ++rr, dst += 2 * row_bytes)
                            if (2 * rr + sub < rows_valid) *reinterpret_cast<float4 *>(dst) = val[rr];
                    }
                    __syncwarp();
                }
            }
            if (!skip && lane < rows_valid) p.lse[(row0 + lane) * p.Hq + h] = lse_row;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 2) tmem_dealloc(tmem, kTmemCols);
}

// ------------------------------------------------------------------------------------------ host
}  // namespace pf

int launch_attn_prefill_bf16(const AttnParams &p, cudaStream_t stream)
{
    using namespace pf;
    if (!p.status) { set_error("pec_prefill_attn: the bf16 path needs a status word"); return PEC_ERR_INVALID_ARG; }
    if (p.splits != 1) { set_error("pec_prefill_attn: this kernel takes no split launches"); return PEC_ERR_INVALID_ARG; }
    // Rows the maps may touch: queries up to the last segment's end, keys up to the end of the visible subset.
    int64_t q_rows = 0, kv_rows = 0, tiles = 0;
    if (p.cu_seqlens) {
        q_rows = p.total_rows; kv_rows = p.total_rows;
        tiles = p.worklist ? p.n_items : (p.total_rows + kBlockM - 1) / kBlockM + p.B;   // without a list every request may end in a ragged tile
    } else {
        for (int s = 0; s < p.n_qseg; ++s) {
            q_rows = p.q_hi[s] > q_rows ? p.q_hi[s] : q_rows;
            tiles += (p.q_hi[s] - p.q_lo[s] + kBlockM - 1) / kBlockM;
        }
        for (int t = 0; t < p.n_iv; ++t) kv_rows = p.iv_hi[t] > kv_rows ? p.iv_hi[t] : kv_rows;
    }
    if (tiles == 0) return PEC_OK;
    if (q_rows >= ((int64_t)1 << 31) || kv_rows >= ((int64_t)1 << 31)) {
        set_error("pec_prefill_attn: more than 2^31 rows unsupported");
        return PEC_ERR_UNSUPPORTED;
    }
    CUtensorMap tm_q, tm_k, tm_v;
    if (!host::make_qkv_map(&tm_q, p.q, q_rows, p.Hq, p.q_stride_t, p.q_stride_h) ||
        !host::make_qkv_map(&tm_k, p.k, kv_rows, p.Hkv, p.k_stride_t, p.k_stride_h) ||
        !host::make_qkv_map(&tm_v, p.v, kv_rows, p.Hkv, p.v_stride_t, p.v_stride_h)) {
        set_error("pec_prefill_attn: cuTensorMapEncodeTiled failed (driver too old, or strides/addresses not encodable)");
        return PEC_ERR_CUDA;
    }
    // Once per device: raise the shared-memory limit, and check that the launch allocation (registers per
    // thread x threads) covers the split in which the softmax warpgroups take registers the third gives up.
    static unsigned char ready[host::kMaxDevices] = {};
    static std::mutex ready_mutex;
    const bool ok = host::once_per_device(ready, ready_mutex, [] {
        if (cudaFuncSetAttribute(attn_prefill_bf16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes) != cudaSuccess) return false;
        cudaFuncAttributes attr;
        return cudaFuncGetAttributes(&attr, attn_prefill_bf16_kernel) == cudaSuccess &&
               attr.numRegs * kThreads >= kSoftmaxWarps * 32 * kSoftmaxRegs + (kThreads - kSoftmaxWarps * 32) * kLightRegs;
    });
    if (!ok) {
        (void)cudaGetLastError();
        set_error("pec_prefill_attn: kernel set-up failed (shared-memory limit, or the register allocation does not cover the warp-role split)");
        return PEC_ERR_CUDA;
    }
    if (tiles > 0x7fffffff || p.Hq > 65535) { set_error("pec_prefill_attn: grid too large"); return PEC_ERR_UNSUPPORTED; }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)tiles, (unsigned)p.Hq, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = kSmemBytes;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = p.overlap_previous ? 1 : 0;
    cudaError_t err = cudaLaunchKernelEx(&cfg, attn_prefill_bf16_kernel, tm_q, tm_k, tm_v, p);
    if (err == cudaSuccess) err = cudaGetLastError();
    if (err != cudaSuccess) { set_error("pec_prefill_attn: launch failed: %s", cudaGetErrorString(err)); return PEC_ERR_CUDA; }
    return PEC_OK;
}

}  // namespace pec
