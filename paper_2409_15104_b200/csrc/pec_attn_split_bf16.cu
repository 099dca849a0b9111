// bf16 partial attention of a few query rows against a long key range, split over the keys: the
// kernel behind pec_decode_attn (Eq. 3-4 as KV-tile partial attention with online-softmax state;
// the partials of the key slices are merged by their LSE afterwards).
//
// One CTA = one group of query heads (up to 128 rows) x two key slices.  Both 128-row "stages" hold
// the same query rows and each walks its own slice, so a CTA keeps two slices in flight and one
// slice's softmax runs under the other's MMAs.  Warp roles (three warpgroups):
//   warps 0-3   softmax of stage 0 (one query row per thread = one TMEM lane)
//   warps 4-7   softmax of stage 1
//   warp  8     MMA issuer (one elected lane issues every tcgen05.mma)
//   warp  9     TMA loader (Q once, then K and V tiles through a ring of shared-memory slots)
//   warps 10-11 idle; they complete the third warpgroup so that it can hand its registers to the
//               softmax warpgroups (setmaxnreg acts on whole warpgroups)
// S = Q K^T lands in tensor memory, the softmax warps turn it into P (bf16, written back over the
// first half of S), and O += P V accumulates in tensor memory.  The accumulator is rescaled lazily:
// the reference maximum of a row only moves when the new maximum exceeds it by 2^8.  The kernel is
// bound by the K/V stream from HBM, not by the tensor pipe.
//
// TMEM columns: S_0 [0,128) (P_0 in [0,64)), S_1 [128,256) (P_1 in [128,192)), O_0 [256,384),
// O_1 [384,512).
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include "pec_host.h"
#include "pec_internal.h"
#include "pec_sm100.cuh"
#include "pec_tile.cuh"

namespace pec {
using namespace sm100;
namespace splitk {

constexpr int kTile = 128;                                 // rows per stage, keys per KV tile
constexpr int kBlockM = 2 * kTile;                         // query rows per CTA
constexpr int kStages = 4;                                 // K/V ring slots
constexpr int kThreads = 384;                              // three full warpgroups
constexpr int kSoftmaxWarps = 8, kMmaWarp = 8, kLoadWarp = 9;
constexpr int kLightRegs = 56, kSoftmaxRegs = 224;          // 256 * 224 + 128 * 56 = 384 * 168 (the launch allocation)
constexpr uint32_t kHalfTileBytes = 128 * 64 * 2;          // one TMA box: 128 rows x 64 bf16
constexpr uint32_t kTileBytes = 2 * kHalfTileBytes;        // 128 x 128 bf16
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0, kColO = 256;                 // + 128 * stage
constexpr float kRescaleThreshold = 8.0f;                  // log2 units

// What a CTA works on, worked out once by thread 0 and shared through shared memory.  All rows and
// positions fit in 32 bits (the host rejects larger problems).
struct Geom {
    int32_t found;               // 0: tile index past the end (or the launch was already aborted)
    int32_t q_row0, out_row0, kv_row0;
    int32_t rows[2];             // valid query rows per stage
    int32_t pos0[2];             // position of each stage's first row in its request
    int32_t n[2];                // key tiles each stage takes part in (a prefix of the CTA's walk)
    int32_t lo[2], hi[2];        // visible-key intervals (positions)
    int32_t cnt[2];              // key tiles per interval walked by the CTA (union over both stages)
    int32_t n_max;               // the larger of the two stages' counts
    int32_t out_st_stride;       // output-row distance between the stages' slices (rows per slice)
};

struct Shared {
    uint64_t bar_q;
    uint64_t kv_full[kStages], kv_empty[kStages];
    uint64_t s_full[2], p_ready[2], o_final[2];
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
attn_split_bf16_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                 const __grid_constant__ CUtensorMap tm_v, const AttnParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t tiles = (raw + 1023u) & ~1023u;           // swizzled tiles need 1024-byte alignment
    const uint32_t sQ = tiles, sRing = tiles + 2 * kTileBytes;
    Shared *sh = reinterpret_cast<Shared *>(smem_raw + (tiles - raw) + (2 + kStages) * kTileBytes);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int h = blockIdx.y, kvh = h / p.group;

    // Thread 0 works out the CTA's geometry: per stage the key slice and the number of key tiles.
    if (tid == 0) {
        Geom g;
        TileJob job;
        g.found = locate_tile(p, (int64_t)gridDim.x - 1 - blockIdx.x, kBlockM, job) ? 1 : 0;
        // An earlier CTA's wait expired: the launch is already lost, leave at once.
        if (p.status && *reinterpret_cast<volatile int32_t *>(p.status) != 0) g.found = 0;
        sh->abort_flag = 0;
        if (g.found) {                                        // stage st takes key slice 2 * blockIdx.z + st (interval st)
            g.q_row0 = (int32_t)job.q_row0; g.kv_row0 = (int32_t)job.kv_row0;
            g.out_st_stride = (int32_t)p.total_rows;
            g.out_row0 = (int32_t)job.out_row0 + 2 * (int32_t)blockIdx.z * (int32_t)p.total_rows;
            g.n_max = 0;
            for (int st = 0; st < 2; ++st) {
                const int64_t slice = 2 * (int64_t)blockIdx.z + st;
                int64_t lo = job.iv_lo[0] + slice * p.split_keys;
                int64_t hi = lo + p.split_keys < job.iv_hi[0] ? lo + p.split_keys : job.iv_hi[0];
                if (job.n_iv == 0 || hi < lo) hi = lo;
                const int32_t rows = (slice < p.splits) ? (job.n_rows > kTile ? kTile : job.n_rows) : 0;
                g.rows[st] = rows;
                g.pos0[st] = (int32_t)job.q_pos0;
                g.lo[st] = (int32_t)lo; g.hi[st] = (int32_t)hi;
                int32_t end = g.hi[st];
                if (p.causal && end > g.pos0[st] + rows) end = g.pos0[st] + rows;
                g.cnt[st] = (rows > 0 && end > g.lo[st]) ? (end - g.lo[st] + kTile - 1) / kTile : 0;
                g.n[st] = g.cnt[st];
                g.n_max = g.cnt[st] > g.n_max ? g.cnt[st] : g.n_max;
            }
        }
        sh->g = g;
    }
    __syncthreads();
    if (!sh->g.found) return;
    const int n_max = sh->g.n_max;

    if (tid == 0) {
        mbar_init(smem_u32(&sh->bar_q), 1);
        for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&sh->kv_full[s]), 1); mbar_init(smem_u32(&sh->kv_empty[s]), 1); }
        for (int st = 0; st < 2; ++st) {
            mbar_init(smem_u32(&sh->s_full[st]), 1);
            mbar_init(smem_u32(&sh->p_ready[st]), 4);         // one arrival per softmax warp
            mbar_init(smem_u32(&sh->o_final[st]), 1);
        }
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

    // Warps 8-11 (the whole third warpgroup) give registers up, warps 0-7 take them.
    if (warp == kLoadWarp) {
        // ------------------------------------------------------------------ TMA loader
        reg_dealloc<kLightRegs>();
        if (lane == 0 && n_max > 0) {
            const uint32_t bar_q = smem_u32(&sh->bar_q);
            mbar_arrive_expect_tx(bar_q, 2 * kTileBytes);
#pragma unroll
            for (int st = 0; st < 2; ++st) {
                const int row = sh->g.q_row0;                  // both stages hold the same rows
                tma_load_3d(sQ + st * kTileBytes, &tm_q, bar_q, 0, h, row);
                tma_load_3d(sQ + st * kTileBytes + kHalfTileBytes, &tm_q, bar_q, 64, h, row);
            }
            int filled = 0;                                    // ring items issued so far
            auto load_tile = [&](const void *map, int krow) {
                const int slot = filled % kStages, fill = filled / kStages;
                if (fill > 0 && !wait_bar(smem_u32(&sh->kv_empty[slot]), (fill - 1) & 1, sh, p)) return false;
                const uint32_t dst = sRing + slot * kTileBytes, bar = smem_u32(&sh->kv_full[slot]);
                mbar_arrive_expect_tx(bar, kTileBytes);
                tma_load_3d(dst, map, bar, 0, kvh, krow);
                tma_load_3d(dst + kHalfTileBytes, map, bar, 64, kvh, krow);
                ++filled;
                return true;
            };
            bool ok = true;
            {
                // Each stage has its own key slice; items in the order the MMA issuer consumes them:
                // K_0(0), K_1(0), then per step V_0(j), K_0(j+1), V_1(j), K_1(j+1).
                const int n0 = sh->g.n[0], n1 = sh->g.n[1];
                const int base0 = sh->g.kv_row0 + sh->g.lo[0], base1 = sh->g.kv_row0 + sh->g.lo[1];
                if (n0 > 0) ok = load_tile(&tm_k, base0);
                if (ok && n1 > 0) ok = load_tile(&tm_k, base1);
                for (int j = 0; j < n_max && ok; ++j) {
                    if (ok && j < n0) ok = load_tile(&tm_v, base0 + j * kTile);
                    if (ok && j + 1 < n0) ok = load_tile(&tm_k, base0 + (j + 1) * kTile);
                    if (ok && j < n1) ok = load_tile(&tm_v, base1 + j * kTile);
                    if (ok && j + 1 < n1) ok = load_tile(&tm_k, base1 + (j + 1) * kTile);
                }
            }
        }
        __syncwarp();
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------------ MMA issuer
        reg_dealloc<kLightRegs>();
        if (lane == 0 && n_max > 0) {
            constexpr uint32_t idesc_qk = idesc_bf16_f32(kTile, kTile, 0, 0);
            constexpr uint32_t idesc_pv = idesc_bf16_f32(kTile, kHeadDim, 0, 1);
            auto kv_wait = [&](int item) {
                return wait_bar(smem_u32(&sh->kv_full[item % kStages]), (item / kStages) & 1, sh, p);
            };
            auto kv_release = [&](int item) { tc_commit(smem_u32(&sh->kv_empty[item % kStages])); };
            // S_st = Q_st K^T: both operands K-major; 8 steps of 16 channels, 4 per 64-channel half tile
            auto issue_qk = [&](int st, int item) {
                const uint32_t a = sQ + st * kTileBytes, b = sRing + (item % kStages) * kTileBytes;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks) {
                    const uint32_t off = (uint32_t)(ks >> 2) * kHalfTileBytes + (uint32_t)(ks & 3) * 32u;
                    mma_ss(tmem + kColS + st * kTile, smem_desc_sw128(a + off, 16, 1024), smem_desc_sw128(b + off, 16, 1024),
                           idesc_qk, ks > 0 ? 1u : 0u);
                }
                tc_commit(smem_u32(&sh->s_full[st]));
            };
            // O_st (+)= P_st V: A = P from TMEM (8 columns per 16 keys), B = V tile stored [key][channel]
            // (N-contiguous): 16 keys = 2048 bytes per step, channel halves 16 KiB apart.
            auto issue_pv = [&](int st, int item, bool accumulate) {
                const uint32_t b = sRing + (item % kStages) * kTileBytes;
#pragma unroll
                for (int ks = 0; ks < 8; ++ks)
                    mma_ts(tmem + kColO + st * kTile, tmem + kColS + st * kTile + ks * 8,
                           smem_desc_sw128(b + ks * 2048u, kHalfTileBytes, 1024), idesc_pv, (accumulate || ks > 0) ? 1u : 0u);
            };

            const int n_st[2] = {sh->g.n[0], sh->g.n[1]};
            bool ok = wait_bar(smem_u32(&sh->bar_q), 0, sh, p);
            if (ok) {
                // Every ring item has one consumer; items arrive in the order used here.
                int item = 0;
#pragma unroll
                for (int st = 0; st < 2 && ok; ++st) {
                    if (n_st[st] > 0) {
                        ok = kv_wait(item);
                        if (ok) { issue_qk(st, item); kv_release(item); ++item; }
                    }
                }
                for (int j = 0; j < n_max && ok; ++j) {
#pragma unroll
                    for (int st = 0; st < 2 && ok; ++st) {
                        if (j < n_st[st]) {
                            ok = wait_bar(smem_u32(&sh->p_ready[st]), j & 1, sh, p) && kv_wait(item);   // P_st(j), V_st(j)
                            if (!ok) break;
                            tc_fence_after();
                            issue_pv(st, item, j > 0);
                            if (j == n_st[st] - 1) tc_commit(smem_u32(&sh->o_final[st]));
                            kv_release(item);
                            ++item;
                        }
                        if (j + 1 < n_st[st]) {
                            ok = kv_wait(item);                // K_st(j+1)
                            if (!ok) break;
                            issue_qk(st, item);
                            kv_release(item);
                            ++item;
                        }
                    }
                }
            }
        }
        __syncwarp();
    } else if (warp >= kSoftmaxWarps) {
        reg_dealloc<kLightRegs>();
    } else {
        // ------------------------------------------------------------------ softmax + epilogue
        reg_alloc<kSoftmaxRegs>();
        const int st = warp >> 2, quarter = warp & 3;
        const int row_in_tile = quarter * 32 + lane;
        const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
        const uint32_t tS = tmem + lane_base + kColS + st * kTile;
        const uint32_t tO = tmem + lane_base + kColO + st * kTile;
        const int n_mine = sh->g.n[st];
        const uint32_t bar_s = smem_u32(&sh->s_full[st]), bar_p = smem_u32(&sh->p_ready[st]);
        // Where the stage's slice ends, and the first key position that some row of this stage cannot
        // see (tiles reaching past it need the mask).
        const int pos0 = sh->g.pos0[st], my_pos = pos0 + row_in_tile;
        const int hi_st = sh->g.hi[st];
        const int iv_full = (p.causal && pos0 + 1 < hi_st) ? pos0 + 1 : hi_st;
        const int iv_mine = (p.causal && my_pos + 1 < hi_st) ? my_pos + 1 : hi_st;
        int k0 = sh->g.lo[st];

        float m_ref = -INFINITY, l_run = 0.f;                // m_ref in log2 units of the scaled scores
        bool ok = true;
        for (int j = 0; j < n_mine; ++j, k0 += kTile) {
            ok = __all_sync(0xffffffffu, wait_bar(bar_s, j & 1, sh, p));     // warp-uniform
            if (!ok) break;
            tc_fence_after();

            uint32_t r[kTile];
            tmem_ld128(tS, r);
            // Mask only when some row of this stage cannot see the whole tile.
            const bool masked = k0 + kTile > iv_full;
            if (masked) {
                int n_vis = iv_mine - k0;
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
            if (j > 0 && __any_sync(0xffffffffu, grow)) {
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
            // half) and 2c+1 (high half).
#pragma unroll
            for (int i = 0; i < kTile / 2; ++i) {
                const float2 x = __ffma2_rn(make_float2(__uint_as_float(r[2 * i]), __uint_as_float(r[2 * i + 1])), sc2, nm2);
                const float2 e = make_float2(ex2(x.x), ex2(x.y));
                sum[i & 3] = __fadd2_rn(sum[i & 3], e);
                r[i] = pack_bf16(e.x, e.y);
            }
            const float2 s01 = __fadd2_rn(__fadd2_rn(sum[0], sum[1]), __fadd2_rn(sum[2], sum[3]));
            l_run += s01.x + s01.y;
            tmem_st32(tS, r);
            tmem_st32(tS + 32, r + 32);
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_p);
        }

        // Epilogue: O / l and LSE = ln2 * m + ln l; rows without any visible key give 0 and -inf.
        if (ok && n_mine > 0) ok = __all_sync(0xffffffffu, wait_bar(smem_u32(&sh->o_final[st]), 0, sh, p));
        if (ok && sh->g.rows[st] > 0) {
            tc_fence_after();
            const bool valid = row_in_tile < sh->g.rows[st];
            const bool empty = (l_run == 0.f);
            const float inv = empty ? 0.f : 1.f / l_run;
            const int64_t row = (int64_t)sh->g.out_row0 + st * sh->g.out_st_stride + row_in_tile;
            const int64_t obase = (row * p.Hq + h) * kHeadDim;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t r[32];
                if (n_mine == 0) {
#pragma unroll
                    for (int i = 0; i < 32; ++i) r[i] = 0u;
                } else {
                    tmem_ld32(tO + c * 32, r);                // warp-wide; only the stores are predicated
                }
                if (!valid) continue;
                if (p.o_is_bf16) {
                    __nv_bfloat16 *o = static_cast<__nv_bfloat16 *>(p.o) + obase + c * 32;
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        uint4 pk;
                        pk.x = pack_bf16(__uint_as_float(r[i + 0]) * inv, __uint_as_float(r[i + 1]) * inv);
                        pk.y = pack_bf16(__uint_as_float(r[i + 2]) * inv, __uint_as_float(r[i + 3]) * inv);
                        pk.z = pack_bf16(__uint_as_float(r[i + 4]) * inv, __uint_as_float(r[i + 5]) * inv);
                        pk.w = pack_bf16(__uint_as_float(r[i + 6]) * inv, __uint_as_float(r[i + 7]) * inv);
                        *reinterpret_cast<uint4 *>(o + i) = pk;
                    }
                } else {
                    float *o = static_cast<float *>(p.o) + obase + c * 32;
#pragma unroll
                    for (int i = 0; i < 32; i += 4)
                        *reinterpret_cast<float4 *>(o + i) = make_float4(__uint_as_float(r[i]) * inv, __uint_as_float(r[i + 1]) * inv,
                                                                         __uint_as_float(r[i + 2]) * inv, __uint_as_float(r[i + 3]) * inv);
                }
            }
            if (valid) p.lse[row * p.Hq + h] = empty ? -INFINITY : m_ref * 0.6931471805599453f + logf(l_run);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, kTmemCols);
}

// ------------------------------------------------------------------------------------------ host
}  // namespace splitk

int launch_attn_split_bf16(const AttnParams &p, cudaStream_t stream)
{
    using namespace splitk;
    if (!p.status) { set_error("pec_decode_attn: the bf16 path needs a status word"); return PEC_ERR_INVALID_ARG; }
    // Rows the maps may touch: queries up to the chunk end, keys up to the end of the visible subset.
    if (p.cu_seqlens) { set_error("pec_decode_attn: packed batches are not split"); return PEC_ERR_INVALID_ARG; }
    const int64_t q_rows = p.q_hi[0];
    int64_t kv_rows = 0;
    for (int t = 0; t < p.n_iv; ++t) kv_rows = p.iv_hi[t] > kv_rows ? p.iv_hi[t] : kv_rows;
    if (q_rows >= ((int64_t)1 << 31) || kv_rows >= ((int64_t)1 << 31)) {
        set_error("pec_decode_attn: more than 2^31 rows unsupported");
        return PEC_ERR_UNSUPPORTED;
    }
    CUtensorMap tm_q, tm_k, tm_v;
    if (!host::make_qkv_map(&tm_q, p.q, q_rows, p.Hq, p.q_stride_t, p.q_stride_h) ||
        !host::make_qkv_map(&tm_k, p.k, kv_rows, p.Hkv, p.k_stride_t, p.k_stride_h) ||
        !host::make_qkv_map(&tm_v, p.v, kv_rows, p.Hkv, p.v_stride_t, p.v_stride_h)) {
        set_error("pec_decode_attn: cuTensorMapEncodeTiled failed (driver too old, or strides/addresses not encodable)");
        return PEC_ERR_CUDA;
    }
    // Once per device: raise the shared-memory limit, and check that the launch allocation (registers per
    // thread x threads) covers the split in which the softmax warpgroups take registers the third gives up.
    static unsigned char ready[host::kMaxDevices] = {};
    static std::mutex ready_mutex;
    const bool ok = host::once_per_device(ready, ready_mutex, [] {
        if (cudaFuncSetAttribute(attn_split_bf16_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes) != cudaSuccess) return false;
        cudaFuncAttributes attr;
        return cudaFuncGetAttributes(&attr, attn_split_bf16_kernel) == cudaSuccess &&
               attr.numRegs * kThreads >= kSoftmaxWarps * 32 * kSoftmaxRegs + (kThreads - kSoftmaxWarps * 32) * kLightRegs;
    });
    if (!ok) {
        (void)cudaGetLastError();
        set_error("pec_decode_attn: kernel set-up failed (shared-memory limit, or the register allocation does not cover the warp-role split)");
        return PEC_ERR_CUDA;
    }
    const int64_t tiles = (p.total_rows + kBlockM - 1) / kBlockM;
    if (tiles > 0x7fffffff || p.Hq > 65535) { set_error("pec_decode_attn: grid too large"); return PEC_ERR_UNSUPPORTED; }
    if (p.splits < 1 || p.splits > 65535) { set_error("pec_decode_attn: bad split count"); return PEC_ERR_INVALID_ARG; }
    if (p.total_rows > kTile) { set_error("pec_decode_attn: split launches take at most 128 query rows"); return PEC_ERR_UNSUPPORTED; }
    // Each CTA's two stages take two consecutive key slices.
    dim3 grid((unsigned)tiles, (unsigned)p.Hq, (unsigned)((p.splits + 1) / 2));
    attn_split_bf16_kernel<<<grid, kThreads, kSmemBytes, stream>>>(tm_q, tm_k, tm_v, p);
    const cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) { set_error("pec_decode_attn: launch failed: %s", cudaGetErrorString(err)); return PEC_ERR_CUDA; }
    return PEC_OK;
}

}  // namespace pec
