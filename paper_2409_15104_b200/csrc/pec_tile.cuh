// Device-side mapping from a linear tile index to the rows and key intervals it covers.
#pragma once
#include "pec_internal.h"

namespace pec {

struct TileJob {
    int64_t q_row0;      // first row of the tile in q
    int64_t out_row0;    // first row of the tile in o / lse
    int64_t q_pos0;      // position of that row in its request
    int32_t n_rows;      // valid rows in the tile
    int64_t kv_row0;     // row of key position 0 in k / v
    int64_t iv_lo[2], iv_hi[2];   // visible-key intervals (positions), before the causal cut
    int32_t n_iv;
};

__device__ __forceinline__ void packed_job(int64_t req_start, int64_t pos0, int64_t req_len, int block_m, TileJob &job)
{
    job.q_row0 = req_start + pos0;
    job.out_row0 = req_start + pos0;
    job.q_pos0 = pos0;
    job.n_rows = (int32_t)((req_len - pos0) < block_m ? (req_len - pos0) : block_m);
    job.kv_row0 = req_start;
    job.n_iv = 1;
    job.iv_lo[0] = 0; job.iv_hi[0] = req_len;
    job.iv_lo[1] = 0; job.iv_hi[1] = 0;
}

// Returns false when `tile` is past the last tile.  A single request's tiles run through its query
// segments in ascending position, each segment starting a fresh tile.  Packed batches either read
// entry `tile` of the work-list or walk cu_seqlens: request b contributes ceil(len_b / block_m)
// tiles, each request starting a fresh tile.
__device__ __forceinline__ bool locate_tile(const AttnParams &p, int64_t tile, int block_m, TileJob &job)
{
    if (p.cu_seqlens == nullptr) {
        int64_t t = tile;
#pragma unroll
        for (int s = 0; s < 2; ++s) {
            if (s >= p.n_qseg) break;
            const int64_t len = p.q_hi[s] - p.q_lo[s];
            const int64_t nt = (len + block_m - 1) / block_m;
            if (t < nt) {
                const int64_t r0 = p.q_lo[s] + t * block_m;
                job.q_row0 = r0;
                job.out_row0 = r0 - p.out_pos0;
                job.q_pos0 = r0;
                job.n_rows = (int32_t)((p.q_hi[s] - r0) < block_m ? (p.q_hi[s] - r0) : block_m);
                job.kv_row0 = 0;
                job.n_iv = p.n_iv;
                job.iv_lo[0] = p.iv_lo[0]; job.iv_hi[0] = p.iv_hi[0];
                job.iv_lo[1] = p.iv_lo[1]; job.iv_hi[1] = p.iv_hi[1];
                return true;
            }
            t -= nt;
        }
        return false;
    }
    if (p.worklist != nullptr) {
        if (tile >= p.n_items) return false;
        const int4 it = reinterpret_cast<const int4 *>(p.worklist)[tile];
        packed_job(it.x, it.y, it.w, block_m, job);
        return true;
    }
    int64_t t = tile;
    for (int b = 0; b < p.B; ++b) {
        const int64_t s = p.cu_seqlens[b], e = p.cu_seqlens[b + 1];
        const int64_t nt = (e - s + block_m - 1) / block_m;
        if (t < nt) {
            packed_job(s, t * block_m, e - s, block_m, job);
            return true;
        }
        t -= nt;
    }
    return false;
}

// The same search done by a whole converged warp: for a packed batch without a work-list each lane
// takes every 32nd request (the two table reads of all requests are in flight together instead of
// one dependent pair per request), tile counts are prefix-summed with shuffles, and the lane that
// owns the tile's request broadcasts it.  Every lane returns the same job.
__device__ __forceinline__ bool locate_tile_warp(const AttnParams &p, int64_t tile, int block_m, TileJob &job)
{
    if (p.cu_seqlens == nullptr || p.worklist != nullptr) return locate_tile(p, tile, block_m, job);
    const int lane = threadIdx.x & 31;
    int64_t before = 0;                                   // tiles of the requests in earlier groups of 32
    for (int b0 = 0; b0 < p.B; b0 += 32) {
        const int b = b0 + lane;
        int64_t s = 0, e = 0;
        if (b < p.B) { s = p.cu_seqlens[b]; e = p.cu_seqlens[b + 1]; }
        const int64_t nt = (e - s + block_m - 1) / block_m;
        int64_t incl = nt;                                // inclusive prefix sum over the lanes
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int64_t up = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += up;
        }
        const bool mine = b < p.B && tile >= before + incl - nt && tile < before + incl;
        const unsigned who = __ballot_sync(0xffffffffu, mine);
        if (who) {
            const int src = __ffs(who) - 1;
            const int64_t s_b = __shfl_sync(0xffffffffu, s, src), e_b = __shfl_sync(0xffffffffu, e, src);
            const int64_t first = __shfl_sync(0xffffffffu, before + incl - nt, src);
            packed_job(s_b, (tile - first) * block_m, e_b - s_b, block_m, job);
            return true;
        }
        before += __shfl_sync(0xffffffffu, incl, 31);
    }
    return false;
}

}  // namespace pec
