// Host planner: zigzag sequence partitions, preemptible chunks, causal tile classes.
// Integer arithmetic only; the rule is stated in pec.h.  The paper asks for segments handled
// by different replicas (Section 2.2) and for prefills that pause between kernels
// (Section 5.1); pairing block p with block 2P-1-p equalises the causal work per partition.
#include <algorithm>
#include <vector>
#include "pec_internal.h"

namespace pec {

static inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }

static inline int64_t bound_at(int64_t k, int64_t units, int64_t two_p, int64_t align, int64_t seq_len)
{
    // k <= 2P and units <= 2^63 / (2P) for any realistic length: the product fits in int64.
    const int64_t b = align * ((k * units) / two_p);
    return b < seq_len ? b : seq_len;
}

void zigzag_intervals(int64_t seq_len, int32_t num_parts, int32_t part_id, int32_t align,
                      int64_t lo[2], int64_t hi[2])
{
    const int64_t two_p = 2 * (int64_t)num_parts;
    const int64_t units = ceil_div(seq_len, align);
    const int64_t a = part_id, b = two_p - 1 - part_id;
    lo[0] = bound_at(a, units, two_p, align, seq_len);
    hi[0] = bound_at(a + 1, units, two_p, align, seq_len);
    lo[1] = bound_at(b, units, two_p, align, seq_len);
    hi[1] = bound_at(b + 1, units, two_p, align, seq_len);
}

}  // namespace pec

using namespace pec;

extern "C" int pec_plan_partitions(int64_t seq_len, int32_t num_parts, int64_t chunk_len, int32_t align,
                                   int32_t block_m, int32_t block_n, int32_t causal, pec_plan *plan)
{
    if (!plan) { set_error("pec_plan_partitions: plan is NULL"); return PEC_ERR_INVALID_ARG; }
    if (seq_len < 0 || num_parts < 1 || align < 1 || block_m < 1 || block_n < 1) {
        set_error("pec_plan_partitions: need seq_len >= 0, num_parts >= 1, align >= 1, block_m/n >= 1");
        return PEC_ERR_INVALID_ARG;
    }
    const int64_t P = num_parts, two_p = 2 * P;
    const int64_t units = ceil_div(seq_len, align);
    const int64_t C = chunk_len > 0 ? chunk_len : (seq_len > 0 ? seq_len : 1);
    plan->n_bounds = two_p + 1;
    plan->n_parts = P;
    plan->n_chunks = ceil_div(seq_len, C);
    plan->nq_tiles = ceil_div(seq_len, block_m);
    plan->nk_tiles = ceil_div(seq_len, block_n);

    if ((plan->bounds && plan->bounds_cap < plan->n_bounds) ||
        ((plan->part_lo || plan->part_hi) && plan->part_cap < two_p) ||
        (plan->pairs && plan->pairs_cap < P) ||
        ((plan->chunk_start || plan->chunk_len) && plan->chunk_cap < plan->n_chunks) ||
        (plan->tile_class && plan->tile_cap < plan->nq_tiles * plan->nk_tiles)) {
        set_error("pec_plan_partitions: a caller array is smaller than the count it must hold");
        return PEC_ERR_CAPACITY;
    }

    if (plan->bounds)
        for (int64_t k = 0; k <= two_p; ++k) plan->bounds[k] = bound_at(k, units, two_p, align, seq_len);

    for (int64_t p = 0; p < P; ++p) {
        int64_t lo[2], hi[2];
        zigzag_intervals(seq_len, num_parts, (int32_t)p, align, lo, hi);
        if (plan->part_lo) { plan->part_lo[2 * p] = lo[0]; plan->part_lo[2 * p + 1] = lo[1]; }
        if (plan->part_hi) { plan->part_hi[2 * p] = hi[0]; plan->part_hi[2 * p + 1] = hi[1]; }
        if (plan->pairs) {
            // sum_{j=lo}^{hi-1} (S - j) = n*S - (lo + hi - 1)*n/2, kept exact in 128-bit.
            __int128 total = 0;
            for (int t = 0; t < 2; ++t) {
                const __int128 n = hi[t] - lo[t];
                if (n <= 0) continue;
                if (causal) total += n * seq_len - ((__int128)(lo[t] + hi[t] - 1) * n) / 2;
                else        total += n * seq_len;
            }
            plan->pairs[p] = (int64_t)total;
        }
    }

    for (int64_t c = 0; c < plan->n_chunks; ++c) {
        const int64_t s = c * C;
        const int64_t e = (s + C < seq_len) ? s + C : seq_len;
        if (plan->chunk_start) plan->chunk_start[c] = s;
        if (plan->chunk_len) plan->chunk_len[c] = e - s;
    }

    if (plan->tile_class) {
        for (int64_t a = 0; a < plan->nq_tiles; ++a) {
            const int64_t q0 = a * block_m;
            const int64_t q1 = (q0 + block_m < seq_len) ? q0 + block_m : seq_len;   // exclusive
            uint8_t *row = plan->tile_class + a * plan->nk_tiles;
            for (int64_t b = 0; b < plan->nk_tiles; ++b) {
                const int64_t k0 = b * block_n;
                const int64_t k1 = (k0 + block_n < seq_len) ? k0 + block_n : seq_len;
                uint8_t cls = PEC_TILE_FULL;
                if (causal) {
                    if (k0 > q1 - 1) cls = PEC_TILE_SKIP;
                    else if (k1 - 1 <= q0) cls = PEC_TILE_FULL;
                    else cls = PEC_TILE_PARTIAL;
                }
                row[b] = cls;
            }
        }
    }
    return PEC_OK;
}

extern "C" int pec_plan_worklist(const int32_t *cu_seqlens, int32_t B, int32_t block_m, int32_t block_n, int32_t causal,
                                 int32_t *items, int64_t items_cap, int64_t *n_items)
{
    if (!cu_seqlens || !n_items || B < 0 || block_m < 1 || block_n < 1) {
        set_error("pec_plan_worklist: need cu_seqlens, n_items, B >= 0 and block sizes >= 1");
        return PEC_ERR_INVALID_ARG;
    }
    int64_t total = 0;
    for (int32_t b = 0; b < B; ++b) {
        if (cu_seqlens[b + 1] < cu_seqlens[b]) { set_error("pec_plan_worklist: cu_seqlens decreases at request %d", (int)b); return PEC_ERR_INVALID_ARG; }
        total += ceil_div((int64_t)cu_seqlens[b + 1] - cu_seqlens[b], block_m);
    }
    *n_items = total;
    if (!items) return PEC_OK;
    if (items_cap < total) { set_error("pec_plan_worklist: items holds %lld entries, %lld needed", (long long)items_cap, (long long)total); return PEC_ERR_CAPACITY; }
    struct Entry { int64_t weight; int32_t start, pos0, rows, len; };
    std::vector<Entry> list;
    list.reserve((size_t)total);
    for (int32_t b = 0; b < B; ++b) {
        const int64_t len = (int64_t)cu_seqlens[b + 1] - cu_seqlens[b];
        for (int64_t pos0 = 0; pos0 < len; pos0 += block_m) {
            const int64_t rows = len - pos0 < block_m ? len - pos0 : block_m;
            const int64_t keys = causal ? pos0 + rows : len;      // the tile's last row sees keys [0, pos0 + rows)
            list.push_back({ceil_div(keys, block_n), cu_seqlens[b], (int32_t)pos0, (int32_t)rows, (int32_t)len});
        }
    }
    // Entries were generated by request, then by position: a stable sort keeps that order among equal weights.
    std::stable_sort(list.begin(), list.end(), [](const Entry &x, const Entry &y) { return x.weight > y.weight; });
    for (size_t i = 0; i < list.size(); ++i) {
        items[4 * i + 0] = list[i].start; items[4 * i + 1] = list[i].pos0;
        items[4 * i + 2] = list[i].rows;  items[4 * i + 3] = list[i].len;
    }
    return PEC_OK;
}

// Visible (query, key) pairs between query rows [a, b) and keys [c, d): a key j counts for row i
// when j <= i (causal) or always.  Rows below the first key see nothing, rows i in [c, d-1) see
// i + 1 - c keys (an arithmetic series), rows from d - 1 on see all d - c.
static __int128 interval_pairs(int64_t a, int64_t b, int64_t c, int64_t d, bool causal)
{
    if (b <= a || d <= c) return 0;
    const __int128 n = d - c;
    if (!causal) return (__int128)(b - a) * n;
    __int128 total = 0;
    const int64_t lo1 = a > c ? a : c, hi1 = b < d - 1 ? b : d - 1;
    if (hi1 > lo1) {
        const __int128 m = hi1 - lo1;
        total += m * (lo1 + 1 - c) + m * (m - 1) / 2;
    }
    const int64_t lo2 = a > d - 1 ? a : d - 1;
    if (b > lo2) total += (__int128)(b - lo2) * n;
    return total;
}

// The (up to two) row intervals of ring rank r under a layout.
static int rank_intervals(int64_t seq_len, int32_t num_parts, int32_t r, int32_t align, int32_t layout,
                          int64_t lo[2], int64_t hi[2])
{
    if (layout == PEC_LAYOUT_ZIGZAG) { zigzag_intervals(seq_len, num_parts, r, align, lo, hi); return 2; }
    const int64_t units = ceil_div(seq_len, align);
    lo[0] = bound_at(r, units, num_parts, align, seq_len);
    hi[0] = bound_at((int64_t)r + 1, units, num_parts, align, seq_len);
    lo[1] = hi[1] = 0;
    return 1;
}

extern "C" int pec_plan_ring(int64_t seq_len, int32_t num_parts, int32_t align, int32_t layout, int32_t causal,
                             int64_t *pairs, int64_t pairs_cap, int64_t *step_max, int64_t *rank_total, int64_t vec_cap)
{
    if (seq_len < 0 || num_parts < 1 || align < 1 || (layout != PEC_LAYOUT_ZIGZAG && layout != PEC_LAYOUT_CONTIGUOUS)) {
        set_error("pec_plan_ring: need seq_len >= 0, num_parts >= 1, align >= 1 and a known layout");
        return PEC_ERR_INVALID_ARG;
    }
    const int64_t P = num_parts;
    if ((pairs && pairs_cap < P * P) || ((step_max || rank_total) && vec_cap < P)) {
        set_error("pec_plan_ring: a caller array is smaller than the count it must hold");
        return PEC_ERR_CAPACITY;
    }
    for (int64_t t = 0; t < P; ++t) {
        if (step_max) step_max[t] = 0;
        if (rank_total) rank_total[t] = 0;
    }
    for (int32_t r = 0; r < num_parts; ++r) {
        int64_t qlo[2], qhi[2];
        const int nq = rank_intervals(seq_len, num_parts, r, align, layout, qlo, qhi);
        for (int32_t t = 0; t < num_parts; ++t) {
            const int32_t src = (int32_t)(((int64_t)r - t + P) % P);
            int64_t klo[2], khi[2];
            const int nk = rank_intervals(seq_len, num_parts, src, align, layout, klo, khi);
            __int128 total = 0;
            for (int a = 0; a < nq; ++a)
                for (int b = 0; b < nk; ++b) total += interval_pairs(qlo[a], qhi[a], klo[b], khi[b], causal != 0);
            const int64_t v = (int64_t)total;
            if (pairs) pairs[(int64_t)r * P + t] = v;
            if (step_max && v > step_max[t]) step_max[t] = v;
            if (rank_total) rank_total[r] += v;
        }
    }
    return PEC_OK;
}

extern "C" int pec_balance_batches(const int32_t *lengths, int32_t n, int32_t replicas, int32_t *assign, int64_t *tokens)
{
    if (n < 0 || replicas < 1 || (n > 0 && (!lengths || !assign))) {
        set_error("pec_balance_batches: need n >= 0, replicas >= 1 and non-NULL lengths/assign");
        return PEC_ERR_INVALID_ARG;
    }
    for (int32_t i = 0; i < n; ++i)
        if (lengths[i] < 0) { set_error("pec_balance_batches: request %d has a negative length", (int)i); return PEC_ERR_INVALID_ARG; }
    std::vector<int32_t> order((size_t)n);
    for (int32_t i = 0; i < n; ++i) order[(size_t)i] = i;
    std::stable_sort(order.begin(), order.end(), [&](int32_t x, int32_t y) { return lengths[x] > lengths[y]; });
    std::vector<int64_t> load((size_t)replicas, 0);
    for (int32_t i : order) {
        int32_t best = 0;
        for (int32_t rep = 1; rep < replicas; ++rep)
            if (load[(size_t)rep] < load[(size_t)best]) best = rep;
        assign[i] = best;
        load[(size_t)best] += lengths[i];
    }
    if (tokens) for (int32_t rep = 0; rep < replicas; ++rep) tokens[rep] = load[(size_t)rep];
    return PEC_OK;
}

// Section 5.3's closed forms for the hybrid SP strategy choice (host arithmetic only).
extern "C" int pec_select_sp(const pec_sp_inputs *in, pec_sp_choice *out)
{
    if (!in || !out) { set_error("pec_select_sp: NULL argument"); return PEC_ERR_INVALID_ARG; }
    const double s = in->s, d = in->d, nh = in->n_h, nkv = in->n_kv, dh = in->d_h, T = in->T, G = in->G;
    if (!(s > 0 && d > 0 && nh > 0 && nkv > 0 && dh > 0 && T >= 1 && G >= 1 && in->elem_bytes > 0 && in->node_bw > 0 && in->gpu_flops > 0)) {
        set_error("pec_select_sp: sizes and rates must be positive, T and G at least 1");
        return PEC_ERR_INVALID_ARG;
    }
    const double heads = (nh + nkv) * dh;
    out->comm[0][0] = 2 * s * d * (T - 1) * G;
    out->comp[0][0] = 2 * s * d * heads / T + 4 * (s * T) * (s * T) * d / T + 2 * s * d * d;
    out->comm[0][1] = 2 * s * heads * (G - 1) + (d * heads + d * d) * G * (T - 1) / T;
    out->comp[0][1] = 2 * s * d * heads + 4 * (s * G) * (s * G) * d / G + 2 * s * d * d;
    out->comm[1][0] = 2 * s * d * (T - 1) * G;
    out->comp[1][0] = 16 * s * d * d;
    out->comm[1][1] = 8 * d * d * (T - 1) * G / T;
    out->comp[1][1] = 16 * s * d * d;
    int best = 0;
    for (int a = 0; a < 2; ++a)
        for (int m = 0; m < 2; ++m) {
            const double t = (out->comm[0][a] + out->comm[1][m]) * in->elem_bytes / in->node_bw +
                             (out->comp[0][a] + out->comp[1][m]) / in->gpu_flops;
            out->seconds[2 * a + m] = t;
            if (t < out->seconds[best]) best = 2 * a + m;
        }
    out->attn_strategy = best >> 1;
    out->mlp_strategy = best & 1;
    return PEC_OK;
}
