// C-ABI entry points: argument checks, resolution of the key subset, kernel dispatch.
#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <climits>
#include "pec_internal.h"

namespace pec {

static thread_local char g_last_error[512] = "";

void set_error(const char *fmt, ...)
{
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_last_error, sizeof(g_last_error), fmt, ap);
    va_end(ap);
}

static std::atomic<int64_t> g_wait_limit_cycles{2000000000LL};   // about a second of SM clock
static std::atomic<int32_t> g_test_skip_last_load{0};
int64_t wait_limit_cycles() { return g_wait_limit_cycles.load(std::memory_order_relaxed); }
int32_t test_skip_last_load() { return g_test_skip_last_load.load(std::memory_order_relaxed); }

constexpr int32_t kBlockMBf16 = 256, kBlockMF32 = 64;   // query rows per CTA of the two attention kernels

static inline bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Checks the arguments and fills the launch description.  Returns a pec_status.
static int resolve(const pec_attn_args *a, AttnParams &p)
{
    if (!a) { set_error("pec_prefill_attn: args is NULL"); return PEC_ERR_INVALID_ARG; }
    if (!a->q || !a->k || !a->v || !a->o || !a->lse) {
        set_error("pec_prefill_attn: q, k, v, o and lse must be non-NULL");
        return PEC_ERR_INVALID_ARG;
    }
    if (a->D != kHeadDim) { set_error("pec_prefill_attn: D=%d unsupported (only 128)", a->D); return PEC_ERR_UNSUPPORTED; }
    if (a->Hq < 1 || a->Hkv < 1 || a->Hq % a->Hkv != 0) {
        set_error("pec_prefill_attn: need Hq >= 1, Hkv >= 1 and Hkv | Hq (got %d, %d)", a->Hq, a->Hkv);
        return PEC_ERR_INVALID_ARG;
    }
    if (a->in_dtype != PEC_BF16 && a->in_dtype != PEC_F32) { set_error("pec_prefill_attn: unknown in_dtype %d", a->in_dtype); return PEC_ERR_UNSUPPORTED; }
    if (a->o_dtype != PEC_BF16 && a->o_dtype != PEC_F32) { set_error("pec_prefill_attn: unknown o_dtype %d", a->o_dtype); return PEC_ERR_UNSUPPORTED; }
    if (a->in_dtype == PEC_F32 && a->o_dtype != PEC_F32) {
        set_error("pec_prefill_attn: fp32 inputs produce fp32 output only");
        return PEC_ERR_UNSUPPORTED;
    }
    if (a->causal != 0 && a->causal != 1) { set_error("pec_prefill_attn: causal must be 0 or 1"); return PEC_ERR_INVALID_ARG; }
    if (a->seq_len < 0 || a->chunk_start < 0 || a->chunk_len < 0 || a->kv_len < 0) {
        set_error("pec_prefill_attn: negative length");
        return PEC_ERR_INVALID_ARG;
    }
    if (a->seq_len > (int64_t)1 << 30) { set_error("pec_prefill_attn: seq_len above 2^30 unsupported"); return PEC_ERR_UNSUPPORTED; }
    if (a->chunk_start + a->chunk_len > a->seq_len || a->kv_len > a->seq_len) {
        set_error("pec_prefill_attn: chunk [%lld,+%lld) or kv_len %lld exceeds seq_len %lld",
                  (long long)a->chunk_start, (long long)a->chunk_len, (long long)a->kv_len, (long long)a->seq_len);
        return PEC_ERR_INVALID_ARG;
    }
    if (a->causal && a->kv_len < a->chunk_start + a->chunk_len) {
        set_error("pec_prefill_attn: causal chunk ending at %lld needs kv_len >= that (got %lld)",
                  (long long)(a->chunk_start + a->chunk_len), (long long)a->kv_len);
        return PEC_ERR_INVALID_ARG;
    }
    if (a->num_parts < 1 || a->part_id < 0 || a->part_id >= a->num_parts || a->part_align < 1) {
        set_error("pec_prefill_attn: need 0 <= part_id < num_parts and part_align >= 1");
        return PEC_ERR_INVALID_ARG;
    }
    if (!(a->softmax_scale >= 0.f) || std::isinf(a->softmax_scale)) { set_error("pec_prefill_attn: softmax_scale must be finite and >= 0"); return PEC_ERR_INVALID_ARG; }
    if ((a->acc_o == nullptr) != (a->acc_lse == nullptr)) { set_error("pec_prefill_attn: acc_o and acc_lse go together"); return PEC_ERR_INVALID_ARG; }
    if (a->acc_o) {
        const bool alias_o = static_cast<const void *>(a->acc_o) == a->o, alias_l = a->acc_lse == a->lse;
        if (alias_o != alias_l || (alias_o && a->o_dtype != PEC_F32)) {
            set_error("pec_prefill_attn: o / lse may be the incoming state's buffers only both at once and with fp32 output");
            return PEC_ERR_INVALID_ARG;
        }
        if (!aligned16(a->acc_o) || (reinterpret_cast<uintptr_t>(a->acc_lse) & 3u)) {
            set_error("pec_prefill_attn: acc_o must be 16-byte aligned (acc_lse 4-byte)");
            return PEC_ERR_ALIGNMENT;
        }
    }
    if (a->q_num_parts > 1 && (a->q_part_id < 0 || a->q_part_id >= a->q_num_parts || a->cu_seqlens)) {
        set_error("pec_prefill_attn: need 0 <= q_part_id < q_num_parts, single request only");
        return PEC_ERR_INVALID_ARG;
    }
    if (a->overlap_previous != 0 && a->overlap_previous != 1) { set_error("pec_prefill_attn: overlap_previous must be 0 or 1"); return PEC_ERR_INVALID_ARG; }
    if (a->in_dtype == PEC_BF16 && !a->status) { set_error("pec_prefill_attn: bf16 inputs need a status word"); return PEC_ERR_INVALID_ARG; }
    if (a->worklist) {
        if (!a->cu_seqlens || a->n_items < 0 || (reinterpret_cast<uintptr_t>(a->worklist) & 15u)) {
            set_error("pec_prefill_attn: a work-list needs cu_seqlens, n_items >= 0 and 16-byte alignment");
            return PEC_ERR_INVALID_ARG;
        }
        if (a->worklist_block_m != pec_worklist_block_m(a->in_dtype)) {
            set_error("pec_prefill_attn: work-list built for tiles of %d rows, this kernel uses %d", a->worklist_block_m, pec_worklist_block_m(a->in_dtype));
            return PEC_ERR_INVALID_ARG;
        }
    }
    if (a->cu_seqlens) {
        if (a->B < 1) { set_error("pec_prefill_attn: packed batch needs B >= 1"); return PEC_ERR_INVALID_ARG; }
        if (a->chunk_start != 0 || a->chunk_len != a->seq_len || a->kv_len != a->seq_len || a->num_parts != 1) {
            set_error("pec_prefill_attn: packed batch needs chunk_start=0, chunk_len=kv_len=seq_len, num_parts=1");
            return PEC_ERR_INVALID_ARG;
        }
    }
    const int64_t esz = a->in_dtype == PEC_BF16 ? 2 : 4;
    const int64_t strides[6] = {a->q_stride_t, a->q_stride_h, a->k_stride_t, a->k_stride_h, a->v_stride_t, a->v_stride_h};
    for (int i = 0; i < 6; ++i) {
        if (strides[i] < kHeadDim) { set_error("pec_prefill_attn: strides must be >= D"); return PEC_ERR_INVALID_ARG; }
        if ((strides[i] * esz) % 16 != 0) { set_error("pec_prefill_attn: strides must be multiples of 16 bytes"); return PEC_ERR_ALIGNMENT; }
    }
    if (!aligned16(a->q) || !aligned16(a->k) || !aligned16(a->v) || !aligned16(a->o) ||
        (reinterpret_cast<uintptr_t>(a->lse) & 3u) || (a->status && (reinterpret_cast<uintptr_t>(a->status) & 3u))) {
        set_error("pec_prefill_attn: q, k, v, o must be 16-byte aligned (lse, status 4-byte)");
        return PEC_ERR_ALIGNMENT;
    }
    if (a->workspace_bytes < pec_workspace_size(a) || (pec_workspace_size(a) > 0 && !a->workspace)) {
        set_error("pec_prefill_attn: workspace too small (%zu < %zu)", a->workspace_bytes, pec_workspace_size(a));
        return PEC_ERR_WORKSPACE;
    }

    std::memset(&p, 0, sizeof(p));
    p.q = a->q; p.k = a->k; p.v = a->v; p.o = a->o; p.lse = a->lse;
    p.q_stride_t = a->q_stride_t; p.q_stride_h = a->q_stride_h;
    p.k_stride_t = a->k_stride_t; p.k_stride_h = a->k_stride_h;
    p.v_stride_t = a->v_stride_t; p.v_stride_h = a->v_stride_h;
    p.Hq = a->Hq; p.Hkv = a->Hkv; p.group = a->Hq / a->Hkv;
    p.cu_seqlens = a->cu_seqlens; p.B = a->cu_seqlens ? a->B : 1;
    p.worklist = a->worklist; p.n_items = a->worklist ? a->n_items : 0;
    p.total_rows = a->chunk_len;
    p.out_pos0 = a->chunk_start;
    p.acc_o = a->acc_o; p.acc_lse = a->acc_lse;
    p.overlap_previous = a->overlap_previous;
    p.wait_cycles = wait_limit_cycles();
    p.test_skip_last_load = test_skip_last_load();
    // Query rows: the chunk, or its intersection with the two blocks of zigzag partition q_part_id.
    p.n_qseg = 0;
    if (!a->cu_seqlens) {
        int64_t qlo[2] = {a->chunk_start, 0}, qhi[2] = {a->chunk_start + a->chunk_len, 0};
        int nq = 1;
        if (a->q_num_parts > 1) { zigzag_intervals(a->seq_len, a->q_num_parts, a->q_part_id, a->part_align, qlo, qhi); nq = 2; }
        for (int t = 0; t < nq; ++t) {
            const int64_t lo = qlo[t] > a->chunk_start ? qlo[t] : a->chunk_start;
            const int64_t hi = qhi[t] < a->chunk_start + a->chunk_len ? qhi[t] : a->chunk_start + a->chunk_len;
            if (hi > lo) { p.q_lo[p.n_qseg] = lo; p.q_hi[p.n_qseg] = hi; ++p.n_qseg; }
        }
    }
    p.causal = a->causal;
    p.scale = a->softmax_scale > 0.f ? a->softmax_scale : (float)(1.0 / std::sqrt((double)kHeadDim));
    p.scale_log2 = (float)((double)p.scale * 1.4426950408889634074);
    p.o_is_bf16 = a->o_dtype == PEC_BF16;
    p.status = a->status;
    p.splits = 1;
    p.split_keys = 0;

    // Key subset of a single request: zigzag partition cut to the stored K/V prefix.
    int64_t lo[2], hi[2];
    if (a->num_parts == 1) { lo[0] = 0; hi[0] = a->seq_len; lo[1] = hi[1] = a->seq_len; }
    else zigzag_intervals(a->seq_len, a->num_parts, a->part_id, a->part_align, lo, hi);
    p.n_iv = 0;
    for (int t = 0; t < 2; ++t) {
        const int64_t h = hi[t] < a->kv_len ? hi[t] : a->kv_len;
        if (h > lo[t]) { p.iv_lo[p.n_iv] = lo[t]; p.iv_hi[p.n_iv] = h; ++p.n_iv; }
    }
    for (int t = p.n_iv; t < 2; ++t) { p.iv_lo[t] = 0; p.iv_hi[t] = 0; }
    return PEC_OK;
}

}  // namespace pec

using namespace pec;

extern "C" const char *pec_last_error(void) { return g_last_error; }

extern "C" size_t pec_workspace_size(const pec_attn_args *) { return 0; }

extern "C" int32_t pec_worklist_block_m(int32_t in_dtype)
{
    return in_dtype == PEC_BF16 ? kBlockMBf16 : (in_dtype == PEC_F32 ? kBlockMF32 : 0);
}

extern "C" int pec_control(int32_t what, int64_t value)
{
    if (what == PEC_CTL_WAIT_LIMIT_CYCLES && value >= 1000) { g_wait_limit_cycles.store(value); return PEC_OK; }
    if (what == PEC_CTL_TEST_SKIP_LAST_LOAD && (value == 0 || value == 1)) { g_test_skip_last_load.store((int32_t)value); return PEC_OK; }
    set_error("pec_control: unknown setting %d or value %lld out of range", (int)what, (long long)value);
    return PEC_ERR_INVALID_ARG;
}

extern "C" int pec_prefill_attn(const pec_attn_args *args, void *cuda_stream)
{
    AttnParams p;
    int rc = resolve(args, p);
    if (rc != PEC_OK) return rc;
    if (p.total_rows == 0) return PEC_OK;   // nothing to write
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (!p.cu_seqlens) {
        // Rows below the subset's first key see nothing under the causal mask (and no row sees anything of an
        // empty subset).  Whole 256-row tiles of such rows get no CTA: an in-place merge leaves them as they
        // are, any other call has them filled (zero / -inf, or a copy of the incoming state).
        int64_t first_vis = INT64_MAX;
        for (int t = 0; t < p.n_iv; ++t) first_vis = p.iv_lo[t] < first_vis ? p.iv_lo[t] : first_vis;
        if (p.n_iv > 0 && !p.causal) first_vis = 0;
        const bool in_place = p.acc_o && static_cast<const void *>(p.acc_o) == p.o;
        int kept = 0;
        for (int s = 0; s < p.n_qseg; ++s) {
            int64_t lo = p.q_lo[s];
            const int64_t hi = p.q_hi[s];
            const int64_t blind_end = first_vis < lo ? lo : (first_vis > hi ? hi : first_vis);
            int64_t cut = lo + ((blind_end - lo) / kBlockMBf16) * kBlockMBf16;
            if (blind_end == hi) cut = hi;                 // the whole segment sees nothing
            if (cut > lo && !in_place) {
                rc = launch_fill_rows(p, lo - p.out_pos0, cut - p.out_pos0, stream);
                if (rc != PEC_OK) return rc;
            }
            lo = cut;
            if (hi > lo) { p.q_lo[kept] = lo; p.q_hi[kept] = hi; ++kept; }
        }
        p.n_qseg = kept;
        if (kept == 0) return PEC_OK;
    }
    if (args->in_dtype != PEC_BF16) return launch_attn_f32(p, stream);
    return launch_attn_prefill_bf16(p, stream);
}

extern "C" int pec_attn_merge(const void *o_a, const float *lse_a, const void *o_b, const float *lse_b,
                              void *o_out, float *lse_out, int64_t rows, int32_t Hq, int32_t D,
                              int32_t part_dtype, int32_t out_dtype, void *cuda_stream)
{
    if (!o_a || !lse_a || !o_b || !lse_b || !o_out || !lse_out) { set_error("pec_attn_merge: NULL pointer"); return PEC_ERR_INVALID_ARG; }
    if (rows < 0 || Hq < 1) { set_error("pec_attn_merge: need rows >= 0 and Hq >= 1"); return PEC_ERR_INVALID_ARG; }
    if (D != kHeadDim) { set_error("pec_attn_merge: D=%d unsupported (only 128)", D); return PEC_ERR_UNSUPPORTED; }
    if (part_dtype != PEC_F32) { set_error("pec_attn_merge: partials must be fp32"); return PEC_ERR_UNSUPPORTED; }
    if (out_dtype != PEC_F32 && out_dtype != PEC_BF16) { set_error("pec_attn_merge: unknown out_dtype %d", out_dtype); return PEC_ERR_UNSUPPORTED; }
    if (!aligned16(o_a) || !aligned16(o_b) || !aligned16(o_out) || !aligned16(lse_a) || !aligned16(lse_b) || !aligned16(lse_out)) {
        set_error("pec_attn_merge: buffers must be 16-byte aligned");
        return PEC_ERR_ALIGNMENT;
    }
    const bool alias_o = (o_out == o_a), alias_l = (lse_out == lse_a);
    if (alias_o != alias_l || (alias_o && out_dtype != PEC_F32) || o_out == o_b || lse_out == lse_b) {
        set_error("pec_attn_merge: outputs may alias side a only (both o and lse, fp32 output)");
        return PEC_ERR_INVALID_ARG;
    }
    if (rows == 0) return PEC_OK;
    return launch_merge(static_cast<const float *>(o_a), lse_a, static_cast<const float *>(o_b), lse_b,
                        o_out, lse_out, rows * (int64_t)Hq, out_dtype == PEC_BF16, alias_o ? 1 : 0,
                        static_cast<cudaStream_t>(cuda_stream));
}

extern "C" int pec_attn_merge_n(const void *const *o_parts, const float *const *lse_parts, int32_t n,
                                void *o_out, float *lse_out, int64_t rows, int32_t Hq, int32_t D,
                                int32_t part_dtype, int32_t out_dtype, void *cuda_stream)
{
    if (!o_parts || !lse_parts || !o_out || !lse_out) { set_error("pec_attn_merge_n: NULL pointer"); return PEC_ERR_INVALID_ARG; }
    if (n < 2 || n > PEC_MERGE_MAX_PARTS) { set_error("pec_attn_merge_n: need 2 <= n <= %d (got %d)", PEC_MERGE_MAX_PARTS, n); return PEC_ERR_INVALID_ARG; }
    if (rows < 0 || Hq < 1) { set_error("pec_attn_merge_n: need rows >= 0 and Hq >= 1"); return PEC_ERR_INVALID_ARG; }
    if (D != kHeadDim) { set_error("pec_attn_merge_n: D=%d unsupported (only 128)", D); return PEC_ERR_UNSUPPORTED; }
    if (part_dtype != PEC_F32) { set_error("pec_attn_merge_n: partials must be fp32"); return PEC_ERR_UNSUPPORTED; }
    if (out_dtype != PEC_F32 && out_dtype != PEC_BF16) { set_error("pec_attn_merge_n: unknown out_dtype %d", out_dtype); return PEC_ERR_UNSUPPORTED; }
    MergeParts parts;
    parts.n = n;
    for (int k = 0; k < PEC_MERGE_MAX_PARTS; ++k) { parts.o[k] = nullptr; parts.lse[k] = nullptr; }
    for (int k = 0; k < n; ++k) {
        if (!o_parts[k] || !lse_parts[k]) { set_error("pec_attn_merge_n: part %d is NULL", k); return PEC_ERR_INVALID_ARG; }
        if (!aligned16(o_parts[k]) || !aligned16(lse_parts[k])) { set_error("pec_attn_merge_n: buffers must be 16-byte aligned"); return PEC_ERR_ALIGNMENT; }
        parts.o[k] = static_cast<const float *>(o_parts[k]);
        parts.lse[k] = lse_parts[k];
        const bool alias_o = (o_out == o_parts[k]), alias_l = (lse_out == lse_parts[k]);
        if ((alias_o || alias_l) && (k != 0 || alias_o != alias_l || out_dtype != PEC_F32)) {
            set_error("pec_attn_merge_n: outputs may alias part 0 only (both o and lse, fp32 output)");
            return PEC_ERR_INVALID_ARG;
        }
    }
    if (!aligned16(o_out) || !aligned16(lse_out)) { set_error("pec_attn_merge_n: buffers must be 16-byte aligned"); return PEC_ERR_ALIGNMENT; }
    if (rows == 0) return PEC_OK;
    return launch_merge_n(parts, o_out, lse_out, rows * (int64_t)Hq, out_dtype == PEC_BF16, static_cast<cudaStream_t>(cuda_stream));
}
