// C-ABI entry points: argument checks, resolution of the key subset, kernel dispatch.
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
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
    p.chunk_start = a->chunk_start; p.chunk_len = a->chunk_len;
    p.total_rows = a->chunk_len;
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

extern "C" int pec_prefill_attn(const pec_attn_args *args, void *cuda_stream)
{
    AttnParams p;
    const int rc = resolve(args, p);
    if (rc != PEC_OK) return rc;
    if (p.total_rows == 0) return PEC_OK;   // nothing to write
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
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
