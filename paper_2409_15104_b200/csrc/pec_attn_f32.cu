// fp32 accuracy path of the partial causal attention (Eq. 3-4): fp32 inputs, fp32 FMA products,
// fp32 online-softmax state.  Exists because fp32 inputs are held to a 1e-4 output tolerance,
// which a single bf16 or tf32 tensor-core product of the scores cannot meet.
//
// One CTA = one (64-row query tile, head).  256 threads as 16x16: thread (ty, tx) owns score
// rows ty*4..+3 and columns tx+16*j of each 64-key tile, and output rows ty*4..+3 with channels
// tx*4..+3 and 64+tx*4..+3.  Q, K, V tiles and the probability tile are staged in shared memory.
#include <cuda_runtime.h>
#include "pec_host.h"
#include "pec_internal.h"
#include "pec_tile.cuh"

namespace pec {

constexpr int kBM = 64, kBN = 64;
constexpr int kLd = kHeadDim + 4;     // padded row of Q/K tiles (floats), keeps 16-byte alignment
constexpr int kLdP = kBN + 4;
constexpr int kF32Threads = 256;
constexpr size_t kF32Smem = sizeof(float) * (2 * kBM * kLd + kBN * kHeadDim + kBM * kLdP);

__global__ void __launch_bounds__(kF32Threads)
attn_f32_kernel(const AttnParams p)
{
    extern __shared__ __align__(16) float smem[];
    float *sQ = smem;                       // [kBM][kLd]
    float *sK = sQ + kBM * kLd;             // [kBN][kLd]
    float *sV = sK + kBN * kLd;             // [kBN][kHeadDim]
    float *sP = sV + kBN * kHeadDim;        // [kBM][kLdP]

    TileJob job;
    if (!locate_tile(p, blockIdx.x, kBM, job)) return;
    const int h = blockIdx.y, kvh = h / p.group;
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;

    const float *q = static_cast<const float *>(p.q);
    const float *k = static_cast<const float *>(p.k);
    const float *v = static_cast<const float *>(p.v);

    // Q tile -> shared (rows past the tile end are zero)
    for (int i = tid; i < kBM * (kHeadDim / 4); i += kF32Threads) {
        const int r = i / (kHeadDim / 4), c = (i % (kHeadDim / 4)) * 4;
        float4 val = make_float4(0.f, 0.f, 0.f, 0.f);
        if (r < job.n_rows)
            val = *reinterpret_cast<const float4 *>(q + (job.q_row0 + r) * p.q_stride_t + (int64_t)h * p.q_stride_h + c);
        *reinterpret_cast<float4 *>(sQ + r * kLd + c) = val;
    }

    float m_run[4], l_run[4], acc[4][8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        m_run[i] = -INFINITY; l_run[i] = 0.f;
#pragma unroll
        for (int c = 0; c < 8; ++c) acc[i][c] = 0.f;
    }
    const int64_t last_pos = job.q_pos0 + job.n_rows - 1;

    for (int t = 0; t < job.n_iv; ++t) {
        const int64_t lo = job.iv_lo[t];
        int64_t hi = job.iv_hi[t];
        if (p.causal && hi > last_pos + 1) hi = last_pos + 1;
        for (int64_t k0 = lo; k0 < hi; k0 += kBN) {
            __syncthreads();   // previous tile's sK/sV/sP reads are done (also orders the Q stores)
            for (int i = tid; i < kBN * (kHeadDim / 4); i += kF32Threads) {
                const int r = i / (kHeadDim / 4), c = (i % (kHeadDim / 4)) * 4;
                float4 kk = make_float4(0.f, 0.f, 0.f, 0.f), vv = kk;
                if (k0 + r < hi) {
                    const int64_t row = job.kv_row0 + k0 + r;
                    kk = *reinterpret_cast<const float4 *>(k + row * p.k_stride_t + (int64_t)kvh * p.k_stride_h + c);
                    vv = *reinterpret_cast<const float4 *>(v + row * p.v_stride_t + (int64_t)kvh * p.v_stride_h + c);
                }
                *reinterpret_cast<float4 *>(sK + r * kLd + c) = kk;
                *reinterpret_cast<float4 *>(sV + r * kHeadDim + c) = vv;
            }
            __syncthreads();

            // scores of a 4x4 micro-tile
            float s[4][4];
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) s[i][j] = 0.f;
#pragma unroll 4
            for (int d = 0; d < kHeadDim; d += 4) {
                float4 qa[4], kb[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) qa[i] = *reinterpret_cast<const float4 *>(sQ + (ty * 4 + i) * kLd + d);
#pragma unroll
                for (int j = 0; j < 4; ++j) kb[j] = *reinterpret_cast<const float4 *>(sK + (tx + 16 * j) * kLd + d);
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        s[i][j] = fmaf(qa[i].x, kb[j].x, s[i][j]);
                        s[i][j] = fmaf(qa[i].y, kb[j].y, s[i][j]);
                        s[i][j] = fmaf(qa[i].z, kb[j].z, s[i][j]);
                        s[i][j] = fmaf(qa[i].w, kb[j].w, s[i][j]);
                    }
            }

            // mask, online softmax (state replicated over the 16 threads sharing a row)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int64_t pos = job.q_pos0 + ty * 4 + i;
                int64_t lim = hi;                                  // keys < lim are visible
                if (p.causal && pos + 1 < lim) lim = pos + 1;
                float mx = -INFINITY;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const bool vis = (k0 + tx + 16 * j) < lim;
                    s[i][j] = vis ? s[i][j] * p.scale_log2 : -INFINITY;
                    mx = fmaxf(mx, s[i][j]);
                }
#pragma unroll
                for (int o = 8; o >= 1; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                const float m_new = fmaxf(m_run[i], mx);
                const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
                const float alpha = exp2f(m_run[i] - m_use);       // 0 while the row is still empty
                float rs = 0.f;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const float pj = exp2f(s[i][j] - m_use);
                    rs += pj;
                    sP[(ty * 4 + i) * kLdP + tx + 16 * j] = pj;
                }
#pragma unroll
                for (int o = 8; o >= 1; o >>= 1) rs += __shfl_xor_sync(0xffffffffu, rs, o);
                l_run[i] = l_run[i] * alpha + rs;
                m_run[i] = m_new;
#pragma unroll
                for (int c = 0; c < 8; ++c) acc[i][c] *= alpha;
            }
            __syncthreads();

            // acc += P V
#pragma unroll 4
            for (int j = 0; j < kBN; ++j) {
                const float4 v0 = *reinterpret_cast<const float4 *>(sV + j * kHeadDim + tx * 4);
                const float4 v1 = *reinterpret_cast<const float4 *>(sV + j * kHeadDim + 64 + tx * 4);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const float pj = sP[(ty * 4 + i) * kLdP + j];
                    acc[i][0] = fmaf(pj, v0.x, acc[i][0]); acc[i][1] = fmaf(pj, v0.y, acc[i][1]);
                    acc[i][2] = fmaf(pj, v0.z, acc[i][2]); acc[i][3] = fmaf(pj, v0.w, acc[i][3]);
                    acc[i][4] = fmaf(pj, v1.x, acc[i][4]); acc[i][5] = fmaf(pj, v1.y, acc[i][5]);
                    acc[i][6] = fmaf(pj, v1.z, acc[i][6]); acc[i][7] = fmaf(pj, v1.w, acc[i][7]);
                }
            }
        }
    }

    // epilogue: O / l, LSE = ln 2 * m + ln l (m holds log2-scaled scores); with an incoming state the
    // row's own result is merged into it by the LSE rule first (online softmax across launches).
    float *o = static_cast<float *>(p.o);
    const int64_t out_row0 = job.out_row0;
    const bool in_place = p.acc_o != nullptr && static_cast<const void *>(p.acc_o) == p.o;
    // The 16 threads of a row all need the row's incoming LSE, and lse may be that very buffer: every
    // read comes before the barrier, every write after it.
    float la_in[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = ty * 4 + i;
        la_in[i] = (p.acc_o != nullptr && r < job.n_rows) ? p.acc_lse[(out_row0 + r) * p.Hq + h] : -INFINITY;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int r = ty * 4 + i;
        if (r >= job.n_rows) continue;
        const bool empty = (l_run[i] == 0.f);
        if (empty && in_place) continue;                       // the row gained no key: its state stays
        float c_own = empty ? 0.f : 1.f / l_run[i], c_acc = 0.f;
        float lse_row = empty ? -INFINITY : m_run[i] * 0.6931471805599453f + logf(l_run[i]);
        const int64_t item = (out_row0 + r) * p.Hq + h;
        float4 a0 = make_float4(0.f, 0.f, 0.f, 0.f), a1 = a0;
        if (p.acc_o != nullptr) {
            const float la = la_in[i];
            const float mx = fmaxf(lse_row, la);
            if (mx != -INFINITY) {
                const float e_own = empty ? 0.f : expf(lse_row - mx), e_acc = (la == -INFINITY) ? 0.f : expf(la - mx);
                const float inv_tot = 1.f / (e_own + e_acc);
                c_own *= e_own * inv_tot;
                c_acc = e_acc * inv_tot;
                lse_row = mx + logf(e_own + e_acc);
            }
            if (c_acc != 0.f) {
                a0 = *reinterpret_cast<const float4 *>(p.acc_o + item * kHeadDim + tx * 4);
                a1 = *reinterpret_cast<const float4 *>(p.acc_o + item * kHeadDim + 64 + tx * 4);
            }
        }
        float *dst = o + item * kHeadDim;
        *reinterpret_cast<float4 *>(dst + tx * 4) = make_float4(fmaf(c_acc, a0.x, acc[i][0] * c_own), fmaf(c_acc, a0.y, acc[i][1] * c_own),
                                                                fmaf(c_acc, a0.z, acc[i][2] * c_own), fmaf(c_acc, a0.w, acc[i][3] * c_own));
        *reinterpret_cast<float4 *>(dst + 64 + tx * 4) = make_float4(fmaf(c_acc, a1.x, acc[i][4] * c_own), fmaf(c_acc, a1.y, acc[i][5] * c_own),
                                                                     fmaf(c_acc, a1.z, acc[i][6] * c_own), fmaf(c_acc, a1.w, acc[i][7] * c_own));
        if (tx == 0) p.lse[item] = lse_row;
    }
}

int launch_attn_f32(const AttnParams &p, cudaStream_t stream)
{
    static unsigned char ready[host::kMaxDevices] = {};
    static std::mutex ready_mutex;
    if (!host::once_per_device(ready, ready_mutex, [] {
            return cudaFuncSetAttribute(attn_f32_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kF32Smem) == cudaSuccess; })) {
        set_error("pec_prefill_attn: cannot raise the shared-memory limit: %s", cudaGetErrorString(cudaGetLastError()));
        return PEC_ERR_CUDA;
    }
    int64_t tiles = 0;
    if (p.cu_seqlens) tiles = p.worklist ? p.n_items : (p.total_rows + kBM - 1) / kBM + p.B;   // each request may end in a ragged tile
    else for (int s = 0; s < p.n_qseg; ++s) tiles += (p.q_hi[s] - p.q_lo[s] + kBM - 1) / kBM;
    if (tiles == 0) return PEC_OK;
    if (tiles > 0x7fffffff || p.Hq > 65535) { set_error("pec_prefill_attn: grid too large"); return PEC_ERR_UNSUPPORTED; }
    dim3 grid((unsigned)tiles, (unsigned)p.Hq);
    attn_f32_kernel<<<grid, kF32Threads, kF32Smem, stream>>>(p);
    const cudaError_t err = cudaGetLastError();
    if (err != cudaSuccess) { set_error("pec_prefill_attn: launch failed: %s", cudaGetErrorString(err)); return PEC_ERR_CUDA; }
    return PEC_OK;
}

}  // namespace pec
