/*
 * pec.h - C ABI of the partial causal prefill attention library (sm_100a).
 *
 * The library computes the attention step that PecSched's fast sequence
 * parallelism and prefill preemption revolve around (arXiv 2409.15104):
 * causal softmax attention (Eq. 3, with the row softmax of Eq. 4 summing over
 * the keys up to and including the row's own token) evaluated as a *partial*
 * result over a subset of the keys, with the per-row log-sum-exp kept so that
 * partials over disjoint key subsets can be merged exactly (the online-softmax
 * combination that ring attention relies on, Section 2.2) and so that a
 * preempted prefill can resume chunk by chunk from its stored K/V prefix
 * (Section 5.1).
 *
 * Conventions for every call:
 *   - returns PEC_OK (0) or a negative pec_status; never throws, never aborts;
 *   - never allocates or frees device memory and never synchronises: kernels
 *     are enqueued on the caller's CUDA stream (`cuda_stream` is a
 *     cudaStream_t passed as void*, NULL = the legacy default stream);
 *   - the caller owns every buffer; outputs are undefined after an error;
 *   - pointers marked "device" must be device-accessible, "host" host memory.
 */
#ifndef PEC_H_
#define PEC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    PEC_OK = 0,
    PEC_ERR_INVALID_ARG = -1, /* NULL pointer, negative size, inconsistent ranges      */
    PEC_ERR_UNSUPPORTED = -2, /* head_dim != 128, dtype combination not implemented   */
    PEC_ERR_ALIGNMENT = -3,   /* pointer or stride not aligned as required             */
    PEC_ERR_WORKSPACE = -4,   /* workspace smaller than pec_workspace_size()           */
    PEC_ERR_CUDA = -5,        /* a CUDA runtime/driver call or the launch failed       */
    PEC_ERR_TIMEOUT = -6,     /* value a kernel stores in *status when a bounded wait  */
                              /* inside it gave up (read it after synchronising)       */
    PEC_ERR_CAPACITY = -7     /* a caller array of pec_plan is too small               */
} pec_status;

typedef enum { PEC_BF16 = 1, PEC_F32 = 2 } pec_dtype;

/* Tile classes written by pec_plan_partitions. */
enum { PEC_TILE_SKIP = 0, PEC_TILE_PARTIAL = 1, PEC_TILE_FULL = 2 };

/*
 * Arguments of pec_prefill_attn.
 *
 * Layout: q is [Tq, Hq, D], k and v are [Tk, Hkv, D] with D contiguous; token
 * and head strides are given in elements.  Query head h reads KV head
 * h / (Hq / Hkv) (grouped-query attention, Section 5.3).  D must be 128.
 *
 * Single request (cu_seqlens == NULL): row t of q/k/v is the token at position
 * t of a request of `seq_len` tokens.  The call handles query rows
 * [chunk_start, chunk_start + chunk_len) and may read keys [0, kv_len) only:
 * this is one preemptible chunk resumed from the stored K/V prefix
 * (Section 5.1).  Output row r of o / lse belongs to position chunk_start + r.
 *
 * Packed batch (cu_seqlens != NULL): request b owns rows
 * [cu_seqlens[b], cu_seqlens[b+1]) of q, k, v, o and lse and attends only to
 * itself, each request starting at position 0 (short-request batches,
 * Section 5.2).  seq_len is the total number of packed rows (cu_seqlens[B]),
 * chunk_start must be 0, chunk_len and kv_len must equal seq_len, num_parts
 * must be 1.
 *
 * Query subset: with q_num_parts <= 1 every row of the chunk; otherwise only those rows of the
 * chunk that lie in zigzag partition q_part_id of q_num_parts (same rule and part_align as the key
 * partitions): the rows one rank of ring-attention sequence parallelism keeps (Section 2.2), so that
 * one call with part_id = (q_part_id - t) mod num_parts is that rank's ring step t.  o and lse keep
 * their chunk layout; rows outside the query subset are neither read nor written.  Single request only.
 *
 * Key subset: with num_parts == 1 all keys of [0, kv_len); otherwise zigzag
 * partition part_id of num_parts as defined by pec_plan_partitions(seq_len,
 * num_parts, ..., part_align, ...), intersected with [0, kv_len).  With
 * `causal`, key j is visible to the query at position i iff j <= i.
 *
 * Results: o[r, h, :] = sum_j p_j v_j over the visible keys of the subset with
 * p the softmax of softmax_scale * q.k restricted to that subset, and
 * lse[r, h] = ln sum_j exp(softmax_scale * q.k_j) (natural log, fp32).  A row
 * with no visible key gets o = 0 and lse = -inf, the identity of
 * pec_attn_merge.  o_dtype PEC_F32 gives a partial fit for merging;
 * PEC_BF16 rounds to nearest-even (allowed with in_dtype PEC_BF16 only).
 *
 * Incoming state (acc_o, acc_lse; both or neither): a partial result of the SAME rows over a key
 * subset disjoint from this call's, fp32, laid out like o / lse.  The call then returns the merge of
 * the two - lse = ln(exp(acc_lse) + exp(lse_own)), o = the correspondingly weighted sum, i.e. the
 * online-softmax step across key segments of Section 2.2, what pec_attn_merge computes - instead of
 * its own partial, so a chain of calls over the key partitions needs no partial buffers and no merge
 * pass.  o / lse may be the very buffers acc_o / acc_lse (both, o_dtype PEC_F32): rows that see no key
 * of this call's subset then stay untouched.  Only the last call of a chain should round to PEC_BF16.
 *
 * overlap_previous = 1 tells the library that q, k and v (and cu_seqlens / worklist) were complete before the kernel
 * that precedes this call on the stream was enqueued - true for every launch but the first of a chain over the key
 * partitions, or of a ring rank's steps.  The bf16 kernel may then start on SMs that the preceding kernel has already
 * left (programmatic dependent launch) and work through its key tiles while that kernel's last CTAs finish; it still
 * waits for the preceding kernel to complete before it reads the incoming state or writes o / lse.  Chains of short
 * launches lose their launch gaps and partial last waves that way.  With 0 (default) the call is ordered after
 * everything enqueued before it, as any kernel is.
 *
 * Packed batches may pass a work-list (worklist, n_items, worklist_block_m) made by pec_plan_worklist
 * and copied to the device by the caller: tiles then run heaviest first across requests and no CTA
 * searches cu_seqlens.  worklist_block_m must equal pec_worklist_block_m(in_dtype).
 *
 * in_dtype PEC_BF16 runs the tcgen05 tensor-core kernel (bf16 products, fp32
 * accumulation); PEC_F32 runs an fp32 FMA kernel (accuracy path).
 */
typedef struct {
    const void *q, *k, *v;      /* device; 16-byte aligned                              */
    int64_t q_stride_t, q_stride_h;
    int64_t k_stride_t, k_stride_h;
    int64_t v_stride_t, v_stride_h;   /* elements; bf16: multiples of 8               */
    int32_t in_dtype;           /* pec_dtype of q, k, v                                  */
    void *o;                    /* device; [rows, Hq, D] contiguous, 16-byte aligned     */
    int32_t o_dtype;            /* pec_dtype of o                                        */
    float *lse;                 /* device; [rows, Hq] contiguous                         */
    int32_t Hq, Hkv, D;
    const int32_t *cu_seqlens;  /* device; [B+1] non-decreasing, or NULL                 */
    int32_t B;                  /* number of packed requests (ignored when NULL above)   */
    int64_t seq_len;
    int64_t chunk_start, chunk_len;
    int64_t kv_len;             /* causal calls need kv_len >= chunk_start + chunk_len   */
    int32_t part_id, num_parts;
    int32_t part_align;         /* partition alignment in tokens (>= 1)                  */
    int32_t causal;             /* 0 or 1                                                */
    float softmax_scale;        /* 0 selects 1/sqrt(D)                                   */
    void *workspace;            /* device scratch of pec_workspace_size() bytes or NULL  */
    size_t workspace_bytes;
    int32_t *status;            /* device word the caller zeroes; a kernel stores        */
                                /* PEC_ERR_TIMEOUT there if a wait expired.  Required    */
                                /* for in_dtype PEC_BF16, may be NULL for PEC_F32        */
    const float *acc_o;         /* device; incoming state [rows, Hq, D] fp32, or NULL    */
    const float *acc_lse;       /* device; [rows, Hq] fp32, or NULL                      */
    int32_t q_part_id, q_num_parts;   /* q_num_parts <= 1: all rows of the chunk         */
    const int32_t *worklist;    /* device; [n_items][4] from pec_plan_worklist, or NULL  */
    int32_t n_items;
    int32_t worklist_block_m;
    int32_t overlap_previous;   /* 0 or 1, see above                                     */
} pec_attn_args;

/*
 * Partial attention of one chunk / partition / packed batch (Eq. 3-4; see the
 * struct above).  Validates the arguments on the host, then enqueues the attention
 * kernel over the row tiles that can see a key of the subset and, where whole tiles
 * of rows see none and still have to be written, one small fill kernel for those.
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, WORKSPACE, CUDA.
 */
int pec_prefill_attn(const pec_attn_args *args, void *cuda_stream);

/* Bytes of device scratch pec_prefill_attn needs for these arguments (may be 0). */
size_t pec_workspace_size(const pec_attn_args *args);

/*
 * Merge two partial results of the same rows over disjoint key subsets
 * (online-softmax combination, Section 2.2; the two-GPU outputs O_1, O_2 of one
 * request in Section 5.2's colocation example are combined this way):
 *     lse = ln(exp(lse_a) + exp(lse_b))
 *     o   = exp(lse_a - lse) * o_a + exp(lse_b - lse) * o_b
 * per (row, head); a side with lse = -inf contributes nothing, both -inf give
 * o = 0, lse = -inf.  o_a, o_b: device [rows, Hq, D] fp32 (part_dtype must be
 * PEC_F32); lse_*: device [rows, Hq] fp32; o_out: device [rows, Hq, D] of
 * out_dtype (PEC_F32 or PEC_BF16); all contiguous and 16-byte aligned.  o_out /
 * lse_out may alias o_a / lse_a (running merge) when out_dtype == PEC_F32.
 * D must be 128.  Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, CUDA.
 */
int pec_attn_merge(const void *o_a, const float *lse_a, const void *o_b, const float *lse_b,
                   void *o_out, float *lse_out, int64_t rows, int32_t Hq, int32_t D,
                   int32_t part_dtype, int32_t out_dtype, void *cuda_stream);

/*
 * The same merge over n partials at once (2 <= n <= PEC_MERGE_MAX_PARTS): one pass over
 * memory instead of n-1, which is what a rank holding several ring steps' partials, or a
 * single GPU running virtual partitions, wants (Section 2.2):
 *     lse = ln sum_i exp(lse_i);   o = sum_i exp(lse_i - lse) * o_i
 * o_parts / lse_parts: HOST arrays of n DEVICE pointers ([rows, Hq, D] fp32 and [rows, Hq]
 * fp32, contiguous, 16-byte aligned); the arrays are read during the call only.  o_out /
 * lse_out as in pec_attn_merge; they may alias part 0 (both, fp32 output) and no other part.
 * Parts whose lse is -inf for a row are not read for that row.
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, CUDA.
 */
#define PEC_MERGE_MAX_PARTS 16
int pec_attn_merge_n(const void *const *o_parts, const float *const *lse_parts, int32_t n,
                     void *o_out, float *lse_out, int64_t rows, int32_t Hq, int32_t D,
                     int32_t part_dtype, int32_t out_dtype, void *cuda_stream);

/*
 * Decode attention of a long request's single new token over part of its K/V cache
 * (Section 5.2: the long request in decode has one query token; its Q is sent to each GPU that
 * holds part of the K/V, every GPU computes attention over its own part with Eq. 3, and the
 * partial outputs are merged).  This call is one GPU's share: keys [kv_lo, kv_hi) of
 * k, v [Tk, Hkv, D] (same layout and strides as pec_prefill_attn; row t = position t), all
 * visible to the token.  q: device [Hq, D] bf16, head stride q_stride_h elements.  Results:
 * o [Hq, D] (o_dtype PEC_F32 for a partial to merge, PEC_BF16 for a final output), lse [Hq] fp32,
 * as defined for pec_prefill_attn; an empty range gives o = 0, lse = -inf.  Two GPUs' results are
 * combined with pec_attn_merge (rows = 1).
 *
 * The key range is cut into num_splits slices (0 = the library chooses) that run in parallel and
 * leave their partial results in `workspace` (device, 16-byte aligned, at least
 * pec_decode_workspace_size() bytes, which depends on Hq, the range and num_splits); a second
 * small kernel combines them.  The workspace contents are scratch: undefined after the call.
 * `status` as in pec_attn_args, but required.  Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT,
 * WORKSPACE, CUDA.
 */
typedef struct {
    const void *q;              /* device; [Hq, D] bf16, 16-byte aligned                        */
    int64_t q_stride_h;
    const void *k, *v;          /* device; [Tk, Hkv, D] bf16                                   */
    int64_t k_stride_t, k_stride_h, v_stride_t, v_stride_h;
    void *o;                    /* device; [Hq, D] contiguous                                  */
    int32_t o_dtype;
    float *lse;                 /* device; [Hq]                                                */
    int32_t Hq, Hkv, D;         /* D must be 128; Hkv | Hq; Hq / Hkv <= 128                    */
    int64_t kv_lo, kv_hi;       /* 0 <= kv_lo <= kv_hi <= Tk                                   */
    int32_t num_splits;         /* 0 = choose; otherwise 1..4096                               */
    float softmax_scale;        /* 0 selects 1/sqrt(D)                                         */
    void *workspace;
    size_t workspace_bytes;
    int32_t *status;
} pec_decode_args;

int pec_decode_attn(const pec_decode_args *args, void *cuda_stream);

/* Bytes of workspace pec_decode_attn needs for these arguments (0 if they are invalid). */
size_t pec_decode_workspace_size(const pec_decode_args *args);

/*
 * pec_decode_attn without a workspace argument.  (The paper has no counterpart for this call; it
 * exists for the way such a kernel gets deployed.)
 *
 * Who needs it: a serving engine of the kind the paper builds on hands every free byte of HBM
 * to its KV-cache pool at start-up, and the decode step of a colocated long request is issued
 * from a scheduler loop that must not stall.  Such a caller cannot ask the driver for memory at
 * that point: cudaMalloc may simply fail because nothing is left, and even when it succeeds it
 * synchronises the whole device, which is exactly the pause the scheduler is trying to avoid.
 * Nor may the call be handed a slice of the engine's pool by a layer that does not own it.
 *
 * So this variant keeps its scratch inside the library: a fixed array of
 * PEC_DECODE_STATIC_SCRATCH_BYTES in device memory that every GPU loading the library carries
 * from load until the process exits.  It performs no allocation and frees nothing.  Arguments
 * and results are those of pec_decode_attn, except that `workspace` and `workspace_bytes` are
 * ignored.  A call whose slices need more scratch than the array holds (slices x Hq x 516
 * bytes; see pec_decode_workspace_size) is refused with PEC_ERR_WORKSPACE and a message that
 * names both sizes: lower num_splits, or use pec_decode_attn.
 *
 * The first call on each device looks up the array's device address (with that device
 * current) and remembers it; make that first call outside any stream capture.  Under CUDA's
 * default lazy module loading that first call may also be the moment the driver loads the part
 * of the library that holds the array, i.e. the moment the array's memory is actually taken: an
 * engine should therefore make one priming call per device at start-up, before it sizes its
 * pool (or run with CUDA_MODULE_LOADING=EAGER).  Every later call takes and returns no memory.  All calls on a
 * device share the one array and it keeps whatever the previous call left there.  Nothing in
 * it has to start at zero - each call overwrites every partial it later reads - but two calls
 * that overlap on the GPU (different streams, or one stream replayed concurrently) would
 * overwrite each other's partials: keep them ordered.
 * Errors: as pec_decode_attn, plus PEC_ERR_CUDA if the address lookup fails.
 */
#define PEC_DECODE_STATIC_SCRATCH_BYTES (4 * 1024 * 1024)
int pec_decode_attn_static(const pec_decode_args *args, void *cuda_stream);

/*
 * Host-side plan of how a request of seq_len tokens is split.  All arrays are
 * host memory owned by the caller; an array pointer may be NULL to skip that
 * output.  Capacities are element counts; the needed counts are always written
 * to the n_* fields, so a first call with NULL arrays is a size query.
 *
 * The paper cuts a long input into segments handled by different replicas
 * (Section 2.2) and pauses a prefill between kernels (Section 5.1) without
 * fixing either rule; this library's integer rule is:
 *   U = ceil(seq_len / align);  bounds[k] = min(seq_len, align * floor(k*U / (2P))), k = 0..2P
 *   block k = [bounds[k], bounds[k+1]);  partition p owns blocks p and 2P-1-p (zigzag)
 *   part_lo/part_hi[2p], [2p+1] = those two intervals (an interval may be empty)
 *   pairs[p] = number of (query, key) pairs with the key in partition p, over all
 *              seq_len query rows: sum (seq_len - j) if causal, else seq_len per key
 *   chunk c = [c*chunk_len, min(seq_len, (c+1)*chunk_len));  chunk_len <= 0: one chunk
 *   tile_class[a*nk_tiles + b] for query tile a (block_m rows) and key tile b
 *   (block_n keys): causal: SKIP if the tile's first key is after its last query,
 *   FULL if its last key is not after its first query, else PARTIAL; non-causal: FULL.
 */
typedef struct {
    int64_t *bounds;      int64_t bounds_cap;  /* 2P+1                      */
    int64_t *part_lo;     int64_t *part_hi;    int64_t part_cap;   /* 2P    */
    int64_t *pairs;       int64_t pairs_cap;   /* P                         */
    int64_t *chunk_start; int64_t *chunk_len;  int64_t chunk_cap;  /* n_chunks */
    uint8_t *tile_class;  int64_t tile_cap;    /* nq_tiles * nk_tiles       */
    int64_t n_bounds, n_parts, n_chunks, nq_tiles, nk_tiles;       /* outputs */
} pec_plan;

/* Errors: INVALID_ARG (seq_len < 0, num_parts < 1, align/block < 1, NULL plan), CAPACITY. */
int pec_plan_partitions(int64_t seq_len, int32_t num_parts, int64_t chunk_len, int32_t align,
                        int32_t block_m, int32_t block_n, int32_t causal, pec_plan *plan);

/*
 * Work-list of a packed batch of short requests (Section 5.2): one entry per tile of block_m query
 * rows, every request starting a fresh tile, ordered so that the kernel's CTAs take the tiles with
 * the most key tiles first (a heavy tile started late would leave the other SMs idle at the end).
 *   weight of the tile at positions [pos0, pos0 + n) of a request of length L:
 *       causal: ceil(min(L, pos0 + n) / block_n), otherwise ceil(L / block_n)
 *   order: weight descending; equal weights by request index, then pos0, ascending
 *   items[4 i .. 4 i + 3] = { cu_seqlens[b], pos0, n, L } of entry i (request b)
 * cu_seqlens: HOST [B + 1], non-decreasing, starting anywhere; items: HOST, capacity items_cap entries
 * (may be NULL for a size query); *n_items receives the number of entries, sum_b ceil(L_b / block_m).
 * The caller copies items to the device and passes it as pec_attn_args.worklist.
 * Errors: INVALID_ARG (NULL cu_seqlens or n_items, B < 0, decreasing offsets, block < 1), CAPACITY.
 */
int pec_plan_worklist(const int32_t *cu_seqlens, int32_t B, int32_t block_m, int32_t block_n, int32_t causal,
                      int32_t *items, int64_t items_cap, int64_t *n_items);

/* Query rows per tile of the kernel behind pec_prefill_attn for this input type (0: unknown type). */
int32_t pec_worklist_block_m(int32_t in_dtype);

/*
 * Work plan of ring-attention sequence parallelism over num_parts ranks (Section 2.2: each replica
 * keeps the queries of its own segment and the K/V segments travel round the ring, one hop per
 * step).  Rank r owns the query rows of its segment; at ring step t it holds the K/V segment of
 * rank (r - t) mod num_parts.  pairs[r * num_parts + t] = number of visible (query, key) pairs of
 * that rank at that step: the attention work of the step (x 4 * D * Hq FLOPs).  step_max[t] = the
 * largest entry of step t over the ranks (a ring step lasts as long as its slowest rank),
 * rank_total[r] = the row sum of rank r.
 * layout PEC_LAYOUT_ZIGZAG: segment r = zigzag partition r of pec_plan_partitions (blocks r and
 * 2P-1-r).  layout PEC_LAYOUT_CONTIGUOUS: segment r = [c[r], c[r+1]) with
 * c[k] = min(seq_len, align * floor(k * U / P)), U = ceil(seq_len / align): the split that leaves
 * the last rank with about 2P-1 times the causal work of the first, which the zigzag pairing
 * removes (there every off-diagonal step costs the same on every rank).  The paper names neither
 * rule; both are this library's.
 * All arrays are host memory owned by the caller and may be NULL to skip; pairs_cap >= P*P,
 * vec_cap >= P where given.  Errors: INVALID_ARG (sizes, unknown layout), CAPACITY.
 */
typedef enum { PEC_LAYOUT_ZIGZAG = 0, PEC_LAYOUT_CONTIGUOUS = 1 } pec_layout;
int pec_plan_ring(int64_t seq_len, int32_t num_parts, int32_t align, int32_t layout, int32_t causal,
                  int64_t *pairs, int64_t pairs_cap, int64_t *step_max, int64_t *rank_total, int64_t vec_cap);

/*
 * Token-balanced short-request batches (Section 5.2: when short prefills preempt a long one, the
 * batches are built so that the total number of tokens per batch is balanced across the model
 * replicas).  The paper states the goal, not the rule; this library's rule is longest-first
 * greedy: requests are taken in order of decreasing length (equal lengths: lower index first) and
 * each goes to the replica that has the fewest tokens so far (equal totals: lowest replica id).
 * The largest replica total is then at most 4/3 - 1/(3 R) times the best possible one.
 * lengths: host [n], each >= 0; assign: host [n], receives the replica id of every request;
 * tokens: host [replicas] or NULL, receives the token total of every replica.
 * Errors: INVALID_ARG (NULL lengths/assign with n > 0, n < 0, replicas < 1, a negative length).
 */
int pec_balance_batches(const int32_t *lengths, int32_t n, int32_t replicas, int32_t *assign, int64_t *tokens);

/*
 * Intra-node SP strategy selection for a long prefill (Section 5.3).  With TP size T, G GPUs per
 * node, per-GPU segment length s, model width d, N_h query heads and N_kv KV heads of size d_h, the
 * paper gives, per stage and strategy, the communication volume in a node and the computation
 * volume on a GPU:
 *   attention stage, Megatron SP: comm 2sd(T-1)G            comp 2sd(N_h+N_kv)d_h/T + 4(sT)^2 d/T + 2sd^2
 *   attention stage, Ulysses SP : comm 2s(N_h+N_kv)d_h(G-1) + (d(N_h+N_kv)d_h + d^2)G(T-1)/T
 *                                 comp 2sd(N_h+N_kv)d_h + 4(sG)^2 d/G + 2sd^2
 *   MLP stage, Megatron SP      : comm 2sd(T-1)G            comp 16sd^2
 *   MLP stage, Ulysses SP       : comm 8d^2(T-1)G/T         comp 16sd^2
 * and picks, among the four combinations, the one with the lowest estimated latency.  The paper
 * does not say how volumes become time; this library's reading: seconds = comm elements *
 * elem_bytes / node_bw + comp / gpu_flops, summed over the two stages.  Host arithmetic in
 * double; ties go to the lower index (Megatron before Ulysses).  Strategy codes: 0 = Megatron SP,
 * 1 = Ulysses SP.  comm[stage][strategy] and comp[stage][strategy] (stage 0 = attention,
 * 1 = MLP) return the volumes, seconds[2*attn + mlp] the four estimates.
 * Errors: INVALID_ARG (NULL, non-positive sizes, T or G below 1, non-positive rates).
 */
typedef struct {
    double s, d, n_h, n_kv, d_h, T, G;
    double elem_bytes;          /* bytes per communicated element (2 for bf16)                  */
    double node_bw;             /* bytes per second the node moves in total                     */
    double gpu_flops;           /* operations per second of one GPU                             */
} pec_sp_inputs;
typedef struct {
    int32_t attn_strategy, mlp_strategy;
    double comm[2][2], comp[2][2], seconds[4];
} pec_sp_choice;
int pec_select_sp(const pec_sp_inputs *in, pec_sp_choice *out);

/*
 * y = x w^T, bf16 inputs and output, fp32 accumulation: the dense steps on either side of the
 * attention.  With w = the W_Q, W_K, W_V of all heads stacked row-wise it is the QKV generation
 * of Eq. 2 (y is then the fused [T, (Hq + 2 Hkv) * D] tensor whose column slices are the q, k, v
 * of pec_prefill_attn, addressed through its stride arguments); with w = W_L^T it is the
 * post-self-attention linear layer of Eq. 5.
 * x: device [M, K], w: device [N, K], y: device [M, N]; row-major with row strides in elements
 * (multiples of 8), 16-byte aligned; N and K multiples of 8.  `status`: required device word, used as
 * in pec_attn_args.  Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, CUDA.
 */
int pec_linear(const void *x, int64_t x_stride, const void *w, int64_t w_stride, void *y, int64_t y_stride,
               int64_t M, int32_t N, int32_t K, int32_t *status, void *cuda_stream);

/*
 * QKV generation (Eq. 2) with rotary position encoding of the query and key heads applied to the
 * fp32 accumulator before it is rounded to bf16.  The paper states no position encoding; the Llama
 * models it serves (Section 6.1) use this one (RoFormer's rotation in its "rotate-half" pairing):
 * the leading rot_cols columns of y are heads of 128 channels, channel i < 64 of a head pairs with
 * channel i + 64, and for the row at position p
 *     y'[i]      = y[i] cos(a) - y[i + 64] sin(a)
 *     y'[i + 64] = y[i + 64] cos(a) + y[i] sin(a),      a = p * theta^(-2 i / 128).
 * Columns from rot_cols on (the value heads) are left as they are.  rot_cols: multiple of 128, <= N.
 * rope_table: device table for positions 0 .. n_pos - 1, pec_rope_table_floats(n_pos) floats filled
 * by pec_rope_table, 16-byte aligned.  Row r is at position positions[r] (device int32 [M], e.g. a
 * packed batch's positions within their requests) or, with positions == NULL, at pos0 + r (a chunk
 * of one request, Section 5.1); positions outside [0, n_pos) are clamped to the table's ends, and
 * the host rejects pos0 + M > n_pos.  Everything else as in pec_linear.
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, CUDA.
 */
int pec_linear_rope(const void *x, int64_t x_stride, const void *w, int64_t w_stride, void *y, int64_t y_stride,
                    int64_t M, int32_t N, int32_t K, const float *rope_table, int64_t n_pos,
                    const int32_t *positions, int64_t pos0, int32_t rot_cols, int32_t *status, void *cuda_stream);

/*
 * The table pec_linear_rope reads, for positions 0 .. n_pos - 1 and D = 128.  The angle of position
 * p = 64 a + b and channel i is split by the addition theorem,
 *     cos(p f_i) = C[a][i] F[i][b] - S[a][i] G[i][b],   sin(p f_i) = S[a][i] F[i][b] + C[a][i] G[i][b],
 *     f_i = theta^(-2 i / D),  C, S = cos, sin(64 a f_i),  F, G = cos, sin(b f_i),
 * so that the kernel's reads are small and contiguous.  Layout, in floats:
 * F [64][64] | G [64][64] | C [na][64] | S [na][64] with na = ceil(n_pos / 64); every entry is worked
 * out in fp64 on the device and stored as fp32.  pec_rope_table_floats returns the table's length
 * (0 for a negative or too large n_pos); theta > 0 (500000 for Llama-3).
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, CUDA.
 */
size_t pec_rope_table_floats(int64_t n_pos);
int pec_rope_table(double theta, int64_t n_pos, int32_t D, float *table, void *cuda_stream);

/*
 * The post-self-attention linear layer (Eq. 5) taking partial attention results as they are:
 *     y = merge(o_1 .. o_n) w^T,   merge as in pec_attn_merge_n:
 *     lse = ln sum_i exp(lse_i);   o = sum_i exp(lse_i - lse) * o_i   per (row, head),
 * the merged o rounded to bf16 (nearest even) as the GEMM's operand and never written to memory.
 * This is what the GPU that finishes a shared long request does with its own and its peer's
 * outputs O_1, O_2 in Section 5.2's colocation example (n = 2), or a GPU holding the partials of
 * n key partitions (Section 2.2).
 * o_parts / lse_parts: HOST arrays of n DEVICE pointers (1 <= n <= PEC_LINEAR_MERGED_MAX_PARTS),
 * [rows, Hq, D] fp32 and [rows, Hq] fp32, contiguous, o 16-byte aligned; the arrays are read
 * during the call only.  What a part holds where its lse is -inf is not used (it may be anything,
 * NaN included); where every part's lse is -inf the merged row is 0.  D must be 128; the contraction runs over K = Hq * D.
 * w: device [N, K] bf16, y: device [rows, N] bf16; row strides in elements (multiples of 8),
 * 16-byte aligned; N a multiple of 8.  `status`: required device word, used as in pec_attn_args.
 * Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, CUDA.
 */
#define PEC_LINEAR_MERGED_MAX_PARTS 8
int pec_linear_merged(const void *const *o_parts, const float *const *lse_parts, int32_t n, int64_t rows, int32_t Hq,
                      int32_t D, const void *w, int64_t w_stride, void *y, int64_t y_stride, int32_t N,
                      int32_t *status, void *cuda_stream);

/*
 * Process-wide settings (the paper has no counterpart; they exist for operations and tests).
 *   PEC_CTL_WAIT_LIMIT_CYCLES   limit of every barrier wait inside the kernels, in SM clock cycles
 *                               (default 2e9, about a second).  A wait that runs out makes its CTA
 *                               leave through the normal exit and stores PEC_ERR_TIMEOUT in the
 *                               status word; a serving engine that would rather lose a request than
 *                               stall every short request queued behind a stuck kernel (Section 5.1's
 *                               preemption works between kernels only) sets it lower.  value >= 1000.
 *   PEC_CTL_TEST_SKIP_LAST_LOAD test hook, 0 / 1: the loader of the tensor-core kernels leaves out its
 *                               last tile (attention: the last V tile of a CTA that walks at least two
 *                               key tiles; pec_linear, pec_linear_merged: the last K step (pec_linear: of its last tile)
 *                               of the second CTA of each pair),
 *                               so that the waits for it run out and the timeout path can be checked.
 *                               Results of such a launch are undefined; the status word tells.
 * Applies to launches enqueued after the call.  Errors: INVALID_ARG.
 */
enum { PEC_CTL_WAIT_LIMIT_CYCLES = 1, PEC_CTL_TEST_SKIP_LAST_LOAD = 2 };
int pec_control(int32_t what, int64_t value);

/* Text describing the last non-zero return on this thread (never NULL). */
const char *pec_last_error(void);

#ifdef __cplusplus
}
#endif
#endif /* PEC_H_ */
