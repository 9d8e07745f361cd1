/*
 * shareprefill.h - C ABI of the SharePrefill prefill-attention library for
 * NVIDIA B200 (sm_100a).
 *
 * The library computes the attention of ONE transformer layer during prefill
 * the way SharePrefill (arXiv 2505.19578) does it, with the per-head pattern
 * decision given by the caller:
 *
 *   1. "pivot" heads run exact dense causal attention and, in the same pass,
 *      emit a block-importance map: the softmax probability mass of every
 *      (query-block, key-block) tile                       [sp_dense_pivot_attn]
 *   2. each row-block of the map is reduced to a block mask by a cumulative
 *      mass threshold gamma (Algorithm "Construct Pivotal Pattern")
 *                                                [sp_block_mask_from_importance]
 *   3. the mask is shared with every head of the pivot's cluster (Algorithm
 *      "Share Pivotal Pattern"), and those heads run block-sparse causal
 *      attention over the selected tiles only (Section 5.1, masked attention
 *      A(Q,K,V,M))                                         [sp_block_sparse_attn]
 *
 *   sp_prefill_attn chains 1-3 on one stream.
 *
 * General conventions
 *   - Every function returns an int: SP_OK (0) or a negative SP_ERR_* code.
 *     Nothing throws, prints or exits.
 *   - Pointers are DEVICE pointers unless the comment says "host".
 *   - Calls validate on the host, enqueue kernels on `stream` (a cudaStream_t
 *     passed as void*; NULL = the default stream) and return WITHOUT
 *     synchronising.  Errors detected on the device (a bounded wait that ran
 *     out) are reported by sp_get_status after the caller has synchronised.
 *   - The caller owns every tensor and the stream.  The library owns only the
 *     sp_ctx (its workspace and status word).  A context belongs to one device
 *     and must not be used from two streams at the same time.
 *   - Tensors are bf16, logical shape [batch, heads, seq, head_dim], element
 *     strides given explicitly; stride[3] must be 1 and the other strides must
 *     be multiples of 8 elements (16 bytes); data must be 16-byte aligned.
 *     batch must be 1.
 *   - Supported: head_dim in {64, 128}; block in {64, 128}; seq a multiple of
 *     block; n_q_heads a multiple of n_kv_heads; seq / block <= 1024.
 *     Anything else returns SP_ERR_UNSUPPORTED.
 *   - Query head h reads KV head h / (n_q_heads / n_kv_heads).
 *   - Nb = seq / block.  Row-block i = query rows [i*block, (i+1)*block);
 *     key-block j likewise.  Attention is causal: key c is visible to query r
 *     iff c <= r, so only tiles j <= i exist.
 */
#ifndef SHAREPREFILL_H_
#define SHAREPREFILL_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  SP_OK = 0,
  SP_ERR_INVALID_ARG = -1, /* NULL pointer, bad shape/stride, gamma not in (0, +inf), ... */
  SP_ERR_UNSUPPORTED = -2, /* a size outside the supported set listed above            */
  SP_ERR_WORKSPACE = -3,   /* workspace allocation failed                              */
  SP_ERR_CUDA = -4,        /* a CUDA runtime / driver call failed                      */
  SP_ERR_TIMEOUT = -5,     /* a bounded device-side wait ran out (see sp_get_status)   */
  SP_ERR_SCRATCH_LIMIT = -6, /* sp_dense_pivot_attn_fixed_scratch: problem too large for the fixed array */
  SP_ERR_RANGE = -7         /* range-checked debug build only: an index left its range (see sp_get_status) */
};

/* bf16 tensor view: device pointer, sizes and strides in ELEMENTS. */
typedef struct {
  void* data;
  int64_t shape[4];  /* [batch, heads, seq, head_dim] */
  int64_t stride[4]; /* stride[3] == 1                 */
} sp_tensor;

typedef struct sp_ctx sp_ctx;

/* Create / destroy a context on CUDA device `device`.  Creation allocates a
 * small status buffer; the workspace grows on demand (cudaMalloc, which
 * synchronises the device) or ahead of time with sp_ctx_reserve. */
int sp_ctx_create(sp_ctx** out, int device);
int sp_ctx_destroy(sp_ctx* ctx);

/* Bytes of workspace sp_prefill_attn needs for a problem of this size
 * (importance maps, masks, compacted lists, per-tile softmax statistics; the
 * statistics are sized for the SM count of the current CUDA device).
 *
 * Which calls may allocate: any call that takes a context grows the context's
 * workspace when the problem needs more than it holds (cudaDeviceSynchronize,
 * cudaFree, cudaMalloc: it synchronises the device that one time), and
 * sp_prefill_attn_host does the same for its device copies of q, k, v and out.
 * Reserve ahead (sp_ctx_reserve) to keep the calls free of both: the figure
 * returned here covers sp_prefill_attn, sp_dense_pivot_attn,
 * sp_block_sparse_attn and the workspace part of sp_prefill_attn_host. */
int sp_workspace_bytes(int64_t seq, int n_q_heads, int n_kv_heads, int head_dim, int block,
                       int n_pivots, size_t* bytes /* host, out */);

/* The same for the calls that decide the pattern on the device (head_dim 128, block 128): *auto_bytes for
 * sp_prefill_attn_auto with n_pivots listed pivots, *layer_bytes for sp_prefill_attn_layer in a layer that
 * creates at most n_pivots new pivots.  Either pointer may be NULL.  (sp_prefill_attn_host also keeps device
 * copies of q, k, v and out, 2 q + 2 k sizes, allocated on its first call.) */
int sp_workspace_bytes_patterns(int64_t seq, int n_q_heads, int n_kv_heads, int head_dim, int block,
                                int n_pivots, int pooled_construction, size_t* auto_bytes /* host, out */,
                                size_t* layer_bytes /* host, out */);

/* Make sure the context's workspace holds at least `bytes`. */
int sp_ctx_reserve(sp_ctx* ctx, size_t bytes);

/* Read and clear the device status word.  The caller must have synchronised
 * the stream(s) it used.  *code is SP_OK or SP_ERR_TIMEOUT; *where identifies
 * the wait that gave up (kernel-internal id).  Either pointer may be NULL.
 * SP_ERR_UNSUPPORTED with *where = 90 means the device laid out a CTA's shared
 * memory window or tensor memory differently from what the attention kernel was
 * built for (it then does no work).
 * The range-checked debug build of the library (compiled with SP_DEBUG; the
 * stand-in for a memory checker) also reports SP_ERR_RANGE here: an index that a
 * kernel computed from its inputs (a listed key-block, a head, a statistics
 * slot) was out of range; the kernel then used the nearest valid index instead
 * of touching memory it does not own, and *where names the check. */
int sp_get_status(sp_ctx* ctx, int* code /* host, out */, int* where /* host, out */);

/* Self-test of the bounded device-side waits: launches one warp that waits,
 * for at most `limit_cycles` SM cycles (1 .. 2e9), on a barrier nothing arrives
 * at.  The wait runs out, the kernel returns normally, and after the caller has
 * synchronised sp_get_status reports SP_ERR_TIMEOUT with where = 99.  Until
 * sp_get_status has cleared the status word every kernel of this context does
 * no work (outputs are left untouched), exactly as after a real timeout.  No
 * device fault, trap or unbounded loop is involved.  The paper has no
 * counterpart; this exists so that the failure path can be tested. */
int sp_selftest_wait_timeout(sp_ctx* ctx, int64_t limit_cycles, void* stream);

/* Static string for an SP_* code. */
const char* sp_strerror(int code);

/*
 * Step 1 - dense causal attention of selected heads, with block importance.
 *   (Algorithm "Share Pivotal Pattern": a head without a pivotal pattern gets
 *   the all-ones pattern and computes full attention; Section 5.2, "Sparse
 *   Attention Computation": the kernel emits a per-block statistic in the same
 *   pass that produces the output.)
 *
 *   heads           host, [n_heads]: query-head indices to process.
 *   out             same shape as q; rows of the listed heads are overwritten.
 *   importance_out  device fp32 [n_heads, Nb, Nb], or NULL for plain dense
 *                   attention.  Entry [t][i][j] = (1/block) * sum over rows r of
 *                   row-block i and keys c of key-block j (c <= r) of the softmax
 *                   probability P[r][c] of head heads[t]; each row-block's entries
 *                   sum to 1; entries with j > i are written as 0.
 *   lse_out         device fp32 [n_heads, seq] natural-log-sum-exp of the scaled
 *                   logits of each query row, or NULL.
 */
int sp_dense_pivot_attn(sp_ctx* ctx, const sp_tensor* q, const sp_tensor* k, const sp_tensor* v,
                        const int32_t* heads, int n_heads, int block, sp_tensor* out,
                        float* importance_out, float* lse_out, void* stream);

/*
 * Step 1 again, for callers that must not allocate device memory.
 *   (The paper has no counterpart: this is a deployment variant of the call above.)
 *
 *   Some hosts cannot call cudaMalloc at the moment they need attention: an
 *   inference-engine plugin whose enqueue hook is forbidden to allocate, a server
 *   whose memory pool already owns the whole device so that a raw allocation
 *   fails, a latency-critical loop that cannot afford the device-wide
 *   synchronisation an allocation implies.  sp_dense_pivot_attn needs a context
 *   (allocated) and a workspace (allocated, grown on demand) for the per-tile
 *   softmax statistics behind the importance map.  This variant needs neither:
 *   it takes no context and keeps those statistics in an array that is part of
 *   the library image, SP_FIXED_SCRATCH_BYTES (64 MiB) on every GPU that loads the
 *   library, held until the process exits.  It calls no cudaMalloc / cudaFree and
 *   no allocating library routine.
 *
 *   Same arguments and results as sp_dense_pivot_attn, plus `device`, the CUDA
 *   device the tensors live on, and the same kernels: at head_dim 128 and block 128
 *   the persistent kernel that gives a CTA two adjacent row-blocks, otherwise the
 *   one-row-block kernel.  Limits and rules:
 *   - with importance_out != NULL the launch needs statistics scratch: at head_dim
 *     128 / block 128, min(SMs of the device, n_heads * ceil(Nb / 2)) * 2 * Nb * 128 * 4
 *     bytes (148 SMs: any number of heads up to seq 56576); for the other shapes
 *     n_heads * Nb * (Nb + 1) / 2 * block * 4 bytes.  Beyond 64 MiB the call returns
 *     SP_ERR_SCRATCH_LIMIT and launches nothing.  Without importance no scratch is
 *     used and there is no limit.
 *   - the first call on a device looks up the array's device address (a host-side
 *     query, done with that device current).  With lazy module loading that query is
 *     also what loads the array's module, i.e. the moment the 64 MiB are taken from
 *     the device: it can synchronise, and on a device whose memory is already all in
 *     use it fails (SP_ERR_CUDA).  Make that first call at start-up, outside any
 *     stream capture.
 *   - all calls on a device share the one array, one status word and one work
 *     counter.  The array keeps whatever the last call left in it; nothing in it
 *     needs to start at zero, and status word and counter are cleared on the stream
 *     before every launch.  Two calls whose kernels may run at the same time on the
 *     same device (different streams, or different host threads) race on them:
 *     serialise them.
 *   - a device-side wait that runs out makes the kernel stop early, as in the
 *     context version: outputs are then incomplete.  sp_fixed_scratch_status reads
 *     that status word (after the caller has synchronised): *code is SP_OK or
 *     SP_ERR_TIMEOUT.  It allocates nothing either.
 */
#define SP_FIXED_SCRATCH_BYTES (64ull << 20)
int sp_dense_pivot_attn_fixed_scratch(int device, const sp_tensor* q, const sp_tensor* k, const sp_tensor* v,
                                      const int32_t* heads, int n_heads, int block, sp_tensor* out,
                                      float* importance_out, float* lse_out, void* stream);
int sp_fixed_scratch_status(int device, int* code /* host, out */, int* where /* host, out */);

/*
 * Step 2 - importance map -> block mask and compacted key-block lists.
 *   (Algorithm "Construct Pivotal Pattern": sort the scores, take the minimum
 *   budget K whose top-K sum reaches gamma, turn the index set into a mask.)
 *   Each row-block i of each of the `n_maps` maps is treated independently over
 *   its causal entries j = 0..i: order by importance descending (equal values:
 *   smaller j first), running sum in that order, K_i = first k whose sum >= gamma
 *   (all i+1 entries if the sum never gets there); the first K_i entries of the
 *   order are selected.  The running sum is exact (fixed point in units of 2^-50:
 *   it equals a float64 running sum unless that sum passes within 1e-12 of gamma).
 *
 *   importance   device fp32 [n_maps, nb, nb]; entries are probabilities: finite and
 *                >= 0 (anything else is read as 0; an entry above 4 counts as 4 in
 *                the running sum); entries with j > i are ignored.
 *   gamma        > 0.  Compared as the double nearest to this float.
 *   mask_out     device u8  [n_maps, nb, nb]: 1 = compute, 0 = skip (j > i: 0); may be NULL.
 *   counts_out   device i32 [n_maps, nb]: K_i.
 *   indices_out  device i32 [n_maps, nb, nb]: row i holds the K_i selected
 *                key-blocks in ascending order, then -1 up to nb.
 */
int sp_block_mask_from_importance(sp_ctx* ctx, const float* importance, int n_maps, int nb,
                                  float gamma, uint8_t* mask_out, int32_t* counts_out,
                                  int32_t* indices_out, void* stream);

/*
 * Step 3 - block-sparse causal attention (Section 5.1: A(Q,K,V,M) =
 *   softmax(QK^T/sqrt(d) - c(1-M)) V with c -> infinity, causal).
 *
 *   heads         host, [n_heads]: query heads to process.
 *   list_of_head  host, [n_heads]: which list (first index of counts/indices)
 *                 each listed head walks; -1 = all causal tiles (dense).
 *   counts        device i32 [n_lists, nb]; indices device i32 [n_lists, nb, nb]
 *                 as written by sp_block_mask_from_importance.  Every listed
 *                 row must select at least one key-block and only j <= i.
 *   out           rows of the listed heads are overwritten.
 */
int sp_block_sparse_attn(sp_ctx* ctx, const sp_tensor* q, const sp_tensor* k, const sp_tensor* v,
                         const int32_t* heads, int n_heads, const int32_t* list_of_head,
                         const int32_t* counts, const int32_t* indices, int n_lists, int block,
                         sp_tensor* out, void* stream);

/*
 * The whole layer (Algorithm "Sparse Attention" with the pattern decision fixed
 * by the caller): pivots dense + importance, importance -> mask, members sparse.
 *
 *   cluster_map  host, [n_q_heads]: cluster id of each query head; < 0 = no cluster.
 *   pivot_heads  host, [n_pivots]: heads that run dense and construct a pattern.
 *                The pivot of a cluster is the FIRST listed pivot head belonging
 *                to it.  A non-pivot head whose cluster has no pivot (or whose
 *                id is < 0) runs dense.
 *   gamma, block as above.
 *   out          bf16, same shape as q; fully overwritten.
 *   mask_out     device u8 [n_q_heads, Nb, Nb] or NULL: the pattern of each head:
 *                for a member its cluster pivot's mask, for a pivot the mask it
 *                constructed (its own output is dense), for a head that ran dense
 *                without constructing anything the causal all-ones mask.
 */
int sp_prefill_attn(sp_ctx* ctx, const sp_tensor* q, const sp_tensor* k, const sp_tensor* v,
                    const int32_t* cluster_map, const int32_t* pivot_heads, int n_pivots,
                    float gamma, int block, sp_tensor* out, uint8_t* mask_out, void* stream);

/*
 * The whole layer with HOST buffers: the same steps as sp_prefill_attn (same
 * algorithms of the paper), with the transfers pipelined around them, cluster by
 * cluster with the pivots one cluster ahead: pivot 0, pivot 1, the members of
 * cluster 0, pivot 2, the members of cluster 1, and so on.  A pivot's KV head and
 * queries are copied in, its dense attention and mask construction run, its
 * output is copied back; members follow in groups of one or two heads (their KV
 * head, if it is not on the device yet, and their queries in; attention; output
 * back) while the next bytes arrive.  Heads of clusters without a pivot run
 * dense, first.  Copies use two streams owned by the context; when the
 * call returns everything is enqueued, and `stream` is made to wait for the last
 * copy, so synchronising `stream` is enough before reading out_host.  The same
 * holds when the call fails part-way: whatever copies it had already enqueued
 * are joined into `stream` before it returns the error.
 *
 *   q_host             host bf16 [n_q_heads, seq, head_dim], contiguous
 *   k_host, v_host     host bf16 [n_kv_heads, seq, head_dim], contiguous
 *   out_host           host bf16, like q_host; fully overwritten
 *   mask_out_host      host u8 [n_q_heads, Nb, Nb] or NULL (as mask_out above)
 *   cluster_map, pivot_heads, gamma, block   as for sp_prefill_attn
 * Host buffers should be page-locked (cudaHostAlloc / cudaHostRegister):
 * pageable memory works but the copies then do not overlap anything.  The
 * buffers must stay valid and unmodified until `stream` has been synchronised.
 * The context keeps device copies of q, k, v and out (2 q + 2 k sizes, allocated
 * on first use, grown on demand) next to its workspace.
 */
int sp_prefill_attn_host(sp_ctx* ctx, const void* q_host, const void* k_host, const void* v_host,
                         int n_q_heads, int n_kv_heads, int64_t seq, int head_dim,
                         const int32_t* cluster_map, const int32_t* pivot_heads, int n_pivots,
                         float gamma, int block, void* out_host, uint8_t* mask_out_host, void* stream);

/*
 * Paper-literal pattern construction (the library's default pattern is the true
 * softmax mass per block, cut per row-block; these three calls follow the text
 * of the paper instead, so that the two can be compared).
 *
 * sp_pooled_logits - the block-wise average of the QK values, A~ (Section 5.2,
 *   "Sparse Attention Computation": computed next to the output; a block that is
 *   not computed gets -infinity).  Entry [t][i][j], j <= i, is the mean of
 *   q_r . k_c / sqrt(head_dim) over the visible (c <= r) entries of the block of
 *   head heads[t]; entries with j > i are -infinity.  The mean over a full block
 *   equals the product of the block means of Q and K, which is how it is
 *   computed, in float64 (the cut below compares a cumulative sum over up to half a
 *   million scores with gamma; fp32 averages of logits of order 1..30 would move it
 *   by 1e-5).
 *     heads host [n_heads]; pooled_out device FLOAT64 [n_heads, Nb, Nb].
 *
 * sp_pattern_from_pooled - Algorithm "Construct Pivotal Pattern": softmax of the
 *   block averages along each row-block, the last row kept as the pivotal
 *   representative a~, the map flattened and normalised by its total, sorted
 *   descending (equal scores: smaller row-major index first), minimum budget K
 *   whose scores sum to >= gamma (every existing block if they never do), index
 *   set -> mask.  A row-block left without a selected block receives its diagonal
 *   block.  The softmax is taken in float64 and every score rounded to fp32 once;
 *   the cumulative sums are exact fixed-point sums of those fp32 scores.
 *     pooled device FLOAT64 [n_maps, nb, nb] (as written by sp_pooled_logits).
 *   Outputs as for sp_block_mask_from_importance (mask_out required), plus
 *   last_row_out device fp32 [n_maps, nb] or NULL.
 *
 * sp_determine_pattern - Algorithm "Determine Sparse Pattern": a^ = softmax of
 *   the pooled QK values of the last block of queries against every key-block,
 *   d_sparse = sqrt(JSD(a^ || uniform)), d_sim = sqrt(JSD(a^ || a~)) (natural
 *   logarithm, float64 arithmetic on the device, the distances returned as fp32),
 *   pattern = shared pivot iff d_sparse < delta and d_sim < tau, else vertical-slash.
 *     pivot_last_rows device fp32 [n_rows, Nb] (a~ of the pivots, as written by
 *     sp_pattern_from_pooled); row_of_head host [n_heads]: which row each head is
 *     compared with, -1 = none (d_sim = +infinity).
 *     pattern_out device i32 [n_heads]: 0 = shared pivot, 1 = vertical-slash;
 *     dist_out device fp32 [n_heads, 2] = (d_sparse, d_sim), or NULL.
 */
int sp_pooled_logits(sp_ctx* ctx, const sp_tensor* q, const sp_tensor* k, const int32_t* heads,
                     int n_heads, int block, double* pooled_out, void* stream);
int sp_pattern_from_pooled(sp_ctx* ctx, const double* pooled, int n_maps, int nb, float gamma,
                           uint8_t* mask_out, int32_t* counts_out, int32_t* indices_out,
                           float* last_row_out, void* stream);
int sp_determine_pattern(sp_ctx* ctx, const sp_tensor* q, const sp_tensor* k, const int32_t* heads,
                         int n_heads, int block, const float* pivot_last_rows,
                         const int32_t* row_of_head, float delta, float tau, int32_t* pattern_out,
                         float* dist_out, void* stream);

/*
 * sp_vertical_slash_pattern - Algorithm "Search Vertical Slash Pattern" (the
 *   fallback pattern of heads that do not share a pivotal pattern): A^ =
 *   softmax(Q^ K^T / sqrt(head_dim)), causal, for Q^ = the last block of queries;
 *   its sums per key column (vertical) and per offset o = query - key >= 0 (slash),
 *   each normalised, ordered descending (equal scores: smaller index first) and cut
 *   at the minimum budget whose scores sum to >= gamma; the union of the selected
 *   lines is turned into a block mask: block (i, j), j <= i, is computed if
 *   key-block j contains a selected column or a selected offset lies in
 *   [(i-j) block - (block-1), (i-j) block + (block-1)].  A row-block left empty
 *   receives its diagonal block.  head_dim 128 and block 128 only.
 *     heads host [n_heads]; mask_out / counts_out / indices_out as for
 *     sp_block_mask_from_importance (all required), directly usable by
 *     sp_block_sparse_attn; sel_v_out, sel_s_out device u8 [n_heads, seq] or NULL:
 *     the selected columns and offsets.
 */
int sp_vertical_slash_pattern(sp_ctx* ctx, const sp_tensor* q, const sp_tensor* k, const int32_t* heads,
                              int n_heads, float gamma, int block, uint8_t* mask_out, int32_t* counts_out,
                              int32_t* indices_out, uint8_t* sel_v_out, uint8_t* sel_s_out, void* stream);

/*
 * sp_prefill_attn_auto - one layer of Algorithm "Sparse Attention" with the
 *   pattern decision made on the device, no host synchronisation:
 *     1. the listed pivot heads (heads whose cluster has no pivotal pattern yet)
 *        run dense and construct their pattern (Algorithm "Construct Pivotal
 *        Pattern": pooled_construction = 0: true softmax mass cut per row-block,
 *        as sp_prefill_attn does; 1: the paper-literal block-averaged QK values
 *        with one global cut, as sp_pattern_from_pooled does);
 *     2. every other head that has a pivot in its cluster is classified by
 *        Algorithm "Determine Sparse Pattern" (d_sparse < delta and d_sim < tau:
 *        it shares the pivot's pattern; otherwise it searches its own
 *        vertical-slash pattern, Algorithm "Search Vertical Slash Pattern");
 *     3. those heads run block-sparse attention over the list chosen for them;
 *        a head whose cluster has no pivot (or id < 0) runs dense.
 *   head_dim 128 and block 128 only.
 *     pattern_out  device i32 [n_q_heads] or NULL: 0 dense, 1 shared pivot,
 *                  2 vertical-slash.
 *     mask_out     device u8 [n_q_heads, Nb, Nb] or NULL: the pattern each head
 *                  used (a pivot: the pattern it constructed).
 *   Other arguments as for sp_prefill_attn.
 */
int sp_prefill_attn_auto(sp_ctx* ctx, const sp_tensor* q, const sp_tensor* k, const sp_tensor* v,
                         const int32_t* cluster_map, const int32_t* pivot_heads, int n_pivots,
                         float gamma, float delta, float tau, int block, int pooled_construction,
                         sp_tensor* out, uint8_t* mask_out, int32_t* pattern_out, void* stream);

/*
 * Cross-layer dictionary of pivotal patterns and the layer call that uses it
 * (Section 5.2: clusters span layers; the first head of a cluster that is met
 * constructs the pivotal pattern, every later head of the cluster, in this or a
 * later layer, reuses it after the similarity check).
 *
 *   sp_dict_create   a dictionary for up to `max_clusters` cluster ids, layers of
 *                    `n_q_heads` heads, sequences of `seq` tokens, `block` = 128.
 *                    It owns device memory for a mask, lists and a representative
 *                    per cluster plus scratch lists for one layer.
 *   sp_dict_clear    forget every stored pattern (a new prompt).
 *   sp_dict_count    clusters that currently have a stored pattern.
 *
 *   sp_prefill_attn_layer - one layer of Algorithm "Sparse Attention", heads taken in
 *   order:
 *     - a head of the noise cluster (id < 0), or with d_sparse >= delta (highly
 *       sparse), searches its own vertical-slash pattern;
 *     - otherwise, if its cluster has a pattern (stored, or constructed by an
 *       earlier head of this layer), it shares it when d_sim < tau and falls back
 *       to vertical-slash when not;
 *     - otherwise it becomes its cluster's pivot: dense attention, pattern
 *       constructed and stored with its representative (pooled_construction as
 *       for sp_prefill_attn_auto).
 *   Who becomes a pivot depends on d_sparse, which is computed on the device: the
 *   call synchronises `stream` ONCE (a few hundred bytes) before it enqueues the
 *   rest; the share / vertical-slash decisions stay on the device.
 *     cluster_of_head  host [n_q_heads]: cluster id in [0, max_clusters) or < 0.
 *     pattern_out      device i32 [n_q_heads] or NULL: 0 dense (new pivot), 1 shared,
 *                      2 vertical-slash.  mask_out as for sp_prefill_attn_auto.
 *   head_dim 128, block 128.  One dictionary serves one context and one sequence
 *   length; layers must be issued in order on one stream.
 */
typedef struct sp_pattern_dict sp_pattern_dict;
int sp_dict_create(sp_ctx* ctx, int max_clusters, int n_q_heads, int64_t seq, int block, sp_pattern_dict** out);
int sp_dict_destroy(sp_pattern_dict* dict);
int sp_dict_clear(sp_pattern_dict* dict);
int sp_dict_count(const sp_pattern_dict* dict);
int sp_prefill_attn_layer(sp_ctx* ctx, sp_pattern_dict* dict, const sp_tensor* q, const sp_tensor* k,
                          const sp_tensor* v, const int32_t* cluster_of_head, float gamma, float delta,
                          float tau, int block, int pooled_construction, sp_tensor* out,
                          uint8_t* mask_out, int32_t* pattern_out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* SHAREPREFILL_H_ */
