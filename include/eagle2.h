/*
 * eagle2.h -- C ABI of the B200 (sm_100a) library for the data-parallel hot path of EAGLE-2's
 * draft-and-verify cycle: draft-tree expansion, reranking, tree mask, tree-masked attention,
 * acceptance and KV compaction.
 *
 * Conventions that hold for every entry point
 *   - Every array pointer is a DEVICE pointer owned by the caller unless marked [host].  The
 *     library allocates nothing: scratch memory comes from a caller-supplied workspace whose size
 *     eagle2_workspace_bytes() reports.  A workspace must be 256-byte aligned and must have been
 *     passed through eagle2_workspace_init() once after allocation (it zeroes the arrival counters
 *     that the kernels leave zeroed again on exit; they occupy the first 4*B bytes, rounded up to
 *     256, in every operation's layout, so one workspace of the largest reported size serves all
 *     operations).  Calls that share a workspace must be ordered on one stream.
 *   - Every call only enqueues work on `stream` and returns; nothing synchronises, so a sequence of
 *     calls can be captured in a CUDA graph.
 *   - Return value: EAGLE2_OK, or a negative EAGLE2_ERR_* found on the host before anything was
 *     launched.  Conditions found on the device are OR-ed into *d_status (EAGLE2_STATUS_* bits, an
 *     int32 in device memory that the caller zeroes); the kernel still ends normally.
 *   - Tree layout (part of the interface).  k children per expanded node and k frontier nodes per
 *     level, depth D, N = k + (D-1)k^2 candidate nodes, R = 1 + (D-1)k draft-logit rows per cycle.
 *     Level-1 nodes have candidate index c in [0,k); a node of level l >= 2 has index
 *     k + (l-2)k^2 + j*k + c with j the frontier slot of its parent and c the rank of the child in
 *     its parent's draft distribution.  parent = -1 is the root (the last committed token).  Draft
 *     row 0 produces level 1; row 1 + (s-1)k + j belongs to frontier slot j of step s >= 1.
 *     Lower index implies shallower-or-equal level, so "ties to the lower index" is the paper's
 *     "ties to the shallower node", and ascending index is a topological order.
 */
#ifndef EAGLE2_H_
#define EAGLE2_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st* eagle2_stream_t; /* a cudaStream_t */

/* host-side errors (return values) */
#define EAGLE2_OK 0
#define EAGLE2_ERR_NULL (-1)        /* a required pointer is NULL */
#define EAGLE2_ERR_SHAPE (-2)       /* a size is outside the supported range */
#define EAGLE2_ERR_ALIGN (-3)       /* a base pointer or stride breaks the stated alignment */
#define EAGLE2_ERR_WORKSPACE (-4)   /* workspace missing, misaligned or too small */
#define EAGLE2_ERR_CUDA (-5)        /* the CUDA runtime refused the launch */
#define EAGLE2_ERR_STATIC_LIMIT (-6) /* sizes need more scratch than the library's built-in buffer holds */

/* device-side conditions (bits of *d_status) */
#define EAGLE2_STATUS_NONFINITE_LOGIT 1 /* NaN or +Inf logit, or a row of only -Inf */
#define EAGLE2_STATUS_NOT_CLOSED 2      /* a selected node's parent was not selected */
#define EAGLE2_STATUS_KV_OVERFLOW 4     /* a sequence's rows exceed the stated cache capacity */
#define EAGLE2_STATUS_TIMEOUT 8         /* a bounded device-side wait ran out */
/* (bit 16 is not used) */
#define EAGLE2_STATUS_BAD_TREE 32       /* parent/path arrays are not a valid topological tree */

/* limits */
#define EAGLE2_MAX_K 32        /* children per node / frontier size */
#define EAGLE2_MAX_M 128       /* rerank budget */
#define EAGLE2_MAX_NODES 4096  /* N = k + (D-1)k^2 */
#define EAGLE2_MAX_DEPTH 64

/* operations, for eagle2_workspace_bytes */
#define EAGLE2_OP_EXPAND 0
#define EAGLE2_OP_RERANK 1
#define EAGLE2_OP_TREE_MASK 2
#define EAGLE2_OP_TREE_ATTENTION 3
#define EAGLE2_OP_ACCEPT 4
#define EAGLE2_OP_KV_COMPACT 5
#define EAGLE2_OP_LM_HEAD_EXPAND 6

int eagle2_version(void);
const char* eagle2_strerror(int code);

/* Bytes of workspace the given operation needs at these sizes (0 if it needs none; sizes that do
 * not apply to the operation are ignored).  max_kv_len is the largest kv_len of any sequence. */
size_t eagle2_workspace_bytes(int op, int B, int V, int k, int D, int m, int Hq, int Hkv, int d,
                              int max_kv_len);

/* Zero a freshly allocated workspace (asynchronous on `stream`). */
int eagle2_workspace_init(void* ws, size_t ws_bytes, eagle2_stream_t stream);

/*
 * Bound of the device-side waits (no counterpart in the paper; it belongs to the library's failure
 * detection).  The tensor-path kernels (tree attention, LM head) and the streaming expansion hand
 * tiles and candidates between warps through barriers and queues; every such wait gives up after
 * `cycles` SM clock cycles, the kernel then lets its copies and tensor instructions in flight
 * finish, frees what it holds, raises EAGLE2_STATUS_TIMEOUT and ends normally, its outputs
 * undefined.  The default is 2^31 cycles (about a second); cycles <= 0 restores it.  The value is
 * process-wide, read on the host when a call is made and passed with the launch, so it applies to
 * calls made after it was set.  A deployment may lower it to learn of a stuck kernel sooner; a
 * test sets a few cycles to see the give-up path run.  Returns the bound in force before the call.
 */
long long eagle2_set_wait_limit(long long cycles);

/*
 * Before step 1 -- the LM head (paper Section 4.1: the draft model's feature of a token goes through
 * the LM head of the original LLM to give the draft distribution):
 *   logits[r][v] = sum_h hidden[r][h] * weight[v][h]      (no bias)
 * bf16 operands, fp32 accumulation on the tensor path, fp32 result: the [rows][V] array that
 * eagle2_expand takes as draft_logits (for B sequences pass rows = B*n_s and batch_stride = n_s*V).
 *   hidden  bf16 [rows][H], 16-byte aligned
 *   weight  bf16 [V][H], 16-byte aligned (the matrix is read once per call)
 *   logits  fp32 [rows][V], written
 * Limits: rows >= 0, H a multiple of 64, V >= 1.  Up to 256 rows are one pass over the weights; more
 * rows take one pass per 256.  Needs no workspace.  A bounded wait that
 * runs out raises EAGLE2_STATUS_TIMEOUT.
 */
int eagle2_lm_head(const void* hidden, const void* weight, int rows, int H, int V, float* logits,
                   int32_t* d_status, eagle2_stream_t stream);

/*
 * The LM head and the expansion of one step in one pass over the weights (paper Section 4.1: the
 * draft features go through the original LLM's LM head, and the expansion keeps every row's k most
 * probable tokens).  Same result as eagle2_lm_head followed by eagle2_expand on its logits, but the
 * logits are never written: the kernel that forms them folds them into per-row maxima, sums of
 * exponentials and k best (value, token) keys, and a merge launch builds the tree level and the
 * next frontier from those.  Meant for many feature rows (B * k of the order of 100 and more),
 * where the logits would cost as much traffic as the weights; with few rows the two separate calls
 * are as fast.
 *   hidden  bf16 [B][n_s][H] (n_s = 1 at s == 0, else k: the features of frontier slot j of sequence b
 *           at row b * n_s + j), 16-byte aligned;  weight  bf16 [V][H], 16-byte aligned
 *   tree_token, tree_parent, tree_value, frontier: as for eagle2_expand (level s + 1 is written,
 *           frontier is read at s > 0 and overwritten)
 *   ws      eagle2_workspace_bytes(EAGLE2_OP_LM_HEAD_EXPAND, B, V, k, ...) bytes
 * Up to 128 rows (B * n_s) ride on one pass over the weights, one block per SM; up to 256 on one
 * pass of block pairs; more rows take a pass per 256 and one for the rest.  Three kinds of launch per
 * call: the passes, a merge of every row's partial results, and the expansion's own merge.
 * Limits: those of eagle2_expand, and k <= 16, H a multiple of 64.  Logits are fp32 sums of bf16
 * products, as eagle2_lm_head forms them; a row's k-th and (k+1)-th logits closer than that sum's
 * rounding may come out in either order.  Status bits as for eagle2_expand; a bounded wait that
 * runs out raises EAGLE2_STATUS_TIMEOUT.
 */
int eagle2_lm_head_expand(const void* hidden, const void* weight, int H, int B, int V, int k, int D, int s,
                          int32_t* tree_token, int32_t* tree_parent, double* tree_value, int32_t* frontier,
                          void* ws, size_t ws_bytes, int32_t* d_status, eagle2_stream_t stream);

/*
 * Step 1 -- expansion (paper Section 4.1, the value equation V_i = prod c_j over Path(root, t_i)).
 * Called for s = 0..D-1.  For each of the n_s input rows (n_s = 1 at s = 0, else k; row j belongs
 * to frontier[b][j]) it takes the log-softmax over the vocabulary, makes the k most probable tokens
 * the node's children (ties: lower token id) and gives each the value parent value + log-probability,
 * i.e. the log of the product of draft confidences on the path (the root counts as 1).  The k best
 * new candidates by value (ties: lower index) become the next frontier.
 *   draft_logits  fp32 [B][n_s][V]; sequence b starts at draft_logits + b*batch_stride (elements).
 *                 16-byte aligned base and V % 4 == 0 select the vectorised path; anything else is
 *                 still handled.
 *   tree_token, tree_parent  int32 [B][N], tree_value fp64 [B][N]: level s+1 is written; earlier
 *                 levels are read (values of the frontier nodes).
 *   frontier      int32 [B][k]: read when s > 0, overwritten with the new frontier.
 * Limits: 1 <= k <= min(V, EAGLE2_MAX_K), N <= EAGLE2_MAX_NODES.
 */
int eagle2_expand(const float* draft_logits, long long batch_stride, int B, int V, int k, int D, int s,
                  int32_t* tree_token, int32_t* tree_parent, double* tree_value, int32_t* frontier,
                  void* ws, size_t ws_bytes, int32_t* d_status, eagle2_stream_t stream);

/*
 * Expansion with a choice of ranking score (paper Section 5.2, the ablation "without value").
 * The ablation compares expanding on the value with expanding on the confidence score, so only the
 * choice of the nodes to expand changes.  flags = 0 is eagle2_expand.  With
 * EAGLE2_EXPAND_BY_CONFIDENCE the next frontier is the k best new candidates by their own confidence
 * (the log-probability the draft model gives the token after its path; ties: lower index) instead
 * of by value.  Children, their order, tree_value (still the sum of log-probabilities along the
 * path) and everything else are unchanged, so eagle2_rerank afterwards ranks by value as always.
 * Every other argument, the workspace and the errors are those of eagle2_expand; an unknown flag
 * bit is EAGLE2_ERR_SHAPE.
 */
#define EAGLE2_EXPAND_BY_CONFIDENCE 1u
int eagle2_expand_variant(const float* draft_logits, long long batch_stride, int B, int V, int k, int D,
                          int s, unsigned flags, int32_t* tree_token, int32_t* tree_parent,
                          double* tree_value, int32_t* frontier, void* ws, size_t ws_bytes,
                          int32_t* d_status, eagle2_stream_t stream);

/*
 * Expansion without a caller workspace (the paper has no counterpart; this is a packaging variant of
 * eagle2_expand, same arguments minus ws/ws_bytes, same kernels, same results).  It is meant for
 * callers that cannot obtain device memory at the moment they need this step: a serving process
 * that handed all of HBM to its KV-cache pool at start-up and has no allocator left to ask, or a
 * host loop in which a cudaMalloc is unacceptable because it synchronises the whole device.  The
 * scratch memory is a fixed array of EAGLE2_EXPAND_STATIC_BYTES that is part of the library image:
 * every GPU context that loads the library holds it until the process exits.
 *   - Sizes whose scratch need (what eagle2_workspace_bytes(EAGLE2_OP_EXPAND, B, V, k, ...) reports:
 *     the larger of the first step's and the later steps' need, so every step s of one tree gets the
 *     same answer) exceeds EAGLE2_EXPAND_STATIC_BYTES are refused with EAGLE2_ERR_STATIC_LIMIT;
 *     nothing is launched.  The call itself never allocates or frees device memory.
 *   - The first call on a device looks up the array's device address (one runtime query, made with
 *     that device current); make that first call outside any stream capture.  The address is kept
 *     per device ordinal for the life of the process: a process that destroys the device's context
 *     (cudaDeviceReset) must not call this entry point on that device afterwards.
 *   - All calls on a device share the one array.  Each call clears the few counters that must
 *     start at zero, on `stream`, before its kernel.  Two calls that can run on the GPU at the same
 *     time (different streams, no dependency) would overwrite each other's partial results: order
 *     them, or give one of them eagle2_expand with its own workspace.
 */
#define EAGLE2_EXPAND_STATIC_BYTES (1 << 20)
int eagle2_expand_static(const float* draft_logits, long long batch_stride, int B, int V, int k, int D,
                         int s, int32_t* tree_token, int32_t* tree_parent, double* tree_value,
                         int32_t* frontier, int32_t* d_status, eagle2_stream_t stream);

/*
 * Step 2a -- reranking (paper Section 4.2): the n_sel = min(m, N) nodes with the highest value among
 * ALL candidates, equal values preferring the shallower (lower-index) node, which keeps the set
 * closed under parents.  Values are clamped to the parent's effective value first, which changes
 * nothing for trees made by eagle2_expand and keeps closure for arbitrary values.  The selection is
 * flattened in ascending candidate index.
 *   sel_index [B][m] candidate index, sel_parent [B][m] flat position of the parent (-1: root),
 *   sel_token [B][m], sel_depth [B][m] (level - 1), n_sel [B].  Rows >= n_sel are padding
 *   (index -1, parent -1, token 0, depth 0).
 * Limits: 1 <= m <= EAGLE2_MAX_M, N <= EAGLE2_MAX_NODES.  Needs no workspace.
 */
int eagle2_rerank(const int32_t* tree_token, const int32_t* tree_parent, const double* tree_value,
                  int B, int k, int D, int m, int32_t* sel_index, int32_t* sel_parent,
                  int32_t* sel_token, int32_t* sel_depth, int32_t* n_sel, int32_t* d_status,
                  eagle2_stream_t stream);

/*
 * Step 2a without the reranking (paper Section 5.2, the ablation "without reranking").  The paper does
 * not list the nodes verified in that case; the reading taken here is the selection the expansion
 * phase made by itself: the frontier of every step, k nodes per step and at most kD in all, which is
 * a connected tree.  They are the nodes that some node names as its parent, plus the last step's
 * frontier, which the caller passes (the array eagle2_expand left after step D-1).  If there are
 * more than m, the m lowest indices (shallowest levels) are kept.  Outputs, padding, limits and
 * status bits are those of eagle2_rerank; n_sel[b] = min(m, number of such nodes); a frontier entry
 * outside [0, N) raises EAGLE2_STATUS_BAD_TREE and is skipped.  tree_value is read only for the NaN
 * check.
 *   frontier  int32 [B][k]
 */
int eagle2_rerank_skipped(const int32_t* tree_token, const int32_t* tree_parent, const double* tree_value,
                          const int32_t* frontier, int B, int k, int D, int m, int32_t* sel_index,
                          int32_t* sel_parent, int32_t* sel_token, int32_t* sel_depth, int32_t* n_sel,
                          int32_t* d_status, eagle2_stream_t stream);

/*
 * Step 2b -- tree attention mask and position ids (paper Section 4.2: a draft token sees only its
 * ancestors).  Row i of the mask has bit i and the bits of all ancestors of flat node i set; padding
 * rows have only their own bit.  pos_ids = kv_len + depth (the root is the last committed token).
 *   mask_bits  uint64 [B][m][ceil(m/64)], bit j of row i = token i sees token j.
 *   mask_dense uint8 [B][m][m], optional (NULL to skip).
 *   pos_ids    int32 [B][m].
 */
int eagle2_tree_mask(const int32_t* sel_parent, const int32_t* sel_depth, const int32_t* n_sel,
                     const int32_t* kv_len, int B, int m, uint64_t* mask_bits, uint8_t* mask_dense,
                     int32_t* pos_ids, int32_t* d_status, eagle2_stream_t stream);

/*
 * Steps 2a and 2b in one launch (paper Section 4.2): eagle2_rerank followed by eagle2_tree_mask on
 * its selection, with the same outputs, limits and status bits as the two calls; the block that has
 * chosen a sequence's nodes writes their mask rows and position ids itself.
 */
int eagle2_rerank_mask(const int32_t* tree_token, const int32_t* tree_parent, const double* tree_value,
                       const int32_t* kv_len, int B, int k, int D, int m, int32_t* sel_index, int32_t* sel_parent,
                       int32_t* sel_token, int32_t* sel_depth, int32_t* n_sel, uint64_t* mask_bits,
                       uint8_t* mask_dense, int32_t* pos_ids, int32_t* d_status, eagle2_stream_t stream);

/* Kernels one eagle2_tree_attention call launches at these sizes (bookkeeping for benchmarks and
 * graph builders; 0 for sizes the call would refuse): the attention kernel, a list kernel in front
 * of it when a ragged batch is served longest first, and a merge kernel behind it when the splits of
 * a sequence are not combined inside the attention kernel. */
int eagle2_tree_attention_launches(int B, int m, int Hq, int Hkv, int d, int max_kv_len);

/*
 * Step 3 -- tree-masked attention of the verification pass (paper Section 4.2), one layer per call:
 *   out[b,i,h,:] = sum_j softmax_j(scale * q[b,i,h,:].k[j,h/g,:]) v[j,h/g,:]
 * over the keys token i may see: every committed cache row [0, kv_len[b]) of its sequence and the
 * tree rows j whose bit is set in mask row i.  bf16 operands, fp32 accumulation, bf16 result.
 *   q        bf16 [B][m][Hq][d]
 *   k_cache, v_cache  bf16 [cache_rows][Hkv][d]; sequence b owns rows kv_off[b] ..
 *            kv_off[b]+kv_len[b]+m-1, the K/V of tree token j at local row kv_len[b]+j.
 *   cache_rows [host value] rows allocated in k_cache and in v_cache.  The kernel streams whole
 *            128-row tiles, so it may read (and ignore) rows of the allocation that follow a
 *            sequence's last key; rows at or beyond cache_rows are never touched.
 *   kv_off   int64 [B], kv_len int32 [B], mask_bits as written by eagle2_tree_mask.
 *            A launch for a single sequence reads kv_off and kv_len before it waits for the kernel
 *            ahead of it in the stream: they must not be written by a kernel that lets its
 *            dependents start before it completes (programmatic dependent launch with an early
 *            trigger).  Ordinary kernels and copies, and eagle2_kv_compact's own update, are fine.
 *   out      bf16 [B][m][Hq][d];  lse fp32 [B][Hq][m], optional natural-log sum of exponentials.
 *   max_kv_len [host value] upper bound of kv_len[], used to size the launch and the workspace.
 * A sequence with kv_len outside [0, max_kv_len] or whose rows do not fit in cache_rows raises
 * EAGLE2_STATUS_KV_OVERFLOW and its output rows are left untouched.
 * Limits: d in {64,128}; Hq % Hkv == 0 with Hq/Hkv <= 8; scale > 0; cache_rows < 2^31; 16-byte
 * aligned q, caches and out.
 */
int eagle2_tree_attention(const void* q, const void* k_cache, const void* v_cache, long long cache_rows,
                          const int64_t* kv_off, const int32_t* kv_len, const uint64_t* mask_bits,
                          int B, int m, int Hq, int Hkv, int d, int max_kv_len, float scale, void* out,
                          float* lse, void* ws, size_t ws_bytes, int32_t* d_status,
                          eagle2_stream_t stream);

/*
 * Step 4 -- acceptance (paper Section 2.1 rule, walked over the tree as in Section 2.2).
 * Rows of target_logits: row 0 belongs to the root, row 1+x to flat node x.  The children of a node
 * are the selected nodes whose sel_parent is that node, in ascending flat position.
 *   temperature == 0: follow the child whose token is the arg-max (lowest id on ties) of the target
 *     row of the current node; the extra token is the arg-max at the node where the walk stops.
 *   temperature  > 0: at the current node p = softmax(target/T), q = softmax(draft/T) with the draft
 *     row that produced the node's children; child x is accepted iff u_accept[x] < min(1, p(x)/q(x));
 *     after a rejection p <- norm(max(p-q,0)) and q loses the rejected token and is renormalised.
 *     With draft_logits_all == NULL the proposal is the point mass on the candidate (accept with
 *     probability p(x), then remove x from p), which is lossless for deterministic top-k children.
 *     The extra token is drawn from the p in force when the walk stops, by inverse CDF in ascending
 *     token id: the first t with sum_{v<=t} p(v) > u_bonus * sum_v p(v).
 *   target_logits     fp32 [B][m+1][V], sequence stride t_stride elements (0 shares one set).
 *   draft_logits_all  fp32 [B][R][V], stride d_stride; may be NULL (see above).
 *   u_accept fp32 [B][m] indexed by flat node, u_bonus fp32 [B], both in [0,1); unused at T == 0.
 *   acc_len [B] accepted draft tokens, acc_path [B][D] their flat positions (-1 padded),
 *   bonus_token [B].
 */
int eagle2_accept(const float* target_logits, long long t_stride, const float* draft_logits_all,
                  long long d_stride, const int32_t* sel_index, const int32_t* sel_parent,
                  const int32_t* sel_token, const int32_t* n_sel, int B, int V, int k, int D, int m,
                  float temperature, const float* u_accept, const float* u_bonus, int32_t* acc_len,
                  int32_t* acc_path, int32_t* bonus_token, void* ws, size_t ws_bytes,
                  int32_t* d_status, eagle2_stream_t stream);

/*
 * Step 5 -- KV compaction (paper Section 2.1: rejected draft tokens are discarded; Appendix A: the
 * cache is pre-allocated).  For every layer, K and V, the accepted tree rows move to the front of
 * the tree region: local row kv_len+acc_path[j] -> kv_len+j for j < acc_len, then kv_len += acc_len.
 *   k_layers, v_layers  device arrays of n_layers device pointers to bf16 [rows][Hkv][d] caches.
 *   kv_len in/out.  acc_path must be strictly increasing with acc_path[j] >= j (a root path in
 *   topological order); otherwise EAGLE2_STATUS_BAD_TREE is raised and that sequence is left alone.
 * Limits: Hkv*d*2 bytes per row a multiple of 16; D <= 16.
 */
int eagle2_kv_compact(void* const* k_layers, void* const* v_layers, int n_layers,
                      const int64_t* kv_off, int32_t* kv_len, const int32_t* acc_path,
                      const int32_t* acc_len, int B, int m, int D, int Hkv, int d, int32_t* d_status,
                      eagle2_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* EAGLE2_H_ */
