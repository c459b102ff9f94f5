/*
 * mirror.h -- C ABI of the B200 (sm_100a) library for the target-side verify step of
 * Mirror Speculative Decoding.
 *
 * One verify step scores a token tree of draft proposals hanging off the last committed token
 * (the hypothesis tree T_t of Sec. 3.1: kappa branches x gamma lookahead tokens) with the target
 * model and decides what to commit:
 *
 *   mirror_attn_verify    branch-tree attention of every tree node against the paged KV cache of
 *                         the verified prefix plus the tree's own K/V under the branch-causal mask
 *                         (each branch is scored as if decoded alone: "verifies left-to-right", Eq. 3)
 *   mirror_lmhead_reduce  logits = W h (the output head of Eq. 1; applied to an intermediate state it
 *                         is the early-exit proxy of Eq. 5) fused with per-row argmax / log-sum-exp /
 *                         Top-kappa (ids + log-probabilities: the token-channel message of Eq. 6)
 *   mirror_accept_select  acceptance operator of Eq. 3 / Eq. 10 per branch (greedy), or the standard
 *                         speculative-sampling rule (Sec. 3.1) with residual resampling; the longest
 *                         accepted branch, the correction / bonus token, and the reuse lookup of
 *                         Sec. 3.1 ("Verification vs. reuse criterion")
 *   mirror_verify_step    the three chained on one stream
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless its comment says "host".  The caller owns every buffer;
 *     inputs are never written.  bf16 tensors are passed as `const void*`.
 *   - All compute calls only enqueue work on `stream` (a cudaStream_t passed as void*) and return without
 *     synchronising.  Host-side argument errors are returned immediately; device-side problems (a bounded
 *     wait that ran out, an index outside its table) set a status word read by mirror_device_status().
 *   - The library allocates device memory only inside mirror_create() (one status word).  Scratch memory
 *     is a caller-provided workspace, sized by mirror_workspace_bytes() and attached with
 *     mirror_set_workspace(); its contents need not survive between calls but two calls that use the
 *     same ctx must not overlap on the GPU.
 *   - Token tree: node 0 is the root (the last committed token, whose row verifies every branch's first
 *     token); parent[i] < i.  A "branch" is a root-to-leaf path, leaves taken in increasing node order.
 *     Row r of any [batch*n_nodes, ...] tensor is (request r / n_nodes, node r % n_nodes): the target's
 *     distribution for the token that follows that node.
 *   - Ties: argmax and Top-kappa prefer the lowest token id; branch selection the lowest branch index.
 */
#ifndef MIRROR_H_
#define MIRROR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct mirror_ctx mirror_ctx;

typedef enum {
    MIRROR_OK = 0,
    MIRROR_ERR_ARG = 1,          /* null pointer / negative size */
    MIRROR_ERR_SHAPE = 2,        /* inconsistent or out-of-range dimensions */
    MIRROR_ERR_UNSUPPORTED = 3,  /* head_dim not in {64,128}, page_size != 16, device is not sm_100, ... */
    MIRROR_ERR_WORKSPACE = 4,    /* workspace missing or too small */
    MIRROR_ERR_CUDA = 5,         /* a CUDA runtime / driver call failed */
    MIRROR_ERR_DEVICE_CHECK = 6, /* device-side bounds check tripped (reported by mirror_device_status) */
    MIRROR_ERR_TIMEOUT = 7       /* a bounded device-side wait expired (reported by mirror_device_status) */
} mirror_status;

#define MIRROR_MAX_NODES 128     /* tree nodes per request, root included */
#define MIRROR_MAX_BRANCHES 64   /* root-to-leaf paths */
#define MIRROR_MAX_DEPTH 32      /* nodes on a path below the root (gamma) */
#define MIRROR_MAX_TOPK 32

typedef struct {
    int hidden;            /* H: width of the rows fed to the LM head */
    int n_q_heads;         /* Hq */
    int n_kv_heads;        /* Hkv, divides Hq */
    int head_dim;          /* d: 64 or 128 */
    int vocab;             /* |V| */
    int page_size;         /* tokens per KV page: 16 */
    float softmax_scale;   /* attention score scale; 0 selects 1/sqrt(head_dim) */
    float temperature;     /* T > 0: probabilities are Softmax(logits / T); 0 selects 1.  Greedy ignores it. */
} mirror_model_desc;

typedef struct {
    int batch;             /* B independent requests, all with the same tree shape */
    int n_nodes;           /* n <= MIRROR_MAX_NODES, root included */
    int kappa;             /* branches of the canonical tree (used when parent == NULL) */
    int gamma;             /* maximum branch length; width of the per-request outputs */
    const int32_t* tokens; /* device [B, n]: token id of each node (node 0: last committed token) */
    const int32_t* parent; /* HOST [n], parent[0] = -1, parent[i] < i; NULL selects the canonical comb:
                              branch i = chain of nodes 1+i*gamma .. 1+i*gamma+gamma-1 (n = 1+kappa*gamma) */
} mirror_tree;

typedef struct {
    const void* k_pool;        /* device bf16 [num_layers][num_pages, Hkv, page_size, d] */
    const void* v_pool;        /* same layout */
    int64_t layer_stride;      /* elements between consecutive layers' pools; a multiple of Hkv*page_size*d */
    int num_layers;
    int num_pages;             /* pages in one layer's pool */
    int max_pages_per_req;
    const int32_t* page_table; /* device [B, max_pages_per_req]: physical page of each logical page (shared by layers) */
    const int32_t* prefix_len; /* device [B]: verified-prefix length in tokens, <= max_pages_per_req*page_size */
} mirror_kv;

typedef enum {
    MIRROR_ACCEPT_GREEDY = 0,        /* Eq. 3 / Eq. 10 on every branch, longest branch wins */
    MIRROR_ACCEPT_SPEC_SAMPLING = 1, /* speculative-sampling rule on every branch independently, longest wins */
    MIRROR_ACCEPT_SPEC_TREE = 2      /* lossless rule over the tree: sequential rejection over siblings (below) */
} mirror_accept_mode;

typedef struct {
    mirror_accept_mode mode;
    int emit_bonus;               /* 1: when a whole branch is accepted also emit the token of its last row */
    const int32_t* target_argmax; /* [B*n]  greedy: the target's token for each row */
    const float* logits;          /* [B*n, V] fp32   spec sampling */
    const float* lse;             /* [B*n] fp32      spec sampling: log sum exp(logits / T) per row */
    const float* q_probs;         /* [B, n-1, V] fp32 spec sampling: draft distribution that proposed node i+1 */
    const float* u_accept;        /* [B, n] fp32 in [0,1): uniform of node c's accept test */
    const float* u_resample;      /* [B, n] fp32 in [0,1): uniform of the correction / bonus draw at row R */
    const int32_t* cand_ids;      /* nullable [B*n, n_cand]: ids the draft already expanded below each row
                                     (e.g. the early-exit Top-kappa of that row) for the reuse lookup */
    int n_cand;
} mirror_accept_in;

typedef struct {
    int32_t* n_accepted;     /* [B]   A: accepted draft tokens */
    int32_t* best_branch;    /* [B]   lowest branch index attaining A */
    int32_t* n_emitted;      /* [B]   A + 1 (A when a whole branch is accepted and emit_bonus == 0) */
    int32_t* emitted;        /* [B, gamma+1] accepted tokens then the correction / bonus token, -1 padded */
    int32_t* accepted_nodes; /* [B, gamma] node ids of the accepted tokens, -1 padded (for the caller's KV commit) */
    int32_t* decide_row;     /* [B]   node whose row produced the correction / bonus token */
    int32_t* reuse_slot;     /* [B]   index of that token in cand_ids[row], or -1 (fallback: fresh rollout) */
} mirror_accept_out;

/* What mirror_workspace_bytes should size for. */
#define MIRROR_WS_ATTN 1u           /* mirror_attn_verify */
#define MIRROR_WS_LMHEAD 2u         /* mirror_lmhead_reduce (M = batch * n_nodes rows) */
#define MIRROR_WS_LMHEAD_LOGITS 10u /* mirror_lmhead_reduce with a workspace that can hold the fp32 logits [M, V] */
#define MIRROR_WS_LMHEAD_TOPK 34u   /* mirror_lmhead_reduce with topk > 0, mirror_early_exit_tap.  Up to 256 rows the Top-kappa is
                                       selected inside the GEMM's epilogue: candidate lists instead of an [M, V] buffer; with more
                                       rows this sizes like MIRROR_WS_LMHEAD_LOGITS (the selection reads spilled logits) */
#define MIRROR_WS_STEP_GREEDY 7u    /* mirror_verify_step, greedy */
#define MIRROR_WS_STEP_SPEC 15u     /* mirror_verify_step, speculative sampling (holds the fp32 logits) */
#define MIRROR_WS_ACCEPT_TREE 16u   /* adds the fp64 scratch of MIRROR_ACCEPT_SPEC_TREE (optional: without it the rule
                                       re-evaluates the running distribution instead of storing it, which is slower) */
#define MIRROR_WS_STEP_TREE 31u     /* mirror_verify_step, MIRROR_ACCEPT_SPEC_TREE */

/* Create a context for one model shape on CUDA device `device` (made current for the call).
 * Allocates one device status word.  Fails with MIRROR_ERR_UNSUPPORTED on a device that is not sm_100. */
mirror_status mirror_create(mirror_ctx** out, const mirror_model_desc* desc, int device);
mirror_status mirror_destroy(mirror_ctx* ctx);

/* Bytes of workspace needed for the calls selected by `what` (OR of MIRROR_WS_*) on this tree / cache
 * shape.  `tree` and `kv` are read for their sizes only (pointers inside may be NULL). */
mirror_status mirror_workspace_bytes(const mirror_ctx* ctx, const mirror_tree* tree, const mirror_kv* kv,
                                     unsigned what, size_t* bytes);
/* Attach a device workspace (256-byte aligned).  The ctx keeps the pointer, not the memory. */
mirror_status mirror_set_workspace(mirror_ctx* ctx, void* dev_ptr, size_t bytes);

/* Branch-tree attention for all layers of `kv` (a1 + a2 of the verify step).
 *   q      bf16 [L, B, n, Hq, d]   queries of the tree nodes (already position-encoded)
 *   k_new  bf16 [L, B, n, Hkv, d]  this step's keys of the tree nodes;  v_new likewise
 *   out    bf16 [L, B, n, Hq, d]   softmax(scale * q k^T over Vis(node)) v, with
 *                                  Vis(node) = verified prefix  U  {node and its ancestors}
 *   lse_out fp32 [L, B, Hq, n], nullable: natural-log softmax denominator of each row
 * Needs a workspace sized for MIRROR_WS_ATTN. */
mirror_status mirror_attn_verify(mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree,
                                 const void* q, const void* k_new, const void* v_new,
                                 void* out, float* lse_out, void* stream);

/* The same attention over an 8-bit cache.  The paper states no storage precision for the target's cache (Sec. 3,
 * Eq. 1); this mode is the library's own option and halves the bytes the step reads.  Its definition:
 *   kv->k_pool, kv->v_pool, k_new, v_new hold e4m3 codes (one byte per element; same shapes, kv->layer_stride counts
 *   elements), value = code * scale[layer, KV head] with k_scale, v_scale: device fp32 [L, Hkv];
 *   the queries enter as q8 = q_scale * e4m3(q / q_scale) (q stays bf16 in memory; q_scale: host fp32 > 0, one for
 *   the call, e.g. max|q| / 448; fp32 division, round to nearest even, saturating);
 *   out = softmax(scale * q8 (k_scale K)^T) (v_scale V) over the same visible set.
 * Inside, the unnormalised softmax weights are rounded to e4m3 too (both operands of an 8-bit tensor-core product are
 * 8-bit), relative to a running offset per row: weights below 2^-12 of it round to zero; the row sum, and so lse_out,
 * is taken before that rounding.  Head dimension 128 only (MIRROR_ERR_UNSUPPORTED otherwise); q, out, lse_out and
 * the workspace as for mirror_attn_verify. */
mirror_status mirror_attn_verify_fp8(mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree, const void* q,
                                     const void* k_new_fp8, const void* v_new_fp8, const float* k_scale,
                                     const float* v_scale, float q_scale, void* out, float* lse_out, void* stream);

/* Scales and codes of a bf16 K or V tensor for that cache.  The tensor is addressed as [layer][...][head][inner]:
 * `inner` consecutive elements (a multiple of 8) belong to one KV head -- page_size * d for a pool, d for the tree's
 * own k_new / v_new -- and heads cycle above that; `layer_elems` elements of each layer are in use, layers are
 * `layer_stride` elements apart (codes are written at the same element offsets).
 *   mirror_kv_scales_fp8:   scale[layer, head] = max|x| / 448 over the layer's and head's elements (1 if all zero)
 *   mirror_kv_quantize_fp8: code = e4m3(x / scale[layer, head]), fp32 division, round to nearest even, saturating
 * x: device bf16, 16-byte aligned; scale: device fp32 [n_layers, Hkv]; out_fp8: device bytes, 8-byte aligned. */
mirror_status mirror_kv_scales_fp8(mirror_ctx* ctx, const void* x, int n_layers, int64_t layer_stride, int64_t layer_elems,
                                   int inner, float* scale, void* stream);
mirror_status mirror_kv_quantize_fp8(mirror_ctx* ctx, const void* x, int n_layers, int64_t layer_stride,
                                     int64_t layer_elems, int inner, const float* scale, void* out_fp8, void* stream);

/* LM head with fused row reductions: logits[r][v] = sum_k hidden[r][k] * W[v][k]  (Eq. 1, Eq. 5).
 *   hidden bf16 [M, H] (row stride H);  W bf16 [V, H]
 *   argmax   int32 [M]  lowest id attaining the maximum          (nullable)
 *   maxlogit fp32 [M]   that maximum                              (nullable)
 *   lse      fp32 [M]   log sum_v exp(logits/T)                   (nullable)
 *   topk > 0: topk_id int32 [M, topk], topk_logprob fp32 [M, topk] = logits/T - lse, ordered by
 *             (logit descending, id ascending): the Top-kappa message of Eq. 6.  topk <= MIRROR_MAX_TOPK.
 *   gather_row/gather_tok int32 [n_gather] -> gather_logit fp32 [n_gather] = logits[row][tok]  (nullable)
 *   logits_out fp32 [M, V], nullable: the full logits (needed by speculative sampling)
 * Needs a workspace sized for MIRROR_WS_LMHEAD; with topk > 0 one sized for MIRROR_WS_LMHEAD_TOPK: with up to 256 rows the
 * Top-kappa is then selected inside the GEMM's epilogue (sorted lists per epilogue warp and row that live as long as the
 * CTA, merged afterwards) and the logits never reach memory; with more rows the selection runs over spilled fp32 logits. */
mirror_status mirror_lmhead_reduce(mirror_ctx* ctx, const void* hidden, int M, const void* W, int topk,
                                   const int32_t* gather_row, const int32_t* gather_tok, int n_gather,
                                   int32_t* argmax, float* maxlogit, float* lse,
                                   int32_t* topk_id, float* topk_logprob, float* gather_logit,
                                   float* logits_out, void* stream);

/* Low-precision LM head (Eq. 1 / Eq. 5 with quantised operands; the paper states no precision for the LM head:
 * an opt-in mode for the weight stream, the bf16 head stays the default).
 * mirror_quantize_rows_fp8: x bf16 [rows, cols] (device) -> out_fp8 [rows, cols] e4m3 bytes and out_scale [rows] fp32 with
 *   scale = max|x_row| / 448 (1 for an all-zero row) and code = e4m3(x / scale), round to nearest even (fp32 division).
 *   Use it once for W [V, H] (one scale per vocabulary row) and per step for the hidden rows.
 * mirror_lmhead_reduce_fp8: logits[r, v] = w_scale[v] * h_scale[r] * sum_k W8[v, k] * h8[r, k] (exact e4m3 products,
 *   fp32 accumulation on the tensor cores), then argmax (ties -> lowest id), max and lse = log sum exp(logits / T) as in
 *   mirror_lmhead_reduce; logits_out nullable fp32 [M, V].  hidden must be a multiple of 128; 16-byte aligned pointers.
 *   Needs a workspace sized for MIRROR_WS_LMHEAD.  Outputs nullable. */
mirror_status mirror_quantize_rows_fp8(mirror_ctx* ctx, const void* x, int rows, int cols, void* out_fp8, float* out_scale,
                                       void* stream);
mirror_status mirror_lmhead_reduce_fp8(mirror_ctx* ctx, const void* hidden_fp8, const float* h_scale, int M, const void* W_fp8,
                                       const float* w_scale, int32_t* argmax, float* maxlogit, float* lse, float* logits_out,
                                       void* stream);

/* LM head with fused argmax / max / log-sum-exp for callers that must not allocate device memory
 * (the paper has no counterpart: this is a deployment variant of mirror_lmhead_reduce, same kernels).
 * Who needs it: a host that has given all device memory to its own pool, a plugin called inside an
 * allocator-guarded region, or any code path where cudaMalloc is forbidden.  No context and no workspace:
 * the kernel's scratch (one partial per CTA and row, two CTAs per SM) is a fixed array inside the library image,
 * 491,776 bytes on every GPU that loads the library, held until the process exits.
 *   device       CUDA device ordinal (made current for the call)
 *   hidden, W    bf16 [M, H] and [V, H] as in mirror_lmhead_reduce; H a multiple of 64
 *   M            at most 128 rows; more returns MIRROR_ERR_SHAPE (use mirror_lmhead_reduce with a workspace)
 *   temperature  T > 0 (0 selects 1): lse = log sum exp(logits / T)
 *   argmax, maxlogit, lse   device [M] outputs, each nullable
 * Calls no cudaMalloc / cudaFree and no allocating library routine.  The first call on a device resolves the
 * scratch array's device address (cudaGetSymbolAddress) and the tensor-map encoder; make that first call
 * before any stream capture begins.  Every call on a device shares the one scratch array: calls that
 * overlap on the GPU (different streams, no ordering) race on it and give wrong results -- order them.
 * The partials are rewritten by every call before they are read.  A device-side problem (a bounded wait that ran
 * out) is recorded in the array's first words and kept until mirror_lmhead_noalloc_status asks for it; the
 * outputs of such a call are not valid.  The one-time set-up is guarded, so first calls may come from any thread. */
mirror_status mirror_lmhead_reduce_noalloc(int device, const void* hidden, int M, const void* W, int V, int H,
                                           float temperature, int32_t* argmax, float* maxlogit, float* lse,
                                           void* stream);

/* Device-side status of the mirror_lmhead_reduce_noalloc calls made on `device` (they have no context to ask;
 * the paper has no counterpart): synchronises the device, returns in *code the first problem since the last query
 * (MIRROR_OK, MIRROR_ERR_TIMEOUT or MIRROR_ERR_DEVICE_CHECK) with a detail word in *detail (nullable), and clears it.
 * Allocates nothing. */
mirror_status mirror_lmhead_noalloc_status(int device, int* code, int* detail);

/* Acceptance, branch selection, emitted tokens and reuse lookup (a5 + a6).
 * Greedy (Eq. 3 / Eq. 10): branch length a = number of leading nodes c with tokens[c] == target_argmax[parent(c)].
 * Speculative sampling: node c (token x, parent row r) passes iff u_accept[c] * q_c[x] <= p_r[x] with
 * p_r[v] = exp(logits[r][v]/T - lse[r]), evaluated in fp64; the extra token is drawn by inverse CDF with
 * u_resample[R] from the normalised residual max(0, p_R - q_c') of the first rejected node c' of the chosen
 * branch, or from p_R when the whole branch was accepted (or the residual has no mass).
 * Selecting the longest of several independently tested branches is distribution-preserving only for a
 * single branch.
 * MIRROR_ACCEPT_SPEC_TREE (same inputs; tree drafts, Sec. 3.1's rule applied to sibling sets): walk down from the
 * root; at row r the current distribution m starts as p_r, the children of r are tested in node order, child c
 * (token x) passes iff u_accept[c] * q_c[x] <= m[x] and the walk moves to c; a child that fails turns m into the
 * normalised residual max(0, m - q_c) (left as it is when that residual has no mass).  When every child of r has
 * failed -- or r is a leaf and emit_bonus is set -- the extra token is drawn from m by inverse CDF with
 * u_resample[r].  If the siblings of each node are independent draws from one q, the emitted tokens are distributed
 * exactly as the target's own samples for any tree.  best_branch is the lowest-index branch that contains the
 * accepted path.  All decision arithmetic is fp64. */
mirror_status mirror_accept_select(mirror_ctx* ctx, const mirror_tree* tree, const mirror_accept_in* in,
                                   const mirror_accept_out* out, void* stream);

/* Early-exit tap (Sec. 3.1, Eq. 5 and Eq. 6): the LM head applied to the hidden states of an intermediate layer,
 * reduced per row to the Top-kappa message M_t that the token channel carries to the draft.
 *   hidden_le        bf16 [M, H]: early-exit hidden rows (one per window position / tree node)
 *   msg_ids          int32 [M, kappa]: candidate ids ordered by (logit descending, id ascending)
 *   msg_logprob_bf16 bf16 [M, kappa]: their log-probabilities logit/T - lse under the early-exit proxy (the token
 *                    channel's payload type)
 * kappa <= MIRROR_MAX_TOPK.  Needs a workspace sized for MIRROR_WS_LMHEAD_TOPK with M rows (up to 256 rows the selection
 * happens in the GEMM's epilogue and there is no [M, V] buffer).  msg_ids is what mirror_accept_select / mirror_verify_step take as cand_ids (n_cand =
 * kappa) for the reuse decision of the same rows. */
mirror_status mirror_early_exit_tap(mirror_ctx* ctx, const void* hidden_le, int M, const void* W, int kappa,
                                    int32_t* msg_ids, void* msg_logprob_bf16, void* stream);

/* Overlap mass (Eq. 7): omega[row] = sum over the row's kappa message ids y of q(y), with
 * q(y) = exp(logits_final[row][y]/T - lse_final[row]) the target's final distribution of that row; by Proposition 1,
 * 1 - omega is the probability that a rejection at the row falls back to a fresh rollout.
 *   logits_final fp32 [M, V], lse_final fp32 [M] (e.g. from mirror_lmhead_reduce with logits_out), msg_ids int32
 *   [M, kappa], omega fp32 [M] (device).  Ids outside [0, V) are skipped and reported as a device-side check. */
mirror_status mirror_overlap_mass(mirror_ctx* ctx, const float* logits_final, const float* lse_final,
                                  const int32_t* msg_ids, int M, int kappa, float* omega, void* stream);

/* Roll-forward of the paged cache after a verify step (Sec. 3.1): for every request b the K/V rows of the root
 * (node 0, the last committed token) and of its accepted nodes, in path order, are written as tokens
 * prefix_len[b] .. prefix_len[b] + n_accepted[b] of every layer and KV head, then prefix_len[b] += n_accepted[b] + 1.
 *   kv              the cache: k_pool / v_pool are WRITTEN here (the struct's const is not honoured by this call);
 *                   page_table must already hold pages for the new positions (it is not modified);
 *                   kv->prefix_len is ignored in favour of the prefix_len argument
 *   k_new, v_new    bf16 [L, B, n, Hkv, d]: the tree's own K/V of the step just verified
 *   accepted_nodes  int32 [B, gamma], n_accepted int32 [B]: as written by mirror_accept_select / mirror_verify_step
 *   prefix_len      int32 [B], device, read and updated in place
 * A position beyond max_pages_per_req*16, a page outside the pool or a node id outside the tree is skipped and
 * reported through mirror_device_status.  Enqueues two small kernels; runs after the step on the same stream. */
mirror_status mirror_kv_commit(mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree, const void* k_new,
                               const void* v_new, const int32_t* accepted_nodes, const int32_t* n_accepted,
                               int32_t* prefix_len, void* stream);
/* The same roll-forward of an e4m3 cache (see mirror_attn_verify_fp8): pools, k_new_fp8 and v_new_fp8 hold codes, one
 * byte per element, already under the cache's scales (mirror_kv_quantize_fp8); d must be a multiple of 16. */
mirror_status mirror_kv_commit_fp8(mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree, const void* k_new_fp8,
                                   const void* v_new_fp8, const int32_t* accepted_nodes, const int32_t* n_accepted,
                                   int32_t* prefix_len, void* stream);

/* HOST helper (no device work): merge kappa branches of gamma tokens -- the branch-complete proposal of Sec. 3.1 --
 * into a token tree without duplicated prefixes ("tree drafts"): branches that agree on their first r tokens share
 * their first r nodes, so shared tokens are scored once.  All pointers are HOST pointers.
 *   branch_tokens int32 [kappa, gamma]; root_token: the last committed token (node 0)
 *   parent, tokens int32 [1 + kappa*gamma] (capacity; *n_nodes entries are written): node ids in order of first
 *                  appearance, parent[i] < i -- the arrays mirror_tree takes (tokens go to the device per request)
 *   node_of        int32 [kappa, gamma]: the node that holds position j of branch i
 * kappa <= MIRROR_MAX_BRANCHES, gamma <= MIRROR_MAX_DEPTH, at most MIRROR_MAX_NODES nodes (else MIRROR_ERR_SHAPE). */
mirror_status mirror_trie_build(const int32_t* branch_tokens, int kappa, int gamma, int32_t root_token, int32_t* parent,
                                int32_t* tokens, int32_t* node_of, int* n_nodes);

/* One whole verify step on one stream: attention over all layers -> LM head rows -> reductions -> acceptance.
 *   hidden   bf16 [B*n, H], or NULL to feed the last layer's attention output (requires Hq*d == H)
 *   attn_out bf16 [L, B, n, Hq, d]  (required: it is also the chained LM-head input)
 *   acc      mode, emit_bonus, q_probs, u_accept, u_resample, cand_ids are read; target_argmax / logits / lse
 *            are produced internally (in the workspace)
 *   argmax_out int32 [B*n], nullable: the target's greedy token per row, for inspection
 * Needs a workspace sized for MIRROR_WS_STEP_GREEDY or MIRROR_WS_STEP_SPEC. */
mirror_status mirror_verify_step(mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree,
                                 const void* q, const void* k_new, const void* v_new,
                                 const void* hidden, const void* W, const mirror_accept_in* acc,
                                 const mirror_accept_out* out, void* attn_out, int32_t* argmax_out,
                                 void* stream);

/* ------------------------------------------------------------------------------------------------------------
 * The target's layers around the verify attention (the "target forward" of Sec. 3.1 that runs between the early
 * exit and the final verification; Sec. 4.1 names pre-norm decoder stacks as targets).  The paper fixes no layer
 * structure; this is the common pre-norm decoder layer: RMSNorm -> Q/K/V projection -> rotary embedding
 * (rotate-half pairs i, i + d/2; angle = position * rope_theta^(-2i/d)) -> mirror_attn_verify for that layer ->
 * output projection + residual -> RMSNorm -> SiLU(gate) * up -> down projection + residual.  Activations are stored
 * in bf16 between the steps; sums are fp32.  Row r = (request, node) sits at position prefix_len[request] + depth(node).
 * ------------------------------------------------------------------------------------------------------------ */
typedef struct {
    const void* w_qkv;      /* bf16 [(Hq + 2*Hkv)*d, H]: query rows, then key rows, then value rows */
    const void* w_o;        /* bf16 [H, Hq*d] */
    const void* w_gate_up;  /* bf16 [2*I, H]: gate rows, then up rows */
    const void* w_down;     /* bf16 [H, I] */
    const void* norm_attn;  /* bf16 [H]: RMSNorm weight ahead of attention */
    const void* norm_mlp;   /* bf16 [H]: RMSNorm weight ahead of the MLP */
} mirror_layer_weights;

typedef struct {
    int n_layers;                        /* layers to run; layer l uses kv layer l and k_new / v_new slab l */
    int intermediate;                    /* I, a multiple of 64 (H and Hq*d must be multiples of 64 too) */
    float rope_theta;                    /* e.g. 1e6 */
    float rms_eps;                       /* e.g. 1e-6 */
    const mirror_layer_weights* layers;  /* HOST array [n_layers] of device pointers */
    const void* norm_final;              /* bf16 [H]: RMSNorm weight ahead of the LM head */
} mirror_target;

/* out[M, N] (bf16) = x[M, K] (bf16) * W[N, K]^T (bf16) (+ residual[M, N], bf16, nullable), fp32 accumulation, one
 * rounding.  K a multiple of 64; x, W, out 16-byte aligned.  scratch: device memory of at least
 * mirror_linear_scratch_bytes() bytes (fp32 partial sums of the K slices the GEMM is split into when it has fewer
 * output tiles than the GPU has CTA pairs; the slices are added in a fixed order). */
mirror_status mirror_linear_scratch_bytes(const mirror_ctx* ctx, int M, int N, int K, size_t* bytes);
mirror_status mirror_linear(mirror_ctx* ctx, const void* x, int M, const void* W, int N, int K, const void* residual,
                            void* out, void* scratch, size_t scratch_bytes, void* stream);

/* out[r, :] = table[tokens[r], :] for the M rows of a step: the residual rows that enter layer 0.
 *   table bf16 [V, H] (V, H of the ctx; H a multiple of 8), tokens int32 [M] (device), out bf16 [M, H]
 * A token outside [0, V) zeroes its row and is reported through mirror_device_status. */
mirror_status mirror_embed_rows(mirror_ctx* ctx, const void* table, const int32_t* tokens, int M, void* out, void* stream);

/* out[M, H] (bf16) = x / sqrt(mean(x^2) + eps) * gamma, row by row (x bf16 [M, H], gamma bf16 [H]; H even). */
mirror_status mirror_rmsnorm(mirror_ctx* ctx, const void* x, const void* gamma, int M, int H, float eps, void* out,
                             void* stream);

/* All layers of `t` on the step's rows, one after the other on `stream`:
 *   x        bf16 [B*n, H]: the residual stream entering layer 0 (the embeddings of the tree's tokens); not written
 *   kv, tree as for mirror_attn_verify (kv->num_layers >= t->n_layers; cached keys are already rotated)
 *   q_out    bf16 [n_layers, B, n, Hq, d], k_new_out / v_new_out bf16 [n_layers, B, n, Hkv, d]: the projected and
 *            rotated queries and the tree's own K/V of every layer (k_new_out / v_new_out are what
 *            mirror_kv_commit appends afterwards)
 *   attn_out bf16 [n_layers, B, n, Hq, d]
 *   x_out    bf16 [B*n, H]: the residual stream after the last layer
 *   hidden_out bf16 [B*n, H]: RMSNorm(x_out) with norm_final -- the LM-head rows (`hidden` of mirror_verify_step /
 *            mirror_lmhead_reduce)
 *   scratch  device memory of at least mirror_target_scratch_bytes() bytes
 * Needs the workspace of mirror_attn_verify.  Per layer it enqueues 4 GEMMs, 4 fused finishing kernels (split-K sum
 * + rotary embedding / residual + RMSNorm / SiLU gate) and the two attention kernels. */
mirror_status mirror_target_scratch_bytes(const mirror_ctx* ctx, const mirror_tree* tree, const mirror_target* t,
                                          size_t* bytes);
mirror_status mirror_target_forward(mirror_ctx* ctx, const mirror_target* t, const mirror_kv* kv, const mirror_tree* tree,
                                    const void* x, void* q_out, void* k_new_out, void* v_new_out, void* attn_out,
                                    void* x_out, void* hidden_out, void* scratch, size_t scratch_bytes, void* stream);
/* The same layers over an e4m3 KV cache (see mirror_attn_verify_fp8; head dimension 128).  kv holds codes; k_scale and
 * v_scale are the cache's scales (device fp32 [n_layers, Hkv]); h_q_scale is a HOST array [n_layers] with one Q scale
 * per layer (e.g. from a calibration pass: max|q| / 448 with some head room; larger values saturate).  Every layer's new
 * K/V rows are written as bf16 (k_new_out, v_new_out, as before) and as codes under the cache's scales (k_new8_out,
 * v_new8_out: bytes [n_layers, B, n, Hkv, d], what mirror_kv_commit_fp8 appends); the layer's attention reads the codes.
 * Two more small kernels per layer. */
mirror_status mirror_target_forward_fp8(mirror_ctx* ctx, const mirror_target* t, const mirror_kv* kv, const mirror_tree* tree,
                                        const void* x, const float* k_scale, const float* v_scale, const float* h_q_scale,
                                        void* q_out, void* k_new_out, void* v_new_out, void* k_new8_out, void* v_new8_out,
                                        void* attn_out, void* x_out, void* hidden_out, void* scratch, size_t scratch_bytes,
                                        void* stream);

/* mirror_verify_step over an e4m3 KV cache: the attention is mirror_attn_verify_fp8's (kv, k_new_fp8, v_new_fp8, the
 * scales and q_scale as there; head dimension 128), everything behind it (attn_out in bf16, LM head, acceptance) is
 * unchanged. */
mirror_status mirror_verify_step_fp8(mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree, const void* q,
                                     const void* k_new_fp8, const void* v_new_fp8, const float* k_scale,
                                     const float* v_scale, float q_scale, const void* hidden, const void* W,
                                     const mirror_accept_in* acc, const mirror_accept_out* out, void* attn_out,
                                     int32_t* argmax_out, void* stream);

/* mirror_verify_step for callers whose step inputs live in HOST memory (pinned for the copies to be asynchronous):
 *   h_q bf16 [L, B, n, Hq, d], h_k_new / h_v_new bf16 [L, B, n, Hkv, d], h_tokens int32 [B, n]: HOST inputs of this step
 *   d_q, d_k_new, d_v_new: DEVICE staging buffers of the same shapes, and tree->tokens (device, written here);
 *                   they must not be in use by work on other streams
 *   h_out           HOST copies of the decision (any member may be NULL); valid once `stream` has been synchronised
 * Copies run on an internal stream (created on first use) and begin after all work already queued on `stream`.  The
 * layers' attention problems are independent and the LM head reads only the last layer's output, so the last layer is
 * copied and attended to first, the LM head and the acceptance follow, and the other layers arrive in up to eleven pieces
 * while the LM head runs; each is attended to once it has landed, after the decision has been sent back.
 * Everything else as in mirror_verify_step (attn_out holds all layers when `stream` has drained).  Does not synchronise. */
typedef struct {
    int32_t* n_accepted;   /* [B] */
    int32_t* best_branch;  /* [B] */
    int32_t* n_emitted;    /* [B] */
    int32_t* emitted;      /* [B, gamma + 1] */
} mirror_accept_host_out;
mirror_status mirror_verify_step_host(mirror_ctx* ctx, const mirror_kv* kv, const mirror_tree* tree, const void* h_q,
                                      const void* h_k_new, const void* h_v_new, const int32_t* h_tokens, void* d_q,
                                      void* d_k_new, void* d_v_new, const void* hidden, const void* W,
                                      const mirror_accept_in* acc, const mirror_accept_out* out,
                                      const mirror_accept_host_out* h_out, void* attn_out, void* stream);

/* Optional timing hooks for mirror_verify_step: four cudaEvent_t (passed as void*) that every later
 * mirror_verify_step on this ctx records on its stream -- before attention, after attention, after the
 * LM-head GEMM kernel, after acceptance -- until cleared with NULL.  The caller owns the events. */
mirror_status mirror_set_stage_events(mirror_ctx* ctx, void* const* events4);

/* Synchronises the device and returns the sticky device-side status (MIRROR_OK, MIRROR_ERR_TIMEOUT or
 * MIRROR_ERR_DEVICE_CHECK) in *code, with a detail word in *detail (nullable); then clears it. */
mirror_status mirror_device_status(mirror_ctx* ctx, int* code, int* detail);

/* Number of kernels the library has launched through this ctx since creation (for accounting). */
mirror_status mirror_launch_count(const mirror_ctx* ctx, long long* count);

const char* mirror_status_str(mirror_status s);

#ifdef __cplusplus
}
#endif
#endif /* MIRROR_H_ */
