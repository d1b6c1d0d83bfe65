/*
 * sparrow_attn.h -- C ABI of libsparrow_attn: the attention of one speculative decoding step of
 * Sparrow (video-LLM speculative decoding) on one NVIDIA B200 (sm_100a).
 *
 * Two modes:
 *   (a) verification -- T draft tokens arranged as a chain or tree attend over the target model's
 *       whole KV cache (visual + text prefix) plus their own ancestors.  The paper's Appendix A
 *       ("Speculative Decoding") and Section 4 ("Metrics") state that the target verifies all
 *       candidates of a (dynamic) draft tree in a single parallel forward pass and that the method
 *       is lossless, i.e. this is the target's ordinary softmax attention under the tree mask.
 *   (b) text-anchored window attention -- Eq. 2 (Section 3.1, VATA): Softmax(Q_t K_T^T/sqrt(d)) V_T
 *       with K_T, V_T restricted to the text-anchored positions T; the visual KV rows are never
 *       touched.  sparrow_anchor_attn_tree() is the same for a draft tree.
 * Around them, for a whole speculative step on the device: sparrow_kv_append(),
 * sparrow_compact_anchors() (row movers), sparrow_accept_greedy(), sparrow_accept_sample(),
 * sparrow_kv_keep_accepted() (acceptance of the draft tree at temperature 0 and 1, and the move of
 * the accepted rows).
 *
 * For every batch entry b, query head h (KV head h / g, g = n_q_heads / n_kv_heads query heads
 * per KV head; g = 7 for the paper's Qwen2-7B-shaped targets), draft token t and visible key set Vis:
 *     s_j = softmax_scale * <q[b,t,h,:], k[b,h/g,j,:]>,   lse = log sum_{j in Vis} exp(s_j),
 *     out = sum_{j in Vis} exp(s_j - lse) * v[b,h/g,j,:].
 *
 * Conventions
 *   - Every function returns a sparrow_status; nothing aborts or throws.  Argument errors are
 *     detected on the host before anything is launched.  Problems only the device can see (a
 *     malformed device-side parent array, an anchor index outside the buffer) set a sticky status
 *     word, read by sparrow_last_device_status(); the kernels always terminate, never read out of
 *     bounds, and treat a bad parent as "root" and a bad anchor row as "not visible".
 *   - "DEV" pointers are device memory of the context's GPU, "HOST" pointers are host memory.
 *   - The caller owns every buffer including the workspace; the library owns only the context.
 *   - The two attention calls allocate nothing, copy nothing from the host and do not
 *     synchronise: they enqueue kernels on `stream` and return.
 *   - bf16 tensors are passed as void*; element strides are in elements, not bytes.
 */
#ifndef SPARROW_ATTN_H_
#define SPARROW_ATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    SPARROW_OK            = 0,
    SPARROW_ERR_NULL      = 1,  /* a required pointer is NULL */
    SPARROW_ERR_SHAPE     = 2,  /* unsupported head geometry, T, batch, lengths, alignment */
    SPARROW_ERR_TREE      = 3,  /* parents[] is not a topologically ordered forest */
    SPARROW_ERR_ANCHOR    = 4,  /* anchor list not strictly increasing / out of range */
    SPARROW_ERR_WORKSPACE = 5,  /* workspace missing, misaligned or too small */
    SPARROW_ERR_CUDA      = 6,  /* a CUDA runtime / driver call failed */
    SPARROW_ERR_TIMEOUT   = 7,  /* a bounded device-side wait gave up */
    SPARROW_ERR_ARCH      = 8   /* the device is not compute capability 10.x */
} sparrow_status;

#define SPARROW_MAX_T      64   /* draft tokens per sequence (one 64-bit ancestor word per token) */
#define SPARROW_MAX_BATCH  64   /* sequences per call */
#define SPARROW_HEAD_DIM   128  /* only value accepted */
#define SPARROW_MAX_GQA_GROUP 16 /* query heads per KV head: 1 .. 16 (7 for the paper's Qwen2-7B-shaped targets) */

/* Fixed per context.  K/V buffers hold, for batch b and KV head g, `kv_capacity` rows of 128 bf16:
 * element offset of (b, g, row, d) = b*kv_stride_batch + g*kv_stride_head + row*128 + d.
 * Both strides must be multiples of 8 elements and the base pointers 16-byte aligned. */
typedef struct {
    int32_t batch;           /* 1 .. SPARROW_MAX_BATCH */
    int32_t n_q_heads;       /* g * n_kv_heads, 1 <= g <= SPARROW_MAX_GQA_GROUP */
    int32_t n_kv_heads;
    int32_t head_dim;        /* must be 128 */
    int32_t kv_capacity;     /* rows per (batch, KV head) */
    float   softmax_scale;   /* e.g. 1/sqrt(128); applied in fp32 to the fp32 scores */
    int64_t kv_stride_batch;
    int64_t kv_stride_head;
} sparrow_layout;

typedef struct sparrow_ctx sparrow_ctx;

/* Creates a context on CUDA device `device` (queries the SM count, loads the kernels).  With
 * SPARROW_LOG=1 in the environment the context prints one line per verification call on stderr
 * (the split plan and how the call is launched); SPARROW_NO_PDL=1 switches programmatic launch off.
 * SPARROW_ERR_ARCH unless the device is sm_100; SPARROW_ERR_CUDA when no usable device exists. */
sparrow_status sparrow_create(sparrow_ctx** ctx, const sparrow_layout* layout, int device);
sparrow_status sparrow_destroy(sparrow_ctx* ctx);

/* How sparrow_verify_attn() cuts the key range into work items (one CTA each; the paper says
 * nothing about scheduling, this is a property of this implementation).  Calls in fused mode
 * overlap their neighbours in the stream, so the number of items trades single-call latency
 * against sustained throughput of a stream of calls:
 *   LATENCY     one wave over all SMs (about n_sm items): shortest time for a call on an idle GPU;
 *   BALANCED    about 3/8 n_sm items (the default);
 *   THROUGHPUT  about n_sm / 7 items: longest pieces, several calls resident at once; best when
 *               many independent calls are queued back to back (one per layer or per request).
 * Results differ between policies only by the rounding order of the split-KV merge.  Calls that
 * cannot overlap (graph capture, SPARROW_NO_PDL, sparrow_anchor_attn, sparrow_verify_attn_static)
 * always use one wave over all SMs. */
typedef enum {
    SPARROW_PLAN_LATENCY    = 0,
    SPARROW_PLAN_BALANCED   = 1,
    SPARROW_PLAN_THROUGHPUT = 2
} sparrow_plan_policy;

/* Sets the policy for later calls (host state only; may be changed between any two calls).
 * SPARROW_ERR_SHAPE for an unknown value. */
sparrow_status sparrow_set_plan_policy(sparrow_ctx* ctx, int32_t policy);

/* enable != 0: single sparrow_verify_attn() calls of this context may start early too (see the
 * ordering rules at sparrow_verify_attn()).  Off by default.  Host state only. */
sparrow_status sparrow_set_call_overlap(sparrow_ctx* ctx, int32_t enable);

/* Work items the planner currently aims for in fused mode (pass it to sparrow_plan_splits() as
 * n_sm to see the schedule of a call).  0 when ctx is NULL. */
int32_t sparrow_plan_target_items(const sparrow_ctx* ctx);

/* Bytes of device scratch the calls need for draft blocks of up to max_T tokens (split-KV partial
 * outputs, the device status word, staging for the host-buffer entry point).  0 on bad arguments. */
size_t sparrow_workspace_bytes(const sparrow_ctx* ctx, int32_t max_T);
/* Registers caller-owned scratch (256-byte aligned, >= sparrow_workspace_bytes(max_T) for the
 * largest T that will be used).  Clears the device status word with a cudaMemset (synchronising).
 * Calls that share one workspace must be ordered on the GPU (same stream, or event dependencies). */
sparrow_status sparrow_set_workspace(sparrow_ctx* ctx, void* dev_ptr, size_t bytes);

/* (a) Verification attention (Appendix A; Section 4 "Metrics": tree-structured, lossless).
 *   q        DEV bf16 [batch][T][n_q_heads][128], dense
 *   k_cache,
 *   v_cache  DEV bf16, layout above; rows [0, kv_len[b]) are the committed prefix, rows
 *            [kv_len[b], kv_len[b]+T) already hold the T draft tokens' keys / values; rows past
 *            that may hold anything (including NaN patterns) and are ignored
 *   kv_len   HOST int32 [batch]; 0 <= kv_len[b], kv_len[b] + T <= kv_capacity
 *   parents  DEV int32 [batch][T]; parents[i] = parent node of draft token i, -1 for a root,
 *            parents[i] < i.  Token t sees the prefix, itself and its ancestors.
 *   T        1 .. SPARROW_MAX_T
 *   out      DEV bf16 [batch][T][n_q_heads][128]
 *   lse      DEV fp32 [batch][n_q_heads][T], natural log of the softmax normaliser
 *   stream   cudaStream_t (NULL = default stream)
 * One kernel per call: a split-KV pass over ~one work item per SM whose last CTAs merge the
 * pieces by log-sum-exp.
 *
 * Ordering.  By default a call is an ordinary launch: it starts after everything enqueued before
 * it on `stream` has finished.  Where the library knows that the kernel directly before a call in
 * the stream is this context's previous verification call, the call starts early (programmatic
 * stream serialisation): it reads q / k_cache / v_cache / parents while that call is still
 * finishing, and several calls can be resident at once.  That is the case
 *   - for the second and later calls of one sparrow_verify_attn_batch(), and
 *   - for every call after sparrow_set_call_overlap(ctx, 1), by which the caller vouches that
 *     whatever it enqueues on the stream between two calls of this context either is an ordinary
 *     kernel / copy (which completes before its successors start) or writes none of the next
 *     call's inputs.  (A kernel that lets its dependents launch early -- many library GEMM, norm
 *     and RoPE kernels do -- and then writes q or the new K/V rows is what must not sit there.)
 * A call that would start early but reads memory that one of this context's calls which may
 * still be running writes (its out / lse) is launched in plain stream order instead, as is a call
 * that follows a call of another context.  Writes of consecutive calls of one context are ordered
 * through counters in its workspace.  All calls of a context belong on one stream (or must be kept
 * from running concurrently by events): the counters assume that calls run in the order they were
 * enqueued.  While a stream is being captured into a graph, or with SPARROW_NO_PDL=1 in the
 * environment when the context is created, a call is two ordinary launches (split-KV pass over
 * one wave of pieces, combine kernel) ordered by the stream alone and touches no counter.
 * Results are deterministic for fixed arguments. */
sparrow_status sparrow_verify_attn(sparrow_ctx* ctx, const void* q, const void* k_cache,
                                   const void* v_cache, const int32_t* kv_len,
                                   const int32_t* parents, int32_t T, void* out, float* lse,
                                   void* stream);

/* (a) generalised for the draft model's attention on a COMPACTED text-anchored cache (Eq. 2,
 * Section 3.1; sparrow_compact_anchors() builds such a cache): the text-anchored window mode as a
 * contiguous stream for the tensor-core kernel.
 *   - The draft block holds the T_tree nodes of the draft tree (rows [kv_len[b], kv_len[b] +
 *     T_tree), parents DEV int32 [batch][T_tree]); the queries are its last T_new nodes
 *     (q, out: [batch][T_new][n_q_heads][128]; lse: [batch][n_q_heads][T_new]).  T_new = T_tree
 *     is sparrow_verify_attn().
 *   - first_visible  DEV int32 [batch][T_new] or NULL: query t sees prefix key j only if
 *     j >= first_visible[b][t] (values above kv_len[b] count as kv_len[b]); the draft block is
 *     governed by the tree alone.  With anchors in increasing order the window rule of
 *     sparrow_anchor_attn() ("qpos - window < p") selects exactly such a run of compact rows;
 *     sparrow_window_first_visible() / _device() compute the index.
 *   - first_visible_min  HOST int32 [batch] or NULL: a lower bound of first_visible[b][*] that the
 *     caller knows on the host (0 <= value <= kv_len[b]); keys left of it (rounded down to a
 *     128-key tile) are not streamed at all.  A device-side bound below it is reported through
 *     the anchor status bit and treated as the first streamed key.
 * Ordering, errors and everything else as for sparrow_verify_attn(); SPARROW_ERR_SHAPE unless
 * 1 <= T_new <= T_tree <= SPARROW_MAX_T and kv_len[b] + T_tree <= kv_capacity. */
sparrow_status sparrow_verify_attn_window(sparrow_ctx* ctx, const void* q, const void* k_cache,
                                          const void* v_cache, const int32_t* kv_len,
                                          const int32_t* parents, int32_t T_tree, int32_t T_new,
                                          const int32_t* first_visible, const int32_t* first_visible_min,
                                          void* out, float* lse, void* stream);

/* The window rule of mode (b) on a compacted cache.  anchor_idx: n_anchor strictly increasing
 * rows, the last T_tree of them the draft tree's nodes, the queries its last T_new nodes (as in
 * sparrow_anchor_attn_tree()); compact row j holds anchor j.  first_visible[t] = the first text
 * anchor j (j < n_anchor - T_tree) with anchor_idx[j] > qpos_t - window, qpos_t = the query's own
 * row; n_anchor - T_tree if there is none; 0 when window <= 0.
 * Host version: one sequence, HOST arrays, also returns the smallest of them (may be NULL);
 * SPARROW_ERR_ANCHOR unless the list is strictly increasing and n_anchor >= T_tree.
 * Device version: DEV anchor_idx [batch][n_anchor] -> DEV first_visible [batch][T_new], one small
 * kernel on `stream` (a binary search per query). */
sparrow_status sparrow_window_first_visible(const int32_t* anchor_idx, int32_t n_anchor, int32_t window,
                                            int32_t T_tree, int32_t T_new, int32_t* first_visible,
                                            int32_t* first_visible_min);
sparrow_status sparrow_window_first_visible_device(sparrow_ctx* ctx, const int32_t* anchor_idx,
                                                   int32_t n_anchor, int32_t window, int32_t T_tree,
                                                   int32_t T_new, int32_t* first_visible, void* stream);

/* Several verification calls enqueued back to back on one stream -- e.g. the layers of one
 * decode step, each with its own KV cache (Section 4: the target verifies the draft tree in one
 * forward pass, i.e. one such call per decoder layer).  Same results as calling
 * sparrow_verify_attn() n_calls times; the calls after the first start early (nothing can sit
 * between them in the stream).  Stops at the first error.  `calls` is HOST memory. */
typedef struct {
    const void*    q;
    const void*    k_cache;
    const void*    v_cache;
    const int32_t* kv_len;    /* HOST */
    const int32_t* parents;   /* DEV */
    int32_t        T;
    void*          out;
    float*         lse;
} sparrow_verify_call;
sparrow_status sparrow_verify_attn_batch(sparrow_ctx* ctx, const sparrow_verify_call* calls,
                                         int32_t n_calls, void* stream);

/* (b) Text-anchored window attention (Eq. 2, Section 3.1).
 *   k, v        DEV bf16 full-length buffers (layout above); only rows named by anchor_idx are read
 *   anchor_idx  DEV int32 [batch][n_anchor], strictly increasing per sequence, every entry in
 *               [0, kv_capacity); the last T entries are the T query tokens' own rows
 *   n_anchor    T .. kv_capacity
 *   window      query t, at position qpos = anchor_idx[n_anchor-T+t], sees anchor p iff
 *               qpos - window < p <= qpos; window <= 0 removes the lower bound.  (The paper names
 *               a window but does not define it; this is the library's rule.)
 *   T           1 .. SPARROW_MAX_T query tokens
 *   q, out, lse as in (a). */
sparrow_status sparrow_anchor_attn(sparrow_ctx* ctx, const void* q, const void* k, const void* v,
                                   const int32_t* anchor_idx, int32_t n_anchor, int32_t window,
                                   int32_t T, void* out, float* lse, void* stream);

/* (b) with tree-structured draft tokens (the paper drafts a dynamic tree, Section 4; Eq. 2 is
 * written for one chain step, so the visibility among draft tokens is this library's reading).
 * The last T_tree entries of anchor_idx are the rows of the draft tree's nodes, node i at
 * anchor_idx[n_anchor - T_tree + i]; the queries are the last T_new nodes (T_new = T_tree: the
 * whole tree; T_new < T_tree: only the nodes added by the latest drafting step).
 *   parents   DEV int32 [batch][T_tree], -1 = root, parents[i] < i (as in (a))
 *   q, out    DEV bf16 [batch][T_new][n_q_heads][128];  lse DEV fp32 [batch][n_q_heads][T_new]
 * A query node at row qpos sees a text anchor p (one of the first n_anchor - T_tree entries) iff
 * p <= qpos and (window <= 0 or qpos - window < p), and a tree node iff it is the query itself or
 * one of its ancestors.  With parents = chain and a window wider than the draft block this equals
 * sparrow_anchor_attn().  SPARROW_ERR_SHAPE unless 1 <= T_new <= T_tree <= SPARROW_MAX_T,
 * SPARROW_ERR_ANCHOR unless T_tree <= n_anchor <= kv_capacity; a malformed device-side parent
 * array sets the tree status bit (the node counts as a root). */
sparrow_status sparrow_anchor_attn_tree(sparrow_ctx* ctx, const void* q, const void* k, const void* v,
                                        const int32_t* anchor_idx, int32_t n_anchor, int32_t window,
                                        const int32_t* parents, int32_t T_tree, int32_t T_new,
                                        void* out, float* lse, void* stream);

/* Row movers (Section 3.1: the draft model keeps the text-anchored states and discards the visual
 * KV cache; the paper gives no procedure, these two calls are this library's).  Both are plain
 * copies, bit-exact, one ordinary kernel each, ordered by the stream like any other kernel.
 *
 * sparrow_kv_append: writes the T new rows of every (sequence, KV head) into cache rows
 * [kv_len[b], kv_len[b] + T) -- what sparrow_verify_attn() expects to find there.
 *   k_new, v_new  DEV bf16 [batch][n_kv_heads][T][128], contiguous
 *   k_cache, v_cache  DEV, the context's layout;  kv_len HOST int32 [batch]
 * SPARROW_ERR_SHAPE unless 1 <= T <= SPARROW_MAX_T and kv_len[b] + T <= kv_capacity.
 *
 * sparrow_compact_anchors: copies rows anchor_idx[b][0 .. n_anchor) of k / v (the context's layout)
 * to rows [dst_row, dst_row + n_anchor) of a compact cache laid out
 * [batch][n_kv_heads][compact_capacity][128], contiguous.  On the compact cache the anchored mode
 * is sparrow_verify_attn_window() with kv_len = (anchors before the draft block): a contiguous
 * stream for the tensor-core kernel instead of a gather.
 *   anchor_idx  DEV int32 [batch][n_anchor]; an entry outside [0, kv_capacity) is not read: its
 *               row is written as zeros and the anchor status bit is set.
 * SPARROW_ERR_ANCHOR unless 1 <= n_anchor <= kv_capacity; SPARROW_ERR_SHAPE unless
 * 0 <= dst_row and dst_row + n_anchor <= compact_capacity.  Both need a workspace (status word). */
sparrow_status sparrow_kv_append(sparrow_ctx* ctx, const void* k_new, const void* v_new, void* k_cache,
                                 void* v_cache, const int32_t* kv_len, int32_t T, void* stream);
sparrow_status sparrow_compact_anchors(sparrow_ctx* ctx, const void* k, const void* v,
                                       const int32_t* anchor_idx, int32_t n_anchor, void* k_compact,
                                       void* v_compact, int32_t compact_capacity, int32_t dst_row,
                                       void* stream);

/* Hidden-state reuse: the draft model's input (Section 3.1, Eq. 1)
 *     z_t = FC(e_t (+) h_t):
 * the projection FC of the concatenation of the token embedding e_t and the target model's hidden
 * state h_t (second-to-last layer, previous position), 2 d features down to d_out, for the M tokens
 * of a drafting step.  FC is read as a linear layer z = W x (+ b); the paper does not say whether it
 * has a bias, so `bias` may be NULL.  The concatenation is never materialised.
 *   e, h     DEV bf16 [M][d], dense          w  DEV bf16 [d_out][2 d], dense (torch.nn.Linear layout)
 *   bias     DEV bf16 [d_out] or NULL        z  DEV bf16 [M][d_out]
 * One kernel, ordered by the stream: a split-K pass whose slices meet inside a thread-block
 * cluster (no scratch memory, no counters); fp32 accumulation in a fixed order (results are
 * deterministic).  The context provides the status word (its workspace must be registered) -- its
 * layout is not used.
 * SPARROW_ERR_SHAPE unless 1 <= M <= 64, d a multiple of 64, d_out a multiple of 128 and the
 * pointers 16-byte aligned. */
sparrow_status sparrow_hsr_fuse(sparrow_ctx* ctx, const void* e, const void* h, const void* w, const void* bias,
                                int32_t M, int32_t d, int32_t d_out, void* z, void* stream);

/* After the verification pass (Appendix A, "Speculative Decoding": the target keeps exactly what it
 * would have produced itself; the paper relies on the standard procedure and does not restate it).
 *
 * sparrow_accept_greedy: temperature-0 acceptance of a draft tree.
 *   draft_tokens DEV int32 [batch][T]      token of every draft node
 *   parents      DEV int32 [batch][T]      as in (a)
 *   target_next  DEV int32 [batch][T + 1]  [0]: the target's next token after the committed prefix,
 *                                          [1 + i]: its next token after node i (argmax of the logits
 *                                          the verification pass produced at that node)
 *   path_out     DEV int32 [batch][T]      nodes of the deepest accepted chain, root first, then -1
 *   n_accept_out DEV int32 [batch]         its length (0 .. T)
 *   bonus_out    DEV int32 [batch]         the target's token after the chain's last node
 * A node is accepted iff its token equals target_next[parent + 1] and its parent is accepted (a
 * root: iff it equals target_next[0]); among chains of equal depth the one ending at the smallest
 * node index wins.  A malformed parent sets the tree status bit and counts as a root.
 *
 * sparrow_kv_keep_accepted: moves the K/V rows of the accepted nodes, rows kv_len[b] + path[i], to
 * rows kv_len[b] + i (i < n_accept[b]) of one cache pair, in place; afterwards the committed
 * length is kv_len[b] + n_accept[b].  One call per layer.  kv_len is HOST, path / n_accept are the
 * device arrays sparrow_accept_greedy() wrote.
 * Both: SPARROW_ERR_SHAPE unless 1 <= T <= SPARROW_MAX_T (and kv_len[b] + T <= kv_capacity). */
sparrow_status sparrow_accept_greedy(sparrow_ctx* ctx, const int32_t* draft_tokens, const int32_t* parents,
                                     const int32_t* target_next, int32_t T, int32_t* path_out,
                                     int32_t* n_accept_out, int32_t* bonus_out, void* stream);
/* sparrow_accept_sample: temperature-1 acceptance of a draft tree by multi-round rejection sampling
 * (Appendix A: the verification keeps the target's output distribution exactly; Section 4 reports
 * every result at temperature 0 and 1.  The paper relies on the standard procedure; the reading
 * taken here: at the current node, with target distribution p and draft distribution q, the
 * children are tried in index order; a child with token x is accepted with probability
 * min(1, p(x) / q(x)); after a rejection p becomes the normalised positive part of (p - q) and q
 * loses x, the siblings having been drawn without replacement; when no child is accepted the
 * next token is drawn from what p has become.)
 *   draft_tokens DEV int32 [batch][T];  parents DEV int32 [batch][T] as in (a)
 *   p_target,
 *   p_draft      DEV fp32 [batch][T + 1][vocab]: row 0 belongs to the committed prefix, row 1 + i to
 *                node i -- the target's next-token distribution there and the draft distribution
 *                that node's children were drawn from; entries in [0, 1]
 *   u_node       DEV uint32 [batch][T]      the uniform of node i's acceptance test
 *   u_bonus      DEV uint32 [batch][T + 1]  the uniform of the token drawn when the walk stops at a row
 *   path_out, n_accept_out, bonus_out as for sparrow_accept_greedy (the accepted chain, its length,
 *                the token emitted after it); sparrow_kv_keep_accepted() takes them as they are.
 * The outputs are integers, so the arithmetic is fixed: P = floor(p 2^30 + 1/2) (likewise Q), and
 * with A = sum P, B = sum Q, r the node's uniform: accept iff Q[x] > 0 and r Q[x] A < P[x] B 2^32;
 * after a rejection P <- max(B P - A Q, 0) >> 30 (unless B == 0), A <- sum P, B <- B - Q[x],
 * Q[x] <- 0; the bonus token is the smallest v with P[0] + ... + P[v] > (u_bonus A) >> 32, P
 * being the row's original target row again if A == 0.  Integer sums: the result does not depend
 * on how the reduction is parallelised.  A token outside [0, vocab) is never accepted and sets
 * the tree status bit, as does a malformed parent (which counts as a root).
 * SPARROW_ERR_SHAPE unless 1 <= T <= SPARROW_MAX_T and vocab >= 1. */
sparrow_status sparrow_accept_sample(sparrow_ctx* ctx, const int32_t* draft_tokens, const int32_t* parents,
                                     const float* p_target, const float* p_draft, const uint32_t* u_node,
                                     const uint32_t* u_bonus, int32_t vocab, int32_t T, int32_t* path_out,
                                     int32_t* n_accept_out, int32_t* bonus_out, void* stream);
sparrow_status sparrow_kv_keep_accepted(sparrow_ctx* ctx, void* k_cache, void* v_cache,
                                        const int32_t* kv_len, const int32_t* path,
                                        const int32_t* n_accept, int32_t T, void* stream);

/* Verification step with HOST buffers (what a caller without device-side glue uses): copies q,
 * the T new K/V rows per (batch, KV head) and parents to the device, writes the new rows into
 * cache rows [kv_len[b], kv_len[b]+T), runs (a), copies out / lse back and synchronises `stream`.
 *   q_host       HOST bf16 [batch][T][n_q_heads][128]      (pinned memory recommended)
 *   k_new_host,
 *   v_new_host   HOST bf16 [batch][n_kv_heads][T][128]
 *   parents_host HOST int32 [batch][T]  (validated on the host: SPARROW_ERR_TREE)
 *   out_host     HOST bf16 [batch][T][n_q_heads][128];  lse_host HOST fp32 [batch][n_q_heads][T]
 * Device staging comes from the registered workspace; nothing is allocated.
 * When all six host buffers are page-locked (cudaHostAlloc / cudaHostRegister) and 16-byte
 * aligned, no copy engine is involved: one kernel reads q, parents and the new rows from host
 * memory (q and parents into staging, the rows into the cache) and the attention kernel stores
 * out / lse into the host buffers; otherwise every buffer goes through cudaMemcpyAsync.  The
 * results are the same bits either way; the host buffers must not change until the call returns. */
sparrow_status sparrow_verify_step_host(sparrow_ctx* ctx, const void* q_host,
                                        const void* k_new_host, const void* v_new_host,
                                        void* k_cache, void* v_cache, const int32_t* kv_len,
                                        const int32_t* parents_host, int32_t T, void* out_host,
                                        float* lse_host, void* stream);

/* Verification attention without a context and without a caller-provided workspace.
 * (The paper has no counterpart to this call; it exists for integration reasons only.)
 *
 * Who it is for: callers that are not allowed to allocate.  Some hosts own every byte of device
 * memory themselves (a serving engine with a fixed pool, a plugin loaded into another framework)
 * and forbid cudaMalloc in extension code; others run a latency-critical loop in which
 * cudaMalloc's device-wide synchronisation, or its failure under fragmentation, is not
 * acceptable.  sparrow_create / sparrow_set_workspace push that problem to the caller; this call
 * removes it: the scratch memory (split-KV partials, status word) is a fixed array of
 * SPARROW_STATIC_SCRATCH_BYTES that is part of the library's device image.  Every GPU that loads
 * the library therefore holds that much memory until the process exits, whether or not the call
 * is ever used.
 *
 * Arguments are those of sparrow_verify_attn(), with the layout passed by value of pointer in
 * place of a context; the call works on the CURRENT device.  It calls no cudaMalloc / cudaFree
 * and no allocating library routine, and keeps its bookkeeping in static host storage.
 *   - First call on a device: one-time set-up (device query, kernel attributes, address of the
 *     scratch array, clearing its header with a synchronising cudaMemset).  Make that first call
 *     outside any stream capture.
 *   - Argument errors are reported as by sparrow_verify_attn(), before anything is enqueued.
 *     SPARROW_ERR_WORKSPACE when the split-KV partials of the call do not fit the array behind its
 *     1 KiB header: a call has max(SM count, batch x KV heads x row groups) work items of at most
 *     70 KB each, so on a 148-SM part everything fits except very large batches of draft blocks
 *     longer than 18 tokens (e.g. 32 sequences x 64 tokens); nothing is enqueued then either.
 *   - The call always runs in the stream-ordered mode: two ordinary kernel launches on `stream`
 *     (one when no sequence needs more than one piece).
 *   - All calls on a device share the one array, which keeps the previous call's contents.  What
 *     must start clean (the status word) is cleared on `stream` at the start of every call;
 *     partials are always written before they are read.  Calls that overlap on the GPU (two
 *     streams without an event between them) race on the array and give undefined results; so do
 *     concurrent calls from several host threads.
 *   - Device-detected input problems (a parent index outside [-1, i)) are handled as everywhere
 *     else (the node is treated as a root) but cannot be queried: there is no context to ask. */
#define SPARROW_STATIC_SCRATCH_BYTES (16u * 1024u * 1024u)
sparrow_status sparrow_verify_attn_static(const sparrow_layout* layout, const void* q, const void* k_cache,
                                          const void* v_cache, const int32_t* kv_len,
                                          const int32_t* parents, int32_t T, void* out, float* lse,
                                          void* stream);

/* Host helpers, exported so mask / index construction can be checked bit for bit.
 * Ancestor words of a draft tree (Section 4: dynamic draft trees): masks[i] has bit a set iff
 * a == i or a is an ancestor of i.  SPARROW_ERR_TREE unless -1 <= parents[i] < i. */
sparrow_status sparrow_build_ancestor_masks(const int32_t* parents_host, int32_t T,
                                            uint64_t* masks_host);
/* Anchor list for Eq. 2's index set T: positions p of [0, seq_len) outside every visual span
 * [begin, end) with p >= seq_len - window (window <= 0: all), increasing, then the T draft rows
 * seq_len .. seq_len+T-1.  idx_host must hold seq_len + T entries. */
sparrow_status sparrow_build_anchor_idx(int32_t seq_len, const int32_t* vis_spans, int32_t n_spans,
                                        int32_t window, int32_t T, int32_t* idx_host,
                                        int32_t* n_anchor_out);
/* Runs the kernels' own device-side mask construction: parents_dev DEV int32 [T] ->
 * masks_dev DEV uint64 [T]. */
sparrow_status sparrow_debug_ancestor_masks_device(sparrow_ctx* ctx, const int32_t* parents_dev,
                                                   int32_t T, uint64_t* masks_dev, void* stream);

/* Host-side split schedule, exported for inspection (pure host code, needs no GPU): for `batch`
 * sequences of n_keys[b] keys, gqa_group query heads per KV head, draft blocks of T tokens and a
 * target of n_sm work items (the SM
 * count, or sparrow_plan_target_items() for calls in fused mode), writes
 * splits_out[b] = key-range pieces per (sequence, KV head, row group) and the total number of
 * work items.  Pieces are whole 128-key tiles, as even as whole tiles allow (the last one takes
 * the ragged end): sparrow_plan_piece_range() gives the keys [begin, end) of piece `piece` of
 * `n_splits`; SPARROW_ERR_SHAPE unless 0 <= piece < n_splits <= ceil(n_keys / 128). */
sparrow_status sparrow_plan_splits(int32_t n_sm, int32_t batch, int32_t n_kv_heads, int32_t gqa_group,
                                   const int32_t* n_keys, int32_t T, int32_t* splits_out,
                                   int32_t* n_items_out);
sparrow_status sparrow_plan_piece_range(int32_t n_keys, int32_t n_splits, int32_t piece,
                                        int32_t* begin_out, int32_t* end_out);

/* Exercises the bounded device-side wait the kernels use between consecutive calls: enqueues a
 * one-thread kernel that waits until the finisher counter of even calls reaches its current
 * expected value plus `ahead`.  With ahead == 0 it returns once all earlier calls are done; with
 * ahead > 0 nothing will ever satisfy it, the wait gives up after about one second, the kernel
 * sets the timeout status bit and ends -- the context stays usable. */
sparrow_status sparrow_debug_wait_counter(sparrow_ctx* ctx, uint32_t ahead, void* stream);

/* Test aid for the ordering rules of sparrow_verify_attn(): enqueues a small kernel that lets its
 * dependents launch at once, idles for about delay_us microseconds (at most 10 ms) and only then
 * copies `bytes` (a multiple of 16, both pointers 16-byte aligned, DEV) from src to dst -- the
 * behaviour of a foreign kernel with an early launch trigger in front of a verification call. */
sparrow_status sparrow_debug_early_trigger_copy(sparrow_ctx* ctx, const void* src, void* dst, size_t bytes,
                                               uint32_t delay_us, void* stream);

/* Synchronises `stream`, returns the sticky device status (SPARROW_OK, SPARROW_ERR_TREE,
 * SPARROW_ERR_ANCHOR or SPARROW_ERR_TIMEOUT) and clears it.  Not for the hot path. */
sparrow_status sparrow_last_device_status(sparrow_ctx* ctx, void* stream);

/* The raw status word that the most recent sparrow_last_device_status() call on this context read
 * (0 before the first call).  Bits 0..2: malformed tree, bad anchor, timeout.  A wait that gave up
 * also sets bit 8 + site: 0 TMA producer, 1 MMA issuer, 2 softmax warps, 3 / 4 the waits in front
 * of a CTA's first global write (same / other call parity), 5 finisher waiting for the call's
 * pieces, 6 finisher waiting for the previous call, 7 finisher's bulk copies, 8 the debug wait.
 * For diagnosis only. */
uint32_t sparrow_debug_status_word(const sparrow_ctx* ctx);

/* Number of kernels the library has launched through this context (for launch accounting). */
int64_t sparrow_launch_count(const sparrow_ctx* ctx);

const char* sparrow_status_string(sparrow_status s);

#ifdef __cplusplus
}
#endif
#endif /* SPARROW_ATTN_H_ */
