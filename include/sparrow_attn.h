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
 * sparrow_compact_anchors() (row movers), sparrow_accept_greedy(), sparrow_kv_keep_accepted()
 * (temperature-0 acceptance of the draft tree and the move of the accepted rows).
 *
 * For every batch entry b, query head h (KV head h / 7), draft token t and visible key set Vis:
 *     s_j = softmax_scale * <q[b,t,h,:], k[b,h/7,j,:]>,   lse = log sum_{j in Vis} exp(s_j),
 *     out = sum_{j in Vis} exp(s_j - lse) * v[b,h/7,j,:].
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
#define SPARROW_GQA_GROUP  7    /* query heads per KV head; only value accepted */

/* Fixed per context.  K/V buffers hold, for batch b and KV head g, `kv_capacity` rows of 128 bf16:
 * element offset of (b, g, row, d) = b*kv_stride_batch + g*kv_stride_head + row*128 + d.
 * Both strides must be multiples of 8 elements and the base pointers 16-byte aligned. */
typedef struct {
    int32_t batch;           /* 1 .. SPARROW_MAX_BATCH */
    int32_t n_q_heads;       /* must equal 7 * n_kv_heads */
    int32_t n_kv_heads;
    int32_t head_dim;        /* must be 128 */
    int32_t kv_capacity;     /* rows per (batch, KV head) */
    float   softmax_scale;   /* e.g. 1/sqrt(128); applied in fp32 to the fp32 scores */
    int64_t kv_stride_batch;
    int64_t kv_stride_head;
} sparrow_layout;

typedef struct sparrow_ctx sparrow_ctx;

/* Creates a context on CUDA device `device` (queries the SM count, loads the kernels).
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
 * cannot overlap (stream-ordered mode, graph capture, sparrow_anchor_attn,
 * sparrow_verify_attn_static) always use one wave over all SMs. */
typedef enum {
    SPARROW_PLAN_LATENCY    = 0,
    SPARROW_PLAN_BALANCED   = 1,
    SPARROW_PLAN_THROUGHPUT = 2
} sparrow_plan_policy;

/* Sets the policy for later calls (host state only; may be changed between any two calls).
 * SPARROW_ERR_SHAPE for an unknown value. */
sparrow_status sparrow_set_plan_policy(sparrow_ctx* ctx, int32_t policy);

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
 * pieces by log-sum-exp.  Consecutive calls on one stream overlap: the kernel is launched with
 * programmatic stream serialisation and starts reading q / k_cache / v_cache / parents while the
 * previous kernel in the stream is finishing, as soon as that kernel lets its dependents launch
 * (the library's own kernels do; an ordinary kernel never does before it completes).  So the
 * inputs of a call must not be the out / lse of the library call enqueued directly before it on
 * the same stream; anything else in between (another kernel, a copy) restores plain stream order.
 * Writes of consecutive calls of one context are ordered through counters in its workspace; a
 * call that follows a call of another context takes plain stream order.  All fused calls of a
 * context belong on one stream (or must be kept from running concurrently by events): the
 * counters assume that calls run in the order they were enqueued.  While a stream is being
 * captured into a graph, or with SPARROW_NO_PDL=1 in the environment when the context is created,
 * a call is two ordinary launches (split-KV pass, combine) ordered by the stream alone.
 * Results are deterministic for fixed arguments. */
sparrow_status sparrow_verify_attn(sparrow_ctx* ctx, const void* q, const void* k_cache,
                                   const void* v_cache, const int32_t* kv_len,
                                   const int32_t* parents, int32_t T, void* out, float* lse,
                                   void* stream);

/* Several verification calls enqueued back to back on one stream -- e.g. the layers of one
 * decode step, each with its own KV cache (Section 4: the target verifies the draft tree in one
 * forward pass, i.e. one such call per decoder layer).  Equivalent to calling
 * sparrow_verify_attn() n_calls times; stops at the first error.  `calls` is HOST memory. */
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
 * without a lower window bound is sparrow_verify_attn() with kv_len = (anchors before the draft
 * block): a contiguous stream for the tensor-core kernel instead of a gather.
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
 * Device staging comes from the registered workspace; nothing is allocated. */
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
 *   - SPARROW_ERR_WORKSPACE when the layout / T need more scratch than the array holds (on a
 *     148-SM part: blocks of more than 36 draft tokens, or large batches); nothing is launched then.
 *   - The call always runs in the stream-ordered mode: two ordinary kernel launches on `stream`.
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
 * sequences of n_keys[b] keys, draft blocks of T tokens and a target of n_sm work items (the SM
 * count, or sparrow_plan_target_items() for calls in fused mode), writes
 * splits_out[b] = key-range pieces per (sequence, KV head, row group) and the total number of
 * work items.  Pieces are whole 128-key tiles, as even as whole tiles allow (the last one takes
 * the ragged end): sparrow_plan_piece_range() gives the keys [begin, end) of piece `piece` of
 * `n_splits`; SPARROW_ERR_SHAPE unless 0 <= piece < n_splits <= ceil(n_keys / 128). */
sparrow_status sparrow_plan_splits(int32_t n_sm, int32_t batch, int32_t n_kv_heads,
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
