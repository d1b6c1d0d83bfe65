/*
 * sparrow_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, obviously-correct CPU statement of what the speculative-step attention of
 * Sparrow computes.  It is used by the tests, by the smoke check and by the benchmark's CPU
 * baseline leg; the product (the CUDA library) never links, imports or calls anything here, and
 * this file shares no code, header, table or helper with the CUDA path.
 *
 * What it follows:
 *   - Eq. 2 (Section 3.1, VATA):  Attention = Softmax(Q_t K_T^T / sqrt(d)) V_T, with K_T, V_T the
 *     key / value rows restricted to the text-anchored index set T.
 *   - Appendix A ("Speculative Decoding") and Section 4 ("Metrics"): the target model verifies all
 *     draft candidates in one parallel forward pass, the candidates forming a (dynamic) tree; the
 *     method is lossless, so the verification attention is the target's ordinary softmax
 *     attention under the tree's ancestor mask.
 *
 * Both modes are therefore the textbook definition, written out:
 *     s_j  = scale * sum_d q[d] * k_j[d]                     for every visible key j
 *     lse  = log sum_{j visible} exp(s_j)                    (natural log)
 *     out  = sum_{j visible} exp(s_j - lse) * v_j
 * evaluated in IEEE double with a two-pass softmax (max first, then the sum).  No tiling, no
 * online rescaling, no fusion: a reader can check it against the formula by eye.  Inputs are
 * bf16 bit patterns (uint16_t), converted exactly to double.
 *
 * The visibility sets are built by separate functions so each can be pinned on its own:
 *   verification:  Vis(t) = {0..kv_len-1}  U  {kv_len + i : i is t itself or an ancestor of t}
 *   anchored   :   Vis(t) = {anchor_idx[j] : qpos_t - window < anchor_idx[j] <= qpos_t},
 *                  qpos_t = anchor_idx[n_anchor - T + t]   (window <= 0: no lower bound)
 * The paper never defines the "window" of VATA; the rule above is this build's reading.
 *
 * Pins (tests marked "not gpu"): closed forms (equal keys -> mean of V and s + log n; two keys ->
 * logistic weights), softmax invariants (shift, permutation, split-and-merge by log-sum-exp),
 * torch's scaled_dot_product_attention in float64 for causal / unmasked / gathered-dense cases,
 * scipy's logsumexp, exhaustive tree enumeration against a parent walk, closed-form masks for
 * chains and forests, brute-force filtering for the anchor list.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_ERR_ARG 1
#define ORACLE_ERR_TREE 3
#define ORACLE_ERR_ANCHOR 4

/* bf16 -> double, exact: a bf16 is the top 16 bits of an IEEE binary32. */
static double bf16_to_double(uint16_t h)
{
    uint32_t u = ((uint32_t)h) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* ------------------------------------------------------------------------------------------
 * Tree mask.  parents[i] is the parent of draft node i, -1 for a root; nodes are in
 * topological order (parents[i] < i).  anc[i] has bit a set iff a == i or a is an ancestor of i.
 * Defined here by the recurrence  anc[i] = bit(i) | anc[parents[i]].
 * ---------------------------------------------------------------------------------------- */
int oracle_ancestor_masks(const int32_t *parents, int32_t T, uint64_t *anc)
{
    if (!parents || !anc || T < 1 || T > 64) return ORACLE_ERR_ARG;
    for (int32_t i = 0; i < T; ++i) {
        int32_t p = parents[i];
        if (p < -1 || p >= i) return ORACLE_ERR_TREE;
        uint64_t m = (uint64_t)1 << i;
        if (p >= 0) m |= anc[p];
        anc[i] = m;
    }
    return ORACLE_OK;
}

/* vis[t][j], j in [0, n_keys), n_keys = kv_len + T, row stride = vis_stride bytes. */
int oracle_verify_visibility(int32_t kv_len, int32_t T, const uint64_t *anc, uint8_t *vis,
                             int64_t vis_stride)
{
    if (!anc || !vis || kv_len < 0 || T < 1 || T > 64) return ORACLE_ERR_ARG;
    for (int32_t t = 0; t < T; ++t) {
        uint8_t *row = vis + (int64_t)t * vis_stride;
        for (int32_t j = 0; j < kv_len; ++j) row[j] = 1;
        for (int32_t i = 0; i < T; ++i) row[kv_len + i] = (uint8_t)((anc[t] >> i) & 1u);
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------
 * Anchor list (the index set T of Eq. 2 under this build's window reading): every position p of
 * [0, seq_len) that lies in no visual span [begin, end) and satisfies p >= seq_len - window
 * (window <= 0: no bound), in increasing order, followed by the T draft positions
 * seq_len .. seq_len+T-1.
 * ---------------------------------------------------------------------------------------- */
int oracle_anchor_idx(int32_t seq_len, const int32_t *vis_spans, int32_t n_spans, int32_t window,
                      int32_t T, int32_t *idx, int32_t *n_anchor)
{
    if (!idx || !n_anchor || seq_len < 0 || T < 0 || n_spans < 0 || (n_spans > 0 && !vis_spans))
        return ORACLE_ERR_ARG;
    int32_t n = 0;
    for (int32_t p = 0; p < seq_len; ++p) {
        int visual = 0;
        for (int32_t s = 0; s < n_spans; ++s)
            if (p >= vis_spans[2 * s] && p < vis_spans[2 * s + 1]) visual = 1;
        if (visual) continue;
        if (window > 0 && p < seq_len - window) continue;
        idx[n++] = p;
    }
    for (int32_t t = 0; t < T; ++t) idx[n++] = seq_len + t;
    *n_anchor = n;
    return ORACLE_OK;
}

/* vis[t][j] over the n_anchor gathered keys (j indexes anchor_idx, not the sequence). */
int oracle_anchor_visibility(const int32_t *anchor_idx, int32_t n_anchor, int32_t window,
                             int32_t T, uint8_t *vis, int64_t vis_stride)
{
    if (!anchor_idx || !vis || T < 1 || n_anchor < T) return ORACLE_ERR_ARG;
    for (int32_t j = 1; j < n_anchor; ++j)
        if (anchor_idx[j] <= anchor_idx[j - 1]) return ORACLE_ERR_ANCHOR;
    if (anchor_idx[0] < 0) return ORACLE_ERR_ANCHOR;
    for (int32_t t = 0; t < T; ++t) {
        int64_t qpos = anchor_idx[n_anchor - T + t];
        uint8_t *row = vis + (int64_t)t * vis_stride;
        for (int32_t j = 0; j < n_anchor; ++j) {
            int64_t p = anchor_idx[j];
            int ok = (p <= qpos);
            if (window > 0 && !(qpos - window < p)) ok = 0;
            row[j] = (uint8_t)ok;
        }
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------
 * Attention core.
 *
 *   q    : [B][T][Hq][D] bf16, dense
 *   k, v : element offset of (b, kv head, row, d) = b*stride_b + head*stride_h + row*D + d
 *   key_rows : NULL (key j lives in row j) or int32 [B][n_keys] (key j lives in row key_rows[j])
 *   vis  : uint8 [B][T][n_keys]; only entries j < n_keys_b[b] are read for sequence b
 *   rows : NULL (every (b,t,h)) or int32 [n_rows][3] = (b, t, h) triples to evaluate
 *   out  : double, [B][T][Hq][D] when rows == NULL, else [n_rows][D]
 *   lse  : double, [B][Hq][T]     when rows == NULL, else [n_rows]
 * Query head h reads KV head h / (Hq/Hkv).  A row with no visible key gets out = 0, lse = -inf.
 * ---------------------------------------------------------------------------------------- */
typedef struct {
    const uint16_t *q, *k, *v;
    const int32_t *key_rows;
    const uint8_t *vis;
    const int32_t *n_keys_b;
    const int32_t *rows;
    int64_t n_rows;
    int32_t B, T, Hq, Hkv, D, n_keys;
    int64_t stride_b, stride_h;
    double scale;
    double *out, *lse;
    int64_t next;            /* work counter (guarded by mu) */
    pthread_mutex_t mu;
} job_t;

static void one_row(const job_t *J, int64_t r, double *s)
{
    int32_t b, t, h;
    double *out, *lse;
    if (J->rows) {
        b = J->rows[3 * r]; t = J->rows[3 * r + 1]; h = J->rows[3 * r + 2];
        out = J->out + r * J->D;
        lse = J->lse + r;
    } else {
        b = (int32_t)(r / ((int64_t)J->T * J->Hq));
        t = (int32_t)((r / J->Hq) % J->T);
        h = (int32_t)(r % J->Hq);
        out = J->out + (((int64_t)b * J->T + t) * J->Hq + h) * J->D;
        lse = J->lse + ((int64_t)b * J->Hq + h) * J->T + t;
    }
    const int32_t D = J->D;
    const int32_t kvh = h / (J->Hq / J->Hkv);
    const int32_t n = J->n_keys_b[b];
    const uint16_t *qrow = J->q + (((int64_t)b * J->T + t) * J->Hq + h) * D;
    const uint16_t *kb = J->k + (int64_t)b * J->stride_b + (int64_t)kvh * J->stride_h;
    const uint16_t *vb = J->v + (int64_t)b * J->stride_b + (int64_t)kvh * J->stride_h;
    const uint8_t *visrow = J->vis + ((int64_t)b * J->T + t) * J->n_keys;
    const int32_t *krows = J->key_rows ? J->key_rows + (int64_t)b * J->n_keys : NULL;

    /* pass 1: scores and their maximum over the visible set */
    double m = -INFINITY;
    for (int32_t j = 0; j < n; ++j) {
        if (!visrow[j]) continue;
        const uint16_t *krow = kb + (int64_t)(krows ? krows[j] : j) * D;
        double dot = 0.0;
        for (int32_t d = 0; d < D; ++d) dot += bf16_to_double(qrow[d]) * bf16_to_double(krow[d]);
        s[j] = J->scale * dot;
        if (s[j] > m) m = s[j];
    }
    for (int32_t d = 0; d < D; ++d) out[d] = 0.0;
    if (m == -INFINITY) { *lse = -INFINITY; return; }
    /* pass 2: normaliser */
    double l = 0.0;
    for (int32_t j = 0; j < n; ++j)
        if (visrow[j]) l += exp(s[j] - m);
    const double L = m + log(l);
    *lse = L;
    /* pass 3: weighted sum of values */
    for (int32_t j = 0; j < n; ++j) {
        if (!visrow[j]) continue;
        const double p = exp(s[j] - L);
        const uint16_t *vrow = vb + (int64_t)(krows ? krows[j] : j) * D;
        for (int32_t d = 0; d < D; ++d) out[d] += p * bf16_to_double(vrow[d]);
    }
}

static void *worker(void *arg)
{
    job_t *J = (job_t *)arg;
    double *s = (double *)malloc(sizeof(double) * (size_t)(J->n_keys > 0 ? J->n_keys : 1));
    if (!s) return NULL;
    for (;;) {
        pthread_mutex_lock(&J->mu);
        int64_t r = J->next++;
        pthread_mutex_unlock(&J->mu);
        if (r >= J->n_rows) break;
        one_row(J, r, s);
    }
    free(s);
    return NULL;
}

int oracle_attention(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                     const int32_t *key_rows, const uint8_t *vis, const int32_t *n_keys_b,
                     int32_t B, int32_t T, int32_t Hq, int32_t Hkv, int32_t D, int32_t n_keys,
                     int64_t stride_b, int64_t stride_h, double scale,
                     const int32_t *rows, int64_t n_rows, int32_t n_threads,
                     double *out, double *lse)
{
    if (!q || !k || !v || !vis || !n_keys_b || !out || !lse) return ORACLE_ERR_ARG;
    if (B < 1 || T < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv || D < 1 || n_keys < 0) return ORACLE_ERR_ARG;
    for (int32_t b = 0; b < B; ++b)
        if (n_keys_b[b] < 0 || n_keys_b[b] > n_keys) return ORACLE_ERR_ARG;
    job_t J;
    memset(&J, 0, sizeof J);
    J.q = q; J.k = k; J.v = v; J.key_rows = key_rows; J.vis = vis; J.n_keys_b = n_keys_b;
    J.rows = rows; J.n_rows = rows ? n_rows : (int64_t)B * T * Hq;
    J.B = B; J.T = T; J.Hq = Hq; J.Hkv = Hkv; J.D = D; J.n_keys = n_keys;
    J.stride_b = stride_b; J.stride_h = stride_h; J.scale = scale;
    J.out = out; J.lse = lse; J.next = 0;
    pthread_mutex_init(&J.mu, NULL);
    if (n_threads < 1) n_threads = 1;
    if (n_threads > 256) n_threads = 256;
    if (n_threads == 1) {
        worker(&J);
    } else {
        pthread_t th[256];
        int started = 0;
        for (int i = 0; i < n_threads; ++i)
            if (pthread_create(&th[started], NULL, worker, &J) == 0) ++started;
        if (started == 0) worker(&J);
        for (int i = 0; i < started; ++i) pthread_join(th[i], NULL);
    }
    pthread_mutex_destroy(&J.mu);
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------------
 * The two modes, assembled from the pieces above.
 *
 * Verification (one call = B sequences): rows [kv_len[b], kv_len[b]+T) of the cache already hold
 * the draft tokens' K/V.  parents: [B][T].
 * ---------------------------------------------------------------------------------------- */
int oracle_verify_attn(const uint16_t *q, const uint16_t *k_cache, const uint16_t *v_cache,
                       const int32_t *kv_len, const int32_t *parents,
                       int32_t B, int32_t T, int32_t Hq, int32_t Hkv, int32_t D,
                       int64_t stride_b, int64_t stride_h, double scale,
                       const int32_t *rows, int64_t n_rows, int32_t n_threads,
                       double *out, double *lse)
{
    if (!kv_len || !parents || B < 1 || T < 1 || T > 64) return ORACLE_ERR_ARG;
    int32_t n_keys = 0;
    for (int32_t b = 0; b < B; ++b) {
        if (kv_len[b] < 0) return ORACLE_ERR_ARG;
        if (kv_len[b] + T > n_keys) n_keys = kv_len[b] + T;
    }
    uint8_t *vis = (uint8_t *)calloc((size_t)B * T * n_keys, 1);
    int32_t *nk = (int32_t *)malloc(sizeof(int32_t) * (size_t)B);
    if (!vis || !nk) { free(vis); free(nk); return ORACLE_ERR_ARG; }
    int rc = ORACLE_OK;
    for (int32_t b = 0; b < B && rc == ORACLE_OK; ++b) {
        uint64_t anc[64];
        rc = oracle_ancestor_masks(parents + (int64_t)b * T, T, anc);
        if (rc == ORACLE_OK)
            rc = oracle_verify_visibility(kv_len[b], T, anc, vis + (int64_t)b * T * n_keys, n_keys);
        nk[b] = kv_len[b] + T;
    }
    if (rc == ORACLE_OK)
        rc = oracle_attention(q, k_cache, v_cache, NULL, vis, nk, B, T, Hq, Hkv, D, n_keys,
                              stride_b, stride_h, scale, rows, n_rows, n_threads, out, lse);
    free(vis); free(nk);
    return rc;
}

/* Text-anchored window mode: anchor_idx [B][n_anchor], strictly increasing per sequence, the
 * last T entries being the draft tokens' own rows. */
int oracle_anchor_attn(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                       const int32_t *anchor_idx, int32_t n_anchor, int32_t window,
                       int32_t B, int32_t T, int32_t Hq, int32_t Hkv, int32_t D,
                       int64_t stride_b, int64_t stride_h, double scale,
                       const int32_t *rows, int64_t n_rows, int32_t n_threads,
                       double *out, double *lse)
{
    if (!anchor_idx || B < 1 || T < 1 || n_anchor < T) return ORACLE_ERR_ARG;
    uint8_t *vis = (uint8_t *)calloc((size_t)B * T * n_anchor, 1);
    int32_t *nk = (int32_t *)malloc(sizeof(int32_t) * (size_t)B);
    if (!vis || !nk) { free(vis); free(nk); return ORACLE_ERR_ARG; }
    int rc = ORACLE_OK;
    for (int32_t b = 0; b < B && rc == ORACLE_OK; ++b) {
        rc = oracle_anchor_visibility(anchor_idx + (int64_t)b * n_anchor, n_anchor, window, T,
                                      vis + (int64_t)b * T * n_anchor, n_anchor);
        nk[b] = n_anchor;
    }
    if (rc == ORACLE_OK)
        rc = oracle_attention(q, k, v, anchor_idx, vis, nk, B, T, Hq, Hkv, D, n_anchor,
                              stride_b, stride_h, scale, rows, n_rows, n_threads, out, lse);
    free(vis); free(nk);
    return rc;
}
