/*
 * fp64 CPU oracle for APE attention (Adaptive Parallel Encoding, arxiv 2502.05431).
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * GPU library must compute.  It shares no code with the CUDA path, and nothing in
 * the product path may call it: only the test-suite, the smoke check and the
 * benchmark's CPU-baseline leg do.
 *
 * What it evaluates
 *   ape_oracle_attend  : the modified softmax attention of the paper's Eq. 5
 *                        (section "Formulation"), written out per query row, and,
 *                        behind a switch, the per-context hierarchical form of the
 *                        appendix "Hierarchical Formula for APE" (Eq. 11-12).
 *   ape_oracle_attend_tree : the same attention when the contexts form trees (appendix "Future
 *                        Directions": each context a tree-like hierarchy, evaluated along each
 *                        branch with intermediate results merged on the way): the hierarchical
 *                        formulas of the appendix applied node by node, bottom-up.
 *   ape_oracle_encode  : the block-diagonal attention that pre-caches each
 *                        context (section "Parallel Encoding", pre-caching step,
 *                        with the shared prefix of section "Prepending Shared
 *                        Prefix"): plain softmax, no T, no S.
 *
 * Inputs are bf16 bit patterns (uint16) that are widened exactly to double; all
 * arithmetic is fp64.  No blocking, no online softmax, no reordering: every
 * logit of a row is formed, the log-sum-exps are taken, then the weights.
 *
 * Readings of the paper taken here (the text is silent or inconsistent):
 *   - S multiplies the log-sum-exp of ALL context tokens together (Eq. 5 and the
 *     "Efficient Implementation" listing); per_context=1 selects Eq. 11-12.
 *     This choice is pinned by no printed value: PARITY UNPINNED for the choice
 *     between the two readings; each reading itself is pinned by the tests.
 *   - Context trees: the paper prints no formula for a hierarchy deeper than one level.  Reading
 *     taken: inside a tree, a node's members (its own tokens and its child nodes) merge by the
 *     plain hierarchical softmax identity; a node marked as SCALED hands S * LogSumExp to its
 *     parent, as A^{h'}_{C_i} does in Eq. 11; by default the scaled nodes are the roots, i.e. every
 *     top-level tree is one context of Eq. 11-12.  PARITY UNPINNED for where S applies along a
 *     branch; the arithmetic of the reading is pinned by the tests (both ends of the family are
 *     printed formulas: one tree over everything is Eq. 5, one node per context is Eq. 11-12).
 *   - T applies to context logits only (Eq. 5; the T in the non-context term of
 *     the appendix's "Relation" paragraph is a typo).
 *   - Query rows are causal inside the query segment, bottom-right aligned when
 *     the segment holds more keys than rows; they see every prefix and context
 *     token unmasked.
 *   - Consecutive query heads share a KV head: g = h / (H_q / H_kv).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    const uint16_t *k;      /* bf16 bits, element (t, g, e) at k[t*token_stride + g*head_stride + e] */
    const uint16_t *v;
    int64_t len;            /* tokens */
    int64_t token_stride;   /* in elements */
    int64_t head_stride;    /* in elements */
} orc_kv_t;

static inline double bf16_to_f64(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

static double dot_qk(const double *q, const uint16_t *k, int d) {
    double s = 0.0;
    for (int e = 0; e < d; ++e) s += q[e] * bf16_to_f64(k[e]);
    return s;
}

/* log(sum(exp(x[0..n)))) by the textbook max-shift; -inf for n == 0 */
static double logsumexp(const double *x, int64_t n) {
    if (n <= 0) return -INFINITY;
    double m = x[0];
    for (int64_t i = 1; i < n; ++i) if (x[i] > m) m = x[i];
    if (isinf(m) && m < 0) return -INFINITY;
    double s = 0.0;
    for (int64_t i = 0; i < n; ++i) s += exp(x[i] - m);
    return m + log(s);
}

static double logaddexp(double a, double b) {
    if (isinf(a) && a < 0) return b;
    if (isinf(b) && b < 0) return a;
    double m = a > b ? a : b;
    return m + log(exp(a - m) + exp(b - m));
}

int ape_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * APE attention for one request.
 *
 * q            bf16 [l_q, H_q, d], element (i, h, e) at q[i*q_token_stride + h*q_head_stride + e]
 * prefix       shared prefix K_P, V_P (len may be 0)
 * ctx[n_ctx]   the cached contexts K_Ci, V_Ci (n_ctx may be 0)
 * qkv          the query segment's own K, V: len l_k >= l_q
 * c            logit scale (1/sqrt(d) in the paper)
 * T, S         temperature and scaling factor of Eq. 5
 * per_context  0: Eq. 5 (one context segment);  1: Eq. 11-12 (S on each context's LSE)
 * rows [row_begin,row_end) and heads [head_begin,head_end) are evaluated; the others are left untouched.
 * out          fp64 [l_q, H_q, d] dense
 * lse          fp64 [l_q, H_q]   log of the Eq. 5 denominator           (nullable)
 * lse_ctx      fp64 [l_q, H_q]   LogSumExp of the tempered context logits (nullable)
 * wsum         fp64 [l_q, H_q]   sum of all final weights (must be 1)     (nullable)
 * returns 0, or -1 on bad arguments, -2 on allocation failure.
 */
int ape_oracle_attend(const uint16_t *q, int64_t l_q, int64_t q_token_stride, int64_t q_head_stride,
                      int H_q, int H_kv, int d, double c,
                      const orc_kv_t *prefix, const orc_kv_t *ctx, int n_ctx, const orc_kv_t *qkv,
                      double T, double S, int per_context,
                      int64_t row_begin, int64_t row_end, int head_begin, int head_end,
                      double *out, double *lse, double *lse_ctx, double *wsum)
{
    if (!q || !out || !prefix || !qkv || H_q <= 0 || H_kv <= 0 || H_q % H_kv || d <= 0) return -1;
    if (!(T > 0.0) || !(S > 0.0) || n_ctx < 0 || (n_ctx > 0 && !ctx)) return -1;
    if (qkv->len < l_q || row_begin < 0 || row_end > l_q || head_begin < 0 || head_end > H_q) return -1;

    const int G = H_q / H_kv;
    const int64_t l_P = prefix->len, l_k = qkv->len;
    int64_t L_C = 0;
    for (int n = 0; n < n_ctx; ++n) L_C += ctx[n].len;

    const int64_t n_rows = row_end - row_begin, n_heads = head_end - head_begin;
    if (n_rows <= 0 || n_heads <= 0) return 0;
    int failed = 0;

    #pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int64_t i = row_begin; i < row_end; ++i) {
        for (int h = head_begin; h < head_end; ++h) {
            const int g = h / G;
            double *qd  = (double *)malloc(sizeof(double) * (size_t)d);
            double *x_P = (double *)malloc(sizeof(double) * (size_t)(l_P > 0 ? l_P : 1));
            double *x_C = (double *)malloc(sizeof(double) * (size_t)(L_C > 0 ? L_C : 1));
            double *x_Q = (double *)malloc(sizeof(double) * (size_t)(l_k > 0 ? l_k : 1));
            double *lse_n = (double *)malloc(sizeof(double) * (size_t)(n_ctx > 0 ? n_ctx : 1));
            if (!qd || !x_P || !x_C || !x_Q || !lse_n) {
                #pragma omp atomic write
                failed = 1;
                free(qd); free(x_P); free(x_C); free(x_Q); free(lse_n);
                continue;
            }
            for (int e = 0; e < d; ++e) qd[e] = bf16_to_f64(q[i * q_token_stride + h * q_head_stride + e]);

            /* logits of the shared prefix: a_{P,j} = exp(q k_{P,j} / sqrt(d))  (Eq. 5) */
            for (int64_t j = 0; j < l_P; ++j)
                x_P[j] = c * dot_qk(qd, prefix->k + j * prefix->token_stride + g * prefix->head_stride, d);

            /* tempered logits of every context token, unmasked: a'_{Ci,j} = exp(q k_{Ci,j} / (T sqrt(d))) */
            int64_t t = 0;
            for (int n = 0; n < n_ctx; ++n)
                for (int64_t j = 0; j < ctx[n].len; ++j, ++t)
                    x_C[t] = (c / T) * dot_qk(qd, ctx[n].k + j * ctx[n].token_stride + g * ctx[n].head_stride, d);

            /* logits of the query's own keys, causal: row i sees keys j <= i + (l_k - l_q) */
            const int64_t n_vis = i + (l_k - l_q) + 1;
            for (int64_t j = 0; j < n_vis; ++j)
                x_Q[j] = c * dot_qk(qd, qkv->k + j * qkv->token_stride + g * qkv->head_stride, d);

            /* segment log-sum-exps (appendix, hierarchical softmax identity) */
            const double lse_P = logsumexp(x_P, l_P);
            const double lse_Q = logsumexp(x_Q, n_vis);
            const double lse_o = logaddexp(lse_P, lse_Q);
            const double lse_C = logsumexp(x_C, L_C);

            /* log of the context mass after the scaling factor */
            double lse_C_scaled;
            if (!per_context) {
                /* Eq. 5: (sum_i sum_j a'_{Ci,j})^S */
                lse_C_scaled = (L_C > 0) ? S * lse_C : -INFINITY;
            } else {
                /* Eq. 11-12: sum_i (sum_j a'_{Ci,j})^S */
                lse_C_scaled = -INFINITY;
                int64_t off = 0;
                for (int n = 0; n < n_ctx; ++n) {
                    lse_n[n] = logsumexp(x_C + off, ctx[n].len);
                    if (ctx[n].len > 0) lse_C_scaled = logaddexp(lse_C_scaled, S * lse_n[n]);
                    off += ctx[n].len;
                }
            }
            /* log of the denominator  Z_P + Z_C^S + Z_Q  of Eq. 5 */
            const double Lambda = logaddexp(lse_o, lse_C_scaled);

            double *o = out + ((size_t)i * H_q + h) * (size_t)d;
            for (int e = 0; e < d; ++e) o[e] = 0.0;
            double ws = 0.0;

            for (int64_t j = 0; j < l_P; ++j) {
                const double w = exp(x_P[j] - Lambda);
                const uint16_t *vr = prefix->v + j * prefix->token_stride + g * prefix->head_stride;
                for (int e = 0; e < d; ++e) o[e] += w * bf16_to_f64(vr[e]);
                ws += w;
            }
            /* context weights: a' * (context sum)^(S-1) / denominator */
            t = 0;
            for (int n = 0; n < n_ctx; ++n) {
                const double bias = per_context ? (S - 1.0) * lse_n[n] : (S - 1.0) * lse_C;
                for (int64_t j = 0; j < ctx[n].len; ++j, ++t) {
                    const double w = exp(x_C[t] + bias - Lambda);
                    const uint16_t *vr = ctx[n].v + j * ctx[n].token_stride + g * ctx[n].head_stride;
                    for (int e = 0; e < d; ++e) o[e] += w * bf16_to_f64(vr[e]);
                    ws += w;
                }
            }
            for (int64_t j = 0; j < n_vis; ++j) {
                const double w = exp(x_Q[j] - Lambda);
                const uint16_t *vr = qkv->v + j * qkv->token_stride + g * qkv->head_stride;
                for (int e = 0; e < d; ++e) o[e] += w * bf16_to_f64(vr[e]);
                ws += w;
            }
            if (lse)     lse[(size_t)i * H_q + h] = Lambda;
            if (lse_ctx) lse_ctx[(size_t)i * H_q + h] = lse_C;
            if (wsum)    wsum[(size_t)i * H_q + h] = ws;
            free(qd); free(x_P); free(x_C); free(x_Q); free(lse_n);
        }
    }
    return failed ? -2 : 0;
}

/*
 * Block-diagonal context encoding (pre-caching step): row r of context i attends to
 * the whole shared prefix and to tokens 0..r of its own context, nothing else;
 * plain softmax with scale c.
 *
 * ctx_q[n]     bf16 [len_n, H_q, d] queries of context n (same strides for all contexts)
 * ctx[n]       K, V of context n
 * out[n]       fp64 [len_n, H_q, d] dense; lse[n] fp64 [len_n, H_q] (array or its entries nullable)
 * Rows [row_begin,row_end) of every context are evaluated (clamped to its length).
 */
int ape_oracle_encode(const uint16_t *const *ctx_q, int64_t q_token_stride, int64_t q_head_stride,
                      int H_q, int H_kv, int d, double c,
                      const orc_kv_t *prefix, const orc_kv_t *ctx, int n_ctx,
                      int64_t row_begin, int64_t row_end,
                      double *const *out, double *const *lse)
{
    if (!ctx_q || !prefix || !ctx || !out || H_q <= 0 || H_kv <= 0 || H_q % H_kv || d <= 0 || n_ctx < 0) return -1;
    const int G = H_q / H_kv;
    const int64_t l_P = prefix->len;
    int failed = 0;

    for (int n = 0; n < n_ctx; ++n) {
        const int64_t r0 = row_begin < 0 ? 0 : row_begin;
        const int64_t r1 = row_end > ctx[n].len ? ctx[n].len : row_end;
        #pragma omp parallel for collapse(2) schedule(dynamic, 1)
        for (int64_t r = r0; r < r1; ++r) {
            for (int h = 0; h < H_q; ++h) {
                const int g = h / G;
                const int64_t n_keys = l_P + r + 1;
                double *qd = (double *)malloc(sizeof(double) * (size_t)d);
                double *x  = (double *)malloc(sizeof(double) * (size_t)n_keys);
                if (!qd || !x) {
                    #pragma omp atomic write
                    failed = 1;
                    free(qd); free(x);
                    continue;
                }
                for (int e = 0; e < d; ++e) qd[e] = bf16_to_f64(ctx_q[n][r * q_token_stride + h * q_head_stride + e]);
                for (int64_t j = 0; j < l_P; ++j)
                    x[j] = c * dot_qk(qd, prefix->k + j * prefix->token_stride + g * prefix->head_stride, d);
                for (int64_t j = 0; j <= r; ++j)
                    x[l_P + j] = c * dot_qk(qd, ctx[n].k + j * ctx[n].token_stride + g * ctx[n].head_stride, d);
                const double L = logsumexp(x, n_keys);
                double *o = out[n] + ((size_t)r * H_q + h) * (size_t)d;
                for (int e = 0; e < d; ++e) o[e] = 0.0;
                for (int64_t j = 0; j < n_keys; ++j) {
                    const double w = exp(x[j] - L);
                    const uint16_t *vr = (j < l_P)
                        ? prefix->v + j * prefix->token_stride + g * prefix->head_stride
                        : ctx[n].v + (j - l_P) * ctx[n].token_stride + g * ctx[n].head_stride;
                    for (int e = 0; e < d; ++e) o[e] += w * bf16_to_f64(vr[e]);
                }
                if (lse && lse[n]) lse[n][(size_t)r * H_q + h] = L;
                free(qd); free(x);
            }
        }
    }
    return failed ? -2 : 0;
}

/*
 * APE attention over context TREES for one request (appendix "Hierarchical Formula for APE" applied along the
 * branches of the hierarchy sketched in the appendix "Future Directions").
 *
 * ctx[n], n = 0..n_ctx-1, are the nodes: node n holds its own tokens (possibly none: a pure grouping node) and has the
 * parent parent[n], -1 for a top-level node; parent[n] < n, so children always come after their parent.
 * scaled[n] != 0 marks the nodes that hand S * LogSumExp to their parent (Eq. 11: A^{h'} = S * LogSumExp); the others
 * hand their LogSumExp unchanged (appendix "Hierarchical Formula for Softmax Attention").
 *
 * Per (row, head), level by level:
 *   1. every node's own tokens: V_own = Softmax(q K_n / (T sqrt(d))) V_n, A_own = LogSumExp(q K_n / (T sqrt(d)));
 *   2. from the last node to the first (children before parents): the node's members are its own tokens and its
 *      finished children; A_n = LogSumExp(member A's), V_n = Softmax(member A's) x [member V's]; then the node hands
 *      (V_n, s_n * A_n) to its parent, s_n = S if scaled[n] else 1;
 *   3. the final softmax over [A_other, handed A of every top-level node] x [V_other, V of every top-level node],
 *      A_other / V_other being the non-context segment (prefix + causal query keys), unchanged.
 * Other arguments and outputs as in ape_oracle_attend; lse is the log of the final softmax's denominator.
 */
int ape_oracle_attend_tree(const uint16_t *q, int64_t l_q, int64_t q_token_stride, int64_t q_head_stride,
                           int H_q, int H_kv, int d, double c,
                           const orc_kv_t *prefix, const orc_kv_t *ctx, const int32_t *parent, const uint8_t *scaled,
                           int n_ctx, const orc_kv_t *qkv, double T, double S,
                           int64_t row_begin, int64_t row_end, int head_begin, int head_end,
                           double *out, double *lse)
{
    if (!q || !out || !prefix || !qkv || H_q <= 0 || H_kv <= 0 || H_q % H_kv || d <= 0) return -1;
    if (!(T > 0.0) || !(S > 0.0) || n_ctx < 0 || (n_ctx > 0 && (!ctx || !parent || !scaled))) return -1;
    if (qkv->len < l_q || row_begin < 0 || row_end > l_q || head_begin < 0 || head_end > H_q) return -1;
    for (int n = 0; n < n_ctx; ++n) if (parent[n] < -1 || parent[n] >= n) return -1;

    const int G = H_q / H_kv;
    const int64_t l_P = prefix->len, l_k = qkv->len;
    int64_t max_len = 1;
    for (int n = 0; n < n_ctx; ++n) if (ctx[n].len > max_len) max_len = ctx[n].len;
    if (row_end <= row_begin || head_end <= head_begin) return 0;
    int failed = 0;

    #pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int64_t i = row_begin; i < row_end; ++i) {
        for (int h = head_begin; h < head_end; ++h) {
            const int g = h / G;
            const int64_t n_vis = i + (l_k - l_q) + 1;
            const int64_t n_oth = l_P + n_vis;
            double *qd  = (double *)malloc(sizeof(double) * (size_t)d);
            double *x   = (double *)malloc(sizeof(double) * (size_t)(max_len > n_oth ? max_len : n_oth));
            double *A   = (double *)malloc(sizeof(double) * (size_t)(n_ctx + 1));        /* [n_ctx]: the non-context segment */
            double *V   = (double *)malloc(sizeof(double) * (size_t)(n_ctx + 1) * (size_t)d);
            if (!qd || !x || !A || !V) {
                #pragma omp atomic write
                failed = 1;
                free(qd); free(x); free(A); free(V);
                continue;
            }
            for (int e = 0; e < d; ++e) qd[e] = bf16_to_f64(q[i * q_token_stride + h * q_head_stride + e]);

            /* step 1: every node's own tokens, tempered logits */
            for (int n = 0; n < n_ctx; ++n) {
                double *Vn = V + (size_t)n * d;
                for (int e = 0; e < d; ++e) Vn[e] = 0.0;
                for (int64_t j = 0; j < ctx[n].len; ++j)
                    x[j] = (c / T) * dot_qk(qd, ctx[n].k + j * ctx[n].token_stride + g * ctx[n].head_stride, d);
                A[n] = logsumexp(x, ctx[n].len);
                for (int64_t j = 0; j < ctx[n].len; ++j) {
                    const double w = exp(x[j] - A[n]);
                    const uint16_t *vr = ctx[n].v + j * ctx[n].token_stride + g * ctx[n].head_stride;
                    for (int e = 0; e < d; ++e) Vn[e] += w * bf16_to_f64(vr[e]);
                }
            }
            /* the non-context segment: prefix keys, then the causal query keys, plain scale */
            {
                double *Vo = V + (size_t)n_ctx * d;
                for (int e = 0; e < d; ++e) Vo[e] = 0.0;
                for (int64_t j = 0; j < l_P; ++j)
                    x[j] = c * dot_qk(qd, prefix->k + j * prefix->token_stride + g * prefix->head_stride, d);
                for (int64_t j = 0; j < n_vis; ++j)
                    x[l_P + j] = c * dot_qk(qd, qkv->k + j * qkv->token_stride + g * qkv->head_stride, d);
                A[n_ctx] = logsumexp(x, n_oth);
                for (int64_t j = 0; j < n_oth; ++j) {
                    const double w = exp(x[j] - A[n_ctx]);
                    const uint16_t *vr = (j < l_P) ? prefix->v + j * prefix->token_stride + g * prefix->head_stride
                                                   : qkv->v + (j - l_P) * qkv->token_stride + g * qkv->head_stride;
                    for (int e = 0; e < d; ++e) Vo[e] += w * bf16_to_f64(vr[e]);
                }
            }
            /* step 2: bottom-up.  When node n is reached every child of it (index > n) has been finished and has
             * already been merged into n, one child at a time: merging [own, child_1, ..., child_k] by one softmax
             * equals merging them pairwise (the identity is associative), and at this point A[n] / V[n] hold node n's
             * own tokens and all its children.  Finish n and hand it to its parent. */
            for (int n = n_ctx - 1; n >= 0; --n) {
                const double handed = (scaled[n] && !(isinf(A[n]) && A[n] < 0)) ? S * A[n] : A[n];
                A[n] = handed;
                const int par = parent[n];
                if (par < 0) continue;
                const double An = logaddexp(A[par], handed);
                double *Vp = V + (size_t)par * d, *Vn = V + (size_t)n * d;
                if (!(isinf(An) && An < 0)) {
                    const double wp = (isinf(A[par]) && A[par] < 0) ? 0.0 : exp(A[par] - An);
                    const double wn = (isinf(handed) && handed < 0) ? 0.0 : exp(handed - An);
                    for (int e = 0; e < d; ++e) Vp[e] = wp * Vp[e] + wn * Vn[e];
                }
                A[par] = An;
            }
            /* step 3: the final softmax over the non-context segment and the top-level nodes */
            double Lambda = A[n_ctx];
            for (int n = 0; n < n_ctx; ++n) if (parent[n] < 0) Lambda = logaddexp(Lambda, A[n]);
            double *o = out + ((size_t)i * H_q + h) * (size_t)d;
            {
                const double w = exp(A[n_ctx] - Lambda);
                const double *Vo = V + (size_t)n_ctx * d;
                for (int e = 0; e < d; ++e) o[e] = w * Vo[e];
            }
            for (int n = 0; n < n_ctx; ++n) {
                if (parent[n] >= 0 || (isinf(A[n]) && A[n] < 0)) continue;
                const double w = exp(A[n] - Lambda);
                const double *Vn = V + (size_t)n * d;
                for (int e = 0; e < d; ++e) o[e] += w * Vn[e];
            }
            if (lse) lse[(size_t)i * H_q + h] = Lambda;
            free(qd); free(x); free(A); free(V);
        }
    }
    return failed ? -2 : 0;
}
