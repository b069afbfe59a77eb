/*
 * specroll_ref.c -- CPU oracle for the SpecRoll per-step speculative hot path.
 *
 * TEST INFRASTRUCTURE, NOT PRODUCT CODE.  Only the test-suite, the smoke check and the
 * benchmark's CPU-baseline leg may call this file.  It shares no code with the CUDA
 * library.  Everything is written as the plain definition: literal loops over
 * sequences, nodes and the vocabulary, fp64 arithmetic, dense vocabulary-length
 * residual vectors, no tiling, no online softmax, no sparse-residual shortcut.
 * OpenMP is used only across independent sequences / rows.
 *
 * bf16 tensors arrive as uint16 bit patterns.  bf16 rounding (nearest, ties to even)
 * is applied only where the method's tensors are declared bf16:
 *   - the LayerNorm output fed to the head matrices,
 *   - the corrected head state fed to the vocabulary projection,
 *   - the attention output.
 *
 * Parity status: every function below is pinned by tests that do not go through this
 * file's own formulas (closed forms, brute force, library special cases, the paper's
 * worked example, Monte-Carlo marginals).  What stays "parity unpinned" is absolute
 * agreement with a real trained model: no weights exist here, inputs are synthetic.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define REF_OK 0
#define REF_EINVAL 1
#define REF_MAX_NODES 64
#define REF_MAX_K 64

/* ------------------------------------------------------------------ bf16 <-> fp64 */

static double bf16_to_f64(uint16_t x)
{
    uint32_t u = (uint32_t)x << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* fp64 -> bf16, round to nearest, ties to even, with no intermediate double rounding. */
static uint16_t f64_to_bf16(double v)
{
    float f = (float)v; /* nearest fp32 */
    uint32_t u;
    memcpy(&u, &f, 4);
    if (isnan(v)) return 0x7FC0;
    uint32_t low = u & 0xFFFFu, hi = u >> 16;
    if (low == 0x8000u) {
        /* fp32 value sits on a bf16 midpoint: decide with the exact fp64 value */
        double fd = (double)f;
        if (fd == v) {
            if (hi & 1u) hi += 1; /* true tie -> even */
        } else if (fabs(fd) < fabs(v)) {
            hi += 1; /* true value is beyond the midpoint (away from zero) */
        }
        return (uint16_t)hi;
    }
    if (low > 0x8000u) hi += 1;
    return (uint16_t)hi;
}

int specroll_ref_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void specroll_ref_round_bf16(int64_t n, const double *x, uint16_t *out)
{
    for (int64_t i = 0; i < n; ++i) out[i] = f64_to_bf16(x[i]);
}

/* ------------------------------------------------------------------ topology */

static int tree_depths(int N, const int32_t *parent, int *depth)
{
    if (N < 1 || N > REF_MAX_NODES || parent[0] != -1) return REF_EINVAL;
    depth[0] = 0;
    for (int n = 1; n < N; ++n) {
        if (parent[n] < 0 || parent[n] >= n) return REF_EINVAL;
        depth[n] = depth[parent[n]] + 1;
    }
    return REF_OK;
}

/* ------------------------------------------------------------------ proposal: heads
 *
 * Future-token heads (Eq. "heads" of Sec. 3.2 with the residual MLP of App. C
 * "Future-token proposer"):   z_h = h + SiLU(A_h LN(h) + b_h),
 * followed by the gated hidden-state correction (Eq. "reflex-correction", Sec. 3.4):
 *   u = m / (RMS(m) + eps),  dz = alpha * RMS(z) * u,  z~ = z + dz,
 * with alpha == 0 (or m == NULL) meaning "abstain", and an optional L2 clip
 * |dz| <= clip_c * |z|.
 *
 * h[B,d], A[K,d,d] (row = output unit), bias[K,d], gamma/beta[K,d] nullable,
 * m[B,K,d] fp32 nullable, alpha[B,K] fp32 nullable.
 * Outputs (all nullable): xhat[B,K,d] bf16, z[B,K,d] fp64 (before the correction),
 * zc[B,K,d] fp64 (after it), zt[B,K,d] bf16 (= zc rounded).
 */
int specroll_ref_heads(int B, int K, int d, double ln_eps, double rms_eps, double clip_c,
                       const uint16_t *h, const uint16_t *A, const uint16_t *bias,
                       const uint16_t *gamma, const uint16_t *beta, const float *m,
                       const float *alpha, uint16_t *xhat_out, double *z_out, double *zc_out,
                       uint16_t *zt_out)
{
    if (B < 0 || K < 1 || d < 1) return REF_EINVAL;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        for (int hd = 0; hd < K; ++hd) {
            double *hv = (double *)malloc(sizeof(double) * d);
            double *xh = (double *)malloc(sizeof(double) * d);
            double *z = (double *)malloc(sizeof(double) * d);
            /* LayerNorm: mean, biased variance */
            double mu = 0.0;
            for (int i = 0; i < d; ++i) {
                hv[i] = bf16_to_f64(h[(size_t)b * d + i]);
                mu += hv[i];
            }
            mu /= d;
            double var = 0.0;
            for (int i = 0; i < d; ++i) var += (hv[i] - mu) * (hv[i] - mu);
            var /= d;
            double rstd = 1.0 / sqrt(var + ln_eps);
            for (int i = 0; i < d; ++i) {
                double x = (hv[i] - mu) * rstd;
                if (gamma) x *= bf16_to_f64(gamma[(size_t)hd * d + i]);
                if (beta) x += bf16_to_f64(beta[(size_t)hd * d + i]);
                uint16_t xb = f64_to_bf16(x); /* tensor boundary: bf16 */
                if (xhat_out) xhat_out[((size_t)b * K + hd) * d + i] = xb;
                xh[i] = bf16_to_f64(xb);
            }
            /* residual SiLU MLP */
            const uint16_t *Ah = A + (size_t)hd * d * d;
            for (int o = 0; o < d; ++o) {
                double y = bf16_to_f64(bias[(size_t)hd * d + o]);
                for (int i = 0; i < d; ++i) y += bf16_to_f64(Ah[(size_t)o * d + i]) * xh[i];
                z[o] = hv[o] + y / (1.0 + exp(-y));
            }
            if (z_out)
                for (int i = 0; i < d; ++i) z_out[((size_t)b * K + hd) * d + i] = z[i];
            /* bounded correction */
            double a = (alpha && m) ? (double)alpha[(size_t)b * K + hd] : 0.0;
            if (a != 0.0) {
                const float *mv = m + ((size_t)b * K + hd) * d;
                double sz = 0.0, sm = 0.0;
                for (int i = 0; i < d; ++i) {
                    sz += z[i] * z[i];
                    sm += (double)mv[i] * (double)mv[i];
                }
                double rms_z = sqrt(sz / d), rms_m = sqrt(sm / d);
                double coef = a * rms_z / (rms_m + rms_eps);
                double nd = fabs(coef) * sqrt(sm); /* |dz|_2 */
                double nz = sqrt(sz);
                if (clip_c > 0.0 && nd > clip_c * nz) coef *= clip_c * nz / nd;
                for (int i = 0; i < d; ++i) z[i] += coef * (double)mv[i];
            }
            if (zc_out)
                for (int i = 0; i < d; ++i) zc_out[((size_t)b * K + hd) * d + i] = z[i];
            if (zt_out)
                for (int i = 0; i < d; ++i) zt_out[((size_t)b * K + hd) * d + i] = f64_to_bf16(z[i]);
            free(hv);
            free(xh);
            free(z);
        }
    }
    return REF_OK;
}

/* ------------------------------------------------------------------ proposal: correction before the heads
 *
 * Secondary form of the bounded correction (Sec. 3.4, Eq. "reflex-correction", applied to the last hidden
 * state instead of to each head's output; the wording of this repository's task statement: "Reflex applies
 * its bounded correction to the last hidden state, the K future-token heads run over it").  One memory row
 * and one ratio per sequence:
 *     dh = alpha_b RMS(h_b) m_b / (RMS(m_b) + eps),   |dh|_2 <= clip_c |h_b|_2 if clip_c > 0,
 *     h~_b = h_b + dh   (alpha_b = 0 or m NULL: h~_b = h_b exactly),  rounded to bf16 (it replaces h).
 * hc[B,d] fp64 (unrounded), ht[B,d] bf16; either may be NULL.
 */
int specroll_ref_prehead(int B, int d, double rms_eps, double clip_c, const uint16_t *h, const float *m,
                         const float *alpha, double *hc_out, uint16_t *ht_out)
{
    if (B < 0 || d < 1) return REF_EINVAL;
    for (int b = 0; b < B; ++b) {
        double a = (alpha && m) ? (double)alpha[b] : 0.0;
        double coef = 0.0;
        if (a != 0.0) {
            const float *mv = m + (size_t)b * d;
            double sh = 0.0, sm = 0.0;
            for (int i = 0; i < d; ++i) {
                double hv = bf16_to_f64(h[(size_t)b * d + i]);
                sh += hv * hv;
                sm += (double)mv[i] * (double)mv[i];
            }
            double rms_h = sqrt(sh / d), rms_m = sqrt(sm / d);
            coef = a * rms_h / (rms_m + rms_eps);
            double nd = fabs(coef) * sqrt(sm); /* |dh|_2 */
            double nh = sqrt(sh);
            if (clip_c > 0.0 && nd > clip_c * nh) coef *= clip_c * nh / nd;
        }
        for (int i = 0; i < d; ++i) {
            double hv = bf16_to_f64(h[(size_t)b * d + i]);
            double v = (a != 0.0) ? hv + coef * (double)m[(size_t)b * d + i] : hv;
            if (hc_out) hc_out[(size_t)b * d + i] = v;
            if (ht_out) ht_out[(size_t)b * d + i] = (a != 0.0) ? f64_to_bf16(v) : h[(size_t)b * d + i];
        }
    }
    return REF_OK;
}

/* ------------------------------------------------------------------ proposal: vocabulary projection
 *
 * logits[r, v] = W_v . zt_r  (shared, frozen projection; Eq. "heads", second line).
 */
static void lm_row(int V, int d, const uint16_t *zt_row, const uint16_t *W, double *out)
{
    double *x = (double *)malloc(sizeof(double) * d);
    for (int i = 0; i < d; ++i) x[i] = bf16_to_f64(zt_row[i]);
    for (int v = 0; v < V; ++v) {
        const uint16_t *wr = W + (size_t)v * d;
        double s = 0.0;
        for (int i = 0; i < d; ++i) s += bf16_to_f64(wr[i]) * x[i];
        out[v] = s;
    }
    free(x);
}

int specroll_ref_lm_logits(int M, int V, int d, const uint16_t *zt, const uint16_t *W,
                           double *logits)
{
#pragma omp parallel for schedule(dynamic)
    for (int r = 0; r < M; ++r) lm_row(V, d, zt + (size_t)r * d, W, logits + (size_t)r * V);
    return REF_OK;
}

/* k largest of a row, ordered by (value descending, index ascending). Plain selection. */
static void topk_row(int V, int k, const double *x, int32_t *id, float *val)
{
    for (int j = 0; j < k; ++j) {
        int best = -1;
        for (int v = 0; v < V; ++v) {
            int taken = 0;
            for (int t = 0; t < j; ++t)
                if (id[t] == v) taken = 1;
            if (taken) continue;
            if (best < 0 || x[v] > x[best]) best = v; /* strict > keeps the lowest index on ties */
        }
        id[j] = best;
        val[j] = (float)x[best];
    }
}

int specroll_ref_topk(int M, int V, int k, const double *logits, int32_t *cand_id, float *cand_logit)
{
    if (k < 1 || k > V || k > REF_MAX_K) return REF_EINVAL;
#pragma omp parallel for schedule(dynamic)
    for (int r = 0; r < M; ++r)
        topk_row(V, k, logits + (size_t)r * V, cand_id + (size_t)r * k, cand_logit + (size_t)r * k);
    return REF_OK;
}

int specroll_ref_lm_topk(int M, int V, int d, int k, const uint16_t *zt, const uint16_t *W,
                         int32_t *cand_id, float *cand_logit)
{
    if (k < 1 || k > V || k > REF_MAX_K) return REF_EINVAL;
#pragma omp parallel for schedule(dynamic)
    for (int r = 0; r < M; ++r) {
        double *row = (double *)malloc(sizeof(double) * V);
        lm_row(V, d, zt + (size_t)r * d, W, row);
        topk_row(V, k, row, cand_id + (size_t)r * k, cand_logit + (size_t)r * k);
        free(row);
    }
    return REF_OK;
}

/* ------------------------------------------------------------------ proposal: tree draw
 *
 * Tree proposal law (App. B.1, Eq. "slotq" / "childlist"): the children of node u are an
 * ordered list drawn WITHOUT replacement from the support C_u = the k candidates of
 * head depth(u)+1.  Slot j draws from the head distribution renormalised on the
 * candidates not yet taken:  q_{u,j}(v) = 1[v in R_{u,j}] qbar(v) / sum_{R_{u,j}} qbar.
 * qbar is softmax(logit / T); restricted to R it only needs the candidate logits.
 * The draw is inverse-CDF in candidate order with the caller's uniform.
 *
 * slot_weights(): q_{u,j} on the k candidate slots (0 on taken ones).
 */
static void slot_weights(int k, const float *cl, const int *taken, double T, double *q)
{
    double mx = -INFINITY;
    for (int c = 0; c < k; ++c)
        if (!taken[c] && (double)cl[c] > mx) mx = (double)cl[c];
    double s = 0.0;
    for (int c = 0; c < k; ++c) {
        q[c] = taken[c] ? 0.0 : exp(((double)cl[c] - mx) / T);
        s += q[c];
    }
    for (int c = 0; c < k; ++c) q[c] /= s;
}

int specroll_ref_tree_draw(int B, int N, int K, int k, double T, const int32_t *parent,
                           const int32_t *anchor, const int32_t *cand_id, const float *cand_logit,
                           const float *u_draw, int32_t *tree_tok, uint8_t *tree_cand,
                           double *slot_q)
{
    int depth[REF_MAX_NODES];
    if (tree_depths(N, parent, depth) != REF_OK || k < 1 || k > REF_MAX_K) return REF_EINVAL;
    for (int n = 0; n < N; ++n)
        if (depth[n] > K) return REF_EINVAL;
#pragma omp parallel for schedule(static)
    for (int b = 0; b < B; ++b) {
        tree_tok[(size_t)b * N] = anchor[b];
        tree_cand[(size_t)b * N] = 255;
        slot_q[(size_t)b * N] = 1.0;
        for (int n = 1; n < N; ++n) {
            int u = parent[n], hd = depth[n] - 1;
            const float *cl = cand_logit + ((size_t)b * K + hd) * k;
            const int32_t *ci = cand_id + ((size_t)b * K + hd) * k;
            int taken[REF_MAX_K] = {0};
            for (int e = 1; e < n; ++e) /* earlier children of the same parent */
                if (parent[e] == u) taken[tree_cand[(size_t)b * N + e]] = 1;
            double q[REF_MAX_K];
            slot_weights(k, cl, taken, T, q);
            double uu = (double)u_draw[(size_t)b * N + n], cum = 0.0;
            int pick = -1, last = -1;
            for (int c = 0; c < k; ++c) {
                if (taken[c]) continue;
                last = c;
                cum += q[c];
                if (cum > uu) {
                    pick = c;
                    break;
                }
            }
            if (pick < 0) pick = last;
            tree_tok[(size_t)b * N + n] = ci[pick];
            tree_cand[(size_t)b * N + n] = (uint8_t)pick;
            slot_q[(size_t)b * N + n] = q[pick];
        }
    }
    return REF_OK;
}

/* Whole proposal step: heads -> projection -> per-head top-k -> tree draw. */
int specroll_ref_propose(int B, int N, int K, int k, int d, int V, double T, double ln_eps,
                         double rms_eps, double clip_c, const uint16_t *h, const int32_t *anchor,
                         const uint16_t *A, const uint16_t *bias, const uint16_t *gamma,
                         const uint16_t *beta, const uint16_t *W, const float *m,
                         const float *alpha, const int32_t *parent, const float *u_draw,
                         int32_t *cand_id, float *cand_logit, int32_t *tree_tok,
                         uint8_t *tree_cand, double *slot_q)
{
    uint16_t *zt = (uint16_t *)malloc(sizeof(uint16_t) * (size_t)B * K * d);
    int rc = specroll_ref_heads(B, K, d, ln_eps, rms_eps, clip_c, h, A, bias, gamma, beta, m, alpha,
                                NULL, NULL, NULL, zt);
    if (rc == REF_OK) rc = specroll_ref_lm_topk(B * K, V, d, k, zt, W, cand_id, cand_logit);
    if (rc == REF_OK)
        rc = specroll_ref_tree_draw(B, N, K, k, T, parent, anchor, cand_id, cand_logit, u_draw,
                                    tree_tok, tree_cand, slot_q);
    free(zt);
    return rc;
}

/* ------------------------------------------------------------------ tree attention
 *
 * Packed target verification (App. B.1, Eq. "nodep"): node n must see exactly what an
 * ordinary autoregressive forward at prefix (x<=t, path(n)) sees, i.e. the sequence's
 * cached keys/values followed by the tree rows of n's ancestors and n itself.
 *
 * Q[B,N,Hq,D], Kc/Vc[T_kv,Hkv,D] ragged by kv_indptr[B+1], Kt/Vt[B,N,Hkv,D].
 * Outputs (nullable): O64[B,N,Hq,D] fp64, Obf[B,N,Hq,D] bf16, lse[B,N,Hq] (natural log).
 */
int specroll_ref_tree_attn(int B, int N, int Hq, int Hkv, int D, double scale, const uint16_t *Q,
                           const uint16_t *Kc, const uint16_t *Vc, const int32_t *kv_indptr,
                           const uint16_t *Kt, const uint16_t *Vt, const int32_t *parent,
                           double *O64, uint16_t *Obf, double *lse)
{
    int depth[REF_MAX_NODES];
    if (tree_depths(N, parent, depth) != REF_OK || Hkv < 1 || Hq % Hkv) return REF_EINVAL;
    int G = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        for (int n = 0; n < N; ++n) {
            int L = kv_indptr[b + 1] - kv_indptr[b];
            /* ancestors of n, including n, root first */
            int anc[REF_MAX_NODES], na = 0;
            for (int a = n; a >= 0; a = parent[a]) anc[na++] = a;
            int nk = L + na;
            double *s = (double *)malloc(sizeof(double) * nk);
            for (int hq = 0; hq < Hq; ++hq) {
                int hk = hq / G;
                const uint16_t *q = Q + (((size_t)b * N + n) * Hq + hq) * D;
                for (int j = 0; j < nk; ++j) {
                    const uint16_t *kr;
                    if (j < L)
                        kr = Kc + ((size_t)(kv_indptr[b] + j) * Hkv + hk) * D;
                    else
                        kr = Kt + (((size_t)b * N + anc[na - 1 - (j - L)]) * Hkv + hk) * D;
                    double acc = 0.0;
                    for (int t = 0; t < D; ++t) acc += bf16_to_f64(q[t]) * bf16_to_f64(kr[t]);
                    s[j] = acc * scale;
                }
                double mx = -INFINITY;
                for (int j = 0; j < nk; ++j)
                    if (s[j] > mx) mx = s[j];
                double den = 0.0;
                for (int j = 0; j < nk; ++j) {
                    s[j] = exp(s[j] - mx);
                    den += s[j];
                }
                size_t oo = (((size_t)b * N + n) * Hq + hq) * D;
                for (int t = 0; t < D; ++t) {
                    double acc = 0.0;
                    for (int j = 0; j < nk; ++j) {
                        const uint16_t *vr;
                        if (j < L)
                            vr = Vc + ((size_t)(kv_indptr[b] + j) * Hkv + hk) * D;
                        else
                            vr = Vt + (((size_t)b * N + anc[na - 1 - (j - L)]) * Hkv + hk) * D;
                        acc += s[j] * bf16_to_f64(vr[t]);
                    }
                    acc /= den;
                    if (O64) O64[oo + t] = acc;
                    if (Obf) Obf[oo + t] = f64_to_bf16(acc);
                }
                if (lse) lse[((size_t)b * N + n) * Hq + hq] = mx + log(den);
            }
            free(s);
        }
    }
    return REF_OK;
}

/* ------------------------------------------------------------------ exact verification
 *
 * Node-wise acceptance and residuals (App. B.2, Eq. "nodeaccept" / "noderesidual",
 * Algorithm "Exact node-wise tree verification"):
 *   r <- p_u ; for each child slot j: y, q = q_{u,j};
 *     accept with probability min(1, r(y)/q(y))  -> commit y, recurse into the child
 *     else r <- [r - q]_+ / sum [r - q]_+
 *   all rejected -> fallback token ~ r ; accepted childless node -> bonus token ~ p_node.
 * p_u = softmax(logits_u / T) over the full vocabulary.
 *
 * Readings fixed here: the acceptance test is  U < min(1, ratio)  with 24-bit uniforms
 * in [0,1); if q(y) underflows to 0 the ratio is +inf when r(y) > 0 and 0 otherwise; if
 * the residual normaliser is <= 1e-300 the residual is left unchanged.  The terminal
 * token is the first token id whose cumulative (token-id order) mass exceeds
 * u_fin * total; the last token with positive mass if none does.
 *
 * logits[B,N,V] bf16; tree_tok[B,N]; tree_cand[B,N] (candidate slot index of each node's
 * token in its head's list); cand_id/cand_logit[B,K,k]; u_acc[B,N]; u_fin[B].
 * Outputs: n_acc[B]; path_node[B,K+1] (node at depth i of the committed path, -1 after);
 * out_tok[B,K+1] (accepted tokens then the terminal token, -1 after); term_node[B];
 * term_kind[B] (0 fallback, 1 bonus); row_max,row_sum[B,N] (M_n and S_n of the softmax);
 * min_margin[B] = min |U - ratio| over tested slots (+inf if none);
 * fin_margin[B] = distance of u_fin*total to the nearest bracket end, over total.
 */
/* Nucleus truncation of one target distribution (the experiments sample the target at nucleus threshold 0.95,
 * App. "Implementation and Reproducibility Details"; the paper does not say how ties are cut).  Reading: the
 * tokens are taken in order of decreasing probability until their mass first reaches top_p, and every token
 * that ties with the last one taken is kept as well, so the kept set does not depend on how equal
 * probabilities are ordered.  p[V] (sums to 1) is replaced by its renormalised restriction to the kept set.
 * thr_p = smallest kept probability, kept_mass = mass kept (before renormalising),
 * margin = distance of top_p to the nearer of the two cumulative masses that bracket it. */
typedef struct { double p; int v; } nuc_item;
static int nuc_cmp(const void *a, const void *b)
{
    const nuc_item *x = (const nuc_item *)a, *y = (const nuc_item *)b;
    if (x->p > y->p) return -1;
    if (x->p < y->p) return 1;
    return (x->v > y->v) - (x->v < y->v);
}
static void nucleus(int V, double *p, double top_p, nuc_item *scratch, double *thr_p, double *kept_mass,
                    double *margin)
{
    for (int v = 0; v < V; ++v) {
        scratch[v].p = p[v];
        scratch[v].v = v;
    }
    qsort(scratch, (size_t)V, sizeof(nuc_item), nuc_cmp);
    double cum = 0.0, above = 0.0; /* above = mass of the probabilities strictly larger than the current one */
    int i = 0;
    for (; i < V; ++i) {
        if (i > 0 && scratch[i].p < scratch[i - 1].p) above = cum;
        cum += scratch[i].p;
        if (cum >= top_p) break;
    }
    if (i >= V) i = V - 1; /* rounding kept the total below top_p: keep everything */
    const double pv = scratch[i].p;
    double all = above; /* mass of everything >= pv */
    for (int j = 0; j < V; ++j)
        if (scratch[j].p == pv) all += scratch[j].p;
    for (int v = 0; v < V; ++v) p[v] = (p[v] >= pv) ? p[v] / all : 0.0;
    *thr_p = pv;
    *kept_mass = all;
    double m1 = top_p - above, m2 = all - top_p;
    if (m1 < 0) m1 = -m1;
    if (m2 < 0) m2 = -m2;
    *margin = m1 < m2 ? m1 : m2;
}

static int verify_impl(int B, int N, int K, int k, int V, double T, double top_p, const uint16_t *logits,
                        const int32_t *parent, const int32_t *tree_tok, const uint8_t *tree_cand,
                        const int32_t *cand_id, const float *cand_logit, const float *u_acc,
                        const float *u_fin, int32_t *n_acc, int32_t *path_node, int32_t *out_tok,
                        int32_t *term_node, int32_t *term_kind, double *row_max, double *row_sum,
                        double *min_margin, double *fin_margin, double *nuc_thr, double *nuc_sum,
                        double *nuc_margin)
{
    const int truncate = top_p > 0.0 && top_p < 1.0;
    int depth[REF_MAX_NODES];
    if (tree_depths(N, parent, depth) != REF_OK || k < 1 || k > REF_MAX_K || V < 1) return REF_EINVAL;
    for (int n = 0; n < N; ++n)
        if (depth[n] > K) return REF_EINVAL;
#pragma omp parallel for schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        double *r = (double *)malloc(sizeof(double) * V);
        double *q = (double *)malloc(sizeof(double) * V);
        nuc_item *scratch = truncate ? (nuc_item *)malloc(sizeof(nuc_item) * V) : NULL;
        double nmin = INFINITY; /* smallest nucleus margin among the nodes whose distribution was used */
        /* softmax statistics of every node */
        for (int n = 0; n < N; ++n) {
            const uint16_t *lg = logits + ((size_t)b * N + n) * V;
            double mx = -INFINITY;
            for (int v = 0; v < V; ++v) {
                double x = bf16_to_f64(lg[v]);
                if (x > mx) mx = x;
            }
            double s = 0.0;
            for (int v = 0; v < V; ++v) s += exp((bf16_to_f64(lg[v]) - mx) / T);
            row_max[(size_t)b * N + n] = mx;
            row_sum[(size_t)b * N + n] = s;
        }
        int32_t *pn = path_node + (size_t)b * (K + 1), *ot = out_tok + (size_t)b * (K + 1);
        for (int i = 0; i <= K; ++i) pn[i] = ot[i] = -1;
        int u = 0, nacc = 0, kind = 0;
        double mm = INFINITY;
        pn[0] = 0;
        for (;;) {
            /* r <- p_u */
            const uint16_t *lg = logits + ((size_t)b * N + u) * V;
            double mx = row_max[(size_t)b * N + u], s = row_sum[(size_t)b * N + u];
            for (int v = 0; v < V; ++v) r[v] = exp((bf16_to_f64(lg[v]) - mx) / T) / s;
            if (truncate) { /* the target distribution of this node is its nucleus */
                double thr_p, kept, mg;
                nucleus(V, r, top_p, scratch, &thr_p, &kept, &mg);
                if (mg < nmin) nmin = mg;
                if (nuc_thr) nuc_thr[(size_t)b * N + u] = mx + T * log(thr_p * s); /* logit of the smallest kept token */
                if (nuc_sum) nuc_sum[(size_t)b * N + u] = kept * s;               /* kept mass in units of exp((l-M)/T) */
            }
            int nchild = 0, accepted = -1;
            for (int c = u + 1; c < N; ++c)
                if (parent[c] == u) ++nchild;
            if (nchild == 0) { /* childless: bonus if reached by acceptance, else (lone root) fallback */
                kind = (u != 0) ? 1 : 0;
                break;
            }
            int hd = depth[u]; /* children of u are proposed by head depth(u)+1 (0-based index depth(u)) */
            const float *cl = cand_logit + ((size_t)b * K + hd) * k;
            const int32_t *ci = cand_id + ((size_t)b * K + hd) * k;
            int taken[REF_MAX_K] = {0};
            for (int c = u + 1; c < N && accepted < 0; ++c) {
                if (parent[c] != u) continue;
                double qs[REF_MAX_K];
                slot_weights(k, cl, taken, T, qs);
                for (int v = 0; v < V; ++v) q[v] = 0.0;
                for (int j = 0; j < k; ++j) q[ci[j]] += qs[j];
                int y = tree_tok[(size_t)b * N + c];
                double ratio;
                if (q[y] > 0.0)
                    ratio = r[y] / q[y];
                else
                    ratio = (r[y] > 0.0) ? INFINITY : 0.0;
                double uu = (double)u_acc[(size_t)b * N + c];
                double mg = fabs(uu - ratio);
                if (mg < mm) mm = mg;
                if (uu < (ratio < 1.0 ? ratio : 1.0)) {
                    accepted = c;
                } else {
                    double Z = 0.0;
                    for (int v = 0; v < V; ++v) {
                        double t = r[v] - q[v];
                        q[v] = t > 0.0 ? t : 0.0; /* reuse q as the clipped difference */
                        Z += q[v];
                    }
                    if (Z > 1e-300)
                        for (int v = 0; v < V; ++v) r[v] = q[v] / Z;
                    taken[tree_cand[(size_t)b * N + c]] = 1;
                }
            }
            if (accepted < 0) {
                kind = 0; /* all siblings rejected: fallback from the final residual r */
                break;
            }
            ot[nacc] = tree_tok[(size_t)b * N + accepted];
            ++nacc;
            pn[nacc] = accepted;
            u = accepted;
        }
        /* terminal token from mass r (fallback residual, or p_u for a bonus: r == p_u here) */
        double total = 0.0;
        for (int v = 0; v < V; ++v) total += r[v];
        double target = (double)u_fin[b] * total, cum = 0.0, prev = 0.0;
        int tok = -1, lastpos = -1;
        for (int v = 0; v < V; ++v) {
            if (r[v] > 0.0) lastpos = v;
            prev = cum;
            cum += r[v];
            if (cum > target) {
                tok = v;
                break;
            }
        }
        if (tok < 0) {
            tok = lastpos;
            prev = cum;
        }
        double fm = fabs(target - prev);
        if (fabs(cum - target) < fm) fm = fabs(cum - target);
        ot[nacc] = tok;
        n_acc[b] = nacc;
        term_node[b] = u;
        term_kind[b] = kind;
        if (min_margin) min_margin[b] = mm;
        if (fin_margin) fin_margin[b] = fm / total;
        if (nuc_margin) nuc_margin[b] = nmin;
        free(r);
        free(q);
        free(scratch);
    }
    return REF_OK;
}

int specroll_ref_verify(int B, int N, int K, int k, int V, double T, const uint16_t *logits,
                        const int32_t *parent, const int32_t *tree_tok, const uint8_t *tree_cand,
                        const int32_t *cand_id, const float *cand_logit, const float *u_acc,
                        const float *u_fin, int32_t *n_acc, int32_t *path_node, int32_t *out_tok,
                        int32_t *term_node, int32_t *term_kind, double *row_max, double *row_sum,
                        double *min_margin, double *fin_margin)
{
    return verify_impl(B, N, K, k, V, T, 1.0, logits, parent, tree_tok, tree_cand, cand_id, cand_logit, u_acc, u_fin,
                       n_acc, path_node, out_tok, term_node, term_kind, row_max, row_sum, min_margin, fin_margin,
                       NULL, NULL, NULL);
}

/* The same walk against nucleus-truncated target distributions (top_p in (0,1); >= 1 keeps everything).
 * Extra outputs: nuc_thr, nuc_sum [B,N], written for the nodes the walk visited only (others untouched):
 * the logit of the smallest kept token and the kept mass in units of exp((l - M)/T);
 * nuc_margin[B] = smallest distance of top_p to a bracketing cumulative mass over the visited nodes. */
int specroll_ref_verify_nucleus(int B, int N, int K, int k, int V, double T, double top_p, const uint16_t *logits,
                                const int32_t *parent, const int32_t *tree_tok, const uint8_t *tree_cand,
                                const int32_t *cand_id, const float *cand_logit, const float *u_acc,
                                const float *u_fin, int32_t *n_acc, int32_t *path_node, int32_t *out_tok,
                                int32_t *term_node, int32_t *term_kind, double *row_max, double *row_sum,
                                double *min_margin, double *fin_margin, double *nuc_thr, double *nuc_sum,
                                double *nuc_margin)
{
    return verify_impl(B, N, K, k, V, T, top_p, logits, parent, tree_tok, tree_cand, cand_id, cand_logit, u_acc,
                       u_fin, n_acc, path_node, out_tok, term_node, term_kind, row_max, row_sum, min_margin,
                       fin_margin, nuc_thr, nuc_sum, nuc_margin);
}

/* Node budget N_t = clip(floor(C_hw / B_t), N_min, N_max)  (Eq. "verification-budget"). */
int32_t specroll_ref_node_budget(int32_t C_hw, int32_t B_active, int32_t N_min, int32_t N_max)
{
    if (B_active < 1) return N_max;
    int32_t n = C_hw / B_active;
    if (n < N_min) n = N_min;
    if (n > N_max) n = N_max;
    return n;
}
