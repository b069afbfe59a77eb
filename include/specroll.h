/*
 * specroll.h -- C ABI of the SpecRoll per-step speculative hot path for NVIDIA B200 (sm_100a).
 *
 * One speculative round of the rollout engine (Algorithm "One exact speculative round") is,
 * per step: proposal -> packed target forward (tree attention in every layer) -> exact
 * node-wise verification.  This library provides those three pieces as stateless calls.
 *
 * Conventions (all entry points):
 *   - Pointers whose name ends in _host are HOST pointers, read during the call only.
 *     Every other pointer is a DEVICE pointer owned by the caller; the library never
 *     allocates, frees or retains memory and never synchronises the device.
 *   - bf16 tensors are passed as `const void*` / `void*` to 2-byte bf16 elements.
 *   - All tensors are dense, row-major, 16-byte aligned at their base.
 *   - All work is enqueued on `cuda_stream` (a cudaStream_t; NULL = default stream).
 *   - Scratch memory comes from `workspace` (device, 256-byte aligned), whose size is given
 *     by the matching *_workspace_bytes query.  Calls that share a workspace must not
 *     overlap on the device.
 *   - Return value: SPECROLL_OK or an error code; on error nothing has been enqueued
 *     (except SPECROLL_ECUDA, where earlier launches of the call may have been).
 *   - An empty batch (B = 0, or R = 0 records) is valid: the descriptor and the topology are
 *     checked, nothing is enqueued, and the per-sequence arrays, which are empty, may be NULL.
 *   - Tree topology: parent_host[N] with parent[0] = -1 and 0 <= parent[n] < n; the tree is
 *     shared by all B sequences of a call.  depth(n) <= K, every node has <= k children,
 *     N <= 64.  The children of a node, in increasing node index, are its ordered slots.
 *     Node 0 is the anchor (an exact target sample) and carries no proposal.
 */
#ifndef SPECROLL_H
#define SPECROLL_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPECROLL_OK 0
#define SPECROLL_EINVAL 1     /* bad shape / limit / NULL pointer / malformed topology */
#define SPECROLL_EALIGN 2     /* a base pointer is not 16-byte aligned */
#define SPECROLL_EWORKSPACE 3 /* workspace too small or misaligned */
#define SPECROLL_ECUDA 4      /* a CUDA runtime call or kernel launch failed */
#define SPECROLL_ETIMEOUT 5   /* a bounded device-side wait ran out (read from a status word) */
#define SPECROLL_ELIMIT 6     /* problem larger than a fixed limit: of an allocation-free entry point, of the kernel a
                                 paged cache needs, or of a sequence's own pages */

#define SPECROLL_EINDEX 7     /* debug build only: an index in a caller's device array is out of range */

#define SPECROLL_MAX_NODES 64
#define SPECROLL_MAX_HEADS 8
#define SPECROLL_MAX_TOPK 64

/* Library version (major * 10000 + minor * 100 + patch). */
int specroll_version(void);

/* Debug builds (compiled with -DSPECROLL_CHECK; the paper has no counterpart).  There the kernels check the
 * indices they read from the caller's device arrays (candidate token ids and candidate slots of the
 * verification walk, cache lengths of the attention plan):
 * a bad index is not followed (index 0 is used instead, so the launch completes and nothing is read or
 * written out of bounds) and the first one is remembered.  This call returns SPECROLL_OK, or
 * SPECROLL_EINDEX with *detail (nullable) = the sequence or record it was found in; reset != 0 clears the
 * memory.  It copies from the device synchronously: synchronise the streams the calls were enqueued on
 * first.  In a normal build the checks do not exist and the call returns -1. */
int specroll_check_status(int32_t *detail, int32_t reset);

/* Debug builds only (the paper has no counterpart): arranges for one bounded device-side wait to run out, so
 * that the path on which a kernel gives up can be tested without a fault or a hang.  what == 1: the next
 * specroll_propose leaves out one barrier arrival in its projection kernel (nothing asynchronous is abandoned);
 * the waiting warps give up after the debug build's 20 ms limit, the kernel returns, and
 * specroll_workspace_status reports SPECROLL_ETIMEOUT.  Returns SPECROLL_OK, SPECROLL_EINVAL for an unknown
 * `what`, -1 in a normal build (where nothing of this exists). */
int specroll_check_inject(int32_t what);

/* Human-readable text for a return code; for SPECROLL_ECUDA includes the last CUDA error
 * string seen by the calling thread.  The pointer stays valid until the thread's next call. */
const char *specroll_strerror(int code);

/* Concurrency-aware node budget, Eq. "verification-budget" (Sec. 3.2):
 *   N_t = clip(floor(C_hw / B_active), N_min, N_max);  B_active < 1 gives N_max. */
int32_t specroll_node_budget(int32_t C_hw, int32_t B_active, int32_t N_min, int32_t N_max);

/* ------------------------------------------------------------------------------------------
 * Proposal (Sec. 3.2 Eq. "heads"; App. C "Future-token proposer"; Sec. 3.4 Eq.
 * "reflex-correction"; App. B.1 Eq. "slotq" / "childlist").
 *
 * For every sequence b and head h (predicting position t+h+1):
 *   x^   = LN(h_b) * gamma_h + beta_h           (fp32 statistics, biased variance; bf16 out)
 *   z    = h_b + SiLU(A_h x^ + bias_h)          (bf16 tensor-core product, fp32 accumulate)
 *   z~   = z + alpha_{b,h} RMS(z) m_{b,h} / (RMS(m_{b,h}) + rms_eps), optionally rescaled so
 *          that |z~ - z|_2 <= clip_c |z|_2; alpha = 0 (or m/alpha NULL) abstains; bf16 out
 *   l_v  = W_v . z~  for all v (never written to memory); the k largest, ordered by
 *          (logit descending, token id ascending), go to cand_logit / cand_id
 * and the tree is drawn: node n >= 1 with parent u and depth dd takes a token from head dd's
 * candidates not already used by an earlier child of u, with probability softmax(l / T)
 * renormalised on that remaining set (inverse CDF in candidate order, uniform u_draw[b,n]).
 *
 * Shapes: h[B,d] bf16; anchor_tok[B] i32; A[K,d,d] bf16 (row = output unit); bias[K,d] bf16;
 * ln_gamma/ln_beta[K,d] bf16 or NULL (1 / 0); W[V,d] bf16 (row = token); m[B,K,d] fp32 or NULL;
 * alpha[B,K] fp32 or NULL; u_draw[B,N] fp32 in [0,1).
 * Outputs: cand_id[B,K,k] i32; cand_logit[B,K,k] fp32; tree_tok[B,N] i32 (node 0 = anchor);
 * tree_cand[B,N] u8 (slot of the node's token in its head's list; 255 for node 0);
 * slot_q[B,N] fp32 (probability the node's token had when drawn; 1 for node 0).
 * Limits: d % 64 == 0, V % 8 == 0, 1 <= k <= 64, K <= 8, N <= 64.
 */
typedef struct {
    int32_t B, N, K, k, d, V;
    float temperature; /* T > 0 */
    float ln_eps;      /* LayerNorm epsilon (1e-5 if the caller has no other value) */
    float rms_eps;     /* epsilon of the RMS normalisation of the memory */
    float clip_c;      /* <= 0: no L2 clip */
    int32_t flags;     /* 0, or an OR of the SPECROLL_PROPOSE_* / SPECROLL_REFLEX_* flags below */
} specroll_propose_desc;

/* Run the vocabulary projection on the mma.sync kernel instead of the tcgen05 one (kept for
 * comparison and for k > 8, where it is used anyway). */
#define SPECROLL_PROPOSE_LEGACY_MMA 1
/* Secondary form of the bounded correction (Sec. 3.4 Eq. "reflex-correction" applied once, to the last
 * hidden state, before the heads; the paper's own form corrects each head's output and is the default):
 *   h~_b = bf16(h_b + alpha_b RMS(h_b) m_b / (RMS(m_b) + rms_eps)),  |h~_b - h_b|_2 <= clip_c |h_b|_2,
 * the heads and the projection then run on h~ and their outputs are not corrected.  With this flag
 * m is [B, d] and alpha is [B] (one memory row and one ratio per sequence); alpha_b = 0 or NULL
 * leaves h_b untouched bit for bit. */
#define SPECROLL_REFLEX_PRE_HEAD 2

size_t specroll_propose_workspace_bytes(const specroll_propose_desc *desc);

int specroll_propose(const specroll_propose_desc *desc, const void *h, const int32_t *anchor_tok,
                     const void *A, const void *bias, const void *ln_gamma, const void *ln_beta,
                     const void *W, const float *m, const float *alpha,
                     const int32_t *parent_host, const float *u_draw, int32_t *cand_id,
                     float *cand_logit, int32_t *tree_tok, uint8_t *tree_cand, float *slot_q,
                     void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Reads back the status word that the last specroll_propose or specroll_tree_attn using this
 * workspace left behind: SPECROLL_OK, or SPECROLL_ETIMEOUT if a bounded wait inside a kernel ran
 * out (the call's results are then invalid).  Unlike the other calls this one synchronises
 * `cuda_stream`.  (Housekeeping; the paper has no counterpart.) */
int specroll_workspace_status(const void *workspace, void *cuda_stream);

/* The last step of the proposal alone (App. B.1): draw the tree from given candidate lists.
 * Same arguments and outputs as the corresponding ones of specroll_propose; needs no workspace. */
int specroll_tree_draw(int32_t B, int32_t N, int32_t K, int32_t k, float temperature,
                       const int32_t *parent_host, const int32_t *anchor_tok,
                       const int32_t *cand_id, const float *cand_logit, const float *u_draw,
                       int32_t *tree_tok, uint8_t *tree_cand, float *slot_q, void *cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Tree-verification attention of one layer (App. B.1 Eq. "nodep": the packed forward must
 * equal an ordinary autoregressive forward at every node's own prefix).
 *
 * For sequence b, node n, query head hq (KV head hq / (Hq/Hkv)):
 *   O = softmax(scale * q . [K_cache(b) ; K_tree(b, anc(n))]^T) [V_cache(b) ; V_tree(b, anc(n))]
 * where anc(n) are the ancestors of n including n.
 *
 * Shapes: Q[B,N,Hq,D] bf16; Kc,Vc[T_kv,Hkv,D] bf16, sequence b owning rows
 * kv_indptr[b] .. kv_indptr[b+1]-1; kv_indptr_dev/_host[B+1] i32 (same values; the host copy
 * sizes the launch so no device read-back is needed); kv_indptr[0] must be 0 (Kc and Vc point at
 * the first sequence's first token), else SPECROLL_EINVAL; Kt,Vt[B,N,Hkv,D] bf16.
 * Outputs: O[B,N,Hq,D] bf16; lse[B,N,Hq] fp32 or NULL (natural-log sum-exp of the scaled scores).
 * Limits: D == 64 or 128, Hq % Hkv == 0, N <= 64.
 */
typedef struct {
    int32_t B, N, Hq, Hkv, D;
    float scale;   /* softmax scale (> 0); the method uses 1/sqrt(D) */
    int32_t flags; /* 0, or an OR of the SPECROLL_ATTN_* flags below */
} specroll_attn_desc;

/* Run the attention on the mma.sync kernel instead of the tcgen05 one (kept for comparison). */
#define SPECROLL_ATTN_LEGACY_MMA 1
/* The workspace still holds the work plan of an earlier specroll_tree_attn call with the same
 * descriptor and the same kv_indptr values (typically the previous layer of the same step): do not
 * rebuild it.  Tensors (Q, K, V, O) may differ.  Ignored by the mma.sync kernel. */
#define SPECROLL_ATTN_REUSE_PLAN 2
/* The cache (Kc, Vc, or the pool and its page table) was last written before the kernel that
 * precedes this call in the stream was launched, as is the case for every layer of a verification
 * step whose cache was committed at the end of the step before.  Together with
 * SPECROLL_ATTN_REUSE_PLAN this lets the attention kernel, which is launched as a programmatic
 * dependent of that preceding kernel, fetch its first cache tiles while that kernel is still
 * finishing; Q, the tree's K/V and the outputs are touched only after it has completed.  Without the
 * flag nothing is read before then.  (Scheduling only; results do not depend on it.) */
#define SPECROLL_ATTN_CACHE_SETTLED 4
/* The tcgen05 attention kernels are launched with programmatic stream serialization: their CTAs are
 * set up while the kernel before them in the stream finishes, and they wait for that kernel before
 * they read or write anything, except as the flag above allows.  This flag makes the launch an
 * ordinary one (for comparison; results do not depend on it). */
#define SPECROLL_ATTN_NO_PDL 8
#define SPECROLL_ATTN_ALL_FLAGS \
    (SPECROLL_ATTN_LEGACY_MMA | SPECROLL_ATTN_REUSE_PLAN | SPECROLL_ATTN_CACHE_SETTLED | SPECROLL_ATTN_NO_PDL)

size_t specroll_tree_attn_workspace_bytes(const specroll_attn_desc *desc,
                                          const int32_t *kv_indptr_host);

/* Number of kernels one specroll_tree_attn call with this descriptor and these lengths enqueues
 * (plan kernel unless the plan is reused, attention kernel, merge kernel when a sequence is cut into
 * many chunks); -1 for an invalid descriptor.  (Housekeeping for reports; the paper has no counterpart.) */
int specroll_tree_attn_launches(const specroll_attn_desc *desc, const int32_t *kv_indptr_host);

int specroll_tree_attn(const specroll_attn_desc *desc, const void *Q, const void *Kc,
                       const void *Vc, const int32_t *kv_indptr_dev,
                       const int32_t *kv_indptr_host, const void *Kt, const void *Vt,
                       const int32_t *parent_host, void *O, float *lse, void *workspace,
                       size_t workspace_bytes, void *cuda_stream);

/* ------------------------------------------------------------------------------------------
 * The same attention over a paged cache, and the two operations that turn one speculative step
 * into the next (the paper lists "accepted-path KV extraction" among the contents of generation
 * time, Sec. on the experimental protocol, and gives no formula; the layout below is this
 * library's).
 *
 * A layer's cache is a pool Kp,Vp[n_pages, SPECROLL_PAGE_TOKENS, Hkv, D] bf16.  Sequence b owns the
 * slots page_indptr[b] .. page_indptr[b+1]-1 of page_table (i32, device); slot i names the pool
 * page that holds its tokens [128 i, 128 i + 128).  kv_len[b] tokens are valid (device and host
 * copies with the same values); a sequence may own more pages than it fills.  Rows of a sequence's last
 * page beyond kv_len[b] are read and multiplied by a zero weight: they must hold finite values (any
 * finite bit pattern; a pool that was zero-filled once, or only ever written by the commit below, does).
 *
 * specroll_tree_attn_paged computes exactly what specroll_tree_attn computes on the cache that the
 * table describes.  It needs the tcgen05 kernel: Hq/Hkv <= 128 and B <= 4096, no
 * SPECROLL_ATTN_LEGACY_MMA (else SPECROLL_ELIMIT).  SPECROLL_ATTN_REUSE_PLAN: same lengths and same
 * page_indptr as the call that built the plan.  Page numbers outside [0, n_pages) read as zeros.
 */
#define SPECROLL_PAGE_TOKENS 128

size_t specroll_tree_attn_paged_workspace_bytes(const specroll_attn_desc *desc,
                                                const int32_t *kv_len_host);

int specroll_tree_attn_paged(const specroll_attn_desc *desc, const void *Q, const void *Kp,
                             const void *Vp, int64_t n_pages, const int32_t *page_table_dev,
                             const int32_t *page_indptr_dev, const int32_t *kv_len_dev,
                             const int32_t *kv_len_host, const void *Kt, const void *Vt,
                             const int32_t *parent_host, void *O, float *lse, void *workspace,
                             size_t workspace_bytes, void *cuda_stream);

/* Appends the committed path of every sequence to one layer's paged cache: the tree rows
 * Kt,Vt[b, path_node[b,i], :, :] for i = 0 .. n_acc[b] (the anchor and the accepted nodes, as
 * specroll_verify wrote them) go to cache positions kv_len[b] + i.  The step's last token
 * (out_tok[b, n_acc[b]]) has no key yet: it is the next step's anchor.
 * kv_len_out[B] (device, nullable, may be kv_len itself) receives kv_len[b] + n_acc[b] + 1; pass it
 * with the last layer only.  A token that does not fit the sequence's own pages is not written and
 * sets *status (device word, nullable) to SPECROLL_ELIMIT; the length is advanced regardless, so
 * the caller must check the word before relying on the cache.  All pointers device; nothing is
 * allocated. */
int specroll_commit_path(int32_t B, int32_t N, int32_t K, int32_t Hkv, int32_t D, const void *Kt,
                         const void *Vt, const int32_t *path_node, const int32_t *n_acc, void *Kp,
                         void *Vp, int64_t n_pages, const int32_t *page_table,
                         const int32_t *page_indptr, const int32_t *kv_len, int32_t *kv_len_out,
                         int32_t *status, void *cuda_stream);

/* The same for all layers of a model in one launch per 64 layers: Kt, Vt, Kp, Vp are HOST arrays of
 * n_layers device pointers (read during the call, not retained); every layer shares the page table,
 * the lengths and n_pages.  kv_len_out is written once, after the last layer's copies. */
int specroll_commit_path_layers(int32_t B, int32_t N, int32_t K, int32_t Hkv, int32_t D,
                                int32_t n_layers, const void *const *Kt, const void *const *Vt,
                                const int32_t *path_node, const int32_t *n_acc, void *const *Kp,
                                void *const *Vp, int64_t n_pages, const int32_t *page_table,
                                const int32_t *page_indptr, const int32_t *kv_len,
                                int32_t *kv_len_out, int32_t *status, void *cuda_stream);

/* Next step's input state: h_next[b,:] = hidden[b, term_node[b], :], the target's final hidden
 * state at the node whose distribution (or residual) produced the step's last token.
 * hidden[B,N,d] and h_next[B,d] bf16, d % 8 == 0, term_node[B] i32 as written by specroll_verify. */
int specroll_gather_hidden(int32_t B, int32_t N, int32_t d, const void *hidden,
                           const int32_t *term_node, void *h_next, void *cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Verifier-derived feedback of matured proposals and the trajectory memory update (Sec. 3.3 Eq.
 * "acceptance-gap-decomposition"; Sec. 3.4 Eq. "support", "distdir", "covdir", "unified-feedback",
 * "ema").  It produces the memory m that specroll_propose consumes.  Per record r (one matured
 * proposal node), with p = softmax(logits[rec_row[r]] / T) and q = softmax(cand_logit[r] / T) on the
 * candidates C = cand_id[r, :] (sorted by logit, as specroll_propose writes them):
 *   S = C u Top_kS(p) u {y_star[r]};  p_S, q_S = p, q renormalised on S
 *   r_dist = sum_{v in S} (p_S(v) - q_S(v)) W_v
 *   C* = Top_k(p), O = C* \ C, b* = weakest (last) candidate;  r_cov = sum_{y in O} p_S(y) (W_y - W_b*)
 *   d_dist = p(C) TV(p_C, q_C),  d_cov = p(C*) - p(C)
 *   rbar = r / (RMS(r) + eps);  g = d_dist rbar_dist + d_cov rbar_cov;  e = (d_dist + d_cov) g / (RMS(g) + eps)
 *   m[rec_mem[r], :] <- rho[r] m[rec_mem[r], :] + (1 - rho[r]) e
 * Top sets are ordered by (logit desc, id asc).  k <= k_support <= 64 (the support must cover the target's
 * top-k).  The records of one call must address distinct memory rows.
 *
 * Shapes (device): logits[rows, V] bf16 with row_max, row_sum[rows] fp32 as specroll_verify wrote them;
 * rec_row, rec_mem, y_star[R] i32; cand_id[R,k] i32; cand_logit[R,k] fp32; W[V,d] bf16; rho[R] fp32;
 * m[mem_rows, d] fp32 in/out; d_dist, d_cov, tv[R] fp32 outputs, each nullable.
 * Severity weighting and discarding: the flag below.  Sketches, reliability score and gate: specroll_reflex_sketch
 * and specroll_reflex_gate. */
typedef struct {
    int32_t R, k, k_support, d, V;
    float temperature;
    float eps;     /* RMS stabiliser (> = 0) */
    int32_t flags; /* 0, or SPECROLL_FEEDBACK_SEVERITY */
    float severity_min; /* with SPECROLL_FEEDBACK_SEVERITY: observations with w below it are discarded (paper: 0.03) */
} specroll_feedback_desc;

/* The observation's severity weights the update and small ones are discarded (App. "Implementation details",
 * paragraph "Verifier-derived feedback"):  w = clip(0.3 TV(p_S, q_S) + 0.7 p_out, 0, 1)  with  p_out = 1 - p(C)
 * the target mass outside the candidates;  m <- rho m + (1 - rho) w e  when  w >= severity_min, else the memory
 * row is left as it is.  (How w enters the update is not printed in the paper; weighting the observation is
 * this implementation's reading.) */
#define SPECROLL_FEEDBACK_SEVERITY 1

size_t specroll_reflex_feedback_workspace_bytes(const specroll_feedback_desc *desc);

int specroll_reflex_feedback(const specroll_feedback_desc *desc, const void *logits,
                             const int32_t *rec_row, const float *row_max, const float *row_sum,
                             const int32_t *cand_id, const float *cand_logit, const int32_t *y_star,
                             const void *W, const float *rho, const int32_t *rec_mem, float *m,
                             float *d_dist, float *d_cov, float *tv, void *workspace,
                             size_t workspace_bytes, void *cuda_stream);

/* The same with two more outputs (device, each nullable): severity[R] fp32, the w above (written whether or
 * not the flag is set), and e_out[R, d] fp32, the feedback vector e of every record (also of discarded ones),
 * which specroll_reflex_sketch turns into the record's verifier-feedback sketch. */
int specroll_reflex_feedback_ex(const specroll_feedback_desc *desc, const void *logits,
                                const int32_t *rec_row, const float *row_max, const float *row_sum,
                                const int32_t *cand_id, const float *cand_logit, const int32_t *y_star,
                                const void *W, const float *rho, const int32_t *rec_mem, float *m,
                                float *d_dist, float *d_cov, float *tv, float *severity, float *e_out,
                                void *workspace, size_t workspace_bytes, void *cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Reliability from delayed alignment and the gate of the correction (Sec. 3.4, paragraphs "Reliability from
 * delayed alignment" and "Gated hidden-state correction", Eq. "reliability-score" and the indicator of Eq.
 * "reflex-correction"; App. "Implementation details", paragraph "Reflex configuration").
 *
 * specroll_reflex_sketch: normalised random-projection sketch of R vectors,
 *   sketch[r, :] = Pi x_r / ||Pi x_r||_2   (the zero vector when Pi x_r = 0),  x_r = X[rows[r], :] (rows nullable:
 *   then x_r = X[r, :]).  X[*, d] fp32, Pi[rank, d] fp32 (rank <= 32; the paper uses rank 24 and draws Pi with
 *   seed 29; the matrix is an input here), sketch[R, rank] fp32.  Used at proposal time on the memory rows
 *   (s_j) and at maturity on the feedback vectors (xi_j).
 *
 * specroll_reflex_gate: takes R matured records in order.  A kept record (keep nullable = all kept; else
 * keep[r] != 0, e.g. severity >= severity_min) of slot j = slot[r] contributes its realised alignment
 * a_r = cos(s_r, xi_r) (0 when either sketch is zero) to the slot's count n, mean and sum of squared
 * deviations M2 (Welford's recurrences: the exact online sample moments) and to its feedback count n_fb.
 * Then for every slot j (a trajectory-horizon pair) with horizon h = horizon[j]:
 *   Rel = mean - z_delta sqrt(M2 / (n - 1)) / sqrt(n)      (n >= 2, else -inf)
 *   open = n >= n_align_min[h] && n_fb >= n_fb_min[h] && Rel > 0 && RMS(m[j, :]) > mem_eps
 *   alpha[j] = open ? alpha_lo[h] + (alpha_hi[h] - alpha_lo[h]) min(Rel, 1) : 0
 * alpha is what specroll_propose takes per (sequence, head).  The paper puts the ratio of an eligible score
 * inside [alpha_lo, alpha_hi] without printing the map; linear in the score is this implementation's reading.
 * Shapes (device): s, xi[R, rank] fp32; slot[R] i32 in [0, S); keep[R] u8 nullable; n, n_fb[S] i32 in/out;
 * mean, M2[S] fp32 in/out; m[S, d] fp32; horizon[S] i32 in [0, H); n_align_min, n_fb_min[H] i32; alpha_lo,
 * alpha_hi[H] fp32; outputs a[R] (nullable; NaN for records not kept), rel[S], alpha[S] fp32. */
typedef struct {
    int32_t R, S, d, rank, H;
    float z_delta; /* paper: 0.60 */
    float mem_eps; /* a memory row with RMS at or below this is "negligible" */
    int32_t flags; /* reserved, must be 0 */
} specroll_gate_desc;

int specroll_reflex_sketch(int32_t R, int32_t d, int32_t rank, const float *X, const int32_t *rows,
                           const float *Pi, float *sketch, void *cuda_stream);

int specroll_reflex_gate(const specroll_gate_desc *desc, const float *s, const float *xi,
                         const int32_t *slot, const uint8_t *keep, int32_t *n, float *mean, float *M2,
                         int32_t *n_fb, const float *m, const int32_t *horizon,
                         const int32_t *n_align_min, const int32_t *n_fb_min, const float *alpha_lo,
                         const float *alpha_hi, float *a, float *rel, float *alpha, void *cuda_stream);

/* ------------------------------------------------------------------------------------------
 * The target's vocabulary projection with the verification's row statistics fused in, so that the
 * logits of the tree nodes never reach memory (Sec. 3.2: p_u of every tree prefix from one packed
 * target forward; App. B.2 uses, per node, the softmax normaliser and the probabilities of the node's
 * candidate tokens only).  The paper does not describe this fusion; it computes the same quantities:
 *   l[r, v]        = bf16( H[r, :] . W[v, :] )            (rounded as a storing projection would)
 *   row_max[r]     = max_v l[r, v];   row_sum[r] = sum_v exp((l[r, v] - row_max[r]) / T)
 *   want_logit[r,q] = l[r, want_id[r, q]]                  q < kw <= 8
 * H[R, d] bf16 (rows = (sequence, node) in the order of the logits tensor of specroll_verify), W[V, d]
 * bf16, want_id[R, kw] i32 (tokens in [0, V); nullable when kw == 0), row_max, row_sum[R] fp32,
 * want_logit[R, kw] bf16.  d % 64 == 0, V % 8 == 0.  The workspace is scratch of this call.
 *
 * specroll_target_head_rows is the same product storing its logits[R, V] bf16: the one full row per
 * sequence that the terminal draw reads (H then holds the hidden states of the terminal nodes, e.g. from
 * specroll_gather_hidden).  status: one i32 on the device, SPECROLL_ETIMEOUT if a wait ran out. */
size_t specroll_target_head_stats_workspace_bytes(int32_t R, int32_t d, int32_t V);

int specroll_target_head_stats(int32_t R, int32_t d, int32_t V, float temperature, const void *H,
                               const void *W, const int32_t *want_id, int32_t kw, float *row_max,
                               float *row_sum, void *want_logit, void *workspace,
                               size_t workspace_bytes, void *cuda_stream);

int specroll_target_head_rows(int32_t R, int32_t d, int32_t V, const void *H, const void *W,
                              void *logits, int32_t *status, void *cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Exact target verification (App. B.2 Eq. "nodeaccept" / "noderesidual", Algorithm "Exact
 * node-wise tree verification").
 *
 * p_n = softmax(logits[b,n,:] / T) at every node.  Starting at the root u with residual
 * r = p_u, the children of u are tested in slot order: child c with token y is accepted iff
 * u_acc[b,c] < min(1, r(y) / q(y)), q being the slot's proposal (recomputed from
 * cand_logit exactly as the proposal drew it); on rejection r <- [r - q]_+ / sum[r - q]_+.
 * An accepted child becomes u.  The round ends with one more token drawn with u_fin[b] by
 * inverse CDF in token-id order: from the final residual when every child of u was rejected
 * (fallback), or from p_u when u was accepted and has no children (bonus).
 *
 * Shapes: logits[B,N,V] bf16; tree_tok[B,N] i32; tree_cand[B,N] u8; cand_id[B,K,k] i32;
 * cand_logit[B,K,k] fp32; u_acc[B,N] fp32; u_fin[B] fp32 (uniforms in [0,1)).
 * Outputs: n_acc[B] i32 (accepted proposals); path_node[B,K+1] i32 (node at each depth of the
 * committed path, -1 after); out_tok[B,K+1] i32 (accepted tokens, then the terminal token, -1
 * after); term_node[B]; term_kind[B] (0 fallback, 1 bonus); row_max,row_sum[B,N] fp32
 * (max logit and sum exp((l - max)/T) of every node); min_margin[B] fp32 or NULL (smallest
 * |u - ratio| over the tested slots; +inf if none).
 * Limits: V % 8 == 0, k <= 64, K <= 8, N <= 64.
 * Workspace: scratch of the call, specroll_verify_workspace_bytes(desc) bytes, 256-byte aligned: the residual the
 * walk hands to the terminal draw (12 bytes per candidate slot of a sequence) and, without
 * SPECROLL_VERIFY_LAZY_STATS, 64 bytes per logits row in which the statistics pass leaves the maximum and the sum
 * of each eighth of the row, so that the terminal draw reads only the eighth that holds the drawn token.
 */
typedef struct {
    int32_t B, N, K, k, V;
    float temperature;
    int32_t flags; /* 0, or SPECROLL_VERIFY_LAZY_STATS */
} specroll_verify_desc;

/* Compute the softmax statistics only of the rows the walk visits (at most K + 1 per sequence instead of all N):
 * same walk and same tokens; row_max / row_sum are then written for the visited nodes only and the other entries
 * are left untouched.  (The method evaluates every node's distribution; this reads fewer bytes, for callers that do
 * not need the statistics of the nodes that were never reached.) */
#define SPECROLL_VERIFY_LAZY_STATS 1

size_t specroll_verify_workspace_bytes(const specroll_verify_desc *desc);

int specroll_verify(const specroll_verify_desc *desc, const void *logits,
                    const int32_t *parent_host, const int32_t *tree_tok,
                    const uint8_t *tree_cand, const int32_t *cand_id, const float *cand_logit,
                    const float *u_acc, const float *u_fin, int32_t *n_acc, int32_t *path_node,
                    int32_t *out_tok, int32_t *term_node, int32_t *term_kind, float *row_max,
                    float *row_sum, float *min_margin, void *workspace, size_t workspace_bytes,
                    void *cuda_stream);

/* Verification without the logits tensor (the same algorithm as specroll_verify, which see for the
 * arguments; only where the target's numbers come from differs):
 *   specroll_verify_want_ids     want_id[(b, u), j] = cand_id[b, depth(u), j], the tokens whose target logit the
 *                                walk reads at node u (input of specroll_target_head_stats with kw = k <= 8);
 *   specroll_verify_walk_sparse  the node-wise walk from row_max, row_sum[B*N] and cand_target[B, N, k] bf16 (the
 *                                wanted logits); writes n_acc, path_node, the accepted tokens of out_tok, term_node,
 *                                term_kind, min_margin (nullable) and leaves the residual in the workspace;
 *   specroll_verify_terminal_rows  the step's last token from term_logits[B, V] bf16, the full logits row of
 *                                every sequence's terminal node, with the same workspace.
 * The workspace has specroll_verify_workspace_bytes(desc) bytes; desc.flags must be 0. */
int specroll_verify_want_ids(const specroll_verify_desc *desc, const int32_t *parent_host,
                             const int32_t *cand_id, int32_t *want_id, void *cuda_stream);

int specroll_verify_walk_sparse(const specroll_verify_desc *desc, const void *cand_target,
                                const float *row_max, const float *row_sum, const int32_t *parent_host,
                                const int32_t *tree_tok, const uint8_t *tree_cand, const int32_t *cand_id,
                                const float *cand_logit, const float *u_acc, int32_t *n_acc,
                                int32_t *path_node, int32_t *out_tok, int32_t *term_node,
                                int32_t *term_kind, float *min_margin, void *workspace,
                                size_t workspace_bytes, void *cuda_stream);

int specroll_verify_terminal_rows(const specroll_verify_desc *desc, const void *term_logits,
                                  const float *row_max, const int32_t *n_acc, const int32_t *term_node,
                                  const float *u_fin, int32_t *out_tok, void *workspace,
                                  size_t workspace_bytes, void *cuda_stream);

/* The same verification against nucleus-truncated target distributions (App. "Implementation and
 * Reproducibility Details": rollouts sample at temperature 1.0 and nucleus threshold 0.95).  p_n is
 * replaced by its renormalised restriction to the nucleus: tokens in order of decreasing probability
 * until their mass first reaches top_p, plus every token that ties with the last one taken (the
 * paper does not say how ties are cut; this rule does not depend on the order of equal
 * probabilities).  top_p in (0,1); top_p >= 1 is specroll_verify.  Acceptance, residuals and the
 * terminal draw then use the truncated distributions, so the emitted tokens are exact samples of them.
 * row_max / row_sum are still those of the plain softmax.  Optional outputs (device, nullable):
 * nucleus_thr[B,N] fp32 = logit of the smallest kept token, nucleus_sum[B,N] fp32 = sum of
 * exp((l - row_max)/T) over the kept tokens.  Workspace: specroll_verify_nucleus_workspace_bytes. */
size_t specroll_verify_nucleus_workspace_bytes(const specroll_verify_desc *desc);

int specroll_verify_nucleus(const specroll_verify_desc *desc, float top_p, const void *logits,
                            const int32_t *parent_host, const int32_t *tree_tok,
                            const uint8_t *tree_cand, const int32_t *cand_id,
                            const float *cand_logit, const float *u_acc, const float *u_fin,
                            int32_t *n_acc, int32_t *path_node, int32_t *out_tok,
                            int32_t *term_node, int32_t *term_kind, float *row_max, float *row_sum,
                            float *min_margin, float *nucleus_thr, float *nucleus_sum,
                            void *workspace, size_t workspace_bytes, void *cuda_stream);

/* ------------------------------------------------------------------------------------------
 * Allocation-free variant of specroll_verify.  (The paper has no counterpart: this is a
 * deployment convenience of this library, not a step of the method.)
 *
 * Who needs it: hosts that cannot supply a workspace because they cannot allocate device memory
 * at the point of the call.  Examples are a rollout server that hands the whole device to its
 * KV-cache pool at start-up and then runs with allocation switched off (a cudaMalloc there either
 * fails for lack of memory or stalls every stream while the driver serialises the device), and a
 * plain-C client that only receives device pointers from another component and owns no allocator.
 *
 * Same arguments, outputs and results as specroll_verify, minus `workspace` (where the per-row table of
 * specroll_verify's workspace does not fit the fixed array beside the residual, the terminal draw reads its whole
 * row instead): the scratch is a
 * fixed array inside the library image (about 0.2 MB, present once on every GPU that loads the
 * library, until the process exits).  The call performs no cudaMalloc/cudaFree and calls no
 * allocating routine.
 *
 * Limits: B <= SPECROLL_STATIC_MAX_B and B * k <= SPECROLL_STATIC_MAX_BK; anything larger returns
 * SPECROLL_ELIMIT and enqueues nothing (use specroll_verify with a caller workspace instead).
 *
 * First use on a device: the first call made with a given device current looks up the scratch
 * array's device address (cudaGetSymbolAddress) and remembers it.  Make that first call outside
 * any stream capture.  Later calls on that device do no set-up.
 *
 * Sharing: every call on a device uses the same array and finds the previous call's contents in
 * it.  Nothing in it needs to start at zero (each call overwrites every entry it later reads), but
 * two calls that overlap on the GPU (different streams, or different host threads without ordering)
 * race on it.  Serialise them, or use specroll_verify with separate workspaces.
 */
#define SPECROLL_STATIC_MAX_B 4096
#define SPECROLL_STATIC_MAX_BK 16384

int specroll_verify_static(const specroll_verify_desc *desc, const void *logits,
                           const int32_t *parent_host, const int32_t *tree_tok,
                           const uint8_t *tree_cand, const int32_t *cand_id, const float *cand_logit,
                           const float *u_acc, const float *u_fin, int32_t *n_acc,
                           int32_t *path_node, int32_t *out_tok, int32_t *term_node,
                           int32_t *term_kind, float *row_max, float *row_sum, float *min_margin,
                           void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SPECROLL_H */
