/*
 * ARL^2 hybrid attention layer -- CPU float64 oracle.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
 * layer computes, written from the paper's equations.  It shares no code with the
 * CUDA library and must never be reached from the product path: only the tests,
 * the smoke check and the bench's CPU-baseline leg may build or call it.
 *
 * Everything is double precision, plain loops, no blocking, no fusion.  The only
 * parallelism is an OpenMP loop over independent (stream, head, row) units, used
 * when the file is built with -fopenmp for the timed CPU baseline.
 *
 * Layouts (all host pointers, row-major, contiguous):
 *   q, k, v, out   [B, L, H, D]   token-major, the shape of x*W reshaped to heads
 *   g              [B, L, H]      combine-gate logits x*W_g (Eq. 6)
 *   S              [B, H, D, D]   recurrent state, row = key dim, column = value dim
 *   w_phi_*        [H, D, D]      per-head feature map, applied as row-vector * W
 *                                 (index [h][in][out]); NULL = identity
 *   rope_cos/sin   [L, D/2]       rotation tables; NULL = no rotation
 *   a              [B, H]         decay-gate logits, alpha = sigmoid(a)
 *   beta_logit     [B, L, H]      learning-rate logits (delta rules only)
 *
 * Readings of the paper where it is silent (each is an interface choice, listed
 * again in the design notes):
 *   - RoPE rotates adjacent pairs (2m, 2m+1) by the angle whose cos/sin the caller
 *     supplies per token: (x0, x1) -> (x0 c - x1 s, x0 s + x1 c).      [parity unpinned]
 *   - L2Norm(x) = x / sqrt(sum_d x_d^2 + eps), over the head dimension.  [eps: parity unpinned]
 *   - phi is a bias-free linear map per head (a grouped 1x1 convolution).
 *   - softmax scale is 1/sqrt(D) as in Eq. 1 unless the caller passes another.
 *   - gates are the logistic sigmoid of the supplied logits.
 */
#include <math.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

static double sigmoid(double x) { return 1.0 / (1.0 + exp(-x)); }

int arl2_oracle_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* RoPE of one head vector x[D] at token position `pos` (Eq. 2, Eq. 3), in place. */
static void rope(double *x, int D, const double *cos_t, const double *sin_t, int pos)
{
    if (!cos_t || !sin_t) return;
    for (int m = 0; m < D / 2; ++m) {
        double c = cos_t[(size_t)pos * (D / 2) + m];
        double s = sin_t[(size_t)pos * (D / 2) + m];
        double x0 = x[2 * m], x1 = x[2 * m + 1];
        x[2 * m]     = x0 * c - x1 * s;
        x[2 * m + 1] = x0 * s + x1 * c;
    }
}

/* y = x * W_h  (row vector times the head's D x D map); W == NULL is the identity. */
static void phi(const double *x, const double *W, int h, int D, double *y)
{
    if (!W) { memcpy(y, x, sizeof(double) * D); return; }
    const double *Wh = W + (size_t)h * D * D;
    for (int o = 0; o < D; ++o) {
        double acc = 0.0;
        for (int i = 0; i < D; ++i) acc += x[i] * Wh[(size_t)i * D + o];
        y[o] = acc;
    }
}

static void l2norm(double *x, int D, double eps)
{
    double ss = 0.0;
    for (int d = 0; d < D; ++d) ss += x[d] * x[d];
    double r = 1.0 / sqrt(ss + eps);
    for (int d = 0; d < D; ++d) x[d] *= r;
}

/*
 * Feature maps of Eq. 3 for one tensor x [B, L, H, D]:
 *   mode 0: y = L2Norm(RoPE(phi(x)))   (Q' and K')
 *   mode 1: y = phi(x)                 (V')
 */
void arl2_oracle_feature(int B, int H, int L, int D, const double *x, const double *W,
                         const double *rope_cos, const double *rope_sin, double eps,
                         int mode, double *y)
{
    for (int b = 0; b < B; ++b)
        for (int l = 0; l < L; ++l)
            for (int h = 0; h < H; ++h) {
                size_t off = (((size_t)b * L + l) * H + h) * D;
                phi(x + off, W, h, D, y + off);
                if (mode == 0) {
                    rope(y + off, D, rope_cos, rope_sin, l);
                    l2norm(y + off, D, eps);
                }
            }
}

/*
 * One output row of the layer: token i of head h of stream b.
 *   O_intra = softmax_j(<RoPE(Q_i), RoPE(K_j)> * scale) V_j   over all L tokens (Eq. 2)
 *   Q'_i    = L2Norm(RoPE(phi_q(Q_i)))                          (Eq. 3)
 *   O_inter = Q'_i S                                            (Eq. 5 / Eq. 8)
 *   O_i     = O_intra + sigmoid(g_i) * O_inter                  (Eq. 6-7, Algorithm 1)
 * S is read, never written (clean-pass-only update, Sec. 3.3).
 * gate_mode selects the granularity of the combine gate (the paper's layer is headwise; the other
 * two are the variants of its gate ablation): 0 headwise g [B, L, H]; 1 scalar g [B, L], one gate
 * per token shared by all heads; 2 elementwise g [B, L, H, D], one gate per output channel.
 * Sh: the D x D state of this (stream, head).  scratch: at least L + 3*D doubles.
 */
static void step_row(int b, int h, int i, int H, int L, int D, int gate_mode,
                     const double *q, const double *k, const double *v, const double *g,
                     const double *Sh, const double *wq,
                     const double *rope_cos, const double *rope_sin,
                     double scale, double eps, double *o, double *scratch)
{
    double *p = scratch;          /* L  */
    double *qr = p + L;           /* D  */
    double *kr = qr + D;          /* D  */
    double *qf = kr + D;          /* D  */
    size_t qoff = (((size_t)b * L + i) * H + h) * D;

    memcpy(qr, q + qoff, sizeof(double) * D);
    rope(qr, D, rope_cos, rope_sin, i);

    /* scores over the whole block: bidirectional, no mask */
    double mx = -INFINITY;
    for (int j = 0; j < L; ++j) {
        size_t koff = (((size_t)b * L + j) * H + h) * D;
        memcpy(kr, k + koff, sizeof(double) * D);
        rope(kr, D, rope_cos, rope_sin, j);
        double s = 0.0;
        for (int d = 0; d < D; ++d) s += qr[d] * kr[d];
        p[j] = s * scale;
        if (p[j] > mx) mx = p[j];
    }
    double den = 0.0;
    for (int j = 0; j < L; ++j) { p[j] = exp(p[j] - mx); den += p[j]; }

    for (int d = 0; d < D; ++d) o[d] = 0.0;
    for (int j = 0; j < L; ++j) {
        size_t voff = (((size_t)b * L + j) * H + h) * D;
        double w = p[j] / den;
        for (int d = 0; d < D; ++d) o[d] += w * v[voff + d];
    }

    /* inter branch: every token reads the same pre-update state */
    phi(q + qoff, wq, h, D, qf);
    rope(qf, D, rope_cos, rope_sin, i);
    l2norm(qf, D, eps);
    for (int e = 0; e < D; ++e) {
        size_t gi = gate_mode == 1 ? (size_t)b * L + i
                  : gate_mode == 2 ? (((size_t)b * L + i) * H + h) * D + e
                                   : ((size_t)b * L + i) * H + h;
        double gate = sigmoid(g[gi]);
        double acc = 0.0;
        for (int d = 0; d < D; ++d) acc += qf[d] * Sh[(size_t)d * D + e];
        o[e] += gate * acc;
    }
}

/* Full denoise-step output, every (b, h, i). */
void arl2_oracle_step(int B, int H, int L, int D,
                      const double *q, const double *k, const double *v, const double *g,
                      const double *S, const double *wq,
                      const double *rope_cos, const double *rope_sin,
                      double scale, double eps, double *out)
{
    long total = (long)B * H * L;
#pragma omp parallel
    {
        double *scratch = (double *)malloc(sizeof(double) * ((size_t)L + 3 * (size_t)D));
#pragma omp for schedule(dynamic, 16)
        for (long t = 0; t < total; ++t) {
            int i = (int)(t % L);
            int h = (int)((t / L) % H);
            int b = (int)(t / ((long)L * H));
            step_row(b, h, i, H, L, D, 0, q, k, v, g, S + ((size_t)b * H + h) * D * D, wq, rope_cos, rope_sin,
                     scale, eps, out + (((size_t)b * L + i) * H + h) * D, scratch);
        }
        free(scratch);
    }
}

/* The same with the combine gate at another granularity (see step_row): the gate ablation's variants. */
void arl2_oracle_step_gate_mode(int B, int H, int L, int D, int gate_mode,
                                const double *q, const double *k, const double *v, const double *g,
                                const double *S, const double *wq,
                                const double *rope_cos, const double *rope_sin,
                                double scale, double eps, double *out)
{
    long total = (long)B * H * L;
#pragma omp parallel
    {
        double *scratch = (double *)malloc(sizeof(double) * ((size_t)L + 3 * (size_t)D));
#pragma omp for schedule(dynamic, 16)
        for (long t = 0; t < total; ++t) {
            int i = (int)(t % L);
            int h = (int)((t / L) % H);
            int b = (int)(t / ((long)L * H));
            step_row(b, h, i, H, L, D, gate_mode, q, k, v, g, S + ((size_t)b * H + h) * D * D, wq, rope_cos,
                     rope_sin, scale, eps, out + (((size_t)b * L + i) * H + h) * D, scratch);
        }
        free(scratch);
    }
}

/*
 * Sampled denoise-step output: n (b, h, i) triples; out_rows is [n, D].
 * Used where the full L x L work per head is too slow to compare in full.
 */
void arl2_oracle_step_rows(int B, int H, int L, int D,
                           const double *q, const double *k, const double *v, const double *g,
                           const double *S, const double *wq,
                           const double *rope_cos, const double *rope_sin,
                           double scale, double eps,
                           int n, const int *bs, const int *hs, const int *is, double *out_rows)
{
    (void)B;
#pragma omp parallel
    {
        double *scratch = (double *)malloc(sizeof(double) * ((size_t)L + 3 * (size_t)D));
#pragma omp for schedule(dynamic, 4)
        for (int t = 0; t < n; ++t)
            step_row(bs[t], hs[t], is[t], H, L, D, 0, q, k, v, g, S + ((size_t)bs[t] * H + hs[t]) * D * D, wq,
                     rope_cos, rope_sin, scale, eps, out_rows + (size_t)t * D, scratch);
        free(scratch);
    }
}

/*
 * Token-level state access, the comparison mode of Sec. 4.3 ("State access granularity"): instead of
 * one pre-update state for the whole block, token i reads the state advanced by the block's tokens
 * before it (each token sees its own sequentially accumulated state), the gated-linear update with
 * one forget gate per token being applied token by token on a private copy:
 *   S^(0) = S,   O_i = O_intra_i + sigmoid(g_i) Q'_i S^(i),   S^(i+1) = alpha_i S^(i) + K'_i^T V'_i,
 * K' = L2Norm(RoPE(phi_k(K))), V' = phi_v(V) from the pass's own K, V; alpha_i = sigmoid(alpha_logit)
 * or 1 when alpha_logit is NULL.  Token 0 reads S itself.  The intra-block softmax is unchanged
 * (bidirectional over the block) and the caller's S is not written.
 */
void arl2_oracle_step_token_level(int B, int H, int L, int D,
                                  const double *q, const double *k, const double *v, const double *g,
                                  const double *alpha_logit, const double *S,
                                  const double *wq, const double *wk, const double *wv,
                                  const double *rope_cos, const double *rope_sin,
                                  double scale, double eps, double *out)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int bh = 0; bh < B * H; ++bh) {
        int b = bh / H, h = bh % H;
        double *scratch = (double *)malloc(sizeof(double) * ((size_t)L + 3 * (size_t)D));
        double *Sloc = (double *)malloc(sizeof(double) * D * D);
        double *kf = (double *)malloc(sizeof(double) * D);
        double *vf = (double *)malloc(sizeof(double) * D);
        memcpy(Sloc, S + (size_t)bh * D * D, sizeof(double) * D * D);
        for (int i = 0; i < L; ++i) {
            size_t off = (((size_t)b * L + i) * H + h) * D;
            /* the row of the layer against the state as this token sees it */
            step_row(b, h, i, H, L, D, 0, q, k, v, g, Sloc, wq, rope_cos, rope_sin, scale, eps,
                     out + off, scratch);
            /* then the token's own write */
            phi(k + off, wk, h, D, kf);
            rope(kf, D, rope_cos, rope_sin, i);
            l2norm(kf, D, eps);
            phi(v + off, wv, h, D, vf);
            double alpha = alpha_logit ? sigmoid(alpha_logit[((size_t)b * L + i) * H + h]) : 1.0;
            for (int d = 0; d < D; ++d)
                for (int e = 0; e < D; ++e)
                    Sloc[(size_t)d * D + e] = alpha * Sloc[(size_t)d * D + e] + kf[d] * vf[e];
        }
        free(vf); free(kf); free(Sloc); free(scratch);
    }
}

/*
 * Eq. 1: the teacher's softmax attention of L queries over a key/value cache of Lk tokens,
 * every cached token visible to every query (the cache holds the blocks so far and the current
 * one).  q, out: [B, L, H, D]; k, v: [B, Lk, H, D].  No rotation, no state.
 *   out_i = sum_j softmax_j(<q_i, k_j> scale) v_j
 */
void arl2_oracle_attend_cache(int B, int H, int L, int Lk, int D,
                              const double *q, const double *k, const double *v,
                              double scale, double *out)
{
#pragma omp parallel
    {
        double *w = (double *)malloc(sizeof(double) * (size_t)Lk);
#pragma omp for collapse(2) schedule(dynamic, 8)
        for (int bh = 0; bh < B * H; ++bh)
            for (int i = 0; i < L; ++i) {
                int b = bh / H, h = bh % H;
                const double *qi = q + (((size_t)b * L + i) * H + h) * D;
                double mx = -INFINITY;
                for (int j = 0; j < Lk; ++j) {
                    const double *kj = k + (((size_t)b * Lk + j) * H + h) * D;
                    double sc = 0.0;
                    for (int d = 0; d < D; ++d) sc += qi[d] * kj[d];
                    w[j] = sc * scale;
                    if (w[j] > mx) mx = w[j];
                }
                double sum = 0.0;
                for (int j = 0; j < Lk; ++j) { w[j] = exp(w[j] - mx); sum += w[j]; }
                double *o = out + (((size_t)b * L + i) * H + h) * D;
                for (int e = 0; e < D; ++e) o[e] = 0.0;
                for (int j = 0; j < Lk; ++j) {
                    const double *vj = v + (((size_t)b * Lk + j) * H + h) * D;
                    double pj = w[j] / sum;
                    for (int e = 0; e < D; ++e) o[e] += pj * vj[e];
                }
            }
        free(w);
    }
}

/*
 * State commit for one (b, h), run once per block from the clean pass's K, V
 * (Algorithm 1, clean-pass branch).  K' = L2Norm(RoPE(phi_k(K))), V' = phi_v(V).
 *
 *   rule 0  gated linear:  S <- alpha S + sum_j K'_j^T V'_j
 *           (Eq. 4 with the correction term dropped and beta = 1; one decay per
 *            head per block)
 *   rule 1  Eq. 4 as printed, frame level:
 *           S <- alpha S + K'^T diag(beta) (V' - K' S_old),  beta_j = sigmoid(beta_logit)
 *   rule 2  Eq. 4 applied token by token in order j = 0..L-1, the decay alpha
 *           applied once before the first token:
 *           S <- alpha S;  for j: S <- S + beta_j K'_j^T (V'_j - K'_j S)
 */
static void commit_head(int b, int h, int H, int L, int D,
                        const double *kc, const double *vc, double alpha,
                        const double *beta_logit, const double *wk, const double *wv,
                        const double *rope_cos, const double *rope_sin, double eps,
                        int rule, double *S)
{
    double *Sh = S + ((size_t)b * H + h) * D * D;
    double *kf = (double *)malloc(sizeof(double) * D);
    double *vf = (double *)malloc(sizeof(double) * D);
    double *pred = (double *)malloc(sizeof(double) * D);
    double *dS = (double *)calloc((size_t)D * D, sizeof(double));
    double *Sold = NULL;
    if (rule == 1) {
        Sold = (double *)malloc(sizeof(double) * D * D);
        memcpy(Sold, Sh, sizeof(double) * D * D);
    }
    if (rule == 2)
        for (size_t t = 0; t < (size_t)D * D; ++t) Sh[t] *= alpha;

    for (int j = 0; j < L; ++j) {
        size_t off = (((size_t)b * L + j) * H + h) * D;
        phi(kc + off, wk, h, D, kf);
        rope(kf, D, rope_cos, rope_sin, j);
        l2norm(kf, D, eps);
        phi(vc + off, wv, h, D, vf);
        double beta = 1.0;
        if (rule != 0 && beta_logit) beta = sigmoid(beta_logit[((size_t)b * L + j) * H + h]);
        if (rule == 0) {
            for (int d = 0; d < D; ++d)
                for (int e = 0; e < D; ++e) dS[(size_t)d * D + e] += kf[d] * vf[e];
        } else {
            const double *Sref = (rule == 1) ? Sold : Sh;
            for (int e = 0; e < D; ++e) {
                double acc = 0.0;
                for (int d = 0; d < D; ++d) acc += kf[d] * Sref[(size_t)d * D + e];
                pred[e] = acc;
            }
            double *dst = (rule == 1) ? dS : Sh;
            for (int d = 0; d < D; ++d)
                for (int e = 0; e < D; ++e)
                    dst[(size_t)d * D + e] += beta * kf[d] * (vf[e] - pred[e]);
        }
    }
    if (rule == 0 || rule == 1)
        for (size_t t = 0; t < (size_t)D * D; ++t) Sh[t] = alpha * Sh[t] + dS[t];

    free(Sold); free(dS); free(pred); free(vf); free(kf);
}

/* heads: optional list of n_heads (b, h) pairs to commit; NULL = all of them. */
void arl2_oracle_commit(int B, int H, int L, int D,
                        const double *kc, const double *vc, const double *a,
                        const double *beta_logit, const double *wk, const double *wv,
                        const double *rope_cos, const double *rope_sin, double eps,
                        int rule, int n_heads, const int *bs, const int *hs, double *S)
{
    int total = bs ? n_heads : B * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (int t = 0; t < total; ++t) {
        int b = bs ? bs[t] : t / H;
        int h = bs ? hs[t] : t % H;
        double alpha = sigmoid(a[(size_t)b * H + h]);
        commit_head(b, h, H, L, D, kc, vc, alpha, beta_logit, wk, wv, rope_cos, rope_sin, eps,
                    rule, S);
    }
}

/*
 * The clean pass of one block (Algorithm 1, clean-pass branch; Sec. 3.3): the layer's output for
 * the clean latent's Q, K, V, read against the state as it stands (Eq. 8: every token queries the
 * same PRE-update state), and only then the gated-linear commit of that block from the same K, V:
 *   out = step(q, kc, vc, g; S),   S <- sigmoid(a) S + sum_j K'_j^T V'_j.
 */
void arl2_oracle_clean_pass(int B, int H, int L, int D,
                            const double *q, const double *kc, const double *vc, const double *g,
                            const double *a, const double *wq, const double *wk, const double *wv,
                            const double *rope_cos, const double *rope_sin, double scale, double eps,
                            double *S, double *out)
{
    arl2_oracle_step(B, H, L, D, q, kc, vc, g, S, wq, rope_cos, rope_sin, scale, eps, out);
    arl2_oracle_commit(B, H, L, D, kc, vc, a, NULL, wk, wv, rope_cos, rope_sin, eps, 0, 0, NULL, NULL, S);
}

/*
 * Eq. 4 applied token by token with per-token gates (the sentence after Eq. 4: the update
 * runs sequentially over the L tokens of the frame, with gates alpha^(j), beta^(j)):
 *   for j = 0..L-1:   S <- alpha_j S + beta_j K'_j^T (V'_j - K'_j S)
 * where the S on the right is the state before token j (both uses), alpha_j =
 * sigmoid(alpha_logit[b,j,h]), beta_j = sigmoid(beta_logit[b,j,h]).  Eq. 4 is taken as
 * printed: the prediction K'_j S uses the undecayed previous state.  With `decayed` non-zero the
 * other reading is taken instead, the one of the Gated DeltaNet the paper builds on: the token's
 * prediction is made against the state after its forget gate,
 *   S <- alpha_j S + beta_j K'_j^T (V'_j - K'_j (alpha_j S)).
 *   alpha_logit, beta_logit  [B, L, H]; NULL = gate fixed at 1.
 */
static void commit_head_tokens(int b, int h, int H, int L, int D,
                               const double *kc, const double *vc,
                               const double *alpha_logit, const double *beta_logit,
                               const double *wk, const double *wv,
                               const double *rope_cos, const double *rope_sin, double eps,
                               int decayed, double *S)
{
    double *Sh = S + ((size_t)b * H + h) * D * D;
    double *kf = (double *)malloc(sizeof(double) * D);
    double *vf = (double *)malloc(sizeof(double) * D);
    double *err = (double *)malloc(sizeof(double) * D);
    for (int j = 0; j < L; ++j) {
        size_t off = (((size_t)b * L + j) * H + h) * D;
        size_t gi = ((size_t)b * L + j) * H + h;
        phi(kc + off, wk, h, D, kf);
        rope(kf, D, rope_cos, rope_sin, j);
        l2norm(kf, D, eps);
        phi(vc + off, wv, h, D, vf);
        double alpha = alpha_logit ? sigmoid(alpha_logit[gi]) : 1.0;
        double beta = beta_logit ? sigmoid(beta_logit[gi]) : 1.0;
        for (int e = 0; e < D; ++e) {   /* V'_j - K'_j S, with the state before this token */
            double acc = 0.0;
            for (int d = 0; d < D; ++d) acc += kf[d] * Sh[(size_t)d * D + e];
            err[e] = vf[e] - (decayed ? alpha * acc : acc);
        }
        for (int d = 0; d < D; ++d)
            for (int e = 0; e < D; ++e)
                Sh[(size_t)d * D + e] = alpha * Sh[(size_t)d * D + e] + beta * kf[d] * err[e];
    }
    free(err); free(vf); free(kf);
}

/* heads: optional list of n_heads (b, h) pairs to commit; NULL = all of them. */
void arl2_oracle_commit_tokens(int B, int H, int L, int D,
                               const double *kc, const double *vc,
                               const double *alpha_logit, const double *beta_logit,
                               const double *wk, const double *wv,
                               const double *rope_cos, const double *rope_sin, double eps,
                               int n_heads, const int *bs, const int *hs, int decayed, double *S)
{
    int total = bs ? n_heads : B * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (int t = 0; t < total; ++t) {
        int b = bs ? bs[t] : t / H;
        int h = bs ? hs[t] : t % H;
        commit_head_tokens(b, h, H, L, D, kc, vc, alpha_logit, beta_logit, wk, wv, rope_cos,
                           rope_sin, eps, decayed, S);
    }
}

/*
 * The gated-linear update (Eq. 4 without the correction term) with the per-token forget gates
 * the paper states, token by token:  for j = 0..L-1:  S <- alpha_j S + K'_j^T V'_j,
 * alpha_j = sigmoid(alpha_logit[b,j,h]).
 */
void arl2_oracle_commit_decay_tokens(int B, int H, int L, int D,
                                     const double *kc, const double *vc, const double *alpha_logit,
                                     const double *wk, const double *wv,
                                     const double *rope_cos, const double *rope_sin, double eps,
                                     int n_heads, const int *bs, const int *hs, double *S)
{
    int total = bs ? n_heads : B * H;
#pragma omp parallel for schedule(dynamic, 1)
    for (int t = 0; t < total; ++t) {
        int b = bs ? bs[t] : t / H;
        int h = bs ? hs[t] : t % H;
        double *Sh = S + ((size_t)b * H + h) * D * D;
        double *kf = (double *)malloc(sizeof(double) * D);
        double *vf = (double *)malloc(sizeof(double) * D);
        for (int j = 0; j < L; ++j) {
            size_t off = (((size_t)b * L + j) * H + h) * D;
            phi(kc + off, wk, h, D, kf);
            rope(kf, D, rope_cos, rope_sin, j);
            l2norm(kf, D, eps);
            phi(vc + off, wv, h, D, vf);
            double alpha = sigmoid(alpha_logit[((size_t)b * L + j) * H + h]);
            for (int d = 0; d < D; ++d)
                for (int e = 0; e < D; ++e)
                    Sh[(size_t)d * D + e] = alpha * Sh[(size_t)d * D + e] + kf[d] * vf[e];
        }
        free(vf); free(kf);
    }
}

/*
 * The projections around the core (Sec. 3.1: Q = x W_q, K = x W_k, V = x W_v; Eq. 6-7: the gate logits
 * x W_g and the output projection y = O W_o).  x, o, y: [rows, d] with rows = B * L and d = H * D, so that
 * Q, K, V and O are the [B, L, H, D] tensors of the core; weights are (in, out), row-major; g: [rows, H].
 */
static void matmul_rows(long rows, int K, int N, const double *x, const double *w, double *y)
{
#pragma omp parallel for schedule(static)
    for (long r = 0; r < rows; ++r)
        for (int n = 0; n < N; ++n) {
            double acc = 0.0;
            for (int kk = 0; kk < K; ++kk) acc += x[(size_t)r * K + kk] * w[(size_t)kk * N + n];
            y[(size_t)r * N + n] = acc;
        }
}

void arl2_oracle_project_in(long rows, int d, int H, const double *x,
                            const double *w_q, const double *w_k, const double *w_v, const double *w_g,
                            double *q, double *k, double *v, double *g)
{
    matmul_rows(rows, d, d, x, w_q, q);
    matmul_rows(rows, d, d, x, w_k, k);
    matmul_rows(rows, d, d, x, w_v, v);
    matmul_rows(rows, d, H, x, w_g, g);
}

void arl2_oracle_project_out(long rows, int d, const double *o, const double *w_o, double *y)
{
    matmul_rows(rows, d, d, o, w_o, y);
}

/* S <- 0 for stream `stream` (or all streams when stream < 0): Algorithm 1, first line. */
void arl2_oracle_reset(int B, int H, int D, int stream, double *S)
{
    size_t per = (size_t)H * D * D;
    if (stream < 0) memset(S, 0, sizeof(double) * per * B);
    else memset(S + per * stream, 0, sizeof(double) * per);
}
