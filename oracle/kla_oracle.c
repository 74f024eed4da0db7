/*
 * fp64 CPU oracle for Kaczmarz Linear Attention (KLA).
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing on the product path may call this file; it exists so that
 * the CUDA kernels can be compared against an independent, obviously-correct implementation.
 * It shares no code with the CUDA path.
 *
 * What it computes: the token-by-token recurrence of Algorithm 1 (left panel, "Tokenwise update")
 * with the Kaczmarz coefficient of Eq. (3), applied to every (sequence, head) independently:
 *
 *     S~   = alpha_t * S_{t-1}                alpha_t = exp(log_alpha_t)      (Alg. 1 left: decay)
 *     e_t  = v_t - S~^T k_t                                                    (residual)
 *     beta = eta_t / (||k_t||^2 + eps)                                         (coefficient, Eq. 3)
 *     S_t  = S~ + beta * k_t e_t^T                                             (rank-one write)
 *     o_t  = S_t^T q_t                                                         (read-out, see below)
 *
 * The state S is d_k x d_v (Section 2), stored row-major with d_v contiguous.
 * Readings taken where the paper is ambiguous:
 *   - the read-out is NOT divided by ||q_t||: Algorithm 1 right, Eq. (8) and Appendix B use the
 *     un-normalised o_i = R_i q_i; a caller who wants the normalised read-out passes q/||q||;
 *   - no 1/sqrt(d_k) scale;
 *   - the stabiliser enters as ||k||^2 + eps (Eq. 3), not (||k|| + eps)^2;
 *   - eps = 0 together with k_t = 0 gives the IEEE result (0/0 = NaN); nothing is clamped.
 *
 * Parallelism: OpenMP over (sequence, head) pairs only; they are independent, so the arithmetic
 * order inside one pair is exactly the loop below.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

/* One token of one head; S is updated in place, o receives d_v values. */
/* The two layer-edge variants the paper names, selected per call (0 = the default above):
 *   coeff_eta  beta_t = eta_t, the gated-delta-rule baseline coefficient without the key-norm division
 *              (Section 2; the comparison model of Section 5);
 *   qnorm      o_t = S_t^T q_t / ||q_t||, the read-out exactly as Algorithm 1 (left) prints it. */
static int g_coeff_eta = 0, g_qnorm = 0;
void kla_oracle_set_variant(int coeff_eta, int qnorm)
{
    g_coeff_eta = coeff_eta;
    g_qnorm = qnorm;
}

static void kla_token_update(double *S, int d_k, int d_v, const double *q, const double *k,
                             const double *v, double log_alpha, double eta, double eps,
                             double *e /* scratch d_v */, double *o)
{
    const double alpha = exp(log_alpha);
    /* decay */
    for (int i = 0; i < d_k; ++i)
        for (int j = 0; j < d_v; ++j) S[(size_t)i * d_v + j] *= alpha;
    /* residual e = v - S~^T k */
    for (int j = 0; j < d_v; ++j) e[j] = v[j];
    for (int i = 0; i < d_k; ++i)
        for (int j = 0; j < d_v; ++j) e[j] -= S[(size_t)i * d_v + j] * k[i];
    /* Kaczmarz coefficient, Eq. 3 */
    double nk = 0.0;
    for (int i = 0; i < d_k; ++i) nk += k[i] * k[i];
    const double beta = g_coeff_eta ? eta : eta / (nk + eps);
    /* rank-one write */
    for (int i = 0; i < d_k; ++i) {
        const double bk = beta * k[i];
        for (int j = 0; j < d_v; ++j) S[(size_t)i * d_v + j] += bk * e[j];
    }
    /* read-out from the post-write state */
    for (int j = 0; j < d_v; ++j) o[j] = 0.0;
    for (int i = 0; i < d_k; ++i)
        for (int j = 0; j < d_v; ++j) o[j] += S[(size_t)i * d_v + j] * q[i];
    if (g_qnorm) {
        double nq = 0.0;
        for (int i = 0; i < d_k; ++i) nq += q[i] * q[i];
        const double inv = 1.0 / sqrt(nq);
        for (int j = 0; j < d_v; ++j) o[j] *= inv;
    }
}

/*
 * Packed (variable-length) forward.  Tokens of all sequences are concatenated; sequence n owns
 * tokens cu_seqlens[n] .. cu_seqlens[n+1]-1.
 *   q, k        [n_tok, H, d_k]      v, out  [n_tok, H, d_v]      log_alpha, eta  [n_tok, H]
 *   init_state  [n_seq, H, d_k, d_v] or NULL (zeros)   final_state same shape or NULL (skipped)
 * A sequence of length 0 leaves final_state equal to its initial state.
 * Returns the number of OpenMP threads used.
 */
int kla_oracle_forward(int n_seq, const int64_t *cu_seqlens, int H, int d_k, int d_v,
                       const double *q, const double *k, const double *v,
                       const double *log_alpha, const double *eta, double eps,
                       const double *init_state, double *out, double *final_state)
{
    int threads = 1;
#ifdef _OPENMP
    threads = omp_get_max_threads();
#endif
    const size_t ss = (size_t)d_k * d_v;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int n = 0; n < n_seq; ++n) {
        for (int h = 0; h < H; ++h) {
            double *S = (double *)malloc(ss * sizeof(double));
            double *e = (double *)malloc((size_t)d_v * sizeof(double));
            if (init_state)
                memcpy(S, init_state + ((size_t)n * H + h) * ss, ss * sizeof(double));
            else
                memset(S, 0, ss * sizeof(double));
            for (int64_t t = cu_seqlens[n]; t < cu_seqlens[n + 1]; ++t) {
                const size_t th = (size_t)t * H + h;
                kla_token_update(S, d_k, d_v, q + th * d_k, k + th * d_k, v + th * d_v,
                                 log_alpha[th], eta[th], eps, e, out + th * d_v);
            }
            if (final_state)
                memcpy(final_state + ((size_t)n * H + h) * ss, S, ss * sizeof(double));
            free(S);
            free(e);
        }
    }
    return threads;
}

/*
 * One decode step for a batch: the loop body above applied once per (b, h), state in place.
 *   q, k [B, H, d_k]   v, out [B, H, d_v]   log_alpha, eta [B, H]   state [B, H, d_k, d_v]
 */
int kla_oracle_decode_step(int B, int H, int d_k, int d_v, const double *q, const double *k,
                           const double *v, const double *log_alpha, const double *eta,
                           double eps, double *state, double *out)
{
    int threads = 1;
#ifdef _OPENMP
    threads = omp_get_max_threads();
#endif
    const size_t ss = (size_t)d_k * d_v;
#pragma omp parallel for schedule(static)
    for (int bh = 0; bh < B * H; ++bh) {
        double *e = (double *)malloc((size_t)d_v * sizeof(double));
        kla_token_update(state + (size_t)bh * ss, d_k, d_v, q + (size_t)bh * d_k,
                         k + (size_t)bh * d_k, v + (size_t)bh * d_v, log_alpha[bh], eta[bh], eps,
                         e, out + (size_t)bh * d_v);
        free(e);
    }
    return threads;
}

/*
 * Diagonal-gated KLA (Appendix B.5, "Extension to diagonal gating"; the decay-agnostic remark of the proofs): the decay
 * operator is D_t = diag(alpha_t) with alpha_t a vector over d_k, so the decay scales the ROWS of S,
 *
 *     S~ = diag(exp(log_alpha_t)) S_{t-1},
 *
 * and everything after it (residual, coefficient of Eq. 3, rank-one write, read-out) is the loop body above unchanged:
 * the Kaczmarz coefficient depends on S~ and k_t only, not on how S~ was produced.  Same layouts as kla_oracle_forward
 * except log_alpha [n_tok, H, d_k].
 */
static void kla_token_update_dg(double *S, int d_k, int d_v, const double *q, const double *k, const double *v,
                                const double *log_alpha, double eta, double eps, double *e, double *o)
{
    /* row-wise decay, then the scalar-gated update with alpha = 1 (log_alpha = 0) */
    for (int i = 0; i < d_k; ++i) {
        const double a = exp(log_alpha[i]);
        for (int j = 0; j < d_v; ++j) S[(size_t)i * d_v + j] *= a;
    }
    kla_token_update(S, d_k, d_v, q, k, v, 0.0, eta, eps, e, o);
}

int kla_oracle_forward_dg(int n_seq, const int64_t *cu_seqlens, int H, int d_k, int d_v,
                          const double *q, const double *k, const double *v,
                          const double *log_alpha, const double *eta, double eps,
                          const double *init_state, double *out, double *final_state)
{
    int threads = 1;
#ifdef _OPENMP
    threads = omp_get_max_threads();
#endif
    const size_t ss = (size_t)d_k * d_v;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int n = 0; n < n_seq; ++n) {
        for (int h = 0; h < H; ++h) {
            double *S = (double *)malloc(ss * sizeof(double));
            double *e = (double *)malloc((size_t)d_v * sizeof(double));
            if (init_state)
                memcpy(S, init_state + ((size_t)n * H + h) * ss, ss * sizeof(double));
            else
                memset(S, 0, ss * sizeof(double));
            for (int64_t t = cu_seqlens[n]; t < cu_seqlens[n + 1]; ++t) {
                const size_t th = (size_t)t * H + h;
                kla_token_update_dg(S, d_k, d_v, q + th * d_k, k + th * d_k, v + th * d_v,
                                    log_alpha + th * d_k, eta[th], eps, e, out + th * d_v);
            }
            if (final_state)
                memcpy(final_state + ((size_t)n * H + h) * ss, S, ss * sizeof(double));
            free(S);
            free(e);
        }
    }
    return threads;
}

/*
 * Reverse-mode derivative of the recurrence above (the models of Section 5.1 are trained through it; the paper prints no
 * backward pass, so this is the chain rule applied to the five lines of the loop body, last line first).  For a scalar
 * loss L with dO_t = dL/do_t given for every token and dS_T = dL/dS_T given for the final state:
 *
 *   read-out   o = S_t^T qh  (qh = q, or q / ||q|| with the qnorm variant)
 *                  G  += qh dO^T                 (G holds dL/dS_t)
 *                  dqh = S_t dO ;  dq = dqh, or (dqh - qh (qh . dqh)) / ||q||
 *   write      S_t = S~ + beta k e^T
 *                  dbeta = k^T G e ;  dk = beta G e ;  de = beta G^T k
 *   residual   e = v - S~^T k
 *                  dv = de ;  dk -= S~ de ;  G -= k de^T   (G now holds dL/dS~)
 *   coefficient  beta = eta / n, n = ||k||^2 + eps  (Eq. 3)
 *                  deta = dbeta / n ;  dk += 2 k (-dbeta eta / n^2)        (beta = eta: deta = dbeta)
 *   decay      S~ = exp(log_alpha) S_{t-1}
 *                  dlog_alpha = <G, S~> ;  G <- exp(log_alpha) G            (G now holds dL/dS_{t-1})
 *
 * `Sprev` is S_{t-1}; the forward quantities of the token are recomputed from it.  `work` holds 2 d_k d_v + 2 d_v doubles.
 */
static void kla_token_backward(const double *Sprev, int d_k, int d_v, const double *q, const double *k,
                               const double *v, double log_alpha, double eta, double eps, const double *dout,
                               double *G, double *dq, double *dk, double *dv, double *dlog_alpha, double *deta,
                               double *work)
{
    const size_t ss = (size_t)d_k * d_v;
    double *St = work;          /* S~ = alpha S_{t-1} */
    double *Sn = work + ss;     /* S_t */
    double *e = work + 2 * ss;
    double *de = e + d_v;
    const double alpha = exp(log_alpha);
    /* forward quantities of this token */
    for (size_t x = 0; x < ss; ++x) St[x] = alpha * Sprev[x];
    for (int j = 0; j < d_v; ++j) e[j] = v[j];
    for (int i = 0; i < d_k; ++i)
        for (int j = 0; j < d_v; ++j) e[j] -= St[(size_t)i * d_v + j] * k[i];
    double nk = 0.0;
    for (int i = 0; i < d_k; ++i) nk += k[i] * k[i];
    const double n = nk + eps;
    const double beta = g_coeff_eta ? eta : eta / n;
    for (int i = 0; i < d_k; ++i)
        for (int j = 0; j < d_v; ++j) Sn[(size_t)i * d_v + j] = St[(size_t)i * d_v + j] + beta * k[i] * e[j];
    /* read-out */
    double qnrm = 1.0;
    if (g_qnorm) {
        double nq = 0.0;
        for (int i = 0; i < d_k; ++i) nq += q[i] * q[i];
        qnrm = sqrt(nq);
    }
    double proj = 0.0;   /* qh . dqh */
    for (int i = 0; i < d_k; ++i) {
        const double qh = q[i] / qnrm;
        double s = 0.0;
        for (int j = 0; j < d_v; ++j) {
            G[(size_t)i * d_v + j] += qh * dout[j];
            s += Sn[(size_t)i * d_v + j] * dout[j];
        }
        dq[i] = s;       /* dqh for now */
        proj += qh * s;
    }
    if (g_qnorm)
        for (int i = 0; i < d_k; ++i) dq[i] = (dq[i] - (q[i] / qnrm) * proj) / qnrm;
    /* rank-one write */
    double dbeta = 0.0;
    for (int j = 0; j < d_v; ++j) de[j] = 0.0;
    for (int i = 0; i < d_k; ++i) {
        double ge = 0.0;
        for (int j = 0; j < d_v; ++j) {
            ge += G[(size_t)i * d_v + j] * e[j];
            de[j] += beta * G[(size_t)i * d_v + j] * k[i];
        }
        dbeta += k[i] * ge;
        dk[i] = beta * ge;
    }
    /* residual */
    for (int j = 0; j < d_v; ++j) dv[j] = de[j];
    for (int i = 0; i < d_k; ++i) {
        double s = 0.0;
        for (int j = 0; j < d_v; ++j) {
            s += St[(size_t)i * d_v + j] * de[j];
            G[(size_t)i * d_v + j] -= k[i] * de[j];
        }
        dk[i] -= s;
    }
    /* coefficient, Eq. 3 */
    if (g_coeff_eta) {
        *deta = dbeta;
    } else {
        *deta = dbeta / n;
        const double dn = -dbeta * eta / (n * n);
        for (int i = 0; i < d_k; ++i) dk[i] += 2.0 * k[i] * dn;
    }
    /* decay */
    double dla = 0.0;
    for (size_t x = 0; x < ss; ++x) {
        dla += G[x] * St[x];
        G[x] *= alpha;
    }
    *dlog_alpha = dla;
}

/*
 * Packed backward.  Inputs as kla_oracle_forward, plus dout [n_tok, H, d_v] and dfinal [n_seq, H, d_k, d_v] or NULL
 * (zeros).  Outputs dq, dk [n_tok, H, d_k], dv [n_tok, H, d_v], dlog_alpha, deta [n_tok, H], dinit [n_seq, H, d_k, d_v]
 * or NULL (skipped).  The reverse sweep needs S_{t-1} of every token: the forward sweep keeps the state at the start of
 * every block of 64 tokens, and the states inside one block are recomputed from its start when the sweep reaches it.
 */
#define KLA_ORACLE_BWD_BLOCK 64
int kla_oracle_backward(int n_seq, const int64_t *cu_seqlens, int H, int d_k, int d_v,
                        const double *q, const double *k, const double *v,
                        const double *log_alpha, const double *eta, double eps,
                        const double *init_state, const double *dout, const double *dfinal,
                        double *dq, double *dk, double *dv, double *dlog_alpha, double *deta, double *dinit)
{
    int threads = 1;
#ifdef _OPENMP
    threads = omp_get_max_threads();
#endif
    const size_t ss = (size_t)d_k * d_v;
    const int L = KLA_ORACLE_BWD_BLOCK;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
    for (int n = 0; n < n_seq; ++n) {
        for (int h = 0; h < H; ++h) {
            const int64_t t0 = cu_seqlens[n], len = cu_seqlens[n + 1] - t0;
            const int64_t n_blocks = (len + L - 1) / L;
            double *starts = (double *)malloc((size_t)(n_blocks + 1) * ss * sizeof(double));  /* state at each block start */
            double *inside = (double *)malloc((size_t)(L + 1) * ss * sizeof(double));         /* S_{t-1} of a block's tokens */
            double *G = (double *)malloc(ss * sizeof(double));
            double *work = (double *)malloc((2 * ss + 2 * (size_t)d_v) * sizeof(double));
            double *o = (double *)malloc((size_t)d_v * sizeof(double));
            double *S = inside;   /* running state of the forward sweep */
            if (init_state)
                memcpy(S, init_state + ((size_t)n * H + h) * ss, ss * sizeof(double));
            else
                memset(S, 0, ss * sizeof(double));
            for (int64_t i = 0; i < len; ++i) {
                if (i % L == 0) memcpy(starts + (size_t)(i / L) * ss, S, ss * sizeof(double));
                const size_t th = (size_t)(t0 + i) * H + h;
                kla_token_update(S, d_k, d_v, q + th * d_k, k + th * d_k, v + th * d_v, log_alpha[th], eta[th], eps,
                                 work, o);
            }
            if (dfinal)
                memcpy(G, dfinal + ((size_t)n * H + h) * ss, ss * sizeof(double));
            else
                memset(G, 0, ss * sizeof(double));
            for (int64_t b = n_blocks - 1; b >= 0; --b) {
                const int64_t i0 = b * L, i1 = (i0 + L < len) ? i0 + L : len;
                memcpy(inside, starts + (size_t)b * ss, ss * sizeof(double));
                for (int64_t i = i0; i + 1 < i1; ++i) {   /* inside[j] = state before token i0 + j */
                    double *nxt = inside + (size_t)(i - i0 + 1) * ss;
                    memcpy(nxt, inside + (size_t)(i - i0) * ss, ss * sizeof(double));
                    const size_t th = (size_t)(t0 + i) * H + h;
                    kla_token_update(nxt, d_k, d_v, q + th * d_k, k + th * d_k, v + th * d_v, log_alpha[th], eta[th],
                                     eps, work, o);
                }
                for (int64_t i = i1 - 1; i >= i0; --i) {
                    const size_t th = (size_t)(t0 + i) * H + h;
                    kla_token_backward(inside + (size_t)(i - i0) * ss, d_k, d_v, q + th * d_k, k + th * d_k, v + th * d_v,
                                       log_alpha[th], eta[th], eps, dout + th * d_v, G, dq + th * d_k, dk + th * d_k,
                                       dv + th * d_v, dlog_alpha + th, deta + th, work);
                }
            }
            if (dinit) memcpy(dinit + ((size_t)n * H + h) * ss, G, ss * sizeof(double));
            free(starts); free(inside); free(G); free(work); free(o);
        }
    }
    return threads;
}

void kla_oracle_set_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}
