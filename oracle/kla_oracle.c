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

void kla_oracle_set_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}
