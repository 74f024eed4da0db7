// Diagonal-gated KLA (Appendix B.5, "Extension to diagonal gating"): the decay is a vector over d_k,
//
//     S~ = diag(exp(log_alpha_t)) S_{t-1},   e_t = v_t - S~^T k_t,   beta_t = eta_t / (||k_t||^2 + eps)   (Eq. 3)
//     S_t = S~ + beta_t k_t e_t^T,           o_t = S_t^T q_t
//
// (the Kaczmarz coefficient is unchanged: it depends on the decayed state and the key only).  This kernel evaluates the
// recurrence token by token on CUDA cores, for whole sequences (kla_dg_fwd) and for one new token per sequence with the
// state updated in place (kla_dg_decode_step, the same kernel with one token).  It is the correct-first path of the
// extension: the chunkwise form with elementwise decay products is not built.
//
// One warp owns WC = 8 columns of the state of one (sequence, head); lane l holds rows l, l + 32, ... of those columns
// in registers for the whole sequence (columns never interact: the write is k e^T).  Per token: the decayed state is
// never stored -- a_c = sum_j alpha_j S_jc k_j is reduced over the warp with a reduce-scatter butterfly (9 shuffles for
// the 8 columns instead of 40), the residuals are gathered back (8 shuffles), S_jc <- alpha_j S_jc + beta k_j e_c is one
// FMA on top of the decay, and the read-out is a second reduce-scatter.  The next token's operands are loaded while
// the current one is processed.
#include "common.cuh"

namespace kla {

namespace {

constexpr int WC = 8;          // state columns per warp
constexpr int WARPS = 4;       // warps (column groups) per block

// Sums over the warp of x[0..7], by halving: afterwards every lane holds the complete sum of column (lane >> 2) & 7.
__device__ __forceinline__ float reduce_scatter8(const float (&x)[WC], int lane)
{
    float y[4], z[2], w;
    const bool b4 = lane & 16, b3 = lane & 8, b2 = lane & 4;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const float keep = b4 ? x[4 + i] : x[i], give = b4 ? x[i] : x[4 + i];
        y[i] = keep + __shfl_xor_sync(0xffffffffu, give, 16);
    }
#pragma unroll
    for (int i = 0; i < 2; ++i) {
        const float keep = b3 ? y[2 + i] : y[i], give = b3 ? y[i] : y[2 + i];
        z[i] = keep + __shfl_xor_sync(0xffffffffu, give, 8);
    }
    {
        const float keep = b2 ? z[1] : z[0], give = b2 ? z[0] : z[1];
        w = keep + __shfl_xor_sync(0xffffffffu, give, 4);
    }
    w += __shfl_xor_sync(0xffffffffu, w, 2);
    w += __shfl_xor_sync(0xffffffffu, w, 1);
    return w;
}
__device__ __forceinline__ float warp_sum(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

struct DgParams {
    const void *q, *k, *v;
    const float *log_alpha;     // [n_tok, H, D]
    const float *eta;           // [n_tok, H]
    const float *init_state;    // [n_seq, H, D, D] or null
    void *out;                  // [n_tok, H, D]
    float *final_state;         // [n_seq, H, D, D] or null (may alias init_state: every warp reads its columns first)
    const int32_t *cu_seqlens;  // null: fixed length T
    int32_t T, H, n_seq;
    float eps;
    int32_t coeff_eta, qnorm;
};

template <int D, typename IO, typename OUT>
__global__ void __launch_bounds__(32 * WARPS) kla_dg_scan_kernel(DgParams p)
{
    constexpr int J = D / 32;              // rows per lane
    constexpr int GROUPS = D / WC;         // column groups per head
    const int lane = threadIdx.x & 31;
    const int unit = blockIdx.x * WARPS + (threadIdx.x >> 5);     // (sequence, head, column group)
    const int cg = unit % GROUPS, h = (unit / GROUPS) % p.H, n = unit / (GROUPS * p.H);
    if (n >= p.n_seq) return;
    int tok0, len;
    if (p.cu_seqlens) {
        tok0 = p.cu_seqlens[n];
        len = p.cu_seqlens[n + 1] - tok0;
    } else {
        tok0 = n * p.T;
        len = p.T;
    }
    const int c0 = cg * WC;                 // first column of this warp
    const int myc = (lane >> 2) & 7;        // the column whose sums this lane ends up with
    const size_t sbase = ((size_t)n * p.H + h) * D * D;

    float S[J][WC];
#pragma unroll
    for (int j = 0; j < J; ++j) {
        if (p.init_state) {
            const float4 a = *reinterpret_cast<const float4 *>(p.init_state + sbase + (size_t)(lane + 32 * j) * D + c0);
            const float4 b = *reinterpret_cast<const float4 *>(p.init_state + sbase + (size_t)(lane + 32 * j) * D + c0 + 4);
            S[j][0] = a.x; S[j][1] = a.y; S[j][2] = a.z; S[j][3] = a.w;
            S[j][4] = b.x; S[j][5] = b.y; S[j][6] = b.z; S[j][7] = b.w;
        } else {
#pragma unroll
            for (int c = 0; c < WC; ++c) S[j][c] = 0.f;
        }
    }

    const IO *qp = reinterpret_cast<const IO *>(p.q), *kp = reinterpret_cast<const IO *>(p.k), *vp = reinterpret_cast<const IO *>(p.v);
    OUT *op = reinterpret_cast<OUT *>(p.out);
    // operands of one token: this lane's rows of q, k and of the decay; the value of this lane's column; the gate
    struct Tok { float q[J], k[J], a[J], v, eta; };
    auto load = [&](int t) {
        Tok x;
        const size_t th = (size_t)(tok0 + t) * p.H + h;
#pragma unroll
        for (int j = 0; j < J; ++j) {
            x.q[j] = to_f32(qp[th * D + lane + 32 * j]);
            x.k[j] = to_f32(kp[th * D + lane + 32 * j]);
            x.a[j] = __expf(p.log_alpha[th * D + lane + 32 * j]);
        }
        x.v = to_f32(vp[th * D + c0 + myc]);
        x.eta = p.eta[th];
        return x;
    };
    Tok cur;
    if (len > 0) cur = load(0);
    for (int t = 0; t < len; ++t) {
        Tok nxt = cur;
        if (t + 1 < len) nxt = load(t + 1);
        // ||k||^2 (and ||q||^2 for the normalised read-out)
        float nk = 0.f, nq = 0.f;
#pragma unroll
        for (int j = 0; j < J; ++j) {
            nk += cur.k[j] * cur.k[j];
            nq += cur.q[j] * cur.q[j];
        }
        nk = warp_sum(nk);
        const float beta = p.coeff_eta ? cur.eta : cur.eta / (nk + p.eps);
        // a_c = sum_j alpha_j S_jc k_j
        float part[WC];
#pragma unroll
        for (int c = 0; c < WC; ++c) {
            float s = 0.f;
#pragma unroll
            for (int j = 0; j < J; ++j) s += (cur.a[j] * cur.k[j]) * S[j][c];
            part[c] = s;
        }
        const float e_mine = cur.v - reduce_scatter8(part, lane);   // residual of column myc
        // S_jc <- alpha_j S_jc + beta k_j e_c;  o_c = sum_j S_jc q_j
#pragma unroll
        for (int c = 0; c < WC; ++c) {
            const float e = __shfl_sync(0xffffffffu, e_mine, c << 2);
            float s = 0.f;
#pragma unroll
            for (int j = 0; j < J; ++j) {
                S[j][c] = cur.a[j] * S[j][c] + (beta * cur.k[j]) * e;
                s += S[j][c] * cur.q[j];
            }
            part[c] = s;
        }
        float o = reduce_scatter8(part, lane);
        if (p.qnorm) o *= rsqrtf(warp_sum(nq));
        if ((lane & 3) == 0) op[((size_t)(tok0 + t) * p.H + h) * D + c0 + myc] = from_f32<OUT>(o);
        cur = nxt;
    }
    if (p.final_state) {
#pragma unroll
        for (int j = 0; j < J; ++j) {
            float *d = p.final_state + sbase + (size_t)(lane + 32 * j) * D + c0;
            *reinterpret_cast<float4 *>(d) = make_float4(S[j][0], S[j][1], S[j][2], S[j][3]);
            *reinterpret_cast<float4 *>(d + 4) = make_float4(S[j][4], S[j][5], S[j][6], S[j][7]);
        }
    }
}

template <int D, typename IO>
cudaError_t launch_io(const DgParams &p, int out_dtype, cudaStream_t stream)
{
    const int units = p.n_seq * p.H * (D / WC);
    if (units == 0) return cudaSuccess;
    const int blocks = (units + WARPS - 1) / WARPS;
    if (out_dtype == KLA_BF16)
        kla_dg_scan_kernel<D, IO, __nv_bfloat16><<<blocks, 32 * WARPS, 0, stream>>>(p);
    else
        kla_dg_scan_kernel<D, IO, float><<<blocks, 32 * WARPS, 0, stream>>>(p);
    count_launch(1);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_dg_scan(const void *q, const void *k, const void *v, const float *log_alpha, const float *eta,
                           const float *init_state, void *out, float *final_state, const int32_t *cu_seqlens, int T, int H,
                           int n_seq, int d, float eps, int coeff_eta, int qnorm, int io_dtype, int out_dtype, cudaStream_t stream)
{
    DgParams p;
    p.q = q; p.k = k; p.v = v;
    p.log_alpha = log_alpha; p.eta = eta;
    p.init_state = init_state; p.out = out; p.final_state = final_state;
    p.cu_seqlens = cu_seqlens;
    p.T = T; p.H = H; p.n_seq = n_seq;
    p.eps = eps;
    p.coeff_eta = coeff_eta; p.qnorm = qnorm;
    if (d == 128) return io_dtype == KLA_BF16 ? launch_io<128, __nv_bfloat16>(p, out_dtype, stream) : launch_io<128, float>(p, out_dtype, stream);
    return io_dtype == KLA_BF16 ? launch_io<64, __nv_bfloat16>(p, out_dtype, stream) : launch_io<64, float>(p, out_dtype, stream);
}

}  // namespace kla
