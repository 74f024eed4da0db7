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
// FMA on top of the decay, and the read-out is a second reduce-scatter.  Operands are requested three tokens ahead and
// prepared one token ahead (see the loop).
#include "common.cuh"
#include "scan_pieces.cuh"

namespace kla {

namespace {

#ifndef DG_WC
#define DG_WC 8   // state columns per warp (4: twice the warps, but every warp prepares every token: 3.4 ms against 3.0 ms)
#endif
constexpr int WARPS = 4;       // warps (column groups) per block

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

template <int D, int WC, typename IO, typename OUT>
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
    const int c0 = cg * WC;                    // first column of this warp
    const int myc = col_of_lane<WC>(lane);     // the column whose sums this lane ends up with
    const size_t sbase = ((size_t)n * p.H + h) * D * D;

    float S[J][WC];
#pragma unroll
    for (int j = 0; j < J; ++j) {
#pragma unroll
        for (int c = 0; c < WC; c += 4) {
            float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
            if (p.init_state) a = *reinterpret_cast<const float4 *>(p.init_state + sbase + (size_t)(lane + 32 * j) * D + c0 + c);
            S[j][c] = a.x; S[j][c + 1] = a.y; S[j][c + 2] = a.z; S[j][c + 3] = a.w;
        }
    }

    const IO *qp = reinterpret_cast<const IO *>(p.q), *kp = reinterpret_cast<const IO *>(p.k), *vp = reinterpret_cast<const IO *>(p.v);
    OUT *op = reinterpret_cast<OUT *>(p.out);
    // Three-stage software pipeline per warp.  Raw operands of token t + 3 are requested from global memory and not touched
    // (any use, even a conversion, would wait for them); the operands of token t + 1 are prepared from raw values requested two
    // iterations earlier -- everything that does not depend on the state: alpha_j, alpha_j k_j, beta k_j (Eq. 3), 1 / ||q||;
    // token t is applied to the state.
    struct Raw { IO q[J], k[J], v; float la[J], eta; };
    struct Tok { float q[J], a[J], ak[J], bk[J], v, qinv; };
    auto request = [&](int t) {
        Raw r;
        const size_t th = (size_t)(tok0 + min(t, len - 1)) * p.H + h;   // (past the end: the last token again, never used)
#pragma unroll
        for (int j = 0; j < J; ++j) {
            r.q[j] = qp[th * D + lane + 32 * j];
            r.k[j] = kp[th * D + lane + 32 * j];
            r.la[j] = p.log_alpha[th * D + lane + 32 * j];
        }
        r.v = vp[th * D + c0 + myc];
        r.eta = p.eta[th];
        return r;
    };
    auto prepare = [&](const Raw &r) {
        Tok x;
        float k[J], nk = 0.f, nq = 0.f;
#pragma unroll
        for (int j = 0; j < J; ++j) {
            x.q[j] = to_f32(r.q[j]);
            k[j] = to_f32(r.k[j]);
            x.a[j] = __expf(r.la[j]);
            nk += k[j] * k[j];
            nq += x.q[j] * x.q[j];
        }
        x.v = to_f32(r.v);
        nk = warp_sum(nk);
        const float beta = p.coeff_eta ? r.eta : r.eta / (nk + p.eps);   // Eq. 3
        x.qinv = p.qnorm ? rsqrtf(warp_sum(nq)) : 1.f;
#pragma unroll
        for (int j = 0; j < J; ++j) {
            x.ak[j] = x.a[j] * k[j];
            x.bk[j] = beta * k[j];
        }
        return x;
    };
    if (len > 0) {
        Raw r1 = request(1), r2 = request(2);
        Tok cur = prepare(request(0));
        for (int t = 0; t < len; ++t) {
            const Raw r3 = request(t + 3);
            const Tok nxt = prepare(r1);
            // a_c = sum_j alpha_j S_jc k_j, residual e_c = v_c - a_c
            float part[WC];
#pragma unroll
            for (int c = 0; c < WC; ++c) {
                float s = 0.f;
#pragma unroll
                for (int j = 0; j < J; ++j) s += cur.ak[j] * S[j][c];
                part[c] = s;
            }
            const float e_mine = cur.v - reduce_scatter<WC>(part, lane);   // residual of column myc
            // S_jc <- alpha_j S_jc + beta k_j e_c;  o_c = sum_j S_jc q_j
#pragma unroll
            for (int c = 0; c < WC; ++c) {
                const float e = __shfl_sync(0xffffffffu, e_mine, lane_of_col<WC>(c));
                float s = 0.f;
#pragma unroll
                for (int j = 0; j < J; ++j) {
                    S[j][c] = cur.a[j] * S[j][c] + cur.bk[j] * e;
                    s += S[j][c] * cur.q[j];
                }
                part[c] = s;
            }
            const float o = reduce_scatter<WC>(part, lane) * cur.qinv;
            if ((lane & (WC == 8 ? 3 : 7)) == 0) op[((size_t)(tok0 + t) * p.H + h) * D + c0 + myc] = from_f32<OUT>(o);
            cur = nxt;
            r1 = r2;
            r2 = r3;
        }
    }
    if (p.final_state) {
#pragma unroll
        for (int j = 0; j < J; ++j)
#pragma unroll
            for (int c = 0; c < WC; c += 4)
                *reinterpret_cast<float4 *>(p.final_state + sbase + (size_t)(lane + 32 * j) * D + c0 + c) =
                    make_float4(S[j][c], S[j][c + 1], S[j][c + 2], S[j][c + 3]);
    }
}

template <int D, typename IO>
cudaError_t launch_io(const DgParams &p, int out_dtype, cudaStream_t stream)
{
    constexpr int WC = DG_WC;   // state columns per warp
    const int units = p.n_seq * p.H * (D / WC);
    if (units == 0) return cudaSuccess;
    const int blocks = (units + WARPS - 1) / WARPS;
    if (out_dtype == KLA_BF16)
        kla_dg_scan_kernel<D, WC, IO, __nv_bfloat16><<<blocks, 32 * WARPS, 0, stream>>>(p);
    else
        kla_dg_scan_kernel<D, WC, IO, float><<<blocks, 32 * WARPS, 0, stream>>>(p);
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
