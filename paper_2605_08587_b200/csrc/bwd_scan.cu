// Reverse-mode derivative of the KLA recurrence (the training pass of Section 5.1; the paper prints no backward, so this
// is the chain rule over the loop body of Algorithm 1 left with the coefficient of Eq. 3), token by token on CUDA cores.
//
// For a scalar loss with dO_t = dL/do_t and dS_T = dL/dS_T given, one token in reverse order, G = dL/dS_t on entry:
//
//     read-out     G += qh dO^T ;  dqh = S_t dO                      (qh = q, or q / ||q|| with its projection for dq)
//     write        dbeta = k^T G e ;  dk = beta G e ;  de = beta G^T k
//     residual     dv = de ;  dk -= S~ de ;  G -= k de^T
//     coefficient  deta = dbeta / n ;  dk += 2 k (-dbeta beta / n)    (n = ||k||^2 + eps; beta = eta: deta = dbeta)
//     decay        dlog_alpha = <G, S~> ;  G <- alpha G               (G = dL/dS_{t-1} on exit)
//
// The step needs S_{t-1}, which only a forward sweep can give.  States are kept every L = 16 tokens on the way forward
// (one state per 16 tokens of workspace); on the way back each block of 16 tokens is first re-run from its stored state
// with the state before every token written to a per-head scratch area (16 states, L2-resident), then walked in reverse.
// Every thread reads back only what it wrote itself, so no fence or barrier guards the stored states.
//
// Work split: columns of S and G never interact, so a block owns 64 columns of one (sequence, head), one warp 8 of them,
// lane l rows l, l + 32, ... (S_{t-1}, G and the prefetched next S_{t-1} in registers).  Sums over rows (S~^T k, G^T k)
// are reduce-scatter butterflies inside the warp; sums over columns (dq, dk, dbeta, dlog_alpha) are per-warp partials
// added up through shared memory once per token.  With d = 128 the two blocks of a head add their halves into
// zero-initialised outputs with one atomic each: two commutative additions, so the result does not depend on their order.
#include "common.cuh"
#include "scan_pieces.cuh"

namespace kla {

namespace {

constexpr int WC = 8;         // state columns per warp
constexpr int WARPS = 8;      // warps per block (64 columns)
constexpr int NT = 32 * WARPS;
constexpr int L = 16;         // tokens between stored states (kla_bwd_workspace_bytes in api.cu uses the same figure)

struct BwdParams {
    const void *q, *k, *v, *dout;
    const float *log_alpha, *eta;      // [n_tok, H]
    const float *init_state, *dfinal;  // [n_seq, H, D, D] or null
    float *dq, *dk, *dv;               // [n_tok, H, D]
    float *dlog_alpha, *deta;          // [n_tok, H]
    float *dinit;                      // [n_seq, H, D, D] or null
    float *stored;                     // states every L tokens: slot (tok0 / L + n + block) * H + h
    float *scratch;                    // L states per (sequence, head)
    const int32_t *cu_seqlens;         // null: fixed length T
    int32_t T, H, n_seq;
    float eps;
    int32_t coeff_eta;
};

template <int D, typename IO, bool QN>
__global__ void __launch_bounds__(NT, 1) kla_bwd_scan_kernel(BwdParams p)
{
    constexpr int J = D / 32;            // rows per lane
    constexpr int SPLIT = D / 64;        // blocks per head
    constexpr int NRED = 2 * D + 2;      // per-token sums over columns: dq, dk, dlog_alpha, deta
    __shared__ float red[2][WARPS][NRED];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int split = blockIdx.x % SPLIT, h = (blockIdx.x / SPLIT) % p.H, n = blockIdx.x / (SPLIT * p.H);
    int tok0, len;
    if (p.cu_seqlens) {
        tok0 = p.cu_seqlens[n];
        len = p.cu_seqlens[n + 1] - tok0;
    } else {
        tok0 = n * p.T;
        len = p.T;
    }
    const int cg = split * WARPS + warp;         // column group within the head
    const int c0 = cg * WC;                      // first column of this warp
    const int myc = col_of_lane<WC>(lane);       // the column whose row sums this lane ends up with
    const size_t sbase = ((size_t)n * p.H + h) * D * D;
    // Stored states use a layout of their own, [column group][j][half][lane] float4, so that every access is 512 contiguous bytes.
    const size_t soff = ((size_t)cg * J * 2) * 128 + lane * 4;
    float *const stored = p.stored + ((size_t)(tok0 / L + n) * p.H + h) * D * D + soff;
    float *const scratch = p.scratch + ((size_t)n * p.H + h) * L * D * D + soff;
    auto put = [&](float *dst, const float (&S)[J][WC]) {
#pragma unroll
        for (int j = 0; j < J; ++j) {
            store4(dst + (j * 2) * 128, make_float4(S[j][0], S[j][1], S[j][2], S[j][3]));
            store4(dst + (j * 2 + 1) * 128, make_float4(S[j][4], S[j][5], S[j][6], S[j][7]));
        }
    };
    auto get = [&](const float *src, float (&S)[J][WC]) {
#pragma unroll
        for (int j = 0; j < J; ++j) {
            const float4 a = load4(src + (j * 2) * 128), b = load4(src + (j * 2 + 1) * 128);
            S[j][0] = a.x; S[j][1] = a.y; S[j][2] = a.z; S[j][3] = a.w;
            S[j][4] = b.x; S[j][5] = b.y; S[j][6] = b.z; S[j][7] = b.w;
        }
    };
    // the caller's states are [row][column]
    auto get_natural = [&](const float *src, float (&S)[J][WC]) {
#pragma unroll
        for (int j = 0; j < J; ++j)
#pragma unroll
            for (int c = 0; c < WC; c += 4) {
                float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
                if (src) a = load4(src + sbase + (size_t)(lane + 32 * j) * D + c0 + c);
                S[j][c] = a.x; S[j][c + 1] = a.y; S[j][c + 2] = a.z; S[j][c + 3] = a.w;
            }
    };

    const IO *qp = reinterpret_cast<const IO *>(p.q), *kp = reinterpret_cast<const IO *>(p.k), *vp = reinterpret_cast<const IO *>(p.v);
    const IO *dop = reinterpret_cast<const IO *>(p.dout);

    // ---- forward steps (no read-out): operands of the next token are requested while this one is applied ----
    struct FRaw { IO k[J], v; float la, eta; };
    auto frequest = [&](int i) {
        FRaw r;
        const size_t th = (size_t)(tok0 + max(min(i, len - 1), 0)) * p.H + h;
#pragma unroll
        for (int j = 0; j < J; ++j) r.k[j] = kp[th * D + lane + 32 * j];
        r.v = vp[th * D + c0 + myc];
        r.la = p.log_alpha[th];
        r.eta = p.eta[th];
        return r;
    };
    auto fstep = [&](float (&S)[J][WC], const FRaw &r) {
        float k[J], nk = 0.f;
#pragma unroll
        for (int j = 0; j < J; ++j) {
            k[j] = to_f32(r.k[j]);
            nk += k[j] * k[j];
        }
        const float alpha = __expf(r.la);
        const float beta = p.coeff_eta ? r.eta : r.eta / (warp_sum(nk) + p.eps);   // Eq. 3
        float part[WC];
#pragma unroll
        for (int c = 0; c < WC; ++c) {
            float s = 0.f;
#pragma unroll
            for (int j = 0; j < J; ++j) s += k[j] * S[j][c];
            part[c] = s;
        }
        const float e_mine = to_f32(r.v) - alpha * reduce_scatter<WC>(part, lane);
#pragma unroll
        for (int c = 0; c < WC; ++c) {
            const float be = beta * __shfl_sync(0xffffffffu, e_mine, lane_of_col<WC>(c));
#pragma unroll
            for (int j = 0; j < J; ++j) S[j][c] = alpha * S[j][c] + k[j] * be;
        }
    };

    float S[J][WC], G[J][WC];
    get_natural(p.init_state, S);
    get_natural(p.dfinal, G);
    const int n_blocks = (len + L - 1) / L;
    // forward sweep up to the start of the last block, keeping the state at the start of every block
    if (n_blocks > 1) {
        FRaw r = frequest(0);
        for (int i = 0; i < (n_blocks - 1) * L; ++i) {
            if (i % L == 0) put(stored + (size_t)(i / L) * p.H * D * D, S);
            const FRaw rn = frequest(i + 1);
            fstep(S, r);
            r = rn;
        }
    }

    // ---- reverse sweep, block by block ----
    struct BRaw { alignas(16) IO dout[WC]; IO q[J], k[J], v; float la, eta; };
    auto brequest = [&](int i) {
        BRaw r;
        const size_t th = (size_t)(tok0 + max(i, 0)) * p.H + h;
#pragma unroll
        for (int j = 0; j < J; ++j) {
            r.q[j] = qp[th * D + lane + 32 * j];
            r.k[j] = kp[th * D + lane + 32 * j];
        }
        r.v = vp[th * D + c0 + myc];
        r.la = p.log_alpha[th];
        r.eta = p.eta[th];
#pragma unroll
        for (int c = 0; c < WC; c += 4) {   // the same WC values for every lane
            if constexpr (sizeof(IO) == 2) {
                const uint2 raw = *reinterpret_cast<const uint2 *>(dop + th * D + c0 + c);
                *reinterpret_cast<uint2 *>(&r.dout[c]) = raw;
            } else {
                const float4 raw = *reinterpret_cast<const float4 *>(dop + th * D + c0 + c);
                *reinterpret_cast<float4 *>(&r.dout[c]) = raw;
            }
        }
        return r;
    };
    for (int b = n_blocks - 1; b >= 0; --b) {
        const int i0 = b * L, i1 = min(i0 + L, len);
        if (b != n_blocks - 1) get(stored + (size_t)b * p.H * D * D, S);
        {   // the state before every token of the block (the last one stays in registers)
            FRaw r = frequest(i0);
            for (int i = i0; i + 1 < i1; ++i) {
                put(scratch + (size_t)(i - i0) * D * D, S);
                const FRaw rn = frequest(i + 1);
                fstep(S, r);
                r = rn;
            }
        }
        BRaw raw = brequest(i1 - 1);
        for (int i = i1 - 1; i >= i0; --i) {
            // S holds S_{i-1}; the state and the operands of the token before are requested now and used next iteration
            float Sn[J][WC];
            if (i > i0) get(scratch + (size_t)(i - 1 - i0) * D * D, Sn);
            const BRaw rawn = brequest(i - 1);
            const size_t th = (size_t)(tok0 + i) * p.H + h;
            float q[J], k[J], dout[WC], nk = 0.f, nq = 0.f;
#pragma unroll
            for (int j = 0; j < J; ++j) {
                q[j] = to_f32(raw.q[j]);
                k[j] = to_f32(raw.k[j]);
                nk += k[j] * k[j];
                nq += q[j] * q[j];
            }
#pragma unroll
            for (int c = 0; c < WC; ++c) dout[c] = to_f32(raw.dout[c]);
            const float alpha = __expf(raw.la);
            const float nrm = warp_sum(nk) + p.eps;
            const float beta = p.coeff_eta ? raw.eta : raw.eta / nrm;   // Eq. 3
            float qinv = 1.f;
            if (QN) {
                qinv = rsqrtf(warp_sum(nq));
#pragma unroll
                for (int j = 0; j < J; ++j) q[j] *= qinv;   // qh
            }
            // forward quantities of the token: S~ = alpha S_{i-1} (in place), e = v - S~^T k
            float part[WC], e[WC], de[WC];
#pragma unroll
            for (int c = 0; c < WC; ++c) {
                float s = 0.f;
#pragma unroll
                for (int j = 0; j < J; ++j) {
                    S[j][c] *= alpha;
                    s += k[j] * S[j][c];
                }
                part[c] = s;
            }
            const float e_mine = to_f32(raw.v) - reduce_scatter<WC>(part, lane);
#pragma unroll
            for (int c = 0; c < WC; ++c) e[c] = __shfl_sync(0xffffffffu, e_mine, lane_of_col<WC>(c));
            // read-out: dqh = S_t dO with S_t = S~ + beta k e^T formed on the fly; G += qh dO^T; then u = G^T k
            float dq[J], dk[J];
#pragma unroll
            for (int j = 0; j < J; ++j) dq[j] = 0.f;
#pragma unroll
            for (int c = 0; c < WC; ++c) {
                const float be = beta * e[c];
                float s = 0.f;
#pragma unroll
                for (int j = 0; j < J; ++j) {
                    dq[j] += (S[j][c] + k[j] * be) * dout[c];
                    G[j][c] += q[j] * dout[c];
                    s += G[j][c] * k[j];
                }
                part[c] = s;
            }
            const float u_mine = reduce_scatter<WC>(part, lane);
            const float de_mine = beta * u_mine;                                      // de = beta G^T k  (= dv)
            const float dbeta = warp_sum((lane & 3) == 0 ? u_mine * e_mine : 0.f);   // this warp's columns of k^T G e
#pragma unroll
            for (int c = 0; c < WC; ++c) de[c] = __shfl_sync(0xffffffffu, de_mine, lane_of_col<WC>(c));
            // dk = beta G e - S~ de;  G <- alpha (G - k de^T);  dlog_alpha = <G - k de^T, S~>
            float dla = 0.f;
#pragma unroll
            for (int j = 0; j < J; ++j) {
                float ge = 0.f, sd = 0.f;
#pragma unroll
                for (int c = 0; c < WC; ++c) {
                    ge += G[j][c] * e[c];
                    sd += S[j][c] * de[c];
                    const float g = G[j][c] - k[j] * de[c];
                    dla += g * S[j][c];
                    G[j][c] = alpha * g;
                }
                dk[j] = beta * ge - sd;
            }
            dla = warp_sum(dla);
            float deta = dbeta;
            if (!p.coeff_eta) {   // beta = eta / n: deta = dbeta / n, dn = -dbeta eta / n^2 = -dbeta beta / n, dk += 2 k dn
                deta = dbeta / nrm;
                const float dn2 = -2.f * dbeta * beta / nrm;
#pragma unroll
                for (int j = 0; j < J; ++j) dk[j] += k[j] * dn2;
            }
            if (QN) {   // o = S^T q / ||q||: dq = (dqh - qh (qh . dqh)) / ||q||, a linear map, applied to this warp's part
                float pr = 0.f;
#pragma unroll
                for (int j = 0; j < J; ++j) pr += q[j] * dq[j];
                pr = warp_sum(pr);
#pragma unroll
                for (int j = 0; j < J; ++j) dq[j] = (dq[j] - q[j] * pr) * qinv;
            }
            if ((lane & 3) == 0) p.dv[th * D + c0 + myc] = de_mine;
            // sums over the block's columns
            float *mine = red[i & 1][warp];
#pragma unroll
            for (int j = 0; j < J; ++j) {
                mine[lane + 32 * j] = dq[j];
                mine[D + lane + 32 * j] = dk[j];
            }
            if (lane == 0) {
                mine[2 * D] = dla;
                mine[2 * D + 1] = deta;
            }
            __syncthreads();   // one barrier per token: the buffers alternate, and nobody is two tokens ahead of anybody
            for (int x = threadIdx.x; x < NRED; x += NT) {
                float s = 0.f;
#pragma unroll
                for (int w = 0; w < WARPS; ++w) s += red[i & 1][w][x];
                float *dst = x < D ? p.dq + th * D + x : x < 2 * D ? p.dk + th * D + (x - D) : x == 2 * D ? p.dlog_alpha + th : p.deta + th;
                if (SPLIT == 1) *dst = s;
                else atomicAdd(dst, s);
            }
            if (i > i0) {
#pragma unroll
                for (int j = 0; j < J; ++j)
#pragma unroll
                    for (int c = 0; c < WC; ++c) S[j][c] = Sn[j][c];
            }
            raw = rawn;
        }
    }
    if (p.dinit) {
#pragma unroll
        for (int j = 0; j < J; ++j)
#pragma unroll
            for (int c = 0; c < WC; c += 4)
                store4(p.dinit + sbase + (size_t)(lane + 32 * j) * D + c0 + c, make_float4(G[j][c], G[j][c + 1], G[j][c + 2], G[j][c + 3]));
    }
}

template <int D, typename IO>
cudaError_t launch_io(const BwdParams &p, int qnorm, cudaStream_t stream)
{
    const int blocks = p.n_seq * p.H * (D / 64);
    if (blocks == 0) return cudaSuccess;
    if (qnorm)
        kla_bwd_scan_kernel<D, IO, true><<<blocks, NT, 0, stream>>>(p);
    else
        kla_bwd_scan_kernel<D, IO, false><<<blocks, NT, 0, stream>>>(p);
    count_launch(1);
    return cudaGetLastError();
}

}  // namespace

size_t bwd_workspace_bytes(int n_seq, long long n_tok, int H, int d)
{
    const size_t state = (size_t)d * d * sizeof(float);
    return ((size_t)(n_tok / L + n_seq) * H + (size_t)n_seq * H * L) * state;
}

cudaError_t launch_bwd_scan(const void *q, const void *k, const void *v, const float *log_alpha, const float *eta,
                            const float *init_state, const void *dout, const float *dfinal, float *dq, float *dk, float *dv,
                            float *dlog_alpha, float *deta, float *dinit, void *workspace, const int32_t *cu_seqlens, int T,
                            long long n_tok, int H, int n_seq, int d, float eps, int coeff_eta, int qnorm, int io_dtype,
                            cudaStream_t stream)
{
    BwdParams p;
    p.q = q; p.k = k; p.v = v; p.dout = dout;
    p.log_alpha = log_alpha; p.eta = eta;
    p.init_state = init_state; p.dfinal = dfinal;
    p.dq = dq; p.dk = dk; p.dv = dv; p.dlog_alpha = dlog_alpha; p.deta = deta; p.dinit = dinit;
    p.stored = reinterpret_cast<float *>(workspace);
    p.scratch = p.stored + (size_t)(n_tok / L + n_seq) * H * d * d;
    p.cu_seqlens = cu_seqlens;
    p.T = T; p.H = H; p.n_seq = n_seq;
    p.eps = eps;
    p.coeff_eta = coeff_eta;
    if (d == 128) {   // two blocks per head add into the outputs that are sums over columns
        cudaError_t e = cudaMemsetAsync(dq, 0, (size_t)n_tok * H * d * sizeof(float), stream);
        if (e == cudaSuccess) e = cudaMemsetAsync(dk, 0, (size_t)n_tok * H * d * sizeof(float), stream);
        if (e == cudaSuccess) e = cudaMemsetAsync(dlog_alpha, 0, (size_t)n_tok * H * sizeof(float), stream);
        if (e == cudaSuccess) e = cudaMemsetAsync(deta, 0, (size_t)n_tok * H * sizeof(float), stream);
        if (e != cudaSuccess) return e;
        return io_dtype == KLA_BF16 ? launch_io<128, __nv_bfloat16>(p, qnorm, stream) : launch_io<128, float>(p, qnorm, stream);
    }
    return io_dtype == KLA_BF16 ? launch_io<64, __nv_bfloat16>(p, qnorm, stream) : launch_io<64, float>(p, qnorm, stream);
}

}  // namespace kla
