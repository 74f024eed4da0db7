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
// with the state before every token written to the thread block's scratch area (16 states, L2-resident), then walked in
// reverse.  One block per SM is resident; (sequence, head, half) units beyond that are taken in turn.
// Every thread reads back only what it wrote itself, so no fence or barrier guards the stored states.
//
// Work split: columns of S and G never interact, so a block owns 64 columns of one (sequence, head), one warp 8 of them,
// lane l rows l, l + 32, ... (S_{t-1}, G and the prefetched next S_{t-1} in registers).  Sums over rows (S~^T k, G^T k)
// are reduce-scatter butterflies inside the warp; sums over columns (dq, dk, dbeta, dlog_alpha) are per-warp partials
// added up through shared memory once per block of 16 tokens.  With d = 128 the two blocks of a head add their halves into
// zero-initialised outputs with one atomic each: two commutative additions, so the result does not depend on their order.
#include "common.cuh"
#include "scan_pieces.cuh"

namespace kla {

namespace {

#ifndef BWD_WC
#define BWD_WC 8   // state columns per warp (4: sixteen warps per block, 8.7 ms against 8.4 ms on the layer shape)
#endif
constexpr int WC = BWD_WC;
constexpr int WARPS = 64 / WC;   // warps per block (64 columns)
constexpr int NT = 32 * WARPS;
constexpr int L = 16;         // tokens between stored states
constexpr int RL = WC == 8 ? 16 : 8;   // tokens between two additions of the warps' partial sums (shared memory: RL x WARPS x (2 d + 2) floats)

struct BwdParams {
    const void *q, *k, *v, *dout;
    const float *log_alpha, *eta;      // [n_tok, H]
    const float *init_state, *dfinal;  // [n_seq, H, D, D] or null
    float *dq, *dk, *dv;               // [n_tok, H, D]
    float *dlog_alpha, *deta;          // [n_tok, H]
    float *dinit;                      // [n_seq, H, D, D] or null
    float *stored;                     // states every L tokens: slot (tok0 / L + n + block) * H + h
    float *scratch;                    // L states of 64 columns per resident block
    const int32_t *cu_seqlens;         // null: fixed length T
    int32_t T, H, n_seq;
    float eps;
    int32_t coeff_eta;
    int32_t n_units;                   // (sequence, head, 64-column half) units; the resident blocks take them in turn
    int32_t *next_unit;                // zeroed before the launch: units beyond the first gridDim.x are handed out in order
};

// One block of L tokens as the steps read it.
template <int D>
struct Stage {
    float k[L][D], q[L][D];       // q already divided by ||q|| when the read-out is normalised
    float v[L][64], dout[L][64];  // the 64 columns of this thread block
    float alpha[L], beta[L], nrm[L], qinv[L];
};

template <int D, typename IO, bool QN>
__global__ void __launch_bounds__(NT, 1) kla_bwd_scan_kernel(BwdParams p)
{
    constexpr int J = D / 32;            // rows per lane
    constexpr int SPLIT = D / 64;        // blocks per head
    constexpr int NRED = 2 * D + 2;      // per-token sums over columns: dq, dk, dlog_alpha, deta
    extern __shared__ __align__(16) float smem_all[];
    Stage<D> *const stage = reinterpret_cast<Stage<D> *>(smem_all);                    // two buffers
    float *const red_all = smem_all + 2 * sizeof(Stage<D>) / sizeof(float);            // [RL][WARPS][NRED]: the warps' partial sums over their columns
    auto red = [&](int slot, int w) { return red_all + ((size_t)slot * WARPS + w) * NRED; };
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int myc = col_of_lane<WC>(lane);       // the column whose row sums this lane ends up with
    const IO *qp = reinterpret_cast<const IO *>(p.q), *kp = reinterpret_cast<const IO *>(p.k), *vp = reinterpret_cast<const IO *>(p.v);
    const IO *dop = reinterpret_cast<const IO *>(p.dout);
    // the scratch states belong to the block, not to the unit it is working on
    float *const scratch = p.scratch + (size_t)blockIdx.x * L * 64 * D + ((size_t)warp * J * (WC / 4)) * 128 + lane * 4;
    __shared__ int unit_s;
    for (int unit = blockIdx.x; unit < p.n_units;) {
        const int split = unit % SPLIT, h = (unit / SPLIT) % p.H, n = unit / (SPLIT * p.H);
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
        const size_t sbase = ((size_t)n * p.H + h) * D * D;
        // Stored states use a layout of their own, [column group][j][quad of columns][lane] float4, so that every access is 512 contiguous bytes.
        const size_t soff = ((size_t)cg * J * (WC / 4)) * 128 + lane * 4;
        float *const stored = p.stored + ((size_t)(tok0 / L + n) * p.H + h) * D * D + soff;
        auto put = [&](float *dst, const float (&S)[J][WC]) {
#pragma unroll
            for (int j = 0; j < J; ++j)
#pragma unroll
                for (int c = 0; c < WC; c += 4)
                    store4(dst + (j * (WC / 4) + c / 4) * 128, make_float4(S[j][c], S[j][c + 1], S[j][c + 2], S[j][c + 3]));
        };
        auto get = [&](const float *src, float (&S)[J][WC]) {
#pragma unroll
            for (int j = 0; j < J; ++j)
#pragma unroll
                for (int c = 0; c < WC; c += 4) {
                    const float4 a = load4(src + (j * (WC / 4) + c / 4) * 128);
                    S[j][c] = a.x; S[j][c + 1] = a.y; S[j][c + 2] = a.z; S[j][c + 3] = a.w;
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

        float S[J][WC], G[J][WC];
        get_natural(p.init_state, S);
        get_natural(p.dfinal, G);
        const int n_blocks = (len + L - 1) / L;

        // ---- operands of one block of L tokens, staged in shared memory as fp32 together with the per-token scalars ----
        // Each warp fetches whole tokens (TPW of them): the raw values are requested into registers before the block in hand
        // is processed and touched only after it (a use, even a conversion, would wait for them), then converted, reduced to
        // alpha, beta (Eq. 3), ||k||^2 + eps and 1 / ||q||, and written to the buffer that is not being read.
        constexpr int TPW = L / WARPS;
        struct Pre { IO k[J], q[J]; IO v[2], dout[2]; float la, eta; };
        Pre pre[TPW];
        auto request_block = [&](int b, bool full) {
#pragma unroll
            for (int u = 0; u < TPW; ++u) {
                const int i = min(b * L + warp + u * WARPS, len - 1);
                const size_t th = (size_t)(tok0 + i) * p.H + h;
#pragma unroll
                for (int j = 0; j < J; ++j) {
                    pre[u].k[j] = kp[th * D + lane + 32 * j];
                    if (full) pre[u].q[j] = qp[th * D + lane + 32 * j];
                }
                const size_t col = th * D + split * 64 + 2 * lane;   // this block's 64 columns, two per lane
                if constexpr (sizeof(IO) == 2) {
                    *reinterpret_cast<uint32_t *>(pre[u].v) = *reinterpret_cast<const uint32_t *>(vp + col);
                    if (full) *reinterpret_cast<uint32_t *>(pre[u].dout) = *reinterpret_cast<const uint32_t *>(dop + col);
                } else {
                    *reinterpret_cast<float2 *>(pre[u].v) = *reinterpret_cast<const float2 *>(vp + col);
                    if (full) *reinterpret_cast<float2 *>(pre[u].dout) = *reinterpret_cast<const float2 *>(dop + col);
                }
                pre[u].la = p.log_alpha[th];
                pre[u].eta = p.eta[th];
            }
        };
        auto commit_block = [&](Stage<D> &st, bool full) {
#pragma unroll
            for (int u = 0; u < TPW; ++u) {
                const int tok = warp + u * WARPS;
                float nk = 0.f, nq = 0.f, q[J];
#pragma unroll
                for (int j = 0; j < J; ++j) {
                    const float k = to_f32(pre[u].k[j]);
                    st.k[tok][lane + 32 * j] = k;
                    nk += k * k;
                    if (full) {
                        q[j] = to_f32(pre[u].q[j]);
                        nq += q[j] * q[j];
                    }
                }
                const float nrm = warp_sum(nk) + p.eps;
                float qinv = 1.f;
                if (QN && full) qinv = rsqrtf(warp_sum(nq));
                store2(&st.v[tok][2 * lane], to_f32(pre[u].v[0]), to_f32(pre[u].v[1]));
                if (full) {
#pragma unroll
                    for (int j = 0; j < J; ++j) st.q[tok][lane + 32 * j] = q[j] * qinv;   // qh
                    store2(&st.dout[tok][2 * lane], to_f32(pre[u].dout[0]), to_f32(pre[u].dout[1]));
                }
                if (lane == 0) {
                    st.alpha[tok] = __expf(pre[u].la);
                    st.beta[tok] = p.coeff_eta ? pre[u].eta : pre[u].eta / nrm;   // Eq. 3
                    st.nrm[tok] = nrm;
                    st.qinv[tok] = qinv;
                }
            }
        };
        // one forward step without read-out
        auto fstep = [&](const Stage<D> &st, int tok) {
            float2 k[J];   // (k_j, k_j)
            float part[WC];
#pragma unroll
            for (int j = 0; j < J; ++j) k[j] = f2(st.k[tok][lane + 32 * j]);
            const float alpha = st.alpha[tok], beta = st.beta[tok];
#pragma unroll
            for (int c = 0; c < WC; c += 2) {
                float2 s = f2(0.f);
#pragma unroll
                for (int j = 0; j < J; ++j) s = fma2(k[j], f2(S[j][c], S[j][c + 1]), s);
                part[c] = s.x;
                part[c + 1] = s.y;
            }
            const float e_mine = st.v[tok][warp * WC + myc] - alpha * reduce_scatter<WC>(part, lane);
            const float2 a2 = f2(alpha);
#pragma unroll
            for (int c = 0; c < WC; c += 2) {
                const float2 be = f2(beta * __shfl_sync(0xffffffffu, e_mine, lane_of_col<WC>(c)),
                                     beta * __shfl_sync(0xffffffffu, e_mine, lane_of_col<WC>(c + 1)));
#pragma unroll
                for (int j = 0; j < J; ++j) {
                    const float2 r = fma2(a2, f2(S[j][c], S[j][c + 1]), mul2(k[j], be));
                    S[j][c] = r.x;
                    S[j][c + 1] = r.y;
                }
            }
        };

        if (n_blocks > 0) {
            int cur = 0;
            request_block(0, n_blocks == 1);
            commit_block(stage[0], n_blocks == 1);
            __syncthreads();
            // forward sweep up to the start of the last block, keeping the state at the start of every block
            for (int b = 0; b + 1 < n_blocks; ++b) {
                const bool next_full = b + 2 == n_blocks;   // the last block is the first one the reverse sweep works on
                request_block(b + 1, next_full);
                put(stored + (size_t)b * p.H * D * D, S);
                for (int tok = 0; tok < L; ++tok) fstep(stage[cur], tok);
                commit_block(stage[cur ^ 1], next_full);
                __syncthreads();   // one barrier per block: the buffer written is the one nobody reads
                cur ^= 1;
            }
            // ---- reverse sweep, block by block ----
            for (int b = n_blocks - 1; b >= 0; --b) {
                const int i0 = b * L, cnt = min(L, len - i0);
                const Stage<D> &st = stage[cur];
                if (b > 0) request_block(b - 1, true);
                if (b != n_blocks - 1) get(stored + (size_t)b * p.H * D * D, S);
                // the state before every token of the block (the last one stays in registers)
                for (int tok = 0; tok + 1 < cnt; ++tok) {
                    put(scratch + (size_t)tok * 64 * D, S);
                    fstep(st, tok);
                }
                for (int tok = cnt - 1; tok >= 0; --tok) {
                    // S holds the state before this token; the one before the previous token is requested now, used next iteration
                    float Sn[J][WC];
                    if (tok > 0) get(scratch + (size_t)(tok - 1) * 64 * D, Sn);
                    const size_t th = (size_t)(tok0 + i0 + tok) * p.H + h;
                    float q[J], k[J], dout[WC];
#pragma unroll
                    for (int j = 0; j < J; ++j) {
                        q[j] = st.q[tok][lane + 32 * j];   // qh
                        k[j] = st.k[tok][lane + 32 * j];
                    }
#pragma unroll
                    for (int c = 0; c < WC; c += 4) {
                        const float4 x = load4(&st.dout[tok][warp * WC + c]);
                        dout[c] = x.x; dout[c + 1] = x.y; dout[c + 2] = x.z; dout[c + 3] = x.w;
                    }
                    const float alpha = st.alpha[tok], beta = st.beta[tok], nrm = st.nrm[tok];
                    // forward quantities of the token: S~ = alpha S_{t-1} (in place), e = v - S~^T k
                    float part[WC], e[WC], de[WC];
                    float2 k2[J], q2[J];
#pragma unroll
                    for (int j = 0; j < J; ++j) {
                        k2[j] = f2(k[j]);
                        q2[j] = f2(q[j]);
                    }
                    const float2 a2 = f2(alpha);
#pragma unroll
                    for (int c = 0; c < WC; c += 2) {
                        float2 s = f2(0.f);
#pragma unroll
                        for (int j = 0; j < J; ++j) {
                            const float2 st2 = mul2(a2, f2(S[j][c], S[j][c + 1]));
                            S[j][c] = st2.x;
                            S[j][c + 1] = st2.y;
                            s = fma2(k2[j], st2, s);
                        }
                        part[c] = s.x;
                        part[c + 1] = s.y;
                    }
                    const float e_mine = st.v[tok][warp * WC + myc] - reduce_scatter<WC>(part, lane);
#pragma unroll
                    for (int c = 0; c < WC; ++c) e[c] = __shfl_sync(0xffffffffu, e_mine, lane_of_col<WC>(c));
                    // read-out: dqh = S_t dO = S~ dO + k (beta e . dO); G += qh dO^T; then u = G^T k
                    float dq[J], dk[J];
                    float2 dq2[J];
                    float bed = 0.f;   // beta e . dO over this warp's columns
#pragma unroll
                    for (int c = 0; c < WC; ++c) bed += e[c] * dout[c];
                    bed *= beta;
#pragma unroll
                    for (int j = 0; j < J; ++j) dq2[j] = f2(0.f);
#pragma unroll
                    for (int c = 0; c < WC; c += 2) {
                        const float2 do2 = f2(dout[c], dout[c + 1]);
                        float2 s = f2(0.f);
#pragma unroll
                        for (int j = 0; j < J; ++j) {
                            dq2[j] = fma2(f2(S[j][c], S[j][c + 1]), do2, dq2[j]);
                            const float2 g = fma2(q2[j], do2, f2(G[j][c], G[j][c + 1]));
                            G[j][c] = g.x;
                            G[j][c + 1] = g.y;
                            s = fma2(g, k2[j], s);
                        }
                        part[c] = s.x;
                        part[c + 1] = s.y;
                    }
#pragma unroll
                    for (int j = 0; j < J; ++j) dq[j] = dq2[j].x + dq2[j].y + k[j] * bed;
                    const float u_mine = reduce_scatter<WC>(part, lane);
                    const float de_mine = beta * u_mine;                                                   // de = beta G^T k  (= dv)
                    const float dbeta = warp_sum((lane & (32 / WC - 1)) == 0 ? u_mine * e_mine : 0.f);   // this warp's columns of k^T G e
#pragma unroll
                    for (int c = 0; c < WC; ++c) de[c] = __shfl_sync(0xffffffffu, de_mine, lane_of_col<WC>(c));
                    // dk = beta G e - S~ de;  G <- alpha (G - k de^T);  dlog_alpha = <G - k de^T, S~>
                    float2 dla2 = f2(0.f);
#pragma unroll
                    for (int j = 0; j < J; ++j) {
                        float2 ge = f2(0.f), sd = f2(0.f);
                        const float2 nk2 = f2(-k[j]);
#pragma unroll
                        for (int c = 0; c < WC; c += 2) {
                            const float2 g0 = f2(G[j][c], G[j][c + 1]), s0 = f2(S[j][c], S[j][c + 1]), de2 = f2(de[c], de[c + 1]);
                            ge = fma2(g0, f2(e[c], e[c + 1]), ge);
                            sd = fma2(s0, de2, sd);
                            const float2 g = fma2(nk2, de2, g0);
                            dla2 = fma2(g, s0, dla2);
                            const float2 ga = mul2(a2, g);
                            G[j][c] = ga.x;
                            G[j][c + 1] = ga.y;
                        }
                        dk[j] = beta * (ge.x + ge.y) - (sd.x + sd.y);
                    }
                    float dla = dla2.x + dla2.y;
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
                        const float qinv = st.qinv[tok];
#pragma unroll
                        for (int j = 0; j < J; ++j) dq[j] = (dq[j] - q[j] * pr) * qinv;
                    }
                    if ((lane & (32 / WC - 1)) == 0) p.dv[th * D + c0 + myc] = de_mine;
                    // this warp's part of the sums over columns; added up every RL tokens
                    float *mine = red(tok % RL, warp);
#pragma unroll
                    for (int j = 0; j < J; ++j) {
                        mine[lane + 32 * j] = dq[j];
                        mine[D + lane + 32 * j] = dk[j];
                    }
                    if (lane == 0) {
                        mine[2 * D] = dla;
                        mine[2 * D + 1] = deta;
                    }
                    if (tok > 0) {
#pragma unroll
                        for (int j = 0; j < J; ++j)
#pragma unroll
                            for (int c = 0; c < WC; ++c) S[j][c] = Sn[j][c];
                    }
                    if (tok % RL == 0) {   // add up the partial sums of tokens tok .. tok + RL - 1 (fewer at the end of the sequence)
                        __syncthreads();
                        const int n_sum = min(RL, cnt - tok);
                        for (int idx = threadIdx.x; idx < n_sum * NRED; idx += NT) {
                            const int slot = idx / NRED, x = idx - slot * NRED;
                            float s = 0.f;
#pragma unroll
                            for (int w = 0; w < WARPS; ++w) s += red(slot, w)[x];
                            const size_t tq = th + (size_t)slot * p.H;
                            float *dst = x < D ? p.dq + tq * D + x : x < 2 * D ? p.dk + tq * D + (x - D) : x == 2 * D ? p.dlog_alpha + tq : p.deta + tq;
                            if (SPLIT == 1) *dst = s;
                            else atomicAdd(dst, s);
                        }
                        __syncthreads();
                    }
                }
                if (b > 0) commit_block(stage[cur ^ 1], true);
                __syncthreads();
                cur ^= 1;
            }
        }
        if (p.dinit) {
#pragma unroll
            for (int j = 0; j < J; ++j)
#pragma unroll
                for (int c = 0; c < WC; c += 4)
                    store4(p.dinit + sbase + (size_t)(lane + 32 * j) * D + c0 + c, make_float4(G[j][c], G[j][c + 1], G[j][c + 2], G[j][c + 3]));
        }
        // the next unit, in the order blocks become free (packed input: lengths differ)
        __syncthreads();
        if (threadIdx.x == 0) unit_s = (int)gridDim.x + atomicAdd(p.next_unit, 1);
        __syncthreads();
        unit = unit_s;
    }
}

// One block per SM (registers and shared memory); more units than that are taken in turn.
int bwd_resident_blocks()
{
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
        return 148;
    return n;
}

template <int D, typename IO>
cudaError_t launch_io(const BwdParams &p, int qnorm, cudaStream_t stream)
{
    if (p.n_units == 0) return cudaSuccess;
    const int blocks = p.n_units < bwd_resident_blocks() ? p.n_units : bwd_resident_blocks();
    constexpr int smem = 2 * (int)sizeof(Stage<D>) + RL * WARPS * (2 * D + 2) * (int)sizeof(float);
    auto kern = qnorm ? kla_bwd_scan_kernel<D, IO, true> : kla_bwd_scan_kernel<D, IO, false>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    kern<<<blocks, NT, smem, stream>>>(p);
    count_launch(1);
    return cudaGetLastError();
}

}  // namespace

size_t bwd_workspace_bytes(int n_seq, long long n_tok, int H, int d)
{
    const size_t state = (size_t)d * d * sizeof(float);
    const long long units = (long long)n_seq * H * (d / 64);
    const size_t blocks = (size_t)(units < bwd_resident_blocks() ? units : bwd_resident_blocks());
    return 256 + (size_t)(n_tok / L + n_seq) * H * state + blocks * L * 64 * d * sizeof(float);   // (256: the unit counter)
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
    p.next_unit = reinterpret_cast<int32_t *>(workspace);
    p.stored = reinterpret_cast<float *>(reinterpret_cast<char *>(workspace) + 256);
    p.scratch = p.stored + (size_t)(n_tok / L + n_seq) * H * d * d;
    if (cudaMemsetAsync(p.next_unit, 0, sizeof(int32_t), stream) != cudaSuccess) return cudaGetLastError();
    p.cu_seqlens = cu_seqlens;
    p.T = T; p.H = H; p.n_seq = n_seq;
    p.eps = eps;
    p.coeff_eta = coeff_eta;
    p.n_units = n_seq * H * (d / 64);
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
