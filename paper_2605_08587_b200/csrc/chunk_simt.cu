// Chunkwise forward on CUDA cores in fp32 (Algorithm 1, right panel; Eqs. 7-9).
//
// Serves fp32 inputs (where fp32 FMA accuracy is wanted), chunk lengths 16/32, and acts as the
// device-side cross-check of the chunk algebra for the tensor-core kernel.
//
// One CTA (256 threads) owns NS = 32 consecutive d_v columns of one (sequence, head) and walks
// the chunks of that sequence in order, carrying its d_k x NS slice of the state in shared
// memory.  Columns of the state never interact (the write is k e^T), so slices need no exchange.
// Per chunk, with g_i = sum_{r<=i} log alpha_r (chunk-local), gamma_i = exp(g_i):
//   beta_i = eta_i / (||k_i||^2 + eps)                                         (Eq. 3)
//   L_ij = beta_i exp(g_i - g_j) k_i.k_j (j < i),  P_ij = exp(g_i - g_j) q_i.k_j (j <= i)
//   rhs_i = beta_i (v_i - gamma_i k_i^T S_0)                                   (right side of Eq. 7)
//   (I + L) U = rhs   by forward substitution                                  (Eq. 7)
//   O = D_gamma Q S_0 + P U                                                    (Eq. 8)
//   S <- gamma_C S_0 + K^T diag(exp(g_C - g_j)) U                              (Eq. 9)
// Decay ratios are always exp of a difference of running sums, never 1/gamma_j.
// Rows past the end of a sequence's last chunk are zero with beta = 0 and log alpha = 0, which
// makes them inert in every formula above.
#include "common.cuh"

namespace kla {

namespace {

constexpr int NS = 32;        // state columns per CTA
constexpr int NTHREADS = 256;

template <int D, int C>
struct SimtSmem {
    static constexpr int LDK = D + 4;  // padded row length of the K/Q tiles
    static constexpr int LDL = C + 1;
    float K[C][LDK];
    float Q[C][LDK];
    float V[C][NS];
    float X[C][NS];    // rhs, then U
    float O[C][NS];    // gamma_i (Q S_0)_i
    float S[D][NS];
    float L[C][LDL];
    float P[C][LDL];
    double g[C];       // chunk-local running sum of log alpha; kept in fp64 so that the
                       // differences g_i - g_j below do not cancel away fp32 digits
    float beta[C], la[C], eta[C];
    float qn[C];       // 1 / ||q_i|| when the normalised read-out is asked for, else 1
};

template <typename IO>
struct Vec8 {};
template <>
struct Vec8<float> {
    float4 a, b;
    __device__ void load(const float *p) { a = *reinterpret_cast<const float4 *>(p); b = *reinterpret_cast<const float4 *>(p + 4); }
    __device__ void zero() { a = make_float4(0, 0, 0, 0); b = a; }
    __device__ void store_f32(float *s) const { *reinterpret_cast<float4 *>(s) = a; *reinterpret_cast<float4 *>(s + 4) = b; }
};
template <>
struct Vec8<__nv_bfloat16> {
    uint4 r;
    __device__ void load(const __nv_bfloat16 *p) { r = *reinterpret_cast<const uint4 *>(p); }
    __device__ void zero() { r = make_uint4(0, 0, 0, 0); }
    __device__ void store_f32(float *s) const
    {
        const __nv_bfloat162 *h = reinterpret_cast<const __nv_bfloat162 *>(&r);
        float2 f0 = __bfloat1622float2(h[0]), f1 = __bfloat1622float2(h[1]);
        float2 f2 = __bfloat1622float2(h[2]), f3 = __bfloat1622float2(h[3]);
        *reinterpret_cast<float4 *>(s) = make_float4(f0.x, f0.y, f1.x, f1.y);
        *reinterpret_cast<float4 *>(s + 4) = make_float4(f2.x, f2.y, f3.x, f3.y);
    }
};

template <int D, int C, typename IO, typename OUT>
__global__ void __launch_bounds__(NTHREADS) kla_chunk_simt_kernel(ChunkParams p)
{
    using Smem = SimtSmem<D, C>;
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Smem &sm = *reinterpret_cast<Smem *>(smem_raw);

    constexpr int SLICES = D / NS;
    constexpr int KQ_ITEMS = C * D / 8;               // 8-element vectors in a K (or Q) tile
    constexpr int KQ_PER_THREAD = (KQ_ITEMS + NTHREADS - 1) / NTHREADS;
    constexpr int V_ITEMS = C * NS / 8;
    constexpr int TD = C / 4;                         // 4x4 tiles per side of the C x C matrices
    constexpr int RD = D / 32;                        // state rows per thread in the update

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sl = blockIdx.x % SLICES;
    const int h = (blockIdx.x / SLICES) % p.H;
    const int n = blockIdx.x / (SLICES * p.H);

    int tok0, len;
    if (p.cu_seqlens) {
        tok0 = p.cu_seqlens[n];
        len = p.cu_seqlens[n + 1] - tok0;
    } else {
        tok0 = n * p.T;
        len = p.T;
    }
    const IO *qg = reinterpret_cast<const IO *>(p.q);
    const IO *kg = reinterpret_cast<const IO *>(p.k);
    const IO *vg = reinterpret_cast<const IO *>(p.v);
    OUT *og = reinterpret_cast<OUT *>(p.out);
    const size_t HD = (size_t)p.H * D;

    // initial state slice
    for (int i = tid; i < D * NS / 4; i += NTHREADS) {
        const int r = i / (NS / 4), c4 = (i % (NS / 4)) * 4;
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (p.init_state) x = *reinterpret_cast<const float4 *>(p.init_state + (((size_t)n * p.H + h) * D + r) * D + sl * NS + c4);
        *reinterpret_cast<float4 *>(&sm.S[r][c4]) = x;
    }

    Vec8<IO> rk[KQ_PER_THREAD], rq[KQ_PER_THREAD], rv;
    float r_la = 0.f, r_eta = 0.f;

    auto fetch = [&](int c0) {
        const int rows = min(C, len - c0);
#pragma unroll
        for (int u = 0; u < KQ_PER_THREAD; ++u) {
            const int it = tid + u * NTHREADS;
            const int r = it / (D / 8), c8 = (it % (D / 8)) * 8;
            if (it < KQ_ITEMS && r < rows) {
                const size_t off = (size_t)(tok0 + c0 + r) * HD + (size_t)h * D + c8;
                rk[u].load(kg + off);
                rq[u].load(qg + off);
            } else {
                rk[u].zero();
                rq[u].zero();
            }
        }
        {
            const int r = tid / (NS / 8), c8 = (tid % (NS / 8)) * 8;
            if (tid < V_ITEMS && r < rows)
                rv.load(vg + (size_t)(tok0 + c0 + r) * HD + (size_t)h * D + sl * NS + c8);
            else
                rv.zero();
        }
        if (tid < C) {
            const bool ok = tid < rows;
            r_la = ok ? p.log_alpha[(size_t)(tok0 + c0 + tid) * p.H + h] : 0.f;
            r_eta = ok ? p.eta[(size_t)(tok0 + c0 + tid) * p.H + h] : 0.f;
        }
    };
    auto stash = [&]() {
#pragma unroll
        for (int u = 0; u < KQ_PER_THREAD; ++u) {
            const int it = tid + u * NTHREADS;
            if (it < KQ_ITEMS) {
                const int r = it / (D / 8), c8 = (it % (D / 8)) * 8;
                rk[u].store_f32(&sm.K[r][c8]);
                rq[u].store_f32(&sm.Q[r][c8]);
            }
        }
        if (tid < V_ITEMS) {
            const int r = tid / (NS / 8), c8 = (tid % (NS / 8)) * 8;
            rv.store_f32(&sm.V[r][c8]);
        }
        if (tid < C) {
            sm.la[tid] = r_la;
            sm.eta[tid] = r_eta;
        }
    };

    if (len > 0) fetch(0);

    for (int c0 = 0; c0 < len; c0 += C) {
        const int rows = min(C, len - c0);
        __syncthreads();  // previous chunk fully consumed (tiles and state)
        stash();
        __syncthreads();
        if (c0 + C < len) fetch(c0 + C);  // next chunk's loads fly during the compute below

        // ---- prologue: beta and chunk-local cumulative log decay -----------------------------
        for (int r = warp; r < C; r += NTHREADS / 32) {
            float s = 0.f, sq = 0.f;
            for (int d = lane; d < D; d += 32) {
                s += sm.K[r][d] * sm.K[r][d];
                sq += sm.Q[r][d] * sm.Q[r][d];
            }
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                s += __shfl_xor_sync(0xffffffffu, s, o);
                sq += __shfl_xor_sync(0xffffffffu, sq, o);
            }
            if (lane == 0) {
                // Eq. 3, or beta = eta (the gated-delta-rule coefficient) when asked for
                sm.beta[r] = (r < rows) ? ((p.variant & VARIANT_COEFF_ETA) ? sm.eta[r] : sm.eta[r] / (s + p.eps)) : 0.f;
                sm.qn[r] = (p.variant & VARIANT_QNORM) ? 1.f / sqrtf(sq) : 1.f;
            }
        }
        if (warp == 0) {
            // inclusive scan of C values, C/32 (or fewer) per lane
            constexpr int PER = (C + 31) / 32;
            double loc[PER];
            double run = 0.0;
#pragma unroll
            for (int u = 0; u < PER; ++u) {
                const int i = lane * PER + u;
                run += (i < C) ? (double)sm.la[i] : 0.0;
                loc[u] = run;
            }
            double incl = run;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const double t = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += t;
            }
            const double excl = incl - run;
#pragma unroll
            for (int u = 0; u < PER; ++u) {
                const int i = lane * PER + u;
                if (i < C) sm.g[i] = excl + loc[u];
            }
        }
        __syncthreads();

        // ---- L and P: 4x4 register tiles over the lower triangle -----------------------------
        if (tid < TD * TD) {
            const int ti = tid / TD, tj = tid % TD;
            if (tj <= ti) {
                float aG[4][4] = {}, aP[4][4] = {};
                for (int d = 0; d < D; d += 4) {
                    float4 ki[4], qi[4], kj[4];
#pragma unroll
                    for (int a = 0; a < 4; ++a) {
                        ki[a] = *reinterpret_cast<const float4 *>(&sm.K[4 * ti + a][d]);
                        qi[a] = *reinterpret_cast<const float4 *>(&sm.Q[4 * ti + a][d]);
                        kj[a] = *reinterpret_cast<const float4 *>(&sm.K[4 * tj + a][d]);
                    }
#pragma unroll
                    for (int a = 0; a < 4; ++a)
#pragma unroll
                        for (int b = 0; b < 4; ++b) {
                            aG[a][b] += ki[a].x * kj[b].x + ki[a].y * kj[b].y + ki[a].z * kj[b].z + ki[a].w * kj[b].w;
                            aP[a][b] += qi[a].x * kj[b].x + qi[a].y * kj[b].y + qi[a].z * kj[b].z + qi[a].w * kj[b].w;
                        }
                }
#pragma unroll
                for (int a = 0; a < 4; ++a)
#pragma unroll
                    for (int b = 0; b < 4; ++b) {
                        const int i = 4 * ti + a, j = 4 * tj + b;
                        const float ratio = (j <= i) ? expf((float)(sm.g[i] - sm.g[j])) : 0.f;
                        sm.L[i][j] = (j < i) ? sm.beta[i] * ratio * aG[a][b] : 0.f;
                        sm.P[i][j] = ratio * aP[a][b];
                    }
            }
        }

        // ---- K S_0 and Q S_0 (4x4 tiles), then rhs and the decayed state read-out -------------
        if (tid < 2 * TD * (NS / 4)) {
            const int which = tid / (TD * (NS / 4));
            const int ti = (tid % (TD * (NS / 4))) / (NS / 4), tc = tid % (NS / 4);
            float acc[4][4] = {};
            float (*Xs)[Smem::LDK] = which ? sm.Q : sm.K;
            for (int d = 0; d < D; d += 4) {
                float4 x[4], s[4];
#pragma unroll
                for (int a = 0; a < 4; ++a) {
                    x[a] = *reinterpret_cast<const float4 *>(&Xs[4 * ti + a][d]);
                    s[a] = *reinterpret_cast<const float4 *>(&sm.S[d + a][4 * tc]);
                }
#pragma unroll
                for (int a = 0; a < 4; ++a) {
                    acc[a][0] += x[a].x * s[0].x + x[a].y * s[1].x + x[a].z * s[2].x + x[a].w * s[3].x;
                    acc[a][1] += x[a].x * s[0].y + x[a].y * s[1].y + x[a].z * s[2].y + x[a].w * s[3].y;
                    acc[a][2] += x[a].x * s[0].z + x[a].y * s[1].z + x[a].z * s[2].z + x[a].w * s[3].z;
                    acc[a][3] += x[a].x * s[0].w + x[a].y * s[1].w + x[a].z * s[2].w + x[a].w * s[3].w;
                }
            }
#pragma unroll
            for (int a = 0; a < 4; ++a) {
                const int i = 4 * ti + a;
                const float gam = expf((float)sm.g[i]);
                if (which == 0) {
                    const float b = sm.beta[i];
                    const float4 vv = *reinterpret_cast<const float4 *>(&sm.V[i][4 * tc]);
                    *reinterpret_cast<float4 *>(&sm.X[i][4 * tc]) =
                        make_float4(b * (vv.x - gam * acc[a][0]), b * (vv.y - gam * acc[a][1]),
                                    b * (vv.z - gam * acc[a][2]), b * (vv.w - gam * acc[a][3]));
                } else {
                    *reinterpret_cast<float4 *>(&sm.O[i][4 * tc]) =
                        make_float4(gam * acc[a][0], gam * acc[a][1], gam * acc[a][2], gam * acc[a][3]);
                }
            }
        }
        __syncthreads();

        // ---- forward substitution (I + L) U = rhs; 8 lanes share one column -------------------
        {
            const int col = tid / 8, part = tid % 8;
            float xr[(C + 7) / 8];
#pragma unroll
            for (int u = 0; u < (C + 7) / 8; ++u) xr[u] = 0.f;
#pragma unroll
            for (int i = 0; i < C; ++i) {
                float s = 0.f;
#pragma unroll
                for (int u = 0; u < (i + 7) / 8; ++u) {
                    const int j = u * 8 + part;
                    if (j < i) s += sm.L[i][j] * xr[u];
                }
                s += __shfl_xor_sync(0xffffffffu, s, 1);
                s += __shfl_xor_sync(0xffffffffu, s, 2);
                s += __shfl_xor_sync(0xffffffffu, s, 4);
                const float xi = sm.X[i][col] - s;
                if ((i % 8) == part) xr[i / 8] = xi;
                if (part == 0) sm.X[i][col] = xi;
            }
        }
        __syncthreads();

        // ---- outputs: O_i = gamma_i (Q S_0)_i + sum_{j<=i} P_ij u_j ---------------------------
        {
            constexpr int RO = C / 32;  // rows per thread (2 for C = 64)
            const int tc = tid % 8, tr = tid / 8;
            if (RO > 0) {
                constexpr int ROe = RO > 0 ? RO : 1;
                float acc[ROe][4];
#pragma unroll
                for (int a = 0; a < ROe; ++a) {
                    const float4 o0 = *reinterpret_cast<const float4 *>(&sm.O[ROe * tr + a][4 * tc]);
                    acc[a][0] = o0.x; acc[a][1] = o0.y; acc[a][2] = o0.z; acc[a][3] = o0.w;
                }
                const int jmax = ROe * tr + ROe - 1;
                for (int j = 0; j <= jmax; ++j) {
                    const float4 u = *reinterpret_cast<const float4 *>(&sm.X[j][4 * tc]);
#pragma unroll
                    for (int a = 0; a < ROe; ++a) {
                        const int i = ROe * tr + a;
                        const float pij = (j <= i) ? sm.P[i][j] : 0.f;
                        acc[a][0] += pij * u.x; acc[a][1] += pij * u.y; acc[a][2] += pij * u.z; acc[a][3] += pij * u.w;
                    }
                }
#pragma unroll
                for (int a = 0; a < ROe; ++a) {
                    const int i = ROe * tr + a;
                    const float rn = sm.qn[i];
                    if (i < rows)
                        store4(og + (size_t)(tok0 + c0 + i) * HD + (size_t)h * D + sl * NS + 4 * tc,
                               make_float4(rn * acc[a][0], rn * acc[a][1], rn * acc[a][2], rn * acc[a][3]));
                }
            } else {
                // C = 16: 128 threads, one row x 4 columns each
                if (tr < C) {
                    const int i = tr;
                    const float4 o0 = *reinterpret_cast<const float4 *>(&sm.O[i][4 * tc]);
                    float a0 = o0.x, a1 = o0.y, a2 = o0.z, a3 = o0.w;
                    for (int j = 0; j <= i; ++j) {
                        const float4 u = *reinterpret_cast<const float4 *>(&sm.X[j][4 * tc]);
                        const float pij = sm.P[i][j];
                        a0 += pij * u.x; a1 += pij * u.y; a2 += pij * u.z; a3 += pij * u.w;
                    }
                    const float rn = sm.qn[i];
                    if (i < rows)
                        store4(og + (size_t)(tok0 + c0 + i) * HD + (size_t)h * D + sl * NS + 4 * tc,
                               make_float4(rn * a0, rn * a1, rn * a2, rn * a3));
                }
            }
        }

        // ---- state: S <- gamma_C S + K^T diag(exp(g_C - g_j)) U -------------------------------
        {
            const int tc = tid % 8, td = tid / 8;  // RD rows x 4 columns per thread
            const double gC = sm.g[C - 1];
            const float gamC = expf((float)gC);
            float acc[RD][4];
#pragma unroll
            for (int a = 0; a < RD; ++a) {
                const float4 s0 = *reinterpret_cast<const float4 *>(&sm.S[RD * td + a][4 * tc]);
                acc[a][0] = gamC * s0.x; acc[a][1] = gamC * s0.y; acc[a][2] = gamC * s0.z; acc[a][3] = gamC * s0.w;
            }
            for (int j = 0; j < C; ++j) {
                const float dj = expf((float)(gC - sm.g[j]));
                float4 u = *reinterpret_cast<const float4 *>(&sm.X[j][4 * tc]);
                u.x *= dj; u.y *= dj; u.z *= dj; u.w *= dj;
#pragma unroll
                for (int a = 0; a < RD; ++a) {
                    const float kv = sm.K[j][RD * td + a];
                    acc[a][0] += kv * u.x; acc[a][1] += kv * u.y; acc[a][2] += kv * u.z; acc[a][3] += kv * u.w;
                }
            }
            __syncthreads();  // everyone has finished reading S, X, K of this chunk
#pragma unroll
            for (int a = 0; a < RD; ++a)
                *reinterpret_cast<float4 *>(&sm.S[RD * td + a][4 * tc]) = make_float4(acc[a][0], acc[a][1], acc[a][2], acc[a][3]);
        }
    }

    __syncthreads();
    if (p.final_state) {
        for (int i = tid; i < D * NS / 4; i += NTHREADS) {
            const int r = i / (NS / 4), c4 = (i % (NS / 4)) * 4;
            *reinterpret_cast<float4 *>(p.final_state + (((size_t)n * p.H + h) * D + r) * D + sl * NS + c4) =
                *reinterpret_cast<const float4 *>(&sm.S[r][c4]);
        }
    }
}

template <int D, int C, typename IO, typename OUT>
cudaError_t launch_t(const ChunkParams &p, cudaStream_t stream)
{
    using Smem = SimtSmem<D, C>;
    auto kern = kla_chunk_simt_kernel<D, C, IO, OUT>;
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(Smem));
    if (err != cudaSuccess) return err;
    const int grid = p.n_seq * p.H * (D / NS);
    if (grid == 0) return cudaSuccess;
    kern<<<grid, NTHREADS, sizeof(Smem), stream>>>(p);
    count_launch(1);
    return cudaGetLastError();
}

template <int D, int C>
cudaError_t launch_dc(const ChunkParams &p, int io_dtype, int out_dtype, cudaStream_t stream)
{
    if (io_dtype == KLA_BF16) {
        if (out_dtype == KLA_BF16) return launch_t<D, C, __nv_bfloat16, __nv_bfloat16>(p, stream);
        return launch_t<D, C, __nv_bfloat16, float>(p, stream);
    }
    if (out_dtype == KLA_BF16) return launch_t<D, C, float, __nv_bfloat16>(p, stream);
    return launch_t<D, C, float, float>(p, stream);
}

}  // namespace

cudaError_t launch_chunk_simt(const ChunkParams &p, int d, int chunk, int io_dtype, int out_dtype, cudaStream_t stream)
{
    if (d == 128) {
        if (chunk == 64) return launch_dc<128, 64>(p, io_dtype, out_dtype, stream);
        if (chunk == 32) return launch_dc<128, 32>(p, io_dtype, out_dtype, stream);
        return launch_dc<128, 16>(p, io_dtype, out_dtype, stream);
    }
    if (chunk == 64) return launch_dc<64, 64>(p, io_dtype, out_dtype, stream);
    if (chunk == 32) return launch_dc<64, 32>(p, io_dtype, out_dtype, stream);
    return launch_dc<64, 16>(p, io_dtype, out_dtype, stream);
}

}  // namespace kla
