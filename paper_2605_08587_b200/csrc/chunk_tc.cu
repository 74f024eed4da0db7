// Chunkwise forward on the 5th-generation tensor cores (tcgen05.mma, TMEM accumulators, TMA-staged
// bf16 tiles) -- Algorithm 1, right panel; Eqs. 7-9.
//
// One CTA (128 threads) owns NS = 64 consecutive d_v columns of one (sequence, head) and walks that
// sequence's chunks (C = 64 tokens) in order.  Its d_k x NS slice of the state lives in registers in
// fp32 (thread r holds row r) and never leaves the SM between chunks.
//
// Per chunk, with g_i the chunk-local running sum of log alpha and gamma_i = exp(g_i):
//   MMA-1  [K;Q] K^T            -> G = K K^T (rows 0..63) and Q K^T (rows 64..127)
//   MMA-2  [K;Q] S_0            -> K S_0 and Q S_0
//          L = B (A^- o G), T = (I + L)^-1 by forward substitution (CUDA cores, fp32)
//          P = A o Q K^T,  rhs = B (V - D_gamma K S_0)                            (Eq. 7, right side)
//   MMA-3  [T_hi;T_lo] rhs      -> U = T rhs                                      (Eq. 7)
//   MMA-4  [P_hi;P_lo] U        -> O = D_gamma Q S_0 + P U                        (Eq. 8)
//   MMA-5  K^T (D U)            -> S <- gamma_C S_0 + K^T diag(exp(g_C - g_j)) U  (Eq. 9)
//
// Precision.  q, k, v are exact bf16 operands.  Every DERIVED operand (S_0, rhs, T, P, U, D U) is
// carried as a pair of bf16 values hi + lo (16 significand bits): a single bf16 rounding of any of
// them costs 1e-2..7e-2 in max|err|/rms on the layer-shaped workloads, far above the 2e-3 bound.
// Where the derived operand is the A matrix (T, P) the pair is stacked along M ([hi; lo], one M=128
// MMA whose two row halves are summed afterwards); where it is the B matrix the two halves are
// accumulated by two MMAs into the same TMEM columns.  All accumulation is fp32.
#include <cuda.h>

#include <mutex>

#include "common.cuh"
#include "umma.cuh"

namespace kla {

namespace {

using namespace umma;

constexpr int C = 64;    // chunk length
constexpr int NS = 64;   // state columns per CTA
constexpr int NT = 128;  // threads
constexpr long long WAIT_LIMIT = 2000000000LL;  // SM clocks (~1 s) before a wait gives up

// TMEM column offsets of the five accumulators (each 128 lanes x 64 fp32 columns)
constexpr uint32_t TM_D1 = 0, TM_D2 = 64, TM_D3 = 128, TM_D4 = 192, TM_D5 = 256, TM_COLS = 512;

template <int D>
struct TcSmem {
    static constexpr int KB = D / 64;             // 64-wide blocks along d_k
    static constexpr int KQ_BYTES = KB * 2 * 8192;  // [K kb0][Q kb0]([K kb1][Q kb1]), 8 KB each
    // all tile bases are multiples of 1024 bytes (128-byte swizzle atom = 8 rows x 128 B)
    alignas(1024) unsigned char kq[2][KQ_BYTES];
    alignas(1024) unsigned char v[2][8192];       // V slice, 64 tokens x 64 bf16
    alignas(1024) unsigned char s_hi[D * 128];    // state slice, D rows (d_k) x 64 bf16
    alignas(1024) unsigned char s_lo[D * 128];
    alignas(1024) unsigned char t[16384];         // [T_hi; T_lo], 128 rows x 64 bf16
    alignas(1024) unsigned char p[16384];         // [P_hi; P_lo]
    alignas(1024) unsigned char ru_hi[8192];      // rhs, later U: 64 tokens x 64 bf16
    alignas(1024) unsigned char ru_lo[8192];
    alignas(1024) unsigned char du_hi[8192];      // diag(exp(g_C - g_j)) U
    alignas(1024) unsigned char du_lo[8192];
    alignas(1024) float x[64 * 64];               // fp32 exchange buffer, 16-byte chunks swizzled
    float l[64][65];                              // strictly lower-triangular L for the solve
    float beta[64];
    float gam[64];                                // exp(g_i)
    float dec[64];                                // exp(g_C - g_i)
    double g[64];
    alignas(8) uint64_t bar_full[2];
    uint64_t bar_mma[5];
    uint32_t tmem_base;
    int abort_flag;
};

// chunk c (0..7) of row r in the fp32 exchange buffer (rows of 64 floats = 16 chunks of 16 B)
__device__ __forceinline__ float4 *xptr(float *x, int r, int c) { return reinterpret_cast<float4 *>(x + r * 64 + ((c ^ (r & 7)) << 2)); }

template <int D, typename OUT>
__global__ void __launch_bounds__(NT, 1)
kla_chunk_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, ChunkParams p)
{
    using Smem = TcSmem<D>;
    constexpr int KB = Smem::KB;
    constexpr int SLICES = D / NS;
    constexpr uint32_t STAGE_BYTES = Smem::KQ_BYTES + 8192;
    constexpr uint32_t ID_KK = idesc_bf16(128, 64, 0, 0);   // A K-major, B K-major
    constexpr uint32_t ID_KM = idesc_bf16(128, NS, 0, 1);   // A K-major, B MN-major
    constexpr uint32_t ID_MM = idesc_bf16(128, NS, 1, 1);   // A MN-major, B MN-major

    extern __shared__ unsigned char smem_dyn[];
    Smem &sm = *reinterpret_cast<Smem *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
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
    const size_t state_off = (((size_t)n * p.H + h) * D) * D + (size_t)sl * NS;

    // ---- state slice: thread r < D holds row r (64 fp32) ---------------------------------------------
    float S[NS];
    if (tid < D && p.init_state) {
#pragma unroll
        for (int c = 0; c < NS; c += 4) {
            const float4 x = *reinterpret_cast<const float4 *>(p.init_state + state_off + (size_t)tid * D + c);
            S[c] = x.x; S[c + 1] = x.y; S[c + 2] = x.z; S[c + 3] = x.w;
        }
    } else {
#pragma unroll
        for (int c = 0; c < NS; ++c) S[c] = 0.f;
    }
    if (len <= 0) {  // empty sequence: the final state is the initial state
        if (p.final_state && tid < D) {
#pragma unroll
            for (int c = 0; c < NS; c += 4)
                *reinterpret_cast<float4 *>(p.final_state + state_off + (size_t)tid * D + c) = make_float4(S[c], S[c + 1], S[c + 2], S[c + 3]);
        }
        return;
    }

    // ---- set-up: barriers, TMEM ----------------------------------------------------------------------
    if (tid == 0) {
        mbar_init(&sm.bar_full[0], 1);
        mbar_init(&sm.bar_full[1], 1);
        for (int i = 0; i < 5; ++i) mbar_init(&sm.bar_mma[i], 1);
        sm.abort_flag = 0;
        mbar_fence_init();
        tma_prefetch_desc(&tm_q);
        tma_prefetch_desc(&tm_k);
        tma_prefetch_desc(&tm_v);
    }
    if (warp == 0) tmem_alloc(&sm.tmem_base, TM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;
    const uint32_t tm_lane = tmem + ((uint32_t)(warp * 32) << 16);  // this warp's 32 TMEM lanes

    const int nchunks = (len + C - 1) / C;

    auto issue_tma = [&](int c) {  // thread 0 only
        const int st = c & 1;
        mbar_expect_tx(&sm.bar_full[st], STAGE_BYTES);
        const int row = tok0 + c * C;
#pragma unroll
        for (int kb = 0; kb < KB; ++kb) {
            tma_load_2d(sm.kq[st] + kb * 16384, &tm_k, h * D + kb * 64, row, &sm.bar_full[st]);
            tma_load_2d(sm.kq[st] + kb * 16384 + 8192, &tm_q, h * D + kb * 64, row, &sm.bar_full[st]);
        }
        tma_load_2d(sm.v[st], &tm_v, h * D + sl * NS, row, &sm.bar_full[st]);
    };

    // writes this thread's state row as the hi/lo B operand of MMA-2 (rows = d_k index, MN-major)
    auto store_state_tiles = [&]() {
        if (tid < D) {
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                uint4 hi, lo;
                split2(S[8 * c + 0], S[8 * c + 1], hi.x, lo.x);
                split2(S[8 * c + 2], S[8 * c + 3], hi.y, lo.y);
                split2(S[8 * c + 4], S[8 * c + 5], hi.z, lo.z);
                split2(S[8 * c + 6], S[8 * c + 7], hi.w, lo.w);
                *reinterpret_cast<uint4 *>(sm.s_hi + sw128(tid, c)) = hi;
                *reinterpret_cast<uint4 *>(sm.s_lo + sw128(tid, c)) = lo;
            }
        }
        fence_async_smem();
    };

    bool ok = true;
    // all threads wait on the barrier; the vote makes a timeout collective
#define KLA_WAIT_ALL(bar, parity)                                   \
    do {                                                            \
        bool w_ = mbar_wait((bar), (parity), WAIT_LIMIT);           \
        if (__syncthreads_or(!w_)) { ok = false; goto done; }       \
    } while (0)

    if (tid == 0) issue_tma(0);
    store_state_tiles();
    float la_next = 0.f, eta_next = 0.f;
    if (tid < C) {
        const bool valid = tid < len;
        la_next = valid ? p.log_alpha[(size_t)(tok0 + tid) * p.H + h] : 0.f;
        eta_next = valid ? p.eta[(size_t)(tok0 + tid) * p.H + h] : 0.f;
    }
    __syncthreads();

    for (int c = 0; c < nchunks; ++c) {
        const int st = c & 1;
        const uint32_t ph = (uint32_t)(c & 1);
        const int rows = min(C, len - c * C);
        const float la_cur = la_next, eta_cur = eta_next;

        if (tid == 0 && c + 1 < nchunks) issue_tma(c + 1);
        if (tid < C && c + 1 < nchunks) {
            const int t = (c + 1) * C + tid;
            const bool valid = t < len;
            la_next = valid ? p.log_alpha[(size_t)(tok0 + t) * p.H + h] : 0.f;
            eta_next = valid ? p.eta[(size_t)(tok0 + t) * p.H + h] : 0.f;
        }
        KLA_WAIT_ALL(&sm.bar_full[st], (uint32_t)((c >> 1) & 1));

        unsigned char *kq = sm.kq[st];
        unsigned char *vt = sm.v[st];
        if (rows < C) {
            // tail chunk: rows past the end of the sequence hold a neighbour's tokens (or TMA zero
            // fill); zero them so that they are inert in every product
            for (int i = tid; i < (C - rows) * 8; i += NT) {
                const int r = rows + i / 8, ch = i % 8;
                const uint4 z = make_uint4(0, 0, 0, 0);
#pragma unroll
                for (int kb = 0; kb < KB; ++kb) {
                    *reinterpret_cast<uint4 *>(kq + kb * 16384 + sw128(r, ch)) = z;
                    *reinterpret_cast<uint4 *>(kq + kb * 16384 + 8192 + sw128(r, ch)) = z;
                }
                *reinterpret_cast<uint4 *>(vt + sw128(r, ch)) = z;
            }
            fence_async_smem();
            __syncthreads();
        }

        // ---- MMA-1 and MMA-2 ----------------------------------------------------------------------------
        if (tid == 0) {
            tc_fence_after();
            const uint32_t a0 = smem_u32(kq);
#pragma unroll
            for (int s = 0; s < D / 16; ++s) {
                const uint32_t off = (uint32_t)((s / 4) * 16384 + (s % 4) * 32);
                mma_bf16_ss(tmem + TM_D1, smem_desc_sw128(a0 + off, 16, 1024), smem_desc_sw128(a0 + off, 16, 1024), ID_KK, s > 0);
            }
            mma_commit(&sm.bar_mma[0]);
            const uint32_t bh = smem_u32(sm.s_hi), bl = smem_u32(sm.s_lo);
#pragma unroll
            for (int s = 0; s < D / 16; ++s) {
                const uint32_t off = (uint32_t)((s / 4) * 16384 + (s % 4) * 32);
                mma_bf16_ss(tmem + TM_D2, smem_desc_sw128(a0 + off, 16, 1024), smem_desc_sw128(bh + s * 2048, 16, 1024), ID_KM, s > 0);
            }
#pragma unroll
            for (int s = 0; s < D / 16; ++s) {
                const uint32_t off = (uint32_t)((s / 4) * 16384 + (s % 4) * 32);
                mma_bf16_ss(tmem + TM_D2, smem_desc_sw128(a0 + off, 16, 1024), smem_desc_sw128(bl + s * 2048, 16, 1024), ID_KM, 1);
            }
            mma_commit(&sm.bar_mma[1]);
        }

        // ---- prologue (overlaps the MMAs): beta_i, g_i, gamma_i, exp(g_C - g_i) --------------------------
        if (tid < C) {
            float nk = 0.f;
#pragma unroll
            for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) {
                    const uint4 raw = *reinterpret_cast<const uint4 *>(kq + kb * 16384 + sw128(tid, ch));
                    const __nv_bfloat162 *h2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 f = __bfloat1622float2(h2[e]);
                        nk += f.x * f.x + f.y * f.y;
                    }
                }
            sm.beta[tid] = (tid < rows) ? eta_cur / (nk + p.eps) : 0.f;
            sm.dec[tid] = la_cur;  // staged for the scan below (overwritten with exp(g_C - g_i) afterwards)
        }
        __syncthreads();
        if (warp == 2) {
            // inclusive scan of the 64 log-decays in fp64 (differences g_i - g_j must not cancel)
            double v0 = (double)sm.dec[2 * lane], v1 = (double)sm.dec[2 * lane + 1];
            double run = v0 + v1, incl = run;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const double t = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= o) incl += t;
            }
            const double excl = incl - run;
            sm.g[2 * lane] = excl + v0;
            sm.g[2 * lane + 1] = excl + run;
        }
        __syncthreads();
        if (tid < C) {
            const double gC = sm.g[C - 1];
            sm.gam[tid] = __expf((float)sm.g[tid]);
            sm.dec[tid] = __expf((float)(gC - sm.g[tid]));
        }

        // ---- L (rows 0..63, warps 0-1) and P (rows 64..127, warps 2-3) from MMA-1 -------------------------
        KLA_WAIT_ALL(&sm.bar_mma[0], ph);
        tc_fence_after();
        {
            const int i = tid & 63;
            const double gi = sm.g[i];
            float acc[32];
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                tmem_ld32(tm_lane + TM_D1 + half * 32, acc);
                if (tid < 64) {
                    const float bi = sm.beta[i];
#pragma unroll
                    for (int jj = 0; jj < 32; ++jj) {
                        const int j = half * 32 + jj;
                        sm.l[i][j] = (j < i) ? bi * __expf((float)(gi - sm.g[j])) * acc[jj] : 0.f;
                    }
                } else {
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
                        float pv[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) {
                            const int j = half * 32 + ch * 8 + e;
                            pv[e] = (j <= i) ? __expf((float)(gi - sm.g[j])) * acc[ch * 8 + e] : 0.f;
                        }
                        uint4 hi, lo;
                        split2(pv[0], pv[1], hi.x, lo.x);
                        split2(pv[2], pv[3], hi.y, lo.y);
                        split2(pv[4], pv[5], hi.z, lo.z);
                        split2(pv[6], pv[7], hi.w, lo.w);
                        *reinterpret_cast<uint4 *>(sm.p + sw128(i, half * 4 + ch)) = hi;
                        *reinterpret_cast<uint4 *>(sm.p + sw128(64 + i, half * 4 + ch)) = lo;
                    }
                }
            }
        }
        __syncthreads();

        // ---- T = (I + L)^-1: column j by the thread pair (2j, 2j+1), rows split by parity -----------------
        {
            const int j = tid >> 1, par = tid & 1;
            float tc[32];  // T[m][j] for m = 2u + par
#pragma unroll
            for (int u = 0; u < 32; ++u) tc[u] = 0.f;
#pragma unroll
            for (int i = 0; i < 64; ++i) {
                float s = 0.f;
#pragma unroll
                for (int u = 0; u < (i + 1) / 2; ++u) {
                    const int m = 2 * u + par;
                    if (m < i) s += sm.l[i][m] * tc[u];
                }
                s += __shfl_xor_sync(0xffffffffu, s, 1);
                const float tij = (i == j) ? 1.f : ((i > j) ? -s : 0.f);
                if ((i & 1) == par) tc[i >> 1] = tij;
            }
            // write column j of [T_hi; T_lo] (K-major rows of 64 bf16)
#pragma unroll
            for (int u = 0; u < 32; ++u) {
                const int m = 2 * u + par;
                const __nv_bfloat16 hi = __float2bfloat16_rn(tc[u]);
                const __nv_bfloat16 lo = __float2bfloat16_rn(tc[u] - __bfloat162float(hi));
                *reinterpret_cast<__nv_bfloat16 *>(sm.t + sw128(m, j >> 3) + (j & 7) * 2) = hi;
                *reinterpret_cast<__nv_bfloat16 *>(sm.t + sw128(64 + m, j >> 3) + (j & 7) * 2) = lo;
            }
        }

        // ---- rhs = B (V - D_gamma K S_0) from MMA-2 (rows 0..63) --------------------------------------------
        KLA_WAIT_ALL(&sm.bar_mma[1], ph);
        tc_fence_after();
        if (tid < 64) {
            const int i = tid;
            const float bi = sm.beta[i], gi = sm.gam[i];
            float acc[32];
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                tmem_ld32(tm_lane + TM_D2 + half * 32, acc);
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    const uint4 raw = *reinterpret_cast<const uint4 *>(vt + sw128(i, half * 4 + ch));
                    const __nv_bfloat162 *h2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
                    float r[8];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float2 f = __bfloat1622float2(h2[e]);
                        r[2 * e] = bi * (f.x - gi * acc[ch * 8 + 2 * e]);
                        r[2 * e + 1] = bi * (f.y - gi * acc[ch * 8 + 2 * e + 1]);
                    }
                    uint4 hi, lo;
                    split2(r[0], r[1], hi.x, lo.x);
                    split2(r[2], r[3], hi.y, lo.y);
                    split2(r[4], r[5], hi.z, lo.z);
                    split2(r[6], r[7], hi.w, lo.w);
                    *reinterpret_cast<uint4 *>(sm.ru_hi + sw128(i, half * 4 + ch)) = hi;
                    *reinterpret_cast<uint4 *>(sm.ru_lo + sw128(i, half * 4 + ch)) = lo;
                }
            }
        }
        fence_async_smem();
        tc_fence_before();
        __syncthreads();

        // ---- MMA-3: [T_hi; T_lo] (rhs_hi + rhs_lo) ------------------------------------------------------------
        if (tid == 0) {
            tc_fence_after();
            const uint32_t a0 = smem_u32(sm.t), bh = smem_u32(sm.ru_hi), bl = smem_u32(sm.ru_lo);
#pragma unroll
            for (int s = 0; s < 4; ++s)
                mma_bf16_ss(tmem + TM_D3, smem_desc_sw128(a0 + s * 32, 16, 1024), smem_desc_sw128(bh + s * 2048, 16, 1024), ID_KM, s > 0);
#pragma unroll
            for (int s = 0; s < 4; ++s)
                mma_bf16_ss(tmem + TM_D3, smem_desc_sw128(a0 + s * 32, 16, 1024), smem_desc_sw128(bl + s * 2048, 16, 1024), ID_KM, 1);
            mma_commit(&sm.bar_mma[2]);
        }
        KLA_WAIT_ALL(&sm.bar_mma[2], ph);
        tc_fence_after();

        // ---- U = hi rows + lo rows; write U and D U as hi/lo B operands --------------------------------------------
        if (tid >= 64) {
            float acc[32];
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                tmem_ld32(tm_lane + TM_D3 + half * 32, acc);
#pragma unroll
                for (int ch = 0; ch < 8; ++ch)
                    *xptr(sm.x, tid - 64, half * 8 + ch) = make_float4(acc[4 * ch], acc[4 * ch + 1], acc[4 * ch + 2], acc[4 * ch + 3]);
            }
        }
        __syncthreads();
        if (tid < 64) {
            const int i = tid;
            const float di = sm.dec[i];
            float acc[32];
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                tmem_ld32(tm_lane + TM_D3 + half * 32, acc);
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) {
                    const float4 x = *xptr(sm.x, i, half * 8 + ch);
                    acc[4 * ch] += x.x; acc[4 * ch + 1] += x.y; acc[4 * ch + 2] += x.z; acc[4 * ch + 3] += x.w;
                }
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    uint4 hi, lo;
                    split2(acc[8 * ch + 0], acc[8 * ch + 1], hi.x, lo.x);
                    split2(acc[8 * ch + 2], acc[8 * ch + 3], hi.y, lo.y);
                    split2(acc[8 * ch + 4], acc[8 * ch + 5], hi.z, lo.z);
                    split2(acc[8 * ch + 6], acc[8 * ch + 7], hi.w, lo.w);
                    *reinterpret_cast<uint4 *>(sm.ru_hi + sw128(i, half * 4 + ch)) = hi;
                    *reinterpret_cast<uint4 *>(sm.ru_lo + sw128(i, half * 4 + ch)) = lo;
                    split2(di * acc[8 * ch + 0], di * acc[8 * ch + 1], hi.x, lo.x);
                    split2(di * acc[8 * ch + 2], di * acc[8 * ch + 3], hi.y, lo.y);
                    split2(di * acc[8 * ch + 4], di * acc[8 * ch + 5], hi.z, lo.z);
                    split2(di * acc[8 * ch + 6], di * acc[8 * ch + 7], hi.w, lo.w);
                    *reinterpret_cast<uint4 *>(sm.du_hi + sw128(i, half * 4 + ch)) = hi;
                    *reinterpret_cast<uint4 *>(sm.du_lo + sw128(i, half * 4 + ch)) = lo;
                }
            }
        }
        fence_async_smem();
        tc_fence_before();
        __syncthreads();

        // ---- MMA-4: [P_hi; P_lo] U  and  MMA-5: K^T (D U) -----------------------------------------------------------
        if (tid == 0) {
            tc_fence_after();
            const uint32_t a0 = smem_u32(sm.p), bh = smem_u32(sm.ru_hi), bl = smem_u32(sm.ru_lo);
#pragma unroll
            for (int s = 0; s < 4; ++s)
                mma_bf16_ss(tmem + TM_D4, smem_desc_sw128(a0 + s * 32, 16, 1024), smem_desc_sw128(bh + s * 2048, 16, 1024), ID_KM, s > 0);
#pragma unroll
            for (int s = 0; s < 4; ++s)
                mma_bf16_ss(tmem + TM_D4, smem_desc_sw128(a0 + s * 32, 16, 1024), smem_desc_sw128(bl + s * 2048, 16, 1024), ID_KM, 1);
            mma_commit(&sm.bar_mma[3]);
            // A = K^T: M = d_k (blocks of 64 KB*8192 bytes apart; for d_k = 64 the second block is the
            // Q tile, whose rows land in TMEM lanes 64..127 and are ignored), K = tokens
            const uint32_t k0 = smem_u32(kq), dh = smem_u32(sm.du_hi), dl = smem_u32(sm.du_lo);
#pragma unroll
            for (int s = 0; s < 4; ++s)
                mma_bf16_ss(tmem + TM_D5, smem_desc_sw128(k0 + s * 2048, KB * 8192, 1024), smem_desc_sw128(dh + s * 2048, 16, 1024), ID_MM, s > 0);
#pragma unroll
            for (int s = 0; s < 4; ++s)
                mma_bf16_ss(tmem + TM_D5, smem_desc_sw128(k0 + s * 2048, KB * 8192, 1024), smem_desc_sw128(dl + s * 2048, 16, 1024), ID_MM, 1);
            mma_commit(&sm.bar_mma[4]);
        }

        // ---- outputs: O_i = gamma_i (Q S_0)_i + (P_hi U)_i + (P_lo U)_i ----------------------------------------------
        KLA_WAIT_ALL(&sm.bar_mma[3], ph);
        tc_fence_after();
        if (tid < 64) {
            float acc[32];
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                tmem_ld32(tm_lane + TM_D4 + half * 32, acc);
#pragma unroll
                for (int ch = 0; ch < 8; ++ch)
                    *xptr(sm.x, tid, half * 8 + ch) = make_float4(acc[4 * ch], acc[4 * ch + 1], acc[4 * ch + 2], acc[4 * ch + 3]);
            }
        }
        __syncthreads();
        if (tid >= 64) {
            const int i = tid - 64;
            const float gi = sm.gam[i];
            OUT *orow = reinterpret_cast<OUT *>(p.out) + ((size_t)(tok0 + c * C + i) * p.H + h) * D + sl * NS;
            float acc[32], qs[32];
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                tmem_ld32(tm_lane + TM_D4 + half * 32, acc);
                tmem_ld32(tm_lane + TM_D2 + half * 32, qs);
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) {
                    const float4 x = *xptr(sm.x, i, half * 8 + ch);
                    float4 o;
                    o.x = gi * qs[4 * ch] + acc[4 * ch] + x.x;
                    o.y = gi * qs[4 * ch + 1] + acc[4 * ch + 1] + x.y;
                    o.z = gi * qs[4 * ch + 2] + acc[4 * ch + 2] + x.z;
                    o.w = gi * qs[4 * ch + 3] + acc[4 * ch + 3] + x.w;
                    if (i < rows) store4(orow + half * 32 + 4 * ch, o);
                }
            }
        }

        // ---- state: S <- gamma_C S + K^T (D U) ---------------------------------------------------------------------------
        KLA_WAIT_ALL(&sm.bar_mma[4], ph);
        tc_fence_after();
        if (tid < D) {
            const float gC = sm.gam[C - 1];
            float acc[32];
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                tmem_ld32(tm_lane + TM_D5 + half * 32, acc);
#pragma unroll
                for (int e = 0; e < 32; ++e) S[half * 32 + e] = gC * S[half * 32 + e] + acc[e];
            }
        }
        if (c + 1 < nchunks) store_state_tiles();
        tc_fence_before();
        __syncthreads();
    }

done:
    if (!ok && tid == 0 && p.status_word) atomicExch(p.status_word, (int)KLA_ERR_TIMEOUT);
    if (ok && p.final_state && tid < D) {
#pragma unroll
        for (int c = 0; c < NS; c += 4)
            *reinterpret_cast<float4 *>(p.final_state + state_off + (size_t)tid * D + c) = make_float4(S[c], S[c + 1], S[c + 2], S[c + 3]);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, TM_COLS);
    }
#undef KLA_WAIT_ALL
}

// ---- host side: tensor maps and launch ---------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    static std::once_flag once;
    std::call_once(once, [] {
        void *ptr = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(ptr);
    });
    return fn;
}

// 2-D view [rows = tokens][cols = H * d] of a bf16 [*, T, H, d] array; box = 64 tokens x 64 columns.
bool make_tmap(CUtensorMap *tm, const void *base, uint64_t n_tok, uint64_t row_elems)
{
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {row_elems, n_tok};
    cuuint64_t strides[1] = {row_elems * 2};
    cuuint32_t box[2] = {64, 64};
    cuuint32_t estr[2] = {1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, typename OUT>
cudaError_t launch_t(const ChunkParams &p, cudaStream_t stream)
{
    using Smem = TcSmem<D>;
    const uint64_t n_tok = (uint64_t)p.B * p.T;
    CUtensorMap tq, tk, tv;
    if (!make_tmap(&tq, p.q, n_tok, (uint64_t)p.H * D) || !make_tmap(&tk, p.k, n_tok, (uint64_t)p.H * D) ||
        !make_tmap(&tv, p.v, n_tok, (uint64_t)p.H * D))
        return cudaErrorInvalidValue;
    auto kern = kla_chunk_tc_kernel<D, OUT>;
    const int smem = (int)sizeof(Smem) + 1024;
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (err != cudaSuccess) return err;
    const int grid = p.n_seq * p.H * (D / NS);
    if (grid == 0) return cudaSuccess;
    kern<<<grid, NT, smem, stream>>>(tq, tk, tv, p);
    count_launch(1);
    return cudaGetLastError();
}

}  // namespace

bool chunk_tc_supported(int d, int chunk, int io_dtype)
{
    return (d == 64 || d == 128) && chunk == 64 && io_dtype == KLA_BF16;
}

cudaError_t launch_chunk_tc(const ChunkParams &p, int d, int io_dtype, int out_dtype, cudaStream_t stream)
{
    (void)io_dtype;
    if (d == 128) {
        if (out_dtype == KLA_BF16) return launch_t<128, __nv_bfloat16>(p, stream);
        return launch_t<128, float>(p, stream);
    }
    if (out_dtype == KLA_BF16) return launch_t<64, __nv_bfloat16>(p, stream);
    return launch_t<64, float>(p, stream);
}

}  // namespace kla
