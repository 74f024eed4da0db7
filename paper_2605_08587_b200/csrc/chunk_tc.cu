// Chunkwise forward on the 5th-generation tensor cores (tcgen05.mma, TMEM accumulators, TMA-staged
// bf16 tiles) -- Algorithm 1, right panel; Eqs. 7-9.
//
// One CTA owns NS = 64 consecutive d_v columns of one (sequence, head) and walks that sequence's
// chunks (C = 64 tokens) in order.  Its d_k x NS slice of the state stays in registers in fp32 for
// the whole sequence.  The CTA is warp-specialised (13 warps):
//
//   control warp (1 thread)  issues every TMA load and every tcgen05.mma, in a fixed order
//   pre group   (4 warps)    state-independent work for chunk c+1 while the chain works on chunk c:
//                            beta, g (Eq. 3, decay sums), L = B (A^- o K K^T), T = (I + L)^-1 by
//                            blocked forward substitution in shared memory, P = A o Q K^T
//   chain group (8 warps)    the serial dependency over chunks:
//                            rhs = B (V - D_gamma K S_0), U = T rhs                      (Eq. 7)
//                            O = D_gamma Q S_0 + P U                                     (Eq. 8)
//                            S <- gamma_C S_0 + K^T diag(exp(g_C - g_j)) U               (Eq. 9)
//
// Tensor-core products per chunk (fp32 accumulation in TMEM):
//   MMA-1  [K;Q] K^T   M=128   -> G (lanes 0..63) and Q K^T (lanes 64..127)
//   MMA-2  K S_0, Q S_0        two M=64 products, S_0 = S_hi + S_lo
//   MMA-3  T rhs       M=64    T_hi rhs_hi + T_hi rhs_lo + T_lo rhs_hi
//   MMA-4  P U         M=64    same three-term form
//   MMA-5  K^T (D U)   M=128   D U = hi + lo
//
// Precision.  q, k, v are exact bf16 operands.  Every DERIVED operand (S_0, rhs, T, P, U, D U) is
// carried as a pair of bf16 values hi + lo (16 significand bits): a single bf16 rounding of any of
// them costs 1e-2..7e-2 in max|err|/rms on the layer-shaped workloads, far above the 2e-3 bound.
//
// Every wait on an mbarrier is bounded; when one gives up the CTA raises an abort flag, reports
// KLA_ERR_TIMEOUT through the status word, releases its TMEM and exits.
#include <cuda.h>

#include <mutex>

#include "common.cuh"
#include "umma.cuh"

namespace kla {

namespace {

using namespace umma;

constexpr int C = 64;    // chunk length
constexpr int NS = 64;   // state columns per CTA
constexpr int PG_T = 128, CG_T = 256;
constexpr int NT = PG_T + CG_T + 32;
constexpr int NSTAGE = 3;
constexpr long long WAIT_LIMIT = 2000000000LL;  // SM clocks (~1 s) before a wait gives up

// TMEM columns (fp32, 128 lanes each)
constexpr uint32_t TM_D1 = 0, TM_KS = 64, TM_QS0 = 128, TM_QS1 = 192, TM_U = 256, TM_PU = 320, TM_DS = 384, TM_COLS = 512;

constexpr int LDT = 68;  // row stride (floats) of the fp32 solve matrix
constexpr int LDM = 36;  // row stride of the solve scratch

enum Bar {
    B_FULL0 = 0,             // +stage: TMA landed
    B_D1_DONE = 3,           // MMA-1(c) complete
    B_D1_FREE = 4,           // pre group finished reading D1(c)
    B_TP_READY = 5,          // T(c), P(c), scalars(c) written
    B_S_READY = 6,           // state tiles for chunk c written
    B_D2_DONE = 7,           // MMA-2(c) complete
    B_RHS_READY = 8,
    B_D3_DONE = 9,
    B_U_READY = 10,
    B_D5_DONE = 11,
    B_D4_DONE = 12,
    B_TAIL_READY = 13,       // masked rows of the last chunk zeroed
    B_COUNT = 14
};

template <int D>
struct TcSmem {
    static constexpr int KB = D / 64;               // 64-wide blocks along d_k
    static constexpr int KQ_BYTES = KB * 2 * 8192;  // [K kb0][Q kb0]([K kb1][Q kb1]), 8 KB each
    // all tile bases are multiples of 1024 bytes (128-byte swizzle atom = 8 rows x 128 B)
    alignas(1024) unsigned char kq[NSTAGE][KQ_BYTES];
    alignas(1024) unsigned char s_hi[D * 128];  // state slice, D rows (d_k) x 64 bf16
    alignas(1024) unsigned char s_lo[D * 128];
    alignas(1024) unsigned char t_hi[8192];     // 64 rows x 64 bf16, K-major
    alignas(1024) unsigned char t_lo[8192];
    alignas(1024) unsigned char p_hi[8192];
    alignas(1024) unsigned char p_lo[8192];
    alignas(1024) unsigned char ru_hi[8192];    // rhs, later U: 64 tokens x 64 bf16, MN-major
    alignas(1024) unsigned char ru_lo[8192];
    alignas(1024) unsigned char du_hi[8192];    // diag(exp(g_C - g_j)) U
    alignas(1024) unsigned char du_lo[8192];
    alignas(16) float tl[64 * LDT];             // L, overwritten in place by T = (I + L)^-1
    alignas(16) float mm[32 * LDM];             // scratch for the block products of the solve
    float beta[NSTAGE][64];
    float gam[NSTAGE][64];                      // exp(g_i)
    float dec[NSTAGE][64];                      // exp(g_C - g_i)
    float la[64];
    double g[64];
    alignas(8) uint64_t bar[B_COUNT];
    uint32_t tmem_base;
    volatile int abort_flag;
};

// ---- small fp32 block products on shared memory, used by the triangular solve ------------------------
// Cm[r][c] = sign * sum_{k = klo(c) .. khi(r)} A[r][k] * Bm[k][c]   for an R x 16*NC4/4.. tile set.
// Each calling thread owns ROWS x 4 outputs: rows r0.., columns c4..c4+3.
// b_lower: Bm is lower triangular (Bm[k][c] = 0 for k < c)  -> start k at c4
// a_lower: A  is lower triangular (A[r][k]  = 0 for k > r)  -> stop k at the tile's last row
template <int ROWS>
__device__ __forceinline__ void tile_mm(float *Cm, int ldc, const float *A, int lda, const float *Bm, int ldb, int r0,
                                        int c4, int K, bool b_lower, bool a_lower, float sign)
{
    float acc[ROWS][4];
#pragma unroll
    for (int a = 0; a < ROWS; ++a) acc[a][0] = acc[a][1] = acc[a][2] = acc[a][3] = 0.f;
    const int k0 = b_lower ? c4 : 0;
    const int k1 = a_lower ? min(K, r0 + ROWS) : K;
#pragma unroll 4
    for (int k = k0; k < k1; ++k) {
        const float4 b = *reinterpret_cast<const float4 *>(Bm + k * ldb + c4);
#pragma unroll
        for (int a = 0; a < ROWS; ++a) {
            const float x = A[(r0 + a) * lda + k];
            acc[a][0] += x * b.x; acc[a][1] += x * b.y; acc[a][2] += x * b.z; acc[a][3] += x * b.w;
        }
    }
#pragma unroll
    for (int a = 0; a < ROWS; ++a)
        *reinterpret_cast<float4 *>(Cm + (r0 + a) * ldc + c4) =
            make_float4(sign * acc[a][0], sign * acc[a][1], sign * acc[a][2], sign * acc[a][3]);
}

__device__ __forceinline__ void pg_sync() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
__device__ __forceinline__ void pg_half_sync() { asm volatile("bar.sync 2, 64;" ::: "memory"); }
// Barrier over the pre group that also ORs a flag: makes "some thread's wait gave up" a collective
// decision, so that no thread is left alone at a later pg_sync().
__device__ __forceinline__ bool pg_any(bool flag)
{
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %1, 0;\n\t"
        "bar.red.or.pred q, 3, 128, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)flag)
        : "memory");
    return r != 0;
}

template <int D, typename OUT>
__global__ void __launch_bounds__(NT, 1)
kla_chunk_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k, ChunkParams p)
{
    using Smem = TcSmem<D>;
    constexpr int KB = Smem::KB;
    constexpr int SLICES = D / NS;
    constexpr int KSTEPS = D / 16;
    constexpr uint32_t STAGE_BYTES = Smem::KQ_BYTES;
    constexpr uint32_t ID_G = idesc_bf16(128, 64, 0, 0);    // [K;Q] K^T : A K-major, B K-major
    constexpr uint32_t ID_S = idesc_bf16(64, NS, 0, 1);     // K S / Q S / T rhs / P U : M=64, B MN-major
    constexpr uint32_t ID_DS = idesc_bf16(128, NS, 1, 1);   // K^T (D U): A MN-major, B MN-major

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

    if (len <= 0) {  // empty sequence: the final state is the initial state
        if (p.final_state) {
            for (int i = tid; i < D * (NS / 4); i += NT) {
                const int r = i / (NS / 4), c = (i % (NS / 4)) * 4;
                float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
                if (p.init_state) x = *reinterpret_cast<const float4 *>(p.init_state + state_off + (size_t)r * D + c);
                *reinterpret_cast<float4 *>(p.final_state + state_off + (size_t)r * D + c) = x;
            }
        }
        return;
    }
    const int nchunks = (len + C - 1) / C;
    const int last_rows = len - (nchunks - 1) * C;

    // ---- set-up ------------------------------------------------------------------------------------------
    if (tid == 0) {
        for (int s = 0; s < NSTAGE; ++s) mbar_init(&sm.bar[B_FULL0 + s], 1);
        mbar_init(&sm.bar[B_D1_DONE], 1);
        mbar_init(&sm.bar[B_D1_FREE], PG_T / 32);
        mbar_init(&sm.bar[B_TP_READY], PG_T / 32);
        mbar_init(&sm.bar[B_S_READY], CG_T / 32);
        mbar_init(&sm.bar[B_D2_DONE], 1);
        mbar_init(&sm.bar[B_RHS_READY], CG_T / 32);
        mbar_init(&sm.bar[B_D3_DONE], 1);
        mbar_init(&sm.bar[B_U_READY], CG_T / 32);
        mbar_init(&sm.bar[B_D5_DONE], 1);
        mbar_init(&sm.bar[B_D4_DONE], 1);
        mbar_init(&sm.bar[B_TAIL_READY], PG_T / 32);
        sm.abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 0) tmem_alloc(&sm.tmem_base, TM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;
    const uint32_t tm_lane = tmem + ((uint32_t)((warp & 3) * 32) << 16);  // this warp's 32 TMEM lanes

    // Bounded wait that also leaves when another role has aborted.
    auto wait = [&](int b, uint32_t parity) -> bool {
        uint64_t *bar = &sm.bar[b];
        if (mbar_try_wait(bar, parity)) return true;
        const long long t0 = clock64();
        while (true) {
#pragma unroll 1
            for (int i = 0; i < 32; ++i)
                if (mbar_try_wait(bar, parity)) return true;
            if (sm.abort_flag) return false;
            if (clock64() - t0 > WAIT_LIMIT) {
                sm.abort_flag = 1;
                return false;
            }
        }
    };
    // one arrival per warp, after the warp's shared-memory writes are visible to the async proxy
    auto warp_arrive = [&](int b) {
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.bar[b]);
    };

    if (warp == NT / 32 - 1) {
        // =============================== control warp =====================================================
        if (lane == 0) {
            tma_prefetch_desc(&tm_q);
            tma_prefetch_desc(&tm_k);
            auto issue_tma = [&](int c) {
                const int st = c % NSTAGE;
                mbar_expect_tx(&sm.bar[B_FULL0 + st], STAGE_BYTES);
                const int row = tok0 + c * C;
#pragma unroll
                for (int kb = 0; kb < KB; ++kb) {
                    tma_load_2d(sm.kq[st] + kb * 16384, &tm_k, h * D + kb * 64, row, &sm.bar[B_FULL0 + st]);
                    tma_load_2d(sm.kq[st] + kb * 16384 + 8192, &tm_q, h * D + kb * 64, row, &sm.bar[B_FULL0 + st]);
                }
            };
            auto mma1 = [&](int c) {  // [K;Q] K^T -> D1
                const uint32_t a0 = smem_u32(sm.kq[c % NSTAGE]);
#pragma unroll
                for (int s = 0; s < KSTEPS; ++s) {
                    const uint32_t off = (uint32_t)((s / 4) * 16384 + (s % 4) * 32);
                    mma_bf16_ss(tmem + TM_D1, smem_desc_sw128(a0 + off, 16, 1024), smem_desc_sw128(a0 + off, 16, 1024), ID_G, s > 0);
                }
                mma_commit(&sm.bar[B_D1_DONE]);
            };
            bool ok = true;
            for (int c = 0; c < NSTAGE && c < nchunks; ++c) issue_tma(c);
            // MMA-1(0)
            ok = wait(B_FULL0, 0);
            if (ok && nchunks == 1 && last_rows < C) ok = wait(B_TAIL_READY, 0);
            if (ok) {
                tc_fence_after();
                mma1(0);
            }
            for (int c = 0; ok && c < nchunks; ++c) {
                const uint32_t ph = (uint32_t)(c & 1);
                const uint32_t k0 = smem_u32(sm.kq[c % NSTAGE]);
                // MMA-1(c+1): as early as its inputs and the D1 buffer allow
                if (c + 1 < nchunks) {
                    if (!(ok = wait(B_FULL0 + (c + 1) % NSTAGE, (uint32_t)(((c + 1) / NSTAGE) & 1)))) break;
                    if (c + 2 == nchunks && last_rows < C)
                        if (!(ok = wait(B_TAIL_READY, 0))) break;
                    if (!(ok = wait(B_D1_FREE, ph))) break;
                    tc_fence_after();
                    mma1(c + 1);
                }
                // MMA-2(c): K S_0 -> TM_KS, Q S_0 -> TM_QS[c&1]
                if (!(ok = wait(B_S_READY, ph))) break;
                tc_fence_after();
                {
                    const uint32_t bh = smem_u32(sm.s_hi), bl = smem_u32(sm.s_lo);
                    const uint32_t tq = tmem + ((c & 1) ? TM_QS1 : TM_QS0);
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        const uint32_t b0 = half ? bl : bh;
#pragma unroll
                        for (int s = 0; s < KSTEPS; ++s) {
                            const uint32_t off = (uint32_t)((s / 4) * 16384 + (s % 4) * 32);
                            mma_bf16_ss(tmem + TM_KS, smem_desc_sw128(k0 + off, 16, 1024), smem_desc_sw128(b0 + s * 2048, 16, 1024), ID_S, (half | s) > 0);
                        }
                    }
#pragma unroll
                    for (int half = 0; half < 2; ++half) {
                        const uint32_t b0 = half ? bl : bh;
#pragma unroll
                        for (int s = 0; s < KSTEPS; ++s) {
                            const uint32_t off = (uint32_t)((s / 4) * 16384 + (s % 4) * 32 + 8192);
                            mma_bf16_ss(tq, smem_desc_sw128(k0 + off, 16, 1024), smem_desc_sw128(b0 + s * 2048, 16, 1024), ID_S, (half | s) > 0);
                        }
                    }
                    mma_commit(&sm.bar[B_D2_DONE]);
                }
                // MMA-3(c): U = T rhs
                if (!(ok = wait(B_TP_READY, ph))) break;
                if (!(ok = wait(B_RHS_READY, ph))) break;
                tc_fence_after();
                {
                    const uint32_t th = smem_u32(sm.t_hi), tl = smem_u32(sm.t_lo), rh = smem_u32(sm.ru_hi), rl = smem_u32(sm.ru_lo);
#pragma unroll
                    for (int s = 0; s < 4; ++s)
                        mma_bf16_ss(tmem + TM_U, smem_desc_sw128(th + s * 32, 16, 1024), smem_desc_sw128(rh + s * 2048, 16, 1024), ID_S, s > 0);
#pragma unroll
                    for (int s = 0; s < 4; ++s)
                        mma_bf16_ss(tmem + TM_U, smem_desc_sw128(th + s * 32, 16, 1024), smem_desc_sw128(rl + s * 2048, 16, 1024), ID_S, 1);
#pragma unroll
                    for (int s = 0; s < 4; ++s)
                        mma_bf16_ss(tmem + TM_U, smem_desc_sw128(tl + s * 32, 16, 1024), smem_desc_sw128(rh + s * 2048, 16, 1024), ID_S, 1);
                    mma_commit(&sm.bar[B_D3_DONE]);
                }
                // MMA-5(c): K^T (D U)   then   MMA-4(c): P U
                if (!(ok = wait(B_U_READY, ph))) break;
                tc_fence_after();
                {
                    const uint32_t dh = smem_u32(sm.du_hi), dl = smem_u32(sm.du_lo);
                    // A = K^T: M = d_k (64-wide blocks KB*8192 bytes apart; for d_k = 64 the second block
                    // is the Q tile, whose rows land in TMEM lanes 64..127 and are ignored), K = tokens
#pragma unroll
                    for (int s = 0; s < 4; ++s)
                        mma_bf16_ss(tmem + TM_DS, smem_desc_sw128(k0 + s * 2048, KB * 8192, 1024), smem_desc_sw128(dh + s * 2048, 16, 1024), ID_DS, s > 0);
#pragma unroll
                    for (int s = 0; s < 4; ++s)
                        mma_bf16_ss(tmem + TM_DS, smem_desc_sw128(k0 + s * 2048, KB * 8192, 1024), smem_desc_sw128(dl + s * 2048, 16, 1024), ID_DS, 1);
                    mma_commit(&sm.bar[B_D5_DONE]);
                    const uint32_t phh = smem_u32(sm.p_hi), pl = smem_u32(sm.p_lo), uh = smem_u32(sm.ru_hi), ul = smem_u32(sm.ru_lo);
#pragma unroll
                    for (int s = 0; s < 4; ++s)
                        mma_bf16_ss(tmem + TM_PU, smem_desc_sw128(phh + s * 32, 16, 1024), smem_desc_sw128(uh + s * 2048, 16, 1024), ID_S, s > 0);
#pragma unroll
                    for (int s = 0; s < 4; ++s)
                        mma_bf16_ss(tmem + TM_PU, smem_desc_sw128(phh + s * 32, 16, 1024), smem_desc_sw128(ul + s * 2048, 16, 1024), ID_S, 1);
#pragma unroll
                    for (int s = 0; s < 4; ++s)
                        mma_bf16_ss(tmem + TM_PU, smem_desc_sw128(pl + s * 32, 16, 1024), smem_desc_sw128(uh + s * 2048, 16, 1024), ID_S, 1);
                    mma_commit(&sm.bar[B_D4_DONE]);
                }
                // the K/Q stage of chunk c is free once MMA-5(c) has read it
                if (c + NSTAGE < nchunks) {
                    if (!(ok = wait(B_D5_DONE, ph))) break;
                    issue_tma(c + NSTAGE);
                }
            }
        }
    } else if (warp < PG_T / 32) {
        // =============================== pre group ==========================================================
        const int pt = tid;  // 0..127
        float la_next = 0.f, eta_next = 0.f;
        if (pt < C) {
            const bool valid = pt < len;
            la_next = valid ? p.log_alpha[(size_t)(tok0 + pt) * p.H + h] : 0.f;
            eta_next = valid ? p.eta[(size_t)(tok0 + pt) * p.H + h] : 0.f;
        }
        for (int c = 0; c < nchunks; ++c) {
            const uint32_t ph = (uint32_t)(c & 1);
            const int rows = (c == nchunks - 1) ? last_rows : C;
            const int sc = c % NSTAGE;
            const float la_cur = la_next, eta_cur = eta_next;
            if (pt < C && c + 1 < nchunks) {
                const int t = (c + 1) * C + pt;
                const bool valid = t < len;
                la_next = valid ? p.log_alpha[(size_t)(tok0 + t) * p.H + h] : 0.f;
                eta_next = valid ? p.eta[(size_t)(tok0 + t) * p.H + h] : 0.f;
            }
            if (pg_any(!wait(B_FULL0 + sc, (uint32_t)((c / NSTAGE) & 1)))) break;
            unsigned char *kq = sm.kq[sc];
            if (rows < C) {
                // last chunk: rows past the end of the sequence hold a neighbour's tokens (or TMA zero
                // fill); zero them so that they are inert in every product
                for (int i = pt; i < (C - rows) * 8; i += PG_T) {
                    const int r = rows + i / 8, ch = i % 8;
                    const uint4 z = make_uint4(0, 0, 0, 0);
#pragma unroll
                    for (int kb = 0; kb < KB; ++kb) {
                        *reinterpret_cast<uint4 *>(kq + kb * 16384 + sw128(r, ch)) = z;
                        *reinterpret_cast<uint4 *>(kq + kb * 16384 + 8192 + sw128(r, ch)) = z;
                    }
                }
                fence_async_smem();
                warp_arrive(B_TAIL_READY);
            }
            // ---- beta_i, g_i, gamma_i, exp(g_C - g_i) ------------------------------------------------------
            if (pt < C) {
                float nk = 0.f;
                if (pt < rows) {
#pragma unroll
                    for (int kb = 0; kb < KB; ++kb)
#pragma unroll
                        for (int ch = 0; ch < 8; ++ch) {
                            const uint4 raw = *reinterpret_cast<const uint4 *>(kq + kb * 16384 + sw128(pt, ch));
                            const __nv_bfloat162 *h2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float2 f = __bfloat1622float2(h2[e]);
                                nk += f.x * f.x + f.y * f.y;
                            }
                        }
                }
                sm.beta[sc][pt] = (pt < rows) ? eta_cur / (nk + p.eps) : 0.f;
                sm.la[pt] = la_cur;
            }
            pg_sync();
            if (warp == 2) {
                // inclusive scan of the 64 log-decays in fp64 (differences g_i - g_j must not cancel)
                const double v0 = (double)sm.la[2 * lane], v1 = (double)sm.la[2 * lane + 1];
                const double run = v0 + v1;
                double incl = run;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const double t = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += t;
                }
                const double excl = incl - run;
                sm.g[2 * lane] = excl + v0;
                sm.g[2 * lane + 1] = excl + run;
            }
            pg_sync();
            if (pt < C) {
                const double gC = sm.g[C - 1];
                sm.gam[sc][pt] = __expf((float)sm.g[pt]);
                sm.dec[sc][pt] = __expf((float)(gC - sm.g[pt]));
            }
            // ---- L (lanes 0..63) and P (lanes 64..127) from MMA-1 -------------------------------------------
            if (pg_any(!wait(B_D1_DONE, ph))) break;
            tc_fence_after();
            uint32_t p_hi[32], p_lo[32];  // this thread's P row, packed bf16 pairs (warps 2, 3 only)
            {
                const int i = pt & 63;
                const double gi = sm.g[i];
                const float bi = sm.beta[sc][i];
                float acc[32];
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    tmem_ld32(tm_lane + TM_D1 + half * 32, acc);
                    if (pt < 64) {
#pragma unroll
                        for (int q4 = 0; q4 < 8; ++q4) {
                            float4 o;
                            float *of = reinterpret_cast<float *>(&o);
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const int j = half * 32 + q4 * 4 + e;
                                of[e] = (j < i) ? bi * __expf((float)(gi - sm.g[j])) * acc[q4 * 4 + e] : 0.f;
                            }
                            *reinterpret_cast<float4 *>(&sm.tl[i * LDT + half * 32 + q4 * 4]) = o;
                        }
                    } else {
#pragma unroll
                        for (int e2 = 0; e2 < 16; ++e2) {
                            const int j = half * 32 + 2 * e2;
                            const float a = (j <= i) ? __expf((float)(gi - sm.g[j])) * acc[2 * e2] : 0.f;
                            const float b = (j + 1 <= i) ? __expf((float)(gi - sm.g[j + 1])) * acc[2 * e2 + 1] : 0.f;
                            split2(a, b, p_hi[half * 16 + e2], p_lo[half * 16 + e2]);
                        }
                    }
                }
            }
            tc_fence_before();
            warp_arrive(B_D1_FREE);

            // ---- T = (I + L)^-1, blocked: 16x16 diagonal blocks, then 16x16 and 32x32 off-diagonal blocks ------
            if (pt < 64) {
                pg_half_sync();  // L rows written by warps 0, 1
                const int blk = pt >> 4, j = pt & 15;
                const float *Lb = sm.tl + (blk * 16) * LDT + blk * 16;
                float x[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    float s0 = 0.f, s1 = 0.f;
#pragma unroll
                    for (int m = 0; m < i; m += 2) {
                        s0 += Lb[i * LDT + m] * x[m];
                        if (m + 1 < i) s1 += Lb[i * LDT + m + 1] * x[m + 1];
                    }
                    x[i] = (i == j) ? 1.f : ((i > j) ? -(s0 + s1) : 0.f);
                }
                pg_half_sync();  // every column of the block has read L_bb
                float *Tb = sm.tl + (blk * 16) * LDT + blk * 16;
#pragma unroll
                for (int i = 0; i < 16; ++i) Tb[i * LDT + j] = x[i];
            }
            pg_sync();
            {
                // level 1: M = L10 T00 and L32 T22 (16x16 each); then T10 = -T11 M, T32 = -T33 M
                const int prod = pt >> 6, r = (pt & 63) >> 2, c4 = (pt & 3) * 4;
                const int rb = prod ? 48 : 16, cb = prod ? 32 : 0;
                tile_mm<1>(sm.mm + prod * 16 * LDM, LDM, sm.tl + rb * LDT + cb, LDT, sm.tl + cb * LDT + cb, LDT, r, c4, 16, true, false, 1.f);
                pg_sync();
                tile_mm<1>(sm.tl + rb * LDT + cb, LDT, sm.tl + rb * LDT + rb, LDT, sm.mm + prod * 16 * LDM, LDM, r, c4, 16, false, true, -1.f);
                pg_sync();
            }
            {
                // level 2: M = L[32..63][0..31] T[0..31][0..31]; T[32..63][0..31] = -T[32..63][32..63] M
                const int r0 = (pt >> 3) * 2, c4 = (pt & 7) * 4;
                tile_mm<2>(sm.mm, LDM, sm.tl + 32 * LDT, LDT, sm.tl, LDT, r0, c4, 32, true, false, 1.f);
                pg_sync();
                tile_mm<2>(sm.tl + 32 * LDT, LDT, sm.tl + 32 * LDT + 32, LDT, sm.mm, LDM, r0, c4, 32, false, true, -1.f);
                pg_sync();
            }
            // ---- write T (after MMA-3(c-1) has read the previous one) and P (after MMA-4(c-1)) ----------------------
            if (c > 0 && pg_any(!wait(B_D3_DONE, ph ^ 1))) break;
            {
                const int i = pt >> 1, half = pt & 1;
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    const float4 a = *reinterpret_cast<const float4 *>(&sm.tl[i * LDT + half * 32 + ch * 8]);
                    const float4 b = *reinterpret_cast<const float4 *>(&sm.tl[i * LDT + half * 32 + ch * 8 + 4]);
                    uint4 hi, lo;
                    split2(a.x, a.y, hi.x, lo.x);
                    split2(a.z, a.w, hi.y, lo.y);
                    split2(b.x, b.y, hi.z, lo.z);
                    split2(b.z, b.w, hi.w, lo.w);
                    *reinterpret_cast<uint4 *>(sm.t_hi + sw128(i, half * 4 + ch)) = hi;
                    *reinterpret_cast<uint4 *>(sm.t_lo + sw128(i, half * 4 + ch)) = lo;
                }
            }
            if (c > 0 && pg_any(!wait(B_D4_DONE, ph ^ 1))) break;
            if (pt >= 64) {
                const int i = pt - 64;
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) {
                    *reinterpret_cast<uint4 *>(sm.p_hi + sw128(i, ch)) = make_uint4(p_hi[4 * ch], p_hi[4 * ch + 1], p_hi[4 * ch + 2], p_hi[4 * ch + 3]);
                    *reinterpret_cast<uint4 *>(sm.p_lo + sw128(i, ch)) = make_uint4(p_lo[4 * ch], p_lo[4 * ch + 1], p_lo[4 * ch + 2], p_lo[4 * ch + 3]);
                }
            }
            fence_async_smem();
            pg_sync();  // the solve matrix is reused by the next chunk
            warp_arrive(B_TP_READY);
        }
    } else {
        // =============================== chain group ==========================================================
        const int ct = tid - PG_T;              // 0..255
        const int q = warp & 3;                 // TMEM lane quadrant
        const int hf = ct >> 7;                 // column half: 0 -> columns 0..31, 1 -> 32..63
        const int srow = q * 32 + lane;         // state row (M = 128 accumulator layout)
        const bool s_act = srow < D;
        const int i = q * 16 + lane;            // chunk row (M = 64 accumulator layout); valid for lane < 16
        const bool r_act = lane < 16;

        float S[32];
        if (s_act && p.init_state) {
#pragma unroll
            for (int c = 0; c < 32; c += 4) {
                const float4 x = *reinterpret_cast<const float4 *>(p.init_state + state_off + (size_t)srow * D + hf * 32 + c);
                S[c] = x.x; S[c + 1] = x.y; S[c + 2] = x.z; S[c + 3] = x.w;
            }
        } else {
#pragma unroll
            for (int c = 0; c < 32; ++c) S[c] = 0.f;
        }
        auto store_state_tiles = [&]() {
            if (s_act) {
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    uint4 hi, lo;
                    split2(S[8 * c + 0], S[8 * c + 1], hi.x, lo.x);
                    split2(S[8 * c + 2], S[8 * c + 3], hi.y, lo.y);
                    split2(S[8 * c + 4], S[8 * c + 5], hi.z, lo.z);
                    split2(S[8 * c + 6], S[8 * c + 7], hi.w, lo.w);
                    *reinterpret_cast<uint4 *>(sm.s_hi + sw128(srow, hf * 4 + c)) = hi;
                    *reinterpret_cast<uint4 *>(sm.s_lo + sw128(srow, hf * 4 + c)) = lo;
                }
            }
            fence_async_smem();
            warp_arrive(B_S_READY);
        };
        const __nv_bfloat16 *vbase = reinterpret_cast<const __nv_bfloat16 *>(p.v) + (size_t)h * D + sl * NS + hf * 32;
        const size_t tokstride = (size_t)p.H * D;
        uint4 vreg[4];
        auto fetch_v = [&](int c) {
            const int t = c * C + i;
            if (r_act && t < len) {
                const uint4 *src = reinterpret_cast<const uint4 *>(vbase + (size_t)(tok0 + t) * tokstride);
#pragma unroll
                for (int u = 0; u < 4; ++u) vreg[u] = src[u];
            } else {
#pragma unroll
                for (int u = 0; u < 4; ++u) vreg[u] = make_uint4(0, 0, 0, 0);
            }
        };
        fetch_v(0);
        store_state_tiles();

        for (int c = 0; c < nchunks; ++c) {
            const uint32_t ph = (uint32_t)(c & 1);
            const int rows = (c == nchunks - 1) ? last_rows : C;
            const int sc = c % NSTAGE;
            // ---- rhs = B (V - D_gamma K S_0) ------------------------------------------------------------------
            if (!wait(B_TP_READY, ph)) break;   // scalars of chunk c
            if (!wait(B_D2_DONE, ph)) break;
            tc_fence_after();
            float bi = 0.f, gi = 0.f, di = 0.f;
            if (r_act) {
                bi = sm.beta[sc][i];
                gi = sm.gam[sc][i];
                di = sm.dec[sc][i];
            }
            const float gC = sm.gam[sc][C - 1];
            {
                float acc[32];
                tmem_ld32(tm_lane + TM_KS + hf * 32, acc);
                if (r_act) {
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
                        const __nv_bfloat162 *h2 = reinterpret_cast<const __nv_bfloat162 *>(&vreg[ch]);
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
                        *reinterpret_cast<uint4 *>(sm.ru_hi + sw128(i, hf * 4 + ch)) = hi;
                        *reinterpret_cast<uint4 *>(sm.ru_lo + sw128(i, hf * 4 + ch)) = lo;
                    }
                }
            }
            fence_async_smem();
            tc_fence_before();
            warp_arrive(B_RHS_READY);
            if (c + 1 < nchunks) fetch_v(c + 1);

            // ---- U and D U as hi/lo operands -------------------------------------------------------------------
            if (!wait(B_D3_DONE, ph)) break;
            tc_fence_after();
            {
                float acc[32];
                tmem_ld32(tm_lane + TM_U + hf * 32, acc);
                if (r_act) {
#pragma unroll
                    for (int ch = 0; ch < 4; ++ch) {
                        uint4 hi, lo;
                        split2(acc[8 * ch + 0], acc[8 * ch + 1], hi.x, lo.x);
                        split2(acc[8 * ch + 2], acc[8 * ch + 3], hi.y, lo.y);
                        split2(acc[8 * ch + 4], acc[8 * ch + 5], hi.z, lo.z);
                        split2(acc[8 * ch + 6], acc[8 * ch + 7], hi.w, lo.w);
                        *reinterpret_cast<uint4 *>(sm.ru_hi + sw128(i, hf * 4 + ch)) = hi;
                        *reinterpret_cast<uint4 *>(sm.ru_lo + sw128(i, hf * 4 + ch)) = lo;
                        split2(di * acc[8 * ch + 0], di * acc[8 * ch + 1], hi.x, lo.x);
                        split2(di * acc[8 * ch + 2], di * acc[8 * ch + 3], hi.y, lo.y);
                        split2(di * acc[8 * ch + 4], di * acc[8 * ch + 5], hi.z, lo.z);
                        split2(di * acc[8 * ch + 6], di * acc[8 * ch + 7], hi.w, lo.w);
                        *reinterpret_cast<uint4 *>(sm.du_hi + sw128(i, hf * 4 + ch)) = hi;
                        *reinterpret_cast<uint4 *>(sm.du_lo + sw128(i, hf * 4 + ch)) = lo;
                    }
                }
            }
            fence_async_smem();
            tc_fence_before();
            warp_arrive(B_U_READY);

            // ---- state: S <- gamma_C S + K^T (D U) -----------------------------------------------------------------
            if (!wait(B_D5_DONE, ph)) break;
            tc_fence_after();
            {
                float acc[32];
                tmem_ld32(tm_lane + TM_DS + hf * 32, acc);
                if (s_act) {
#pragma unroll
                    for (int e = 0; e < 32; ++e) S[e] = gC * S[e] + acc[e];
                }
            }
            tc_fence_before();
            if (c + 1 < nchunks) store_state_tiles();

            // ---- outputs: O_i = gamma_i (Q S_0)_i + (P U)_i (off the chain) -----------------------------------------
            if (!wait(B_D4_DONE, ph)) break;
            tc_fence_after();
            {
                float acc[32], qs[32];
                tmem_ld32(tm_lane + TM_PU + hf * 32, acc);
                tmem_ld32(tm_lane + ((c & 1) ? TM_QS1 : TM_QS0) + hf * 32, qs);
                if (r_act && i < rows) {
                    OUT *orow = reinterpret_cast<OUT *>(p.out) + ((size_t)(tok0 + c * C + i) * p.H + h) * D + sl * NS + hf * 32;
#pragma unroll
                    for (int e = 0; e < 32; e += 4)
                        store4(orow + e, make_float4(gi * qs[e] + acc[e], gi * qs[e + 1] + acc[e + 1],
                                                     gi * qs[e + 2] + acc[e + 2], gi * qs[e + 3] + acc[e + 3]));
                }
            }
            tc_fence_before();
        }
        if (!sm.abort_flag && p.final_state && s_act) {
#pragma unroll
            for (int c = 0; c < 32; c += 4)
                *reinterpret_cast<float4 *>(p.final_state + state_off + (size_t)srow * D + hf * 32 + c) =
                    make_float4(S[c], S[c + 1], S[c + 2], S[c + 3]);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem, TM_COLS);
    }
    if (tid == 0 && sm.abort_flag && p.status_word) atomicExch(p.status_word, (int)KLA_ERR_TIMEOUT);
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
    CUtensorMap tq, tk;
    if (!make_tmap(&tq, p.q, n_tok, (uint64_t)p.H * D) || !make_tmap(&tk, p.k, n_tok, (uint64_t)p.H * D))
        return cudaErrorInvalidValue;
    auto kern = kla_chunk_tc_kernel<D, OUT>;
    const int smem = (int)sizeof(Smem) + 1024;
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (err != cudaSuccess) return err;
    const int grid = p.n_seq * p.H * (D / NS);
    if (grid == 0) return cudaSuccess;
    kern<<<grid, NT, smem, stream>>>(tq, tk, p);
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
