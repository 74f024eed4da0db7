// Chunkwise forward on the 5th-generation tensor cores (tcgen05.mma, TMEM accumulators, TMA-staged
// bf16 tiles) -- Algorithm 1, right panel; Eqs. 7-9.
//
// One CTA owns NS = 64 consecutive d_v columns of one (sequence, head) and walks that sequence's
// chunks (C = 64 tokens) in order.  Its d_k x NS slice of the state stays in registers in fp32 for
// the whole sequence.  The CTA is warp-specialised (17 warps), every role a compact loop:
//
//   control warp             issues every TMA load and every tcgen05.mma, in a fixed order
//   pre group (8 warps)      state-independent work for chunk c+1 while the chain works on chunk c:
//                            g (decay sums), beta (Eq. 3, ||k||^2 read off the diagonal of K K^T),
//                            X = A^- o K K^T, T = (I + B X)^-1 by blocked substitution in shared
//                            memory, and (half of the warps, one chunk behind) P = A o Q K^T
//   chain group (8 warps)    the serial dependency over chunks:
//                            rhs = B (V - D_gamma K S_0), U = T rhs                      (Eq. 7)
//                            O = D_gamma Q S_0 + P U                                     (Eq. 8)
//                            S <- gamma_C S_0 + K^T diag(exp(g_C - g_j)) U               (Eq. 9)
//
// With two column slices per head (d_v = 128) the two CTAs of a head are launched as a thread-block cluster and
// share the pre group's work: each forms X, T and P of every other chunk and copies the operand tiles and the
// per-token scalars into the peer's shared memory (kernel template parameter PAIR).
//
// Tensor-core products per chunk (fp32 accumulation in TMEM):
//   MMA-1  [K;Q] K^T   M=128   -> K K^T (lanes 0..63) and Q K^T (lanes 64..127), double-buffered
//   MMA-2  K S_0, Q S_0        two M=64 products, S_0 = S_hi + S_lo
//   MMA-3  T rhs       M=64    T_hi rhs_hi + T_hi rhs_lo + T_lo rhs_hi
//   MMA-4  P U         M=64    same three-term form, taken as (P D^-1)(D U) so that the chain forms D U only
//   MMA-5  K^T (D U)   M=128   D U = hi + lo
//
// Precision.  q, k, v are exact bf16 operands.  Every DERIVED operand (S_0, rhs, T, P, U, D U) is
// carried as a pair of bf16 values hi + lo (16 significand bits): a single bf16 rounding of any of
// them costs 1e-2..7e-2 in max|err|/rms on the layer-shaped workloads, far above the 2e-3 bound.
//
// Code size matters here: a role whose per-chunk code is one long unrolled stream runs at the speed
// of instruction fetch (measured: three times slower than the same code resident in the instruction
// cache), so loops are kept rolled wherever register arrays do not force unrolling, and the bounded
// barrier wait is one out-of-line function.
//
// Every wait on an mbarrier is bounded; when one gives up the CTA raises an abort flag, reports
// KLA_ERR_TIMEOUT through the status word, releases its TMEM and exits.
#include <cuda.h>

#include <cstddef>
#include <mutex>

#include "common.cuh"
#include "umma.cuh"

namespace kla {

namespace {

using namespace umma;

constexpr int C = 64;    // chunk length
constexpr int NS = 64;   // state columns per CTA
constexpr int PG_T = 256, CG_T = 256;
constexpr int NT = PG_T + CG_T + 32;
// Thread layout: warp 0 control, warps 1..8 chain group, warps 9..16 pre group: the roles on the serial chain
// sit in the lowest warp slots, which the warp schedulers favour when several warps are ready.
constexpr int CG_BASE = 32, PG_BASE = 32 + CG_T;
constexpr int NSTAGE = 3;
constexpr long long WAIT_LIMIT = 2000000000LL;  // SM clocks (~1 s) before a wait gives up
constexpr float LOG2E = 1.4426950408889634f;
// The write weights exp(g_C - g_j) are kept above 2^-DEC_FLOOR_LOG2 (~1e-35): the output product is taken as
// (P D^-1)(D U), and with the floor neither factor leaves the fp32 / bf16 exponent range however strong the decay.  A
// floored weight puts at most 1e-35 of a token into the state instead of less.
constexpr float DEC_FLOOR_LOG2 = 115.f;

// TMEM columns (fp32, 128 lanes each)
constexpr uint32_t TM_D1 = 0 /* two buffers of 64 */, TM_KS = 128, TM_QS0 = 192, TM_QS1 = 256, TM_U = 320, TM_PU = 384,
                   TM_DS = 448, TM_COLS = 512;

constexpr int LDT = 68;  // row stride (floats) of the fp32 solve matrix
constexpr int LDM = 40;  // row stride of the solve scratch

enum Bar {
    B_FULL0 = 0,             // +stage: TMA landed
    B_D1_DONE0 = 3,          // +buffer: MMA-1 complete
    B_D1_FREE0 = 5,          // +buffer: every pre warp finished reading that D1 buffer
    B_T_READY = 7,           // T(c) and the scalars of chunk c written
    B_P_READY = 8,           // P(c) written
    B_S_READY = 9,           // state tiles for chunk c written
    B_D2_DONE = 10,          // K S_0 of chunk c complete
    B_RHS_READY = 11,
    B_D3_DONE = 12,
    B_U_READY = 13,
    B_D5_DONE = 14,
    B_D4_DONE = 15,          // P U (and, earlier in the pipe, Q S_0) of chunk c complete
    B_TAIL_READY = 16,       // masked rows of the last chunk zeroed
    B_V_FULL = 17,           // V slice of chunk c landed
    // Paired CTAs.  A wait tells a phase only from its neighbours, and nothing bounds how far one CTA of a pair runs
    // ahead of the other, so every barrier below is waited on, phase after phase, by one role of one CTA:
    B_T_FREE0 = 18,          // +(c & 1): MMA-3(c) of both CTAs complete (the T tiles may be overwritten); waited on by
                             // the owner of chunk c + 1
    B_P_FREE0 = 20,          // +(c & 1): MMA-4(c) of both CTAs complete; waited on by the owner of chunk c + 1
    B_SCAL_READY0 = 22,      // +(c & 3): beta, gamma, exp(g_C - g) of chunk c written (long before T(c)).  Four deep: the
                             // owner sends those of chunk c + 4 only after it has seen MMA-3(c+1) of the peer complete,
                             // and that chain has then long since waited for those of chunk c
    B_COUNT = 26
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
    alignas(1024) unsigned char ru_hi[8192];    // rhs: 64 tokens x 64 bf16, MN-major
    alignas(1024) unsigned char ru_lo[8192];
    alignas(1024) unsigned char du_hi[8192];    // D U, D = diag(exp(g_C - g_j)): operand of MMA-5 and of MMA-4
    alignas(1024) unsigned char du_lo[8192];
    alignas(1024) unsigned char vt[8192];       // V slice of one chunk: 64 tokens x 64 bf16, same layout as ru_*
    alignas(16) float tl[64 * LDT];             // X = A^- o K K^T, overwritten in place by T = (I + B X)^-1
    alignas(16) float mm[32 * LDM];             // scratch for the block products of the inverse
    alignas(16) float g2[NSTAGE][64];           // log2(e) * chunk-local running sum of log alpha
    float beta[NSTAGE][64];
    float gam[NSTAGE][64];                      // exp(g_i)
    float dec[NSTAGE][64];                      // exp(g_C - g_i)
    alignas(8) uint64_t bar[B_COUNT];
    uint32_t tmem_base;
    volatile int abort_flag;
    float qn[NSTAGE][64];                       // 1 / ||q_i|| (written only when the normalised read-out is asked for)
};

// Bounded wait on an mbarrier phase that also leaves when another role has aborted.  Every lane of the
// calling warp polls: letting one lane poll and broadcasting the result splits the warp, and each later
// warp-collective instruction (elect.sync, tcgen05.ld) then pays for re-forming it.
__device__ __noinline__ bool bar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i) {
            if (mbar_try_wait(bar, parity)) return true;
            __nanosleep(32);   // a polling warp is always ready to issue: keep it from crowding out working warps
        }
        if (*abort_flag) return false;
        if (clock64() - t0 > WAIT_LIMIT) {
            *abort_flag = 1;
            return false;
        }
    }
}

// Warp-uniform wait for the control warp: every lane polls, the warp leaves together.  Out of line: the control
// program calls it a dozen times per chunk.
__device__ __noinline__ bool warp_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag)
{
    const bool ok = mbar_try_wait(bar, parity) || bar_wait(bar, parity, abort_flag);
    return __all_sync(0xffffffffu, ok);
}

__device__ __forceinline__ void pg_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
__device__ __forceinline__ void half_sync() { asm volatile("bar.sync 3, 64;" ::: "memory"); }
// Barrier over the pre group that also ORs a flag: makes "some thread's wait gave up" a collective
// decision, so that no thread is left alone at a later pg_sync().
__device__ __forceinline__ bool pg_any(bool flag)
{
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %1, 0;\n\t"
        "bar.red.or.pred q, 2, 256, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)flag)
        : "memory");
    return r != 0;
}


// 4 x 4 transpose over the four lanes of a quad (t = lane & 3): on entry lane t holds v[j] = element (t, j), on
// exit v[s] = element (s, t).  Two butterfly stages; every lane of the warp must call it.
__device__ __forceinline__ void quad_transpose(uint32_t (&v)[4], int t)
{
    const bool o1 = t & 1, o2 = t & 2;
    uint32_t x = o1 ? v[0] : v[1], y = o1 ? v[2] : v[3];
    x = __shfl_xor_sync(0xffffffffu, x, 1);
    y = __shfl_xor_sync(0xffffffffu, y, 1);
    if (o1) { v[0] = x; v[2] = y; } else { v[1] = x; v[3] = y; }
    x = o2 ? v[0] : v[2];
    y = o2 ? v[1] : v[3];
    x = __shfl_xor_sync(0xffffffffu, x, 2);
    y = __shfl_xor_sync(0xffffffffu, y, 2);
    if (o2) { v[0] = x; v[1] = y; } else { v[2] = x; v[3] = y; }
}

// One level of the blocked inverse of I + B X (X strictly lower triangular, 64 x 64, in `tl`): for every pair
// of adjacent BS x BS diagonal blocks (T_00, T_11 already inverted) the block below the diagonal becomes
//   T_10 = -T_11 (B_1 X_10 T_00).
// All pairs of the level are done at once by the 256 threads of the pre group: 32 result rows x BS columns,
// one 1 x 4 tile per thread; `mm` holds the intermediate product.  Trip counts are warp-uniform.
template <int BS>
__device__ __forceinline__ void merge_level(float *tl, float *mm, const float *bet, int pt)
{
    constexpr int QPR = BS / 4;                 // column quads per row
    constexpr int RMASK = 128 / BS - 1;         // a warp covers 128 / BS consecutive rows
    const bool act = pt < 8 * BS;
    const int R = pt / QPR, c4 = (pt % QPR) * 4;
    const int pr = R / BS, r = R % BS;          // pair, row inside the block
    const int rb = (2 * pr + 1) * BS, cb = 2 * pr * BS;
    if (act) {
        // M = B_1 X_10 T_00
        const float *Ap = tl + (rb + r) * LDT + cb;
        const float *Bp = tl + cb * LDT + cb + c4;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 2
        for (int k = 0; k < BS; k += 4) {
            const float4 a = *reinterpret_cast<const float4 *>(Ap + k);
            const float av[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float4 b = *reinterpret_cast<const float4 *>(Bp + (k + u) * LDT);
                acc.x += av[u] * b.x; acc.y += av[u] * b.y; acc.z += av[u] * b.z; acc.w += av[u] * b.w;
            }
        }
        const float s = bet[rb + r];
        *reinterpret_cast<float4 *>(&mm[R * LDM + c4]) = make_float4(s * acc.x, s * acc.y, s * acc.z, s * acc.w);
    }
    pg_sync();
    if (act) {
        // T_10 = -T_11 M; T_11 is lower triangular: columns k > r of its row r are zero
        const float *Ap = tl + (rb + r) * LDT + rb;
        const float *Bp = mm + (pr * BS) * LDM + c4;
        const int kend = min(BS, (r | RMASK) + 1);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 2
        for (int k = 0; k < kend; k += 4) {
            const float4 a = *reinterpret_cast<const float4 *>(Ap + k);
            const float av[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float4 b = *reinterpret_cast<const float4 *>(Bp + (k + u) * LDM);
                acc.x += av[u] * b.x; acc.y += av[u] * b.y; acc.z += av[u] * b.z; acc.w += av[u] * b.w;
            }
        }
        *reinterpret_cast<float4 *>(&tl[(rb + r) * LDT + cb + c4]) = make_float4(-acc.x, -acc.y, -acc.z, -acc.w);
    }
    pg_sync();
}

// ---- pieces of the pre group's work, shared by the paired and the unpaired form of the group ------------------------------
// Decay scan of one chunk by one warp (lane l holds log alpha of tokens 2l, 2l + 1): log2(e) g_i, gamma_i = exp(g_i),
// d_i = exp(g_C - g_i) (floored, see DEC_FLOOR_LOG2) into slot sc.
template <typename Smem>
__device__ __forceinline__ void decay_scan(Smem &sm, int sc, int lane, float la0, float la1)
{
    float incl = la0 + la1;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const float t = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += t;
    }
    const float gC = __shfl_sync(0xffffffffu, incl, 31);
    const float a2 = (incl - la1) * LOG2E, b2 = incl * LOG2E, c2 = gC * LOG2E;
    *reinterpret_cast<float2 *>(&sm.g2[sc][2 * lane]) = make_float2(a2, b2);
    *reinterpret_cast<float2 *>(&sm.gam[sc][2 * lane]) = make_float2(ex2_approx(a2), ex2_approx(b2));
    *reinterpret_cast<float2 *>(&sm.dec[sc][2 * lane]) =
        make_float2(ex2_approx(fmaxf(c2 - a2, -DEC_FLOOR_LOG2)), ex2_approx(fmaxf(c2 - b2, -DEC_FLOOR_LOG2)));
}

// Last chunk: rows past the end of the sequence hold a neighbour's tokens (or TMA zero fill); zero them in the K and
// Q tiles of the stage so that they are inert in every product.  All PG_T threads of the group.
template <int KB>
__device__ __forceinline__ void zero_tail_rows(unsigned char *kq, int rows, int pt)
{
    for (int e = pt; e < (C - rows) * 8; e += PG_T) {
        const int r = rows + e / 8, ch = e % 8;
        const uint4 z = make_uint4(0, 0, 0, 0);
#pragma unroll
        for (int kb = 0; kb < KB; ++kb) {
            *reinterpret_cast<uint4 *>(kq + kb * 16384 + sw128(r, ch)) = z;
            *reinterpret_cast<uint4 *>(kq + kb * 16384 + 8192 + sw128(r, ch)) = z;
        }
    }
}

// X = A^- o K K^T: this thread's row i, columns chh * 32 .. + 31 of the MMA-1 accumulator at tbase, into the solve
// matrix.  Returns the diagonal element G_ii = ||k_i||^2 if it lies in these columns (else 0).
template <typename Smem>
__device__ __forceinline__ float form_x_row(Smem &sm, int sc, int i, int chh, uint32_t tbase)
{
    const float gi2 = sm.g2[sc][i];
    float dg = 0.f;
#pragma unroll 1
    for (int grp = 0; grp < 4; ++grp) {
        float a[8];
        tmem_ld8(tbase + grp * 8, a);
        const int j0 = chh * 32 + grp * 8;
        const float4 ga = *reinterpret_cast<const float4 *>(&sm.g2[sc][j0]);
        const float4 gb = *reinterpret_cast<const float4 *>(&sm.g2[sc][j0 + 4]);
        const float gj[8] = {ga.x, ga.y, ga.z, ga.w, gb.x, gb.y, gb.z, gb.w};
        float x[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            x[e] = (j0 + e < i) ? ex2_approx(gi2 - gj[e]) * a[e] : 0.f;
            dg = (j0 + e == i) ? a[e] : dg;
        }
        *reinterpret_cast<float4 *>(&sm.tl[i * LDT + j0]) = make_float4(x[0], x[1], x[2], x[3]);
        *reinterpret_cast<float4 *>(&sm.tl[i * LDT + j0 + 4]) = make_float4(x[4], x[5], x[6], x[7]);
    }
    return dg;
}

// P D^-1 with P = A o Q K^T and D = diag(d_j), d_j the (floored) write weights of the decay scan: the chain forms D U
// only (the operand of the state update), and the outputs use P U = (P D^-1)(D U).  Element (i, j <= i) is
// exp(g_i - g_j) / d_j = 2^(g2_i - max(g2_C, g2_j - DEC_FLOOR_LOG2)), at most 2^DEC_FLOOR_LOG2.  This thread's row i,
// columns chh * 32 .. + 31 of the MMA-1 accumulator at tbase, as bf16 hi/lo operand tiles (zeros where `live` is false:
// all 32 columns above the diagonal).
template <typename Smem>
__device__ __forceinline__ void form_p_row(Smem &sm, int sc, int i, int chh, bool live, uint32_t tbase)
{
    const float gi2 = sm.g2[sc][i], gc2 = sm.g2[sc][C - 1];
#pragma unroll 2
    for (int grp = 0; grp < 4; ++grp) {
        uint4 hi = make_uint4(0, 0, 0, 0), lo = hi;
        if (live) {
            float a[8];
            tmem_ld8(tbase + grp * 8, a);
            const int j0 = chh * 32 + grp * 8;
            const float4 ga = *reinterpret_cast<const float4 *>(&sm.g2[sc][j0]);
            const float4 gb = *reinterpret_cast<const float4 *>(&sm.g2[sc][j0 + 4]);
            const float gj[8] = {ga.x, ga.y, ga.z, ga.w, gb.x, gb.y, gb.z, gb.w};
            float x[8];
#pragma unroll
            for (int e = 0; e < 8; ++e)
                x[e] = (j0 + e <= i) ? ex2_approx(gi2 - fmaxf(gc2, gj[e] - DEC_FLOOR_LOG2)) * a[e] : 0.f;
            split2(x[0], x[1], hi.x, lo.x);
            split2(x[2], x[3], hi.y, lo.y);
            split2(x[4], x[5], hi.z, lo.z);
            split2(x[6], x[7], hi.w, lo.w);
        }
        *reinterpret_cast<uint4 *>(sm.p_hi + sw128(i, chh * 4 + grp)) = hi;
        *reinterpret_cast<uint4 *>(sm.p_lo + sw128(i, chh * 4 + grp)) = lo;
    }
}

// 8 x 8 diagonal blocks of T = (I + B X)^-1 by substitution: thread pt < 64 solves column pt % 8 of block pt / 8 in
// registers, then the block's eight threads write their columns over X_bb.
__device__ __forceinline__ void substitute_diag_blocks(float *tl, const float *bet, int pt)
{
    const int blk = pt >> 3, j = pt & 7;
    float *Lb = tl + (blk * 8) * LDT + blk * 8;
    float x[8];
#pragma unroll
    for (int r = 0; r < 8; ++r) {
        const float4 l0 = *reinterpret_cast<const float4 *>(Lb + r * LDT);
        const float4 l1 = *reinterpret_cast<const float4 *>(Lb + r * LDT + 4);
        const float l[8] = {l0.x, l0.y, l0.z, l0.w, l1.x, l1.y, l1.z, l1.w};
        float s = 0.f;
#pragma unroll
        for (int m = 0; m < r; ++m) s += l[m] * x[m];
        x[r] = (r == j) ? 1.f : ((r > j) ? -bet[blk * 8 + r] * s : 0.f);
    }
    half_sync();  // every column of the block has read X_bb
#pragma unroll
    for (int r = 0; r < 8; ++r) Lb[r * LDT + j] = x[r];
}

// T (fp32, in the solve matrix) as bf16 hi/lo operand tiles: thread pt writes 16 columns of row pt % 64.
template <typename Smem>
__device__ __forceinline__ void write_t_tiles(Smem &sm, int pt)
{
    const int r = pt & 63, qq = pt >> 6;  // row, 16-column quarter
#pragma unroll 1
    for (int ch = 0; ch < 2; ++ch) {
        const float4 a = *reinterpret_cast<const float4 *>(&sm.tl[r * LDT + qq * 16 + ch * 8]);
        const float4 b = *reinterpret_cast<const float4 *>(&sm.tl[r * LDT + qq * 16 + ch * 8 + 4]);
        uint4 hi, lo;
        split2(a.x, a.y, hi.x, lo.x);
        split2(a.z, a.w, hi.y, lo.y);
        split2(b.x, b.y, hi.z, lo.z);
        split2(b.z, b.w, hi.w, lo.w);
        *reinterpret_cast<uint4 *>(sm.t_hi + sw128(r, qq * 2 + ch)) = hi;
        *reinterpret_cast<uint4 *>(sm.t_lo + sw128(r, qq * 2 + ch)) = lo;
    }
}

// VAR: compiled with the layer-edge variants (beta = eta, read-out over ||q||); the default instantiation carries
// none of their code.
// PAIR: the two CTAs that hold the two column slices of one (sequence, head) run as a thread-block cluster and
// share the state-independent work: the CTA of rank r forms X, T and P of the chunks c with c mod 2 = r and writes
// the T and P operand tiles (and beta) into both CTAs' shared memory, so that each pre group has two chunk
// periods for one inverse.  The decay scan, every MMA but MMA-1, and the chain stay per CTA.
template <int D, typename OUT, bool VAR, bool PAIR>
__global__ void __launch_bounds__(NT, 1)
kla_chunk_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, ChunkParams p)
{
    using Smem = TcSmem<D>;
    constexpr int KB = Smem::KB;
    constexpr int SLICES = D / NS;
    constexpr uint32_t STAGE_BYTES = Smem::KQ_BYTES;
    // a pair hands T and P over with one copy per hi/lo pair of tiles
    static_assert(sizeof(Smem) + 1024 <= 232448, "shared memory of one CTA");
    static_assert(offsetof(Smem, t_lo) == offsetof(Smem, t_hi) + 8192 && offsetof(Smem, p_lo) == offsetof(Smem, p_hi) + 8192, "tile pairs must be contiguous");
    constexpr uint32_t ID_G = idesc_bf16(128, 64, 0, 0);    // [K;Q] K^T : A K-major, B K-major
    constexpr uint32_t ID_S = idesc_bf16(64, NS, 0, 1);     // K S / Q S / T rhs / P U : M=64, B MN-major
    constexpr uint32_t ID_DS = idesc_bf16(128, NS, 1, 1);   // K^T (D U): A MN-major, B MN-major

    extern __shared__ unsigned char smem_dyn[];
    Smem &sm = *reinterpret_cast<Smem *>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) & ~(uintptr_t)1023);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;   // PAIR: adjacent blocks = the two slices of one head
    // plain launch: block = (sequence, head, slice).  Segment pass 1 doubles the slices (the second set carries
    // the transition map) and skips each sequence's last segment; see ChunkParams.
    const int nslices = p.seg_pass == 1 ? 2 * SLICES : SLICES;
    const int sl2 = blockIdx.x % nslices;
    const bool is_map = sl2 >= SLICES;
    const int sl = sl2 % SLICES;
    const int h = (blockIdx.x / nslices) % p.H;
    int n = blockIdx.x / (nslices * p.H);
    const bool no_out = p.seg_pass == 1;
    // Segment passes: the word after the segment bounds says whether the segments start from decay-bounded warm-up runs
    // (pass 4, or 5 for packed input, alone does the work) or not (passes 1 and 3, or the plain packed launch 6, do);
    // the other kind returns at once.
    if (p.seg_pass == 6) {
        if (p.seq_order[p.seg_G] != 0) return;
    } else if (p.seg_pass != 0 && (p.seg_pass >= 4) != (p.cu_seqlens[p.n_seq + 1] == 1)) {
        return;
    }
    if (p.seg_pass == 1) n = (n / (p.seg_G - 1)) * p.seg_G + n % (p.seg_G - 1);
    else if ((p.seg_pass == 0 || p.seg_pass == 6) && p.seq_order) n = p.seq_order[n];   // packed input: longest sequences first

    int tok0, len;
    if (p.cu_seqlens) {
        tok0 = p.cu_seqlens[n];
        len = p.cu_seqlens[n + 1] - tok0;
    } else {
        tok0 = n * p.T;
        len = p.T;
    }
    // packed input cut into pieces: the piece's sequence, and whether it is the first and the last piece of it
    const int32_t piece = p.seg_pass == 5 ? p.cu_seqlens[p.n_seq + 2 + p.n_seq * p.H + n] : 0;
    const int sq = p.seg_pass == 5 ? (piece & 0x1fffffff) : n;   // index of the states this CTA reads and writes
    const size_t state_off = (((size_t)sq * p.H + h) * D) * D + (size_t)sl * NS;
    // the state before the first token (null: zero) and the number of leading chunks whose outputs are not stored
    const float *init = p.init_state;
    size_t init_off = state_off;
    int first_out = 0;
    if (p.seg_pass == 5 && !((piece >> 29) & 1)) {   // not a sequence's first piece: from zero, so many chunks early
        init = nullptr;
        first_out = p.cu_seqlens[p.n_seq + 2 + n * p.H + h];
        tok0 -= first_out * C;
        len += first_out * C;
    }
    if (p.seg_pass == 4) {
        if (n % p.seg_G == 0) {   // first segment: the sequence's own initial state
            init_off = (((size_t)(n / p.seg_G) * p.H + h) * D) * D + (size_t)sl * NS;
        } else {                  // later segments: from zero, so many chunks before the segment (see seg_warm_plan_kernel)
            init = nullptr;
            first_out = p.cu_seqlens[p.n_seq + 2 + n * p.H + h];
            tok0 -= first_out * C;
            len += first_out * C;
        }
    }
    // where this CTA's final state goes (null: nowhere)
    float *fin = is_map ? p.map_state : p.final_state;
    size_t fin_off = state_off;
    if (p.seg_pass == 5) {
        if (!((piece >> 30) & 1)) fin = nullptr;   // only a sequence's last piece holds its final state
    } else if (p.seg_pass >= 3 && p.seg_pass <= 4 && fin) {
        if (n % p.seg_G != p.seg_G - 1) fin = nullptr;
        else fin_off = (((size_t)(n / p.seg_G) * p.H + h) * D) * D + (size_t)sl * NS;
    }

    if (len <= 0) {  // empty sequence: the final state is the initial state (never a segment: those are non-empty)
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
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sm.bar[B_D1_DONE0 + b], 1);
            mbar_init(&sm.bar[B_D1_FREE0 + b], PG_T / 32);
        }
        // PAIR: one arrival per chunk, local (own chunk) or from the peer together with the bytes of its copy
        mbar_init(&sm.bar[B_T_READY], PAIR ? 1 : PG_T / 32);
        mbar_init(&sm.bar[B_P_READY], PAIR ? 1 : PG_T / 64);
        mbar_init(&sm.bar[B_S_READY], CG_T / 32);
        mbar_init(&sm.bar[B_D2_DONE], 1);
        mbar_init(&sm.bar[B_RHS_READY], CG_T / 32);
        mbar_init(&sm.bar[B_D3_DONE], 1);
        mbar_init(&sm.bar[B_U_READY], CG_T / 32);
        mbar_init(&sm.bar[B_D5_DONE], 1);
        mbar_init(&sm.bar[B_D4_DONE], 1);
        mbar_init(&sm.bar[B_TAIL_READY], PG_T / 32);
        mbar_init(&sm.bar[B_V_FULL], 1);
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sm.bar[B_T_FREE0 + b], 2);
            mbar_init(&sm.bar[B_P_FREE0 + b], 2);
        }
        for (int b = 0; b < 4; ++b) mbar_init(&sm.bar[B_SCAL_READY0 + b], 1);
        sm.abort_flag = 0;
        mbar_fence_init();
    }
    // the block of the solve matrix above the diagonal blocks is never written again
    for (int i = tid; i < 64 * LDT; i += NT) sm.tl[i] = 0.f;
    if (warp == 0) tmem_alloc(&sm.tmem_base, TM_COLS);
    tc_fence_before();
    __syncthreads();
    if constexpr (PAIR) cluster_sync_all();   // the peer's barriers are initialised before anything arrives on them
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;
    const uint32_t tm_lane = tmem + ((uint32_t)((warp & 3) * 32) << 16);  // this warp's 32 TMEM lanes

    // fast path inline (the phase is often complete already), polling loop out of line
    auto wait = [&](int b, uint32_t parity) -> bool {
        if (mbar_try_wait(&sm.bar[b], parity)) return true;
        return bar_wait(&sm.bar[b], parity, &sm.abort_flag);
    };
    // one arrival per warp, after the warp's shared-memory writes are visible to the async proxy
    auto warp_arrive = [&](int b) {
        __syncwarp();
        if (lane == 0) mbar_arrive(&sm.bar[b]);
    };

    if (warp == 0) {
        // =============================== control warp =====================================================
        // The whole warp runs this role in lock step: waits are taken by every lane, TMA loads are issued
        // by lane 0 and tensor-core instructions by the lane that elect.sync picks.
        if (lane == 0) {
            tma_prefetch_desc(&tm_q);
            tma_prefetch_desc(&tm_k);
            tma_prefetch_desc(&tm_v);
        }
        auto issue_tma = [&](int c) {
            if (lane == 0) {
                const int st = c % NSTAGE;
                mbar_expect_tx(&sm.bar[B_FULL0 + st], STAGE_BYTES);
                const int row = tok0 + c * C;
#pragma unroll
                for (int kb = 0; kb < KB; ++kb) {
                    tma_load_2d(sm.kq[st] + kb * 16384, &tm_k, h * D + kb * 64, row, &sm.bar[B_FULL0 + st]);
                    tma_load_2d(sm.kq[st] + kb * 16384 + 8192, &tm_q, h * D + kb * 64, row, &sm.bar[B_FULL0 + st]);
                }
            }
            __syncwarp();
        };
        // V slice of chunk c: one 64 x 64 box; the single buffer is free once every chain warp has posted rhs(c-1).
        // (Fetching V with plain loads into registers a chunk ahead stalled the chain warps for the full
        // global-memory latency at their next barrier wait.)
        auto issue_tma_v = [&](int c) {
            if (lane == 0) {
                mbar_expect_tx(&sm.bar[B_V_FULL], 8192);
                tma_load_2d(sm.vt, &tm_v, h * D + sl * NS, tok0 + c * C, &sm.bar[B_V_FULL]);
            }
            __syncwarp();
        };
        auto wwait = [&](int b, uint32_t parity) -> bool { return warp_wait(&sm.bar[b], parity, &sm.abort_flag); };
        // four MMAs (K = 64): operand descriptors advance by astep / bstep (16-byte units) per K-step
#define KLA_SEQ(d, a, astep, b, bstep, idesc, acc) mma4_bf16_lo<astep, bstep>(d, a, b, idesc, acc)
        // Descriptors: everything except the 14-bit start-address field is fixed, so a K-step is an add.
        const uint32_t d_kq0 = desc_lo(smem_desc_sw128(smem_u32(sm.kq[0]), 16, 1024));             // K-major views of a stage
        const uint32_t d_kt0 = desc_lo(smem_desc_sw128(smem_u32(sm.kq[0]), KB * 8192, 1024));      // K^T (MN-major) view
        const uint32_t d_sh = desc_lo(smem_desc_sw128(smem_u32(sm.s_hi), 16, 1024)), d_sl = desc_lo(smem_desc_sw128(smem_u32(sm.s_lo), 16, 1024));
        const uint32_t d_th = desc_lo(smem_desc_sw128(smem_u32(sm.t_hi), 16, 1024)), d_tl = desc_lo(smem_desc_sw128(smem_u32(sm.t_lo), 16, 1024));
        const uint32_t d_ph = desc_lo(smem_desc_sw128(smem_u32(sm.p_hi), 16, 1024)), d_pl = desc_lo(smem_desc_sw128(smem_u32(sm.p_lo), 16, 1024));
        const uint32_t d_rh = desc_lo(smem_desc_sw128(smem_u32(sm.ru_hi), 16, 1024)), d_rl = desc_lo(smem_desc_sw128(smem_u32(sm.ru_lo), 16, 1024));
        const uint32_t d_dh = desc_lo(smem_desc_sw128(smem_u32(sm.du_hi), 16, 1024)), d_dl = desc_lo(smem_desc_sw128(smem_u32(sm.du_lo), 16, 1024));
        constexpr uint32_t STAGE_STEP = (uint32_t)(Smem::KQ_BYTES >> 4);

        auto mma1 = [&](int c) {  // [K;Q] K^T -> D1 buffer c & 1 (PAIR: this CTA's chunks alternate between the buffers)
            const uint32_t a0 = d_kq0 + (uint32_t)(c % NSTAGE) * STAGE_STEP;
            const int b = PAIR ? (c >> 1) & 1 : c & 1;
#pragma unroll 1
            for (int kb = 0; kb < KB; ++kb) KLA_SEQ(tmem + TM_D1 + (uint32_t)b * 64, a0 + kb * 1024, 2, a0 + kb * 1024, 2, ID_G, kb > 0);
            mma_commit(&sm.bar[B_D1_DONE0 + b]);
        };
        // PAIR: MMA-1 of one of this CTA's own chunks, once its tiles have landed and its D1 buffer (last used by
        // chunk c - 4) has been read
        auto mma1_own = [&](int c) -> bool {
            if (!wwait(B_FULL0 + c % NSTAGE, (uint32_t)((c / NSTAGE) & 1))) return false;
            if (c + 1 == nchunks && last_rows < C)
                if (!wwait(B_TAIL_READY, 0)) return false;
            if (c >= 4)
                if (!wwait(B_D1_FREE0 + ((c >> 1) & 1), (uint32_t)(((c >> 2) - 1) & 1))) return false;
            tc_fence_after();
            mma1(c);
            return true;
        };
        // [K or Q](c) S_0 -> d; qoff = 512 selects the Q tile of a block; S_0 = S_hi + S_lo
        // (blocks t0 .. t1 - 1 of the 2 KB four-MMA blocks: the S_hi term first, then the S_lo term)
        auto mma_xs = [&](uint32_t d, uint32_t k0, uint32_t qoff, int t0, int t1) {
#pragma unroll 1
            for (int t = t0; t < t1; ++t) {
                const uint32_t kb = (uint32_t)t & (KB - 1);
                KLA_SEQ(d, k0 + qoff + kb * 1024, 2, (t >= KB ? d_sl : d_sh) + kb * 512, 128, ID_S, t > 0);
            }
        };
        // three-term product (a_hi + a_lo)(b_hi + b_lo) ~ a_hi b_hi + a_hi b_lo + a_lo b_hi, K = 64
        auto mma_3 = [&](uint32_t d, uint32_t ah, uint32_t al, uint32_t bh, uint32_t bl) {
#pragma unroll 1
            for (int t = 0; t < 3; ++t) KLA_SEQ(d, t == 2 ? al : ah, 2, t == 1 ? bl : bh, 128, ID_S, t > 0);
        };
        bool ok = true;
        for (int c = 0; c < NSTAGE && c < nchunks; ++c) issue_tma(c);
        issue_tma_v(0);
        if constexpr (PAIR) {
            // ---- paired CTAs.  The tensor pipe runs the MMAs in issue order at ~60 cycles each, so what is not on the
            // chain goes where the pipe would idle and can finish before the chain's next product is ready:
            //   K S_0(c) | MMA-1 of this CTA's chunk c + 2 (if due and landed), else half of Q S_0(c)   while rhs(c) forms
            //   MMA-3(c) | the rest of Q S_0(c) (| MMA-1 if due and not issued above)                   while D U(c) forms
            //   MMA-5(c) | MMA-4(c)                                                        while the chain updates S
            // Order constraints: Q S_0(c) before MMA-5(c), whose completion lets the chain overwrite the S tiles;
            // MMA-4(c) before MMA-3(c+1), whose completion lets it overwrite D U.
            auto ready = [&](int b, uint32_t parity) -> bool {
                return __all_sync(0xffffffffu, mbar_test_wait(&sm.bar[b], parity));
            };
            if ((int)rank < nchunks) ok = mma1_own((int)rank);
            for (int c = 0; ok && c < nchunks; ++c) {
                const bool own = (uint32_t)(c & 1) == rank;
                // a chunk of the peer: no MMA-1 here has waited for its tiles
                if (!own)
                    if (!(ok = wwait(B_FULL0 + c % NSTAGE, (uint32_t)((c / NSTAGE) & 1)))) break;
                // the masked rows of the last chunk are zeroed before any product reads its tiles
                if (c + 1 == nchunks && last_rows < C)
                    if (!(ok = wwait(B_TAIL_READY, 0))) break;
                const uint32_t ph = (uint32_t)(c & 1);
                const uint32_t k0 = d_kq0 + (uint32_t)(c % NSTAGE) * STAGE_STEP;
                const uint32_t kt0 = d_kt0 + (uint32_t)(c % NSTAGE) * STAGE_STEP;
                if (!(ok = wwait(B_S_READY, ph))) break;
                tc_fence_after();
                mma_xs(tmem + TM_KS, k0, 0, 0, 2 * KB);
                mma_commit(&sm.bar[B_D2_DONE]);
                const int cn = c + 2;   // this CTA's next chunk
                bool m1_due = own && cn < nchunks;
                int qs_done = no_out ? 2 * KB : 0;   // blocks of Q S_0 issued so far
                if (m1_due && ready(B_FULL0 + cn % NSTAGE, (uint32_t)((cn / NSTAGE) & 1)) &&
                    (!(cn + 1 == nchunks && last_rows < C) || ready(B_TAIL_READY, 0)) &&
                    (cn < 4 || ready(B_D1_FREE0 + ((cn >> 1) & 1), (uint32_t)(((cn >> 2) - 1) & 1)))) {
                    tc_fence_after();
                    mma1(cn);
                    m1_due = false;
                } else if (!no_out) {
                    // no MMA-1 in this window: the S_hi term of Q S_0 fits here instead
                    mma_xs(tmem + ((c & 1) ? TM_QS1 : TM_QS0), k0, 512, 0, KB);
                    qs_done = KB;
                }
                // MMA-3(c): U = T rhs
                if (!(ok = wwait(B_T_READY, ph))) break;
                if (!(ok = wwait(B_RHS_READY, ph))) break;
                tc_fence_after();
                mma_3(tmem + TM_U, d_th, d_tl, d_rh, d_rl);
                bool signal = true;
                if constexpr (VAR) signal = !(p.variant & VARIANT_TEST_TIMEOUT);   // test hook: see the unpaired loop
                if (signal) {
                    mma_commit(&sm.bar[B_D3_DONE]);
                    // Only where a later chunk's owner will wait for it: a signal sent for the last chunk could reach
                    // the peer's SM after that CTA has gone and another block has set up its barriers there.
                    if (c + 1 < nchunks) mma_commit_multicast(&sm.bar[B_T_FREE0 + (c & 1)], 3);
                }
                if (c + 1 < nchunks) issue_tma_v(c + 1);   // every chain warp has posted rhs(c): the V buffer is free
                if (qs_done < 2 * KB) mma_xs(tmem + ((c & 1) ? TM_QS1 : TM_QS0), k0, 512, qs_done, 2 * KB);
                if (m1_due)
                    if (!(ok = mma1_own(cn))) break;
                // MMA-5(c): K^T (D U)
                if (!(ok = wwait(B_U_READY, ph))) break;
                tc_fence_after();
#pragma unroll 1
                for (int t = 0; t < 2; ++t) KLA_SEQ(tmem + TM_DS, kt0, 128, t ? d_dl : d_dh, 128, ID_DS, t);
                mma_commit(&sm.bar[B_D5_DONE]);
                // MMA-4(c): P U
                if (!no_out) {
                    if (!(ok = wwait(B_P_READY, ph))) break;
                    tc_fence_after();
                    mma_3(tmem + TM_PU, d_ph, d_pl, d_dh, d_dl);
                    mma_commit(&sm.bar[B_D4_DONE]);
                    if (c + 1 < nchunks) mma_commit_multicast(&sm.bar[B_P_FREE0 + (c & 1)], 3);   // as for T_FREE
                }
                // (the chain group, which sees MMA-5(c) complete first, refills the K/Q stage of chunk c)
            }
        } else {
        // iteration c issues MMA-1(c+1) first, as early as its inputs and its D1 buffer allow; c = -1 does only that
        for (int c = -1; ok && c < nchunks; ++c) {
            if (c + 1 < nchunks) {
                if (!(ok = wwait(B_FULL0 + (c + 1) % NSTAGE, (uint32_t)(((c + 1) / NSTAGE) & 1)))) break;
                if (c + 2 == nchunks && last_rows < C)
                    if (!(ok = wwait(B_TAIL_READY, 0))) break;
                if (c >= 1)   // the buffer was last used by chunk c - 1: its ((c - 1) / 2)-th use
                    if (!(ok = wwait(B_D1_FREE0 + ((c + 1) & 1), (uint32_t)(((c - 1) >> 1) & 1)))) break;
                tc_fence_after();
                mma1(c + 1);
            }
            if (c < 0) continue;
            const uint32_t ph = (uint32_t)(c & 1);
            const uint32_t k0 = d_kq0 + (uint32_t)(c % NSTAGE) * STAGE_STEP;
            const uint32_t kt0 = d_kt0 + (uint32_t)(c % NSTAGE) * STAGE_STEP;
            // MMA-2(c): K S_0 -> TM_KS (on the chain), then Q S_0 -> TM_QS[c&1] (needed only for the outputs)
            if (!(ok = wwait(B_S_READY, ph))) break;
            tc_fence_after();
#pragma unroll 1
            for (int x = 0; x < (no_out ? 1 : 2); ++x) {
                mma_xs(tmem + (x == 0 ? TM_KS : ((c & 1) ? TM_QS1 : TM_QS0)), k0, x * 512, 0, 2 * KB);
                if (x == 0) mma_commit(&sm.bar[B_D2_DONE]);
            }
            // MMA-3(c): U = T rhs
            if (!(ok = wwait(B_T_READY, ph))) break;
            if (!(ok = wwait(B_RHS_READY, ph))) break;
            if (c + 1 < nchunks) issue_tma_v(c + 1);
            tc_fence_after();
            mma_3(tmem + TM_U, d_th, d_tl, d_rh, d_rl);
            if constexpr (VAR) {
                // test hook: without this signal the chain's bounded wait runs out
                if (!(p.variant & VARIANT_TEST_TIMEOUT)) mma_commit(&sm.bar[B_D3_DONE]);
            } else {
                mma_commit(&sm.bar[B_D3_DONE]);
            }
            // MMA-5(c): K^T (D U)   then   MMA-4(c): P U
            if (!(ok = wwait(B_U_READY, ph))) break;
            tc_fence_after();
            // A = K^T: M = d_k (64-wide blocks KB*8192 bytes apart; for d_k = 64 the second block
            // is the Q tile, whose rows land in TMEM lanes 64..127 and are ignored), K = tokens
#pragma unroll 1
            for (int t = 0; t < 2; ++t) KLA_SEQ(tmem + TM_DS, kt0, 128, t ? d_dl : d_dh, 128, ID_DS, t);
            mma_commit(&sm.bar[B_D5_DONE]);
            if (!no_out) {
                if (!(ok = wwait(B_P_READY, ph))) break;
                tc_fence_after();
                mma_3(tmem + TM_PU, d_ph, d_pl, d_dh, d_dl);
                mma_commit(&sm.bar[B_D4_DONE]);
            }
            // the K/Q stage of chunk c is free once MMA-5(c) has read it
            if (c + NSTAGE < nchunks) {
                if (!(ok = wwait(B_D5_DONE, ph))) break;
                issue_tma(c + NSTAGE);
            }
        }
        }
    } else if (PAIR && warp >= PG_BASE / 32) {
        // =============================== pre group, paired CTAs ============================================
        // This CTA's own chunks (c mod 2 = rank): decay scan, X(c), beta(c), T(c) and P(c); the per-token scalars
        // and the T and P operand tiles go into both CTAs.  The peer's chunks: only the zeroing of the masked rows
        // of the last chunk (the K and Q tiles are per CTA).  Warp roles as in the unpaired group: warps 0, 1, 4, 5
        // hold rows of K K^T, warps 2, 3, 6, 7 rows of Q K^T.
        const int pt = tid - PG_BASE;
        const int q = warp & 3, chh = (warp - PG_BASE / 32) >> 2;
        const bool is_g = q < 2;
        const int i = (q & 1) * 32 + lane;
        const bool live = chh <= (q & 1);
        const bool scan_warp = q == 0 && chh == 1;
        // distance from a shared-memory address of this CTA to the same location in the peer CTA
        const uint32_t peer_off = mapa_u32(smem_u32(&sm), rank ^ 1u) - smem_u32(&sm);
        float la_next0 = 0.f, la_next1 = 0.f, eta_next = 0.f;
        auto fetch_gates = [&](int c) {
            if (scan_warp) {
                const int t = c * C + 2 * lane;
                la_next0 = (t < len) ? p.log_alpha[(size_t)(tok0 + t) * p.H + h] : 0.f;
                la_next1 = (t + 1 < len) ? p.log_alpha[(size_t)(tok0 + t + 1) * p.H + h] : 0.f;
            }
            if (is_g && chh == q) {
                const int t = c * C + i;
                eta_next = (t < len) ? p.eta[(size_t)(tok0 + t) * p.H + h] : 0.f;
            }
        };
        if ((int)rank < nchunks) fetch_gates((int)rank);
        bool okp = true;   // outcome of the P warps' waits, folded into the next collective decision
        for (int c = 0; c < nchunks; ++c) {
            const int rows = (c == nchunks - 1) ? last_rows : C;
            const int sc = c % NSTAGE;
            const bool own = (uint32_t)(c & 1) == rank;
            const float la0 = la_next0, la1 = la_next1, eta_cur = eta_next;
            if (own && c + 2 < nchunks) fetch_gates(c + 2);
            if (own && scan_warp) {
                decay_scan(sm, sc, lane, la0, la1);
                fence_async_smem();   // gam and dec are also copied to the peer
            }
            bool okc = okp;
            if (rows < C && okc) {
                okc = wait(B_FULL0 + sc, (uint32_t)((c / NSTAGE) & 1));
                if (okc) {
                    zero_tail_rows<KB>(sm.kq[sc], rows, pt);
                    fence_async_smem();
                    warp_arrive(B_TAIL_READY);
                }
            }
            if (pg_any(!okc)) break;   // also publishes the decay sums to the whole group
            if (!own) continue;   // the peer's chunk: its scalars, T and P arrive from there

            const int b1 = (c >> 1) & 1;                       // D1 buffer of this CTA's chunk c, ...
            const uint32_t ph1 = (uint32_t)((c >> 2) & 1);     // ... in its (c / 4)-th use
            if (is_g) {
                // ---- X = A^- o K K^T (this thread: row i, 32 columns) and beta_i, Eq. 3 ----------------------
                okc = wait(B_D1_DONE0 + b1, ph1);
                if (okc) {
                    tc_fence_after();
                    if (live) {
                        // G_ii = ||k_i||^2 comes with the row
                        const float dg = form_x_row(sm, sc, i, chh, tm_lane + TM_D1 + (uint32_t)b1 * 64 + chh * 32);
                        if (chh == q) {
                            sm.beta[sc][i] = (i < rows) ? eta_cur / (dg + p.eps) : 0.f;
                            fence_async_smem();
                        }
                    }
                    tc_fence_before();
                    warp_arrive(B_D1_FREE0 + b1);
                }
            } else if (no_out) {
                warp_arrive(B_D1_FREE0 + b1);   // nothing reads Q K^T
            }
            if (pg_any(!okc)) break;
            // The per-token scalars of chunk c (beta, gamma, exp(g_C - g)) go to both chains now, more than a chunk
            // period before T(c): their rhs does not wait for the inverse.  (The peer's slot c mod 3 is free: its
            // chain read the scalars of chunk c - 3 before MMA-3(c-3), which this group saw complete two chunks ago.)
            if (pt == 0) {
                const uint32_t rbar = smem_u32(&sm.bar[B_SCAL_READY0 + (c & 3)]) + peer_off;
                mbar_arrive_expect_tx_cluster(rbar, 768);
                bulk_copy_to_cluster(smem_u32(sm.beta[sc]) + peer_off, smem_u32(sm.beta[sc]), 256, rbar);
                bulk_copy_to_cluster(smem_u32(sm.gam[sc]) + peer_off, smem_u32(sm.gam[sc]), 256, rbar);
                bulk_copy_to_cluster(smem_u32(sm.dec[sc]) + peer_off, smem_u32(sm.dec[sc]), 256, rbar);
                mbar_arrive(&sm.bar[B_SCAL_READY0 + (c & 3)]);
            }

            // ---- T = (I + B X)^-1 ----------------------------------------------------------------------------
            const float *bet = sm.beta[sc];
            if (pt < 64) substitute_diag_blocks(sm.tl, bet, pt);
            pg_sync();
            merge_level<8>(sm.tl, sm.mm, bet, pt);
            merge_level<16>(sm.tl, sm.mm, bet, pt);
            merge_level<32>(sm.tl, sm.mm, bet, pt);
            // ---- T as bf16 hi/lo operand tiles, once MMA-3(c-1) of both CTAs has read the previous ones ------------
            bool okd = true;
            if (c > 0 && pt >= PG_T - 32) okd = wait(B_T_FREE0 + ((c - 1) & 1), (uint32_t)(((c - 1) >> 1) & 1));
            if (pg_any(!okd)) break;
            write_t_tiles(sm, pt);
            fence_async_smem();
            pg_sync();  // every tile write is done (and the solve matrix may be reused by this CTA's next chunk)
            if (pt == 0) {
                // this CTA's copy is ready; the peer's is sent by the copy engine and counted on its barrier
                const uint32_t rbar = smem_u32(&sm.bar[B_T_READY]) + peer_off;
                mbar_arrive_expect_tx_cluster(rbar, 16384);
                bulk_copy_to_cluster(smem_u32(sm.t_hi) + peer_off, smem_u32(sm.t_hi), 16384, rbar);   // t_hi and t_lo
                mbar_arrive(&sm.bar[B_T_READY]);
            }

            // ---- P(c) = A o Q K^T as bf16 hi/lo operand tiles into both CTAs (rows of Q K^T: warps 2, 3, 6, 7) --------
            if (!is_g && !no_out) {
                okp = wait(B_D1_DONE0 + b1, ph1);
                // MMA-4(c-1) of both CTAs has read the P tiles
                if (okp && c > 0) okp = wait(B_P_FREE0 + ((c - 1) & 1), (uint32_t)(((c - 1) >> 1) & 1));
                if (okp) {
                    tc_fence_after();
                    form_p_row(sm, sc, i, chh, live, tm_lane + TM_D1 + (uint32_t)b1 * 64 + chh * 32);
                    tc_fence_before();
                    fence_async_smem();
                    warp_arrive(B_D1_FREE0 + b1);
                }
                // the four P warps meet (also when a wait gave up: nobody is left behind), then one thread publishes
                asm volatile("bar.sync 4, 128;" ::: "memory");
                if (okp && q == 2 && chh == 0 && lane == 0) {
                    const uint32_t rbar = smem_u32(&sm.bar[B_P_READY]) + peer_off;
                    mbar_arrive_expect_tx_cluster(rbar, 16384);
                    bulk_copy_to_cluster(smem_u32(sm.p_hi) + peer_off, smem_u32(sm.p_hi), 16384, rbar);   // p_hi and p_lo
                    mbar_arrive(&sm.bar[B_P_READY]);
                }
            }
        }
    } else if (warp >= PG_BASE / 32) {
        // =============================== pre group ==========================================================
        // Warps 0, 1, 4, 5 hold rows of K K^T (TMEM lanes 0..63), warps 2, 3, 6, 7 rows of Q K^T (lanes 64..127).
        // Iteration c: the first set forms X(c) while the second forms P(c-1); then all eight warps invert.
        const int pt = tid - PG_BASE;             // 0..255
        const int q = warp & 3, chh = (warp - PG_BASE / 32) >> 2;  // TMEM lane quadrant, column half of D1
        const bool is_g = q < 2;
        const int i = (q & 1) * 32 + lane;        // row of K K^T or of Q K^T held by this thread
        const bool live = chh <= (q & 1);         // otherwise all 32 columns are above the diagonal
        const bool scan_warp = q == 0 && chh == 1;         // K K^T rows 0..31 x columns 32..63: no X work
        float la_next0 = 0.f, la_next1 = 0.f, eta_next = 0.f;
        auto fetch_gates = [&](int c) {
            if (scan_warp) {
                const int t = c * C + 2 * lane;
                la_next0 = (t < len) ? p.log_alpha[(size_t)(tok0 + t) * p.H + h] : 0.f;
                la_next1 = (t + 1 < len) ? p.log_alpha[(size_t)(tok0 + t + 1) * p.H + h] : 0.f;
            }
            if (is_g && chh == q) {   // the thread whose 32 columns contain the diagonal element of its row
                const int t = c * C + i;
                eta_next = (t < len) ? p.eta[(size_t)(tok0 + t) * p.H + h] : 0.f;
            }
        };
        // P(c) = A o Q K^T as bf16 hi/lo operand tiles (rows of Q K^T: warps 2, 3, 6, 7 only)
        auto form_p = [&](int c) -> bool {
            // D1(c) complete; the P tiles are free once MMA-4(c-1) has read them
            bool okp = wait(B_D1_DONE0 + (c & 1), (uint32_t)((c >> 1) & 1));
            if (okp && c > 0) okp = wait(B_D4_DONE, (uint32_t)((c - 1) & 1));
            if (!okp) return false;
            tc_fence_after();
            const int sc = c % NSTAGE;
            form_p_row(sm, sc, i, chh, live, tm_lane + TM_D1 + (uint32_t)(c & 1) * 64 + chh * 32);
            if constexpr (VAR) if ((p.variant & VARIANT_QNORM) && chh == 0) {
                // ||q_i||^2 from row i of the Q tile (still resident: its stage is refilled only after MMA-4(c))
                const unsigned char *qt = sm.kq[sc];
                float n = 0.f;
#pragma unroll 1
                for (int e = 0; e < KB * 8; ++e) {
                    const uint4 raw = *reinterpret_cast<const uint4 *>(qt + (e >> 3) * 16384 + 8192 + sw128(i, e & 7));
                    const __nv_bfloat162 *h2 = reinterpret_cast<const __nv_bfloat162 *>(&raw);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const float2 f = __bfloat1622float2(h2[u]);
                        n += f.x * f.x + f.y * f.y;
                    }
                }
                sm.qn[sc][i] = 1.f / sqrtf(n);
            }
            tc_fence_before();
            fence_async_smem();
            warp_arrive(B_D1_FREE0 + (c & 1));
            warp_arrive(B_P_READY);
            return true;
        };
        // barrier over the four K K^T warps (128 threads) that also ORs a flag
        auto kk_any = [&](bool flag) -> bool {
            uint32_t r;
            asm volatile(
                "{\n\t.reg .pred p, q;\n\tsetp.ne.u32 p, %1, 0;\n\t"
                "bar.red.or.pred q, 5, 128, p;\n\tselp.u32 %0, 1, 0, q;\n\t}"
                : "=r"(r)
                : "r"((uint32_t)flag)
                : "memory");
            return r != 0;
        };
        fetch_gates(0);
        int c = 0;
        for (; c < nchunks; ++c) {
            const uint32_t ph = (uint32_t)(c & 1);
            const int rows = (c == nchunks - 1) ? last_rows : C;
            const int sc = c % NSTAGE;
            const float la0 = la_next0, la1 = la_next1, eta_cur = eta_next;
            if (c + 1 < nchunks) fetch_gates(c + 1);
            // ---- g_i (chunk-local running sum of log alpha), gamma_i, exp(g_C - g_i) -----------------------------
            if (scan_warp) {
                decay_scan(sm, sc, lane, la0, la1);
            }
            bool okc = true;
            if (rows < C) {
                // last chunk: rows past the end of the sequence hold a neighbour's tokens (or TMA zero
                // fill); zero them so that they are inert in every product
                okc = wait(B_FULL0 + sc, (uint32_t)((c / NSTAGE) & 1));
                if (okc) {
                    zero_tail_rows<KB>(sm.kq[sc], rows, pt);
                    fence_async_smem();
                    warp_arrive(B_TAIL_READY);
                }
            }
            if (pg_any(!okc)) break;   // also publishes the decay sums to the whole group
            if (is_g) {
                // ---- X = A^- o K K^T from MMA-1 (this thread: row i, 32 columns) and beta_i ----------------------------
                okc = wait(B_D1_DONE0 + (c & 1), (uint32_t)((c >> 1) & 1));
                if (okc) {
                    tc_fence_after();
                    if (live) {
                        // G_ii = ||k_i||^2 comes with the row
                        const float dg = form_x_row(sm, sc, i, chh, tm_lane + TM_D1 + (uint32_t)(c & 1) * 64 + chh * 32);
                        // beta_i = eta_i / (||k_i||^2 + eps), Eq. 3; rows past the end of the sequence get 0
                        if (chh == q) {
                            if constexpr (VAR) sm.beta[sc][i] = (i < rows) ? ((p.variant & VARIANT_COEFF_ETA) ? eta_cur : eta_cur / (dg + p.eps)) : 0.f;
                            else sm.beta[sc][i] = (i < rows) ? eta_cur / (dg + p.eps) : 0.f;
                        }
                    }
                    tc_fence_before();
                    warp_arrive(B_D1_FREE0 + (c & 1));
                }
                // ---- T = (I + B X)^-1, first the 8x8 diagonal blocks by substitution.  The four K K^T warps go on to
                // them at once (forming P takes the Q K^T warps almost twice as long as X takes these): they meet,
                // two of them substitute, and the one with no X work takes the wait that guards the T tiles
                // (MMA-3(c-1) must have read the previous ones; the first look at a barrier completed by the tensor pipe
                // costs several hundred cycles wherever it is taken, so it is taken here).  Letting these four warps
                // do the block merges at sizes 8 and 16 as well (work for 64 and 128 threads) made them the longer half.
                if (!kk_any(!okc)) {
                    const int gt = (chh * 2 + (q & 1)) * 32 + lane;   // 0..127 over the four warps
                    if (gt < 64) substitute_diag_blocks(sm.tl, sm.beta[sc], gt);
                    if (c > 0 && scan_warp) okc = wait(B_D3_DONE, ph ^ 1);
                } else {
                    okc = false;
                }
            } else if (no_out) {
                warp_arrive(B_D1_FREE0 + (c & 1));   // nothing reads Q K^T: release this warp's share of D1(c)
            } else if (c > 0) {
                okc = form_p(c - 1);
            }
            if (pg_any(!okc)) break;   // X, the diagonal blocks and P(c-1) are done

            // ---- then the off-diagonal blocks T_10 = -T_11 (B_1 X_10 T_00) at block sizes 8, 16, 32 -------------------
            const float *bet = sm.beta[sc];
            merge_level<8>(sm.tl, sm.mm, bet, pt);
            merge_level<16>(sm.tl, sm.mm, bet, pt);
            merge_level<32>(sm.tl, sm.mm, bet, pt);
            // ---- write T as bf16 hi/lo operand tiles, after MMA-3(c-1) has read the previous ones ----------------------
            write_t_tiles(sm, pt);
            fence_async_smem();
            pg_sync();  // the solve matrix is reused by the next chunk
            warp_arrive(B_T_READY);
        }
        // P of the last chunk
        if (c == nchunks && !is_g && !no_out) form_p(nchunks - 1);
    } else {
        // =============================== chain group ==========================================================
        const int ct = tid - CG_BASE;           // 0..255
        const int q = warp & 3;                 // TMEM lane quadrant
        const int hf = ct >> 7;                 // column half: 0 -> columns 0..31, 1 -> 32..63
        const int srow = q * 32 + lane;         // state row (M = 128 accumulator layout, 32x32b loads)
        const bool s_act = srow < D;
        // M = 64 accumulators, 16x256b loads: rows i0 and i0 + 8, column pairs cp + 8j (j = 0..3), cp = hf * 32 + 2 (lane % 4)
        const int i0 = q * 16 + (lane >> 2), i1 = i0 + 8;
        const uint32_t tm16 = tmem + ((uint32_t)(q * 32) << 16) + hf * 32;

        float S[32];
        if (is_map) {
            // transition map: start from the identity (columns sl * NS + hf * 32 .. of I)
#pragma unroll
            for (int c = 0; c < 32; ++c) S[c] = (srow == sl * NS + hf * 32 + c) ? 1.f : 0.f;
        } else if (s_act && init) {
#pragma unroll
            for (int c = 0; c < 32; c += 4) {
                const float4 x = *reinterpret_cast<const float4 *>(init + init_off + (size_t)srow * D + hf * 32 + c);
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
        // byte offset of this thread's bf16 pair j (columns cp + 8j, cp + 8j + 1) of row i inside the
        // 64-token x 64-column B-operand tiles
        const uint32_t lo4 = 4 * (lane & 3);
        auto off = [&](int i, int j) -> uint32_t { return sw128(i, hf * 4 + j) + lo4; };
        store_state_tiles();

        for (int c = 0; c < nchunks; ++c) {
            const uint32_t ph = (uint32_t)(c & 1);
            const int rows = (c == nchunks - 1) ? last_rows : C;
            const int sc = c % NSTAGE;
            // ---- rhs = B (V - D_gamma K S_0) ------------------------------------------------------------------
            if (!(PAIR ? wait(B_SCAL_READY0 + (c & 3), (uint32_t)((c >> 2) & 1)) : wait(B_T_READY, ph))) break;   // scalars of chunk c
            const float b0 = sm.beta[sc][i0], b1 = sm.beta[sc][i1];
            const float g0 = sm.gam[sc][i0], g1 = sm.gam[sc][i1];
            const float d0 = sm.dec[sc][i0], d1 = sm.dec[sc][i1];
            const float gC = sm.gam[sc][C - 1];
            if (!wait(B_V_FULL, ph)) break;
            if (!wait(B_D2_DONE, ph)) break;
            tc_fence_after();
#pragma unroll 1
            for (int j = 0; j < 4; ++j) {
                float acc[4];
                tmem_ld16x256b_x1(tm16 + TM_KS + 8 * j, acc);
                const uint32_t o0 = off(i0, j), o1 = o0 + 8 * 128;   // i1 = i0 + 8: same swizzle phase, eight rows on
                // V[i0][cp + 8j .. +1], V[i1][...]; rows past the end of the sequence are another sequence's tokens
                const uint32_t va = (i0 < rows && !is_map) ? *reinterpret_cast<const uint32_t *>(sm.vt + o0) : 0u;
                const uint32_t vb = (i1 < rows && !is_map) ? *reinterpret_cast<const uint32_t *>(sm.vt + o1) : 0u;
                const float2 fa = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&va));
                const float2 fb = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&vb));
                uint32_t hi, lo;
                split2(b0 * (fa.x - g0 * acc[0]), b0 * (fa.y - g0 * acc[1]), hi, lo);
                *reinterpret_cast<uint32_t *>(sm.ru_hi + o0) = hi;
                *reinterpret_cast<uint32_t *>(sm.ru_lo + o0) = lo;
                split2(b1 * (fb.x - g1 * acc[2]), b1 * (fb.y - g1 * acc[3]), hi, lo);
                *reinterpret_cast<uint32_t *>(sm.ru_hi + o1) = hi;
                *reinterpret_cast<uint32_t *>(sm.ru_lo + o1) = lo;
            }
            fence_async_smem();
            tc_fence_before();
            warp_arrive(B_RHS_READY);

            // ---- D U as hi/lo operand: of the state update and, against P D^-1, of the outputs --------------------------------
            if (!wait(B_D3_DONE, ph)) break;
            tc_fence_after();
#pragma unroll 1
            for (int j = 0; j < 4; ++j) {
                float acc[4];
                tmem_ld16x256b_x1(tm16 + TM_U + 8 * j, acc);
                const uint32_t o0 = off(i0, j), o1 = o0 + 8 * 128;   // i1 = i0 + 8: same swizzle phase, eight rows on
                uint32_t hi, lo;
                split2(d0 * acc[0], d0 * acc[1], hi, lo);
                *reinterpret_cast<uint32_t *>(sm.du_hi + o0) = hi;
                *reinterpret_cast<uint32_t *>(sm.du_lo + o0) = lo;
                split2(d1 * acc[2], d1 * acc[3], hi, lo);
                *reinterpret_cast<uint32_t *>(sm.du_hi + o1) = hi;
                *reinterpret_cast<uint32_t *>(sm.du_lo + o1) = lo;
            }
            fence_async_smem();
            tc_fence_before();
            warp_arrive(B_U_READY);

            // ---- state: S <- gamma_C S + K^T (D U) -----------------------------------------------------------------
            if (!wait(B_D5_DONE, ph)) break;
            if constexpr (PAIR) {
                // MMA-5(c) was the last reader of the K/Q stage of chunk c: refill it at once (this CTA's MMA-1 of
                // chunk c + 3 may be due within a fraction of a chunk period)
                if (ct == 0 && c + NSTAGE < nchunks) {
                    const int cn = c + NSTAGE;
                    mbar_expect_tx(&sm.bar[B_FULL0 + sc], STAGE_BYTES);
#pragma unroll
                    for (int kb = 0; kb < KB; ++kb) {
                        tma_load_2d(sm.kq[sc] + kb * 16384, &tm_k, h * D + kb * 64, tok0 + cn * C, &sm.bar[B_FULL0 + sc]);
                        tma_load_2d(sm.kq[sc] + kb * 16384 + 8192, &tm_q, h * D + kb * 64, tok0 + cn * C, &sm.bar[B_FULL0 + sc]);
                    }
                }
            }
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
            if (no_out) continue;
            if (!wait(B_D4_DONE, ph)) break;
            tc_fence_after();
            const int rows_out = c < first_out ? 0 : rows;   // warm-up chunks are computed like any other and not stored
            {
                // This thread's accumulator values are column pairs cp + 8j (j = 0..3) of rows i0 and i1; a 4 x 4 transpose
                // over the four lanes of a quad gives each lane 8 consecutive columns of both rows, so that every
                // store is 16 bytes and a warp's store covers whole 32-byte sectors (2-element stores straight from the
                // accumulator layout backed up the store queue for more than a thousand cycles per chunk).
                float pu[16], qs[16];
                tmem_ld16x256b_x4(tm16 + TM_PU, pu);
                tmem_ld16x256b_x4(tm16 + ((c & 1) ? TM_QS1 : TM_QS0), qs);
                float n0 = g0, n1 = g1, m0 = 1.f, m1 = 1.f;   // o = n * qs + m * pu
                if constexpr (VAR) {
                    if (p.variant & VARIANT_QNORM) {   // read-out over ||q||
                        m0 = sm.qn[sc][i0]; m1 = sm.qn[sc][i1];
                        n0 *= m0; n1 *= m1;
                    }
                }
                const int t4 = lane & 3;
                const size_t col = (size_t)sl * NS + hf * 32 + 8 * t4;
                OUT *o0 = reinterpret_cast<OUT *>(p.out) + ((size_t)(tok0 + c * C + i0) * p.H + h) * D + col;
                OUT *o1 = reinterpret_cast<OUT *>(p.out) + ((size_t)(tok0 + c * C + i1) * p.H + h) * D + col;
                if constexpr (sizeof(OUT) == 2) {
                    uint32_t a[4], b[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const __nv_bfloat162 x = __floats2bfloat162_rn(n0 * qs[4 * j] + m0 * pu[4 * j], n0 * qs[4 * j + 1] + m0 * pu[4 * j + 1]);
                        const __nv_bfloat162 y = __floats2bfloat162_rn(n1 * qs[4 * j + 2] + m1 * pu[4 * j + 2], n1 * qs[4 * j + 3] + m1 * pu[4 * j + 3]);
                        a[j] = *reinterpret_cast<const uint32_t *>(&x);
                        b[j] = *reinterpret_cast<const uint32_t *>(&y);
                    }
                    quad_transpose(a, t4);
                    quad_transpose(b, t4);
                    if (i0 < rows_out) *reinterpret_cast<uint4 *>(o0) = make_uint4(a[0], a[1], a[2], a[3]);
                    if (i1 < rows_out) *reinterpret_cast<uint4 *>(o1) = make_uint4(b[0], b[1], b[2], b[3]);
                } else {
                    uint32_t ax[4], ay[4], bx[4], by[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        ax[j] = __float_as_uint(n0 * qs[4 * j] + m0 * pu[4 * j]);
                        ay[j] = __float_as_uint(n0 * qs[4 * j + 1] + m0 * pu[4 * j + 1]);
                        bx[j] = __float_as_uint(n1 * qs[4 * j + 2] + m1 * pu[4 * j + 2]);
                        by[j] = __float_as_uint(n1 * qs[4 * j + 3] + m1 * pu[4 * j + 3]);
                    }
                    quad_transpose(ax, t4);
                    quad_transpose(ay, t4);
                    quad_transpose(bx, t4);
                    quad_transpose(by, t4);
                    if (i0 < rows_out) {
                        *reinterpret_cast<uint4 *>(o0) = make_uint4(ax[0], ay[0], ax[1], ay[1]);
                        *reinterpret_cast<uint4 *>(o0 + 4) = make_uint4(ax[2], ay[2], ax[3], ay[3]);
                    }
                    if (i1 < rows_out) {
                        *reinterpret_cast<uint4 *>(o1) = make_uint4(bx[0], by[0], bx[1], by[1]);
                        *reinterpret_cast<uint4 *>(o1 + 4) = make_uint4(bx[2], by[2], bx[3], by[3]);
                    }
                }
            }
            tc_fence_before();
        }
        if (!sm.abort_flag && fin && s_act) {
#pragma unroll
            for (int c = 0; c < 32; c += 4)
                *reinterpret_cast<float4 *>(fin + fin_off + (size_t)srow * D + hf * 32 + c) =
                    make_float4(S[c], S[c + 1], S[c + 2], S[c + 3]);
        }
    }

    tc_fence_before();
    __syncthreads();
    // Neither CTA of a pair leaves while the other may still write into its shared memory or signal its barriers.
    // On the normal path everything sent has been waited for by its receiver; after a wait gave up, copies and
    // completion signals issued just before may still be on their way (microseconds): let them land first.
    if constexpr (PAIR) {
        if (sm.abort_flag)
            for (int i = 0; i < 32; ++i) __nanosleep(1000);
        cluster_sync_all();
    }
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

template <int D, typename OUT, bool VAR, bool PAIR>
cudaError_t launch_v(const ChunkParams &p, cudaStream_t stream);

template <int D, typename OUT>
cudaError_t launch_t(const ChunkParams &p, cudaStream_t stream)
{
    const int32_t v = p.variant & ~(VARIANT_NO_PAIR | VARIANT_WY);
    // two slices per head: the CTAs of a head run as a cluster and share the state-independent work (the layer-edge
    // variants are implemented in the unpaired kernel only; the error-path test hook in both)
    if constexpr (D == 2 * NS) {
        if (!(p.variant & VARIANT_NO_PAIR)) {
            if (v == 0) return launch_v<D, OUT, false, true>(p, stream);
            if (v == VARIANT_TEST_TIMEOUT) return launch_v<D, OUT, true, true>(p, stream);
        }
    }
    return v != 0 ? launch_v<D, OUT, true, false>(p, stream) : launch_v<D, OUT, false, false>(p, stream);
}

template <int D, typename OUT, bool VAR, bool PAIR>
cudaError_t launch_v(const ChunkParams &p, cudaStream_t stream)
{
    using Smem = TcSmem<D>;
    const uint64_t n_tok = (uint64_t)p.B * p.T;
    CUtensorMap tq, tk, tv;
    if (!make_tmap(&tq, p.q, n_tok, (uint64_t)p.H * D) || !make_tmap(&tk, p.k, n_tok, (uint64_t)p.H * D) ||
        !make_tmap(&tv, p.v, n_tok, (uint64_t)p.H * D))
        return cudaErrorInvalidValue;
    auto kern = kla_chunk_tc_kernel<D, OUT, VAR, PAIR>;
    const int smem = (int)sizeof(Smem) + 1024;
    cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (err != cudaSuccess) return err;
    // segment pass 1: (seg_G - 1) segments per sequence, twice the slices; p.n_seq counts all segments there
    const int grid = p.seg_pass == 1 ? (p.n_seq / p.seg_G) * (p.seg_G - 1) * p.H * 2 * (D / NS) : p.n_seq * p.H * (D / NS);
    if (grid == 0) return cudaSuccess;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(NT);
    cfg.dynamicSmemBytes = (size_t)smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;   // blocks 2j, 2j + 1 = the two slices of one (sequence, head)
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = PAIR ? 1 : 0;
    err = cudaLaunchKernelEx(&cfg, kern, tq, tk, tv, p);
    count_launch(1);
    return err != cudaSuccess ? err : cudaGetLastError();
}

}  // namespace

bool chunk_tc_supported(int d, int chunk, int io_dtype)
{
    return (d == 64 || d == 128) && chunk == 64 && io_dtype == KLA_BF16;
}

cudaError_t launch_chunk_tc(const ChunkParams &p, int d, int io_dtype, int out_dtype, cudaStream_t stream)
{
    (void)io_dtype;
    if (d == 128 && (p.variant & VARIANT_WY)) return launch_chunk_wy(p, out_dtype, stream);
    if (d == 128) {
        if (out_dtype == KLA_BF16) return launch_t<128, __nv_bfloat16>(p, stream);
        return launch_t<128, float>(p, stream);
    }
    if (out_dtype == KLA_BF16) return launch_t<64, __nv_bfloat16>(p, stream);
    return launch_t<64, float>(p, stream);
}

}  // namespace kla
