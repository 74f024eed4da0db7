// Pieces shared by the two tensor-core chunk kernels (chunk_tc.cu: one CTA per state slice, W-free form of
// Algorithm 1 right; chunk_wy.cu: two CTAs per head, WY form): constants, bounded barrier waits, the decay scan, the
// blocked inverse of I + B X in shared memory, tile helpers and the host side of the tensor maps.
#pragma once
#include <cuda.h>

#include <mutex>

#include "common.cuh"
#include "umma.cuh"

namespace kla {
namespace tc {

using namespace umma;

constexpr int C = 64;    // chunk length
constexpr int NS = 64;   // state columns per CTA
constexpr int NSTAGE = 3;
constexpr long long WAIT_LIMIT = 2000000000LL;  // SM clocks (~1 s) before a wait gives up
constexpr float LOG2E = 1.4426950408889634f;
// The write weights exp(g_C - g_j) are kept above 2^-DEC_FLOOR_LOG2 (~1e-35): the output product is taken as
// (P D^-1)(D U), and with the floor neither factor leaves the fp32 / bf16 exponent range however strong the decay.  A
// floored weight puts at most 1e-35 of a token into the state instead of less.
constexpr float DEC_FLOOR_LOG2 = 115.f;

constexpr int LDT = 68;  // row stride (floats) of the fp32 solve matrix
constexpr int LDM = 40;  // row stride of the solve scratch

// Bounded wait on an mbarrier phase that also leaves when another role has aborted.  Every lane of the
// calling warp polls: letting one lane poll and broadcasting the result splits the warp, and each later
// warp-collective instruction (elect.sync, tcgen05.ld) then pays for re-forming it.
// `sleep_ns`: pause between looks.  A polling warp is always ready to issue and takes issue slots and instruction fetches
// from the working warps (a third of all instructions executed were polls): roles whose waits are long and whose
// reaction time does not matter sleep longer.
static __device__ __noinline__ bool bar_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag, unsigned sleep_ns = 32)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    while (true) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i) {
            if (mbar_try_wait(bar, parity)) return true;
            __nanosleep(sleep_ns);
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
static __device__ __noinline__ bool warp_wait(uint64_t *bar, uint32_t parity, volatile int *abort_flag, unsigned sleep_ns = 32)
{
    const bool ok = mbar_try_wait(bar, parity) || bar_wait(bar, parity, abort_flag, sleep_ns);
    return __all_sync(0xffffffffu, ok);
}

// Named barriers of the pre group (256 threads).
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
// one 1 x 4 tile per thread; `mm` (row stride ldm) holds the intermediate product.  Trip counts are warp-uniform.
template <int BS>
__device__ __forceinline__ void merge_level(float *tl, float *mm, int ldm, const float *bet, int pt)
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
        *reinterpret_cast<float4 *>(&mm[R * ldm + c4]) = make_float4(s * acc.x, s * acc.y, s * acc.z, s * acc.w);
    }
    pg_sync();
    if (act) {
        // T_10 = -T_11 M; T_11 is lower triangular: columns k > r of its row r are zero
        const float *Ap = tl + (rb + r) * LDT + rb;
        const float *Bp = mm + (pr * BS) * ldm + c4;
        const int kend = min(BS, (r | RMASK) + 1);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 2
        for (int k = 0; k < kend; k += 4) {
            const float4 a = *reinterpret_cast<const float4 *>(Ap + k);
            const float av[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const float4 b = *reinterpret_cast<const float4 *>(Bp + (k + u) * ldm);
                acc.x += av[u] * b.x; acc.y += av[u] * b.y; acc.z += av[u] * b.z; acc.w += av[u] * b.w;
            }
        }
        *reinterpret_cast<float4 *>(&tl[(rb + r) * LDT + cb + c4]) = make_float4(-acc.x, -acc.y, -acc.z, -acc.w);
    }
    pg_sync();
}

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
// Q tiles of the stage so that they are inert in every product.  All 256 threads of the pre group.
template <int KB>
__device__ __forceinline__ void zero_tail_rows(unsigned char *kq, int rows, int pt)
{
    for (int e = pt; e < (C - rows) * 8; e += 256) {
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
// 16-byte column groups grp0 .. grp1 - 1 (8 columns each) of the MMA-1 accumulator row at tbase (the address of column
// 0 of the row), as bf16 hi/lo operand tiles.  A warp holds 32 consecutive rows; groups above the diagonal for every row
// of the warp are written as zeros without a read (the TMEM load is warp-collective: the test must be warp-uniform).
template <typename Smem>
__device__ __forceinline__ void form_p_row(Smem &sm, int sc, int i, int grp0, int grp1, uint32_t tbase)
{
    const float gi2 = sm.g2[sc][i], gc2 = sm.g2[sc][C - 1];
#pragma unroll 2
    for (int grp = grp0; grp < grp1; ++grp) {
        uint4 hi = make_uint4(0, 0, 0, 0), lo = hi;
        const int j0 = grp * 8;
        if (j0 <= (i | 31)) {
            float a[8];
            tmem_ld8(tbase + j0, a);
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
        *reinterpret_cast<uint4 *>(sm.p_hi + sw128(i, grp)) = hi;
        *reinterpret_cast<uint4 *>(sm.p_lo + sw128(i, grp)) = lo;
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

// ---- host side: tensor maps ---------------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn get_encode_fn()
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
inline bool make_tmap(CUtensorMap *tm, const void *base, uint64_t n_tok, uint64_t row_elems)
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

}  // namespace tc
}  // namespace kla
