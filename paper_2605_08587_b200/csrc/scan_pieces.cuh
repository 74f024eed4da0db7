// Warp-level pieces shared by the token-by-token kernels (dg_scan.cu, bwd_scan.cu): one warp owns WC columns of a
// d x d state, lane l holds rows l, l + 32, ... of those columns in registers.
#pragma once
#include "common.cuh"

namespace kla {

// Sums over the warp of x[0..WC-1] (WC = 4 or 8 state columns per warp), by halving: afterwards every lane holds the
// complete sum of column col_of_lane<WC>(lane).
template <int WC>
__device__ __forceinline__ int col_of_lane(int lane) { return WC == 8 ? (lane >> 2) & 7 : (lane >> 3) & 3; }
template <int WC>
__device__ __forceinline__ int lane_of_col(int c) { return WC == 8 ? c << 2 : c << 3; }
template <int WC>
__device__ __forceinline__ float reduce_scatter(const float (&x)[WC], int lane)
{
    float y[WC];
#pragma unroll
    for (int i = 0; i < WC; ++i) y[i] = x[i];
    int n = WC, off = 16;
#pragma unroll
    for (; n > 1; n >>= 1, off >>= 1) {   // halve the number of columns held, summing with the partner that keeps the other half
        const bool hi = lane & off;
#pragma unroll
        for (int i = 0; i < n / 2; ++i) {
            const float keep = hi ? y[n / 2 + i] : y[i], give = hi ? y[i] : y[n / 2 + i];
            y[i] = keep + __shfl_xor_sync(0xffffffffu, give, off);
        }
    }
    float w = y[0];
#pragma unroll
    for (; off > 0; off >>= 1) w += __shfl_xor_sync(0xffffffffu, w, off);
    return w;
}
__device__ __forceinline__ float warp_sum(float x)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}

// Packed fp32 arithmetic (two lanes of one instruction, sm_100): the token-by-token kernels are bound by instruction issue,
// and their inner loops run over pairs of adjacent state columns.
__device__ __forceinline__ float2 f2(float a, float b) { return make_float2(a, b); }
__device__ __forceinline__ float2 f2(float a) { return make_float2(a, a); }
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) { return __ffma2_rn(a, b, c); }
__device__ __forceinline__ float2 mul2(float2 a, float2 b) { return __fmul2_rn(a, b); }
__device__ __forceinline__ float2 add2(float2 a, float2 b) { return __fadd2_rn(a, b); }

}  // namespace kla
