// Segment-parallel scan: the small kernels around the chunk kernel.
//
// Every chunk step is affine in the incoming state (Eqs. 7-9 are linear in S_0), so a run of chunks is too:
//     S_end = Phi S_start + N,   Phi (d_k x d_k) = the state reached from the identity with v = 0,
//                                N   (d_k x d_v) = the state reached from zero.
// A long sequence is cut into G segments; pass 1 (the chunk kernel, no outputs) finds (Phi, N) of every segment
// but the last in parallel; `seg_combine` below chains them serially -- G - 1 small fp32 products per head --
// to get each segment's true start state; pass 3 (the chunk kernel again) then runs all segments in parallel.
#include "common.cuh"

namespace kla {

namespace {

// Segment bounds, and after them the plan word (cu_seg[B G + 1]): 1 = the segments are to start from decay-bounded warm-up
// runs unless seg_warm_plan_kernel finds a reason against it, 0 = from chained transition maps.
__global__ void seg_bounds_kernel(int32_t *cu_seg, int B, int T, int G, int seg_len, int try_warm)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i > B * G + 1) return;
    if (i == B * G + 1) {
        cu_seg[i] = try_warm;
        return;
    }
    if (i == B * G) {
        cu_seg[i] = B * T;
        return;
    }
    const int b = i / G, g = i % G;
    cu_seg[i] = b * T + min(g * seg_len, T);
}

// Decay-bounded segment starts.  The state map over a run of tokens is Phi = prod_t alpha_t (I - beta_t k_t k_t^T); every
// factor is symmetric with eigenvalues alpha_t and alpha_t (1 - beta_t ||k_t||^2), and beta_t ||k_t||^2 = eta_t ||k_t||^2 /
// (||k_t||^2 + eps) lies in [0, eta_t] (Eq. 3), so for 0 <= eta_t <= 2 the factor's norm is at most alpha_t and
// ||Phi||_2 <= exp(sum_t log alpha_t).  A segment that is run from the ZERO state starting w chunks early therefore reaches
// its first token with an error of at most exp(sum of log alpha over those w chunks) x ||S||: with the sum below -40
// (4e-18) that is nothing in fp32, and the segment needs neither its predecessors' transition maps nor a second pass.
// One warp per (segment, head): warm[(n H + h)] = the smallest such w, at most max_warm chunks; if there is none, or if
// any eta is outside [0, 2] (blocks past the planning warps check eta), the plan word is cleared and the transition-map
// passes run instead.
constexpr float WARM_LOG_DECAY = -40.f;
__global__ void seg_warm_plan_kernel(int32_t *cu_seg, const float *log_alpha, const float *eta, int n_seg, int G, int H,
                                     int max_warm, int plan_blocks, long long n_gate, const int32_t *unit_seq)
{
    int32_t *plan = cu_seg + n_seg + 1, *warm = cu_seg + n_seg + 2;
    if ((int)blockIdx.x >= plan_blocks) {   // eta in [0, 2] everywhere (a NaN fails the test)
        bool bad = false;
        for (long long i = (long long)(blockIdx.x - plan_blocks) * blockDim.x + threadIdx.x; i < n_gate;
             i += (long long)(gridDim.x - plan_blocks) * blockDim.x) {
            const float e = eta[i];
            bad |= !(e >= 0.f && e <= 2.f);
        }
        if (bad) *plan = 0;
        return;
    }
    const int unit = blockIdx.x * (blockDim.x / 32) + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (unit >= n_seg * H) return;
    const int n = unit / H, h = unit % H;
    // a sequence's first piece starts from the initial state: G equal segments per sequence, or (packed input) the table
    if (unit_seq ? (unit_seq[n] >> 29) & 1 : n % G == 0) {
        if (lane == 0) warm[unit] = 0;
        return;
    }
    const int start = cu_seg[n];   // first token of the segment (a multiple of 64 tokens into its sequence)
    float acc = 0.f;
    int w = 0;
    while (w < max_warm && acc > WARM_LOG_DECAY) {
        ++w;
        const size_t t = (size_t)(start - w * 64 + 2 * lane);
        float x = log_alpha[t * H + h] + log_alpha[(t + 1) * H + h];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
        acc += x;
    }
    if (lane == 0) {
        warm[unit] = w;
        if (!(acc <= WARM_LOG_DECAY)) *plan = 0;   // (also when a gate is NaN)
    }
}

// Packed input: every sequence longer than seg_len tokens is cut into pieces of seg_len (the last one shorter).  One block.
//   ub[u], ub[u + 1]   token range of piece u (pieces tile the packed token axis; empty sequences have none)
//   ub[n_units + 1]    plan word, set to 1 (seg_warm_plan_kernel may clear it)
//   unit_seq[u]        sequence of piece u | first piece << 29 | last piece << 30
// Empty sequences get their final state here (no piece will write it).
constexpr int MAX_PACKED_SEQ = 4096;
__global__ void __launch_bounds__(256) packed_units_kernel(const int32_t *cu_seqlens, int n_seq, int seg_len, int n_units,
                                                           int32_t *ub, int32_t *unit_seq, const float *init_state,
                                                           float *final_state, int state_elems)
{
    __shared__ int first_unit[MAX_PACKED_SEQ + 1];
    for (int n = threadIdx.x; n < n_seq; n += blockDim.x) {
        const int len = cu_seqlens[n + 1] - cu_seqlens[n];
        first_unit[n + 1] = (len + seg_len - 1) / seg_len;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        first_unit[0] = 0;
        for (int n = 0; n < n_seq; ++n) first_unit[n + 1] += first_unit[n];
        ub[n_units] = cu_seqlens[n_seq];
        ub[n_units + 1] = 1;
    }
    __syncthreads();
    for (int n = threadIdx.x; n < n_seq; n += blockDim.x) {
        const int t0 = cu_seqlens[n], t1 = cu_seqlens[n + 1], u0 = first_unit[n], cnt = first_unit[n + 1] - u0;
        for (int g = 0; g < cnt; ++g) {
            ub[u0 + g] = t0 + g * seg_len;
            unit_seq[u0 + g] = n | (g == 0 ? 1 << 29 : 0) | (g == cnt - 1 ? 1 << 30 : 0);
        }
        (void)t1;
    }
    if (final_state) {
        for (int n = 0; n < n_seq; ++n) {
            if (cu_seqlens[n + 1] != cu_seqlens[n]) continue;
            for (int i = threadIdx.x; i < state_elems; i += blockDim.x)
                final_state[(size_t)n * state_elems + i] = init_state ? init_state[(size_t)n * state_elems + i] : 0.f;
        }
    }
}

// Rank of every sequence by decreasing length (ties by index): order[rank] = sequence.
__global__ void seq_order_kernel(const int32_t *cu_seqlens, int n_seq, int32_t *order)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_seq) return;
    const int li = cu_seqlens[i + 1] - cu_seqlens[i];
    int rank = 0;
    for (int j = 0; j < n_seq; ++j) {
        const int lj = cu_seqlens[j + 1] - cu_seqlens[j];
        rank += (lj > li || (lj == li && j < i)) ? 1 : 0;
    }
    order[rank] = i;
}

// One CTA per (sequence, head, 16-column slice of the state); thread r owns row r of the slice.
template <int D>
__global__ void __launch_bounds__(D) seg_combine_kernel(const float *init_state, const float *map, const float *local,
                                                        float *start, int H, int G, const int32_t *skip_if_one)
{
    if (skip_if_one && *skip_if_one == 1) return;   // the segments start from warm-up runs: no maps to chain
    constexpr int W = 16;
    const int sl = blockIdx.x % (D / W);
    const int h = (blockIdx.x / (D / W)) % H;
    const int b = blockIdx.x / ((D / W) * H);
    const int r = threadIdx.x;
    __shared__ __align__(16) float S[2][D][W];

    auto base = [&](int g) -> size_t { return ((size_t)(b * G + g) * H + h) * D * D; };
    float cur[W];
#pragma unroll
    for (int c = 0; c < W; c += 4) {
        float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
        if (init_state) x = *reinterpret_cast<const float4 *>(init_state + ((size_t)b * H + h) * D * D + (size_t)r * D + sl * W + c);
        cur[c] = x.x; cur[c + 1] = x.y; cur[c + 2] = x.z; cur[c + 3] = x.w;
    }
    for (int g = 0; g < G; ++g) {
        // publish the start state of segment g
        float *dst = start + base(g) + (size_t)r * D + sl * W;
#pragma unroll
        for (int c = 0; c < W; c += 4) {
            const float4 x = make_float4(cur[c], cur[c + 1], cur[c + 2], cur[c + 3]);
            *reinterpret_cast<float4 *>(dst + c) = x;
            *reinterpret_cast<float4 *>(&S[g & 1][r][c]) = x;
        }
        if (g + 1 == G) break;
        __syncthreads();
        // next = Phi_g cur + N_g
        const float *Mrow = map + base(g) + (size_t)r * D;
        const float *Nrow = local + base(g) + (size_t)r * D + sl * W;
        float acc[W];
#pragma unroll
        for (int c = 0; c < W; c += 4) {
            const float4 x = *reinterpret_cast<const float4 *>(Nrow + c);
            acc[c] = x.x; acc[c + 1] = x.y; acc[c + 2] = x.z; acc[c + 3] = x.w;
        }
#pragma unroll 2
        for (int k = 0; k < D; k += 4) {
            const float4 m = *reinterpret_cast<const float4 *>(Mrow + k);
            const float mv[4] = {m.x, m.y, m.z, m.w};
#pragma unroll
            for (int u = 0; u < 4; ++u) {
#pragma unroll
                for (int c = 0; c < W; c += 4) {
                    const float4 s4 = *reinterpret_cast<const float4 *>(&S[g & 1][k + u][c]);
                    acc[c] += mv[u] * s4.x; acc[c + 1] += mv[u] * s4.y; acc[c + 2] += mv[u] * s4.z; acc[c + 3] += mv[u] * s4.w;
                }
            }
        }
#pragma unroll
        for (int c = 0; c < W; ++c) cur[c] = acc[c];
        // the other buffer is written next; readers of this one are done after the next barrier
    }
}

}  // namespace

cudaError_t launch_seg_bounds(int32_t *cu_seg, int B, int T, int G, int seg_len, int try_warm, cudaStream_t stream)
{
    const int n = B * G + 2;
    seg_bounds_kernel<<<(n + 127) / 128, 128, 0, stream>>>(cu_seg, B, T, G, seg_len, try_warm);
    count_launch(1);
    return cudaGetLastError();
}

cudaError_t launch_seg_warm_plan(int32_t *cu_seg, const float *log_alpha, const float *eta, int B, int T, int H, int G,
                                 int seg_len, cudaStream_t stream)
{
    const int n_seg = B * G, plan_blocks = (n_seg * H + 3) / 4;   // four planning warps per block
    const long long n_gate = (long long)B * T * H;
    const int eta_blocks = (int)((n_gate + 128 * 16 - 1) / (128 * 16) < 256 ? (n_gate + 128 * 16 - 1) / (128 * 16) : 256);
    const int max_warm = seg_len / 64 / 2 < 32 ? seg_len / 64 / 2 : 32;   // at most half a segment, and 2048 tokens
    seg_warm_plan_kernel<<<plan_blocks + eta_blocks, 128, 0, stream>>>(cu_seg, log_alpha, eta, n_seg, G, H, max_warm, plan_blocks, n_gate, nullptr);
    count_launch(1);
    return cudaGetLastError();
}

cudaError_t launch_packed_units(const int32_t *cu_seqlens, int n_seq, int seg_len, int n_units, int32_t *ub, int32_t *unit_seq,
                                const float *log_alpha, const float *eta, long long n_tok, int H, const float *init_state,
                                float *final_state, int d, cudaStream_t stream)
{
    if (n_seq > MAX_PACKED_SEQ) return cudaErrorInvalidValue;
    packed_units_kernel<<<1, 256, 0, stream>>>(cu_seqlens, n_seq, seg_len, n_units, ub, unit_seq, init_state, final_state, H * d * d);
    const int plan_blocks = (n_units * H + 3) / 4;
    const long long n_gate = n_tok * H;
    const int eta_blocks = (int)((n_gate + 128 * 16 - 1) / (128 * 16) < 256 ? (n_gate + 128 * 16 - 1) / (128 * 16) : 256);
    const int max_warm = seg_len / 64 / 2 < 32 ? seg_len / 64 / 2 : 32;
    seg_warm_plan_kernel<<<plan_blocks + eta_blocks, 128, 0, stream>>>(ub, log_alpha, eta, n_units, 1, H, max_warm, plan_blocks, n_gate, unit_seq);
    count_launch(2);
    return cudaGetLastError();
}

cudaError_t launch_seq_order(const int32_t *cu_seqlens, int n_seq, int32_t *order, cudaStream_t stream)
{
    seq_order_kernel<<<(n_seq + 127) / 128, 128, 0, stream>>>(cu_seqlens, n_seq, order);
    count_launch(1);
    return cudaGetLastError();
}

cudaError_t launch_seg_combine(const float *init_state, const float *map, const float *local, float *start, int B, int H,
                               int G, int d, const int32_t *skip_if_one, cudaStream_t stream)
{
    if (d == 128)
        seg_combine_kernel<128><<<B * H * (128 / 16), 128, 0, stream>>>(init_state, map, local, start, H, G, skip_if_one);
    else
        seg_combine_kernel<64><<<B * H * (64 / 16), 64, 0, stream>>>(init_state, map, local, start, H, G, skip_if_one);
    count_launch(1);
    return cudaGetLastError();
}

}  // namespace kla
