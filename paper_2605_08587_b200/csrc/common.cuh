// Shared device/host helpers for the KLA kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kla.h"

namespace kla {

// Everything a chunk-forward kernel needs; passed by value.
struct ChunkParams {
    const void *q, *k, *v;
    const float *log_alpha, *eta;
    const float *init_state;  // may be null
    void *out;
    float *final_state;       // may be null
    const int32_t *cu_seqlens;  // device, may be null (fixed length)
    int32_t *status_word;       // may be null
    int32_t B, T, H, n_seq;
    float eps;
    // Segment-parallel scan (tensor-core kernel only; all zero / null for a plain launch).
    //   seg_pass 1: "sequence" index = a segment that is not the last of its sequence (seg_G segments per
    //               sequence); no outputs; 2x the slices: the extra ones carry the transition map (state
    //               started at the identity, v = 0) and write it to map_state.
    //   seg_pass 3: every segment from its true start state; only the last segment of a sequence writes
    //               final_state, at the sequence's index.
    //   seg_pass 4: every segment but a sequence's first from the zero state, started as many chunks early as the plan
    //               after the segment bounds says (outputs of those chunks are not stored); init_state is per sequence.
    //   seg_pass 5: packed input cut into pieces (launch_packed_units): cu_seqlens = the piece bounds, n_seq = the number of
    //               pieces; the table after the warm-up lengths (cu_seqlens[n_seq + 2 + n_seq H + u]) names each piece's
    //               sequence and says whether it is the first (initial state) and the last (final state) of it.
    //   seg_pass 6: the plain packed launch, taken only if the pieces' plan word, seq_order[seg_G], is 0.
    //   Passes 1 and 3 return at once when the plan word (cu_seqlens[n_seq + 1]) is 1, passes 4 and 5 when it is not.
    int32_t seg_pass, seg_G;
    int32_t variant;     // bit 0: beta_t = eta_t instead of Eq. 3; bit 1: read-out divided by ||q_t||; bit 2: test hook; bits 3, 4: see VARIANT_NO_PAIR, VARIANT_WY
    union {
        float *map_state;            // segment pass 1
        const int32_t *seq_order;    // packed input, plain launch: block b works on sequence seq_order[b] (longest
                                     // first, so that the long sequences do not end up in the last wave); may be null
    };
};
constexpr int32_t VARIANT_COEFF_ETA = 1, VARIANT_QNORM = 2, VARIANT_TEST_TIMEOUT = 4;
constexpr int32_t VARIANT_NO_PAIR = 8;   // host side only: launch the two slices of a head as independent CTAs
constexpr int32_t VARIANT_WY = 16;       // host side only: head dimension 128 goes to the WY-form kernel (chunk_wy.cu)

struct DecodeParams {
    const void *q, *k, *v;
    const float *log_alpha, *eta;
    float *state;
    void *out;
    int32_t BH;
    float eps;
    // 1: q, k, v, log_alpha, eta were complete before the previous kernel on the stream started (later steps of
    // kla_decode_steps), so they may be read while that kernel drains; 0: they may be its outputs
    int32_t inputs_ready;
    int32_t coeff_eta, qnorm;   // as in ChunkParams
};

// Launchers implemented in the kernel translation units.  Each returns cudaGetLastError().
cudaError_t launch_decode(const DecodeParams &p, int d, int io_dtype, int out_dtype,
                          cudaStream_t stream);
cudaError_t launch_chunk_simt(const ChunkParams &p, int d, int chunk, int io_dtype, int out_dtype,
                              cudaStream_t stream);
cudaError_t launch_chunk_tc(const ChunkParams &p, int d, int io_dtype, int out_dtype,
                            cudaStream_t stream);
// Head dimension 128, the two slices of a head as a cluster of two CTAs (chunk_wy.cu); called by launch_chunk_tc.
cudaError_t launch_chunk_wy(const ChunkParams &p, int out_dtype, cudaStream_t stream);
// Segment-parallel helpers (segscan.cu).  cu_seg[b * G + g] = b * T + min(g * seg_len, T), one more entry = B * T.
// After the bounds come the plan word (cu_seg[B G + 1]; `try_warm` is its initial value) and, from cu_seg[B G + 2] on, one
// warm-up length in chunks per (segment, head): seg_plan_ints(B, G, H) int32 in all.
cudaError_t launch_seg_bounds(int32_t *cu_seg, int B, int T, int G, int seg_len, int try_warm, cudaStream_t stream);
inline size_t seg_plan_ints(int B, int G, int H) { return (size_t)B * G + 2 + (size_t)B * G * H; }
// Decides whether the segments may start from decay-bounded warm-up runs and how long each must be (clears the plan word if not).
cudaError_t launch_seg_warm_plan(int32_t *cu_seg, const float *log_alpha, const float *eta, int B, int T, int H, int G,
                                 int seg_len, cudaStream_t stream);
// order[r] = index of the sequence with the r-th largest length (ties by index); n_seq small (quadratic work)
cudaError_t launch_seq_order(const int32_t *cu_seqlens, int n_seq, int32_t *order, cudaStream_t stream);
// start[b, 0] = init (or 0); start[b, g + 1] = map[b, g] . start[b, g] + local[b, g]   (d x d products, fp32)
// Packed input cut into pieces of at most seg_len tokens (n_units of them, counted by the caller from the host copy of the
// offsets): piece bounds ub[n_units + 1], plan word ub[n_units + 1] = 1, warm-up lengths from ub[n_units + 2] on (cleared
// plan word if some piece has none), unit_seq[n_units]; final states of empty sequences.  Two launches.
cudaError_t launch_packed_units(const int32_t *cu_seqlens, int n_seq, int seg_len, int n_units, int32_t *ub, int32_t *unit_seq,
                                const float *log_alpha, const float *eta, long long n_tok, int H, const float *init_state,
                                float *final_state, int d, cudaStream_t stream);
// (`skip_if_one`: null, or a device word; the kernel does nothing when it holds 1)
cudaError_t launch_seg_combine(const float *init_state, const float *map, const float *local, float *start, int B, int H,
                               int G, int d, const int32_t *skip_if_one, cudaStream_t stream);
// Diagonal-gated recurrence, token by token on CUDA cores (dg_scan.cu); log_alpha [n_tok, H, d].
cudaError_t launch_dg_scan(const void *q, const void *k, const void *v, const float *log_alpha, const float *eta,
                           const float *init_state, void *out, float *final_state, const int32_t *cu_seqlens, int T, int H,
                           int n_seq, int d, float eps, int coeff_eta, int qnorm, int io_dtype, int out_dtype, cudaStream_t stream);
// Reverse-mode derivative of the recurrence, token by token on CUDA cores (bwd_scan.cu); gradients in fp32.
size_t bwd_workspace_bytes(int n_seq, long long n_tok, int H, int d);
cudaError_t launch_bwd_scan(const void *q, const void *k, const void *v, const float *log_alpha, const float *eta,
                            const float *init_state, const void *dout, const float *dfinal, float *dq, float *dk, float *dv,
                            float *dlog_alpha, float *deta, float *dinit, void *workspace, const int32_t *cu_seqlens, int T,
                            long long n_tok, int H, int n_seq, int d, float eps, int coeff_eta, int qnorm, int io_dtype,
                            cudaStream_t stream);
// True when the tensor-core kernel covers this case.
bool chunk_tc_supported(int d, int chunk, int io_dtype);

void count_launch(int n);
// Host-side validation of a chunk-forward call (api.cu); `check_workspace`: also that desc->workspace is large enough.
kla_status check_chunk_args(const kla_desc *d, const void *q, const void *k, const void *v, const float *log_alpha, const float *eta,
                            float eps, int32_t chunk, const float *init_state, void *out, float *final_state, bool check_workspace);

// ---- device helpers -------------------------------------------------------------------------
__device__ __forceinline__ float to_f32(float x) { return x; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 x) { return __bfloat162float(x); }

template <typename T>
__device__ __forceinline__ T from_f32(float x);
template <>
__device__ __forceinline__ float from_f32<float>(float x) { return x; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float x) { return __float2bfloat16_rn(x); }

// Load 4 consecutive elements (16-byte aligned for fp32, 8-byte aligned for bf16) as fp32.
__device__ __forceinline__ float4 load4(const float *p) { return *reinterpret_cast<const float4 *>(p); }
__device__ __forceinline__ float4 load4(const __nv_bfloat16 *p)
{
    uint2 raw = *reinterpret_cast<const uint2 *>(p);
    __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162 *>(&raw.x);
    __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162 *>(&raw.y);
    float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
    return make_float4(fa.x, fa.y, fb.x, fb.y);
}
__device__ __forceinline__ void store4(float *p, float4 x) { *reinterpret_cast<float4 *>(p) = x; }
__device__ __forceinline__ void store4(__nv_bfloat16 *p, float4 x)
{
    __nv_bfloat162 a = __floats2bfloat162_rn(x.x, x.y), b = __floats2bfloat162_rn(x.z, x.w);
    uint2 raw;
    raw.x = *reinterpret_cast<uint32_t *>(&a);
    raw.y = *reinterpret_cast<uint32_t *>(&b);
    *reinterpret_cast<uint2 *>(p) = raw;
}

__device__ __forceinline__ void store2(float *p, float a, float b) { *reinterpret_cast<float2 *>(p) = make_float2(a, b); }
__device__ __forceinline__ void store2(__nv_bfloat16 *p, float a, float b)
{
    *reinterpret_cast<__nv_bfloat162 *>(p) = __floats2bfloat162_rn(a, b);
}

}  // namespace kla
