// Recurrent decode step (Algorithm 1, left panel; Eq. 3) -- memory-bound kernel.
//
// One CTA owns W consecutive d_v columns of one head's d_k x d_v fp32 state.  Columns evolve
// independently (the rank-one write is k e^T), so no CTA talks to another.  The slice is read
// from HBM exactly once with 128-bit loads, kept in registers, and written back once:
//
//   a = S^T k, c = S^T q                       (one sweep over the registers)
//   e = v - alpha a,  beta = eta / (||k||^2 + eps)
//   S <- alpha S + beta k e^T                  (written back)
//   o = S_new^T q = alpha c + beta (k.q) e     (no second sweep over the state)
#include "common.cuh"

namespace kla {

template <int D, int W, typename IO, typename OUT>
__global__ void __launch_bounds__(128) kla_decode_kernel(DecodeParams p)
{
    constexpr int SLICES = D / W;
    constexpr int TPR = W / 4;      // threads per state row (one float4 each)
    constexpr int RPP = 128 / TPR;  // rows covered per pass
    constexpr int NP = D / RPP;     // passes = float4 registers per thread
    static_assert(D % RPP == 0 && TPR <= 32 && (32 % TPR) == 0, "tiling");

    const int bh = blockIdx.x / SLICES;
    const int sl = blockIdx.x % SLICES;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cg = tid % TPR, rg = tid / TPR;

    __shared__ float sk[D], sq[D];
    __shared__ float red_a[4][W], red_c[4][W];
    __shared__ float red_s[3][4];

    // 1. token vectors and their reductions.  The kernel is launched with programmatic stream serialisation, so
    //    it may start while the previous kernel on the stream drains.  When the vectors are known to predate that
    //    kernel (later steps of a multi-step call) they are read right away; otherwise wait first.
    if (!p.inputs_ready) asm volatile("griddepcontrol.wait;" ::: "memory");
    const IO *qp = reinterpret_cast<const IO *>(p.q) + (size_t)bh * D;
    const IO *kp = reinterpret_cast<const IO *>(p.k) + (size_t)bh * D;
    float kk = 0.f, kq = 0.f, qq = 0.f;
    if (tid < D) {
        float kv = to_f32(kp[tid]), qv = to_f32(qp[tid]);
        sk[tid] = kv;
        sq[tid] = qv;
        kk = kv * kv;
        kq = kv * qv;
        qq = qv * qv;
    }
    const float alpha = expf(p.log_alpha[bh]);
    const float eta = p.eta[bh];
    const float4 vv = load4(reinterpret_cast<const IO *>(p.v) + (size_t)bh * D + sl * W + cg * 4);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        kk += __shfl_xor_sync(0xffffffffu, kk, o);
        kq += __shfl_xor_sync(0xffffffffu, kq, o);
        qq += __shfl_xor_sync(0xffffffffu, qq, o);
    }
    if (lane == 0) {
        red_s[0][warp] = kk;
        red_s[1][warp] = kq;
        red_s[2][warp] = qq;
    }

    // 2. the state: written by the previous step, so wait for that kernel (a no-op for an ordinary launch), then
    //    let the next step's kernel start its own prologue
    asm volatile("griddepcontrol.wait;" ::: "memory");
    float *Sp = p.state + (size_t)bh * D * D + sl * W + cg * 4;
    float4 s[NP];
#pragma unroll
    for (int i = 0; i < NP; ++i) s[i] = *reinterpret_cast<const float4 *>(Sp + (size_t)(rg + i * RPP) * D);
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    __syncthreads();
    kk = red_s[0][0] + red_s[0][1] + red_s[0][2] + red_s[0][3];
    kq = red_s[1][0] + red_s[1][1] + red_s[1][2] + red_s[1][3];
    qq = red_s[2][0] + red_s[2][1] + red_s[2][2] + red_s[2][3];

    // 3. a = S^T k and c = S^T q for this thread's 4 columns over its rows
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f), c = a;
#pragma unroll
    for (int i = 0; i < NP; ++i) {
        const float kr = sk[rg + i * RPP], qr = sq[rg + i * RPP];
        a.x += s[i].x * kr; a.y += s[i].y * kr; a.z += s[i].z * kr; a.w += s[i].w * kr;
        c.x += s[i].x * qr; c.y += s[i].y * qr; c.z += s[i].z * qr; c.w += s[i].w * qr;
    }
    // reduce over the row groups: inside a warp lanes with equal (lane % TPR) share columns
#pragma unroll
    for (int o = TPR; o < 32; o <<= 1) {
        a.x += __shfl_xor_sync(0xffffffffu, a.x, o); a.y += __shfl_xor_sync(0xffffffffu, a.y, o);
        a.z += __shfl_xor_sync(0xffffffffu, a.z, o); a.w += __shfl_xor_sync(0xffffffffu, a.w, o);
        c.x += __shfl_xor_sync(0xffffffffu, c.x, o); c.y += __shfl_xor_sync(0xffffffffu, c.y, o);
        c.z += __shfl_xor_sync(0xffffffffu, c.z, o); c.w += __shfl_xor_sync(0xffffffffu, c.w, o);
    }
    if (lane < TPR) {
        *reinterpret_cast<float4 *>(&red_a[warp][lane * 4]) = a;
        *reinterpret_cast<float4 *>(&red_c[warp][lane * 4]) = c;
    }
    __syncthreads();
    {
        float4 t0 = *reinterpret_cast<float4 *>(&red_a[0][cg * 4]), t1 = *reinterpret_cast<float4 *>(&red_a[1][cg * 4]);
        float4 t2 = *reinterpret_cast<float4 *>(&red_a[2][cg * 4]), t3 = *reinterpret_cast<float4 *>(&red_a[3][cg * 4]);
        a = make_float4((t0.x + t1.x) + (t2.x + t3.x), (t0.y + t1.y) + (t2.y + t3.y),
                        (t0.z + t1.z) + (t2.z + t3.z), (t0.w + t1.w) + (t2.w + t3.w));
        t0 = *reinterpret_cast<float4 *>(&red_c[0][cg * 4]); t1 = *reinterpret_cast<float4 *>(&red_c[1][cg * 4]);
        t2 = *reinterpret_cast<float4 *>(&red_c[2][cg * 4]); t3 = *reinterpret_cast<float4 *>(&red_c[3][cg * 4]);
        c = make_float4((t0.x + t1.x) + (t2.x + t3.x), (t0.y + t1.y) + (t2.y + t3.y),
                        (t0.z + t1.z) + (t2.z + t3.z), (t0.w + t1.w) + (t2.w + t3.w));
    }

    // 4. residual, coefficient, write-back, read-out
    const float beta = p.coeff_eta ? eta : eta / (kk + p.eps);   // Eq. 3, or the gated-delta-rule coefficient
    float4 e = make_float4(vv.x - alpha * a.x, vv.y - alpha * a.y, vv.z - alpha * a.z, vv.w - alpha * a.w);
#pragma unroll
    for (int i = 0; i < NP; ++i) {
        const float bk = beta * sk[rg + i * RPP];
        float4 n;
        n.x = alpha * s[i].x + bk * e.x; n.y = alpha * s[i].y + bk * e.y;
        n.z = alpha * s[i].z + bk * e.z; n.w = alpha * s[i].w + bk * e.w;
        *reinterpret_cast<float4 *>(Sp + (size_t)(rg + i * RPP) * D) = n;
    }
    if (rg == 0) {
        const float bq = beta * kq;
        const float rn = p.qnorm ? 1.f / sqrtf(qq) : 1.f;   // read-out over ||q|| (Algorithm 1 left) when asked for
        float4 o = make_float4(rn * (alpha * c.x + bq * e.x), rn * (alpha * c.y + bq * e.y), rn * (alpha * c.z + bq * e.z),
                               rn * (alpha * c.w + bq * e.w));
        store4(reinterpret_cast<OUT *>(p.out) + (size_t)bh * D + sl * W + cg * 4, o);
    }
}

template <int D, typename IO, typename OUT>
static cudaError_t launch_decode_t(const DecodeParams &p, cudaStream_t stream)
{
    constexpr int W = 32;
    // programmatic dependent launch: the kernel's prologue may start while the previous kernel on the stream
    // drains; its state accesses come after griddepcontrol.wait
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(p.BH * (D / W)));
    cfg.blockDim = dim3(128);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t err = cudaLaunchKernelEx(&cfg, kla_decode_kernel<D, W, IO, OUT>, p);
    count_launch(1);
    return err != cudaSuccess ? err : cudaGetLastError();
}

cudaError_t launch_decode(const DecodeParams &p, int d, int io_dtype, int out_dtype, cudaStream_t stream)
{
    const int key = (d == 128 ? 4 : 0) | (io_dtype == KLA_BF16 ? 2 : 0) | (out_dtype == KLA_BF16 ? 1 : 0);
    switch (key) {
        case 0: return launch_decode_t<64, float, float>(p, stream);
        case 1: return launch_decode_t<64, float, __nv_bfloat16>(p, stream);
        case 2: return launch_decode_t<64, __nv_bfloat16, float>(p, stream);
        case 3: return launch_decode_t<64, __nv_bfloat16, __nv_bfloat16>(p, stream);
        case 4: return launch_decode_t<128, float, float>(p, stream);
        case 5: return launch_decode_t<128, float, __nv_bfloat16>(p, stream);
        case 6: return launch_decode_t<128, __nv_bfloat16, float>(p, stream);
        default: return launch_decode_t<128, __nv_bfloat16, __nv_bfloat16>(p, stream);
    }
}

}  // namespace kla
