// extern "C" boundary of the library: argument validation, dispatch, error codes.
#include <atomic>
#include <cmath>

#include "common.cuh"

namespace kla {

static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

static bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static kla_status check_arch()
{
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return KLA_ERR_ARCH;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return KLA_ERR_ARCH;
    return major == 10 ? KLA_OK : KLA_ERR_ARCH;
}

static kla_status check_common(const kla_desc *d)
{
    if (!d) return KLA_ERR_NULL;
    if (d->io_dtype != KLA_F32 && d->io_dtype != KLA_BF16) return KLA_ERR_DTYPE;
    if (d->out_dtype != KLA_F32 && d->out_dtype != KLA_BF16) return KLA_ERR_DTYPE;
    if (d->B < 1 || d->T < 0 || d->H < 1) return KLA_ERR_SHAPE;
    if (!(d->d_k == 64 || d->d_k == 128) || d->d_v != d->d_k) return KLA_ERR_SHAPE;
    if (d->status_word && (reinterpret_cast<uintptr_t>(d->status_word) & 3u)) return KLA_ERR_ALIGN;
    return KLA_OK;
}

// Host-side validation of a chunk-forward call; launches nothing.
static kla_status check_chunk(const kla_desc *d, const void *q, const void *k, const void *v,
                              const float *log_alpha, const float *eta, float eps, int32_t chunk,
                              const float *init_state, void *out, float *final_state)
{
    kla_status st = check_common(d);
    if (st != KLA_OK) return st;
    if (!q || !k || !v || !log_alpha || !eta || !out) return KLA_ERR_NULL;
    if (!(eps >= 0.f) || !std::isfinite(eps)) return KLA_ERR_EPS;
    if (!(chunk == 16 || chunk == 32 || chunk == 64)) return KLA_ERR_CHUNK;
    if (d->cu_seqlens) {
        if (!d->host_seqlens) return KLA_ERR_NULL;
        if (d->B != 1 || d->n_seq < 1) return KLA_ERR_SHAPE;
        if (d->host_seqlens[0] != 0) return KLA_ERR_SEQLENS;
        for (int i = 0; i < d->n_seq; ++i)
            if (d->host_seqlens[i + 1] < d->host_seqlens[i]) return KLA_ERR_SEQLENS;
        if (d->host_seqlens[d->n_seq] != d->T) return KLA_ERR_SEQLENS;
        if (reinterpret_cast<uintptr_t>(d->cu_seqlens) & 3u) return KLA_ERR_ALIGN;
    } else {
        if (d->n_seq != d->B) return KLA_ERR_SHAPE;
    }
    if ((int64_t)d->B * d->T >= (int64_t)1 << 31) return KLA_ERR_SHAPE;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(log_alpha) || !aligned16(eta) ||
        !aligned16(out) || !aligned16(init_state) || !aligned16(final_state))
        return KLA_ERR_ALIGN;
    if (kla_chunk_fwd_workspace_bytes(d, chunk) > 0) {
        if (!d->workspace || d->workspace_bytes < kla_chunk_fwd_workspace_bytes(d, chunk)) return KLA_ERR_WORKSPACE;
        if (!aligned16(d->workspace)) return KLA_ERR_ALIGN;
    }
    return KLA_OK;
}

}  // namespace kla

using namespace kla;

extern "C" {

size_t kla_chunk_fwd_workspace_bytes(const kla_desc *desc, int32_t chunk)
{
    if (check_common(desc) != KLA_OK) return 0;
    (void)chunk;
    return 0;  // both chunk kernels keep every intermediate on chip
}

kla_status kla_chunk_fwd(const kla_desc *desc, const void *q, const void *k, const void *v,
                         const float *log_alpha, const float *eta, float eps, int32_t chunk,
                         const float *init_state, void *out, float *final_state)
{
    kla_status st = check_chunk(desc, q, k, v, log_alpha, eta, eps, chunk, init_state, out, final_state);
    if (st != KLA_OK) return st;
    st = check_arch();
    if (st != KLA_OK) return st;

    ChunkParams p;
    p.q = q; p.k = k; p.v = v;
    p.log_alpha = log_alpha; p.eta = eta;
    p.init_state = init_state;
    p.out = out;
    p.final_state = final_state;
    p.cu_seqlens = desc->cu_seqlens;
    p.status_word = desc->status_word;
    p.trace = nullptr;
    p.B = desc->B; p.T = desc->T; p.H = desc->H; p.n_seq = desc->n_seq;
    p.eps = eps;
    if (desc->T == 0) {
        // nothing to read out; the final state is the initial state
        if (final_state) {
            const size_t bytes = (size_t)desc->n_seq * desc->H * desc->d_k * desc->d_v * sizeof(float);
            cudaError_t e = init_state ? cudaMemcpyAsync(final_state, init_state, bytes, cudaMemcpyDeviceToDevice, (cudaStream_t)desc->stream)
                                       : cudaMemsetAsync(final_state, 0, bytes, (cudaStream_t)desc->stream);
            if (e != cudaSuccess) return KLA_ERR_LAUNCH;
        }
        return KLA_OK;
    }
    cudaStream_t stream = (cudaStream_t)desc->stream;
    cudaError_t err;
    if (!(desc->flags & KLA_FLAG_FORCE_SIMT) && chunk_tc_supported(desc->d_k, chunk, desc->io_dtype))
        err = launch_chunk_tc(p, desc->d_k, desc->io_dtype, desc->out_dtype, stream);
    else
        err = launch_chunk_simt(p, desc->d_k, chunk, desc->io_dtype, desc->out_dtype, stream);
    return err == cudaSuccess ? KLA_OK : KLA_ERR_LAUNCH;
}

static kla_status check_decode(const kla_desc *d, const void *q, const void *k, const void *v,
                               const float *log_alpha, const float *eta, float eps,
                               float *state, void *out)
{
    kla_status st = check_common(d);
    if (st != KLA_OK) return st;
    if (!q || !k || !v || !log_alpha || !eta || !state || !out) return KLA_ERR_NULL;
    if (d->T != 1 || d->cu_seqlens || d->n_seq != d->B) return KLA_ERR_SHAPE;
    if (!(eps >= 0.f) || !std::isfinite(eps)) return KLA_ERR_EPS;
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(log_alpha) || !aligned16(eta) ||
        !aligned16(state) || !aligned16(out))
        return KLA_ERR_ALIGN;
    return KLA_OK;
}

kla_status kla_decode_steps(const kla_desc *desc, int32_t n_steps, const void *q, const void *k,
                            const void *v, const float *log_alpha, const float *eta, float eps,
                            float *state_inout, void *out)
{
    kla_status st = check_decode(desc, q, k, v, log_alpha, eta, eps, state_inout, out);
    if (st != KLA_OK) return st;
    if (n_steps < 0) return KLA_ERR_SHAPE;
    st = check_arch();
    if (st != KLA_OK) return st;
    const size_t bh = (size_t)desc->B * desc->H;
    const size_t io_sz = desc->io_dtype == KLA_BF16 ? 2 : 4, out_sz = desc->out_dtype == KLA_BF16 ? 2 : 4;
    // per-step strides must keep the 16-byte alignment of the gate arrays
    if (n_steps > 1 && ((bh * sizeof(float)) & 15u)) return KLA_ERR_ALIGN;
    for (int32_t s = 0; s < n_steps; ++s) {
        DecodeParams p;
        p.q = (const char *)q + (size_t)s * bh * desc->d_k * io_sz;
        p.k = (const char *)k + (size_t)s * bh * desc->d_k * io_sz;
        p.v = (const char *)v + (size_t)s * bh * desc->d_v * io_sz;
        p.log_alpha = log_alpha + (size_t)s * bh;
        p.eta = eta + (size_t)s * bh;
        p.state = state_inout;
        p.out = (char *)out + (size_t)s * bh * desc->d_v * out_sz;
        p.BH = (int32_t)bh;
        p.eps = eps;
        if (launch_decode(p, desc->d_k, desc->io_dtype, desc->out_dtype, (cudaStream_t)desc->stream) != cudaSuccess)
            return KLA_ERR_LAUNCH;
    }
    return KLA_OK;
}

kla_status kla_decode_step(const kla_desc *desc, const void *q, const void *k, const void *v,
                           const float *log_alpha, const float *eta, float eps,
                           float *state_inout, void *out)
{
    return kla_decode_steps(desc, 1, q, k, v, log_alpha, eta, eps, state_inout, out);
}

const char *kla_status_str(kla_status s)
{
    switch (s) {
        case KLA_OK: return "ok";
        case KLA_ERR_NULL: return "required pointer is NULL";
        case KLA_ERR_SHAPE: return "unsupported or inconsistent shape";
        case KLA_ERR_DTYPE: return "unsupported dtype";
        case KLA_ERR_ALIGN: return "pointer not 16-byte aligned";
        case KLA_ERR_CHUNK: return "chunk must be 16, 32 or 64";
        case KLA_ERR_SEQLENS: return "sequence offsets not monotone from 0 to T";
        case KLA_ERR_WORKSPACE: return "workspace missing or too small";
        case KLA_ERR_EPS: return "eps must be finite and >= 0";
        case KLA_ERR_LAUNCH: return "CUDA launch failed";
        case KLA_ERR_TIMEOUT: return "a bounded device-side wait expired";
        case KLA_ERR_ARCH: return "device is not sm_100";
    }
    return "unknown status";
}

uint64_t kla_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
