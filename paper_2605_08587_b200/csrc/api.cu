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
    if (cudaGetDevice(&dev) != cudaSuccess) return KLA_ERR_ARCH;   // (no usable device: there is no fallback)
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
kla_status check_chunk_args(const kla_desc *d, const void *q, const void *k, const void *v,
                            const float *log_alpha, const float *eta, float eps, int32_t chunk,
                            const float *init_state, void *out, float *final_state, bool check_workspace)
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
    if (check_workspace && kla_chunk_fwd_workspace_bytes(d, chunk) > 0) {
        if (!d->workspace || d->workspace_bytes < kla_chunk_fwd_workspace_bytes(d, chunk)) return KLA_ERR_WORKSPACE;
        if (!aligned16(d->workspace)) return KLA_ERR_ALIGN;
    }
    return KLA_OK;
}

// Packed input: the tensor-core kernel takes its sequences longest first (one int32 per sequence of scratch).
static size_t order_bytes(const kla_desc *d, int32_t chunk)
{
    if (!d->cu_seqlens || d->n_seq < 2 || d->n_seq > 4096 || (d->flags & KLA_FLAG_FORCE_SIMT) ||
        !chunk_tc_supported(d->d_k, chunk, d->io_dtype))
        return 0;
    return ((size_t)d->n_seq * sizeof(int32_t) + 255) & ~(size_t)255;
}

// Packed input, tensor-core path: long sequences are cut into pieces that start from decay-bounded warm-up runs when one
// sequence would otherwise set the length of the launch (or when the caller forces a number of pieces for the longest).
struct PackedPlan {
    int seg_len = 0;      // tokens per piece (a multiple of 64); 0: sequences are not cut
    int n_units = 0;      // pieces in all
    size_t off_plan = 0, bytes = 0;   // the piece tables follow the longest-first order array in the workspace
};

static int sm_count();

static PackedPlan plan_packed(const kla_desc *d, int32_t chunk)
{
    PackedPlan pp;
    if (!order_bytes(d, chunk) || !d->host_seqlens) return pp;
    if (d->flags & (KLA_FLAG_NO_SEGMENTS | KLA_FLAG_EXACT_SEGMENTS | KLA_FLAG_COEFF_ETA)) return pp;
    if ((d->flags & KLA_FLAG_WY_FORM) && d->d_k == 128) return pp;
    long long total = 0;
    int longest = 0;
    for (int n = 0; n < d->n_seq; ++n) {
        if (d->host_seqlens[n + 1] < d->host_seqlens[n]) return pp;   // (refused by the argument check anyway)
        const int c = (d->host_seqlens[n + 1] - d->host_seqlens[n] + 63) / 64;
        total += c;
        longest = c > longest ? c : longest;
    }
    const int forced = (d->flags >> 8) & 0xff;
    int seg_chunks = 0;
    if (forced >= 2) {
        seg_chunks = (longest + forced - 1) / forced;
    } else {
        // chunks per SM if the work were spread evenly; a sequence well beyond that sets the length of the launch
        const long long even = total * d->H * (d->d_k / 64) / sm_count();
        const int target = even > 32 ? (int)even : 32;
        if (longest >= target + target / 4 + 8) seg_chunks = target;
    }
    if (seg_chunks < 2) return pp;   // (the warm-up may take at most half a piece)
    pp.seg_len = seg_chunks * 64;
    for (int n = 0; n < d->n_seq; ++n)
        pp.n_units += (d->host_seqlens[n + 1] - d->host_seqlens[n] + pp.seg_len - 1) / pp.seg_len;
    if (pp.n_units <= d->n_seq) return PackedPlan();   // nothing is actually cut
    pp.off_plan = order_bytes(d, chunk);
    // bounds (n_units + 1), plan word, warm-up lengths (n_units x H), piece table (n_units)
    pp.bytes = pp.off_plan + ((((size_t)pp.n_units * (d->H + 2) + 2) * sizeof(int32_t) + 255) & ~(size_t)255);
    return pp;
}

// ---- segment-parallel scan: when to use it, and the workspace it needs ----------------------------------------------
struct SegPlan {
    int G = 0;            // segments per sequence (0: plain launch)
    int seg_len = 0;      // tokens per segment (a multiple of the chunk length)
    size_t off_map = 0, off_local = 0, off_start = 0, bytes = 0;   // workspace layout; cu_seg sits at offset 0
};

static int sm_count()
{
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
        return 148;
    return n;
}

// Few long sequences leave most SMs idle (one CTA per sequence x head x slice, each walking its chunks in series).
// Cutting every sequence into G segments costs about two more passes of state work but runs G times as many CTAs.
static SegPlan plan_segments(const kla_desc *d, int32_t chunk)
{
    SegPlan pl;
    if (d->cu_seqlens || (d->flags & (KLA_FLAG_FORCE_SIMT | KLA_FLAG_NO_SEGMENTS)) || !chunk_tc_supported(d->d_k, chunk, d->io_dtype))
        return pl;
    const int chunks = (d->T + 63) / 64;
    const int units = d->B * d->H * (d->d_k / 64);
    const int forced = (d->flags >> 8) & 0xff;
    int best_len = 0;
    if (forced >= 2) {
        best_len = (chunks + forced - 1) / forced;
    } else if (forced == 0) {
        const int sms = sm_count();
        auto waves = [&](int ctas) { return (ctas + sms - 1) / sms; };
        const double plain = (double)waves(units) * chunks;
        double best = 0.75 * plain;   // only worth it for a clear win
        for (int G = 2; G <= 32 && chunks / G >= 8; ++G) {
            const int len = (chunks + G - 1) / G, Ge = (chunks + len - 1) / len;
            if (Ge < 2) continue;
            // measured on the 65K single-sequence workload (per-pass device times): a chunk of pass 1 (no outputs) takes 0.86 of a
            // main-pass chunk, and chaining the maps costs 2.2 chunk periods per segment
            const double cost = 0.86 * waves(units * 2 * (Ge - 1)) * len + (double)waves(units * Ge) * len + 2.2 * Ge;
            if (cost < best) {
                best = cost;
                best_len = len;
            }
        }
    }
    if (best_len <= 0) return pl;
    pl.seg_len = best_len * 64;
    pl.G = (d->T + pl.seg_len - 1) / pl.seg_len;
    if (pl.G < 2) return SegPlan();
    const size_t cu_bytes = (seg_plan_ints(d->B, pl.G, d->H) * sizeof(int32_t) + 255) & ~(size_t)255;
    const size_t st = (size_t)d->B * pl.G * d->H * d->d_k * d->d_v * sizeof(float);
    pl.off_map = cu_bytes;
    pl.off_local = cu_bytes + st;
    pl.off_start = cu_bytes + 2 * st;
    pl.bytes = cu_bytes + 3 * st;
    return pl;
}

}  // namespace kla

using namespace kla;

extern "C" {

size_t kla_chunk_fwd_workspace_bytes(const kla_desc *desc, int32_t chunk)
{
    if (check_common(desc) != KLA_OK) return 0;
    // the chunk kernels keep every intermediate on chip; scratch is needed by the segment-parallel scan and, for
    // packed input on the tensor-core path, by the longest-first order of the sequences
    if (order_bytes(desc, chunk)) {
        const PackedPlan pp = plan_packed(desc, chunk);
        return pp.seg_len ? pp.bytes : order_bytes(desc, chunk);
    }
    return plan_segments(desc, chunk).bytes;
}

size_t kla_chunk_fwd_plan_word_offset(const kla_desc *desc, int32_t chunk)
{
    if (check_common(desc) != KLA_OK) return (size_t)-1;
    const SegPlan pl = plan_segments(desc, chunk);
    if (pl.G >= 2) return ((size_t)desc->B * pl.G + 1) * sizeof(int32_t);
    const PackedPlan pp = plan_packed(desc, chunk);
    return pp.seg_len ? pp.off_plan + ((size_t)pp.n_units + 1) * sizeof(int32_t) : (size_t)-1;
}

}  // extern "C"

// The chunk forward proper.  `marks`: null, or five events recorded on the stream around the set-up kernels, segment
// pass 1, the chaining of the segment maps and the main pass (kla_chunk_fwd_timed).
static kla_status chunk_fwd_impl(const kla_desc *desc, const void *q, const void *k, const void *v,
                                 const float *log_alpha, const float *eta, float eps, int32_t chunk,
                                 const float *init_state, void *out, float *final_state, cudaEvent_t *marks)
{
    auto mark = [&](int i) {
        if (marks) cudaEventRecord(marks[i], (cudaStream_t)desc->stream);
    };
    kla_status st = check_chunk_args(desc, q, k, v, log_alpha, eta, eps, chunk, init_state, out, final_state, true);
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
    p.seg_pass = 0; p.seg_G = 0; p.map_state = nullptr;
    p.variant = ((desc->flags & KLA_FLAG_COEFF_ETA) ? VARIANT_COEFF_ETA : 0) | ((desc->flags & KLA_FLAG_QNORM) ? VARIANT_QNORM : 0) |
                ((desc->flags & KLA_INTERNAL_FLAG_TEST_TIMEOUT) ? VARIANT_TEST_TIMEOUT : 0) |
                ((desc->flags & KLA_FLAG_NO_PAIR) ? VARIANT_NO_PAIR : 0) | ((desc->flags & KLA_FLAG_WY_FORM) ? VARIANT_WY : 0);
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
    const SegPlan pl = plan_segments(desc, chunk);
    mark(0);
    if (pl.G >= 2) {
        char *ws = (char *)desc->workspace;
        int32_t *cu_seg = (int32_t *)ws;
        float *map = (float *)(ws + pl.off_map), *local = (float *)(ws + pl.off_local), *start = (float *)(ws + pl.off_start);
        // Decay-bounded segment starts (seg_warm_plan_kernel): tried unless the caller forbids it, the coefficient is not
        // Eq. 3's (beta = eta: no bound on beta ||k||^2) or the WY-form kernel is asked for (it has no such pass).  Both
        // kinds of passes are enqueued; a device word decides which of them does the work, so nothing waits for the host.
        const bool try_warm = !(desc->flags & (KLA_FLAG_EXACT_SEGMENTS | KLA_FLAG_COEFF_ETA)) &&
                              !((desc->flags & KLA_FLAG_WY_FORM) && desc->d_k == 128);
        if (launch_seg_bounds(cu_seg, desc->B, desc->T, pl.G, pl.seg_len, try_warm ? 1 : 0, stream) != cudaSuccess) return KLA_ERR_LAUNCH;
        if (try_warm && launch_seg_warm_plan(cu_seg, log_alpha, eta, desc->B, desc->T, desc->H, pl.G, pl.seg_len, stream) != cudaSuccess)
            return KLA_ERR_LAUNCH;
        mark(1);
        ChunkParams p1 = p;   // pass 1: transition map and zero-start state of every segment but the last
        p1.cu_seqlens = cu_seg; p1.n_seq = desc->B * pl.G;
        p1.init_state = nullptr; p1.final_state = local; p1.map_state = map;
        p1.seg_pass = 1; p1.seg_G = pl.G;
        if (launch_chunk_tc(p1, desc->d_k, desc->io_dtype, desc->out_dtype, stream) != cudaSuccess) return KLA_ERR_LAUNCH;
        mark(2);
        if (launch_seg_combine(init_state, map, local, start, desc->B, desc->H, pl.G, desc->d_k, cu_seg + desc->B * pl.G + 1, stream) != cudaSuccess)
            return KLA_ERR_LAUNCH;
        mark(3);
        ChunkParams p3 = p;   // pass 3: every segment from its true start state
        p3.cu_seqlens = cu_seg; p3.n_seq = desc->B * pl.G;
        p3.init_state = start;
        p3.seg_pass = 3; p3.seg_G = pl.G;
        err = launch_chunk_tc(p3, desc->d_k, desc->io_dtype, desc->out_dtype, stream);
        if (err == cudaSuccess && try_warm) {
            ChunkParams p4 = p;   // pass 4: every segment from a warm-up run (the sequence's first from its initial state)
            p4.cu_seqlens = cu_seg; p4.n_seq = desc->B * pl.G;
            p4.seg_pass = 4; p4.seg_G = pl.G;
            err = launch_chunk_tc(p4, desc->d_k, desc->io_dtype, desc->out_dtype, stream);
        }
        mark(4);
        return err == cudaSuccess ? KLA_OK : KLA_ERR_LAUNCH;
    }
    if (!(desc->flags & KLA_FLAG_FORCE_SIMT) && chunk_tc_supported(desc->d_k, chunk, desc->io_dtype)) {
        const PackedPlan pp = plan_packed(desc, chunk);
        if (order_bytes(desc, chunk)) {
            int32_t *order = (int32_t *)desc->workspace;
            if (launch_seq_order(desc->cu_seqlens, desc->n_seq, order, stream) != cudaSuccess) return KLA_ERR_LAUNCH;
            p.seq_order = order;
        }
        if (pp.seg_len) {
            // pieces from warm-up runs (pass 5) if the decay allows, else the plain launch (pass 6): a device word decides
            int32_t *ub = (int32_t *)((char *)desc->workspace + pp.off_plan);
            int32_t *unit_seq = ub + pp.n_units + 2 + (size_t)pp.n_units * desc->H;
            if (launch_packed_units(desc->cu_seqlens, desc->n_seq, pp.seg_len, pp.n_units, ub, unit_seq, log_alpha, eta,
                                    (long long)desc->T, desc->H, init_state, final_state, desc->d_k, stream) != cudaSuccess)
                return KLA_ERR_LAUNCH;
            mark(1); mark(2); mark(3);
            ChunkParams p5 = p;
            p5.cu_seqlens = ub; p5.n_seq = pp.n_units;
            p5.seg_pass = 5; p5.seg_G = 0; p5.map_state = nullptr;
            if (launch_chunk_tc(p5, desc->d_k, desc->io_dtype, desc->out_dtype, stream) != cudaSuccess) return KLA_ERR_LAUNCH;
            p.seg_pass = 6;
            p.seg_G = (int32_t)((ub + pp.n_units + 1) - p.seq_order);   // where the plan word is, counted from the order array
            err = launch_chunk_tc(p, desc->d_k, desc->io_dtype, desc->out_dtype, stream);
        } else {
            mark(1); mark(2); mark(3);
            err = launch_chunk_tc(p, desc->d_k, desc->io_dtype, desc->out_dtype, stream);
        }
    }
    else {
        mark(1); mark(2); mark(3);
        err = launch_chunk_simt(p, desc->d_k, chunk, desc->io_dtype, desc->out_dtype, stream);
    }
    mark(4);
    return err == cudaSuccess ? KLA_OK : KLA_ERR_LAUNCH;
}

extern "C" {

kla_status kla_chunk_fwd(const kla_desc *desc, const void *q, const void *k, const void *v,
                         const float *log_alpha, const float *eta, float eps, int32_t chunk,
                         const float *init_state, void *out, float *final_state)
{
    return chunk_fwd_impl(desc, q, k, v, log_alpha, eta, eps, chunk, init_state, out, final_state, nullptr);
}

kla_status kla_chunk_fwd_timed(const kla_desc *desc, const void *q, const void *k, const void *v,
                               const float *log_alpha, const float *eta, float eps, int32_t chunk,
                               const float *init_state, void *out, float *final_state, float *pass_ms)
{
    if (!pass_ms) return KLA_ERR_NULL;
    for (int i = 0; i < 4; ++i) pass_ms[i] = 0.f;
    // validated here as well, so that nothing is created for a call that will be refused
    kla_status st = check_chunk_args(desc, q, k, v, log_alpha, eta, eps, chunk, init_state, out, final_state, true);
    if (st != KLA_OK) return st;
    cudaEvent_t ev[5];
    int made = 0;
    for (; made < 5; ++made)
        if (cudaEventCreate(&ev[made]) != cudaSuccess) break;
    if (made == 5) {
        st = chunk_fwd_impl(desc, q, k, v, log_alpha, eta, eps, chunk, init_state, out, final_state, ev);
        if (st == KLA_OK && desc->T > 0) {
            if (cudaStreamSynchronize((cudaStream_t)desc->stream) != cudaSuccess) st = KLA_ERR_LAUNCH;
            for (int i = 0; st == KLA_OK && i < 4; ++i)
                if (cudaEventElapsedTime(&pass_ms[i], ev[i], ev[i + 1]) != cudaSuccess) pass_ms[i] = 0.f;
            // passes that did not run: their marks were recorded back to back
            const bool segments = plan_segments(desc, chunk).G >= 2;
            if (!segments) pass_ms[1] = pass_ms[2] = 0.f;
            if (!segments && !order_bytes(desc, chunk)) pass_ms[0] = 0.f;
        }
    } else {
        st = KLA_ERR_LAUNCH;
    }
    for (int i = 0; i < made; ++i) cudaEventDestroy(ev[i]);
    (void)cudaGetLastError();
    return st;
}


// ---- sequence-parallel prefill: the pieces around the exchange ------------------------------------------------------------
size_t kla_chunk_span_map_workspace_bytes(const kla_desc *desc)
{
    if (check_common(desc) != KLA_OK) return 0;
    // segment bounds of a two-segment cut whose second segment is empty, then both halves of the segment arrays
    const size_t cu_bytes = (seg_plan_ints(desc->B, 2, desc->H) * sizeof(int32_t) + 255) & ~(size_t)255;
    return cu_bytes + 2 * (size_t)desc->B * 2 * desc->H * desc->d_k * desc->d_v * sizeof(float);
}

kla_status kla_chunk_span_map(const kla_desc *desc, const void *k, const void *v, const float *log_alpha, const float *eta,
                              float eps, float *phi_out, float *n_out)
{
    kla_status st = check_common(desc);
    if (st != KLA_OK) return st;
    if (!k || !v || !log_alpha || !eta || !phi_out || !n_out) return KLA_ERR_NULL;
    if (!(eps >= 0.f) || !std::isfinite(eps)) return KLA_ERR_EPS;
    if (desc->cu_seqlens || desc->n_seq != desc->B || desc->T < 1) return KLA_ERR_SHAPE;
    if (desc->io_dtype != KLA_BF16) return KLA_ERR_DTYPE;
    if ((int64_t)desc->B * desc->T >= (int64_t)1 << 31) return KLA_ERR_SHAPE;
    if (!aligned16(k) || !aligned16(v) || !aligned16(log_alpha) || !aligned16(eta) || !aligned16(phi_out) || !aligned16(n_out))
        return KLA_ERR_ALIGN;
    const size_t need = kla_chunk_span_map_workspace_bytes(desc);
    if (!desc->workspace || desc->workspace_bytes < need) return KLA_ERR_WORKSPACE;
    if (!aligned16(desc->workspace)) return KLA_ERR_ALIGN;
    st = check_arch();
    if (st != KLA_OK) return st;
    cudaStream_t stream = (cudaStream_t)desc->stream;
    // The whole input as the first of two segments per sequence (the second is empty): segment pass 1 of the chunk
    // kernel then gives the map and the zero-start state of exactly that span.
    char *ws = (char *)desc->workspace;
    int32_t *cu_seg = (int32_t *)ws;
    const size_t cu_bytes = (seg_plan_ints(desc->B, 2, desc->H) * sizeof(int32_t) + 255) & ~(size_t)255;
    const size_t half = (size_t)desc->B * 2 * desc->H * desc->d_k * desc->d_v;
    float *map = (float *)(ws + cu_bytes), *local = map + half;
    if (launch_seg_bounds(cu_seg, desc->B, desc->T, 2, ((desc->T + 63) / 64) * 64, 0, stream) != cudaSuccess) return KLA_ERR_LAUNCH;
    ChunkParams p;
    p.q = k;   // never read out: pass 1 forms no outputs (the tensor map only needs a valid address)
    p.k = k; p.v = v;
    p.log_alpha = log_alpha; p.eta = eta;
    p.init_state = nullptr;
    p.out = nullptr;
    p.final_state = local;
    p.cu_seqlens = cu_seg;
    p.status_word = desc->status_word;
    p.B = desc->B; p.T = desc->T; p.H = desc->H; p.n_seq = desc->B * 2;
    p.eps = eps;
    p.seg_pass = 1; p.seg_G = 2;
    p.variant = ((desc->flags & KLA_FLAG_COEFF_ETA) ? VARIANT_COEFF_ETA : 0) | ((desc->flags & KLA_FLAG_NO_PAIR) ? VARIANT_NO_PAIR : 0) |
                ((desc->flags & KLA_FLAG_WY_FORM) ? VARIANT_WY : 0);
    p.map_state = map;
    if (launch_chunk_tc(p, desc->d_k, desc->io_dtype, KLA_F32, stream) != cudaSuccess) return KLA_ERR_LAUNCH;
    // segment 0 of sequence b sits at index 2 b of the segment arrays
    const size_t one = (size_t)desc->H * desc->d_k * desc->d_v * sizeof(float);
    if (cudaMemcpy2DAsync(phi_out, one, map, 2 * one, one, (size_t)desc->B, cudaMemcpyDeviceToDevice, stream) != cudaSuccess ||
        cudaMemcpy2DAsync(n_out, one, local, 2 * one, one, (size_t)desc->B, cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
        return KLA_ERR_LAUNCH;
    return KLA_OK;
}

kla_status kla_state_chain(const kla_desc *desc, int32_t n_spans, const float *init_state, const float *phi, const float *n,
                           float *start_out)
{
    kla_status st = check_common(desc);
    if (st != KLA_OK) return st;
    if (!phi || !n || !start_out) return KLA_ERR_NULL;
    if (n_spans < 1) return KLA_ERR_SHAPE;
    if (!aligned16(phi) || !aligned16(n) || !aligned16(start_out) || !aligned16(init_state)) return KLA_ERR_ALIGN;
    st = check_arch();
    if (st != KLA_OK) return st;
    return launch_seg_combine(init_state, phi, n, start_out, desc->B, desc->H, n_spans, desc->d_k, nullptr, (cudaStream_t)desc->stream) == cudaSuccess
               ? KLA_OK : KLA_ERR_LAUNCH;
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
        p.inputs_ready = s > 0 ? 1 : 0;
        p.coeff_eta = (desc->flags & KLA_FLAG_COEFF_ETA) ? 1 : 0;
        p.qnorm = (desc->flags & KLA_FLAG_QNORM) ? 1 : 0;
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

kla_status kla_dg_fwd(const kla_desc *desc, const void *q, const void *k, const void *v,
                      const float *log_alpha, const float *eta, float eps,
                      const float *init_state, void *out, float *final_state)
{
    // the same host-side checks as the chunk forward (chunk 64 stands in: there is no chunk length here)
    kla_status st = check_chunk_args(desc, q, k, v, log_alpha, eta, eps, 64, init_state, out, final_state, false);
    if (st != KLA_OK) return st;
    st = check_arch();
    if (st != KLA_OK) return st;
    cudaStream_t stream = (cudaStream_t)desc->stream;
    if (desc->T == 0) {
        if (final_state) {
            const size_t bytes = (size_t)desc->n_seq * desc->H * desc->d_k * desc->d_v * sizeof(float);
            cudaError_t e = init_state ? cudaMemcpyAsync(final_state, init_state, bytes, cudaMemcpyDeviceToDevice, stream)
                                       : cudaMemsetAsync(final_state, 0, bytes, stream);
            if (e != cudaSuccess) return KLA_ERR_LAUNCH;
        }
        return KLA_OK;
    }
    return launch_dg_scan(q, k, v, log_alpha, eta, init_state, out, final_state, desc->cu_seqlens, desc->T, desc->H, desc->n_seq,
                          desc->d_k, eps, (desc->flags & KLA_FLAG_COEFF_ETA) ? 1 : 0, (desc->flags & KLA_FLAG_QNORM) ? 1 : 0,
                          desc->io_dtype, desc->out_dtype, stream) == cudaSuccess ? KLA_OK : KLA_ERR_LAUNCH;
}

kla_status kla_dg_decode_step(const kla_desc *desc, const void *q, const void *k, const void *v,
                              const float *log_alpha, const float *eta, float eps,
                              float *state_inout, void *out)
{
    kla_status st = check_decode(desc, q, k, v, log_alpha, eta, eps, state_inout, out);
    if (st != KLA_OK) return st;
    st = check_arch();
    if (st != KLA_OK) return st;
    // one token per sequence; every warp reads its columns of the state before it writes them, so the update is in place
    return launch_dg_scan(q, k, v, log_alpha, eta, state_inout, out, state_inout, nullptr, 1, desc->H, desc->B, desc->d_k, eps,
                          (desc->flags & KLA_FLAG_COEFF_ETA) ? 1 : 0, (desc->flags & KLA_FLAG_QNORM) ? 1 : 0, desc->io_dtype,
                          desc->out_dtype, (cudaStream_t)desc->stream) == cudaSuccess ? KLA_OK : KLA_ERR_LAUNCH;
}

size_t kla_bwd_workspace_bytes(const kla_desc *desc)
{
    if (check_common(desc) != KLA_OK || desc->n_seq < 1) return 0;
    return bwd_workspace_bytes(desc->n_seq, (long long)desc->B * desc->T, desc->H, desc->d_k);
}

kla_status kla_bwd(const kla_desc *desc, const void *q, const void *k, const void *v,
                   const float *log_alpha, const float *eta, float eps, const float *init_state,
                   const void *d_out, const float *d_final_state,
                   float *dq, float *dk, float *dv, float *dlog_alpha, float *deta, float *dinit_state)
{
    // the forward's host-side checks (d_out stands where out does: same shape, required, aligned)
    kla_status st = check_chunk_args(desc, q, k, v, log_alpha, eta, eps, 64, init_state, const_cast<void *>(d_out), nullptr, false);
    if (st != KLA_OK) return st;
    if (!dq || !dk || !dv || !dlog_alpha || !deta) return KLA_ERR_NULL;
    if (!aligned16(dq) || !aligned16(dk) || !aligned16(dv) || !aligned16(dlog_alpha) || !aligned16(deta) ||
        !aligned16(d_final_state) || !aligned16(dinit_state))
        return KLA_ERR_ALIGN;
    const size_t need = kla_bwd_workspace_bytes(desc);
    if (need > 0 && (!desc->workspace || desc->workspace_bytes < need)) return KLA_ERR_WORKSPACE;
    if (!aligned16(desc->workspace)) return KLA_ERR_ALIGN;
    st = check_arch();
    if (st != KLA_OK) return st;
    cudaStream_t stream = (cudaStream_t)desc->stream;
    return launch_bwd_scan(q, k, v, log_alpha, eta, init_state, d_out, d_final_state, dq, dk, dv, dlog_alpha, deta, dinit_state,
                           desc->workspace, desc->cu_seqlens, desc->T, (long long)desc->B * desc->T, desc->H, desc->n_seq,
                           desc->d_k, eps, (desc->flags & KLA_FLAG_COEFF_ETA) ? 1 : 0, (desc->flags & KLA_FLAG_QNORM) ? 1 : 0,
                           desc->io_dtype, stream) == cudaSuccess ? KLA_OK : KLA_ERR_LAUNCH;
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
        case KLA_ERR_DEVICE: return "current device could not be queried or its scratch address is unavailable";
    }
    return "unknown status";
}

uint64_t kla_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
