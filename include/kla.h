/*
 * kla.h -- C ABI of the B200 (sm_100a) Kaczmarz Linear Attention hot path.
 *
 * Two operations, both defined by the same per-head recurrence on a d_k x d_v state S
 * (Algorithm 1, left panel; coefficient of Eq. 3; transposed form Eq. 6):
 *
 *     S~  = exp(log_alpha_t) * S_{t-1}
 *     e_t = v_t - S~^T k_t
 *     beta_t = eta_t / (||k_t||^2 + eps)
 *     S_t = S~ + beta_t * k_t e_t^T
 *     o_t = S_t^T q_t            (no division by ||q_t||, no 1/sqrt(d_k) scale: the caller
 *                                 passes the q it wants read out)
 *
 * kla_chunk_fwd evaluates it for whole sequences with the chunkwise-parallel solver
 * (Algorithm 1, right panel; Eqs. 7-9); kla_decode_step applies it to one new token per
 * sequence with the state updated in place.  The result does not depend on the chunk length.
 *
 * General rules
 *  - Every data pointer is a DEVICE pointer unless stated otherwise; every buffer is owned by the
 *    caller.  The library allocates nothing, on host or device.  The only state it keeps between calls is
 *    process-wide bookkeeping that no result depends on: the launch counter read by kla_launch_count, the
 *    driver entry point used to encode tensor maps, and, for kla_chunk_fwd_static_scratch, the device address
 *    of its built-in scratch array (looked up once per device; stale after cudaDeviceReset).
 *  - All arrays are dense, row-major, last index contiguous, 16-byte aligned.
 *  - Work is enqueued on desc->stream and the call returns without synchronising.  Argument
 *    errors are detected on the host before anything is launched and reported through the
 *    return value; nothing is launched in that case.
 *  - There is no CPU fallback: a device that is not compute capability 10.x gives KLA_ERR_ARCH.
 *  - Not thread-safe per stream beyond what CUDA itself guarantees; calls on different streams
 *    with disjoint buffers may overlap.
 */
#ifndef KLA_H_
#define KLA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    KLA_OK = 0,
    KLA_ERR_NULL = -1,      /* a required pointer is NULL                                  */
    KLA_ERR_SHAPE = -2,     /* unsupported or inconsistent B/T/H/d_k/d_v/n_seq             */
    KLA_ERR_DTYPE = -3,     /* io_dtype / out_dtype not one of kla_dtype                   */
    KLA_ERR_ALIGN = -4,     /* a pointer is not 16-byte aligned                            */
    KLA_ERR_CHUNK = -5,     /* chunk not in {16, 32, 64}                                   */
    KLA_ERR_SEQLENS = -6,   /* host_seqlens not monotone / does not end at T               */
    KLA_ERR_WORKSPACE = -7, /* workspace missing or smaller than the query says            */
    KLA_ERR_EPS = -8,       /* eps < 0 or not finite                                       */
    KLA_ERR_LAUNCH = -9,    /* the CUDA runtime rejected a launch (see cudaGetLastError)   */
    KLA_ERR_TIMEOUT = -10,  /* written to *status_word by a kernel whose bounded wait ran out */
    KLA_ERR_ARCH = -11,     /* current device is not sm_100                                */
    KLA_ERR_DEVICE = -12    /* the current device could not be queried, or (static scratch) its index is
                               beyond the table of scratch addresses or the address lookup failed */
} kla_status;

typedef enum { KLA_F32 = 0, KLA_BF16 = 1 } kla_dtype;

/* desc->flags */
#define KLA_FLAG_NONE 0
/* Force the CUDA-core fp32 chunk kernel even where the tensor-core kernel applies (used to
 * cross-check the two device paths against each other and against the oracle). */
#define KLA_FLAG_FORCE_SIMT 1
/* Layer-edge variants named by the paper; both default to off (the recurrence at the top of this file). */
#define KLA_FLAG_COEFF_ETA 4              /* beta_t = eta_t: the gated-delta-rule baseline coefficient of Section 2,
                                             without the key-norm division of Eq. 3 (eps is then unused)          */
#define KLA_FLAG_QNORM 8                  /* o_t = S_t^T q_t / ||q_t||: the read-out as Algorithm 1 (left) prints it */
/* Not part of the supported flag set: used by the library's own tests of the error path.  The tensor-core kernel
 * withholds one internal completion signal, so that a bounded device-side wait runs out (about one second), every
 * CTA gives up in an orderly way and KLA_ERR_TIMEOUT appears in *status_word.  Outputs are then undefined; the
 * context stays usable. */
#define KLA_INTERNAL_FLAG_TEST_TIMEOUT 16
/* With d_v = 128 the two CTAs that hold the two 64-column slices of a head run as a thread-block cluster and share
 * the work that does not depend on the state (each inverts every other chunk's I + B X and hands the result to its
 * peer through distributed shared memory).  This flag launches them as independent CTAs instead, each doing all of
 * that work itself; the arithmetic is the same, so the results are bit-identical.  Used to cross-check the two
 * launch forms. */
#define KLA_FLAG_NO_PAIR 32
/* Head dimension 128 only (ignored otherwise): run the chunk forward in the WY form of Appendix B (Props. 5-6 and the
 * combined representation U^ = U - W S_0, with W = T B D_gamma K and U = T B V formed on tensor cores off the serial
 * chain) instead of the default W-free form of Algorithm 1 right.  Same result up to rounding; the product W S_0 is
 * taken in fp16 (11 significand bits), which holds the 2e-3 bound on layer-shaped inputs but not on inputs with
 * heavy-tailed key norms, and needs the state and W inside the fp16 range. */
#define KLA_FLAG_WY_FORM 64
/* Segment-parallel scan of the tensor-core path (the transition-map form: fixed-length input only).  Every chunk step is affine in the
 * incoming state (Eqs. 7-9), so a sequence can be cut into G segments whose transition maps are found in
 * parallel, chained, and the segments then run in parallel from their true start states: the same result up
 * to rounding, about three times the state work, G times the parallelism.  By default the library decides
 * from the shape (few long sequences -> segments) and the workspace query returns what that decision needs. */
/* When the decay is strong enough the segments need no transition maps at all: the map over a run of tokens has norm
 * at most exp(sum of log_alpha) (every factor alpha (I - beta k k^T) has norm <= alpha when 0 <= eta <= 2, Eq. 3), so a
 * segment run from the zero state, started so many chunks early that this bound is below exp(-40), reaches its first
 * token with the exact state to fp32 accuracy.  A small kernel checks both conditions on the device (eta in [0, 2]
 * everywhere; for every segment and head a warm-up of at most min(half a segment, 2048 tokens)); if they hold, one pass
 * over the segments (plus their warm-up chunks) does the work, otherwise the transition-map passes do.  The decision is
 * taken on the device, the call stays asynchronous; the workspace need is the same either way.  Not attempted with
 * KLA_FLAG_COEFF_ETA (no bound on beta ||k||^2), KLA_FLAG_WY_FORM or KLA_FLAG_EXACT_SEGMENTS.
 * Packed input (cu_seqlens, tensor-core path, 2 <= n_seq <= 4096) is cut the same way, and only this way: when one
 * sequence would set the length of the launch (it is well beyond the work per SM of an even spread), or when
 * KLA_FLAG_SEGMENTS(g) asks for it (the longest sequence in g pieces, every sequence in pieces of that length), the long
 * sequences are cut into pieces that start from warm-up runs; if the decay does not allow that, the plain launch runs
 * instead (again decided on the device).  The workspace then also holds the piece tables. */
#define KLA_FLAG_NO_SEGMENTS 2            /* never cut sequences into segments                              */
#define KLA_FLAG_EXACT_SEGMENTS 128       /* segments always from chained transition maps, never from warm-up runs */
#define KLA_FLAG_SEGMENTS(g) ((g) << 8)   /* force g segments per sequence, 2 <= g <= 255 (fewer if T is short) */

typedef struct {
    int32_t B;        /* sequences in the batch; packed (varlen) input: 1                       */
    int32_t T;        /* tokens per sequence; packed input: total number of tokens              */
    int32_t H;        /* heads                                                                  */
    int32_t d_k;      /* key/query head dimension, 64 or 128                                    */
    int32_t d_v;      /* value head dimension, equal to d_k                                     */
    int32_t n_seq;    /* packed input: number of sequences; otherwise equal to B                */
    const int32_t *cu_seqlens;   /* DEVICE int32[n_seq + 1] cumulative token offsets, or NULL for
                                    fixed-length input.  Sequence n owns tokens
                                    cu_seqlens[n] .. cu_seqlens[n+1]-1 of the packed arrays.    */
    const int32_t *host_seqlens; /* HOST copy of the same array (used for validation and work
                                    partitioning); required when cu_seqlens is given            */
    int32_t io_dtype;   /* kla_dtype of q, k, v                                                 */
    int32_t out_dtype;  /* kla_dtype of out                                                     */
    int32_t flags;      /* KLA_FLAG_*                                                           */
    void *workspace;           /* DEVICE scratch of at least kla_chunk_fwd_workspace_bytes()    */
    size_t workspace_bytes;
    int32_t *status_word;      /* optional DEVICE int32, zeroed by the caller; a kernel whose
                                  bounded wait expires stores KLA_ERR_TIMEOUT there and exits  */
    void *stream;              /* cudaStream_t (NULL = default stream)                          */
} kla_desc;

/*
 * Scratch needed by kla_chunk_fwd for this descriptor (shape, dtypes, flags) and chunk length; 0 unless the
 * segment-parallel scan applies (then: per-segment transition maps and states, 3 x B x G x H x d_k x d_v fp32, after a block of
 * B G (H + 1) + 2 int32 padded to 256 bytes: segment bounds, plan word, warm-up lengths) or the
 * input is packed and goes to the tensor-core kernel (then: one int32 per sequence, for a longest-first order).
 * Computed on the host (it reads the current device's SM count when a device is present); returns 0 for an
 * invalid descriptor.  The same descriptor must be passed to kla_chunk_fwd with a workspace of at least this size.
 */
size_t kla_chunk_fwd_workspace_bytes(const kla_desc *desc, int32_t chunk);

/*
 * Byte offset, inside the workspace of a call with this descriptor and chunk length, of an int32 that holds after the
 * call 1 if the segments were started from decay-bounded warm-up runs and 0 if from chained transition maps (see
 * KLA_FLAG_EXACT_SEGMENTS); (size_t)-1 when the call does not cut its sequences into segments.  Host function.
 */
size_t kla_chunk_fwd_plan_word_offset(const kla_desc *desc, int32_t chunk);

/*
 * Chunkwise-parallel forward (Algorithm 1 right; Eqs. 7-9; Props. 3-4).
 *
 *   q, k        [B, T, H, d_k]   io_dtype          (packed: [1, n_tok, H, d_k])
 *   v           [B, T, H, d_v]   io_dtype
 *   log_alpha   [B, T, H]        fp32, log of the scalar decay alpha_t in (0, 1]
 *   eta         [B, T, H]        fp32, relaxation gate (a sigmoid output in the paper)
 *   eps         stabiliser of Eq. 3, >= 0.  eps = 0 with an all-zero key gives NaN (IEEE 0/0).
 *   chunk       chunk length C in {16, 32, 64}; the tensor-core kernel requires 64
 *   init_state  [n_seq, H, d_k, d_v] fp32 state before the first token, or NULL for zeros;
 *               never written
 *   out         [B, T, H, d_v]   out_dtype, fully overwritten
 *   final_state [n_seq, H, d_k, d_v] fp32 state after the last token, or NULL to skip; fully
 *               overwritten; a zero-length sequence gets its initial state
 *
 * State layout: S[i][j], i over d_k, j over d_v, j contiguous (Section 2), so o_t = S_t^T q_t.
 * Arithmetic: bf16 inputs are used exactly; every contraction accumulates in fp32 and the
 * carried state stays in fp32.
 */
kla_status kla_chunk_fwd(const kla_desc *desc, const void *q, const void *k, const void *v,
                         const float *log_alpha, const float *eta, float eps, int32_t chunk,
                         const float *init_state, void *out, float *final_state);

/*
 * The same chunk forward for callers that cannot allocate device memory (no counterpart in the paper: this is a
 * property of the library, not of the method).  kla_chunk_fwd needs a caller-provided workspace whenever it cuts
 * long sequences into segments; a caller that has no allocator at hand -- code inside a region where its framework
 * serves no allocations, a plugin that is handed nothing but its input and output buffers, a binding without
 * cudaMalloc -- calls this instead.  desc->workspace and desc->workspace_bytes are ignored: the scratch is a fixed
 * array of KLA_STATIC_SCRATCH_BYTES inside the library image, which every GPU that loads the library holds until
 * the process exits.  The call itself allocates and frees nothing, on host or device.
 *
 *  - A shape whose scratch would exceed KLA_STATIC_SCRATCH_BYTES is refused with KLA_ERR_WORKSPACE before
 *    anything is launched (kla_chunk_fwd_workspace_bytes tells what a shape needs; KLA_FLAG_NO_SEGMENTS makes
 *    the need zero at the price of less parallelism).
 *  - The first call on each device looks up that device's address of the array (with the device current, as
 *    for every call); make that first call outside any stream capture.  With the CUDA runtime's lazy module
 *    loading this is also when the device sets the array aside.
 *  - All calls share the one array and it keeps the previous call's contents.  Nothing in it has to start at
 *    zero (a call writes every byte it later reads), but two calls that overlap on the GPU -- different streams,
 *    or host threads racing on one stream -- would overwrite each other's segments: serialise them.
 *  - Arguments are validated exactly as by kla_chunk_fwd (same codes, same order, except that the workspace fields
 *    are not looked at); then comes the size check above; KLA_ERR_DEVICE if the current device's index is beyond the
 *    library's table of scratch addresses (64 devices) or the address lookup fails.  Layouts and results are those
 *    of kla_chunk_fwd.
 */
#define KLA_STATIC_SCRATCH_BYTES (32u << 20)
kla_status kla_chunk_fwd_static_scratch(const kla_desc *desc, const void *q, const void *k, const void *v,
                                        const float *log_alpha, const float *eta, float eps, int32_t chunk,
                                        const float *init_state, void *out, float *final_state);

/*
 * kla_chunk_fwd with per-pass device times (a measurement aid; no counterpart in the paper).  Does exactly the work
 * of kla_chunk_fwd with the same arguments, records CUDA events on desc->stream between the launches, waits for
 * the stream and writes milliseconds to the HOST array pass_ms[4]:
 *   [0] set-up kernels (segment bounds or the order of packed sequences), [1] segment pass 1 (transition maps),
 *   [2] the chaining of the segment maps, [3] the main pass (segment pass 3, or the only pass of a plain launch).
 * Entries of passes that did not run are 0.  Synchronises with the stream (unlike kla_chunk_fwd); creates and
 * destroys four CUDA events; otherwise allocates nothing.
 */
kla_status kla_chunk_fwd_timed(const kla_desc *desc, const void *q, const void *k, const void *v,
                               const float *log_alpha, const float *eta, float eps, int32_t chunk,
                               const float *init_state, void *out, float *final_state, float *pass_ms);

/*
 * Sequence-parallel prefill: one long sequence cut along T across several GPUs (the affine form of Appendix B: every
 * chunk step, hence every span of tokens, maps the incoming state S to Phi S + N).  Each GPU holds one span of the
 * sequence and (1) calls kla_chunk_span_map on it, (2) exchanges (Phi, N) with the other GPUs (one all-gather of
 * 2 x B x H x d_k x d_k fp32 per GPU; the library has no communication of its own), (3) calls kla_state_chain on the
 * gathered maps to get the state at the start of its span, (4) calls kla_chunk_fwd on its span with that state.
 *
 * kla_chunk_span_map: transition map of the whole input (head dimension 128 or 64, bf16, chunk 64, fixed length).
 *   q is not read (no outputs are formed) and may be NULL.
 *   phi_out [B, H, d_k, d_k] fp32: the state reached from the identity with v = 0 (S_end = phi_out . S_start + n_out)
 *   n_out   [B, H, d_k, d_v] fp32: the state reached from zero
 *   desc->workspace: at least kla_chunk_span_map_workspace_bytes(desc) bytes.
 *
 * kla_state_chain: start states of R consecutive spans from their maps, in fp32:
 *   start[b, 0] = init_state[b] (or 0);  start[b, r + 1] = phi[b, r] . start[b, r] + n[b, r]
 *   phi, n [B, R, H, d, d] fp32 (the maps of spans 0 .. R-2 are read); start_out [B, R, H, d, d] fp32.
 *   Uses desc->B, H, d_k, stream only.
 */
size_t kla_chunk_span_map_workspace_bytes(const kla_desc *desc);
kla_status kla_chunk_span_map(const kla_desc *desc, const void *k, const void *v, const float *log_alpha, const float *eta,
                              float eps, float *phi_out, float *n_out);
kla_status kla_state_chain(const kla_desc *desc, int32_t n_spans, const float *init_state, const float *phi, const float *n,
                           float *start_out);

/*
 * One recurrent decode step (Algorithm 1 left) for B sequences x H heads; desc->T must be 1 and
 * desc->cu_seqlens NULL.
 *
 *   q, k [B, H, d_k]   v [B, H, d_v]  io_dtype;   log_alpha, eta [B, H] fp32
 *   state_inout [B, H, d_k, d_v] fp32, read once and overwritten in place with S_t
 *   out [B, H, d_v] out_dtype
 */
kla_status kla_decode_step(const kla_desc *desc, const void *q, const void *k, const void *v,
                           const float *log_alpha, const float *eta, float eps,
                           float *state_inout, void *out);

/*
 * n_steps consecutive decode steps enqueued back to back on desc->stream (Algorithm 1 left applied
 * to tokens 0 .. n_steps-1).  Step s reads q + s*B*H*d_k (and likewise k, v, log_alpha, eta) and
 * writes out + s*B*H*d_v; the state is carried in place.  Equivalent to n_steps calls of
 * kla_decode_step; exists so that a host loop in an interpreted language is not the bottleneck.
 */
kla_status kla_decode_steps(const kla_desc *desc, int32_t n_steps, const void *q, const void *k,
                            const void *v, const float *log_alpha, const float *eta, float eps,
                            float *state_inout, void *out);

/*
 * Diagonal-gated KLA (Appendix B.5, "Extension to diagonal gating"; the decay-agnostic remark of Appendix A): the decay
 * of the recurrence at the top of this file becomes a vector over d_k,
 *
 *     S~ = diag(exp(log_alpha_t)) S_{t-1}         (row i of the state decays by exp(log_alpha_t[i])),
 *
 * and the residual, the coefficient of Eq. 3, the write and the read-out are unchanged.  Arguments as kla_chunk_fwd /
 * kla_decode_step except
 *   log_alpha   [B, T, H, d_k] fp32 (decode: [B, H, d_k])
 * and no chunk length, workspace or segment flags: the recurrence is evaluated token by token on CUDA cores, in fp32,
 * with the state of every (sequence, head) in registers (the chunkwise form with elementwise decay products is not
 * built).  Packed input (cu_seqlens), KLA_FLAG_COEFF_ETA and KLA_FLAG_QNORM are supported; fp32 or bf16 q, k, v.
 */
kla_status kla_dg_fwd(const kla_desc *desc, const void *q, const void *k, const void *v,
                      const float *log_alpha, const float *eta, float eps,
                      const float *init_state, void *out, float *final_state);
kla_status kla_dg_decode_step(const kla_desc *desc, const void *q, const void *k, const void *v,
                              const float *log_alpha, const float *eta, float eps,
                              float *state_inout, void *out);

/*
 * Backward pass (training, Section 5.1): gradients of a scalar loss L through the recurrence at the top of this file.
 * The paper prints no backward; this is reverse-mode differentiation of Algorithm 1 (left) with the coefficient of
 * Eq. 3, token by token in reverse order (G = dL/dS_t carried backwards):
 *
 *     G += q dO_t^T ;  dq_t = S_t dO_t                                   (read-out)
 *     dbeta = k^T G e ;  dk_t = beta G e ;  de = beta G^T k              (write)
 *     dv_t = de ;  dk_t -= S~ de ;  G -= k de^T                          (residual)
 *     deta_t = dbeta / n ;  dk_t -= 2 k dbeta beta / n, n = ||k||^2+eps  (coefficient, Eq. 3)
 *     dlog_alpha_t = <G, S~> ;  G <- alpha_t G                           (decay)
 *
 * Inputs q, k, v, log_alpha, eta, eps, init_state: as kla_chunk_fwd (fixed-length or packed through desc->cu_seqlens /
 * host_seqlens; desc->io_dtype; KLA_FLAG_COEFF_ETA and KLA_FLAG_QNORM are honoured, other flags ignored).
 *   d_out          [B, T, H, d_v] io_dtype, dL/dout
 *   d_final_state  [n_seq, H, d_k, d_v] fp32, dL/dfinal_state, or NULL for zeros
 *   dq, dk         [B, T, H, d_k] fp32; dv [B, T, H, d_v] fp32; dlog_alpha, deta [B, T, H] fp32: fully overwritten
 *   dinit_state    [n_seq, H, d_k, d_v] fp32, dL/dinit_state, or NULL to skip; an empty sequence gets d_final_state
 * All arithmetic is fp32 on CUDA cores.  The forward states are not an input: they are recomputed (a state is kept every
 * 16 tokens on a forward sweep, the ones in between are re-run when the reverse sweep reaches them), which needs
 * desc->workspace of kla_bwd_workspace_bytes(desc) bytes: (B T / 16 + n_seq) x H x d_k x d_v fp32 for the kept states,
 * 16 x 64 x d_k fp32 of scratch per resident thread block (at most one per SM) and 256 bytes (host function; it reads
 * the current device's SM count when a device is present; 0 for an invalid descriptor).  Errors as kla_chunk_fwd.
 */
size_t kla_bwd_workspace_bytes(const kla_desc *desc);
kla_status kla_bwd(const kla_desc *desc, const void *q, const void *k, const void *v,
                   const float *log_alpha, const float *eta, float eps, const float *init_state,
                   const void *d_out, const float *d_final_state,
                   float *dq, float *dk, float *dv, float *dlog_alpha, float *deta, float *dinit_state);

/* Static, NUL-terminated description of a status code. */
const char *kla_status_str(kla_status s);

/* Number of kernels the library has launched in this process so far (monotone counter; host). */
uint64_t kla_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* KLA_H_ */
