"""Thin Python binding of the C ABI declared in include/kla.h: argument marshalling only.

PyTorch supplies device memory and the current stream; every arithmetic step of the path runs in
the library's CUDA kernels.  There is no fallback: a missing library raises at import of the
symbols, and a non-zero status raises `KlaError`.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libkla_b200.so")

KLA_F32, KLA_BF16 = 0, 1
KLA_FLAG_NONE, KLA_FLAG_FORCE_SIMT, KLA_FLAG_NO_SEGMENTS = 0, 1, 2
KLA_FLAG_COEFF_ETA, KLA_FLAG_QNORM, KLA_INTERNAL_FLAG_TEST_TIMEOUT, KLA_FLAG_NO_PAIR, KLA_FLAG_WY_FORM = 4, 8, 16, 32, 64
KLA_FLAG_EXACT_SEGMENTS = 128


def KLA_FLAG_SEGMENTS(g: int) -> int:
    """Force g segments per sequence in the segment-parallel scan (include/kla.h)."""
    return int(g) << 8


EXPORTS = ["kla_chunk_fwd_workspace_bytes", "kla_chunk_fwd_plan_word_offset", "kla_chunk_fwd", "kla_chunk_fwd_timed", "kla_chunk_fwd_static_scratch",
           "kla_chunk_span_map_workspace_bytes", "kla_chunk_span_map", "kla_state_chain", "kla_dg_fwd", "kla_dg_decode_step", "kla_bwd_workspace_bytes", "kla_bwd", "kla_decode_step", "kla_decode_steps",
           "kla_status_str", "kla_launch_count"]


class KlaError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__("kla status %d: %s" % (code, msg))
        self.code = code


class KlaDesc(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("T", ctypes.c_int32), ("H", ctypes.c_int32),
                ("d_k", ctypes.c_int32), ("d_v", ctypes.c_int32), ("n_seq", ctypes.c_int32),
                ("cu_seqlens", ctypes.c_void_p), ("host_seqlens", ctypes.c_void_p),
                ("io_dtype", ctypes.c_int32), ("out_dtype", ctypes.c_int32), ("flags", ctypes.c_int32),
                ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t),
                ("status_word", ctypes.c_void_p), ("stream", ctypes.c_void_p)]


_lib = None


def load():
    """Load libkla_b200.so (built in-tree by `paper_2605_08587_b200.build`).  Raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise FileNotFoundError("%s not found: run `python -m paper_2605_08587_b200.build` "
                                "(there is no CPU or PyTorch fallback)" % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    vp, fp, dp = ctypes.c_void_p, ctypes.c_void_p, ctypes.POINTER(KlaDesc)
    lib.kla_chunk_fwd_workspace_bytes.restype = ctypes.c_size_t
    lib.kla_chunk_fwd_workspace_bytes.argtypes = [dp, ctypes.c_int32]
    lib.kla_chunk_fwd_plan_word_offset.restype = ctypes.c_size_t
    lib.kla_chunk_fwd_plan_word_offset.argtypes = [dp, ctypes.c_int32]
    lib.kla_chunk_fwd.restype = ctypes.c_int
    lib.kla_chunk_fwd.argtypes = [dp, vp, vp, vp, fp, fp, ctypes.c_float, ctypes.c_int32, fp, vp, fp]
    lib.kla_chunk_fwd_timed.restype = ctypes.c_int
    lib.kla_chunk_fwd_timed.argtypes = lib.kla_chunk_fwd.argtypes + [ctypes.POINTER(ctypes.c_float)]
    lib.kla_chunk_fwd_static_scratch.restype = ctypes.c_int
    lib.kla_chunk_fwd_static_scratch.argtypes = lib.kla_chunk_fwd.argtypes
    lib.kla_chunk_span_map_workspace_bytes.restype = ctypes.c_size_t
    lib.kla_chunk_span_map_workspace_bytes.argtypes = [dp]
    lib.kla_chunk_span_map.restype = ctypes.c_int
    lib.kla_chunk_span_map.argtypes = [dp, vp, vp, fp, fp, ctypes.c_float, fp, fp]
    lib.kla_state_chain.restype = ctypes.c_int
    lib.kla_state_chain.argtypes = [dp, ctypes.c_int32, fp, fp, fp, fp]
    lib.kla_decode_step.restype = ctypes.c_int
    lib.kla_decode_step.argtypes = [dp, vp, vp, vp, fp, fp, ctypes.c_float, fp, vp]
    lib.kla_dg_fwd.restype = ctypes.c_int
    lib.kla_dg_fwd.argtypes = [dp, vp, vp, vp, fp, fp, ctypes.c_float, fp, vp, fp]
    lib.kla_dg_decode_step.restype = ctypes.c_int
    lib.kla_dg_decode_step.argtypes = lib.kla_decode_step.argtypes
    lib.kla_bwd_workspace_bytes.restype = ctypes.c_size_t
    lib.kla_bwd_workspace_bytes.argtypes = [dp]
    lib.kla_bwd.restype = ctypes.c_int
    lib.kla_bwd.argtypes = [dp, vp, vp, vp, fp, fp, ctypes.c_float, fp, vp, fp] + [fp] * 6
    lib.kla_decode_steps.restype = ctypes.c_int
    lib.kla_decode_steps.argtypes = [dp, ctypes.c_int32, vp, vp, vp, fp, fp, ctypes.c_float, fp, vp]
    lib.kla_status_str.restype = ctypes.c_char_p
    lib.kla_status_str.argtypes = [ctypes.c_int]
    lib.kla_launch_count.restype = ctypes.c_uint64
    lib.kla_launch_count.argtypes = []
    _lib = lib
    return lib


def status_str(code: int) -> str:
    return load().kla_status_str(int(code)).decode()


def launch_count() -> int:
    return int(load().kla_launch_count())


def _check(code):
    if code != 0:
        raise KlaError(code, status_str(code))


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return KLA_F32
    if t.dtype == torch.bfloat16:
        return KLA_BF16
    raise TypeError("q, k, v, out must be float32 or bfloat16, got %s" % t.dtype)


def _dev(t, name, dtype=None):
    if t is None:
        return None
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous()):
        raise ValueError("%s must be a contiguous CUDA tensor" % name)
    if dtype is not None and t.dtype != dtype:
        raise TypeError("%s must be %s" % (name, dtype))
    return t.data_ptr()


_own_status = {}   # device index -> int32[1] the binding passes as status word when the caller gives none


def _status_for(dev):
    i = torch.device(dev).index
    i = torch.cuda.current_device() if i is None else i
    if i not in _own_status:
        _own_status[i] = torch.zeros(1, dtype=torch.int32, device="cuda:%d" % i)
    return _own_status[i]


def check(device=None):
    """Reads (and clears) the status word the binding passes to kla_chunk_fwd when the caller gives none: raises KlaError
    if a kernel on `device` (default: the current one) gave up on a bounded wait since the last check -- its outputs are
    then undefined.  Waits for the device; meant for the end of a step, not for the hot path."""
    i = torch.cuda.current_device() if device is None else torch.device(device).index
    word = _own_status.get(i)
    if word is None:
        return
    code = int(word.item())
    if code != 0:
        word.zero_()
        raise KlaError(code, status_str(code))


def _stream(dev):
    return torch.cuda.current_stream(dev).cuda_stream


def kla_chunk_fwd(q, k, v, log_alpha, eta, eps, chunk=64, init_state=None, out=None, final_state=None,
                  cu_seqlens=None, host_seqlens=None, out_dtype=None, flags=KLA_FLAG_NONE,
                  want_final_state=True, status_word=None, pass_ms=None, plan_word=None):
    """Chunkwise forward (include/kla.h: kla_chunk_fwd).

    q, k [B, T, H, d_k]; v [B, T, H, d_v]; log_alpha, eta [B, T, H] fp32; all CUDA, contiguous.
    Packed input: B = 1, cu_seqlens int32 CUDA [n_seq + 1] plus `host_seqlens` (CPU int32 copy;
    made from cu_seqlens with one D2H copy if omitted).
    Returns (out, final_state); buffers are allocated here unless passed in.
    `status_word`: CUDA int32[1], zeroed by the caller, that receives KLA_ERR_TIMEOUT if a bounded device-side wait runs
    out; if None the binding passes one of its own per device, read and cleared by `check()`.
    `plan_word`: a list; if given, the int32 of kla_chunk_fwd_plan_word_offset is read back after the call (which
    waits for the device) and appended: 1 = segments started from warm-up runs, 0 = from chained maps, None = no segments.
    `pass_ms`: a list; if given the call goes through kla_chunk_fwd_timed (which waits for the stream) and the four
    per-pass device times in ms (set-up, segment pass 1, chaining, main pass) are appended to it.
    """
    lib = load()
    B, T, H, d_k = q.shape
    d_v = v.shape[-1]
    if tuple(k.shape) != (B, T, H, d_k) or tuple(v.shape) != (B, T, H, d_v):
        raise ValueError("q, k, v shapes disagree")
    if tuple(log_alpha.shape) != (B, T, H) or tuple(eta.shape) != (B, T, H):
        raise ValueError("log_alpha, eta must be [B, T, H]")
    if k.dtype != q.dtype or v.dtype != q.dtype:
        raise TypeError("q, k, v must share one dtype")
    n_seq = B
    hs = None
    if cu_seqlens is not None:
        if cu_seqlens.dtype != torch.int32:
            raise TypeError("cu_seqlens must be int32")
        hs = (cu_seqlens.cpu() if host_seqlens is None else host_seqlens).contiguous()
        if hs.dtype != torch.int32 or hs.is_cuda:
            raise TypeError("host_seqlens must be a CPU int32 tensor")
        n_seq = cu_seqlens.numel() - 1
    if out is None:
        out = torch.empty((B, T, H, d_v), device=q.device, dtype=out_dtype or q.dtype)
    if final_state is None and want_final_state:
        final_state = torch.empty((n_seq, H, d_k, d_v), device=q.device, dtype=torch.float32)
    if init_state is not None and tuple(init_state.shape) != (n_seq, H, d_k, d_v):
        raise ValueError("init_state must be [n_seq, H, d_k, d_v]")
    if status_word is None:   # a timeout must not pass unnoticed: see check()
        status_word = _status_for(q.device)
    desc = KlaDesc(B=B, T=T, H=H, d_k=d_k, d_v=d_v, n_seq=n_seq,
                   cu_seqlens=_dev(cu_seqlens, "cu_seqlens"), host_seqlens=hs.data_ptr() if hs is not None else None,
                   io_dtype=_dt(q), out_dtype=_dt(out), flags=flags, workspace=None, workspace_bytes=0,
                   status_word=_dev(status_word, "status_word", torch.int32), stream=_stream(q.device))
    ws = None
    need = lib.kla_chunk_fwd_workspace_bytes(ctypes.byref(desc), chunk)
    if need:
        ws = torch.empty(need, device=q.device, dtype=torch.uint8)
        desc.workspace, desc.workspace_bytes = ws.data_ptr(), need
    args = (ctypes.byref(desc), _dev(q, "q"), _dev(k, "k"), _dev(v, "v"),
            _dev(log_alpha, "log_alpha", torch.float32), _dev(eta, "eta", torch.float32),
            float(eps), int(chunk), _dev(init_state, "init_state", torch.float32),
            _dev(out, "out"), _dev(final_state, "final_state", torch.float32))
    with torch.cuda.device(q.device):
        if pass_ms is None:
            code = lib.kla_chunk_fwd(*args)
        else:
            ms = (ctypes.c_float * 4)()
            code = lib.kla_chunk_fwd_timed(*args, ms)
            pass_ms.extend(float(x) for x in ms)
    _check(code)
    if plan_word is not None:
        off = lib.kla_chunk_fwd_plan_word_offset(ctypes.byref(desc), chunk)
        plan_word.append(None if off == ctypes.c_size_t(-1).value or ws is None else int(ws[off:off + 4].view(torch.int32).item()))
    return out, final_state


STATIC_SCRATCH_BYTES = 32 << 20


def kla_chunk_fwd_static_scratch(q, k, v, log_alpha, eta, eps, out, final_state=None, chunk=64, init_state=None,
                                 flags=KLA_FLAG_NONE, cu_seqlens=None, host_seqlens=None, status_word=None):
    """Chunk forward for callers that cannot allocate device memory (include/kla.h:
    kla_chunk_fwd_static_scratch).  The scratch (segment-parallel scan; longest-first order of packed sequences) is a
    fixed array inside the library, so this wrapper allocates nothing either: `out` (and `final_state`, if wanted) must
    be passed in, and for packed input both `cu_seqlens` (CUDA int32) and `host_seqlens` (CPU int32 copy).  Shapes whose
    scratch would exceed STATIC_SCRATCH_BYTES raise KlaError (workspace).  Calls must not overlap on the GPU."""
    lib = load()
    B, T, H, d_k = q.shape
    d_v = v.shape[-1]
    if tuple(k.shape) != (B, T, H, d_k) or tuple(v.shape) != (B, T, H, d_v) or tuple(out.shape) != (B, T, H, d_v):
        raise ValueError("q, k, v, out shapes disagree")
    if tuple(log_alpha.shape) != (B, T, H) or tuple(eta.shape) != (B, T, H):
        raise ValueError("log_alpha, eta must be [B, T, H]")
    n_seq = B
    if cu_seqlens is not None:
        if host_seqlens is None or host_seqlens.is_cuda or host_seqlens.dtype != torch.int32 or cu_seqlens.dtype != torch.int32:
            raise TypeError("packed input needs cu_seqlens (CUDA int32) and host_seqlens (CPU int32)")
        n_seq = cu_seqlens.numel() - 1
    desc = KlaDesc(B=B, T=T, H=H, d_k=d_k, d_v=d_v, n_seq=n_seq, cu_seqlens=_dev(cu_seqlens, "cu_seqlens"),
                   host_seqlens=host_seqlens.data_ptr() if host_seqlens is not None else None,
                   io_dtype=_dt(q), out_dtype=_dt(out), flags=flags, workspace=None, workspace_bytes=0,
                   status_word=_dev(status_word, "status_word", torch.int32), stream=_stream(q.device))
    with torch.cuda.device(q.device):
        code = lib.kla_chunk_fwd_static_scratch(
            ctypes.byref(desc), _dev(q, "q"), _dev(k, "k"), _dev(v, "v"), _dev(log_alpha, "log_alpha", torch.float32),
            _dev(eta, "eta", torch.float32), float(eps), int(chunk), _dev(init_state, "init_state", torch.float32),
            _dev(out, "out"), _dev(final_state, "final_state", torch.float32))
    _check(code)
    return out, final_state


def kla_chunk_span_map(k, v, log_alpha, eta, eps, flags=KLA_FLAG_NONE):
    """Transition map of a span of tokens (include/kla.h: kla_chunk_span_map): S_end = phi . S_start + n.
    k [B, T, H, d]; v [B, T, H, d]; log_alpha, eta [B, T, H]; bf16 inputs.  Returns (phi, n), both [B, H, d, d] fp32."""
    lib = load()
    B, T, H, d = k.shape
    phi = torch.empty((B, H, d, d), device=k.device, dtype=torch.float32)
    n = torch.empty((B, H, d, d), device=k.device, dtype=torch.float32)
    desc = KlaDesc(B=B, T=T, H=H, d_k=d, d_v=v.shape[-1], n_seq=B, cu_seqlens=None, host_seqlens=None, io_dtype=_dt(k),
                   out_dtype=KLA_F32, flags=flags, workspace=None, workspace_bytes=0, status_word=None, stream=_stream(k.device))
    need = lib.kla_chunk_span_map_workspace_bytes(ctypes.byref(desc))
    ws = torch.empty(max(need, 16), device=k.device, dtype=torch.uint8)
    desc.workspace, desc.workspace_bytes = ws.data_ptr(), need
    with torch.cuda.device(k.device):
        code = lib.kla_chunk_span_map(ctypes.byref(desc), _dev(k, "k"), _dev(v, "v"), _dev(log_alpha, "log_alpha", torch.float32),
                                      _dev(eta, "eta", torch.float32), float(eps), phi.data_ptr(), n.data_ptr())
    _check(code)
    return phi, n


def kla_state_chain(phi, n, init_state=None):
    """Start states of R consecutive spans from their maps (include/kla.h: kla_state_chain).
    phi, n [B, R, H, d, d] fp32; init_state [B, H, d, d] fp32 or None (zeros).  Returns start [B, R, H, d, d] fp32 with
    start[:, 0] = init_state and start[:, r + 1] = phi[:, r] . start[:, r] + n[:, r]."""
    lib = load()
    B, R, H, d, _ = phi.shape
    start = torch.empty_like(phi)
    desc = KlaDesc(B=B, T=1, H=H, d_k=d, d_v=d, n_seq=B, cu_seqlens=None, host_seqlens=None, io_dtype=KLA_BF16, out_dtype=KLA_F32,
                   flags=0, workspace=None, workspace_bytes=0, status_word=None, stream=_stream(phi.device))
    with torch.cuda.device(phi.device):
        code = lib.kla_state_chain(ctypes.byref(desc), R, _dev(init_state, "init_state", torch.float32), _dev(phi, "phi", torch.float32),
                                   _dev(n, "n", torch.float32), start.data_ptr())
    _check(code)
    return start


def _decode_desc(q, v, out, B, H, d_k, d_v, flags=0):
    return KlaDesc(B=B, T=1, H=H, d_k=d_k, d_v=d_v, n_seq=B, cu_seqlens=None, host_seqlens=None,
                   io_dtype=_dt(q), out_dtype=_dt(out), flags=flags, workspace=None, workspace_bytes=0,
                   status_word=None, stream=_stream(q.device))


def kla_decode_step(q, k, v, log_alpha, eta, eps, state_inout, out=None, out_dtype=None, flags=KLA_FLAG_NONE):
    """One decode step (include/kla.h: kla_decode_step).  q, k [B, H, d_k]; v [B, H, d_v];
    log_alpha, eta [B, H] fp32; state_inout [B, H, d_k, d_v] fp32, updated in place."""
    lib = load()
    B, H, d_k = q.shape
    d_v = v.shape[-1]
    if out is None:
        out = torch.empty((B, H, d_v), device=q.device, dtype=out_dtype or q.dtype)
    desc = _decode_desc(q, v, out, B, H, d_k, d_v, flags)
    with torch.cuda.device(q.device):
        code = lib.kla_decode_step(ctypes.byref(desc), _dev(q, "q"), _dev(k, "k"), _dev(v, "v"),
                                   _dev(log_alpha, "log_alpha", torch.float32), _dev(eta, "eta", torch.float32),
                                   float(eps), _dev(state_inout, "state_inout", torch.float32), _dev(out, "out"))
    _check(code)
    return out


def kla_decode_steps(q, k, v, log_alpha, eta, eps, state_inout, out=None, out_dtype=None, flags=KLA_FLAG_NONE):
    """n consecutive decode steps (include/kla.h: kla_decode_steps).  q, k [n, B, H, d_k];
    v [n, B, H, d_v]; log_alpha, eta [n, B, H]; state carried in place; out [n, B, H, d_v]."""
    lib = load()
    n, B, H, d_k = q.shape
    d_v = v.shape[-1]
    if out is None:
        out = torch.empty((n, B, H, d_v), device=q.device, dtype=out_dtype or q.dtype)
    desc = _decode_desc(q, v, out, B, H, d_k, d_v, flags)
    with torch.cuda.device(q.device):
        code = lib.kla_decode_steps(ctypes.byref(desc), n, _dev(q, "q"), _dev(k, "k"), _dev(v, "v"),
                                    _dev(log_alpha, "log_alpha", torch.float32), _dev(eta, "eta", torch.float32),
                                    float(eps), _dev(state_inout, "state_inout", torch.float32), _dev(out, "out"))
    _check(code)
    return out


def kla_dg_fwd(q, k, v, log_alpha, eta, eps, init_state=None, out=None, final_state=None, cu_seqlens=None, host_seqlens=None,
               out_dtype=None, flags=KLA_FLAG_NONE, want_final_state=True):
    """Diagonal-gated forward (include/kla.h: kla_dg_fwd): as kla_chunk_fwd with log_alpha [B, T, H, d_k], one decay per
    row of the state.  Returns (out, final_state)."""
    lib = load()
    B, T, H, d_k = q.shape
    d_v = v.shape[-1]
    if tuple(log_alpha.shape) != (B, T, H, d_k) or tuple(eta.shape) != (B, T, H):
        raise ValueError("log_alpha must be [B, T, H, d_k] and eta [B, T, H]")
    n_seq, hs = B, None
    if cu_seqlens is not None:
        hs = (cu_seqlens.cpu() if host_seqlens is None else host_seqlens).contiguous()
        n_seq = cu_seqlens.numel() - 1
    if out is None:
        out = torch.empty((B, T, H, d_v), device=q.device, dtype=out_dtype or q.dtype)
    if final_state is None and want_final_state:
        final_state = torch.empty((n_seq, H, d_k, d_v), device=q.device, dtype=torch.float32)
    desc = KlaDesc(B=B, T=T, H=H, d_k=d_k, d_v=d_v, n_seq=n_seq, cu_seqlens=_dev(cu_seqlens, "cu_seqlens"),
                   host_seqlens=hs.data_ptr() if hs is not None else None, io_dtype=_dt(q), out_dtype=_dt(out), flags=flags,
                   workspace=None, workspace_bytes=0, status_word=None, stream=_stream(q.device))
    with torch.cuda.device(q.device):
        code = lib.kla_dg_fwd(ctypes.byref(desc), _dev(q, "q"), _dev(k, "k"), _dev(v, "v"), _dev(log_alpha, "log_alpha", torch.float32),
                              _dev(eta, "eta", torch.float32), float(eps), _dev(init_state, "init_state", torch.float32),
                              _dev(out, "out"), _dev(final_state, "final_state", torch.float32))
    _check(code)
    return out, final_state


def kla_bwd(q, k, v, log_alpha, eta, eps, d_out, init_state=None, d_final_state=None, cu_seqlens=None, host_seqlens=None,
            flags=KLA_FLAG_NONE, want_dinit_state=True, workspace=None):
    """Backward pass (include/kla.h: kla_bwd): gradients of a scalar loss given d_out = dL/dout (dtype of q) and
    d_final_state = dL/dfinal_state (or None).  Returns a dict of fp32 tensors dq, dk, dv, dlog_alpha, deta and
    dinit_state (None unless asked for).  `workspace`: a uint8 CUDA tensor of at least kla_bwd_workspace_bytes, else
    one is allocated here."""
    lib = load()
    B, T, H, d_k = q.shape
    d_v = v.shape[-1]
    if tuple(d_out.shape) != (B, T, H, d_v) or d_out.dtype != q.dtype:
        raise ValueError("d_out must be [B, T, H, d_v] with the dtype of q")
    n_seq, hs = B, None
    if cu_seqlens is not None:
        hs = (cu_seqlens.cpu() if host_seqlens is None else host_seqlens).contiguous()
        n_seq = cu_seqlens.numel() - 1
    f32 = dict(device=q.device, dtype=torch.float32)
    g = dict(dq=torch.empty((B, T, H, d_k), **f32), dk=torch.empty((B, T, H, d_k), **f32), dv=torch.empty((B, T, H, d_v), **f32),
             dlog_alpha=torch.empty((B, T, H), **f32), deta=torch.empty((B, T, H), **f32),
             dinit_state=torch.empty((n_seq, H, d_k, d_v), **f32) if want_dinit_state else None)
    desc = KlaDesc(B=B, T=T, H=H, d_k=d_k, d_v=d_v, n_seq=n_seq, cu_seqlens=_dev(cu_seqlens, "cu_seqlens"),
                   host_seqlens=hs.data_ptr() if hs is not None else None, io_dtype=_dt(q), out_dtype=KLA_F32, flags=flags,
                   workspace=None, workspace_bytes=0, status_word=None, stream=_stream(q.device))
    need = int(lib.kla_bwd_workspace_bytes(ctypes.byref(desc)))
    if workspace is None and need > 0:
        workspace = torch.empty(need, device=q.device, dtype=torch.uint8)
    if workspace is not None:
        desc.workspace = _dev(workspace, "workspace")
        desc.workspace_bytes = workspace.numel() * workspace.element_size()
    with torch.cuda.device(q.device):
        code = lib.kla_bwd(ctypes.byref(desc), _dev(q, "q"), _dev(k, "k"), _dev(v, "v"), _dev(log_alpha, "log_alpha", torch.float32),
                           _dev(eta, "eta", torch.float32), float(eps), _dev(init_state, "init_state", torch.float32),
                           _dev(d_out, "d_out"), _dev(d_final_state, "d_final_state", torch.float32),
                           _dev(g["dq"], "dq"), _dev(g["dk"], "dk"), _dev(g["dv"], "dv"), _dev(g["dlog_alpha"], "dlog_alpha"),
                           _dev(g["deta"], "deta"), _dev(g["dinit_state"], "dinit_state"))
    _check(code)
    return g


def kla_dg_decode_step(q, k, v, log_alpha, eta, eps, state_inout, out=None, out_dtype=None, flags=KLA_FLAG_NONE):
    """One diagonal-gated decode step (include/kla.h: kla_dg_decode_step): log_alpha [B, H, d_k]; state updated in place."""
    lib = load()
    B, H, d_k = q.shape
    d_v = v.shape[-1]
    if out is None:
        out = torch.empty((B, H, d_v), device=q.device, dtype=out_dtype or q.dtype)
    desc = _decode_desc(q, v, out, B, H, d_k, d_v, flags)
    with torch.cuda.device(q.device):
        code = lib.kla_dg_decode_step(ctypes.byref(desc), _dev(q, "q"), _dev(k, "k"), _dev(v, "v"),
                                      _dev(log_alpha, "log_alpha", torch.float32), _dev(eta, "eta", torch.float32), float(eps),
                                      _dev(state_inout, "state_inout", torch.float32), _dev(out, "out"))
    _check(code)
    return out
