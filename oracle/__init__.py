"""fp64 CPU oracle for the KLA hot path -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the CPU-baseline leg of the benchmark may import this
package.  It shares no code with the CUDA path and never imports it.

`forward` / `decode_step` run the token-by-token recurrence of Algorithm 1 (left panel) with
the coefficient of Eq. (3) in fp64 (C, `kla_oracle.c`).  `chunkwise.forward_chunkwise` restates
Algorithm 1 (right panel, Eqs. 7-9) in numpy fp64; the tests use it to pin the reading of the
chunk formulas against the recurrence.

`forward(..., diagonal_gates=True)` is the diagonal-gated extension of Appendix B.5 (a decay per row of the state).
`backward` / `backward_packed` are the reverse-mode derivative of the recurrence (the training pass of Section 5.1),
pinned by central differences of `forward`, closed forms and a library autograd run.

Pins (tests/test_oracle_pins.py): Kaczmarz projection (Theorem 1), residual contraction (Eq. 5),
proximal stationarity (Prop. 1), minimum-norm change, pure decay at eta=0, chunkwise == tokenwise
for several chunk sizes, brute force over the unrolled product form (Table 7) on T<=8, reduction
to causal linear attention on orthonormal keys, row-scaling invariance at eps=0, state hand-off.
No function here is "parity unpinned".
"""
import ctypes
import numpy as np

from .build import build as _build

_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(_build())
        dp = ctypes.POINTER(ctypes.c_double)
        lib.kla_oracle_forward.restype = ctypes.c_int
        lib.kla_oracle_forward.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_int64),
                                           ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                           dp, dp, dp, dp, dp, ctypes.c_double, dp, dp, dp]
        lib.kla_oracle_forward_dg.restype = ctypes.c_int
        lib.kla_oracle_forward_dg.argtypes = lib.kla_oracle_forward.argtypes
        lib.kla_oracle_backward.restype = ctypes.c_int
        lib.kla_oracle_backward.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_int64),
                                            ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                            dp, dp, dp, dp, dp, ctypes.c_double, dp, dp, dp] + [dp] * 6
        lib.kla_oracle_decode_step.restype = ctypes.c_int
        lib.kla_oracle_decode_step.argtypes = [ctypes.c_int] * 4 + [dp] * 5 + [ctypes.c_double, dp, dp]
        lib.kla_oracle_set_variant.restype = None
        lib.kla_oracle_set_variant.argtypes = [ctypes.c_int, ctypes.c_int]
        lib.kla_oracle_set_threads.restype = None
        lib.kla_oracle_set_threads.argtypes = [ctypes.c_int]
        _lib = lib
    return _lib


def _f64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _ptr(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_double)) if a is not None else None


class variant:
    """Context manager selecting the layer-edge variants for the calls inside it:
    `coeff_eta` -- beta_t = eta_t (the gated-delta-rule baseline coefficient, Section 2) instead of Eq. 3;
    `qnorm`     -- read-out divided by ||q_t||, as Algorithm 1 (left) prints it.  Default: neither."""

    def __init__(self, coeff_eta=False, qnorm=False):
        self.args = (int(bool(coeff_eta)), int(bool(qnorm)))

    def __enter__(self):
        _load().kla_oracle_set_variant(*self.args)
        return self

    def __exit__(self, *a):
        _load().kla_oracle_set_variant(0, 0)


def set_threads(n: int) -> None:
    _load().kla_oracle_set_threads(int(n))


def forward_packed(q, k, v, log_alpha, eta, eps, cu_seqlens, init_state=None, want_final=True, diagonal_gates=False):
    """Packed variable-length forward.

    q, k [n_tok, H, d_k]; v [n_tok, H, d_v]; log_alpha, eta [n_tok, H];
    cu_seqlens int[n_seq+1]; init_state [n_seq, H, d_k, d_v] or None (zeros).
    `diagonal_gates`: log_alpha is [n_tok, H, d_k], one decay per row of the state (Appendix B.5).
    Returns (out [n_tok, H, d_v], final_state [n_seq, H, d_k, d_v] or None, threads_used).
    """
    lib = _load()
    q, k, v, la, et = _f64(q), _f64(k), _f64(v), _f64(log_alpha), _f64(eta)
    n_tok, H, d_k = q.shape
    d_v = v.shape[-1]
    assert k.shape == (n_tok, H, d_k) and v.shape == (n_tok, H, d_v)
    assert la.shape == ((n_tok, H, d_k) if diagonal_gates else (n_tok, H)) and et.shape == (n_tok, H)
    cu = np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int64))
    n_seq = cu.shape[0] - 1
    assert cu[0] == 0 and cu[-1] == n_tok and np.all(np.diff(cu) >= 0)
    s0 = None
    if init_state is not None:
        s0 = _f64(init_state)
        assert s0.shape == (n_seq, H, d_k, d_v)
    out = np.zeros((n_tok, H, d_v), dtype=np.float64)
    fin = np.zeros((n_seq, H, d_k, d_v), dtype=np.float64) if want_final else None
    fn = lib.kla_oracle_forward_dg if diagonal_gates else lib.kla_oracle_forward
    thr = fn(n_seq, cu.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), H, d_k, d_v,
                                 _ptr(q), _ptr(k), _ptr(v), _ptr(la), _ptr(et), float(eps),
                                 _ptr(s0), _ptr(out), _ptr(fin))
    return out, fin, thr


def forward(q, k, v, log_alpha, eta, eps, init_state=None, want_final=True, diagonal_gates=False):
    """Fixed-length forward: q, k [B, T, H, d_k]; v [B, T, H, d_v]; log_alpha, eta [B, T, H] (log_alpha
    [B, T, H, d_k] with `diagonal_gates`); init_state [B, H, d_k, d_v] or None.
    Returns (out [B, T, H, d_v], final_state, threads)."""
    q = np.asarray(q)
    B, T, H, d_k = q.shape
    d_v = np.asarray(v).shape[-1]
    cu = np.arange(B + 1, dtype=np.int64) * T
    la = _f64(log_alpha).reshape((B * T, H, d_k) if diagonal_gates else (B * T, H))
    out, fin, thr = forward_packed(_f64(q).reshape(B * T, H, d_k), _f64(k).reshape(B * T, H, d_k),
                                   _f64(v).reshape(B * T, H, d_v), la,
                                   _f64(eta).reshape(B * T, H), eps, cu, init_state, want_final, diagonal_gates)
    return out.reshape(B, T, H, d_v), fin, thr


def backward_packed(q, k, v, log_alpha, eta, eps, cu_seqlens, dout, init_state=None, dfinal=None):
    """Gradients of a scalar loss through the packed forward, given dout = dL/dout [n_tok, H, d_v] and
    dfinal = dL/dfinal_state [n_seq, H, d_k, d_v] or None (zeros).  Layouts as `forward_packed`.
    Returns a dict with dq, dk, dv, dlog_alpha, deta, dinit (dL/dinit_state) and threads."""
    lib = _load()
    q, k, v, la, et, do = _f64(q), _f64(k), _f64(v), _f64(log_alpha), _f64(eta), _f64(dout)
    n_tok, H, d_k = q.shape
    d_v = v.shape[-1]
    assert k.shape == (n_tok, H, d_k) and v.shape == (n_tok, H, d_v) and do.shape == (n_tok, H, d_v)
    assert la.shape == (n_tok, H) and et.shape == (n_tok, H)
    cu = np.ascontiguousarray(np.asarray(cu_seqlens, dtype=np.int64))
    n_seq = cu.shape[0] - 1
    assert cu[0] == 0 and cu[-1] == n_tok and np.all(np.diff(cu) >= 0)
    s0 = _f64(init_state) if init_state is not None else None
    df = _f64(dfinal) if dfinal is not None else None
    for a in (s0, df):
        assert a is None or a.shape == (n_seq, H, d_k, d_v)
    g = dict(dq=np.zeros((n_tok, H, d_k)), dk=np.zeros((n_tok, H, d_k)), dv=np.zeros((n_tok, H, d_v)),
             dlog_alpha=np.zeros((n_tok, H)), deta=np.zeros((n_tok, H)), dinit=np.zeros((n_seq, H, d_k, d_v)))
    g["threads"] = lib.kla_oracle_backward(n_seq, cu.ctypes.data_as(ctypes.POINTER(ctypes.c_int64)), H, d_k, d_v,
                                           _ptr(q), _ptr(k), _ptr(v), _ptr(la), _ptr(et), float(eps),
                                           _ptr(s0), _ptr(do), _ptr(df), _ptr(g["dq"]), _ptr(g["dk"]), _ptr(g["dv"]),
                                           _ptr(g["dlog_alpha"]), _ptr(g["deta"]), _ptr(g["dinit"]))
    return g


def backward(q, k, v, log_alpha, eta, eps, dout, init_state=None, dfinal=None):
    """Fixed-length form of `backward_packed`: q, k [B, T, H, d_k]; v, dout [B, T, H, d_v]; log_alpha, eta [B, T, H]."""
    q = np.asarray(q)
    B, T, H, d_k = q.shape
    d_v = np.asarray(v).shape[-1]
    cu = np.arange(B + 1, dtype=np.int64) * T
    g = backward_packed(_f64(q).reshape(B * T, H, d_k), _f64(k).reshape(B * T, H, d_k), _f64(v).reshape(B * T, H, d_v),
                        _f64(log_alpha).reshape(B * T, H), _f64(eta).reshape(B * T, H), eps, cu,
                        _f64(dout).reshape(B * T, H, d_v), init_state, dfinal)
    for name, last in (("dq", d_k), ("dk", d_k), ("dv", d_v)):
        g[name] = g[name].reshape(B, T, H, last)
    for name in ("dlog_alpha", "deta"):
        g[name] = g[name].reshape(B, T, H)
    return g


def decode_step(q, k, v, log_alpha, eta, eps, state):
    """One recurrent step; `state` (float64 ndarray [B, H, d_k, d_v], C-contiguous) is updated
    IN PLACE.  q, k [B, H, d_k]; v [B, H, d_v]; log_alpha, eta [B, H].  Returns out [B, H, d_v]."""
    lib = _load()
    assert isinstance(state, np.ndarray) and state.dtype == np.float64 and state.flags.c_contiguous
    q, k, v, la, et = _f64(q), _f64(k), _f64(v), _f64(log_alpha), _f64(eta)
    B, H, d_k = q.shape
    d_v = v.shape[-1]
    assert state.shape == (B, H, d_k, d_v)
    out = np.zeros((B, H, d_v), dtype=np.float64)
    lib.kla_oracle_decode_step(B, H, d_k, d_v, _ptr(q), _ptr(k), _ptr(v), _ptr(la), _ptr(et),
                               float(eps), _ptr(state), _ptr(out))
    return out
