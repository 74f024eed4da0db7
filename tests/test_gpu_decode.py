"""GPU parity of the recurrent decode step against the fp64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from helpers import TOL_BF16, TOL_F32, assert_bf16_out_close, np64, rel_err
from paper_2605_08587_b200 import kla_chunk_fwd, kla_decode_step, kla_decode_steps, workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _oracle_decode(w, bsel=None, hsel=None):
    q, k, v, la, eta = (np64(a) for a in (w.q, w.k, w.v, w.log_alpha, w.eta))
    st = np64(w.state)
    if bsel is not None:
        q, k, v, la, eta, st = q[:, bsel], k[:, bsel], v[:, bsel], la[:, bsel], eta[:, bsel], st[bsel]
    if hsel is not None:
        q, k, v, la, eta, st = q[:, :, hsel], k[:, :, hsel], v[:, :, hsel], la[:, :, hsel], eta[:, :, hsel], st[:, hsel]
    st = np.ascontiguousarray(st)
    outs = [oracle.decode_step(q[s], k[s], v[s], la[s], eta[s], w.eps, st) for s in range(q.shape[0])]
    return np.stack(outs), st


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("io", [torch.bfloat16, torch.float32])
def test_decode_small_every_step(d, io):
    w = W.config4(B=3, H=2, d=d, steps=12, seed=3 + d)
    if io == torch.float32:
        w.q, w.k, w.v = w.q.float() * 1.0371, w.k.float() * 0.9713, w.v.float() * 1.0113   # not bf16-representable
    ro, rs = _oracle_decode(w)
    st = w.state.to(DEV).clone()
    tol = TOL_BF16 if io == torch.bfloat16 else TOL_F32
    for s in range(12):
        o = kla_decode_step(w.q[s].to(DEV), w.k[s].to(DEV), w.v[s].to(DEV), w.log_alpha[s].to(DEV), w.eta[s].to(DEV),
                            w.eps, st, out_dtype=torch.float32)
        assert rel_err(np64(o), ro[s]) <= tol
    assert rel_err(np64(st), rs) <= tol


def test_decode_bf16_out_rounding_only():
    w = W.config4(B=2, H=2, d=128, steps=4, seed=9)
    ro, _ = _oracle_decode(w)
    st = w.state.to(DEV).clone()
    out = kla_decode_steps(w.q.to(DEV), w.k.to(DEV), w.v.to(DEV), w.log_alpha.to(DEV), w.eta.to(DEV), w.eps, st)
    assert out.dtype == torch.bfloat16
    assert_bf16_out_close(out, ro)


def test_decode_steps_equals_step_loop_bitwise():
    w = W.config4(B=4, H=4, d=128, steps=8, seed=13)
    a = w.state.to(DEV).clone()
    b = w.state.to(DEV).clone()
    args = [t.to(DEV) for t in (w.q, w.k, w.v, w.log_alpha, w.eta)]
    o_all = kla_decode_steps(*args, w.eps, a, out_dtype=torch.float32)
    for s in range(8):
        o = kla_decode_step(*[t[s] for t in args], w.eps, b, out_dtype=torch.float32)
        assert torch.equal(o, o_all[s])
    assert torch.equal(a, b)


def test_decode_continues_chunk_forward():
    """State hand-off: chunk forward over a prefix, then decode steps, equals the oracle on the whole."""
    wl = W.config2(B=2, H=2, T=80, seed=17)
    args = [t.to(DEV) for t in (wl.q, wl.k, wl.v, wl.log_alpha, wl.eta)]
    _, fin = kla_chunk_fwd(*[t[:, :70].contiguous() for t in args], wl.eps)
    outs = []
    for t in range(70, 80):
        outs.append(kla_decode_step(*[a[:, t].contiguous() for a in args], wl.eps, fin, out_dtype=torch.float32))
    ro, rf, _ = oracle.forward(np64(wl.q), np64(wl.k), np64(wl.v), np64(wl.log_alpha), np64(wl.eta), wl.eps)
    assert rel_err(np64(torch.stack(outs, 1)), ro[:, 70:]) <= TOL_BF16
    assert rel_err(np64(fin), rf) <= TOL_BF16


def test_config4_full_size_sampled():
    """B = 64, H = 8, d = 128, 1024 consecutive steps in place; oracle on a sample of (b, h) pairs."""
    w = W.config4()
    st = w.state.to(DEV).clone()
    out = kla_decode_steps(w.q.to(DEV), w.k.to(DEV), w.v.to(DEV), w.log_alpha.to(DEV), w.eta.to(DEV), w.eps, st,
                           out_dtype=torch.float32)
    torch.cuda.synchronize()
    bsel, hsel = [0, 37, 63], [1, 6]
    ro, rs = _oracle_decode(w, bsel, hsel)
    got = np64(out[:, bsel][:, :, hsel])
    per_step = [rel_err(got[s], ro[s]) for s in range(got.shape[0])]
    assert max(per_step) <= TOL_BF16
    assert rel_err(np64(st[bsel][:, hsel]), rs) <= TOL_BF16
    assert torch.isfinite(out).all() and torch.isfinite(st).all()


@pytest.mark.parametrize("variant", [(True, False), (False, True), (True, True)])
def test_decode_variants(variant):
    """beta = eta (gated-delta-rule coefficient) and the read-out over ||q||, against the oracle's variants."""
    from paper_2605_08587_b200 import KLA_FLAG_COEFF_ETA, KLA_FLAG_QNORM
    coeff_eta, qnorm = variant
    w = W.config4(B=4, H=2, d=128, steps=6, seed=40 + 2 * coeff_eta + qnorm)
    if coeff_eta:
        k = w.k.float()
        w.k = (k / k.norm(dim=-1, keepdim=True)).to(w.k.dtype)
    flags = (KLA_FLAG_COEFF_ETA if coeff_eta else 0) | (KLA_FLAG_QNORM if qnorm else 0)
    with oracle.variant(coeff_eta=coeff_eta, qnorm=qnorm):
        ro, rs = _oracle_decode(w)
    st = w.state.to(DEV).clone()
    out = kla_decode_steps(w.q.to(DEV), w.k.to(DEV), w.v.to(DEV), w.log_alpha.to(DEV), w.eta.to(DEV), w.eps, st,
                           out_dtype=torch.float32, flags=flags)
    assert rel_err(np64(out), ro) <= TOL_BF16
    assert rel_err(np64(st), rs) <= TOL_BF16
