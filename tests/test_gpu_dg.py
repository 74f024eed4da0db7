"""GPU parity of the diagonal-gated extension (kla_dg_fwd, kla_dg_decode_step; Appendix B.5) against the fp64 oracle:
<= 2e-3 (max|err| / rms) for bf16 inputs, <= 1e-5 for fp32 inputs."""
import numpy as np
import pytest
import torch

import oracle
from helpers import TOL_BF16, TOL_F32, assert_bf16_out_close, np64, rel_err
from paper_2605_08587_b200 import (KLA_FLAG_COEFF_ETA, KLA_FLAG_FORCE_SIMT, KLA_FLAG_QNORM, kla_chunk_fwd, kla_dg_decode_step,
                                   kla_dg_fwd, workloads as W)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _gpu(w, out_dtype=torch.float32, flags=0, cu=None):
    out, fin = kla_dg_fwd(w.q.to(DEV), w.k.to(DEV), w.v.to(DEV), w.log_alpha.to(DEV), w.eta.to(DEV), w.eps,
                          init_state=None if w.init_state is None else w.init_state.to(DEV), out_dtype=out_dtype, flags=flags,
                          cu_seqlens=None if cu is None else cu.to(DEV), host_seqlens=cu)
    torch.cuda.synchronize()
    return out, fin


def _ref(w, **kw):
    return oracle.forward(np64(w.q), np64(w.k), np64(w.v), np64(w.log_alpha), np64(w.eta), w.eps,
                          None if w.init_state is None else np64(w.init_state), diagonal_gates=True, **kw)[:2]


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("T", [1, 2, 63, 200, 1000])
def test_bf16_inputs_match_the_oracle(T, d):
    w = W.config_dg(B=2, H=3, T=T, d=d, seed=800 + T)
    out, fin = _gpu(w)
    ro, rf = _ref(w)
    assert rel_err(np64(out), ro) <= TOL_BF16
    assert rel_err(np64(fin), rf) <= TOL_BF16


@pytest.mark.parametrize("d", [64, 128])
def test_fp32_inputs_match_the_oracle(d):
    w = W.config_dg(B=2, H=2, T=300, d=d, seed=811, dtype=torch.float32)
    out, fin = _gpu(w)
    ro, rf = _ref(w)
    assert rel_err(np64(out), ro) <= TOL_F32
    assert rel_err(np64(fin), rf) <= TOL_F32


def test_bf16_out_and_no_initial_state():
    w = W.config_dg(B=1, H=2, T=257, d=128, seed=812, init_state=False)
    out, fin = _gpu(w, out_dtype=torch.bfloat16)
    ro, rf = _ref(w)
    assert_bf16_out_close(out, ro)
    assert rel_err(np64(fin), rf) <= TOL_BF16


def test_packed_input_with_empty_sequences():
    lens = [70, 0, 1, 129, 0, 300]
    w = W.config_dg(B=1, H=2, T=sum(lens), d=64, seed=813, init_state=False)
    cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32)
    w.init_state = (0.05 * torch.randn(len(lens), 2, 64, 64, generator=torch.Generator().manual_seed(814))).float()
    out, fin = _gpu(w, cu=cu)
    ro, rf, _ = oracle.forward_packed(np64(w.q)[0], np64(w.k)[0], np64(w.v)[0], np64(w.log_alpha)[0], np64(w.eta)[0], w.eps,
                                      cu.numpy(), np64(w.init_state), diagonal_gates=True)
    assert rel_err(np64(out)[0], ro) <= TOL_BF16
    assert rel_err(np64(fin), rf) <= TOL_BF16
    for n in (1, 4):
        assert torch.equal(fin[n].cpu(), w.init_state[n])


@pytest.mark.parametrize("variant", [(True, False), (False, True)])
def test_layer_edge_variants(variant):
    coeff_eta, qnorm = variant
    w = W.config_dg(B=2, H=2, T=150, d=128, seed=815)
    if coeff_eta:
        kk = w.k.float()
        w.k = (kk / kk.norm(dim=-1, keepdim=True)).to(w.k.dtype)
    out, fin = _gpu(w, flags=(KLA_FLAG_COEFF_ETA if coeff_eta else 0) | (KLA_FLAG_QNORM if qnorm else 0))
    with oracle.variant(coeff_eta=coeff_eta, qnorm=qnorm):
        ro, rf = _ref(w)
    assert rel_err(np64(out), ro) <= TOL_BF16
    assert rel_err(np64(fin), rf) <= TOL_BF16


def test_a_constant_gate_vector_is_the_scalar_gated_path():
    """With the same decay in every key dimension the extension must agree with the scalar-gated chunk forward."""
    w = W.config3(B=2, H=2, T=333, d=64, seed=816)
    a = [t.to(DEV) for t in (w.q, w.k, w.v)]
    la_vec = w.log_alpha[..., None].expand(-1, -1, -1, 64).contiguous()
    o_dg, f_dg = kla_dg_fwd(*a, la_vec.to(DEV), w.eta.to(DEV), w.eps, init_state=w.init_state.to(DEV), out_dtype=torch.float32)
    o_sc, f_sc = kla_chunk_fwd(*a, w.log_alpha.to(DEV), w.eta.to(DEV), w.eps, init_state=w.init_state.to(DEV), out_dtype=torch.float32,
                               flags=KLA_FLAG_FORCE_SIMT)
    torch.cuda.synchronize()
    assert rel_err(np64(o_dg), np64(o_sc)) <= 1e-4 and rel_err(np64(f_dg), np64(f_sc)) <= 1e-4


@pytest.mark.parametrize("d", [64, 128])
def test_decode_steps_match_the_oracle_and_continue_a_forward(d):
    w = W.config_dg(B=3, H=2, T=40, d=d, seed=817)
    ro, rf = _ref(w)
    # the first 30 tokens through the forward, the last 10 one step at a time from its final state
    a = [t.to(DEV) for t in (w.q, w.k, w.v, w.log_alpha, w.eta)]
    _, st = kla_dg_fwd(*[x[:, :30].contiguous() for x in a], w.eps, init_state=w.init_state.to(DEV), out_dtype=torch.float32)
    for t in range(30, 40):
        o = kla_dg_decode_step(*[x[:, t].contiguous() for x in a], w.eps, st, out_dtype=torch.float32)
        torch.cuda.synchronize()
        assert rel_err(np64(o), ro[:, t]) <= TOL_BF16
    assert rel_err(np64(st), rf) <= TOL_BF16


def test_full_size_layer_shape():
    """The shape of the headline configuration (B=8, H=8, T=4096, d=128) with vector gates, every sequence and head."""
    w = W.config_dg()
    out, fin = _gpu(w)
    ro, rf = _ref(w)
    assert rel_err(np64(out), ro) <= TOL_BF16
    assert rel_err(np64(fin), rf) <= TOL_BF16
