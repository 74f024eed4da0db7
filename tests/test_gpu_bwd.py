"""GPU parity of the backward pass (kla_bwd; the training pass of Section 5.1) against the fp64 oracle's reverse-mode
derivative.  Every gradient tensor is held to the forward's bounds in the same metric: max|err| / rms(ref) <= 2e-3 for
bf16 inputs for bf16 inputs; fp32 inputs get a bound of their own (below).  The arithmetic is fp32 throughout, so the bf16 cases
sit far inside theirs."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from helpers import TOL_BF16, np64, rel_err
from paper_2605_08587_b200 import KLA_FLAG_COEFF_ETA, KLA_FLAG_QNORM, KlaError, binding, kla_bwd, workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
# fp32 inputs: the gradients pass through T dependent fp32 updates of G and S; 64 units of fp32 rounding relative to the
# rms of the tensor covers every case below with a factor of three to spare.
TOL_F32_BWD = 64 * 2.0 ** -24
PAIRS = [("dq", "dq"), ("dk", "dk"), ("dv", "dv"), ("dlog_alpha", "dlog_alpha"), ("deta", "deta"), ("dinit_state", "dinit")]


def _gpu(w, flags=0, final=True, cu=None, want_dinit=True):
    do, df = W.upstream_grads(w, final=final)
    g = kla_bwd(w.q.to(DEV), w.k.to(DEV), w.v.to(DEV), w.log_alpha.to(DEV), w.eta.to(DEV), w.eps, do.to(DEV),
                init_state=None if w.init_state is None else w.init_state.to(DEV),
                d_final_state=None if df is None else df.to(DEV), flags=flags,
                cu_seqlens=None if cu is None else cu.to(DEV), host_seqlens=cu, want_dinit_state=want_dinit)
    torch.cuda.synchronize()
    return g, do, df


def _ref(w, do, df):
    s0 = None if w.init_state is None else np64(w.init_state)
    if w.cu_seqlens is None:
        return oracle.backward(np64(w.q), np64(w.k), np64(w.v), np64(w.log_alpha), np64(w.eta), w.eps, np64(do), s0,
                               None if df is None else np64(df))
    r = oracle.backward_packed(np64(w.q)[0], np64(w.k)[0], np64(w.v)[0], np64(w.log_alpha)[0], np64(w.eta)[0], w.eps,
                               w.cu_seqlens.numpy(), np64(do)[0], s0, None if df is None else np64(df))
    for name in ("dq", "dk", "dv", "dlog_alpha", "deta"):
        r[name] = r[name][None]
    return r


def _assert_close(g, r, tol):
    for name, rname in PAIRS:
        if g[name] is None:
            continue
        err = rel_err(np64(g[name]), r[rname])
        assert err <= tol, "%s: %.3g > %.3g" % (name, err, tol)


def _with_state(w, seed):
    B, _, H, d = w.q.shape
    w.init_state = (0.02 * torch.randn(w.n_seq, H, d, d, generator=torch.Generator().manual_seed(seed))).float()
    return w


@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("T", [1, 2, 15, 16, 17, 33, 200, 1000])
def test_bf16_inputs_match_the_oracle(T, d):
    # lengths around the 16-token spacing of the stored states, and several hundred blocks of it
    w = _with_state(W.config2(B=2, H=3, T=T, d=d, seed=900 + T), T)
    g, do, df = _gpu(w)
    _assert_close(g, _ref(w, do, df), TOL_BF16)


@pytest.mark.parametrize("d", [64, 128])
def test_fp32_inputs_match_the_oracle(d):
    w = W.config1(T=300, d=d, seed=911)      # unnormalised N(0,1) keys, fp32
    g, do, df = _gpu(w)
    _assert_close(g, _ref(w, do, df), TOL_F32_BWD)


def test_no_initial_state_no_final_gradient_no_dinit():
    w = W.config2(B=1, H=2, T=130, d=128, seed=912)
    g, do, df = _gpu(w, final=False, want_dinit=False)
    assert g["dinit_state"] is None and df is None
    _assert_close(g, _ref(w, do, df), TOL_BF16)


def test_packed_input_with_empty_sequences():
    lens = [70, 0, 1, 129, 0, 16, 300]
    w = W.config5(H=2, lengths=lens, seed=913)
    w = _with_state(w, 914)
    g, do, df = _gpu(w, cu=w.cu_seqlens)
    r = _ref(w, do, df)
    _assert_close(g, r, TOL_BF16)
    for n in (1, 4):   # an empty sequence hands the gradient of its final state straight to its initial state
        assert torch.equal(g["dinit_state"][n].cpu(), df[n])


@pytest.mark.parametrize("variant", [(True, False), (False, True), (True, True)])
@pytest.mark.parametrize("d", [64, 128])
def test_layer_edge_variants(variant, d):
    coeff_eta, qnorm = variant
    w = _with_state(W.config2(B=2, H=2, T=150, d=d, seed=915), 916)
    if coeff_eta:   # beta = eta is a contraction only on unit keys
        kk = w.k.float()
        w.k = (kk / kk.norm(dim=-1, keepdim=True)).to(w.k.dtype)
    g, do, df = _gpu(w, flags=(KLA_FLAG_COEFF_ETA if coeff_eta else 0) | (KLA_FLAG_QNORM if qnorm else 0))
    with oracle.variant(coeff_eta=coeff_eta, qnorm=qnorm):
        r = _ref(w, do, df)
    _assert_close(g, r, TOL_BF16)


def test_two_runs_agree_bit_for_bit():
    # d = 128: the two blocks of a head add their halves of dq, dk, dlog_alpha, deta with one atomic each
    w = _with_state(W.config2(B=3, H=4, T=500, d=128, seed=917), 918)
    a, _, _ = _gpu(w)
    b, _, _ = _gpu(w)
    for name, _r in PAIRS:
        assert torch.equal(a[name], b[name]), name


def test_strong_decay_and_near_zero_keys():
    lens = [257, 64]
    w = W.config5(H=2, lengths=lens, seed=919)     # heavy-tailed key norms including near-zero keys
    w.log_alpha = (w.log_alpha * 40).contiguous()  # decay far beyond the fp32 range over a few hundred tokens
    g, do, df = _gpu(w, cu=w.cu_seqlens)
    _assert_close(g, _ref(w, do, df), TOL_BF16)


def test_workspace_is_checked_and_a_caller_supplied_one_is_used():
    w = W.config2(B=1, H=2, T=64, d=64, seed=920)
    do, df = W.upstream_grads(w)
    args = [x.to(DEV) for x in (w.q, w.k, w.v, w.log_alpha, w.eta)]
    desc = binding.KlaDesc(B=1, T=64, H=2, d_k=64, d_v=64, n_seq=1, io_dtype=binding.KLA_BF16, out_dtype=binding.KLA_F32)
    need = int(binding.load().kla_bwd_workspace_bytes(ctypes.byref(desc)))
    # kept states (one per 16 tokens and one more per sequence) per head, scratch of the two resident blocks, unit counter
    assert need == (64 // 16 + 1) * 2 * 64 * 64 * 4 + 2 * 16 * 64 * 64 * 4 + 256
    with pytest.raises(KlaError) as e:
        kla_bwd(*args, w.eps, do.to(DEV), workspace=torch.empty(need - 16, device=DEV, dtype=torch.uint8))
    assert e.value.code == -7   # KLA_ERR_WORKSPACE
    ws = torch.empty(need, device=DEV, dtype=torch.uint8)
    g = kla_bwd(*args, w.eps, do.to(DEV), d_final_state=df.to(DEV), workspace=ws)
    torch.cuda.synchronize()
    _assert_close(g, _ref(w, do, df), TOL_BF16)


def test_config2_full_size_every_sequence_and_head():
    w = W.config2()
    g, do, df = _gpu(w)
    _assert_close(g, _ref(w, do, df), TOL_BF16)


def test_packed_benchmark_workload_full_size_every_sequence_and_head():
    # 32 sequences of 1..8192 tokens, 16 heads, d = 64, heavy-tailed key norms with near-zero and zero keys
    w = W.config5()
    g, do, df = _gpu(w, cu=w.cu_seqlens)
    _assert_close(g, _ref(w, do, df), TOL_BF16)


def test_long_context_workload_full_size_every_head():
    # one sequence of 65 536 tokens: 4096 kept states per head, gradients carried back through all of them
    w = W.config3()
    g, do, df = _gpu(w)
    _assert_close(g, _ref(w, do, df), TOL_BF16)
