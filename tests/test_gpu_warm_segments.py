"""Decay-bounded segment starts of the segment-parallel scan (include/kla.h: KLA_FLAG_EXACT_SEGMENTS): when the decay is
strong enough every segment is run from the zero state a few chunks early instead of from chained transition maps.  The
result must match the fp64 oracle either way; the plan word in the workspace says which way was taken."""
import numpy as np
import pytest
import torch

from helpers import TOL_BF16, assert_bf16_out_close, gpu_chunk, np64, oracle_chunk, rel_err
from paper_2605_08587_b200 import (KLA_FLAG_COEFF_ETA, KLA_FLAG_EXACT_SEGMENTS, KLA_FLAG_NO_PAIR, KLA_FLAG_NO_SEGMENTS,
                                   KLA_FLAG_SEGMENTS, KLA_FLAG_WY_FORM, workloads as W)

pytestmark = pytest.mark.gpu


def _run(w, flags, **kw):
    word = []
    out, fin = gpu_chunk(w, flags=flags, plan_word=word, **kw)
    return out, fin, word[0]


def _check(w, out, fin):
    ro, rf = oracle_chunk(w)
    assert rel_err(np64(out), ro) <= TOL_BF16
    if fin is not None:
        assert rel_err(np64(fin), rf) <= TOL_BF16


@pytest.mark.parametrize("d,flags", [(128, 0), (128, KLA_FLAG_NO_PAIR), (64, 0)])
def test_decaying_input_takes_the_warm_up_path_and_matches_the_oracle(d, flags):
    # log_alpha averages -0.1 per token: exp(-40) is reached within ~7 chunks; segments of 4096 tokens allow 32
    w = W.config3(B=2, H=2, T=16384 + 70, d=d, seed=950)
    out, fin, word = _run(w, KLA_FLAG_SEGMENTS(4) | flags)
    assert word == 1
    _check(w, out, fin)


def test_warm_up_and_transition_maps_agree():
    w = W.config3(B=1, H=3, T=12288, seed=951)
    o_w, f_w, word_w = _run(w, KLA_FLAG_SEGMENTS(3))
    o_e, f_e, word_e = _run(w, KLA_FLAG_SEGMENTS(3) | KLA_FLAG_EXACT_SEGMENTS)
    o_p, f_p = gpu_chunk(w, flags=KLA_FLAG_NO_SEGMENTS)
    assert (word_w, word_e) == (1, 0)
    for o, f in ((o_w, f_w), (o_e, f_e)):
        assert rel_err(np64(o), np64(o_p)) <= 2e-4
        assert rel_err(np64(f), np64(f_p)) <= 2e-4


def test_weak_decay_falls_back_to_transition_maps():
    w = W.config3(B=1, H=2, T=8192, seed=952)
    w.log_alpha = (0.02 * w.log_alpha).contiguous()   # -0.002 per token: exp(-40) would need 20 000 tokens
    out, fin, word = _run(w, KLA_FLAG_SEGMENTS(4))
    assert word == 0
    _check(w, out, fin)


def test_one_head_with_weak_decay_is_enough_to_fall_back():
    w = W.config3(B=1, H=3, T=8192, seed=953)
    w.log_alpha[:, 3000:4096, 1] = 0.0   # one head without decay over the 1024 tokens (half a segment) a warm-up may use
    out, fin, word = _run(w, KLA_FLAG_SEGMENTS(4))
    assert word == 0
    _check(w, out, fin)


@pytest.mark.parametrize("bad", [2.5, -0.1, float("nan")])
def test_eta_outside_the_contraction_range_falls_back(bad):
    w = W.config3(B=1, H=2, T=8192, seed=954)
    w.eta[0, 5000, 1] = bad
    out, fin, word = _run(w, KLA_FLAG_SEGMENTS(4))
    assert word == 0
    if bad == bad:   # (a NaN gate poisons the oracle's outputs too: only the decision is checked)
        _check(w, out, fin)


def test_not_attempted_with_the_baseline_coefficient_or_the_wy_form():
    w = W.config3(B=1, H=2, T=8192, seed=955)
    kk = w.k.float()
    w.k = (kk / kk.norm(dim=-1, keepdim=True)).to(w.k.dtype)
    assert _run(w, KLA_FLAG_SEGMENTS(4) | KLA_FLAG_COEFF_ETA)[2] == 0
    assert _run(w, KLA_FLAG_SEGMENTS(4) | KLA_FLAG_WY_FORM)[2] == 0
    assert _run(w, KLA_FLAG_NO_SEGMENTS)[2] is None


def test_no_initial_state_bf16_out_and_a_ragged_last_segment():
    w = W.config2(B=1, H=2, T=3 * 4096 + 1000 + 13, seed=956)   # zero initial state; last segment shorter than the others
    word = []
    out, fin = gpu_chunk(w, out_dtype=torch.bfloat16, flags=KLA_FLAG_SEGMENTS(4), plan_word=word)
    assert word[0] == 1
    ro, rf = oracle_chunk(w)
    assert_bf16_out_close(out, ro)
    assert rel_err(np64(fin), rf) <= TOL_BF16


def test_strong_decay_needs_a_single_warm_up_chunk():
    w = W.config3(B=1, H=2, T=8192, seed=957)
    w.log_alpha = (20 * w.log_alpha).contiguous()
    out, fin, word = _run(w, KLA_FLAG_SEGMENTS(8))
    assert word == 1
    _check(w, out, fin)


def test_two_runs_agree_bit_for_bit():
    w = W.config3(B=1, H=2, T=16384, seed=958)
    a = _run(w, KLA_FLAG_SEGMENTS(4))
    b = _run(w, KLA_FLAG_SEGMENTS(4))
    assert a[2] == b[2] == 1
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


def test_long_context_workload_by_default_every_head():
    w = W.config3()   # one 65 536-token sequence, 8 heads: the library cuts it into segments by itself
    out, fin, word = _run(w, 0)
    assert word == 1
    _check(w, out, fin)


# ---- packed input: long sequences cut into pieces that start from warm-up runs ------------------------------------------------
def _skewed(lens, H=2, d=64, seed=960, init=True):
    w = W.config5(H=H, d=d, lengths=lens, seed=seed)
    w.log_alpha = (w.log_alpha * 12).contiguous()   # config 5 draws -softplus / 8 ... scaled so that exp(-40) needs ~4 chunks
    if init:
        w.init_state = (0.02 * torch.randn(len(lens), H, d, d, generator=torch.Generator().manual_seed(seed + 1))).float()
    return w


def _check_packed(w, out, fin):
    ro, rf = oracle_chunk(w)[:2]
    o = np64(out)[0]
    assert rel_err(o, ro) <= TOL_BF16
    assert rel_err(np64(fin), rf) <= TOL_BF16
    cu = w.cu_seqlens.numpy()
    for n in range(len(cu) - 1):   # no sequence hides behind the others
        if cu[n + 1] > cu[n]:
            assert rel_err(o[cu[n]:cu[n + 1]], ro[cu[n]:cu[n + 1]]) <= 5 * TOL_BF16


@pytest.mark.parametrize("d", [64, 128])
def test_one_long_sequence_among_short_ones_is_cut_by_default(d):
    lens = [40, 20000 + 37, 0, 64, 130, 1]
    w = _skewed(lens, d=d, seed=961)
    out, fin, word = _run(w, 0)
    assert word == 1            # the library decided to cut, and the decay allowed warm-up starts
    _check_packed(w, out, fin)
    assert torch.equal(fin[2].cpu(), w.init_state[2])   # the empty sequence keeps its state


def test_forced_pieces_match_the_plain_launch_and_the_oracle():
    lens = [3000, 700, 5000 + 11, 64, 0, 2048]
    w = _skewed(lens, d=128, seed=962)
    o_c, f_c, word = _run(w, KLA_FLAG_SEGMENTS(4))        # the longest sequence in four pieces; pieces of that length everywhere
    o_p, f_p, none = _run(w, KLA_FLAG_NO_SEGMENTS)
    assert word == 1 and none is None
    _check_packed(w, o_c, f_c)
    assert rel_err(np64(o_c), np64(o_p)) <= 2e-4 and rel_err(np64(f_c), np64(f_p)) <= 2e-4


def test_packed_pieces_fall_back_to_the_plain_launch_on_weak_decay():
    lens = [3000, 700, 5000 + 11, 64]
    w = _skewed(lens, d=64, seed=963)
    w.log_alpha = (w.log_alpha * 1e-3).contiguous()
    out, fin, word = _run(w, KLA_FLAG_SEGMENTS(4))
    assert word == 0
    _check_packed(w, out, fin)
    plain = gpu_chunk(w, flags=KLA_FLAG_NO_SEGMENTS)
    assert torch.equal(out, plain[0]) and torch.equal(fin, plain[1])   # the fallback IS the plain launch


def test_packed_pieces_without_initial_state_bf16_out():
    lens = [9000, 100, 4100]
    w = _skewed(lens, d=128, seed=964, init=False)
    word = []
    out, fin = gpu_chunk(w, out_dtype=torch.bfloat16, flags=KLA_FLAG_SEGMENTS(3), plan_word=word)
    assert word[0] == 1
    ro, rf = oracle_chunk(w)[:2]
    assert_bf16_out_close(out[0], ro)
    assert rel_err(np64(fin), rf) <= TOL_BF16


def test_the_packed_benchmark_workload_is_not_cut():
    # lengths uniform in [1, 8192]: the launch is bound by total work, no sequence stands out
    from paper_2605_08587_b200 import binding
    import ctypes
    w = W.config5()
    hs = w.cu_seqlens.contiguous()
    desc = binding.KlaDesc(B=1, T=w.q.shape[1], H=16, d_k=64, d_v=64, n_seq=32, cu_seqlens=1 << 20, host_seqlens=hs.data_ptr(),
                           io_dtype=binding.KLA_BF16, out_dtype=binding.KLA_BF16)
    lib = binding.load()
    assert lib.kla_chunk_fwd_plan_word_offset(ctypes.byref(desc), 64) == ctypes.c_size_t(-1).value
    assert lib.kla_chunk_fwd_workspace_bytes(ctypes.byref(desc), 64) == 256   # the longest-first order array alone
