"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on identical
seeded inputs.  Tolerances: max|err|/rms(ref) <= 2e-3 for bf16 inputs (fp32 `out` and the fp32
final state), <= 1e-5 for fp32 inputs; a bf16 `out` is allowed its own rounding on top."""
import numpy as np
import pytest
import torch

from helpers import (TOL_BF16, TOL_F32, assert_bf16_out_close, gpu_chunk, np64, oracle_chunk, rel_err)
from paper_2605_08587_b200 import KLA_FLAG_FORCE_SIMT, workloads as W

pytestmark = pytest.mark.gpu


def _check_fixed(w, tol, flags=0, chunk=None, out_dtype=torch.float32):
    out, fin = gpu_chunk(w, out_dtype=out_dtype, flags=flags, chunk=chunk)
    ro, rf = oracle_chunk(w)
    if out_dtype == torch.bfloat16:
        assert_bf16_out_close(out, ro, tol)
    else:
        assert rel_err(np64(out), ro) <= tol
    assert rel_err(np64(fin), rf) <= tol
    return out, fin


# ---- config 1: fp32, exact shape ------------------------------------------------------------------
@pytest.mark.parametrize("chunk", [16, 32, 64])
def test_config1_fp32_exact_shape(chunk):
    _check_fixed(W.config1(), TOL_F32, chunk=chunk)


def test_config1_fp32_d128_ragged():
    _check_fixed(W.config1(B=2, H=3, T=200, d=128, seed=11), TOL_F32)


# ---- configs 2/3 at sizes the oracle finishes in seconds (several chunks + ragged tail) -----------
@pytest.mark.parametrize("flags", [0, KLA_FLAG_FORCE_SIMT])
def test_config2_small_bf16(flags):
    _check_fixed(W.config2(B=2, H=3, T=1000), TOL_BF16, flags=flags)


@pytest.mark.parametrize("flags", [0, KLA_FLAG_FORCE_SIMT])
def test_config2_small_bf16_out_bf16(flags):
    _check_fixed(W.config2(B=1, H=2, T=333, seed=21), TOL_BF16, flags=flags, out_dtype=torch.bfloat16)


@pytest.mark.parametrize("flags", [0, KLA_FLAG_FORCE_SIMT])
def test_config3_small_with_init_state(flags):
    _check_fixed(W.config3(B=1, H=4, T=2048 + 17), TOL_BF16, flags=flags)


@pytest.mark.parametrize("flags", [0, KLA_FLAG_FORCE_SIMT])
@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("T", [1, 5, 63, 64, 65, 128, 129])
def test_short_and_boundary_lengths(T, d, flags):
    w = W.config3(B=2, H=2, T=T, d=d, seed=100 + T)
    _check_fixed(w, TOL_BF16, flags=flags)


# ---- config 5: packed variable-length ----------------------------------------------------------------
@pytest.mark.parametrize("flags", [0, KLA_FLAG_FORCE_SIMT])
def test_config5_small_varlen(flags):
    w = W.config5(H=4, lengths=[1, 63, 64, 65, 300, 1, 129, 2, 517])
    out, fin = gpu_chunk(w, flags=flags)
    ro, rf, _ = oracle_chunk(w)
    assert rel_err(np64(out)[0], ro) <= TOL_BF16
    assert rel_err(np64(fin), rf) <= TOL_BF16
    cu = w.cu_seqlens.numpy()
    worst = max(rel_err(np64(out)[0, cu[n]:cu[n + 1]], ro[cu[n]:cu[n + 1]]) for n in range(len(cu) - 1))
    assert worst <= 5 * TOL_BF16   # per-sequence figure, reported for the heavy-tailed keys


@pytest.mark.parametrize("flags", [0, KLA_FLAG_FORCE_SIMT])
def test_varlen_zero_length_sequences_keep_their_initial_state(flags):
    w = W.config5(H=2, lengths=[0, 70, 0, 3, 0], seed=5)
    gen = torch.Generator().manual_seed(77)
    w.init_state = (0.05 * torch.randn(5, 2, 64, 64, generator=gen)).float()
    out, fin = gpu_chunk(w, flags=flags)
    ro, rf, _ = oracle_chunk(w)
    assert rel_err(np64(out)[0], ro) <= TOL_BF16
    assert rel_err(np64(fin), rf) <= TOL_BF16
    for n in (0, 2, 4):
        assert torch.equal(fin[n].cpu(), w.init_state[n])


def test_varlen_equals_fixed_length_bitwise():
    """Packing B equal-length sequences must give exactly the fixed-length result."""
    w = W.config2(B=3, H=2, T=130, seed=31)
    out_f, fin_f = gpu_chunk(w)
    wp = W.ChunkWorkload("packed", w.q.reshape(1, -1, 2, 128), w.k.reshape(1, -1, 2, 128), w.v.reshape(1, -1, 2, 128),
                         w.log_alpha.reshape(1, -1, 2), w.eta.reshape(1, -1, 2), w.eps, w.chunk,
                         cu_seqlens=torch.tensor([0, 130, 260, 390], dtype=torch.int32))
    out_p, fin_p = gpu_chunk(wp)
    assert torch.equal(out_p.reshape(3, 130, 2, 128), out_f)
    assert torch.equal(fin_p, fin_f)


# ---- properties that hold at any size -------------------------------------------------------------------
@pytest.mark.parametrize("flags", [0, KLA_FLAG_FORCE_SIMT])
def test_state_handoff_on_gpu(flags):
    w = W.config2(B=2, H=2, T=512, seed=41)
    out, fin = gpu_chunk(w, flags=flags)
    T1 = 192
    def part(a, b, s0):
        return W.ChunkWorkload("p", w.q[:, a:b].contiguous(), w.k[:, a:b].contiguous(), w.v[:, a:b].contiguous(),
                               w.log_alpha[:, a:b].contiguous(), w.eta[:, a:b].contiguous(), w.eps, w.chunk, init_state=s0)
    o1, f1 = gpu_chunk(part(0, T1, None), flags=flags)
    o2, f2 = gpu_chunk(part(T1, 512, f1.cpu()), flags=flags)
    ref = np64(out)
    assert rel_err(np64(torch.cat([o1, o2], 1)), ref) <= 1e-5   # T1 is a chunk multiple: same arithmetic
    assert rel_err(np64(f2), np64(fin)) <= 1e-5


@pytest.mark.parametrize("flags", [0, KLA_FLAG_FORCE_SIMT])
def test_eta_zero_is_pure_decay(flags):
    w = W.config3(B=1, H=2, T=150, seed=51)
    w.eta = torch.zeros_like(w.eta)
    out, fin = gpu_chunk(w, flags=flags)
    gamma = torch.exp(torch.cumsum(w.log_alpha.double(), 1))
    expect = gamma[..., None] * torch.einsum("bhkv,bthk->bthv", w.init_state.double(), w.q.double())
    tol = 1e-5 if flags else 3e-4   # fp32 CUDA-core path / split-bf16 tensor-core path
    assert rel_err(np64(out), expect.numpy()) <= tol
    assert rel_err(np64(fin), (gamma[:, -1][..., None, None] * w.init_state.double()).numpy()) <= tol


@pytest.mark.parametrize("flags", [0, KLA_FLAG_FORCE_SIMT])
def test_kaczmarz_projection_on_gpu(flags):
    """eta = 1, eps = 0: reading the final state with the last key returns the last value."""
    w = W.config2(B=2, H=2, T=100, seed=61)
    w.eta = torch.ones_like(w.eta)
    w.eps = 0.0
    out, fin = gpu_chunk(w, flags=flags)
    pred = torch.einsum("bhkv,bhk->bhv", fin.double().cpu(), w.k[:, -1].double())
    assert rel_err(pred.numpy(), w.v[:, -1].double().numpy()) <= TOL_BF16


def test_run_to_run_determinism():
    w = W.config2(B=2, H=2, T=700, seed=71)
    a = gpu_chunk(w)
    b = gpu_chunk(w)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


def test_final_state_is_optional():
    w = W.config2(B=1, H=2, T=100, seed=81)
    out, fin = gpu_chunk(w, want_final_state=False)
    assert fin is None
    ro, _ = oracle_chunk(w)
    assert rel_err(np64(out), ro) <= TOL_BF16


# ---- guard bands: nothing outside `out`, `final_state` and the workspace is written ---------------------------------
GUARD = 4096   # bytes of sentinel before and after each buffer


def _guarded(nbytes, dev="cuda:0"):
    """A uint8 buffer of nbytes (rounded up to 256) with GUARD sentinel bytes on either side; returns (whole, view)."""
    n = (nbytes + 255) // 256 * 256
    whole = torch.full((GUARD + n + GUARD,), 0xA5, dtype=torch.uint8, device=dev)
    return whole, whole[GUARD:GUARD + n]


def _bands_intact(whole):
    return bool((whole[:GUARD] == 0xA5).all()) and bool((whole[-GUARD:] == 0xA5).all())


@pytest.mark.parametrize("case", ["packed_d64", "packed_d128", "segments_d128", "wy_d128", "simt_d64"])
def test_guard_bands_around_outputs_and_workspace_stay_intact(case):
    """`out`, `final_state` and the workspace sit between sentinel bands; sequences end in the middle of a chunk, so the
    masked stores of the tail chunks are exactly where an off-by-one would write a neighbour's rows.  Inside `out`, rows
    of the next sequence must not be touched by the previous one either: the result has to match the oracle everywhere."""
    import ctypes
    from paper_2605_08587_b200 import binding, KLA_FLAG_SEGMENTS, KLA_FLAG_FORCE_SIMT
    dev = "cuda:0"
    flags = 0
    if case == "packed_d64":
        w = W.config5(H=3, d=64, seed=601, lengths=[70, 1, 129, 63, 200, 65])
    elif case == "packed_d128":
        w = W.config5(H=2, d=128, seed=602, lengths=[130, 5, 64, 191])
    elif case == "segments_d128":
        w = W.config3(B=2, H=2, T=1024 + 37, seed=603)
        flags = KLA_FLAG_SEGMENTS(3)
    elif case == "wy_d128":
        w = W.config5(H=2, d=128, seed=604, lengths=[97, 250, 1, 66])
        flags = binding.KLA_FLAG_WY_FORM
    else:
        w = W.config5(H=2, d=64, seed=605, lengths=[33, 90, 64, 1])
        flags = KLA_FLAG_FORCE_SIMT
    B, T, H, d = w.q.shape
    n_seq = w.n_seq
    out_whole, out_raw = _guarded(B * T * H * d * 4)
    fin_whole, fin_raw = _guarded(n_seq * H * d * d * 4)
    out = out_raw[:B * T * H * d * 4].view(torch.float32).view(B, T, H, d)
    fin = fin_raw[:n_seq * H * d * d * 4].view(torch.float32).view(n_seq, H, d, d)
    lib = binding.load()
    cu = None if w.cu_seqlens is None else w.cu_seqlens.to(dev)
    hs = w.cu_seqlens
    a = [t.to(dev) for t in (w.q, w.k, w.v, w.log_alpha, w.eta)]
    s0 = None if w.init_state is None else w.init_state.to(dev)
    desc = binding.KlaDesc(B=B, T=T, H=H, d_k=d, d_v=d, n_seq=n_seq, cu_seqlens=None if cu is None else cu.data_ptr(),
                           host_seqlens=None if hs is None else hs.data_ptr(), io_dtype=binding.KLA_BF16, out_dtype=binding.KLA_F32,
                           flags=flags, workspace=None, workspace_bytes=0, status_word=None,
                           stream=torch.cuda.current_stream().cuda_stream)
    need = lib.kla_chunk_fwd_workspace_bytes(ctypes.byref(desc), 64)
    ws_whole = None
    if need:
        ws_whole, ws = _guarded(need)
        desc.workspace, desc.workspace_bytes = ws.data_ptr(), need
    code = lib.kla_chunk_fwd(ctypes.byref(desc), a[0].data_ptr(), a[1].data_ptr(), a[2].data_ptr(), a[3].data_ptr(), a[4].data_ptr(),
                             w.eps, 64, None if s0 is None else s0.data_ptr(), out.data_ptr(), fin.data_ptr())
    torch.cuda.synchronize()
    assert code == 0
    assert _bands_intact(out_whole) and _bands_intact(fin_whole)
    if ws_whole is not None:
        assert _bands_intact(ws_whole)
    r = oracle_chunk(w)
    o = np64(out)[0] if w.cu_seqlens is not None else np64(out)
    assert rel_err(o, r[0]) <= TOL_BF16
    assert rel_err(np64(fin), r[1]) <= TOL_BF16


# ---- full-size configurations, in the launch configuration the benchmark times ---------------------------
# The oracle runs the whole workload (every sequence and head): the bound is a maximum over every output element.
_FULL = {}


def _full(name):
    """Workload and oracle result of a full-size configuration, computed once per test session."""
    if name not in _FULL:
        w = {"cfg2": W.config2, "cfg3": W.config3, "cfg5": W.config5}[name]()
        _FULL[name] = (w, oracle_chunk(w))
    return _FULL[name]


def _check_full(name, out_dtype, flags=0):
    w, r = _full(name)
    out, fin = gpu_chunk(w, out_dtype=out_dtype, flags=flags)
    assert torch.isfinite(out).all() and torch.isfinite(fin).all()
    o = out[0] if w.cu_seqlens is not None else out
    if out_dtype == torch.bfloat16:
        assert_bf16_out_close(o, r[0])
    else:
        assert rel_err(np64(o), r[0]) <= TOL_BF16
    assert rel_err(np64(fin), r[1]) <= TOL_BF16
    return out, fin, r


@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])   # bf16 out is the instantiation the benchmark times
def test_config2_full_size_every_sequence_and_head(out_dtype):
    _check_full("cfg2", out_dtype)


def test_config2_full_size_wy_form():
    from paper_2605_08587_b200 import binding
    _check_full("cfg2", torch.float32, flags=binding.KLA_FLAG_WY_FORM)


@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_config3_full_size_every_head(out_dtype):
    _check_full("cfg3", out_dtype)


def test_config3_full_size_from_chained_transition_maps():
    from paper_2605_08587_b200 import binding
    _check_full("cfg3", torch.float32, flags=binding.KLA_FLAG_EXACT_SEGMENTS)


@pytest.mark.parametrize("out_dtype", [torch.float32, torch.bfloat16])
def test_config5_full_size_every_sequence_and_head(out_dtype):
    out, fin, r = _check_full("cfg5", out_dtype)
    if out_dtype == torch.float32:
        # per-sequence figure as well (heavy-tailed keys): no single sequence is far worse than the whole
        w = _full("cfg5")[0]
        cu = w.cu_seqlens.numpy()
        o = np64(out[0])
        worst = max(rel_err(o[cu[n]:cu[n + 1]], r[0][cu[n]:cu[n + 1]]) for n in range(len(cu) - 1))
        assert worst <= 5 * TOL_BF16


# ---- segment-parallel scan (long sequences cut into segments; same result up to rounding) ------------------
from paper_2605_08587_b200 import KLA_FLAG_EXACT_SEGMENTS, KLA_FLAG_NO_SEGMENTS, KLA_FLAG_SEGMENTS  # noqa: E402


@pytest.mark.parametrize("exact", [KLA_FLAG_EXACT_SEGMENTS, 0])   # chained transition maps always / warm-up runs where they apply
@pytest.mark.parametrize("G", [2, 3, 7])
@pytest.mark.parametrize("d", [64, 128])
def test_forced_segments_match_oracle(G, d, exact):
    w = W.config3(B=2, H=2, T=1536 + 17, d=d, seed=200 + G)
    _check_fixed(w, TOL_BF16, flags=KLA_FLAG_SEGMENTS(G) | exact)


def test_segments_equal_plain_launch_closely():
    w = W.config3(B=1, H=3, T=4096, seed=211)
    o_p, f_p = gpu_chunk(w, flags=KLA_FLAG_NO_SEGMENTS)
    o_s, f_s = gpu_chunk(w, flags=KLA_FLAG_SEGMENTS(4))
    assert rel_err(np64(o_s), np64(o_p)) <= 2e-4
    assert rel_err(np64(f_s), np64(f_p)) <= 2e-4


def test_segments_without_init_state_and_without_final_state():
    w = W.config2(B=1, H=2, T=1100, seed=213)
    out, fin = gpu_chunk(w, flags=KLA_FLAG_SEGMENTS(3), want_final_state=False)
    assert fin is None
    ro, _ = oracle_chunk(w)
    assert rel_err(np64(out), ro) <= TOL_BF16


def test_more_segments_than_chunks_is_clamped():
    w = W.config3(B=1, H=2, T=130, seed=215)
    _check_fixed(w, TOL_BF16, flags=KLA_FLAG_SEGMENTS(9))


# ---- layer-edge variants: beta = eta (gated-delta-rule coefficient) and the read-out over ||q|| -------------------
import oracle  # noqa: E402
from paper_2605_08587_b200 import KLA_FLAG_COEFF_ETA, KLA_FLAG_QNORM  # noqa: E402


def _unit_keys(w):
    """beta = eta is only a stable write for keys of about unit norm (the paper's comparison model normalises
    them): rescale k to ||k|| = 1, rounded to the workload's dtype before either side sees it."""
    k = w.k.float()
    w.k = (k / k.norm(dim=-1, keepdim=True).clamp_min(1e-12)).to(w.k.dtype)
    return w


@pytest.mark.parametrize("flags", [0, KLA_FLAG_FORCE_SIMT])
@pytest.mark.parametrize("variant", [(True, False), (False, True), (True, True)])
def test_variants_match_oracle(variant, flags):
    coeff_eta, qnorm = variant
    w = W.config3(B=2, H=2, T=300, seed=400 + 2 * coeff_eta + qnorm)
    if coeff_eta:
        w = _unit_keys(w)
    vf = (KLA_FLAG_COEFF_ETA if coeff_eta else 0) | (KLA_FLAG_QNORM if qnorm else 0)
    out, fin = gpu_chunk(w, flags=flags | vf)
    with oracle.variant(coeff_eta=coeff_eta, qnorm=qnorm):
        ro, rf = oracle_chunk(w)
    assert rel_err(np64(out), ro) <= TOL_BF16
    assert rel_err(np64(fin), rf) <= TOL_BF16


def test_variants_fp32_and_segments():
    w = _unit_keys(W.config1(B=1, H=2, T=200, d=64, seed=410))
    out, fin = gpu_chunk(w, flags=KLA_FLAG_COEFF_ETA | KLA_FLAG_QNORM)
    with oracle.variant(coeff_eta=True, qnorm=True):
        ro, rf = oracle_chunk(w)
    assert rel_err(np64(out), ro) <= TOL_F32
    assert rel_err(np64(fin), rf) <= TOL_F32
    w = _unit_keys(W.config3(B=1, H=2, T=1024, seed=411))
    out, fin = gpu_chunk(w, flags=KLA_FLAG_COEFF_ETA | KLA_FLAG_QNORM | KLA_FLAG_SEGMENTS(4))
    with oracle.variant(coeff_eta=True, qnorm=True):
        ro, rf = oracle_chunk(w)
    assert rel_err(np64(out), ro) <= TOL_BF16
    assert rel_err(np64(fin), rf) <= TOL_BF16


# ---- the bounded-wait error path (no fault, no hang: a wait runs out by design and the kernel reports it) -------------
@pytest.mark.parametrize("no_pair", [0, 32])   # paired CTAs (a cluster per head) and independent CTAs
def test_bounded_wait_reports_timeout_and_context_stays_usable(no_pair):
    from paper_2605_08587_b200 import binding
    w = W.config2(B=1, H=2, T=200, seed=501)
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    dev = "cuda:0"
    a = [t.to(dev) for t in (w.q, w.k, w.v, w.log_alpha, w.eta)]
    from paper_2605_08587_b200 import kla_chunk_fwd
    kla_chunk_fwd(*a, w.eps, flags=binding.KLA_INTERNAL_FLAG_TEST_TIMEOUT | no_pair, status_word=status)
    torch.cuda.synchronize()                      # returns after about a second: the wait is bounded
    assert int(status.item()) == -10              # KLA_ERR_TIMEOUT
    # the same context then runs the normal path correctly, and an untouched status word stays zero
    status.zero_()
    out, fin = kla_chunk_fwd(*a, w.eps, out_dtype=torch.float32, status_word=status)
    torch.cuda.synchronize()
    ro, rf = oracle_chunk(w)
    assert int(status.item()) == 0
    assert rel_err(np64(out), ro) <= TOL_BF16 and rel_err(np64(fin), rf) <= TOL_BF16


def test_timeout_without_a_caller_status_word_is_raised_by_check():
    """The binding passes a status word of its own when the caller gives none; check() reads and clears it."""
    from paper_2605_08587_b200 import KlaError, binding, check, kla_chunk_fwd
    w = W.config2(B=1, H=2, T=200, seed=502)
    a = [t.to("cuda:0") for t in (w.q, w.k, w.v, w.log_alpha, w.eta)]
    kla_chunk_fwd(*a, w.eps)
    check("cuda:0")                               # nothing to report after an ordinary call
    kla_chunk_fwd(*a, w.eps, flags=binding.KLA_INTERNAL_FLAG_TEST_TIMEOUT)
    with pytest.raises(KlaError) as e:
        check("cuda:0")
    assert e.value.code == -10                    # KLA_ERR_TIMEOUT
    check("cuda:0")                               # cleared
    out, fin = kla_chunk_fwd(*a, w.eps, out_dtype=torch.float32)
    check("cuda:0")
    ro, rf = oracle_chunk(w)
    assert rel_err(np64(out), ro) <= TOL_BF16 and rel_err(np64(fin), rf) <= TOL_BF16


# ---- d_v = 128: the two slices of a head as a cluster that shares the solve (default) or as independent CTAs ----------
from paper_2605_08587_b200 import KLA_FLAG_NO_PAIR  # noqa: E402


@pytest.mark.parametrize("T", [1, 64, 65, 129, 1000, 2048 + 17])
def test_independent_ctas_match_oracle_and_paired_launch_bitwise(T):
    """Both launch forms do the same arithmetic on the same operands: the results must be identical, and the
    unpaired form is checked against the oracle by itself."""
    w = W.config3(B=2, H=2, T=T, seed=300 + T)
    out_u, fin_u = _check_fixed(w, TOL_BF16, flags=KLA_FLAG_NO_PAIR)
    out_p, fin_p = gpu_chunk(w)
    assert torch.equal(out_p, out_u)
    assert torch.equal(fin_p, fin_u)


def test_paired_segments_and_packed_input_bitwise():
    w = W.config3(B=1, H=3, T=1536 + 40, seed=311)
    o_p, f_p = gpu_chunk(w, flags=KLA_FLAG_SEGMENTS(3))
    o_u, f_u = gpu_chunk(w, flags=KLA_FLAG_SEGMENTS(3) | KLA_FLAG_NO_PAIR)
    assert torch.equal(o_p, o_u) and torch.equal(f_p, f_u)
    wv = W.config5(H=2, d=128, seed=313, lengths=[300, 1, 64, 700, 129])
    o_p, f_p = gpu_chunk(wv)
    o_u, f_u = gpu_chunk(wv, flags=KLA_FLAG_NO_PAIR)
    assert torch.equal(o_p, o_u) and torch.equal(f_p, f_u)


def test_paired_launch_is_repeatable_over_several_waves():
    """More clusters than the GPU holds at once, many launches: every launch must reproduce the independent-CTA result
    bit for bit (a hand-over between the CTAs of a pair that relied on timing would show up here)."""
    w = W.config2(B=24, H=8, T=640, seed=321)          # 384 CTAs of one CTA per SM
    o_u, f_u = gpu_chunk(w, flags=KLA_FLAG_NO_PAIR)
    for _ in range(12):
        o_p, f_p = gpu_chunk(w)
        assert torch.equal(o_p, o_u) and torch.equal(f_p, f_u)
    wl = W.config3()                                    # one long sequence: segment passes of 256 and 144 CTAs
    o_u, f_u = gpu_chunk(wl, flags=KLA_FLAG_NO_PAIR)
    for _ in range(12):
        o_p, f_p = gpu_chunk(wl)
        assert torch.equal(o_p, o_u) and torch.equal(f_p, f_u)


@pytest.mark.parametrize("flags", [0, KLA_FLAG_NO_PAIR, KLA_FLAG_FORCE_SIMT])
@pytest.mark.parametrize("d", [64, 128])
def test_decay_far_beyond_the_exponent_range_within_one_chunk(d, flags):
    """log alpha of -0.5 .. -4 per token: exp(g_C - g_j) spans hundreds of binades inside a chunk, far below what fp32
    holds.  The tensor-core kernel factors the output product through those weights (with a floor): the outputs of
    tokens next to the writes, where the unfactored decay is ~1, must still be right."""
    w = W.config3(B=2, H=2, T=200, d=d, seed=71)
    g = torch.Generator().manual_seed(72)
    w.log_alpha = -(0.5 + 3.5 * torch.rand(w.log_alpha.shape, generator=g))
    _check_fixed(w, TOL_BF16, flags=flags)


# ---- seeded sweep over shapes and launch forms ------------------------------------------------------------------------------
def _sweep_cases():
    rng = np.random.default_rng(20260501)
    cases = []
    for n in range(24):
        d = int(rng.choice([64, 128]))
        B = int(rng.integers(1, 4))
        H = int(rng.integers(1, 5))
        T = int(rng.choice([rng.integers(1, 64), rng.integers(64, 400), rng.integers(400, 1400)]))
        form = int(rng.choice([0, KLA_FLAG_NO_PAIR, KLA_FLAG_SEGMENTS(int(rng.integers(2, 6))),
                               KLA_FLAG_SEGMENTS(int(rng.integers(2, 6))) | KLA_FLAG_NO_PAIR]))
        bf16_out = bool(rng.integers(0, 2))
        cases.append((n, d, B, H, T, form, bf16_out))
    return cases


@pytest.mark.parametrize("n,d,B,H,T,form,bf16_out", _sweep_cases())
def test_seeded_sweep_of_shapes_and_launch_forms(n, d, B, H, T, form, bf16_out):
    w = (W.config3 if n % 2 else W.config2)(B=B, H=H, T=T, d=d, seed=900 + n)   # with / without an initial state
    _check_fixed(w, TOL_BF16, flags=form, out_dtype=torch.bfloat16 if bf16_out else torch.float32)


# ---- head dimension 128 in the WY form (KLA_FLAG_WY_FORM): same checks as the default form -------------------------------
from paper_2605_08587_b200 import binding as _binding  # noqa: E402

WY = _binding.KLA_FLAG_WY_FORM


@pytest.mark.parametrize("T", [1, 5, 63, 64, 65, 128, 129, 200, 1000, 2048 + 17])
def test_wy_form_lengths(T):
    _check_fixed(W.config3(B=2, H=2, T=T, seed=700 + T), TOL_BF16, flags=WY)


def test_wy_form_without_init_state_bf16_out():
    _check_fixed(W.config2(B=2, H=3, T=777, seed=711), TOL_BF16, flags=WY, out_dtype=torch.bfloat16)


@pytest.mark.parametrize("G", [2, 5])
def test_wy_form_segments(G):
    _check_fixed(W.config3(B=2, H=2, T=1536 + 17, seed=720 + G), TOL_BF16, flags=WY | KLA_FLAG_SEGMENTS(G))


def test_wy_form_packed_input():
    w = W.config3(B=1, H=2, T=300 + 1 + 64 + 700 + 129, seed=731)   # layer-shaped values, packed
    w.cu_seqlens = torch.tensor([0, 300, 301, 365, 1065, 1194], dtype=torch.int32)
    w.init_state = (0.02 * torch.randn(5, 2, 128, 128, generator=torch.Generator().manual_seed(732))).float()
    out, fin = gpu_chunk(w, flags=WY)
    ro, rf, _ = oracle_chunk(w)
    assert rel_err(np64(out)[0], ro) <= TOL_BF16
    assert rel_err(np64(fin), rf) <= TOL_BF16


@pytest.mark.parametrize("variant", [(True, False), (False, True), (True, True)])
def test_wy_form_variants(variant):
    coeff_eta, qnorm = variant
    w = W.config3(B=2, H=2, T=300, seed=740 + 2 * coeff_eta + qnorm)
    if coeff_eta:
        w = _unit_keys(w)
    vf = (KLA_FLAG_COEFF_ETA if coeff_eta else 0) | (KLA_FLAG_QNORM if qnorm else 0)
    out, fin = gpu_chunk(w, flags=WY | vf)
    with oracle.variant(coeff_eta=coeff_eta, qnorm=qnorm):
        ro, rf = oracle_chunk(w)
    assert rel_err(np64(out), ro) <= TOL_BF16
    assert rel_err(np64(fin), rf) <= TOL_BF16


def test_wy_form_is_deterministic_and_close_to_the_default_form():
    w = W.config2(B=6, H=8, T=640, seed=751)   # more clusters than run at once would need many more; several per SM pair
    a = gpu_chunk(w, flags=WY)
    b = gpu_chunk(w, flags=WY)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    d = gpu_chunk(w)
    assert rel_err(np64(a[0]), np64(d[0])) <= 2e-3 and rel_err(np64(a[1]), np64(d[1])) <= 2e-3


def test_wy_form_decay_far_beyond_the_exponent_range():
    w = W.config3(B=2, H=2, T=200, seed=761)
    g = torch.Generator().manual_seed(762)
    w.log_alpha = -(0.5 + 3.5 * torch.rand(w.log_alpha.shape, generator=g))
    _check_fixed(w, TOL_BF16, flags=WY)


def test_wy_form_bounded_wait_reports_timeout():
    w = W.config2(B=1, H=2, T=200, seed=771)
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    a = [t.to("cuda:0") for t in (w.q, w.k, w.v, w.log_alpha, w.eta)]
    from paper_2605_08587_b200 import kla_chunk_fwd
    kla_chunk_fwd(*a, w.eps, flags=WY | _binding.KLA_INTERNAL_FLAG_TEST_TIMEOUT, status_word=status)
    torch.cuda.synchronize()
    assert int(status.item()) == -10
    status.zero_()
    out, fin = kla_chunk_fwd(*a, w.eps, out_dtype=torch.float32, flags=WY, status_word=status)
    torch.cuda.synchronize()
    ro, rf = oracle_chunk(w)
    assert int(status.item()) == 0
    assert rel_err(np64(out), ro) <= TOL_BF16 and rel_err(np64(fin), rf) <= TOL_BF16
