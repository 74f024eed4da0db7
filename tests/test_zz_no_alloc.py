"""kla_chunk_fwd_static_scratch: the chunk forward for callers that cannot allocate device memory.

Such callers (code running where its framework serves no allocations, a plugin that only gets its input and
output buffers, a binding without cudaMalloc) cannot hand kla_chunk_fwd the workspace it wants for the
segment-parallel scan or for the longest-first order of packed sequences; this entry point takes the scratch from a
fixed array inside the library instead.  The tests call it through the C ABI, twice in a row on different shapes (the
array keeps the previous call's contents), and compare with kla_chunk_fwd given an ordinary workspace: both run the
same kernels on the same operands, so the results must be identical bit for bit; one shape is also checked against
the oracle.  This file is collected last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import ctypes

import pytest
import torch

from helpers import TOL_BF16, np64, oracle_chunk, rel_err
from paper_2605_08587_b200 import (KLA_FLAG_SEGMENTS, KlaError, binding, kla_chunk_fwd, kla_chunk_fwd_static_scratch,
                                   workloads as W)

DEV = "cuda:0"


def _both(w, flags, first_call_on_device=False):
    a = [t.to(DEV) for t in (w.q, w.k, w.v, w.log_alpha, w.eta)]
    s0 = None if w.init_state is None else w.init_state.to(DEV)
    cu = None if w.cu_seqlens is None else w.cu_seqlens.to(DEV)
    out_ref, fin_ref = kla_chunk_fwd(*a, w.eps, init_state=s0, out_dtype=torch.float32, flags=flags, cu_seqlens=cu,
                                     host_seqlens=w.cu_seqlens)
    out = torch.full_like(out_ref, float("nan"))
    fin = torch.full_like(fin_ref, float("nan"))
    torch.cuda.synchronize()
    held = torch.cuda.memory_allocated()
    free = torch.cuda.mem_get_info()[0]
    kla_chunk_fwd_static_scratch(*a, w.eps, out, fin, init_state=s0, flags=flags, cu_seqlens=cu, host_seqlens=w.cu_seqlens)
    torch.cuda.synchronize()
    # The call took no device memory: neither through the caching allocator nor from the driver.  (Not checked on the
    # first call: that is when the CUDA runtime loads the part of the library that holds the array.)
    if not first_call_on_device:
        assert torch.cuda.memory_allocated() == held
        assert torch.cuda.mem_get_info()[0] == free
    return out, fin, out_ref, fin_ref


@pytest.mark.gpu
def test_static_scratch_matches_workspace_path_on_two_calls_in_a_row():
    first = W.config3(B=1, H=2, T=2048 + 33, seed=301)      # 5 segments
    second = W.config3(B=2, H=3, T=1024, d=64, seed=302)    # another shape, 3 segments: reuses the same bytes
    _both(first, KLA_FLAG_SEGMENTS(5), first_call_on_device=True)   # looks up the array's address
    for w, g in ((first, 5), (second, 3), (first, 5)):
        out, fin, out_ref, fin_ref = _both(w, KLA_FLAG_SEGMENTS(g))
        assert torch.isfinite(out).all() and torch.isfinite(fin).all()
        assert torch.equal(out, out_ref) and torch.equal(fin, fin_ref)
    ro, rf = oracle_chunk(first)
    assert rel_err(np64(out), ro) <= TOL_BF16
    assert rel_err(np64(fin), rf) <= TOL_BF16


@pytest.mark.gpu
def test_static_scratch_serves_the_order_of_packed_sequences():
    w = W.config5(H=3, d=64, seed=304, lengths=[70, 300, 1, 129, 64, 513])   # packed: one int32 per sequence of scratch
    for i in range(3):
        out, fin, out_ref, fin_ref = _both(w, 0, first_call_on_device=(i == 0))   # (when this test runs alone)
        assert torch.equal(out, out_ref) and torch.equal(fin, fin_ref)
    ro, rf, _ = oracle_chunk(w)
    assert rel_err(np64(out)[0], ro) <= TOL_BF16
    assert rel_err(np64(fin), rf) <= TOL_BF16


@pytest.mark.gpu
def test_static_scratch_without_segments_needs_no_scratch():
    w = W.config3(B=2, H=2, T=200, seed=303)
    out, fin, out_ref, fin_ref = _both(w, 0, first_call_on_device=True)   # (needs no scratch: nothing to check)
    assert torch.equal(out, out_ref) and torch.equal(fin, fin_ref)


def _desc(**kw):
    base = dict(B=64, T=4096, H=8, d_k=128, d_v=128, n_seq=64, cu_seqlens=None, host_seqlens=None,
                io_dtype=binding.KLA_BF16, out_dtype=binding.KLA_BF16, flags=KLA_FLAG_SEGMENTS(8),
                workspace=None, workspace_bytes=0, status_word=None, stream=None)
    base.update(kw)
    return binding.KlaDesc(**base)


def test_shapes_beyond_the_fixed_array_are_refused_before_anything_runs():
    """Host-side check, no GPU needed: 64 sequences x 8 heads x 8 segments of 128 x 128 states need 805 MB."""
    lib = binding.load()
    fake = 0x1000
    desc = _desc()
    assert lib.kla_chunk_fwd_workspace_bytes(ctypes.byref(desc), 64) > binding.STATIC_SCRATCH_BYTES
    code = lib.kla_chunk_fwd_static_scratch(ctypes.byref(desc), fake, fake, fake, fake, fake, 1e-6, 64, None, fake, None)
    assert code == -7
    with pytest.raises(KlaError):
        binding._check(code)


def test_argument_errors_come_before_the_size_check():
    """The same validation as kla_chunk_fwd, in the same order: a NULL pointer, a bad eps or a bad chunk is reported as
    such even when the shape would also be too large for the array."""
    lib = binding.load()
    fake = 0x1000
    desc = _desc()
    call = lib.kla_chunk_fwd_static_scratch
    assert call(ctypes.byref(desc), None, fake, fake, fake, fake, 1e-6, 64, None, fake, None) == -1    # KLA_ERR_NULL
    assert call(ctypes.byref(desc), fake, fake, fake, fake, fake, -1.0, 64, None, fake, None) == -8    # KLA_ERR_EPS
    assert call(ctypes.byref(desc), fake, fake, fake, fake, fake, 1e-6, 48, None, fake, None) == -5    # KLA_ERR_CHUNK
    assert call(ctypes.byref(desc), fake + 4, fake, fake, fake, fake, 1e-6, 64, None, fake, None) == -4  # KLA_ERR_ALIGN
