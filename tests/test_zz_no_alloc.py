"""kla_chunk_fwd_static_scratch: the chunk forward for callers that cannot allocate device memory.

Such callers (code running where its framework serves no allocations, a plugin that only gets its input and
output buffers, a binding without cudaMalloc) cannot hand kla_chunk_fwd the workspace it wants for the
segment-parallel scan; this entry point takes the scratch from a fixed array inside the library instead.  The
tests call it through the C ABI, twice in a row on different shapes (the array keeps the previous call's
contents), and compare with kla_chunk_fwd given an ordinary workspace.  This file is collected last on purpose:
a run that stops at the first failure has then already run every other test.
"""
import ctypes

import pytest
import torch

from helpers import TOL_BF16, np64, rel_err
from paper_2605_08587_b200 import (KLA_FLAG_SEGMENTS, KlaError, binding, kla_chunk_fwd, kla_chunk_fwd_static_scratch,
                                   workloads as W)

DEV = "cuda:0"


def _both(w, flags):
    a = [t.to(DEV) for t in (w.q, w.k, w.v, w.log_alpha, w.eta)]
    s0 = w.init_state.to(DEV)
    out_ref, fin_ref = kla_chunk_fwd(*a, w.eps, init_state=s0, out_dtype=torch.float32, flags=flags)
    out = torch.full_like(out_ref, float("nan"))
    fin = torch.full_like(fin_ref, float("nan"))
    kla_chunk_fwd_static_scratch(*a, w.eps, out, fin, init_state=s0, flags=flags)
    torch.cuda.synchronize()
    return out, fin, out_ref, fin_ref


@pytest.mark.gpu
def test_static_scratch_matches_workspace_path_on_two_calls_in_a_row():
    first = W.config3(B=1, H=2, T=2048 + 33, seed=301)      # 5 segments
    second = W.config3(B=2, H=3, T=1024, d=64, seed=302)    # another shape, 3 segments: reuses the same bytes
    for w, g in ((first, 5), (second, 3)):
        out, fin, out_ref, fin_ref = _both(w, KLA_FLAG_SEGMENTS(g))
        assert torch.isfinite(out).all() and torch.isfinite(fin).all()
        assert rel_err(np64(out), np64(out_ref)) <= TOL_BF16
        assert rel_err(np64(fin), np64(fin_ref)) <= TOL_BF16
    # and once more on the first shape, after the array was used for the second
    out, fin, out_ref, fin_ref = _both(first, KLA_FLAG_SEGMENTS(5))
    assert rel_err(np64(out), np64(out_ref)) <= TOL_BF16
    assert rel_err(np64(fin), np64(fin_ref)) <= TOL_BF16


@pytest.mark.gpu
def test_static_scratch_without_segments_needs_no_scratch():
    w = W.config3(B=2, H=2, T=200, seed=303)
    out, fin, out_ref, fin_ref = _both(w, 0)
    assert rel_err(np64(out), np64(out_ref)) <= TOL_BF16
    assert rel_err(np64(fin), np64(fin_ref)) <= TOL_BF16


def test_shapes_beyond_the_fixed_array_are_refused_before_anything_runs():
    """Host-side check, no GPU needed: 64 sequences x 8 heads x 8 segments of 128 x 128 states need 805 MB."""
    lib = binding.load()
    fake = 0x1000
    desc = binding.KlaDesc(B=64, T=4096, H=8, d_k=128, d_v=128, n_seq=64, cu_seqlens=None, host_seqlens=None,
                           io_dtype=binding.KLA_BF16, out_dtype=binding.KLA_BF16, flags=KLA_FLAG_SEGMENTS(8),
                           workspace=None, workspace_bytes=0, status_word=None, stream=None)
    assert lib.kla_chunk_fwd_workspace_bytes(ctypes.byref(desc), 64) > binding.STATIC_SCRATCH_BYTES
    code = lib.kla_chunk_fwd_static_scratch(ctypes.byref(desc), fake, fake, fake, fake, fake, 1e-6, 64, None, fake, None)
    assert code == -7
    with pytest.raises(KlaError):
        binding._check(code)
