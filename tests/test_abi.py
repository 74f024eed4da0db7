"""CPU-side checks of the C-ABI library: it loads, exports what the header declares, and rejects
bad arguments on the host without touching a GPU."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2605_08587_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.load()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "kla.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(kla_[a-z_0-9]+)\s*\(", text)))


def test_header_symbols_are_exported(lib):
    names = _declared_functions()
    assert {"kla_chunk_fwd", "kla_decode_step", "kla_chunk_fwd_workspace_bytes", "kla_status_str"} <= set(names)
    for n in names:
        assert hasattr(lib, n), "missing export " + n
    assert set(binding.EXPORTS) <= set(names)


def test_status_strings(lib):
    seen = set()
    for code in range(0, -12, -1):
        s = binding.status_str(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 12
    assert binding.status_str(-99) == "unknown status"


def _desc(**kw):
    base = dict(B=1, T=64, H=2, d_k=64, d_v=64, n_seq=1, cu_seqlens=None, host_seqlens=None,
                io_dtype=binding.KLA_BF16, out_dtype=binding.KLA_F32, flags=0, workspace=None,
                workspace_bytes=0, status_word=None, stream=None)
    base.update(kw)
    return binding.KlaDesc(**base)


FAKE = 0x1000  # 16-byte aligned, never dereferenced: validation fails (or no sm_100 device) first


def _call_chunk(lib, desc, q=FAKE, k=FAKE, v=FAKE, la=FAKE, eta=FAKE, eps=1e-6, chunk=64, init=None, out=FAKE, fin=None):
    return lib.kla_chunk_fwd(ctypes.byref(desc), q, k, v, la, eta, eps, chunk, init, out, fin)


def test_chunk_fwd_validation(lib):
    assert _call_chunk(lib, _desc(), q=None) == -1
    assert _call_chunk(lib, _desc(), out=None) == -1
    assert _call_chunk(lib, _desc(d_k=96, d_v=96)) == -2
    assert _call_chunk(lib, _desc(d_v=128)) == -2
    assert _call_chunk(lib, _desc(H=0)) == -2
    assert _call_chunk(lib, _desc(n_seq=3)) == -2
    assert _call_chunk(lib, _desc(io_dtype=7)) == -3
    assert _call_chunk(lib, _desc(out_dtype=-1)) == -3
    assert _call_chunk(lib, _desc(), k=FAKE + 4) == -4
    assert _call_chunk(lib, _desc(), fin=FAKE + 8) == -4
    assert _call_chunk(lib, _desc(), chunk=48) == -5
    assert _call_chunk(lib, _desc(), chunk=128) == -5
    assert _call_chunk(lib, _desc(), eps=-1.0) == -8
    assert _call_chunk(lib, _desc(), eps=float("nan")) == -8
    assert _call_chunk(lib, _desc(), eps=float("inf")) == -8


def test_chunk_fwd_seqlens_validation(lib):
    def with_lens(lens, T, n_seq=None, B=1):
        arr = np.asarray(lens, dtype=np.int32)
        d = _desc(B=B, T=T, n_seq=len(lens) - 1 if n_seq is None else n_seq, cu_seqlens=FAKE,
                  host_seqlens=arr.ctypes.data)
        return _call_chunk(lib, d), arr
    assert with_lens([0, 10, 5, 64], 64)[0] == -6       # not monotone
    assert with_lens([1, 10, 64], 64)[0] == -6          # does not start at 0
    assert with_lens([0, 10, 60], 64)[0] == -6          # does not end at T
    assert with_lens([0, 10, 64], 64, B=2)[0] == -2     # packed input needs B = 1
    d = _desc(cu_seqlens=FAKE, host_seqlens=None)
    assert _call_chunk(lib, d) == -1                    # host copy required


def test_decode_validation(lib):
    d = _desc(T=1, B=4, n_seq=4)
    f = lib.kla_decode_step
    assert f(ctypes.byref(d), FAKE, FAKE, FAKE, FAKE, FAKE, 1e-6, None, FAKE) == -1
    assert f(ctypes.byref(_desc(T=2, B=4, n_seq=4)), FAKE, FAKE, FAKE, FAKE, FAKE, 1e-6, FAKE, FAKE) == -2
    assert f(ctypes.byref(d), FAKE, FAKE + 2, FAKE, FAKE, FAKE, 1e-6, FAKE, FAKE) == -4
    assert f(ctypes.byref(d), FAKE, FAKE, FAKE, FAKE, FAKE, -0.5, FAKE, FAKE) == -8
    assert lib.kla_decode_steps(ctypes.byref(d), -1, FAKE, FAKE, FAKE, FAKE, FAKE, 1e-6, FAKE, FAKE) == -2


def test_no_silent_fallback_without_sm100(lib):
    """Valid arguments on a machine without an sm_100 device must give KLA_ERR_ARCH, not a CPU path."""
    import torch
    if torch.cuda.is_available() and torch.cuda.get_device_capability(0)[0] == 10:
        pytest.skip("an sm_100 device is present")
    assert _call_chunk(lib, _desc()) == -11
    d = _desc(T=1, B=4, n_seq=4)
    assert lib.kla_decode_step(ctypes.byref(d), FAKE, FAKE, FAKE, FAKE, FAKE, 1e-6, FAKE, FAKE) == -11


def test_workspace_query(lib):
    assert lib.kla_chunk_fwd_workspace_bytes(ctypes.byref(_desc(d_k=7, d_v=7)), 64) == 0
    assert lib.kla_chunk_fwd_workspace_bytes(None, 64) == 0
    assert lib.kla_chunk_fwd_workspace_bytes(ctypes.byref(_desc()), 64) >= 0


def test_workspace_grows_only_when_sequences_are_cut_into_segments(lib):
    """Host logic of the segment-parallel scan: few long sequences get a workspace, many short ones do not,
    flags force it on or off, and a missing workspace is refused before anything is launched."""
    many = _desc(B=8, T=4096, H=8, d_k=128, d_v=128, n_seq=8)
    assert lib.kla_chunk_fwd_workspace_bytes(ctypes.byref(many), 64) == 0
    long1 = _desc(B=1, T=65536, H=8, d_k=128, d_v=128, n_seq=1)
    need = lib.kla_chunk_fwd_workspace_bytes(ctypes.byref(long1), 64)
    assert need > 0
    state = 8 * 128 * 128 * 4
    plan = lambda B, G, H: ((B * G + 2 + B * G * H) * 4 + 255) // 256 * 256   # bounds, plan word, warm-up length per (segment, head)
    G = need // (3 * state)
    assert 2 <= G <= 32 and need == plan(1, G, 8) + 3 * G * state   # plan block (padded) + map, local, start per segment
    off = _desc(B=1, T=65536, H=8, d_k=128, d_v=128, n_seq=1, flags=2)
    assert lib.kla_chunk_fwd_workspace_bytes(ctypes.byref(off), 64) == 0
    forced = _desc(B=8, T=4096, H=8, d_k=128, d_v=128, n_seq=8, flags=4 << 8)
    assert lib.kla_chunk_fwd_workspace_bytes(ctypes.byref(forced), 64) == plan(8, 4, 8) + 3 * 8 * 4 * state
    assert lib.kla_chunk_fwd(ctypes.byref(forced), FAKE, FAKE, FAKE, FAKE, FAKE, 1e-6, 64, None, FAKE, None) == -7
    # fp32 inputs and chunk 32 go to the CUDA-core kernel: never segmented
    f32 = _desc(B=1, T=65536, H=8, d_k=128, d_v=128, n_seq=1, io_dtype=binding.KLA_F32)
    assert lib.kla_chunk_fwd_workspace_bytes(ctypes.byref(f32), 64) == 0
    assert lib.kla_chunk_fwd_workspace_bytes(ctypes.byref(long1), 32) == 0


def test_packed_input_asks_for_one_word_per_sequence(lib):
    """Packed input on the tensor-core path is taken longest sequence first: one int32 per sequence of scratch."""
    import numpy as np
    cu = np.array([0, 100, 164, 1000], dtype=np.int32)
    d = _desc(B=1, T=1000, H=2, d_k=64, d_v=64, n_seq=3, cu_seqlens=FAKE, host_seqlens=cu.ctypes.data)
    assert lib.kla_chunk_fwd_workspace_bytes(ctypes.byref(d), 64) == 256
    assert lib.kla_chunk_fwd_workspace_bytes(ctypes.byref(d), 32) == 0        # CUDA-core kernel
    assert _call_chunk(lib, d) == -7                                            # workspace missing


def test_binding_rejects_cpu_tensors():
    import torch
    from paper_2605_08587_b200 import kla_chunk_fwd
    q = torch.zeros(1, 64, 2, 64)
    with pytest.raises((ValueError, RuntimeError, AssertionError)):
        kla_chunk_fwd(q, q, q, torch.zeros(1, 64, 2), torch.zeros(1, 64, 2), 1e-6)
