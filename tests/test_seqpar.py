"""Sequence-parallel prefill (one long sequence cut along T across ranks).

CPU part: the orchestration of paper_2605_08587_b200/seqpar.py with world-size-2 and -3 gloo process groups, the
arithmetic of the steps supplied by the fp64 oracle -- it checks which rank reads which map and that the one all-gather
is enough.  GPU part: the same orchestration on one device that plays every rank in turn (no kernel waits for another),
the steps being the library's kernels, against the oracle on the whole sequence.
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from helpers import TOL_BF16, np64, rel_err
from paper_2605_08587_b200 import seqpar, workloads as W


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _spans(T, world):
    """Token ranges of the ranks: equal chunks-of-64 shares, the remainder on the last rank."""
    per = (T // world) // 64 * 64
    cuts = [r * per for r in range(world)] + [T]
    return [(cuts[r], cuts[r + 1]) for r in range(world)]


def _oracle_steps(gather):
    """The four steps in fp64 on the CPU (test code): the maps come from the oracle's recurrence run from the identity
    with v = 0 and from zero; the chaining is written out."""
    import oracle

    def span_map(k, v, la, eta, eps):
        B, T, H, d = k.shape
        eye = np.broadcast_to(np.eye(d), (B, H, d, d)).copy()
        q0 = np.zeros_like(np64(k))
        _, phi, _ = oracle.forward(q0, np64(k), np.zeros_like(np64(v)), np64(la), np64(eta), eps, eye)
        _, n, _ = oracle.forward(q0, np64(k), np64(v), np64(la), np64(eta), eps, None)
        return torch.from_numpy(phi), torch.from_numpy(n)

    def state_chain(phi, n, s0):
        B, R, H, d, _ = phi.shape
        start = torch.zeros_like(phi)
        cur = torch.zeros(B, H, d, d, dtype=torch.float64) if s0 is None else s0.double().clone()
        for r in range(R):
            start[:, r] = cur
            cur = phi[:, r] @ cur + n[:, r]
        return start

    def forward(q, k, v, la, eta, eps, s0):
        out, fin, _ = oracle.forward(np64(q), np64(k), np64(v), np64(la), np64(eta), eps, s0.numpy())
        return torch.from_numpy(out), torch.from_numpy(fin)

    return seqpar.Steps(span_map=span_map, all_gather=gather, state_chain=state_chain, forward=forward)


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = W.config3(B=2, H=2, T=640 + 37, d=64, seed=40 + world)   # every rank draws the same sequence, keeps its span
    a, b = _spans(w.q.shape[1], world)[rank]

    def gather(x):
        bufs = [torch.empty_like(x) for _ in range(world)]
        dist.all_gather(bufs, x.contiguous())
        return torch.stack(bufs, 1)

    o, fin = seqpar.sequence_parallel_forward(rank, _oracle_steps(gather), w.q[:, a:b], w.k[:, a:b], w.v[:, a:b],
                                              w.log_alpha[:, a:b], w.eta[:, a:b], w.eps, w.init_state.double())
    out[rank] = (o.numpy(), fin.numpy())
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_gloo_ranks_reproduce_the_whole_sequence(world):
    import oracle
    port = _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    w = W.config3(B=2, H=2, T=640 + 37, d=64, seed=40 + world)
    ro, rf, _ = oracle.forward(np64(w.q), np64(w.k), np64(w.v), np64(w.log_alpha), np64(w.eta), w.eps, np64(w.init_state))
    got = np.concatenate([res[r][0] for r in range(world)], axis=1)
    assert rel_err(got, ro) <= 1e-9
    assert rel_err(res[world - 1][1], rf) <= 1e-9          # the last rank ends with the sequence's final state


# ---- GPU: one device plays every rank in turn ---------------------------------------------------------------------------
def _emulated(w, world, flags=0):
    from paper_2605_08587_b200 import binding
    dev = "cuda:0"
    spans = _spans(w.q.shape[1], world)
    g = {k: getattr(w, k).to(dev) for k in ("q", "k", "v", "log_alpha", "eta")}
    s0 = w.init_state.to(dev)
    maps = [binding.kla_chunk_span_map(g["k"][:, a:b].contiguous(), g["v"][:, a:b].contiguous(), g["log_alpha"][:, a:b].contiguous(),
                                       g["eta"][:, a:b].contiguous(), w.eps, flags=flags) for a, b in spans]
    phi_all = torch.stack([m[0] for m in maps], 1)
    n_all = torch.stack([m[1] for m in maps], 1)
    outs, fin = [], None
    for r, (a, b) in enumerate(spans):
        steps = seqpar.Steps(span_map=lambda *x, r=r: maps[r], all_gather=lambda x: phi_all if x is maps[r][0] else n_all,
                             state_chain=binding.kla_state_chain,
                             forward=lambda q, k, v, la, eta, eps, st: binding.kla_chunk_fwd(q, k, v, la, eta, eps, init_state=st,
                                                                                            out_dtype=torch.float32, flags=flags))
        o, fin = seqpar.sequence_parallel_forward(r, steps, *[g[k][:, a:b].contiguous() for k in ("q", "k", "v", "log_alpha", "eta")],
                                                  w.eps, s0)
        outs.append(o)
    torch.cuda.synchronize()
    return torch.cat(outs, 1), fin, phi_all, n_all


@pytest.mark.gpu
@pytest.mark.parametrize("d,world,flags", [(128, 2, 0), (128, 4, 0), (64, 3, 0), (128, 3, 64)])
def test_emulated_ranks_match_the_oracle(d, world, flags):
    import oracle
    w = W.config3(B=2, H=2, T=2048 + 64 * world + 21, d=d, seed=50 + world)
    out, fin, phi_all, n_all = _emulated(w, world, flags)
    ro, rf, _ = oracle.forward(np64(w.q), np64(w.k), np64(w.v), np64(w.log_alpha), np64(w.eta), w.eps, np64(w.init_state))
    assert rel_err(np64(out), ro) <= TOL_BF16
    assert rel_err(np64(fin), rf) <= TOL_BF16


@pytest.mark.gpu
@pytest.mark.parametrize("d", [64, 128])
def test_span_map_matches_the_recurrence_run_from_identity_and_from_zero(d):
    """S_end = phi . S_start + n on a span short enough that phi has not decayed to nothing."""
    import oracle
    from paper_2605_08587_b200 import binding
    w = W.config3(B=2, H=2, T=150, d=d, seed=61)
    dev = "cuda:0"
    phi_g, n_g = binding.kla_chunk_span_map(w.k.to(dev), w.v.to(dev), w.log_alpha.to(dev), w.eta.to(dev), w.eps)
    torch.cuda.synchronize()
    eye = np.broadcast_to(np.eye(d), (2, 2, d, d)).copy()
    k, v, la, eta = (np64(x) for x in (w.k, w.v, w.log_alpha, w.eta))
    _, phi, _ = oracle.forward(np.zeros_like(k), k, np.zeros_like(v), la, eta, w.eps, eye)
    _, n0, _ = oracle.forward(np.zeros_like(k), k, v, la, eta, w.eps, None)
    assert rel_err(np64(phi_g), phi) <= TOL_BF16
    assert rel_err(np64(n_g), n0) <= TOL_BF16
    # chaining: three spans' worth of maps against the written-out recurrence
    gen = torch.Generator().manual_seed(62)
    P = (0.3 * torch.randn(2, 3, 2, d, d, generator=gen)).float()
    N = torch.randn(2, 3, 2, d, d, generator=gen).float()
    start = binding.kla_state_chain(P.to(dev), N.to(dev), w.init_state.to(dev)).cpu().double()
    cur = w.init_state.double()
    for r in range(3):
        assert rel_err(start[:, r].numpy(), cur.numpy()) <= 1e-5
        cur = P[:, r].double() @ cur + N[:, r].double()
