"""Sequence-parallel prefill: one long sequence cut along T across ranks (one GPU per rank).

Every chunk step is affine in the incoming state (Eqs. 7-9 are linear in S_0; Appendix B writes the state after a run
of tokens as a transition applied to the start state plus a term that does not depend on it), so a span of tokens
maps the state S at its start to Phi S + N.  With rank r holding the r-th span of every sequence:

  1. every rank computes (Phi_r, N_r) of its span                  -- kla_chunk_span_map, no outputs, no exchange
  2. one all-gather of (Phi_r, N_r): 2 x B x H x d x d fp32 per rank -- the only communication
  3. every rank chains the maps of the ranks before it to get the state at the start of its span  -- kla_state_chain
  4. every rank runs the ordinary chunk forward on its span from that state                        -- kla_chunk_fwd

The result on rank r is `out` for its span; `final_state` of the last rank is the state after the whole sequence.
The steps are passed in as callables so that the orchestration (which rank reads which map) can be exercised without a
GPU; `cuda_steps()` binds them to the library and to torch.distributed.  Nothing here does arithmetic of the method.
"""
from dataclasses import dataclass
from typing import Callable

import torch


@dataclass
class Steps:
    span_map: Callable      # (k, v, log_alpha, eta, eps) -> (phi [B,H,d,d], n [B,H,d,d])
    all_gather: Callable    # (x [B,H,d,d]) -> [B, R, H, d, d], index r = rank r's tensor
    state_chain: Callable   # (phi [B,R,H,d,d], n [B,R,H,d,d], init_state or None) -> start [B,R,H,d,d]
    forward: Callable       # (q, k, v, log_alpha, eta, eps, init_state [B,H,d,d]) -> (out, final_state)


def sequence_parallel_forward(rank: int, steps: Steps, q, k, v, log_alpha, eta, eps, init_state=None):
    """Forward over this rank's span [B, T_local, H, d] of sequences that are cut along T in rank order.
    `init_state`: the state before the first token of the whole sequence (the same on every rank, or None)."""
    phi, n = steps.span_map(k, v, log_alpha, eta, eps)
    phi_all = steps.all_gather(phi)
    n_all = steps.all_gather(n)
    start = steps.state_chain(phi_all, n_all, init_state)
    return steps.forward(q, k, v, log_alpha, eta, eps, start[:, rank].contiguous())


def cuda_steps(group=None, flags=0) -> Steps:
    """The steps on the GPU: the library's kernels, and torch.distributed (NCCL) for the one all-gather."""
    import torch.distributed as dist

    from . import binding

    def all_gather(x):
        world = dist.get_world_size(group)
        buf = torch.empty((world,) + tuple(x.shape), device=x.device, dtype=x.dtype)
        dist.all_gather_into_tensor(buf, x.contiguous(), group=group)
        return buf.transpose(0, 1).contiguous()   # [B, R, H, d, d]

    def forward(q, k, v, log_alpha, eta, eps, s0):
        return binding.kla_chunk_fwd(q, k, v, log_alpha, eta, eps, init_state=s0, flags=flags)

    return Steps(span_map=lambda k, v, la, eta, eps: binding.kla_chunk_span_map(k, v, la, eta, eps, flags=flags),
                 all_gather=all_gather, state_chain=binding.kla_state_chain, forward=forward)
