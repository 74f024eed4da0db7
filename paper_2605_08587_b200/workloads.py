"""Seeded synthetic inputs shaped like the paper's workloads (0.4B model: 8 heads x head dim 128,
4K training context, 65K evaluation context, 32K-token decode prefix -- Appendix C, Section 5).

This module holds NO arithmetic of the method: it only draws random tensors.  It is the one piece
of code that both the CPU oracle's tests and the CUDA path's callers use, so that both sides see
bit-identical inputs.  bf16 inputs are rounded here, before either side consumes them.

All draws come from one CPU `torch.Generator` seeded per workload, in the fixed order
q, k, v, eta_raw, alpha_raw, [q-scale, k-scale], [init_state], [lengths], [tail masks].
"""
from dataclasses import dataclass, field
from typing import Optional

import torch


@dataclass
class ChunkWorkload:
    name: str
    q: torch.Tensor            # [B, T, H, d_k]  (varlen: B = 1, T = n_tok)
    k: torch.Tensor
    v: torch.Tensor            # [B, T, H, d_v]
    log_alpha: torch.Tensor    # [B, T, H] fp32, <= 0
    eta: torch.Tensor          # [B, T, H] fp32
    eps: float
    chunk: int
    init_state: Optional[torch.Tensor] = None   # [n_seq, H, d_k, d_v] fp32
    cu_seqlens: Optional[torch.Tensor] = None   # int32 [n_seq + 1]
    meta: dict = field(default_factory=dict)

    @property
    def n_seq(self):
        return self.q.shape[0] if self.cu_seqlens is None else self.cu_seqlens.numel() - 1

    @property
    def n_tok(self):
        return self.q.shape[0] * self.q.shape[1]


@dataclass
class DecodeWorkload:
    name: str
    q: torch.Tensor            # [steps, B, H, d_k]
    k: torch.Tensor
    v: torch.Tensor            # [steps, B, H, d_v]
    log_alpha: torch.Tensor    # [steps, B, H] fp32
    eta: torch.Tensor          # [steps, B, H] fp32
    eps: float
    state: torch.Tensor        # [B, H, d_k, d_v] fp32, the state before step 0
    meta: dict = field(default_factory=dict)


def _gates(gen, shape, alpha_div):
    eta = torch.sigmoid(torch.randn(shape, generator=gen))
    log_alpha = -torch.nn.functional.softplus(torch.randn(shape, generator=gen)) / alpha_div
    return eta.float().contiguous(), log_alpha.float().contiguous()


def config1(B=1, H=2, T=256, d=64, chunk=64, seed=0):
    """fp32 chunk forward, unnormalised N(0,1) keys, zero initial state."""
    gen = torch.Generator().manual_seed(seed)
    q = torch.randn(B, T, H, d, generator=gen)
    k = torch.randn(B, T, H, d, generator=gen)
    v = torch.randn(B, T, H, d, generator=gen)
    eta, log_alpha = _gates(gen, (B, T, H), 1.0)
    return ChunkWorkload("cfg1_fp32_B%d_H%d_T%d_d%d" % (B, H, T, d), q, k, v, log_alpha, eta,
                         1e-6, chunk, meta={"dtype": "f32"})


def _layer_shaped(gen, B, T, H, d, norm_sigma):
    q = torch.randn(B, T, H, d, generator=gen) / (d ** 0.5)
    k = torch.randn(B, T, H, d, generator=gen) / (d ** 0.5)
    v = torch.randn(B, T, H, d, generator=gen)
    eta, log_alpha = _gates(gen, (B, T, H), 8.0)
    q = q * torch.exp(0.5 * torch.randn(B, T, H, 1, generator=gen))
    k = k * torch.exp(norm_sigma * torch.randn(B, T, H, 1, generator=gen))
    return q, k, v, eta, log_alpha


def config2(B=8, H=8, T=4096, d=128, chunk=64, seed=1):
    """bf16 chunk forward at the 0.4B-layer shape; q,k ~ N(0, 1/d) x lognormal(0, 0.5) norms."""
    gen = torch.Generator().manual_seed(seed)
    q, k, v, eta, log_alpha = _layer_shaped(gen, B, T, H, d, 0.5)
    return ChunkWorkload("cfg2_bf16_B%d_H%d_T%d_d%d" % (B, H, T, d), q.bfloat16(), k.bfloat16(),
                         v.bfloat16(), log_alpha, eta, 1e-6, chunk, meta={"dtype": "bf16"})


def config3(B=1, H=8, T=65536, d=128, chunk=64, seed=2):
    """bf16 long-context prefill with a random fp32 initial state ~ N(0, std 0.02)."""
    gen = torch.Generator().manual_seed(seed)
    q, k, v, eta, log_alpha = _layer_shaped(gen, B, T, H, d, 0.5)
    s0 = (0.02 * torch.randn(B, H, d, d, generator=gen)).float().contiguous()
    return ChunkWorkload("cfg3_bf16_B%d_H%d_T%d_d%d" % (B, H, T, d), q.bfloat16(), k.bfloat16(),
                         v.bfloat16(), log_alpha, eta, 1e-6, chunk, init_state=s0,
                         meta={"dtype": "bf16"})


def config4(B=64, H=8, d=128, steps=1024, seed=3):
    """Recurrent decode: fp32 state ~ N(0, std 0.02) standing in for a 32K-token prefix; bf16
    q, k, v for `steps` consecutive tokens, same value distributions as config 2."""
    gen = torch.Generator().manual_seed(seed)
    q, k, v, eta, log_alpha = _layer_shaped(gen, steps, B, H, d, 0.5)   # [steps, B, H, .]
    s0 = (0.02 * torch.randn(B, H, d, d, generator=gen)).float().contiguous()
    return DecodeWorkload("cfg4_decode_B%d_H%d_d%d_steps%d" % (B, H, d, steps), q.bfloat16(),
                          k.bfloat16(), v.bfloat16(), log_alpha, eta, 1e-6, s0,
                          meta={"dtype": "bf16"})


def config5(n_seq=32, max_len=8192, H=16, d=64, chunk=64, seed=4, lengths=None):
    """bf16 varlen packed forward: lengths uniform in [1, max_len], heavy-tailed key norms
    lognormal(0, 1.5), 1 % of tokens with k x 1e-4 and 0.1 % with k = 0 exactly (stress eps)."""
    gen = torch.Generator().manual_seed(seed)
    if lengths is None:
        lens = torch.randint(1, max_len + 1, (n_seq,), generator=torch.Generator().manual_seed(seed + 1000))
    else:
        lens = torch.as_tensor(lengths, dtype=torch.int64)
        n_seq = lens.numel()
    n_tok = int(lens.sum())
    q, k, v, eta, log_alpha = _layer_shaped(gen, 1, n_tok, H, d, 1.5)
    u = torch.rand(1, n_tok, H, 1, generator=gen)
    k = torch.where(u < 0.01, k * 1e-4, k)
    k = torch.where(u < 0.001, torch.zeros_like(k), k)
    cu = torch.zeros(n_seq + 1, dtype=torch.int32)
    cu[1:] = torch.cumsum(lens, 0).to(torch.int32)
    return ChunkWorkload("cfg5_varlen_n%d_tok%d_H%d_d%d" % (n_seq, n_tok, H, d), q.bfloat16(),
                         k.bfloat16(), v.bfloat16(), log_alpha, eta, 1e-6, chunk, cu_seqlens=cu,
                         meta={"dtype": "bf16", "lengths": lens.tolist()})


def config_dg(B=8, H=8, T=4096, d=128, seed=5, dtype=torch.bfloat16, init_state=True):
    """Diagonal-gated variant of the layer-shaped workload (Appendix B.5): as config 2, with one decay per key dimension,
    log_alpha [B, T, H, d] = -softplus(N(0,1)) / 8 drawn independently per dimension (drawn last, after the initial state)."""
    gen = torch.Generator().manual_seed(seed)
    q, k, v, eta, _ = _layer_shaped(gen, B, T, H, d, 0.5)
    s0 = (0.02 * torch.randn(B, H, d, d, generator=gen)).float().contiguous() if init_state else None
    log_alpha = (-torch.nn.functional.softplus(torch.randn(B, T, H, d, generator=gen)) / 8.0).float().contiguous()
    return ChunkWorkload("dg_%s_B%d_H%d_T%d_d%d" % ("bf16" if dtype == torch.bfloat16 else "f32", B, H, T, d), q.to(dtype),
                         k.to(dtype), v.to(dtype), log_alpha, eta, 1e-6, 0, init_state=s0, meta={"dtype": str(dtype), "diagonal_gates": True})


def upstream_grads(w: ChunkWorkload, seed=6, final=True):
    """Seeded upstream gradients for a backward pass over workload `w`: d_out ~ N(0,1) in the dtype of v (shape of v)
    and, with `final`, d_final_state ~ N(0,1) fp32 [n_seq, H, d_k, d_v] (else None)."""
    gen = torch.Generator().manual_seed(seed)
    d_out = torch.randn(w.v.shape, generator=gen).to(w.v.dtype).contiguous()
    H, d_k, d_v = w.q.shape[2], w.q.shape[3], w.v.shape[3]
    d_final = torch.randn((w.n_seq, H, d_k, d_v), generator=gen).float().contiguous() if final else None
    return d_out, d_final


def config5_skewed(long_len=65536, n_short=31, max_short=2048, H=16, d=64, seed=7):
    """A packed batch that one sequence dominates: one sequence of `long_len` tokens and `n_short` sequences with lengths
    uniform in [1, max_short]; value distributions of config 5."""
    lens = [long_len] + torch.randint(1, max_short + 1, (n_short,), generator=torch.Generator().manual_seed(seed + 1000)).tolist()
    w = config5(H=H, d=d, seed=seed, lengths=lens)
    w.name = "packed_skewed_1x%d_plus_%d_short_H%d_d%d" % (long_len, n_short, H, d)
    return w
