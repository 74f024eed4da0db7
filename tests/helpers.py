"""Shared test helpers: the parity metric and oracle/GPU call wrappers."""
import numpy as np
import torch

TOL_BF16 = 2e-3   # max|err| / rms(ref) for bf16 inputs with fp32 accumulation
TOL_F32 = 1e-5    # same metric, fp32 inputs


def rel_err(got, ref):
    """max_i |got_i - ref_i| / sqrt(mean_i ref_i^2)."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    rms = np.sqrt(np.mean(ref * ref))
    if rms == 0.0:
        return float(np.abs(got - ref).max())
    return float(np.abs(got - ref).max() / rms)


def np64(t):
    return t.detach().float().cpu().numpy().astype(np.float64) if isinstance(t, torch.Tensor) else np.asarray(t, dtype=np.float64)


def bf16_half_ulp(ref):
    """Half a bf16 unit in the last place at |ref| (8 significand bits), for the output-rounding floor."""
    ref = np.abs(np.asarray(ref, dtype=np.float64))
    e = np.floor(np.log2(np.maximum(ref, 2.0 ** -126)))
    return 0.5 * 2.0 ** (e - 7)


def assert_bf16_out_close(got, ref, tol=TOL_BF16):
    """A bf16-rounded output cannot meet the max/rms bound by itself (its own rounding is up to 2^-9
    relative), so it is held to |got - ref| <= tol * rms(ref) + half a bf16 ulp of ref."""
    got, ref = np64(got), np.asarray(ref, dtype=np.float64)
    rms = np.sqrt(np.mean(ref * ref))
    bound = tol * rms + bf16_half_ulp(ref) * 1.0001
    bad = np.abs(got - ref) > bound
    assert not bad.any(), "bf16 out: %d elements beyond bound, worst excess %g" % (
        bad.sum(), float((np.abs(got - ref) - bound).max()))


def oracle_chunk(w, heads=None, seqs=None):
    """Run the oracle on a ChunkWorkload (optionally on a subset of heads / sequences).
    Returns (out [n_tok_sel, H_sel, d_v], final [n_seq_sel, H_sel, d_k, d_v])."""
    import oracle
    H = w.q.shape[2]
    heads = list(range(H)) if heads is None else list(heads)
    q, k, v = (np64(a[0] if w.cu_seqlens is not None else a)[..., heads, :] for a in (w.q, w.k, w.v))
    la, eta = (np64(a[0] if w.cu_seqlens is not None else a)[..., heads] for a in (w.log_alpha, w.eta))
    s0 = None if w.init_state is None else np64(w.init_state)[:, heads]
    if w.cu_seqlens is None:
        B = q.shape[0]
        seqs = list(range(B)) if seqs is None else list(seqs)
        out, fin, _ = oracle.forward(q[seqs], k[seqs], v[seqs], la[seqs], eta[seqs], w.eps,
                                     None if s0 is None else s0[seqs])
        return out, fin
    cu = w.cu_seqlens.numpy().astype(np.int64)
    n_seq = len(cu) - 1
    seqs = list(range(n_seq)) if seqs is None else list(seqs)
    idx = np.concatenate([np.arange(cu[n], cu[n + 1]) for n in seqs]) if seqs else np.zeros(0, dtype=np.int64)
    lens = np.array([cu[n + 1] - cu[n] for n in seqs], dtype=np.int64)
    cu_sel = np.concatenate([[0], np.cumsum(lens)])
    out, fin, _ = oracle.forward_packed(q[idx], k[idx], v[idx], la[idx], eta[idx], w.eps, cu_sel,
                                        None if s0 is None else s0[seqs])
    return out, fin, idx


def gpu_chunk(w, out_dtype=torch.float32, flags=0, chunk=None, want_final_state=True, plan_word=None):
    from paper_2605_08587_b200 import kla_chunk_fwd
    dev = "cuda:0"
    cu = None if w.cu_seqlens is None else w.cu_seqlens.to(dev)
    out, fin = kla_chunk_fwd(w.q.to(dev), w.k.to(dev), w.v.to(dev), w.log_alpha.to(dev), w.eta.to(dev), w.eps,
                             chunk=chunk or w.chunk,
                             init_state=None if w.init_state is None else w.init_state.to(dev),
                             cu_seqlens=cu, host_seqlens=w.cu_seqlens, out_dtype=out_dtype, flags=flags,
                             want_final_state=want_final_state, plan_word=plan_word)
    torch.cuda.synchronize()
    return out, fin
