#!/usr/bin/env python
"""Benchmark of the KLA hot path on B200.

A "step" is one chunkwise forward (prologue + UT/WY transform + inter-chunk scan, one kernel
launch) over one batch of the headline workload: bf16, B=8, H=8, T=4096, d_k=d_v=128, chunk=64,
synthetic inputs with the value distributions of the 0.4B-layer recipe.  The metric is
chunk-forward throughput in Mtok/s (one token = one position of one sequence, all heads).
With N GPUs every rank processes its own batch (independent sequences, no collective on the data
path): weak scaling, value = N * tokens / max-over-ranks time.

Reported beside it, from the same run: the decode step (B=64, H=8, d=128, 1024 consecutive steps),
the long-context and varlen workloads, an end-to-end figure with host buffers, the roofline
fraction of the chunk kernel, and the fp64 oracle timed on the host cores (a baseline, not the
target).  `--impl reference` times only that oracle.
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "chunk_fwd_throughput"
UNIT = "Mtok/s"
WORKLOAD = "cfg2_bf16_B8_H8_T4096_d128_chunk64"   # the same string in both arms
# dram__bytes_read.sum + dram__bytes_write.sum of one headline launch of the chunk kernel, from the ncu capture
# summarised under profiles/; None while the kernel has changed since the counters were taken.
CHUNK_TC_DRAM_BYTES_PER_LAUNCH = 255039232   # 203.86 MB read + 51.18 MB written
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            with open(path) as f:
                pk = json.load(f)
            return pk, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


# ---- workload accounting (algorithmic bytes / flops per token-head) -----------------------------------
def algorithmic_bytes(n_tok, H, d, n_seq, io_bytes, out_bytes, has_init, want_final):
    """q, k, v read + out written + the two fp32 gates, plus the states that are read/written."""
    per_token_head = d * io_bytes * 3 + d * out_bytes + 8
    state = n_seq * H * d * d * 4
    return n_tok * H * per_token_head + (state if has_init else 0) + (state if want_final else 0)


def algorithmic_flops(n_tok, H, d, C=64):
    """Causal-half count of Algorithm 1 (right): K K^T, K S0, T.rhs, Q S0, Q K^T, (A o QK^T) U, K^T D U, solve."""
    per_token_head = 2 * C * (d + d) + 6 * d * d + C * C / 3.0
    return n_tok * H * per_token_head


# ---- multi-rank aggregation (host logic; covered by a gloo test on CPU) ---------------------------------
def max_over_ranks(value, device):
    """Maximum of a per-rank scalar over all ranks of the default process group (identity without one)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([float(value)], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_mtok_per_s(tokens_per_rank, world, ms_per_step):
    """Every rank processes its own batch (weak scaling): tokens of all ranks over the slowest rank's time."""
    return world * tokens_per_rank / (ms_per_step * 1e-3) / 1e6


# ---- clocks sampling ------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.samples = []
        self._stop = threading.Event()
        self._thr = None

    def _run(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=5).stdout
                parts = [x.strip() for x in out.strip().split(",")]
                if len(parts) >= 7:
                    self.samples.append(parts)
            except Exception:
                pass
            self._stop.wait(0.1)

    def __enter__(self):
        self._thr = threading.Thread(target=self._run, daemon=True)
        self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        self._thr.join(timeout=10)

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            try:
                sm.append(float(s[0]))
                mx.append(float(s[1]))
            except ValueError:
                continue
            for nm, val in zip(names, s[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ---- the oracle leg (CPU baseline / reference arm) ---------------------------------------------------------
def oracle_sample_run(seed=1, B=2, H=8, T=4096, d=128, repeats=1):
    """Time the fp64 oracle, as it stands, on a bounded sample of the headline workload:
    B sequences (of the workload's 8) x all heads x all T tokens.  Returns (Mtok/s, threads, seconds)."""
    import oracle
    from paper_2605_08587_b200 import workloads as W
    w = W.config2(B=B, H=H, T=T, d=d, seed=seed)
    args = [a.float().numpy() for a in (w.q, w.k, w.v)] + [w.log_alpha.numpy(), w.eta.numpy()]
    best, thr = None, 1
    for _ in range(repeats):
        t0 = time.perf_counter()
        _, _, thr = oracle.forward(*args, w.eps)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return B * T / best / 1e6, thr, best


def oracle_chunk_workload(w):
    """The fp64 oracle, as it stands, on a whole chunk-forward workload (one run).  Returns a cpu_baseline dict."""
    import oracle
    packed = w.cu_seqlens is not None
    a = [(x[0] if packed else x).float().numpy() for x in (w.q, w.k, w.v)] + [(x[0] if packed else x).numpy() for x in (w.log_alpha, w.eta)]
    s0 = None if w.init_state is None else w.init_state.numpy()
    t0 = time.perf_counter()
    if packed:
        _, _, thr = oracle.forward_packed(*a, w.eps, w.cu_seqlens.numpy(), s0)
    else:
        _, _, thr = oracle.forward(*a, w.eps, s0)
    dt = time.perf_counter() - t0
    return {"value": w.n_tok / dt / 1e6, "unit": UNIT, "cores": thr, "kind": "oracle",
            "sample": "the whole workload %s, one run, %.1f s" % (w.name, dt)}


def oracle_decode_workload(B=64, H=8, d=128, steps=128):
    """The fp64 oracle's decode step, `steps` consecutive steps of the decode workload.  Returns a cpu_baseline dict."""
    import numpy as np
    import oracle
    from paper_2605_08587_b200 import workloads as W
    w = W.config4(B=B, H=H, d=d, steps=steps)
    st = w.state.numpy().astype(np.float64)
    a = [x.float().numpy() for x in (w.q, w.k, w.v)] + [w.log_alpha.numpy(), w.eta.numpy()]
    t0 = time.perf_counter()
    for s in range(steps):
        oracle.decode_step(a[0][s], a[1][s], a[2][s], a[3][s], a[4][s], w.eps, st)
    dt = time.perf_counter() - t0
    return {"value": B * steps / dt, "unit": "tok/s", "cores": os.cpu_count(), "kind": "oracle",
            "sample": "%d consecutive decode steps of the B=%d workload (of its 1024), %.1f s" % (steps, B, dt)}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    sample = dict(B=8, H=8, T=4096, d=128)
    for _ in range(args.warmup):
        oracle_sample_run(**sample)
    times, thr = [], 1
    for _ in range(args.steps):
        v, thr, dt = oracle_sample_run(**sample)
        times.append(dt)
    ms = 1e3 * sum(times) / len(times)
    value = sample["B"] * sample["T"] / (ms / 1e3) / 1e6
    desc = "the whole headline workload (%d sequences x 8 heads x 4096 tokens) per step" % sample["B"]
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "sampled": desc},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": thr, "kind": "oracle", "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---- GPU legs ----------------------------------------------------------------------------------------------------
def time_launches(fn, steps, warmup, stream, stats=None):
    """Average device time per call of fn() in ms: CUDA events on the launching stream, one after every call, so that
    the median and the minimum of the per-call times can be reported beside the mean (`stats`, a dict, receives them)."""
    import torch
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    ev[0].record(stream)
    for i in range(steps):
        fn()
        ev[i + 1].record(stream)
    torch.cuda.synchronize()
    if stats is not None:
        per = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
        stats.update({"ms_median": statistics.median(per), "ms_min": min(per), "ms_max": max(per), "repetitions": steps})
    return ev[0].elapsed_time(ev[steps]) / steps


def to_dev(w, dev):
    return dict(q=w.q.to(dev), k=w.k.to(dev), v=w.v.to(dev), log_alpha=w.log_alpha.to(dev), eta=w.eta.to(dev),
                init_state=None if w.init_state is None else w.init_state.to(dev),
                cu_seqlens=None if w.cu_seqlens is None else w.cu_seqlens.to(dev), host_seqlens=w.cu_seqlens)


def chunk_leg(w, dev, steps, warmup, peaks, out_dtype):
    """Time one chunk-forward workload; returns a dict of figures."""
    import torch
    from paper_2605_08587_b200 import kla_chunk_fwd
    t = to_dev(w, dev)
    B, T, H, d = w.q.shape
    n_seq = w.n_seq
    out = torch.empty((B, T, H, d), device=dev, dtype=out_dtype)
    fin = torch.empty((n_seq, H, d, d), device=dev, dtype=torch.float32)

    def step():
        kla_chunk_fwd(t["q"], t["k"], t["v"], t["log_alpha"], t["eta"], w.eps, chunk=w.chunk,
                      init_state=t["init_state"], out=out, final_state=fin, cu_seqlens=t["cu_seqlens"],
                      host_seqlens=t["host_seqlens"])

    stats = {}
    ms = time_launches(step, steps, warmup, torch.cuda.current_stream(), stats)
    # per-pass device times of one more call (set-up kernels, segment pass 1, chaining of the maps, main pass)
    passes = []
    kla_chunk_fwd(t["q"], t["k"], t["v"], t["log_alpha"], t["eta"], w.eps, chunk=w.chunk, init_state=t["init_state"], out=out,
                  final_state=fin, cu_seqlens=t["cu_seqlens"], host_seqlens=t["host_seqlens"], pass_ms=passes)
    nbytes = algorithmic_bytes(B * T, H, d, n_seq, w.q.element_size(), out.element_size(), w.init_state is not None, True)
    flops = algorithmic_flops(B * T, H, d, w.chunk)
    gbs = nbytes / (ms * 1e-3) / 1e9
    tfs = flops / (ms * 1e-3) / 1e12
    t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
    t_tc = flops / (peaks["bf16_tflops"] * 1e12)
    return {"workload": w.name, "ms": ms, **stats, "mtok_per_s": B * T / (ms * 1e-3) / 1e6, "tokens": B * T,
            "pass_us": {"setup": 1e3 * passes[0], "segment_pass_1": 1e3 * passes[1], "chain_maps": 1e3 * passes[2], "main_pass": 1e3 * passes[3]},
            "algorithmic_bytes": nbytes, "algorithmic_flops": flops, "achieved_gbs": gbs, "achieved_tflops": tfs,
            "roofline_ms": 1e3 * max(t_hbm, t_tc), "roofline_frac": max(t_hbm, t_tc) / (ms * 1e-3),
            "bound": "hbm" if t_hbm >= t_tc else "tensor"}


def decode_leg(dev, steps_per_call, calls, warmup, peaks, B=64, H=8, d=128, l2_defeat=False):
    import torch
    from paper_2605_08587_b200 import kla_decode_steps, workloads as W
    w = W.config4(B=B, H=H, d=d, steps=steps_per_call)
    args = [a.to(dev) for a in (w.q, w.k, w.v, w.log_alpha, w.eta)]
    st = w.state.to(dev).clone()
    out = torch.empty((steps_per_call, B, H, d), device=dev, dtype=torch.bfloat16)

    def step():
        kla_decode_steps(*args, w.eps, st, out=out)

    stats = {}
    ms = time_launches(step, calls, warmup, torch.cuda.current_stream(), stats) / steps_per_call
    stats = {"us_per_step_median": 1e3 * stats["ms_median"] / steps_per_call, "us_per_step_min": 1e3 * stats["ms_min"] / steps_per_call,
             "calls": calls, "consecutive_steps_per_call": steps_per_call}
    state_bytes = 2 * B * H * d * d * 4
    vec_bytes = B * H * (3 * d * 2 + d * 2 + 8)
    nbytes = state_bytes + vec_bytes
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"workload": w.name, "us_per_step": ms * 1e3, **stats, "tok_per_s": B / (ms * 1e-3), "bytes_per_step": nbytes,
            "effective_gbs": gbs, "frac_of_hbm_peak": gbs / peaks["hbm_gbs"],
            "state_mb": state_bytes / 2 / 1e6, "state_fits_l2": state_bytes / 2 < 126e6}


def wy_leg(w, t, dev, steps, warmup):
    """The headline workload through the WY-form kernel (KLA_FLAG_WY_FORM), for comparison with the default form."""
    import torch
    from paper_2605_08587_b200 import KLA_FLAG_WY_FORM, kla_chunk_fwd
    B, T, H, d = w.q.shape
    out = torch.empty((B, T, H, d), device=dev, dtype=torch.bfloat16)
    fin = torch.empty((B, H, d, d), device=dev, dtype=torch.float32)
    stats = {}
    ms = time_launches(lambda: kla_chunk_fwd(t["q"], t["k"], t["v"], t["log_alpha"], t["eta"], w.eps, chunk=w.chunk, out=out,
                                             final_state=fin, flags=KLA_FLAG_WY_FORM), steps, warmup, torch.cuda.current_stream(), stats)
    return {"workload": w.name, "ms": ms, **stats, "mtok_per_s": B * T / (ms * 1e-3) / 1e6}


def dg_leg(dev, steps, warmup, peaks):
    """Diagonal-gated extension (Appendix B.5) on the headline shape: token-recurrent CUDA-core kernel."""
    import torch
    from paper_2605_08587_b200 import kla_dg_fwd, workloads as W
    w = W.config_dg()
    t = [x.to(dev) for x in (w.q, w.k, w.v, w.log_alpha, w.eta)]
    s0 = w.init_state.to(dev)
    B, T, H, d = w.q.shape
    out = torch.empty((B, T, H, d), device=dev, dtype=torch.bfloat16)
    fin = torch.empty((B, H, d, d), device=dev, dtype=torch.float32)
    stats = {}
    ms = time_launches(lambda: kla_dg_fwd(*t, w.eps, init_state=s0, out=out, final_state=fin), steps, warmup,
                       torch.cuda.current_stream(), stats)
    nbytes = B * T * H * (3 * d * 2 + d * 2 + d * 4 + 4) + 2 * B * H * d * d * 4   # q, k, v, out, the gate vector, eta; states
    return {"workload": w.name, "ms": ms, **stats, "mtok_per_s": B * T / (ms * 1e-3) / 1e6, "algorithmic_bytes": nbytes,
            "achieved_gbs": nbytes / (ms * 1e-3) / 1e9, "roofline_frac": nbytes / (peaks["hbm_gbs"] * 1e9) / (ms * 1e-3), "bound": "hbm"}


def bwd_leg(w, dev, steps, warmup, peaks, cpu_baseline):
    """Backward pass (training, Section 5.1) on the headline shape: reverse sweep over recomputed states, fp32 on CUDA cores."""
    import torch
    from paper_2605_08587_b200 import binding, kla_bwd, workloads as W
    do, df = W.upstream_grads(w)
    t = [x.to(dev) for x in (w.q, w.k, w.v, w.log_alpha, w.eta)]
    dod, dfd = do.to(dev), df.to(dev)
    B, T, H, d = w.q.shape
    desc = binding.KlaDesc(B=B, T=T, H=H, d_k=d, d_v=d, n_seq=B, io_dtype=binding.KLA_BF16, out_dtype=binding.KLA_F32)
    import ctypes
    ws = torch.empty(int(binding.load().kla_bwd_workspace_bytes(ctypes.byref(desc))), device=dev, dtype=torch.uint8)
    stats = {}
    ms = time_launches(lambda: kla_bwd(*t, w.eps, dod, d_final_state=dfd, workspace=ws), steps, warmup,
                       torch.cuda.current_stream(), stats)
    # q, k, v, d_out bf16 and the two gates read; dq, dk, dv and the two gate gradients written in fp32; dS_T read, dS_0 written
    nbytes = B * T * H * (4 * d * 2 + 8 + 3 * d * 4 + 8) + 2 * B * H * d * d * 4
    r = {"workload": w.name, "ms": ms, **stats, "mtok_per_s": B * T / (ms * 1e-3) / 1e6, "algorithmic_bytes": nbytes,
         "workspace_bytes": ws.numel(), "achieved_gbs": nbytes / (ms * 1e-3) / 1e9,
         "roofline_frac": nbytes / (peaks["hbm_gbs"] * 1e9) / (ms * 1e-3), "bound": "hbm"}
    if cpu_baseline:
        import oracle
        a = [x.float().numpy() for x in (w.q, w.k, w.v)] + [w.log_alpha.numpy(), w.eta.numpy()]
        t0 = time.perf_counter()
        thr = oracle.backward(*a, w.eps, do.float().numpy(), None, df.numpy())["threads"]
        dt = time.perf_counter() - t0
        r["cpu_baseline"] = {"value": B * T / dt / 1e6, "unit": UNIT, "cores": thr, "kind": "oracle",
                             "sample": "the whole backward of %s, one run, %.1f s" % (w.name, dt)}
    return r


def e2e_leg(w, dev, steps, warmup, groups=8):
    """Same step, host buffers: pinned host -> device copies of every input, the launches, and the
    device -> host read of out and final state, all inside the timed region.  The batch is cut into `groups`
    groups of sequences (they are independent problems) that go round two streams, so that the upload of one
    group, the kernel of another and the download of a third overlap; the step ends when both streams have."""
    import torch
    from paper_2605_08587_b200 import kla_chunk_fwd
    host = {k: getattr(w, k).pin_memory() for k in ("q", "k", "v", "log_alpha", "eta")}
    B, T, H, d = w.q.shape
    groups = max(1, min(groups, B))
    cuts = [B * g // groups for g in range(groups + 1)]
    devbuf = {k: torch.empty_like(v, device=dev) for k, v in host.items()}
    out = torch.empty((B, T, H, d), device=dev, dtype=torch.bfloat16)
    fin = torch.empty((w.n_seq, H, d, d), device=dev, dtype=torch.float32)
    out_h = torch.empty(out.shape, dtype=out.dtype).pin_memory()
    fin_h = torch.empty(fin.shape, dtype=fin.dtype).pin_memory()
    h2d = sum(v.numel() * v.element_size() for v in host.values())
    d2h = out.numel() * out.element_size() + fin.numel() * fin.element_size()
    main = torch.cuda.current_stream()
    side = [torch.cuda.Stream(device=dev) for _ in range(2)]
    done = [torch.cuda.Event() for _ in range(2)]

    def step():
        start = torch.cuda.Event()
        start.record(main)
        for s in side:
            s.wait_event(start)
        for g in range(groups):
            lo, hi = cuts[g], cuts[g + 1]
            with torch.cuda.stream(side[g % 2]):
                for k in host:
                    devbuf[k][lo:hi].copy_(host[k][lo:hi], non_blocking=True)
                kla_chunk_fwd(devbuf["q"][lo:hi], devbuf["k"][lo:hi], devbuf["v"][lo:hi], devbuf["log_alpha"][lo:hi],
                              devbuf["eta"][lo:hi], w.eps, chunk=w.chunk, out=out[lo:hi], final_state=fin[lo:hi])
                out_h[lo:hi].copy_(out[lo:hi], non_blocking=True)
                fin_h[lo:hi].copy_(fin[lo:hi], non_blocking=True)
        for i, s in enumerate(side):
            done[i].record(s)
            main.wait_event(done[i])

    ms = time_launches(step, steps, warmup, main)
    return ms, h2d, d2h


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2605_08587_b200 import launch_count, workloads as W

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback for the product path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    peaks, peak_src = load_peaks()

    # every rank owns an independent batch of the headline workload (weak scaling)
    w = W.config2(seed=1 + rank)
    t = to_dev(w, dev)
    B, T, H, d = w.q.shape
    out = torch.empty((B, T, H, d), device=dev, dtype=torch.bfloat16)
    fin = torch.empty((B, H, d, d), device=dev, dtype=torch.float32)
    from paper_2605_08587_b200 import kla_chunk_fwd

    def step():
        kla_chunk_fwd(t["q"], t["k"], t["v"], t["log_alpha"], t["eta"], w.eps, chunk=w.chunk, out=out, final_state=fin)

    stream = torch.cuda.current_stream()
    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    n0 = launch_count()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    with ClockSampler(local) as clk:
        ev[0].record(stream)
        for i in range(args.steps):
            step()
            ev[i + 1].record(stream)
        torch.cuda.synchronize()
        launches = launch_count() - n0   # kernels launched inside the timed region
        # The timed region (a few ms) is shorter than one sampling period of nvidia-smi: the same launch is repeated
        # for 0.6 s after it, and the clock samples are taken over the timed steps and those repetitions.
        t_end = time.time() + (0.0 if args.quick else 0.6)
        while time.time() < t_end:
            step()
        torch.cuda.synchronize()
    total_ms = ev[0].elapsed_time(ev[args.steps])
    per_step = [ev[i].elapsed_time(ev[i + 1]) for i in range(args.steps)]
    if world > 1:
        dist.barrier()
    total_ms = max_over_ranks(total_ms, dev)
    ms = total_ms / args.steps
    tokens_all = world * B * T
    value = whole_job_mtok_per_s(B * T, world, ms)

    e2e_ms, h2d, d2h = (float("nan"), 0, 0) if args.quick else e2e_leg(w, dev, max(2, min(args.steps, 5)), 2)
    e2e_ms = max_over_ranks(e2e_ms, dev)

    if rank != 0:
        if world > 1:
            dist.barrier()
            dist.destroy_process_group()
        return

    nbytes = algorithmic_bytes(B * T, H, d, B, 2, 2, False, True)
    flops = algorithmic_flops(B * T, H, d, w.chunk)
    t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
    t_tc = flops / (peaks["bf16_tflops"] * 1e12)
    achieved = nbytes / (ms * 1e-3) / 1e9
    roofline = {"bound": "hbm" if t_hbm >= t_tc else "tensor", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved / peaks["hbm_gbs"], "traffic": None, "peak_source": peak_src + " (burst copy)",
                "kernel": "kla_chunk_tc_kernel",
                "algorithmic_bytes_per_launch": nbytes, "algorithmic_flops_per_launch": flops,
                "tensor_time_us_at_peak": t_tc * 1e6, "hbm_time_us_at_peak": t_hbm * 1e6,
                "frac_of_roofline_time": max(t_hbm, t_tc) / (ms * 1e-3)}
    roofline["traffic"] = CHUNK_TC_DRAM_BYTES_PER_LAUNCH

    extras = {}
    if args.quick and args.also:
        # profiling mode: one extra leg, small launch counts (the ncu captures under profiles/ use these)
        if args.also == "decode":
            extras["decode_l2_defeating_B512"] = decode_leg(dev, 4, 2, 1, peaks, B=512)
        elif args.also == "decode64":
            extras["decode_cfg4"] = decode_leg(dev, 8, 2, 1, peaks)
        elif args.also == "long":
            extras["chunk_cfg3_long_context"] = chunk_leg(W.config3(), dev, 2, 1, peaks, torch.bfloat16)
        elif args.also == "varlen":
            extras["chunk_cfg5_varlen"] = chunk_leg(W.config5(), dev, 2, 1, peaks, torch.bfloat16)
        elif args.also == "wy":
            extras["chunk_cfg2_wy_form"] = wy_leg(w, t, dev, 2, 1)
        elif args.also == "dg":
            extras["dg_fwd_layer_shape"] = dg_leg(dev, 2, 1, peaks)
        elif args.also == "bwd":
            extras["bwd_layer_shape"] = bwd_leg(W.config2(T=512), dev, 2, 1, peaks, False)
    if not args.quick:
        # decode: calls of 1024 consecutive steps on 1024 distinct token vectors, state carried in place
        extras["decode_cfg4"] = decode_leg(dev, 1024, 5, 1, peaks)
        # (B = 512: 128 consecutive steps per call; 1024 steps of inputs would be 4 GB)
        extras["decode_l2_defeating_B512"] = decode_leg(dev, 128, 5, 1, peaks, B=512)
        extras["chunk_cfg3_long_context"] = chunk_leg(W.config3(), dev, 20, 3, peaks, torch.bfloat16)
        extras["chunk_cfg5_varlen"] = chunk_leg(W.config5(), dev, 20, 3, peaks, torch.bfloat16)
        # a packed batch that one long sequence dominates: cut into pieces that start from warm-up runs
        extras["chunk_packed_one_long_sequence"] = chunk_leg(W.config5_skewed(), dev, 10, 3, peaks, torch.bfloat16)
        extras["chunk_cfg2_wy_form"] = wy_leg(w, t, dev, 20, 3)
        extras["dg_fwd_layer_shape"] = dg_leg(dev, 10, 3, peaks)
        extras["bwd_layer_shape"] = bwd_leg(w, dev, 10, 3, peaks, not args.no_cpu_baseline)
        if not args.no_cpu_baseline:
            extras["chunk_cfg3_long_context"]["cpu_baseline"] = oracle_chunk_workload(W.config3())
            extras["chunk_cfg5_varlen"]["cpu_baseline"] = oracle_chunk_workload(W.config5())
            extras["decode_cfg4"]["cpu_baseline"] = oracle_decode_workload()

    cpu = None
    if not (args.no_cpu_baseline or args.quick):
        v, thr, dt = oracle_sample_run(B=8, repeats=3)
        cpu = {"value": v, "unit": UNIT, "cores": thr, "kind": "oracle",
               "sample": "the whole headline workload (8 sequences x 8 heads x 4096 tokens), best of 3 runs, %.1f s each" % dt}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms, "ms_per_step_median": statistics.median(per_step),
            "ms_per_step_min": min(per_step), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": WORKLOAD, "per_gpu": "every GPU runs this workload on its own batch", "tokens_per_step": tokens_all,
                       "arithmetic": "bf16 tensor-core operands (derived operands as hi/lo pairs), fp32 accumulation and state",
                       "l2": "inputs+outputs per step are 271 MB > 126 MB L2, no flush needed",
                       "parallelism": "independent batches per GPU, no collective"},
            "clocks": {**clk.summary(), "sampled_over": "the timed steps and 0.6 s of the same launch repeated right after them"},
            "roofline": roofline, "cpu_baseline": cpu,
            "e2e": {"value": tokens_all / (e2e_ms * 1e-3) / 1e6, "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms},
            "gpu_launches": launches, "extras": extras}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--quick", action="store_true", help="profiling mode: headline kernel only (no e2e, decode, long-context, varlen or CPU legs)")
    ap.add_argument("--also", default="", choices=["", "decode", "decode64", "long", "varlen", "wy", "dg", "bwd"],
                    help="with --quick: run one more leg after the headline kernel (used for profiling)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
