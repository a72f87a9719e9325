#!/usr/bin/env python
"""Benchmark of the ReHyAt hybrid attention operator on B200.

    python bench.py --gpus N --steps K --warmup W [--impl reference] [--workload NAME]

One step = one pass of the whole operator (state increments, scan, linear read-out, softmax
window + joint normaliser) over one synthetic layer input.  At N=1 the workload is the
Wan2.1-1.3B-shaped layer (B=1, 12 heads of 128, 21 latent frames of 30x52 = 32,760 tokens,
chunk 3, overlap 1, bf16).  With N>1 (one process per GPU under torchrun) every rank runs its
own layer input of that shape: the (batch, head) problems are independent, so there is no
collective on the data path and scaling is weak.

`value` is algorithmic TFLOP/s of the whole job with inputs resident in HBM; `e2e` is the same
metric through the host-buffer entry point (pinned host tensors, copies inside the timed
region).  `--impl reference` times the fp64 CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2601_04342_b200 import geometry, synth  # noqa: E402

METRIC = "hybrid-attention TFLOP/s (algorithmic) per layer at 32,760 tokens"
UNIT = "TFLOP/s"

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from one ncu capture of that
# kernel at this workload, together with a digest of the kernel's sources at the time of the capture: the figure
# is reported only for the kernel it was taken on and only while those sources are unchanged.
KERNEL_SOURCES = {"window_tc": ("rehyat_tc.cuh", "rehyat_ptx.cuh", "rehyat_common.cuh"),
                  "window_tc1": ("rehyat_tc_single.cuh", "rehyat_tc.cuh", "rehyat_ptx.cuh", "rehyat_common.cuh")}
NCU_CAPTURES = {   # kernel -> bytes per launch, workload and source digest of the ncu capture the figure was read from
    "window_tc": {"traffic": 394308864 + 84172288, "workload": "wan13b_layer", "sources": "2159efc4c3b5db21"},
}


def kernel_source_digest(kernel):
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES.get(kernel, ()):
        with open(os.path.join(ROOT, "paper_2601_04342_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def ncu_traffic(kernel, workload):
    cap = NCU_CAPTURES.get(kernel)
    if not cap or cap["workload"] != workload or cap["sources"] != kernel_source_digest(kernel):
        return None
    return cap["traffic"]


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"bf16_burst": p["bf16_tflops"], "bf16_sustained": p["bf16_tflops_sustained"],
                "hbm_gbs": p["hbm_gbs"], "source": "measured"}
    return {"bf16_burst": 1590.0, "bf16_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.lines = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20",
                 "-i", str(self.gpu)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._pump, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line))

    def wait_running(self, timeout=5.0):
        """Blocks until the first sample has arrived (nvidia-smi takes a while to start), so that a short timed
        region that follows is sampled from its start."""
        t_end = time.time() + timeout
        while self.proc is not None and not self.lines and time.time() < t_end:
            time.sleep(0.005)

    def stop(self, t0=None, t1=None):
        """Summary of the samples that arrived in the host-time window [t0, t1] (all samples if no window is
        given; the sample nearest to the window if it was shorter than the sampling period)."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.03)                               # one more sampling period: the last sample of the window
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        lines = self.lines
        if t0 is not None and lines:
            inside = [x for x in lines if t0 <= x[0] <= t1 + 0.03]
            lines = inside or [min(lines, key=lambda x: abs(x[0] - 0.5 * (t0 + t1)))]
        sm, smax, reasons, power = [], [], set(), []
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for _, line in lines:
            tok = [t.strip() for t in line.split(",")]
            if len(tok) < 9:
                continue
            try:
                sm.append(float(tok[1])); smax.append(float(tok[2])); power.append(float(tok[3]))
            except ValueError:
                continue
            for name, val in zip(names, tok[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p["num_threads"] for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def oracle_sample(wl, inputs, heads, frames=None):
    """Times the fp64 oracle (recurrent form, as it stands) on `heads` of batch 0 of the workload, optionally on
    its first `frames` latent frames only.  Returns (seconds, algorithmic FLOPs of what was computed)."""
    from oracle import rehyat_oracle as orc
    T = wl.T if frames is None else frames
    n = T * wl.HW
    sel = lambda t: t[:1, heads, :n].to(torch.float64).numpy()
    q, k, v = sel(inputs["q"]), sel(inputs["k"]), sel(inputs["v"])
    pq = {n_: t[heads].to(torch.float64).numpy() for n_, t in inputs["phi_q"].items()}
    pk = {n_: t[heads].to(torch.float64).numpy() for n_, t in inputs["phi_k"].items()}
    t0 = time.perf_counter()
    orc.hybrid_rnn(q, k, v, pq, pk, T, wl.HW, wl.Tc, wl.To, P=wl.P)
    dt = time.perf_counter() - t0
    flops = geometry.flop_model(1, len(heads), wl.head_dim, T, wl.HW, wl.Tc, wl.To, wl.D_h, wl.D_out)["total"]
    return dt, flops


def config_of(wl, extra=None):
    cfg = {"workload": wl.name, "batch": wl.B, "heads": wl.n_heads, "head_dim": wl.head_dim,
           "latent_frames": wl.T, "patch_grid": [wl.H, wl.W], "tokens": wl.N, "chunk_frames": wl.Tc,
           "overlap_frames": wl.To, "phi": {"hidden": wl.D_h, "dim": wl.D_out, "degree": wl.P, "act": "relu/relu",
                                            "param_std": 0.02},
           "c_mode": "rowmax", "qk_rms_norm": wl.rms_norm_qk,
           "l2": "inputs (q,k,v,out = %.0f MB) exceed the 126 MB L2; no flush" %
                 (geometry.io_bytes(wl.B, wl.n_heads, wl.head_dim, wl.N, 2) / 1e6)}
    if extra:
        cfg.update(extra)
    return cfg


def _time_ms(fn, stream, warmup, steps):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        fn()
    e1.record(stream)
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / steps


def full_softmax_comparison(wl, dev, phi_q, phi_k, stream, hybrid_ms, flops, warmup=2, steps=5):
    """Full softmax attention (Eq. 2) at the workload's shape: this operator with one chunk covering
    every frame (exact by the T_c = T limit) and, as an independent time, the library SDPA kernel."""
    from paper_2601_04342_b200 import binding
    op = binding.for_workload(wl, max_chunk_frames=wl.T)
    out = torch.empty_like(dev["q"])
    ours = _time_ms(lambda: op.forward(dev["q"], dev["k"], dev["v"], phi_q, phi_k, wl.T, wl.H, wl.W, wl.T, 0,
                                       out=out, stream=stream), stream, warmup, steps)
    assert op.status() == 0
    op.close()
    lib = _time_ms(lambda: torch.nn.functional.scaled_dot_product_attention(dev["q"], dev["k"], dev["v"]), stream,
                   warmup, steps)
    return {"flop": flops["full_softmax"], "this_operator_chunk_eq_frames_ms": ours,
            "this_operator_tflops": flops["full_softmax"] / (ours * 1e-3) / 1e12,
            "library_sdpa_ms": lib, "library_sdpa_tflops": flops["full_softmax"] / (lib * 1e-3) / 1e12,
            "hybrid_ms": hybrid_ms, "hybrid_speedup_vs_this_operator_full": ours / hybrid_ms,
            "hybrid_speedup_vs_library_sdpa": lib / hybrid_ms}


def workspace_by_frames(wl, device):
    """rehyat_workspace_bytes of contexts made for 21, 41 and 81 latent frames: the workspace is a
    function of the configuration only, not of the video length (Section 3.3, note 3)."""
    from paper_2601_04342_b200 import binding
    out = {}
    for T in (21, 41, 81):
        op = binding.for_workload(wl.with_(T=T), device=device)
        out[str(T)] = op.workspace_bytes
        op.close()
    return out


def stream_timing(wl, dev, phi_q, phi_k, stream, flops):
    """The same layer fed chunk by chunk through rehyat_stream_step (state held by the context)."""
    from paper_2601_04342_b200 import binding
    op = binding.for_workload(wl)
    HW = wl.HW
    n_chunks = -(-wl.T // wl.Tc)
    chunks = []
    for t in range(n_chunks):
        sl = slice(t * wl.Tc * HW, min((t + 1) * wl.Tc, wl.T) * HW)
        chunks.append(tuple(dev[n][:, :, sl].contiguous() for n in ("q", "k", "v")) + (min((t + 1) * wl.Tc, wl.T) - t * wl.Tc,))
    outs = [torch.empty_like(c[0]) for c in chunks]

    def run():
        op.stream_begin(wl.B, wl.H, wl.W, wl.Tc, wl.To, stream=stream)
        for (q, k, v, f), o in zip(chunks, outs):
            op.stream_step(q, k, v, phi_q, phi_k, f, out=o, stream=stream)

    ms = _time_ms(run, stream, 2, 10)
    assert op.status() == 0
    res = {"ms_per_layer": ms, "tflops": flops["total"] / (ms * 1e-3) / 1e12, "steps_per_layer": n_chunks,
           "state_bytes_after_last_step": lib_state_bytes(op)}
    op.close()
    return res


def bidirectional_timing(wl, dev, phi_q, phi_k, stream, causal_ms):
    """The variant of Eq. 10-12 (linear branch over every token outside the window) at the same shape."""
    from paper_2601_04342_b200 import binding
    op = binding.for_workload(wl, bidirectional=True)
    out = torch.empty_like(dev["q"])
    ms = _time_ms(lambda: op.forward(dev["q"], dev["k"], dev["v"], phi_q, phi_k, wl.T, wl.H, wl.W, wl.Tc, wl.To,
                                     out=out, stream=stream), stream, 3, 20)
    assert op.status() == 0
    res = {"ms_per_step": ms, "causal_ms_per_step": causal_ms, "launches_per_step": op.last_launches}
    op.close()
    return res


def qk_transform_timing(wl, dev, phi_q, phi_k, stream, plain_ms, peaks):
    """The same layer with q and k normalised and rotated ahead of the operator by the library's own pass
    (per-head RMS norm with weights, rotary tables of one-dimensional positions): the pass is bound by HBM, it
    reads q, k and writes the transformed q, k once."""
    from paper_2601_04342_b200 import binding
    op = binding.for_workload(wl, qk_transform=True)
    w = torch.ones((wl.n_heads, wl.head_dim), device="cuda", dtype=dev["q"].dtype)
    half = wl.head_dim // 2
    ang = torch.arange(wl.N, device="cuda", dtype=torch.float32)[:, None] * \
        (10000.0 ** (-torch.arange(half, device="cuda", dtype=torch.float32) / half))[None, :]
    cos, sin = torch.cos(ang).contiguous(), torch.sin(ang).contiguous()
    op.set_qk_transform(q_weight=w, k_weight=w, cos=cos, sin=sin)
    out = torch.empty_like(dev["q"])
    run = lambda: op.forward(dev["q"], dev["k"], dev["v"], phi_q, phi_k, wl.T, wl.H, wl.W, wl.Tc, wl.To, out=out, stream=stream)
    for _ in range(3):
        run()
    op.profile_enable(True)
    ms = _time_ms(run, stream, 0, 20)
    prof = op.profile_read()
    op.profile_enable(False)
    assert op.status() == 0
    prep_ms = prof["qk_prep"][0] / max(prof["qk_prep"][1], 1)
    nbytes = 4 * wl.B * wl.n_heads * wl.N * wl.head_dim * dev["q"].element_size()      # q, k read; q', k' written
    res = {"ms_per_step": ms, "plain_ms_per_step": plain_ms, "prepass_ms": prep_ms, "prepass_algorithmic_bytes": nbytes,
           "prepass_gbs": nbytes / (prep_ms * 1e-3) / 1e9 if prep_ms > 0 else None,
           "prepass_frac_of_hbm_peak": nbytes / (prep_ms * 1e-3) / 1e9 / peaks["hbm_gbs"] if prep_ms > 0 else None,
           "workspace_bytes": op.workspace_bytes}
    op.close()
    return res


def lib_state_bytes(op):
    from paper_2601_04342_b200 import binding
    return binding.lib().rehyat_stream_state_bytes(op._h)


def linear_share_summary(op, wl, run):
    """Runs one step with the library's diagnostic output switched on and summarises nL / (nS + nL) (Eq. 8, 9):
    how much of the joint normaliser the linear branch carries, over the rows that have a linear set."""
    share = torch.zeros((wl.B, wl.n_heads, wl.N), device="cuda", dtype=torch.float32)
    op.set_linear_share_output(share)
    run()
    torch.cuda.synchronize()
    op.set_linear_share_output(None)
    first_linear = next((c.q0 for c in geometry.chunk_plan(wl.T, wl.HW, wl.Tc, wl.To) if c.lo > 0), wl.N)
    rows = share[:, :, first_linear:]
    if rows.numel() == 0:
        return {"rows_with_linear_set": 0.0, "mean": 0.0, "median": 0.0, "max": 0.0}
    return {"rows_with_linear_set": (wl.N - first_linear) / wl.N, "mean": float(rows.mean()),
            "median": float(rows.median()), "max": float(rows.max())}


def time_config(wl, device, stream, full_softmax=False, steps=20, rms_norm=True):
    """Kernel-resident timing of another configuration.  Inputs are drawn on the device (seeded torch
    generator, N(0,1), q and k RMS-normalised where the configuration says so) because the host recipe takes
    tens of seconds at these sizes; the parity tests use the host recipe."""
    from paper_2601_04342_b200 import binding
    gen = torch.Generator(device="cuda").manual_seed(wl.seed)
    shape = (wl.B, wl.n_heads, wl.N, wl.head_dim)
    q, k, v = (torch.randn(shape, generator=gen, device="cuda", dtype=torch.float32) for _ in range(3))
    if rms_norm and wl.rms_norm_qk:
        q = q / q.pow(2).mean(-1, keepdim=True).sqrt()
        k = k / k.pow(2).mean(-1, keepdim=True).sqrt()
    q, k, v = q.to(torch.bfloat16), k.to(torch.bfloat16), v.to(torch.bfloat16)
    pq = {n: t.cuda() for n, t in synth.make_phi_params(wl, "phi_q").items()}
    pk = {n: t.cuda() for n, t in synth.make_phi_params(wl, "phi_k").items()}
    out = torch.empty_like(q)
    op = binding.for_workload(wl, device=device)
    run = lambda: op.forward(q, k, v, pq, pk, wl.T, wl.H, wl.W, wl.Tc, wl.To, out=out, stream=stream)
    ms = _time_ms(run, stream, 3, steps)
    assert op.status() == 0
    fl = geometry.flop_model(wl.B, wl.n_heads, wl.head_dim, wl.T, wl.HW, wl.Tc, wl.To, wl.D_h, wl.D_out)
    res = {"workload": wl.name, "batch": wl.B, "heads": wl.n_heads, "head_dim": wl.head_dim, "tokens": wl.N, "chunk_frames": wl.Tc, "overlap_frames": wl.To,
           "steps": steps, "ms_per_step": ms, "tflops": fl["total"] / (ms * 1e-3) / 1e12,
           "tokens_per_s": wl.B * wl.N / (ms * 1e-3), "workspace_bytes": op.workspace_bytes, "launches_per_step": op.last_launches,
           "window_tiles_per_item": op.last_window_tiles, "full_softmax_flop_ratio": fl["full_softmax"] / fl["total"],
           "linear_share_of_normaliser": linear_share_summary(op, wl, run)}
    op.close()
    if full_softmax:
        res["full_softmax_same_shape"] = full_softmax_comparison(wl, {"q": q, "k": k, "v": v}, pq, pk, stream, ms, fl,
                                                                 warmup=1, steps=2)
    return res


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    inputs = synth.make_inputs(wl)
    # Every step is a bounded sample of the workload, sized from one calibration pass so that the whole run of
    # warmup + steps stays within about two and a half minutes: as many heads as fit, else one head on its first frames.
    t_head, _ = oracle_sample(wl, inputs, [0])
    per_step = 150.0 / max(args.warmup + args.steps, 1)
    n_heads = int(min(args.ref_heads, wl.n_heads, max(1, per_step // t_head)))
    frames = None
    if t_head > per_step:
        frames = wl.T
        while frames > wl.Tc + wl.To + 1 and t_head * (frames / wl.T) ** 1.2 > per_step:
            frames -= wl.Tc
    heads = list(range(n_heads))
    times = []
    flops = 0
    for i in range(args.warmup + args.steps):
        dt, flops = oracle_sample(wl, inputs, heads, frames)
        if i >= args.warmup:
            times.append(dt)
    total = sum(times)
    value = flops * len(times) / total / 1e12
    sample = (f"{len(heads)} of {wl.n_heads} heads of batch 0, " +
              (f"all {wl.N} tokens" if frames is None else f"the first {frames} of {wl.T} latent frames ({frames * wl.HW} tokens)") +
              ", recurrent form, fp64 numpy")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_of(wl),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="wan13b_layer", choices=sorted(synth.CONFIGS))
    ap.add_argument("--ref-heads", type=int, default=12, help="heads the oracle sample covers")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--kernel-impl", default="auto", choices=["auto", "simt", "tensor"])
    ap.add_argument("--no-full-softmax", action="store_true", help="skip the full-softmax comparison at the same shape")
    ap.add_argument("--all-configs", action="store_true",
                    help="also the full-softmax comparison at the CFG-batch shape and the bidirectional variant")
    ap.add_argument("--shard", default="replicas", choices=["replicas", "heads"],
                    help="with --gpus N > 1: every rank runs its own layer input (weak scaling, the default), or ONE "
                         "layer's (batch, head) problems are split over the ranks (strong scaling)")
    ap.add_argument("--no-other-configs", action="store_true",
                    help="skip the CFG-batch, long-video, 320x480 and chunk/overlap-sweep timings")
    ap.add_argument("--sustained-seconds", type=float, default=3.0,
                    help="length of the power-capped leg (0 skips it)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    wl = synth.CONFIGS[args.workload]

    if args.impl == "reference":
        run_reference(args, wl)
        return

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the operator has no CPU path")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    from paper_2601_04342_b200 import binding, build
    if rank == 0:
        build.build()
    if dist:
        dist.barrier()

    # every rank draws its own layer input (weak scaling over independent problems); when one layer is split
    # over the ranks, all of them draw the same input and each computes its own (batch, head) problems of it
    shard_heads = args.shard == "heads" and world > 1
    wl_rank = wl if shard_heads else wl.with_(seed=wl.seed + 1000 * rank)
    host = synth.make_inputs(wl_rank)
    dev = {n: host[n].cuda() for n in ("q", "k", "v")}
    phi_q = {n: t.cuda() for n, t in host["phi_q"].items()}
    phi_k = {n: t.cuda() for n, t in host["phi_k"].items()}
    out = torch.empty_like(dev["q"])
    op = binding.for_workload(wl, impl=args.kernel_impl, device=local_rank)
    stream = torch.cuda.current_stream()
    sharded = None
    if shard_heads:
        sharded = binding.ShardedRehyat(world, rank, batch=wl.B, n_heads=wl.n_heads, head_dim=wl.head_dim, dtype=wl.dtype,
                                        phi_hidden=wl.D_h, phi_dim=wl.D_out, poly_degree=wl.P, impl=args.kernel_impl,
                                        max_tokens_per_frame=wl.HW, max_chunk_frames=min(wl.Tc, wl.T), device=local_rank)

    def step():
        if sharded is not None:
            sharded.forward(dev["q"], dev["k"], dev["v"], out, phi_q, phi_k, wl.T, wl.H, wl.W, wl.Tc, wl.To, stream=stream)
        else:
            op.forward(dev["q"], dev["k"], dev["v"], phi_q, phi_k, wl.T, wl.H, wl.W, wl.Tc, wl.To, out=out, stream=stream)

    def barrier():
        if dist:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    assert op.status() == 0 and (sharded is None or sharded.status() == 0), "device status word set during warm-up"
    launches_per_step = sharded.last_launches if sharded is not None else op.last_launches
    kernel_family = op.last_impl
    window_tiles = op.last_window_tiles

    flops = geometry.flop_model(wl.B, wl.n_heads, wl.head_dim, wl.T, wl.HW, wl.Tc, wl.To, wl.D_h, wl.D_out)
    sampler = ClockSampler(local_rank)
    op.profile_enable(True)
    sampler.start()
    sampler.wait_running()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_host0 = time.time()
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    clocks = sampler.stop(t_host0, time.time())
    ms_total = e0.elapsed_time(e1)
    prof = op.profile_read()
    op.profile_enable(False)
    assert op.status() == 0, "device status word set during the timed region"
    if dist:
        t = torch.tensor([ms_total], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total = float(t.item())
    ms_step = ms_total / args.steps
    jobs = 1 if shard_heads else world               # layers the whole job computes per step
    value = jobs * flops["total"] / (ms_step * 1e-3) / 1e12

    # end to end through the host-buffer entry point (pinned host tensors, copies timed)
    pinned = {n: host[n].pin_memory() for n in ("q", "k", "v")}
    out_host = torch.empty_like(host["q"]).pin_memory()
    nbytes = host["q"].numel() * host["q"].element_size()

    def e2e_step():
        op.forward_host(pinned["q"], pinned["k"], pinned["v"], out_host, phi_q, phi_k, wl.T, wl.H, wl.W, wl.Tc, wl.To,
                        stream=stream)

    e2e_step()
    barrier()
    e0.record(stream)
    for _ in range(args.e2e_steps):
        e2e_step()
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1) / args.e2e_steps
    if dist:
        t = torch.tensor([e2e_ms], device="cuda", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())
    e2e_value = world * flops["total"] / (e2e_ms * 1e-3) / 1e12       # the host-buffer entry point always runs a whole layer per rank

    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    timed_s = ms_total * 1e-3
    peak_kind = "sustained" if timed_s >= 2.0 else "burst"
    peak = peaks["bf16_sustained"] if peak_kind == "sustained" else peaks["bf16_burst"]
    win_ms, win_n = prof["window"]
    win_flops_per_launch = flops["window"] * args.steps / max(win_n, 1)
    achieved = win_flops_per_launch / (win_ms / max(win_n, 1) * 1e-3) / 1e12 if win_ms > 0 else None
    kernel_name = ("window_tc" if window_tiles == 2 else "window_tc1") if kernel_family == "tensor" else "window_simt"
    roofline = {"bound": "tensor", "kernel": kernel_name, "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                "frac": achieved / peak if achieved else None, "traffic": ncu_traffic(kernel_name, wl.name),
                "traffic_captured_on": kernel_name if ncu_traffic(kernel_name, wl.name) is not None else None,
                "peak_source": f"{peaks['source']} bf16 {peak_kind} (MEASURED_PEAKS.json)" if peaks["source"] == "measured"
                else "fallback",
                "frac_of_nominal_2250": achieved / 2250.0 if achieved else None,
                "frac_of_measured_sustained": achieved / peaks["bf16_sustained"] if achieved else None,
                "launches": win_n, "avg_launch_ms": win_ms / max(win_n, 1),
                "algorithmic_flop_per_launch": win_flops_per_launch,
                "hbm_gbs_whole_step": geometry.io_bytes(wl.B, wl.n_heads, wl.head_dim, wl.N, 2) / (ms_step * 1e-3) / 1e9,
                "hbm_peak_gbs": peaks["hbm_gbs"]}
    kernel_ms = {k: {"ms_per_step": v[0] / args.steps, "launches_per_step": v[1] / args.steps} for k, v in prof.items()}

    cpu = None
    if not args.no_cpu_baseline and world == 1:
        heads = list(range(args.ref_heads))
        dt, fl = oracle_sample(wl, host, heads)
        cpu = {"value": fl / dt / 1e12, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
               "sample": f"{len(heads)} of {wl.n_heads} heads of batch 0, all {wl.N} tokens, recurrent form, "
                         f"fp64 numpy, {dt:.1f} s"}

    extras = {}
    if world == 1 and args.sustained_seconds > 0:
        # The same step looped for seconds, with the clock sampler running across it: the regime in which the GPU
        # sits at its power cap.  Reported against the sustained peak (a matmul looped for seconds, same regime).
        n_sus = max(int(args.sustained_seconds / (ms_step * 1e-3)), 10)
        sus_sampler = ClockSampler(local_rank)
        torch.cuda.synchronize()
        sus_sampler.start()
        sus_sampler.wait_running()
        sus_ms = _time_ms(step, stream, 3, n_sus)
        sus_clocks = sus_sampler.stop()
        sus_tf = flops["total"] / (sus_ms * 1e-3) / 1e12
        extras["sustained"] = {"steps": n_sus, "seconds": sus_ms * n_sus * 1e-3, "ms_per_step": sus_ms, "value": sus_tf,
                               "unit": UNIT, "clocks": sus_clocks,
                               "ms_x_mhz": sus_ms * sus_clocks["sm_mhz"] if sus_clocks.get("sm_mhz") else None,
                               "frac_of_measured_sustained": sus_tf / peaks["bf16_sustained"],
                               "frac_of_measured_burst": sus_tf / peaks["bf16_burst"]}
    if world == 1:
        # Whether the timed loop above reached the power cap depends on --steps (its clock record is in "clocks").
        # For context (never the headline value): ten steps after the GPU has been idle for a second.
        time.sleep(1.0)
        idle_ms = _time_ms(step, stream, 3, 10)
        extras["ten_steps_after_idle"] = {"ms_per_step": idle_ms, "value": flops["total"] / (idle_ms * 1e-3) / 1e12,
                                          "unit": UNIT, "frac_of_measured_burst": flops["total"] / (idle_ms * 1e-3) / 1e12 / peaks["bf16_burst"],
                                          "frac_of_nominal_2250": flops["total"] / (idle_ms * 1e-3) / 1e12 / 2250.0}
    if world == 1:
        # The timed loop leaves L2 as the previous step left it (the steady state of a layer called again and again;
        # the tensors exceed L2 anyway).  For comparison, ten steps each started after 256 MB of writes have swept L2.
        sweep = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        f0 = [torch.cuda.Event(enable_timing=True) for _ in range(10)]
        f1 = [torch.cuda.Event(enable_timing=True) for _ in range(10)]
        for a, b in zip(f0, f1):
            sweep.zero_()
            a.record(stream)
            step()
            b.record(stream)
        torch.cuda.synchronize()
        extras["l2_swept_before_each_step"] = {"ms_per_step": sum(a.elapsed_time(b) for a, b in zip(f0, f1)) / 10}
        del sweep
    if world == 1 and wl.dtype == "bf16" and not args.no_full_softmax:
        extras["full_softmax_same_shape"] = full_softmax_comparison(wl, dev, phi_q, phi_k, stream, ms_step, flops)
    if world == 1:
        extras["workspace_bytes_by_latent_frames"] = workspace_by_frames(wl, local_rank)
        extras["chunk_by_chunk"] = stream_timing(wl, dev, phi_q, phi_k, stream, flops)
    if world == 1 and wl.dtype == "bf16":
        extras["qk_transform_same_shape"] = qk_transform_timing(wl, dev, phi_q, phi_k, stream, ms_step, peaks)
    if world == 1 and args.all_configs:
        extras["bidirectional_same_shape"] = bidirectional_timing(wl, dev, phi_q, phi_k, stream, ms_step)
    if world == 1:
        extras["linear_share_of_normaliser"] = linear_share_summary(op, wl, step)
    if world == 1 and not args.no_other_configs:
        extras["other_configs"] = [time_config(synth.CONFIGS[n], local_rank, stream, steps=10,
                                               full_softmax=(args.all_configs and n == "cfg_long"))
                                   for n in ("cfg_long", "long_constant_memory", "wan13b_320x480")]
        # the same tokens and model width with heads of 64 channels: tensor-core window, fp32 kernels for phi
        extras["other_configs"].append(time_config(wl.with_(name="heads_of_64", n_heads=2 * wl.n_heads, head_dim=wl.head_dim // 2),
                                                   local_rank, stream, steps=5))
        extras["chunk_overlap_sweep"] = [time_config(w, local_rank, stream, steps=5) for w in synth.sweep_configs()]

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "strong" if shard_heads else "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": config_of(wl, {"kernels": kernel_family, "parallelism": (f"one layer's {wl.B * wl.n_heads} (batch, head) problems split over {world} ranks, "
                                                f"at most {geometry.shard_efficiency(wl.B, wl.n_heads, world):.3f} efficient"
                                                if shard_heads else f"dp{world} over (batch, head) problems")}),
            "tokens_per_s": jobs * wl.B * wl.N / (ms_step * 1e-3),
            "frac_of_bf16_peak": {"measured_burst": value / world / peaks["bf16_burst"],
                                  "measured_sustained": value / world / peaks["bf16_sustained"],
                                  "nominal_2250": value / world / 2250.0},
            "clocks": clocks, "ms_x_mhz": ms_step * clocks["sm_mhz"] if clocks.get("sm_mhz") else None,
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 3 * nbytes, "d2h_bytes_per_step": nbytes,
                    "ms_per_step": e2e_ms},
            "gpu_launches": launches_per_step * args.steps,
            "kernel_ms": kernel_ms, "workspace_bytes": op.workspace_bytes,
            "roofline": roofline, "cpu_baseline": cpu}
    line.update(extras)
    print(json.dumps(line), flush=True)
    op.close()
    if dist:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
