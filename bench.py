#!/usr/bin/env python
"""Benchmark of the RAttention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one training step of one RAttention layer on the "c4_train_step" workload
(B=8, H_q=H_kv=16, T=4096, d=128, w=512, bf16): forward with residuals + backward
(dq, dk, dv), through the C ABI.  `value` is algorithmic TFLOP/s of that step (band pairs
and recurrent-form RLA only: masked tile halves and recomputation are not counted).
The forward-only configuration (c2) and one decode step (c5 shapes) are timed beside it
and reported under "extra".  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import tempfile
import time

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2506_15545_b200 import workloads as W  # noqa: E402

METRIC = "RAttention fwd+bwd TFLOP/s (T=4096,w=512,d=128,bf16)"

# DRAM traffic per launch of the main kernels (dram__bytes_read.sum + dram__bytes_write.sum, one
# ncu capture each on the small training case `--case train`, B = 2), in MB per batch entry of
# this head configuration; it scales with the batch.  See profiles/.  Set an entry to None when
# its kernel changes after the capture.
NCU_TRAFFIC_MB_PER_BATCH_ENTRY = {"tc_fwd": 90.3, "tc_bwd_dq": 107.1, "tc_bwd_dkv": 117.4}


# --------------------------------------------------------------------------- work model
def n_swa_pairs(T, w):
    w = min(w, T - 1)
    return (w + 1) * T - w * (w + 1) // 2


def flops(wl, what):
    """Algorithmic FLOPs.  SWA fwd 4*d per band pair and query head; RLA fwd 2*d^2 per
    residual row and query head (read-out) + 2*d^2 per absorbed token and K/V head (state
    update); backward: SWA 10*d per pair (five products), RLA 4*d^2 + 4*d^2."""
    d, T, w = wl.d, wl.T, wl.w
    n = n_swa_pairs(T, w)
    rows = max(0, T - w - 1)
    bq, bkv = wl.B * wl.H_q, wl.B * wl.H_kv
    fwd_swa = 4 * d * n * bq
    fwd_read = 2 * d * d * rows * bq
    fwd_upd = 2 * d * d * rows * bkv
    parts = {
        "fwd": fwd_swa + fwd_read + fwd_upd,
        "fwd_main": fwd_swa + fwd_read,
        "fwd_state": fwd_upd,
        "bwd": 10 * d * n * bq + 4 * d * d * rows * bq + 4 * d * d * rows * bkv,
        "bwd_dq": 4 * d * n * bq + 2 * d * d * rows * bq,
        "bwd_dkv": 6 * d * n * bq + 2 * d * d * rows * bq + 4 * d * d * rows * bkv,
    }
    parts["step"] = parts["fwd"] + parts["bwd"]
    return parts[what]


def io_bytes_fwd(wl):
    e = 2 if wl.dtype == "bf16" else 4
    return e * wl.d * wl.T * wl.B * (2 * wl.H_q + 2 * wl.H_kv)


def io_bytes_step(wl):
    """Algorithmic bytes of a training step: q, k, v, dO read; out, dq, dk, dv written (the
    residuals the forward leaves for the backward are implementation traffic, not counted)."""
    e = 2 if wl.dtype == "bf16" else 4
    return e * wl.d * wl.T * wl.B * (4 * wl.H_q + 4 * wl.H_kv)


def decode_bytes(wl):
    e = 2
    ring = 2 * wl.B * wl.H_kv * wl.w * wl.d * e
    state = 2 * wl.B * wl.H_kv * wl.d * wl.d * 4
    tok = wl.B * (2 * wl.H_q + 2 * wl.H_kv) * wl.d * e
    return ring + state + tok


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return dict(hbm=j["hbm_gbs"], tf_burst=j["bf16_tflops"], tf_sus=j["bf16_tflops_sustained"],
                    src="measured")
    return dict(hbm=6650.0, tf_burst=1590.0, tf_sus=1400.0, src="fallback")


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "20", "-i", str(index)], stdout=self.f,
                                      stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self, window=None):
        """Summary of the samples; `window` = (t0, t1) wall-clock seconds of the timed region,
        whose own samples are summarised under "timed_region"."""
        if self.p is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "samples": 0, "reasons": ["nvidia-smi unavailable"]}
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        import datetime
        sm, mx, pw, ts, reasons = [], [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1]))
                mx.append(float(c[2]))
            except ValueError:
                continue
            try:
                pw.append(float(c[3]))
            except ValueError:
                pw.append(float("nan"))
            try:
                ts.append(datetime.datetime.strptime(c[0], "%Y/%m/%d %H:%M:%S.%f").timestamp())
            except ValueError:
                ts.append(None)
            for n, v in zip(names, c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        os.unlink(self.f.name)
        out = {"sm_mhz": statistics.median(sm) if sm else None, "sm_min_mhz": min(sm) if sm else None,
               "sm_max_mhz": max(mx) if mx else None, "power_w_max": max(pw) if pw else None,
               "samples": len(sm), "reasons": sorted(reasons)}
        if window is not None:
            inside = [x for x, t in zip(sm, ts) if t is not None and window[0] <= t <= window[1]]
            out["timed_region"] = {"samples": len(inside), "sm_mhz": statistics.median(inside) if inside else None}
        return out


# ------------------------------------------------------------------------ reference arm
def oracle_step(wl, q, k, v, dy, head):
    """One bounded sample of the workload through the fp64 oracle: forward + backward of one
    (batch, head) pair at the full sequence length."""
    from oracle import rattn_oracle as O
    b, h = divmod(head, wl.H_q)
    g = wl.H_q // wl.H_kv
    q64, k64, v64, dy64 = (t.to(torch.float64).numpy() for t in (q[b, h], k[b, h // g], v[b, h // g], dy[b, h]))
    O.forward_head(q64, k64, v64, wl.w, wl.scale)
    O.backward_head(q64, k64, v64, dy64, wl.w, wl.scale)


def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return len(os.sched_getaffinity(0))


def head_flops(wl):
    one = wl.replace(B=1, H_q=1, H_kv=1)
    return flops(one, "step")


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    small = wl.replace(B=1, H_q=min(4, wl.H_q), H_kv=min(4, wl.H_kv))
    q, k, v = W.make_qkv(small)
    dy = W.make_dout(small)
    for i in range(args.warmup):
        oracle_step(small, q, k, v, dy, i % small.H_q)
    t0 = time.perf_counter()
    for i in range(args.steps):
        oracle_step(small, q, k, v, dy, i % small.H_q)
    dt = time.perf_counter() - t0
    val = head_flops(wl) * args.steps / dt / 1e12
    cores = oracle_threads()
    sample = "each step = forward+backward of one (batch, head) pair at T=4096 through the fp64 oracle"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s",
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": {"workload": workload_name(wl), "sample": sample},
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def workload_name(wl):
    return (f"{wl.name}: B={wl.B},H_q={wl.H_q},H_kv={wl.H_kv},T={wl.T},d={wl.d},w={wl.w},{wl.dtype} "
            "forward(with residuals)+backward")


# ----------------------------------------------------------------------------- our arm
def timed(fn, steps, warmup, sync):
    for _ in range(warmup):
        fn()
    sync()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(steps):
        fn()
    b.record()
    sync()
    return a.elapsed_time(b) / steps


def time_decode_steps(R, c5, dev, n_sets=3, steps_per_graph=30, replays=20, flags=0):
    """Milliseconds per decode step of config 5's shapes, device time.  The steps are captured once into a
    CUDA graph (the way a serving loop issues them) and replayed: a step takes about as long as its
    launch costs the host, so timing eager launches would measure the host.  The positions come from
    a device tensor, and the steps rotate over n_sets cache sets (ring 67 MB + state 17 MB each), so
    that with three sets every step reads its ring and state from HBM, not from L2."""
    rings = [(torch.randn(c5.B, c5.H_kv, c5.w, c5.d, device=dev).to(torch.bfloat16),
              torch.randn(c5.B, c5.H_kv, c5.w, c5.d, device=dev).to(torch.bfloat16),
              torch.zeros(c5.B, c5.H_kv, c5.d, c5.d, device=dev)) for _ in range(n_sets)]
    qd, kd, vd = W.make_decode_token(c5, 0, dev)
    od = torch.empty_like(qd)
    posd = torch.full((c5.B,), c5.T, dtype=torch.int32, device=dev)

    def steps(n):
        for i in range(n):
            r = rings[i % n_sets]
            R.rattn_decode_step_ex(qd, kd, vd, r[0], r[1], r[2], 0, scale=c5.scale, out=od, pos_dev=posd, flags=flags)

    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        steps(3)
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            steps(steps_per_graph)
    torch.cuda.synchronize()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(replays):
        graph.replay()
    e1.record()
    torch.cuda.synchronize()
    assert R.rattn_decode_status() == 0, "a device-side wait expired in a decode step"
    return e0.elapsed_time(e1) / (steps_per_graph * replays)


def whole_job(ms_local, units_per_rank, dist=None, device="cpu"):
    """Replicas only: every rank runs the same per-GPU workload with no data-path exchange.
    The job's time is the slowest rank's (MAX over ranks), its work the sum over ranks.
    Returns (ms, total units)."""
    if dist is None:
        return ms_local, units_per_rank
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item()), units_per_rank * dist.get_world_size()


def run_ours(args, wl):
    from paper_2506_15545_b200 import binding as R
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    R.lib()
    pk = peaks()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # every rank runs the same per-GPU workload (independent replicas of the layer's batch)
    wl_r = wl.replace(seed=wl.seed + rank)
    q, k, v = W.make_qkv(wl_r, dev)
    dy = W.make_dout(wl_r, dev)
    ws = R.alloc_workspace(q, k, wl.w, R.MODE_RATTN, R.FLAG_SAVE_RESIDUALS)
    out = torch.empty_like(q)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)

    def step():
        R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, workspace=ws, save_residuals=True, out=out)
        R.rattn_backward_ex(q, k, v, dy, wl.w, ws, scale=wl.scale, dq=dq, dk=dk, dv=dv)

    for _ in range(args.warmup):
        step()
    barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    launches0 = R.rattn_launch_count()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    wall0 = time.time()
    a.record()
    for _ in range(args.steps):
        step()
    b.record()
    barrier()
    wall1 = time.time()
    ms = a.elapsed_time(b) / args.steps
    launches = R.rattn_launch_count() - launches0
    # Per-kernel durations: the same K steps once more with the library's event pair around every
    # launch.  (An event between two kernels makes the second wait for the first to finish, so in
    # this pass the forward's main kernel does not overlap the chunk-state kernel as it does in
    # the timed region above; the sum of the kernels is therefore a little above ms_per_step.)
    R.rattn_timing_enable(True)
    for _ in range(args.steps):
        step()
    torch.cuda.synchronize()
    kernel_ms = R.rattn_timing_read()
    R.rattn_timing_enable(False)
    # The K timed steps last tens of milliseconds, too short for more than a sample or two of
    # nvidia-smi.  The same step is therefore repeated under the same sampler for about two
    # seconds more (timed on its own, reported as "sustained"): the clock record then has
    # dozens of samples of this very load, and the two times show whether the short region ran
    # in the burst regime (same time per step) or ahead of a power-capped steady state.
    sustained = None
    if rank == 0 and args.clock_seconds > 0:
        n_more = max(args.steps, int(args.clock_seconds * 1e3 / max(ms, 1e-3)))
        c, d = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c.record()
        for _ in range(n_more):
            step()
        d.record()
        torch.cuda.synchronize()
        sustained = {"steps": n_more, "ms_per_step": c.elapsed_time(d) / n_more}
    clocks = sampler.stop((wall0, wall1)) if sampler else None
    if clocks is not None and sustained is not None:
        clocks["sustained_loop"] = sustained
        if clocks.get("sm_mhz"):
            clocks["ms_per_step_x_sm_mhz"] = ms * clocks["sm_mhz"]
    barrier()
    assert R.rattn_read_status(ws) == 0, "device-side wait expired"
    ms, total_flops = whole_job(ms, flops(wl, "step"), dist, dev)
    value = total_flops / (ms * 1e-3) / 1e12

    # ---- dominant kernel and its roofline -------------------------------------------
    per_launch = {n: tot / cnt for n, (cnt, tot) in kernel_ms.items() if cnt}
    share = {n: tot for n, (cnt, tot) in kernel_ms.items()}
    top = max(share, key=share.get)
    kflops = {"tc_fwd": "fwd_main", "tc_chunk_delta": "fwd_state", "generic_fwd": "fwd",
              "generic_bwd_dq": "bwd_dq", "generic_bwd_dkv": "bwd_dkv",
              "tc_bwd_dq": "bwd_dq", "tc_bwd_dkv": "bwd_dkv"}
    # Which measured bf16 peak applies is read off the run: the burst figure when the timed
    # region is short and the sampled SM clock sat at its maximum, the sustained one for a
    # region of seconds or a clock held down by the power cap.  Both fractions are printed.
    region_s = ms * args.steps * 1e-3
    # clock of the timed region itself where nvidia-smi caught a sample inside it, else the loop's
    mhz = None
    if clocks:
        mhz = (clocks.get("timed_region") or {}).get("sm_mhz") or clocks.get("sm_mhz")
    at_max = bool(mhz and mhz >= 0.97 * clocks["sm_max_mhz"])
    regime = "burst" if (region_s < 1.0 and (at_max or not mhz)) else "sustained"
    peak = pk["tf_burst"] if regime == "burst" else pk["tf_sus"]
    roof = None
    if top in kflops:
        ach = flops(wl, kflops[top]) / (per_launch[top] * 1e-3) / 1e12
        mb = NCU_TRAFFIC_MB_PER_BATCH_ENTRY.get(top)
        roof = {"kernel": top, "bound": "tensor", "achieved": ach, "peak": peak, "unit": "TFLOP/s",
                "frac": ach / peak, "frac_of_burst_peak": ach / pk["tf_burst"],
                "frac_of_sustained_peak": ach / pk["tf_sus"],
                "traffic": None if mb is None else mb * 1e6 * wl.B,
                "traffic_unit": "bytes per launch (ncu capture at B=2, scaled by the batch)",
                "peak_source": f"{pk['src']} {regime} bf16 peak (timed region {region_s * 1e3:.0f} ms, "
                               f"SM clock there {mhz} MHz)",
                "algorithmic_flops_per_launch": flops(wl, kflops[top]),
                "ms_per_launch": per_launch[top]}
    t_roof_step = max(flops(wl, "step") / (peak * 1e12), io_bytes_step(wl) / (pk["hbm"] * 1e9)) * 1e3
    step_roof = {"roofline_ms": t_roof_step, "frac": t_roof_step / (ms if world == 1 else ms),
                 "flops_per_step": flops(wl, "step"), "bytes_per_step": io_bytes_step(wl),
                 "denominator": f"max(FLOPs / {peak} TF/s, bytes / {pk['hbm']} GB/s), {pk['src']} {regime}"}
    total_k = sum(share.values())
    kernels = {n: {"launches": kernel_ms[n][0], "ms_per_launch": per_launch[n], "share": share[n] / total_k}
               for n in share}

    result = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": workload_name(wl), "global_batch": wl.B * world,
                   "parallelism": f"replicas x{world}" if world > 1 else "single GPU",
                   "l2": "inputs larger than L2 (q,k,v,dO,residuals > 1 GB per step)"},
        "tokens_per_s": wl.B * wl.T * world / (ms * 1e-3),
        "gpu_launches": int(launches), "kernels": kernels, "roofline": roof, "step_roofline": step_roof,
        "clocks": clocks,
    }
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- extra: forward-only (c2) and decode (c5 shapes), device-resident -----------
    extra = {}
    sync = torch.cuda.synchronize
    del dq, dk, dv, dy
    c2 = W.C2
    q2, k2, v2 = W.make_qkv(c2, dev)
    ws2 = R.alloc_workspace(q2, k2, c2.w, R.MODE_RATTN, 0)
    # rotate three input sets (3 x 268 MB > L2) so no launch finds its inputs in L2
    sets = [(q2, k2, v2)] + [tuple(t.clone() for t in (q2, k2, v2)) for _ in range(2)]
    o2 = torch.empty_like(q2)
    it = [0]

    def fwd_only():
        s = sets[it[0] % 3]
        it[0] += 1
        R.rattn_forward_ex(s[0], s[1], s[2], c2.w, scale=c2.scale, workspace=ws2, out=o2)

    ms_f = timed(fwd_only, 60, 5, sync)
    R.rattn_timing_enable(True)      # per-kernel events serialise the two kernels: a second pass
    timed(fwd_only, 12, 0, sync)
    kf = R.rattn_timing_read()
    R.rattn_timing_enable(False)
    t_roof = max(flops(c2, "fwd") / (pk["tf_burst"] * 1e12), io_bytes_fwd(c2) / (pk["hbm"] * 1e9))
    extra["fwd_c2"] = {
        "workload": "c2_3b_fwd: B=4,H=16/16,T=4096,d=128,w=512 forward only, 3 rotating input sets",
        "ms": ms_f, "tflops": flops(c2, "fwd") / (ms_f * 1e-3) / 1e12,
        "tokens_per_s": c2.B * c2.T / (ms_f * 1e-3),
        "roofline_ms": t_roof * 1e3, "roofline_frac": t_roof * 1e3 / ms_f,
        "roofline_denominator": f"max(FLOPs/{pk['tf_burst']} TF/s burst, bytes/{pk['hbm']} GB/s), {pk['src']}",
        "kernels_ms_per_launch": {n: tot / cnt for n, (cnt, tot) in kf.items() if cnt},
    }
    del sets, q2, k2, v2, ws2, o2

    c5 = W.C5
    ms_d = time_decode_steps(R, c5, dev)
    extra["decode_c5"] = {
        "workload": "one decode step, B=32,H=32/8,d=128,w=512, three rotating cache sets, replayed from a CUDA graph",
        "ms": ms_d, "gb_per_s": decode_bytes(c5) / (ms_d * 1e-3) / 1e9,
        "roofline_frac": decode_bytes(c5) / (ms_d * 1e-3) / 1e9 / pk["hbm"],
        "tokens_per_s": c5.B / (ms_d * 1e-3),
        "roofline_denominator": f"{pk['hbm']} GB/s HBM copy, {pk['src']}",
    }
    torch.cuda.empty_cache()
    result["extra"] = extra

    # ---- end to end: host buffers in, gradients out, through the same calls ----------
    hq, hk, hv = (t.cpu().pin_memory() for t in (q, k, v))
    hdy = W.make_dout(wl_r, "cpu").pin_memory()
    dy_d = torch.empty_like(q)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    h_dq, h_dk, h_dv = (torch.empty_like(t, device="cpu").pin_memory() for t in (dq, dk, dv))

    def e2e_step():
        q.copy_(hq, non_blocking=True)
        k.copy_(hk, non_blocking=True)
        v.copy_(hv, non_blocking=True)
        dy_d.copy_(hdy, non_blocking=True)
        R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, workspace=ws, save_residuals=True, out=out)
        R.rattn_backward_ex(q, k, v, dy_d, wl.w, ws, scale=wl.scale, dq=dq, dk=dk, dv=dv)
        h_dq.copy_(dq, non_blocking=True)
        h_dk.copy_(dk, non_blocking=True)
        h_dv.copy_(dv, non_blocking=True)

    n_e2e = max(10, min(args.steps, 20))
    e2e_step()
    sync()
    per = []
    for _ in range(n_e2e):
        ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ea.record()
        e2e_step()
        eb.record()
        sync()
        per.append(ea.elapsed_time(eb))
    ms_e = statistics.median(per)
    nbytes = lambda *ts: int(sum(t.numel() * t.element_size() for t in ts))
    result["e2e"] = {"value": flops(wl, "step") / (ms_e * 1e-3) / 1e12, "unit": "TFLOP/s",
                     "ms_per_step": ms_e, "ms_per_step_min": min(per), "steps": n_e2e,
                     "h2d_bytes_per_step": nbytes(hq, hk, hv, hdy),
                     "d2h_bytes_per_step": nbytes(h_dq, h_dk, h_dv)}

    # ---- CPU baseline: the oracle, as it stands, on a bounded sample ------------------
    if world == 1:
        n_heads = 6
        qc, kc, vc, dyc = hq, hk, hv, hdy
        t0 = time.perf_counter()
        for i in range(n_heads):
            oracle_step(wl, qc, kc, vc, dyc, i * 7 % (wl.B * wl.H_q))
        dt = time.perf_counter() - t0
        result["cpu_baseline"] = {
            "value": head_flops(wl) * n_heads / dt / 1e12, "unit": "TFLOP/s", "cores": oracle_threads(),
            "kind": "oracle", "seconds": dt,
            "sample": f"{n_heads} of {wl.B * wl.H_q} (batch, head) pairs, forward+backward at full T=4096",
        }
    print(json.dumps(result))
    if dist is not None:
        dist.destroy_process_group()


def run_case(args):
    """One small, single-kernel-family case for profiler captures (`--case`): a few launches
    of one entry point on inputs a little larger than L2, no clocks sampling, no oracle."""
    from paper_2506_15545_b200 import binding as R
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    sync = torch.cuda.synchronize
    if args.case in ("fwd", "train"):
        wl = W.C2.replace(B=2)          # q,k,v,out = 134 MB
        q, k, v = W.make_qkv(wl, dev)
        ws = R.alloc_workspace(q, k, wl.w, R.MODE_RATTN, R.FLAG_SAVE_RESIDUALS if args.case == "train" else 0)
        out = torch.empty_like(q)
        if args.case == "fwd":
            fn = lambda: R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, workspace=ws, out=out)
            fl = flops(wl, "fwd")
        else:
            dy = W.make_dout(wl, dev)
            dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)

            def fn():
                R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, workspace=ws, save_residuals=True, out=out)
                R.rattn_backward_ex(q, k, v, dy, wl.w, ws, scale=wl.scale, dq=dq, dk=dk, dv=dv)
            fl = flops(wl, "step")
        ms = timed(fn, args.steps, args.warmup, sync)
        R.rattn_timing_enable(True)
        timed(fn, args.steps, 0, sync)
        km = R.rattn_timing_read()
        R.rattn_timing_enable(False)
        assert R.rattn_read_status(ws) == 0
        print(json.dumps({"case": args.case, "workload": workload_name(wl), "ms": ms,
                          "tflops": fl / (ms * 1e-3) / 1e12,
                          "kernels_ms_per_launch": {n: t / c for n, (c, t) in km.items() if c}}))
    elif args.case == "prologue":
        # qk-norm + rotary embedding over config 4's q and k (2 x 134 MB, larger than L2), then its gradient
        wl = W.C4
        q, k, _ = W.make_qkv(wl, dev)
        gq = torch.ones(wl.d, device=dev)
        qo, ko = torch.empty_like(q), torch.empty_like(k)
        nbytes = 2 * (q.numel() + k.numel()) * q.element_size()
        ms_f = timed(lambda: R.rattn_qk_prologue(q, k, q_gain=gq, k_gain=gq), args.steps, args.warmup, sync)
        wsp = torch.empty(R.rattn_qk_prologue_workspace_bytes(wl.B, wl.H_q, wl.H_kv, wl.T, wl.d), dtype=torch.uint8,
                          device=dev)
        ms_b = timed(lambda: R.rattn_qk_prologue_backward(q, k, qo, ko, q_gain=gq, k_gain=gq, workspace=wsp),
                     args.steps, args.warmup, sync)
        hbm = peaks()["hbm"]
        qt, kt = q.transpose(1, 2).contiguous(), k.transpose(1, 2).contiguous()       # [B, T, H, d]
        ms_ft = timed(lambda: R.rattn_qk_prologue(qt, kt, q_gain=gq, k_gain=gq, layout=R.LAYOUT_BTHD), args.steps,
                      args.warmup, sync)
        print(json.dumps({"case": "prologue", "workload": workload_name(wl),
                          "forward_bthd": {"ms": ms_ft, "gb_per_s": nbytes / ms_ft / 1e6,
                                           "frac_of_hbm_peak": nbytes / ms_ft / 1e6 / hbm},
                          "forward": {"ms": ms_f, "gb_per_s": nbytes / ms_f / 1e6, "frac_of_hbm_peak": nbytes / ms_f / 1e6 / hbm},
                          "backward": {"ms": ms_b, "gb_per_s": 1.5 * nbytes / ms_b / 1e6,
                                       "frac_of_hbm_peak": 1.5 * nbytes / ms_b / 1e6 / hbm},
                          "bytes": "forward: q, k read once and written once; backward: q, k and their output "
                                   "gradients read, input gradients written"}))
    else:
        c5 = W.C5
        ms = time_decode_steps(R, c5, dev, steps_per_graph=max(1, args.steps), replays=max(1, args.warmup))
        print(json.dumps({"case": "decode", "ms": ms, "gb_per_s": decode_bytes(c5) / (ms * 1e-3) / 1e9,
                          "frac_of_hbm_peak": decode_bytes(c5) / (ms * 1e-3) / 1e9 / peaks()["hbm"]}))


def run_all_configs(args):
    """Forward timings of the five named configurations (window sweep and the two control
    modes for config 3, prefill and decode for config 5), one JSON line.  Device-resident
    inputs, CUDA events, each configuration's working set larger than L2 except config 1."""
    from paper_2506_15545_b200 import binding as R
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    sync = torch.cuda.synchronize
    pk = peaks()
    out = {"peaks": pk, "configs": []}

    def roof_ms(wl, fl):
        return 1e3 * max(fl / (pk["tf_burst"] * 1e12), io_bytes_fwd(wl) / (pk["hbm"] * 1e9))

    def time_fwd(wl, mode=R.MODE_RATTN, label=None, steps=20):
        q, k, v = W.make_qkv(wl, dev)
        ws = R.alloc_workspace(q, k, wl.w, mode, 0)
        o = torch.empty_like(q)
        ms = timed(lambda: R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, mode=mode, workspace=ws, out=o),
                   steps, 3, sync)
        assert R.rattn_read_status(ws) == 0
        eff = wl if mode == R.MODE_RATTN else wl.replace(w=wl.T if mode == R.MODE_FULL_CAUSAL else wl.w)
        fl = flops(eff, "fwd") if mode == R.MODE_RATTN else flops(eff, "fwd_main") - 2 * wl.d * wl.d * max(0, eff.T - eff.w - 1) * wl.B * wl.H_q
        rec = {"config": label or wl.name, "B": wl.B, "H_q": wl.H_q, "H_kv": wl.H_kv, "T": wl.T, "w": wl.w,
               "mode": ["rattn", "swa_only", "full_causal"][mode], "ms": ms, "tflops": fl / (ms * 1e-3) / 1e12,
               "tokens_per_s": wl.B * wl.T / (ms * 1e-3), "roofline_ms": roof_ms(wl, fl),
               "roofline_frac": roof_ms(wl, fl) / ms, "tensor_path": bool(R.rattn_uses_tensor_path(wl.d, wl.w, R.RATTN_BF16 if wl.dtype == "bf16" else R.RATTN_F32, mode))}
        out["configs"].append(rec)
        del q, k, v, ws, o
        torch.cuda.empty_cache()

    time_fwd(W.C1, label="c1 (fp32, portable kernels)")
    time_fwd(W.C2)
    for w in W.C3_WINDOWS:
        time_fwd(W.C3.replace(w=w), label=f"c3 w={w}")
    for w in W.C3_WINDOWS:
        time_fwd(W.C3.replace(w=w), mode=R.MODE_SWA_ONLY, label=f"c3 w={w} swa-only")
    time_fwd(W.C3, mode=R.MODE_FULL_CAUSAL, label="c3 full-causal")
    time_fwd(W.C4, label="c4 forward only")
    # the paper's own head shapes (Table 1): 3B = 16 query / 4 K/V heads, 12B = 40 / 8 (groups of 4 and 5)
    time_fwd(W.C2.replace(H_q=16, H_kv=4), label="paper 3B heads 16/4, B=4, T=4096, w=512")
    time_fwd(W.C3.replace(H_q=40, H_kv=8, w=1024), label="paper 12B heads 40/8, B=2, T=8192, w=1024")
    c5 = W.C5.replace(B=args.c5_batch)
    time_fwd(c5, label=f"c5 prefill (B={c5.B} of 32)", steps=3)
    # prefill -> decode hand-off (ring + state out of the prefill's K/V): the library's own
    # per-kernel events around one forward that asks for it
    q, k, v = W.make_qkv(c5, dev)
    ws = R.alloc_workspace(q, k, c5.w, R.MODE_RATTN, 0)
    o = torch.empty_like(q)
    st_o = torch.zeros(c5.B, c5.H_kv, c5.d, c5.d, device=dev)
    kr_o = torch.zeros(c5.B, c5.H_kv, c5.w, c5.d, device=dev, dtype=torch.bfloat16)
    vr_o = torch.zeros_like(kr_o)
    hand = lambda: R.rattn_forward_ex(q, k, v, c5.w, scale=c5.scale, workspace=ws, out=o, state_out=st_o,
                                      k_ring_out=kr_o, v_ring_out=vr_o)
    hand()
    R.rattn_timing_enable(True)
    hand()
    km = R.rattn_timing_read()
    R.rattn_timing_enable(False)
    out["configs"].append({"config": f"c5 prefill + hand-off (B={c5.B}), per kernel",
                           "kernels_ms_per_launch": {n: t / c for n, (c, t) in km.items() if c}})
    del q, k, v, ws, o, st_o, kr_o, vr_o
    torch.cuda.empty_cache()
    ms_d = time_decode_steps(R, W.C5, dev)
    ms_p = time_decode_steps(R, W.C5, dev, flags=R.FLAG_FORCE_GENERIC)
    out["configs"].append({"config": "c5 decode step (B=32)", "ms": ms_d, "gb_per_s": decode_bytes(W.C5) / (ms_d * 1e-3) / 1e9,
                           "roofline_frac": decode_bytes(W.C5) / (ms_d * 1e-3) / 1e9 / pk["hbm"],
                           "tokens_per_s": W.C5.B / (ms_d * 1e-3), "ms_portable_kernel": ms_p,
                           "note": "three rotating cache sets (252 MB), replayed from a CUDA graph"})
    print(json.dumps(out))


def free_port():
    import socket
    with socket.socket() as so:
        so.bind(("127.0.0.1", 0))
        return so.getsockname()[1]


def launch_replicas(argv, n):
    """`bench.py --gpus N` started as a plain process: start the N replica ranks itself (one
    process per GPU under torch.distributed.run on this node) and hand back their exit code.
    Rank 0 of the children prints the JSON line."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__), *argv]
    return subprocess.call(cmd)


def run_replicas_selftest(args):
    """The replica plumbing without a GPU: gloo ranks that pretend to have measured
    10 + 5 * rank milliseconds for 7 units of work each; rank 0 prints the aggregate."""
    import torch.distributed as dist
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
    ms, units = whole_job(10.0 + 5.0 * rank, 7.0, dist if world > 1 else None, "cpu")
    if rank == 0:
        print(json.dumps({"impl": "replicas-selftest", "n_gpus": world, "ms_per_step": ms, "units": units}))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_timeline(args):
    """Where one CTA of the forward kernel spends a work unit: the library is rebuilt with its clock
    stamps compiled in (librattn_tl.so), one forward of the small case (B=2 of config 2; --train for
    the training-mode forward of config 4) is run, and the stamps of CTA 7's two row groups are
    printed as cycles since the unit began.  Stamp ids: 200+i first scores of stream position i
    seen, 300+i row maxima done, 400+i weights handed over, 503 phi(Q) done, 504 phi(K) done,
    501 window accumulator complete, 502 window output parked, 530 residual products complete,
    535 residuals for the backward stored, 540 output stored."""
    import ctypes
    from paper_2506_15545_b200 import binding as R
    from paper_2506_15545_b200 import build as B
    R.LIB_PATH = B.build(timeline=True)
    L = R.lib()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    wl = W.C4 if args.train else W.C2.replace(B=2)
    q, k, v = W.make_qkv(wl, dev)
    ws = R.alloc_workspace(q, k, wl.w, R.MODE_RATTN, R.FLAG_SAVE_RESIDUALS if args.train else 0)
    out = torch.empty_like(q)
    buf = (ctypes.c_ulonglong * 8192)()
    n = (ctypes.c_int * 4)()
    for _ in range(3):
        R.rattn_forward_ex(q, k, v, wl.w, scale=wl.scale, workspace=ws, out=out, save_residuals=args.train)
        torch.cuda.synchronize()
        L.rattn_timeline_read(buf, n)
    units = []
    for role in range(2):
        ev = [(int(buf[role * 2048 + 2 * i]), int(buf[role * 2048 + 2 * i + 1])) for i in range(n[role])]
        start, marks = None, {}
        for e, t in ev:
            if e >= 1000:
                start, marks = t, {"unit": e - 1000}
            elif start is not None:
                marks[e] = t - start
                if e == 540:
                    units.append({"row_group": "AB"[role], **marks})
    print(json.dumps({"case": "timeline", "workload": workload_name(wl), "training_mode": bool(args.train),
                      "units_of_cta_7": units}))


def run_sweep(args):
    """The forward's tuning parameters swept on config 2 and on the paper's own head shapes
    (Table 1: 16 query / 4 K/V heads, 40 / 8), one JSON line per point: stored-state stride m,
    overlap of the chunk-state kernel with the main kernel, unit order.  The chunk size is the
    128-token MMA tile and is not swept.  Device-resident inputs, three rotating input sets."""
    from paper_2506_15545_b200 import binding as R
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    sync = torch.cuda.synchronize
    pk = peaks()
    shapes = [("c2 (B=4, H=16/16, T=4096, w=512)", W.C2),
              ("paper 3B heads 16/4 (B=4, T=4096, w=512)", W.C2.replace(H_q=16, H_kv=4)),
              ("paper 12B heads 40/8 (B=2, T=8192, w=1024)", W.C3.replace(H_q=40, H_kv=8, w=1024))]
    for label, wl in shapes:
        q, k, v = W.make_qkv(wl, dev)
        sets = [(q, k, v)] + [tuple(t.clone() for t in (q, k, v)) for _ in range(2)]
        ws = R.alloc_workspace(q, k, wl.w, R.MODE_RATTN, 0)
        o = torch.empty_like(q)
        it = [0]

        def fwd():
            x = sets[it[0] % 3]
            it[0] += 1
            R.rattn_forward_ex(x[0], x[1], x[2], wl.w, scale=wl.scale, workspace=ws, out=o)

        for m in (1, 2):
            for overlap in (0, 1):
                for order in (1, 2):
                    R.rattn_tune(R.TUNE_STATE_STRIDE, m)
                    R.rattn_tune(R.TUNE_OVERLAP, overlap)
                    R.rattn_tune(R.TUNE_UNIT_ORDER, order)
                    ms = timed(fwd, 40, 5, sync)
                    assert R.rattn_read_status(ws) == 0
                    t_roof = max(flops(wl, "fwd") / (pk["tf_burst"] * 1e12), io_bytes_fwd(wl) / (pk["hbm"] * 1e9)) * 1e3
                    print(json.dumps({"sweep": label, "m": m, "chunk": 128, "overlap": overlap, "unit_order": order,
                                      "ms": round(ms, 4), "tflops": round(flops(wl, "fwd") / (ms * 1e-3) / 1e12, 1),
                                      "roofline_frac": round(t_roof / ms, 4)}), flush=True)
        R.rattn_tune(R.TUNE_STATE_STRIDE, 0)
        R.rattn_tune(R.TUNE_OVERLAP, 1)
        R.rattn_tune(R.TUNE_UNIT_ORDER, 0)
        del sets, q, k, v, ws, o
        torch.cuda.empty_cache()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference", "replicas-selftest"])
    ap.add_argument("--train", action="store_true", help="with --case timeline: the training-mode forward of config 4")
    ap.add_argument("--case", default=None, choices=["fwd", "train", "decode", "timeline", "prologue"],
                    help="run one small case (for profiler captures) instead of the benchmark")
    ap.add_argument("--sweep", action="store_true",
                    help="sweep the forward's tuning parameters (stored-state stride, overlap, unit order)")
    ap.add_argument("--all-configs", action="store_true",
                    help="time the forward of all five named configurations instead of the benchmark")
    ap.add_argument("--c5-batch", type=int, default=32, help="batch entries of config 5's prefill to time")
    ap.add_argument("--clock-seconds", type=float, default=2.0,
                    help="after the K timed steps, repeat the step for about this long under the clock sampler")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and not (args.all_configs or args.case or args.sweep):
        sys.exit(launch_replicas(sys.argv[1:], args.gpus))
    if args.impl == "replicas-selftest":
        run_replicas_selftest(args)
        return
    if args.sweep:
        run_sweep(args)
        return
    if args.all_configs:
        run_all_configs(args)
        return
    if args.case == "timeline":
        run_timeline(args)
        return
    if args.case:
        run_case(args)
        return
    wl = W.C4
    if args.impl == "reference":
        run_reference(args, wl)
    else:
        run_ours(args, wl)


if __name__ == "__main__":
    main()
