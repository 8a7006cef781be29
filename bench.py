#!/usr/bin/env python
"""Benchmark of the GSWA layer: forward + training backward through the C ABI of libgswa.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cM] [--impl reference]

A step is one gswa_forward + gswa_backward over one batch of seeded synthetic input.  One JSON line
is printed by rank 0: whole-job tokens/s with inputs resident in HBM (`value`), the same through the
host-buffer entry point with copies inside the timed region (`e2e`), the roofline fraction of the
dominant kernel, the fp64 CPU checker timed on the host cores (`cpu_baseline`), peak device memory
against an unfused attention-matrix-storing baseline, and the SM clocks seen under load.
`--impl reference` times the CPU checker alone.  With N > 1 (torchrun) every rank runs the same
per-GPU workload on its own GPU (batch items are independent; no collective on the data path).
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

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2409_06206_b200.inputs import CONFIGS, LayerConfig, layer_groups, make_inputs  # noqa: E402

METRIC = "GSWA fwd+bwd tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def flops_per_token(cfg: LayerConfig, backward: bool = True) -> float:
    C, N = cfg.C, cfg.window ** 2
    return (24 * C * C + 12 * N * C) if backward else (8 * C * C + 4 * N * C)


def bytes_per_token(cfg: LayerConfig, backward: bool = True) -> float:
    es = 2 if cfg.dtype == "bf16" else 4
    return (5 if backward else 2) * cfg.C * es       # fwd: x, y; bwd: x, dy, dx


# ------------------------------------------------------------------------------ CPU checker leg
def time_oracle(cfg: LayerConfig, images: int, repeats: int = 1):
    """Times the fp64 CPU checker (as it stands) on `images` batch items of the workload."""
    from oracle import gswa_oracle as orc
    inp = make_inputs(cfg, batch=images)
    gh, gs = layer_groups(cfg, 0)
    args = (inp["w_qkv"], inp["b_qkv"], inp["w_proj"], inp["b_proj"], inp["bias_table"], cfg.window, gh, gs)
    best = None
    for _ in range(repeats):
        t0 = time.perf_counter()
        if cfg.backward:
            orc.forward_backward_chunked(inp["x"], *args, inp["dy"], chunk=2)
        else:
            orc.forward(inp["x"], *args, keep=False)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    tokens = images * cfg.H * cfg.W
    return tokens / best, best, tokens


def oracle_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info()]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def run_reference(args, cfg):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    images = 2
    for _ in range(args.warmup):
        time_oracle(cfg, 1)
    vals = []
    t_all = time.perf_counter()
    for _ in range(args.steps):
        v, dt, tokens = time_oracle(cfg, images)
        vals.append((v, dt))
    wall = time.perf_counter() - t_all
    v = float(np.mean([tokens / dt for _, dt in vals]))
    ms = 1e3 * float(np.mean([dt for _, dt in vals]))
    sample = "%d of %d images of %s per step (%d tokens), numpy float64" % (images, cfg.B, cfg.name, tokens)
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": dict(workload_config(cfg), flags=args.flags),
            "cpu_baseline": {"value": v, "unit": "tokens/s", "cores": oracle_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": v, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "wall_s": wall}
    print(json.dumps(line), flush=True)


def max_over_ranks(value: float) -> float:
    """Largest `value` over all ranks of the default process group (the value itself without one).  Batch items
    are independent, so ranks exchange nothing on the data path; this reduction of the timings is the only
    collective of a multi-GPU run."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([float(value)], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def workload_config(cfg: LayerConfig):
    return {"workload": "%s: x[%d,%d,%d,%d] %s, %d heads (dim %d), groups %s shifts %s, window %d, %s" % (
        cfg.name, cfg.B, cfg.H, cfg.W, cfg.C, cfg.dtype, cfg.num_heads, cfg.head_dim, list(cfg.group_heads),
        list(cfg.group_shift), cfg.window, "fwd+bwd" if cfg.backward else "fwd x%d layers" % cfg.layers),
        "tokens_per_step_per_gpu": cfg.tokens, "l2": "working set larger than L2 (inputs + intermediates)",
        "parallelism": "replicas (batch items independent; no data-path collective)"}


# ------------------------------------------------------------------------------ clocks
class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.rows = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), line.strip()))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, pw = [], [], set(), []
        for t, line in self.rows:
            f = [s.strip() for s in line.split(",")]
            if len(f) < 7 or not (t0 - 0.05 <= t <= t1 + 0.15):
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); pw.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples inside the timed region"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "power_w_max": float(max(pw)), "samples": len(sm)}


# ------------------------------------------------------------------------------ unfused memory baseline
def unfused_peak_bytes(cfg: LayerConfig, dev, batch: int):
    """Peak device memory of a plain torch autograd evaluation of the same layer that materialises the
    rolled / partitioned copies and keeps the [windows, heads, M^2, M^2] attention matrix for backward.
    Measured on `batch` images and reported per image (every term is linear in the batch)."""
    import torch
    M, nh, C, d = cfg.window, cfg.num_heads, cfg.C, cfg.head_dim
    N = M * M
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    x = dev["x"][:batch].clone().requires_grad_(True)
    params = [dev[k].clone().requires_grad_(True) for k in ("w_qkv", "b_qkv", "w_proj", "b_proj", "bias_table")]
    w_qkv, b_qkv, w_proj, b_proj, table = params
    a = torch.arange(N, device="cuda") // M
    c = torch.arange(N, device="cuda") % M
    rel = (a[:, None] - a[None, :] + M - 1) * (2 * M - 1) + (c[:, None] - c[None, :] + M - 1)
    torch.cuda.synchronize()
    torch.cuda.reset_peak_memory_stats()
    base = torch.cuda.memory_allocated()
    B, H, W = batch, cfg.H, cfg.W
    qkv = torch.nn.functional.linear(x, w_qkv, b_qkv)
    outs = []
    h0 = 0
    for gh, s in zip(cfg.group_heads, cfg.group_shift):
        parts = []
        for blk in range(3):
            t = qkv[..., blk * C + h0 * d: blk * C + (h0 + gh) * d]
            if s:
                t = torch.roll(t, shifts=(-s, -s), dims=(1, 2))
            t = t.reshape(B, H // M, M, W // M, M, gh, d).permute(0, 1, 3, 5, 2, 4, 6).reshape(-1, gh, N, d)
            parts.append(t.contiguous())
        q, k, v = parts
        S = (q * d ** -0.5) @ k.transpose(-1, -2) + table[rel][:, :, h0:h0 + gh].permute(2, 0, 1)[None]
        if s:
            r = torch.zeros(H, W, device="cuda")
            for i, sl_i in enumerate((slice(0, H - M), slice(H - M, H - s), slice(H - s, H))):
                for j, sl_j in enumerate((slice(0, W - M), slice(W - M, W - s), slice(W - s, W))):
                    r[sl_i, sl_j] = 3 * i + j
            r = r.reshape(H // M, M, W // M, M).permute(0, 2, 1, 3).reshape(-1, N)
            mask = torch.where(r[:, :, None] == r[:, None, :], 0.0, float("-inf")).to(tdt)
            S = (S.reshape(B, -1, gh, N, N) + mask[None, :, None]).reshape(-1, gh, N, N)
        P = torch.softmax(S.float(), dim=-1).to(tdt)
        O = (P @ v).permute(0, 2, 1, 3).reshape(B, H // M, W // M, M, M, gh * d).permute(0, 1, 3, 2, 4, 5)
        O = O.reshape(B, H, W, gh * d)
        if s:
            O = torch.roll(O, shifts=(s, s), dims=(1, 2))
        outs.append(O)
        h0 += gh
    y = torch.nn.functional.linear(torch.cat(outs, dim=-1), w_proj, b_proj)
    y.backward(dev["dy"][:batch])
    torch.cuda.synchronize()
    peak = torch.cuda.max_memory_allocated() - base
    return int(peak / batch), y.detach()


# ------------------------------------------------------------------------------ our arm
def timed_repeats(args, step, barrier, check_status, gb):
    """Times `--steps` steps, bracketed by a barrier and a device synchronisation on both sides, with CUDA events on
    the launching stream, `--repeats` times over; the reported step time is the median repeat (max over ranks of
    each).  After every repeat the device error word is read: a kernel that gave up a bounded wait returns early,
    which would make the step look faster, so a non-zero word fails the run.
    -> (ms per step, [ms per step of every repeat], launches per repeat, wall-clock start, end)"""
    import torch
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    per_step, launches = [], 0
    t0 = time.perf_counter()
    for _ in range(max(1, args.repeats)):
        barrier()
        n0 = gb.gswa_launch_count()
        e0.record()
        for _ in range(args.steps):
            step()
        e1.record()
        barrier()
        launches = gb.gswa_launch_count() - n0
        check_status()                                   # raises on GSWA_ERR_DEVICE (outside the timed region)
        per_step.append(max_over_ranks(e0.elapsed_time(e1)) / args.steps)
    t1 = time.perf_counter()
    return float(np.median(per_step)), per_step, int(launches), t0, t1


def run_ours(args, cfg):
    import torch
    import torch.distributed as dist
    from paper_2409_06206_b200 import binding as gb
    from paper_2409_06206_b200 import build as gbuild

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        gbuild.build()
    if world > 1:
        dist.barrier()
    gb.lib()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    inp = make_inputs(dataclass_replace(cfg, seed=cfg.seed + 1000 * rank))
    host = {k: torch.from_numpy(v).to(tdt).pin_memory() for k, v in inp.items()}
    torch.cuda.synchronize()
    mem0 = torch.cuda.memory_allocated()
    torch.cuda.reset_peak_memory_stats()
    dev = {k: v.cuda() for k, v in host.items()}
    desc = gb.Desc.from_config(cfg, flags=args.flags)
    saved_b, fwd_b, infer_b, bwd_b = gb.gswa_workspace_query(desc)
    C, M, nh = cfg.C, cfg.window, cfg.num_heads
    y = torch.empty(inp["x"].shape, dtype=tdt, device="cuda")
    dx = torch.empty_like(y)
    saved = torch.empty(max(saved_b, 16), dtype=torch.uint8, device="cuda")
    scratch = torch.empty(max(fwd_b, bwd_b, 16), dtype=torch.uint8, device="cuda")
    grads = {"dw_qkv": torch.empty(3 * C, C, device="cuda"), "db_qkv": torch.empty(3 * C, device="cuda"),
             "dw_proj": torch.empty(C, C, device="cuda"), "db_proj": torch.empty(C, device="cuda"),
             "dbias_table": torch.empty((2 * M - 1) ** 2, nh, device="cuda")}
    fused_bytes = torch.cuda.memory_allocated() - mem0

    def step():
        gb.gswa_forward(desc, dev["x"], dev["w_qkv"], dev["b_qkv"], dev["w_proj"], dev["b_proj"], dev["bias_table"], y,
                        saved, scratch)
        gb.gswa_backward(desc, dev["x"], dev["w_qkv"], dev["b_qkv"], dev["w_proj"], dev["bias_table"], saved,
                         dev["dy"], dx, grads["dw_qkv"], grads["db_qkv"], grads["dw_proj"], grads["db_proj"],
                         grads["dbias_table"], scratch)

    def check_status():
        # the backward call clears the error word its forward call may have set (they share `scratch`), so the
        # forward pass is checked on its own first
        gb.gswa_forward(desc, dev["x"], dev["w_qkv"], dev["b_qkv"], dev["w_proj"], dev["b_proj"], dev["bias_table"], y,
                        saved, scratch)
        gb.gswa_scratch_status(desc, scratch)
        step()
        gb.gswa_scratch_status(desc, scratch)

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    check_status()
    fused_peak = torch.cuda.max_memory_allocated() - mem0
    sampler = ClockSampler(local) if rank == 0 else None
    time.sleep(0.25 if rank == 0 else 0.0)
    ms_step, ms_repeats, launches, t0, t1 = timed_repeats(args, step, barrier, check_status, gb)
    clocks = sampler.stop(t0, t1) if sampler else None
    value = world * cfg.tokens / (ms_step * 1e-3)

    # per-kernel durations (CUDA events on the launching stream, separate pass so the timed region stays clean)
    kernels = per_kernel_times(args, step, gb)

    # end to end through the host-buffer entry point
    hout = {"y": torch.empty(inp["x"].shape, dtype=tdt).pin_memory(), "dx": torch.empty(inp["x"].shape, dtype=tdt).pin_memory()}
    for k, v in grads.items():
        hout[k] = torch.empty(v.shape).pin_memory()
    del saved, scratch
    arena = torch.empty(gb.gswa_step_host_arena_bytes(desc), dtype=torch.uint8, device="cuda")

    def step_host():
        gb.gswa_step_host(desc, host["x"], host["w_qkv"], host["b_qkv"], host["w_proj"], host["b_proj"],
                          host["bias_table"], host["dy"], hout["y"], hout["dx"], hout["dw_qkv"], hout["db_qkv"],
                          hout["dw_proj"], hout["db_proj"], hout["dbias_table"], arena)

    e2e_steps = max(2, min(args.steps, 10))
    for _ in range(2):
        step_host()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        step_host()
    e1.record()
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    e2e_ms = max_over_ranks(e2e_ms)
    e2e_value = world * cfg.tokens / (e2e_ms / e2e_steps * 1e-3)
    es = 2 if cfg.dtype == "bf16" else 4
    nparam = 3 * C * C + 3 * C + C * C + C + (2 * M - 1) ** 2 * nh
    h2d = 2 * cfg.tokens * C * es + nparam * es
    d2h = 2 * cfg.tokens * C * es + nparam * 4
    del arena

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    pk, pk_src = peaks()
    F = flops_per_token(cfg) * cfg.tokens
    Bt = bytes_per_token(cfg) * cfg.tokens
    t_roof = max(F / (pk["bf16_tflops"] * 1e12), Bt / (pk["hbm_gbs"] * 1e9))
    t_roof_sus = max(F / (pk["bf16_tflops_sustained"] * 1e12), Bt / (pk["hbm_gbs"] * 1e9))
    roofline = dominant_roofline(cfg, kernels, pk, pk_src)

    unf = None
    if world == 1 and not args.no_unfused:
        try:
            ub = min(cfg.B, 8)
            per_img, _ = unfused_peak_bytes(cfg, dev, ub)
            unf = {"unfused_bytes_per_image": per_img, "unfused_bytes_at_batch": per_img * cfg.B,
                   "measured_on_images": ub}
        except Exception as ex:  # noqa: BLE001
            unf = {"error": repr(ex)[:200]}
    peak_mem = {"fused_peak_bytes": int(fused_peak), "fused_allocated_bytes": int(fused_bytes),
                "saved_bytes": saved_b, "scratch_bytes": max(fwd_b, bwd_b), "unfused_baseline": unf}

    cpu = None
    if world == 1 and not args.no_cpu:
        images = min(cfg.B, 40)                     # about 10-15 s of CPU work at C = 180
        v, dt, tokens = time_oracle(cfg, images)
        cpu = {"value": v, "unit": "tokens/s", "cores": oracle_threads(), "kind": "oracle",
               "sample": "%d of %d images of %s (%d tokens) in %.1f s, numpy float64 fwd+bwd" % (
                   images, cfg.B, cfg.name, tokens, dt)}

    line = {"metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "repeats": len(ms_repeats),
            "ms_per_step_repeats": [round(v, 5) for v in ms_repeats], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic", "config": dict(workload_config(cfg), flags=args.flags),
            "tflops": F * world / (ms_step * 1e-3) / 1e12,
            "layer_roofline": {"frac_burst": t_roof / (ms_step * 1e-3), "frac_sustained": t_roof_sus / (ms_step * 1e-3),
                               "roofline_us": t_roof * 1e6, "alg_flops": F, "alg_bytes": Bt, "peaks": pk_src},
            "roofline": roofline, "kernels": kernels, "gpu_launches": int(launches),
            "e2e": {"value": e2e_value, "unit": "tokens/s", "h2d_bytes_per_step": int(h2d),
                    "d2h_bytes_per_step": int(d2h), "steps": e2e_steps},
            "peak_mem": peak_mem, "cpu_baseline": cpu, "clocks": clocks}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def per_kernel_times(args, step, gb):
    """Per-kernel durations: CUDA events on the launching stream around every launch, in a separate pass so that
    the timed region stays clean."""
    import torch
    gb.gswa_profile_enable(True)
    for _ in range(args.steps):
        step()
    torch.cuda.synchronize()
    gb.gswa_profile_enable(False)
    per = {}
    for name, t in gb.gswa_profile_read():
        a = per.setdefault(name, [0, 0.0])
        a[0] += 1
        a[1] += t
    total_ms = sum(v[1] for v in per.values())
    return {k: {"launches_per_step": v[0] / args.steps, "ms_per_step": v[1] / args.steps, "share": v[1] / total_ms}
            for k, v in sorted(per.items(), key=lambda kv: -kv[1][1])}


def run_inference(args, cfg):
    """Forward-only workloads: `cfg.layers` stacked layers with alternating group assignment and independent
    weights, activations ping-ponging between two buffers, every call in inference mode (no carry is kept)."""
    import torch
    from paper_2409_06206_b200 import binding as gb
    from paper_2409_06206_b200 import build as gbuild

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        gbuild.build()

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    barrier()
    gb.lib()
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    seeded = dataclass_replace(cfg, seed=cfg.seed + 1000 * rank)
    mem0 = torch.cuda.memory_allocated()
    torch.cuda.reset_peak_memory_stats()
    x0 = torch.from_numpy(make_inputs(seeded, tensors=("x",))["x"]).to(tdt).cuda()
    names = ("w_qkv", "b_qkv", "w_proj", "b_proj", "bias_table")
    params = [{k: torch.from_numpy(v).to(tdt).cuda() for k, v in make_inputs(seeded, layer=l, tensors=names).items()}
              for l in range(cfg.layers)]
    descs = [gb.Desc.from_config(cfg, layer=l, flags=args.flags) for l in range(cfg.layers)]
    infer_b = max(gb.gswa_workspace_query(d)[2] for d in descs)
    scratch = torch.empty(max(infer_b, 16), dtype=torch.uint8, device="cuda")
    bufs = [torch.empty_like(x0), torch.empty_like(x0)]

    def step():
        src = x0
        for l in range(cfg.layers):
            dst = bufs[l & 1]
            p = params[l]
            gb.gswa_forward(descs[l], src, p["w_qkv"], p["b_qkv"], p["w_proj"], p["b_proj"], p["bias_table"], dst, None, scratch)
            src = dst

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()
    gb.gswa_scratch_status(descs[0], scratch)
    peak = torch.cuda.max_memory_allocated() - mem0
    sampler = ClockSampler(local) if rank == 0 else None
    time.sleep(0.25 if rank == 0 else 0.0)
    ms_step, ms_repeats, launches, t0, t1 = timed_repeats(args, step, barrier, lambda: gb.gswa_scratch_status(descs[0], scratch), gb)
    clocks = sampler.stop(t0, t1) if sampler else None
    kernels = per_kernel_times(args, step, gb)
    if rank != 0:
        return
    pk, pk_src = peaks()
    F = flops_per_token(cfg, backward=False) * cfg.tokens * cfg.layers
    Bt = bytes_per_token(cfg, backward=False) * cfg.tokens * cfg.layers
    t_roof = max(F / (pk["bf16_tflops"] * 1e12), Bt / (pk["hbm_gbs"] * 1e9))
    t_roof_sus = max(F / (pk["bf16_tflops_sustained"] * 1e12), Bt / (pk["hbm_gbs"] * 1e9))
    cpu = None
    if world == 1 and not args.no_cpu:
        # one layer of the stack on a 128 x 128 crop-sized draw of the same recipe: about 10 s of CPU work
        small = dataclass_replace(cfg, H=128, W=128)
        v, dt, tokens = time_oracle(small, 1)
        cpu = {"value": v / cfg.layers, "unit": "tokens/s", "cores": oracle_threads(), "kind": "oracle",
               "sample": "one layer on a 128x128 image of the %s recipe (%d tokens) in %.1f s, numpy float64 forward; "
                         "value = that rate / %d layers" % (cfg.name, tokens, dt, cfg.layers)}
    line = {"metric": "GSWA fwd tokens/s through %d stacked layers" % cfg.layers,
            "value": world * cfg.tokens / (ms_step * 1e-3), "unit": "tokens/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "repeats": len(ms_repeats),
            "ms_per_step_repeats": [round(v, 5) for v in ms_repeats], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic", "config": dict(workload_config(cfg), flags=args.flags),
            "token_layers_per_s": world * cfg.tokens * cfg.layers / (ms_step * 1e-3),
            "tflops": F * world / (ms_step * 1e-3) / 1e12,
            "layer_roofline": {"frac_burst": t_roof / (ms_step * 1e-3), "frac_sustained": t_roof_sus / (ms_step * 1e-3),
                               "roofline_us": t_roof * 1e6, "alg_flops": F, "alg_bytes": Bt, "peaks": pk_src},
            "roofline": dominant_roofline(cfg, kernels, pk, pk_src), "kernels": kernels, "gpu_launches": int(launches),
            "e2e": None, "peak_mem": {"fused_peak_bytes": int(peak), "scratch_bytes": infer_b},
            "cpu_baseline": cpu, "clocks": clocks}
    print(json.dumps(line), flush=True)


def dataclass_replace(cfg, **kw):
    import dataclasses
    return dataclasses.replace(cfg, **kw)


# Algorithmic cost of each kernel per token: (flops, bytes) as functions of the layer; un-padded, no
# credit for recomputation or for the padded head dim.  Bytes count every operand the kernel must read
# or write exactly once.
def kernel_cost(cfg: LayerConfig, name: str):
    C, N, nh = cfg.C, cfg.window ** 2, cfg.num_heads
    es = 2 if cfg.dtype == "bf16" else 4
    table = {
        "qkv_gemm": (6 * C * C, (1 + 3) * C * es),                 # read x; write q,k,v
        "attn_fwd": (4 * N * C, (3 + 1) * C * es + 4 * nh),        # read q,k,v; write A and the row log-sum-exp
        "proj_gemm": (2 * C * C, 2 * C * es),                      # read A; write y
        "dattn_gemm": (2 * C * C, 2 * C * es),                     # read dy; write dO = dy W^P
        "dwproj_gemm": (2 * C * C, 2 * C * es),                    # read dy, A; dW^P stays on chip
        "attn_bwd": (8 * N * C, (3 + 1 + 3) * C * es + 4 * nh),    # read q,k,v,dO,L; write dq,dk,dv (no credit for recomputing S)
        "dx_gemm": (6 * C * C, (3 + 1) * C * es),                  # read dqkv; write dx
        "dwqkv_gemm": (6 * C * C, (3 + 1) * C * es),               # read dqkv, x; dW_qkv stays on chip
    }
    alias = {"attn_fwd_generic": "attn_fwd", "attn_bwd_generic": "attn_bwd"}
    return table.get(alias.get(name, name))


# DRAM bytes per token of each kernel: dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture of that
# kernel on workload c3 (131072 tokens; traffic grows in proportion to the tokens) divided by its tokens.
# A kernel is listed only while it is unchanged since its counters were taken (else `traffic` is null).
NCU_DRAM_BYTES_PER_TOKEN = {"attn_bwd": 314.09e6 / 131072}


def dominant_roofline(cfg, kernels, pk, pk_src):
    if not kernels:
        return None
    name = next(iter(kernels))
    k = kernels[name]
    cost = kernel_cost(cfg, name)
    launches = max(k["launches_per_step"], 1e-9)
    dur = k["ms_per_step"] / launches * 1e-3
    per_tok = NCU_DRAM_BYTES_PER_TOKEN.get(name)
    out = {"kernel": name, "launch_us": dur * 1e6, "share_of_step": k["share"], "peak_source": pk_src,
           "traffic": None if per_tok is None else per_tok * cfg.tokens / launches}
    if cost is None:
        out.update({"bound": "hbm", "achieved": None, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": None,
                    "note": "no algorithmic cost model for this kernel"})
        return out
    fl, by = cost
    fl *= cfg.tokens / launches
    by *= cfg.tokens / launches
    t_f, t_b = fl / (pk["bf16_tflops"] * 1e12), by / (pk["hbm_gbs"] * 1e9)
    if t_b >= t_f:
        ach = by / dur / 1e9
        out.update({"bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": ach / pk["hbm_gbs"]})
    else:
        ach = fl / dur / 1e12
        out.update({"bound": "tensor", "achieved": ach, "peak": pk["bf16_tflops"], "unit": "TFLOP/s",
                    "frac": ach / pk["bf16_tflops"]})
    out["alg_bytes_per_launch"] = by
    out["alg_flops_per_launch"] = fl
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--repeats", type=int, default=5, help="the K timed steps are measured this many times; the median is reported")
    ap.add_argument("--workload", default="cM", choices=sorted(CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--flags", type=int, default=0, help="GSWA_FLAG_* bits for the layer descriptor (measured alternatives: "
                    "4 = fused QKV + forward attention, 8 = attention backward on tcgen05)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-checker timing leg")
    ap.add_argument("--no-unfused", action="store_true", help="skip the unfused memory baseline")
    args = ap.parse_args()
    cfg = CONFIGS[args.workload]
    if args.impl == "reference":
        run_reference(args, cfg)
    elif not cfg.backward:
        run_inference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
