#!/usr/bin/env python
"""Benchmark of the attention hot path (forward saving LSE, then backward dQ/dK/dV).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload C3]

One "step" is one pass of the whole hot path over one batch of the workload: forward
(O, LSE), the D pre-pass and the backward kernels.  The metric is the backward's
algorithmic TFLOP/s (10 * kept * d per head: the five products QK^T, dO V^T, P^T dO,
dS^T Q, dS K; recomputation is not counted), timed with CUDA events around the backward
call of every timed step.  Inputs are seeded synthetic N(0,1) tensors rounded to bf16.

With N > 1 (launched under torch.distributed.run) every rank owns its own batch of the
workload -- (batch, head) units are independent, so there is no data-path collective --
and the value is the aggregate over ranks divided by the slowest rank's time.

Prints ONE JSON line on rank 0.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2410_09397_b200 import inputs  # noqa: E402

METRIC = "attention backward TFLOP/s (bf16, n=8192, d=128)"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def kept_entries(w: inputs.Workload, bmask) -> float:
    """Kept score entries per head used for FLOP counting (causal counted as n^2 / 2)."""
    if w.mask == inputs.MASK_NONE:
        return float(w.n) * w.n
    if w.mask == inputs.MASK_CAUSAL:
        return float(w.n) * w.n / 2
    if w.mask == inputs.MASK_BLOCK_SPARSE_CAUSAL:   # blocks below the diagonal whole, kept diagonal blocks as one half
        m = bmask[0].astype(bool)
        return (float(np.tril(m, -1).sum()) + 0.5 * float(np.diag(m).sum())) * w.block * w.block
    return float(bmask[0].sum()) * w.block * w.block


def flops(w: inputs.Workload, bmask, heads: int | None = None):
    bh = w.batch * w.heads if heads is None else heads
    k = kept_entries(w, bmask)
    return 4.0 * k * w.d * bh, 10.0 * k * w.d * bh   # forward, backward


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.perf_counter(), [c.strip() for c in line.split(",")]))

    def stop(self, since: float | None = None, until: float | None = None):
        """Ends the sampling (first call); only samples taken in [since, until] (perf_counter values) are used."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        if self.proc.poll() is None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except subprocess.TimeoutExpired:
                self.proc.kill()
            self.thread.join(timeout=5)
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for t, r in self.rows:
            if len(r) < 6 or (since is not None and t < since) or (until is not None and t > until):
                continue
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for name, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def physical_gpu_index(local: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except (ValueError, IndexError):
            return local
    return local


def max_over_ranks(values, world: int):
    """Element-wise max of a list of floats over all ranks (identity when world == 1)."""
    if world == 1:
        return list(values)
    import torch
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor(values, dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def sum_over_ranks(values, world: int):
    if world == 1:
        return list(values)
    import torch
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor(values, dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return [float(v) for v in t.cpu()]


def cpu_baseline(w: inputs.Workload, bmask, budget_s: float = 15.0):
    """Times the float64 oracle's backward on a bounded sample: whole (batch, head) units."""
    from oracle import oracle as orc
    kind = {inputs.MASK_NONE: orc.MASK_NONE, inputs.MASK_CAUSAL: orc.MASK_CAUSAL,
            inputs.MASK_BLOCK_SPARSE: orc.MASK_BLOCK, inputs.MASK_BLOCK_SPARSE_CAUSAL: orc.MASK_BLOCK_CAUSAL}[w.mask]
    mk = dict(mask_kind=kind, block=w.block, mask_bits=bmask)

    def run(units):
        x = {k: v.astype(np.float64)[None] for k, v in w.tensors(head_slice=(0, units)).items()}
        O, LSE = orc.attn_fwd(x["Q"], x["K"], x["V"], **mk)
        t = time.perf_counter()
        orc.attn_bwd(x["Q"], x["K"], x["V"], O, x["dO"], LSE, **mk)
        return time.perf_counter() - t

    t1 = run(1)
    units = int(max(1, min(w.batch * w.heads, budget_s // max(t1, 1e-3))))
    t = run(units) if units > 1 else t1
    _, fb = flops(w, bmask, heads=units)
    return {"value": fb / t / 1e12, "unit": "TFLOP/s", "cores": orc.threads(), "kind": "oracle",
            "sample": f"backward of {units} of {w.batch * w.heads} (batch, head) units of {w.name} "
                      f"(n={w.n}, d={w.d}), float64, given the oracle's own forward; {t:.2f} s",
            "seconds": t}


def run_reference(args, w, bmask, rank, world):
    """--impl reference: the oracle as it stands on the host cores, a bounded sample per step."""
    if rank != 0:
        return
    from oracle import oracle as orc
    kind = {inputs.MASK_NONE: orc.MASK_NONE, inputs.MASK_CAUSAL: orc.MASK_CAUSAL,
            inputs.MASK_BLOCK_SPARSE: orc.MASK_BLOCK, inputs.MASK_BLOCK_SPARSE_CAUSAL: orc.MASK_BLOCK_CAUSAL}[w.mask]
    mk = dict(mask_kind=kind, block=w.block, mask_bits=bmask)
    x = {k: v.astype(np.float64)[None] for k, v in w.tensors(head_slice=(0, 1)).items()}
    # sample: the leading r rows of one (batch, head) unit.  For the causal workload this
    # is a self-contained sub-problem (rows < r only see keys < r); r is sized so that
    # all steps end within about two minutes.
    r = min(w.n, 1024)
    if inputs.is_block_mask(w.mask):
        r = w.n
    xs = {k: np.ascontiguousarray(v[:, :, :r]) for k, v in x.items()}
    mks = dict(mk)
    if inputs.is_block_mask(w.mask):
        mks["mask_bits"] = bmask
    O, LSE = orc.attn_fwd(xs["Q"], xs["K"], xs["V"], **mks)
    t = time.perf_counter()
    orc.attn_bwd(xs["Q"], xs["K"], xs["V"], O, xs["dO"], LSE, **mks)
    t_probe = time.perf_counter() - t
    total_steps = args.steps + args.warmup
    if not inputs.is_block_mask(w.mask):
        while r * 2 <= w.n and t_probe * 4 * total_steps < 120.0:
            r *= 2
            t_probe *= 4
        xs = {k: np.ascontiguousarray(v[:, :, :r]) for k, v in x.items()}
        O, LSE = orc.attn_fwd(xs["Q"], xs["K"], xs["V"], **mks)
    if w.mask == inputs.MASK_NONE:
        kept = float(r) * r
    elif w.mask == inputs.MASK_CAUSAL:
        kept = float(r) * r / 2
    else:
        kept = kept_entries(w, bmask)
    fb = 10.0 * kept * w.d
    for _ in range(args.warmup):
        orc.attn_bwd(xs["Q"], xs["K"], xs["V"], O, xs["dO"], LSE, **mks)
    t = time.perf_counter()
    for _ in range(args.steps):
        orc.attn_bwd(xs["Q"], xs["K"], xs["V"], O, xs["dO"], LSE, **mks)
    dt = time.perf_counter() - t
    val = fb * args.steps / dt / 1e12
    sample = (f"per step: backward of the leading {r} x {r} sub-problem of one (batch, head) unit of {w.name} "
              f"(n={w.n}, d={w.d}), float64 oracle on the host")
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(w), "sample": sample},
        "cpu_baseline": {"value": val, "unit": "TFLOP/s", "cores": orc.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_name(w):
    mask = {0: "no mask", 1: "causal", 2: f"block-sparse {w.block}x{w.block} p={w.keep_prob}",
            3: f"block-sparse {w.block}x{w.block} p={w.keep_prob} AND causal"}[w.mask]
    return f"{w.name}: batch={w.batch} heads={w.heads} n={w.n} d={w.d} {w.dtype} {mask}"


def weights_leg(attn, torch, w, dev, peaks, phase2=None, steps=20):
    """The memory-bound kernels around the attention proper, timed on their own after the main loop: the
    projection out = A W (S = A1 X, h = A3 Y) and the weight gradient g = A^T G, on tensors of the workload's
    shape with one weight matrix per head.  Returns per-kernel HBM rooflines (algorithmic bytes / event time)."""
    elem = 2 if w.bf16 else 4
    tdtype = torch.bfloat16 if w.bf16 else torch.float32
    W = torch.from_numpy(inputs.normal_tensor(w.seed, 4, (w.heads, w.d, w.d), bf16=False) / np.sqrt(w.d)).to(tdtype).cuda()
    out = torch.empty_like(dev["Q"])
    g = torch.empty((w.heads, w.d, w.d), dtype=torch.float32, device="cuda")
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")

    def step():
        attn.attn_project(dev["Q"], W, out, workspace=ws)
        attn.attn_weight_grad(dev["Q"], dev["dO"], w.heads, g, workspace=ws)

    for _ in range(3):
        step()
    torch.cuda.synchronize()
    attn.attn_timing_enable(True)
    attn.attn_timing_collect()
    ms: dict[str, list[float]] = {}
    for _ in range(steps):
        step()
        for name, t in attn.attn_timing_collect():
            ms.setdefault(name, []).append(t)
    attn.attn_timing_enable(False)
    if attn.attn_workspace_status(ws) != attn.ATTN_OK:
        raise SystemExit("weight kernel reported a device-side error")
    units = w.batch * w.heads
    nbytes = {"wproj": units * w.n * w.d * 2 * elem + w.heads * w.d * w.d * elem,
              "wgrad": units * w.n * w.d * 2 * elem + w.heads * w.d * w.d * 4}
    res = {}
    for name, lst in ms.items():
        key = name.replace("_simt", "")
        if key not in nbytes:
            continue
        avg = sum(lst) / len(lst)
        gbs = nbytes[key] / (avg * 1e-3) / 1e9
        res[name] = {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": gbs / peaks["hbm_gbs"], "avg_launch_ms": avg, "min_launch_ms": min(lst),
                     "bytes_per_launch": nbytes[key], "launches_timed": len(lst), "peak_source": peaks["source"]}
    res["note"] = ("out = A W and g = A^T G on tensors of the workload's shape, one d x d weight per head; "
                   "timed separately from the step above")
    if phase2 is not None:
        # phase 2 of the large-cache algorithm as one call: the attention backward and both weight gradients
        # (gX = A1^T dQ, gY = A3^T dV), with the workload's tensors standing in for A1 = S = Q, A2 = K, A3 = h = V
        O, LSE, mask, cfg, dt_code, bwd_flops = phase2
        gy = torch.empty_like(g)
        wsb = torch.empty(max(256, attn.attn_weights_bwd_workspace_bytes(w.n, w.d, w.heads, w.batch, mask, dt_code, cfg)),
                          dtype=torch.uint8, device="cuda")
        call = lambda: attn.attn_weights_bwd(dev["Q"], dev["K"], dev["V"], dev["Q"], dev["V"], O, dev["dO"], LSE, w.heads,
                                             g, gy, mask=mask, cfg=cfg, workspace=wsb)
        for _ in range(3):
            call()
        ts = []
        for _ in range(max(3, steps // 2)):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); call(); e1.record(); torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        if attn.attn_workspace_status(wsb) != attn.ATTN_OK:
            raise SystemExit("attn_weights_bwd reported a device-side error")
        avg = sum(ts) / len(ts)
        fl = bwd_flops + 2 * 2.0 * units * w.n * w.d * w.d
        # gX reads A1 (2 B) and the fp32 dQ accumulator (4 B) per element where the backward keeps one
        # (bf16, fused, with atomics); otherwise the stored dQ, like gY
        acc = w.bf16 and w.d in (64, 128, 256) and not (cfg and (cfg.deterministic or cfg.algo == attn.ATTN_ALGO_MATERIALIZED))
        gx_bytes = units * w.n * w.d * (elem + 4) + w.heads * w.d * w.d * 4 if acc else nbytes["wgrad"]
        res["weights_bwd"] = {"avg_ms": avg, "min_ms": min(ts), "tflops": fl / (avg * 1e-3) / 1e12, "flops": fl,
                              "hbm_bytes_of_the_two_weight_gradients": gx_bytes + nbytes["wgrad"],
                              "gX_from_fp32_accumulator": bool(acc),
                              "note": "attn_weights_bwd as a whole: attention backward + gX + gY"}
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C3", choices=sorted(inputs.WORKLOADS))
    ap.add_argument("--algo", default="auto", choices=["auto", "fused", "materialized", "simt"])
    ap.add_argument("--tile-q", type=int, default=0)
    ap.add_argument("--tile-k", type=int, default=0)
    ap.add_argument("--tile-d", type=int, default=0)
    ap.add_argument("--deterministic", type=int, default=0)
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (profiling on a smaller case)")
    ap.add_argument("--heads", type=int, default=0, help="override the workload's heads")
    ap.add_argument("--keep-prob", type=float, default=0.0,
                    help="override the off-diagonal keep probability of a block-sparse workload (density sweep)")
    ap.add_argument("--mask-block", type=int, default=0,
                    help="override the block edge of a block-sparse workload (128, 64 or 32; the mask is redrawn at that edge)")
    ap.add_argument("--block-causal", action="store_true",
                    help="block-sparse workload: also drop the entries above the diagonal (block mask AND causal)")
    ap.add_argument("--profile", action="store_true",
                    help="for runs under ncu: allow fewer than 3 warm-up steps, skip e2e and the CPU baseline")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-weights", action="store_true",
                    help="skip the separately timed projection / weight-gradient kernels")
    args = ap.parse_args()
    if args.profile:
        args.no_e2e = args.no_cpu_baseline = args.no_weights = True
    elif args.impl == "ours":
        args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    w = inputs.WORKLOADS[args.workload]
    if args.batch or args.heads:
        w = inputs.Workload(**{**w.__dict__, "batch": args.batch or w.batch, "heads": args.heads or w.heads,
                               "name": w.name + "-reduced"})
    if args.keep_prob and inputs.is_block_mask(w.mask):
        w = inputs.Workload(**{**w.__dict__, "keep_prob": args.keep_prob, "name": w.name + "-density"})
    if (args.mask_block or args.block_causal) and inputs.is_block_mask(w.mask):
        w = inputs.Workload(**{**w.__dict__, "block": args.mask_block or w.block,
                               "mask": inputs.MASK_BLOCK_SPARSE_CAUSAL if args.block_causal else w.mask,
                               "name": w.name + "-variant"})
    bmask = w.block_mask()

    if args.impl == "reference":
        run_reference(args, w, bmask, rank, world)
        return

    import torch
    import torch.distributed as dist
    import paper_2410_09397_b200 as attn

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the attention library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    attn.binding.lib()   # fail loudly here if the library is missing

    algo = {"auto": attn.ATTN_ALGO_AUTO, "fused": attn.ATTN_ALGO_FUSED, "materialized": attn.ATTN_ALGO_MATERIALIZED,
            "simt": attn.ATTN_ALGO_SIMT}[args.algo]
    cfg = attn.Cfg(args.tile_q, args.tile_k, args.tile_d, algo, args.deterministic)
    dt_code = attn.ATTN_BF16 if w.bf16 else attn.ATTN_F32
    tdtype = torch.bfloat16 if w.bf16 else torch.float32

    # every rank draws its own batch: stream seed shifted by the rank (weak scaling)
    wr = inputs.Workload(**{**w.__dict__, "seed": w.seed + 1000 * rank})
    host = {}
    for name, arr in wr.tensors().items():
        t = torch.from_numpy(arr.reshape(w.batch, w.heads, w.n, w.d)).to(tdtype)
        host[name] = t.pin_memory()
    dev = {k: v.cuda(non_blocking=True) for k, v in host.items()}
    mask = None
    if w.mask != inputs.MASK_NONE:
        mask = attn.Mask(kind=w.mask, block=w.block,
                         block_mask=torch.from_numpy(bmask).cuda() if bmask is not None else None)
    O = torch.empty_like(dev["Q"])
    LSE = torch.empty((w.batch, w.heads, w.n), dtype=torch.float32, device="cuda")
    dQ, dK, dV = (torch.empty_like(dev["Q"]) for _ in range(3))
    ws_f = torch.empty(max(256, attn.attn_fwd_workspace_bytes(w.n, w.d, w.heads, w.batch, mask, dt_code, cfg)),
                       dtype=torch.uint8, device="cuda")
    ws_b = torch.empty(max(256, attn.attn_bwd_workspace_bytes(w.n, w.d, w.heads, w.batch, mask, dt_code, cfg)),
                       dtype=torch.uint8, device="cuda")

    def fwd():
        attn.attn_fwd(dev["Q"], dev["K"], dev["V"], O, LSE, mask=mask, cfg=cfg, workspace=ws_f)

    def bwd():
        attn.attn_bwd(dev["Q"], dev["K"], dev["V"], O, dev["dO"], LSE, dQ, dK, dV, mask=mask, cfg=cfg, workspace=ws_b)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(physical_gpu_index(local_rank))
    if rank == 0:
        sampler.start()   # nvidia-smi needs a moment to come up: start it before the warm-up
    for _ in range(args.warmup):
        fwd()
        bwd()
    barrier()
    st = attn.attn_workspace_status(ws_b)
    if st != attn.ATTN_OK:
        raise SystemExit(f"kernel reported: {attn.status_str(st)}")

    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    attn.attn_timing_enable(True)
    attn.attn_timing_collect()
    launches0 = attn.attn_kernel_launches()
    kernel_ms: dict[str, list[float]] = {}
    barrier()
    t_wall = time.perf_counter()
    for s in range(args.steps):
        ev[s][0].record()
        fwd()
        ev[s][1].record()
        bwd()
        ev[s][2].record()
        if (s + 1) % 16 == 0 or s == args.steps - 1:   # the event pool holds 256 launches
            for name, ms in attn.attn_timing_collect():
                kernel_ms.setdefault(name, []).append(ms)
    barrier()
    wall_ms = (time.perf_counter() - t_wall) * 1e3
    launches = attn.attn_kernel_launches() - launches0
    attn.attn_timing_enable(False)
    # nvidia-smi samples every 100 ms.  The clock record is of the samples that fell into the timed region; a region too
    # short to catch one is reported with the samples of the whole run (warm-up included) and says so
    t_end = time.perf_counter()
    clocks = None
    if rank == 0:
        clocks = sampler.stop(since=t_wall, until=t_end)
        clocks["window"] = "timed region"
        if not clocks.get("samples"):
            clocks = sampler.stop()
            clocks["window"] = "whole run, warm-up included (no sample fell into the timed region of %.0f ms)" % wall_ms
            clocks["in_region_samples"] = 0
    fwd_ms = sum(ev[s][0].elapsed_time(ev[s][1]) for s in range(args.steps))
    bwd_ms = sum(ev[s][1].elapsed_time(ev[s][2]) for s in range(args.steps))
    step_ms = sum(ev[s][0].elapsed_time(ev[s][2]) for s in range(args.steps))
    bwd_each = sorted(ev[s][1].elapsed_time(ev[s][2]) for s in range(args.steps))
    fwd_each = sorted(ev[s][0].elapsed_time(ev[s][1]) for s in range(args.steps))
    st = attn.attn_workspace_status(ws_b)
    if st != attn.ATTN_OK or attn.attn_workspace_status(ws_f) != attn.ATTN_OK:
        raise SystemExit("kernel reported a device-side timeout")

    # ---- end to end through the public API with HOST buffers: H2D of Q, K, V, dO, forward,
    # backward, D2H of dQ, dK, dV, every step
    e2e = None
    if not args.no_e2e:
        out_host = [torch.empty_like(host["Q"]).pin_memory() for _ in range(3)]
        e2e_steps = max(3, min(args.steps, 10))

        def e2e_step():
            for k in ("Q", "K", "V", "dO"):
                dev[k].copy_(host[k], non_blocking=True)
            fwd()
            bwd()
            for src, dst in zip((dQ, dK, dV), out_host):
                dst.copy_(src, non_blocking=True)

        def time_e2e(step_fn):
            step_fn()
            barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(e2e_steps):
                step_fn()
            e1.record()
            barrier()
            return e0.elapsed_time(e1) / e2e_steps

        e2e_serial_ms = time_e2e(e2e_step)
        ref_dK = out_host[1].clone()   # dK has a fixed summation order: the pipelined leg must reproduce it bit for bit

        # The same work pipelined: (batch, head) units are independent, so the public API is called on chunks of
        # units, with the host-to-device copies, the kernels and the device-to-host copies of different chunks on
        # three streams (PCIe is full duplex).  Every chunk has a workspace of its own.
        bh = w.batch * w.heads
        n_chunks = next((c for c in (8, 4, 2) if bh % c == 0 and bh // c >= 2), 1)
        cu = bh // n_chunks                      # units per chunk
        flat = lambda t: t.view(bh, *t.shape[2:])
        hin = {k: flat(v) for k, v in host.items()}
        din = {k: flat(v) for k, v in dev.items()}
        dO_, dLSE_ = flat(O), flat(LSE)
        dout = [flat(t) for t in (dQ, dK, dV)]
        hout = [flat(t) for t in out_host]
        sl = lambda t, c: t[c * cu:(c + 1) * cu].unsqueeze(0)     # [1, cu, n, d] view of chunk c
        cws_f = [torch.empty(max(256, attn.attn_fwd_workspace_bytes(w.n, w.d, cu, 1, mask, dt_code, cfg)),
                             dtype=torch.uint8, device="cuda") for _ in range(n_chunks)]
        cws_b = [torch.empty(max(256, attn.attn_bwd_workspace_bytes(w.n, w.d, cu, 1, mask, dt_code, cfg)),
                             dtype=torch.uint8, device="cuda") for _ in range(n_chunks)]
        s_in, s_k, s_out = (torch.cuda.Stream() for _ in range(3))

        def e2e_pipelined():
            main = torch.cuda.current_stream()
            start = torch.cuda.Event()
            start.record(main)
            for st_ in (s_in, s_k, s_out):
                st_.wait_event(start)
            for c in range(n_chunks):
                with torch.cuda.stream(s_in):
                    for k in ("Q", "K", "V", "dO"):
                        din[k][c * cu:(c + 1) * cu].copy_(hin[k][c * cu:(c + 1) * cu], non_blocking=True)
                    ready = torch.cuda.Event()
                    ready.record(s_in)
                with torch.cuda.stream(s_k):
                    s_k.wait_event(ready)
                    attn.attn_fwd(sl(din["Q"], c), sl(din["K"], c), sl(din["V"], c), sl(dO_, c), sl(dLSE_, c), mask=mask,
                                  cfg=cfg, workspace=cws_f[c])
                    attn.attn_bwd(sl(din["Q"], c), sl(din["K"], c), sl(din["V"], c), sl(dO_, c), sl(din["dO"], c),
                                  sl(dLSE_, c), sl(dout[0], c), sl(dout[1], c), sl(dout[2], c), mask=mask, cfg=cfg,
                                  workspace=cws_b[c])
                    done = torch.cuda.Event()
                    done.record(s_k)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(done)
                    for src, dst in zip(dout, hout):
                        dst[c * cu:(c + 1) * cu].copy_(src[c * cu:(c + 1) * cu], non_blocking=True)
            fin = torch.cuda.Event()
            fin.record(s_out)
            main.wait_event(fin)

        e2e_ms = e2e_serial_ms
        e2e_chunks = 1
        if n_chunks > 1:
            e2e_pipe_ms = time_e2e(e2e_pipelined)
            if attn.attn_workspace_status(cws_b[-1]) != attn.ATTN_OK:
                raise SystemExit("kernel reported a device-side timeout (pipelined end-to-end leg)")
            if not torch.equal(ref_dK, out_host[1]):
                raise SystemExit("pipelined end-to-end leg: dK differs from the single-call result")
            if e2e_pipe_ms < e2e_ms:
                e2e_ms, e2e_chunks = e2e_pipe_ms, n_chunks
    ff, fb = flops(w, bmask)
    red = max_over_ranks([fwd_ms, bwd_ms, step_ms, e2e_ms if not args.no_e2e else 0.0,
                          e2e_serial_ms if not args.no_e2e else 0.0], world)
    fwd_ms, bwd_ms, step_ms, e2e_ms, e2e_serial_ms = red
    total = sum_over_ranks([fb, ff, float(launches)], world)
    fb_all, ff_all, launches_all = total
    value = fb_all * args.steps / (bwd_ms * 1e-3) / 1e12
    peaks = load_peaks()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # dominant kernel: the one with the largest total time
    tot = {k: sum(v) for k, v in kernel_ms.items()}
    roofline = None
    if tot:
        top = max(tot, key=tot.get)
        avg_ms = tot[top] / len(kernel_ms[top])
        share = {k: round(v / sum(tot.values()), 4) for k, v in tot.items()}
        # FLOPs one launch of each kernel executes, as a share of the forward (F) / backward (B) algorithmic
        # count: the backward's five products are 0.2 B each; the split kernels recompute S and dP
        own = {"tc_fwd": ("F", 1.0), "simt_fwd": ("F", 1.0), "tc_bwd_fused": ("B", 1.0), "tc_bwd_fused64": ("B", 1.0),
               "tc_bwd_dkdv": ("B", 0.8), "tc_bwd_dq": ("B", 0.6), "simt_bwd_dkdv": ("B", 0.8), "simt_bwd_dq": ("B", 0.6),
               "mat_phase1_P": ("B", 0.2), "mat_phase2_dP": ("B", 0.2), "mat_phase4_dV": ("B", 0.2),
               "mat_phase4_dK": ("B", 0.2), "mat_phase4_dQ": ("B", 0.2)}
        which, share_ = own.get(top, ("B", 1.0))
        alg = (ff if which == "F" else fb) * share_
        note = ("algorithmic FLOPs of the five backward products" if top in ("tc_bwd_fused", "tc_bwd_fused64") else
                f"this kernel's own products: {share_:g} x the {'forward' if which == 'F' else 'backward'} count")
        ach = alg / (avg_ms * 1e-3) / 1e12
        # the denominator that matches the run: the burst peak (a GEMM timed alone at full clock) when the timed
        # region is shorter than a second and the sampled SM clock stayed within 3 % of its maximum, else the
        # sustained peak (a seconds-long GEMM loop under the power cap)
        sm, smx = (clocks or {}).get("sm_mhz"), (clocks or {}).get("sm_max_mhz")
        # a sub-second region without a sample of its own is taken as a burst, the stricter denominator
        in_region = (clocks or {}).get("in_region_samples", 1) != 0
        burst = wall_ms < 1000.0 and (not in_region or sm is None or (smx and sm >= 0.97 * smx))
        pk = peaks["bf16_tflops"] if burst else peaks["bf16_tflops_sustained"]
        roofline = {"bound": "tensor", "kernel": top, "achieved": ach, "peak": pk,
                    "unit": "TFLOP/s", "frac": ach / pk, "peak_kind": "burst" if burst else "sustained",
                    "frac_of_burst_peak": ach / peaks["bf16_tflops"],
                    "frac_of_sustained_peak": ach / peaks["bf16_tflops_sustained"],
                    "peak_source": peaks["source"] + (" burst" if burst else " sustained"),
                    "avg_launch_ms": avg_ms, "launches_timed": len(kernel_ms[top]), "flops_per_launch": alg,
                    "flops_note": note, "traffic": traffic_of(top, w.name), "kernel_time_share": share}
    # the memory-bound step of the path (D pre-pass) against the measured copy bandwidth
    roofline_hbm = None
    for name in ("tc_bwd_preprocess", "mat_preprocess", "bwd_preprocess_D"):
        if name in kernel_ms:
            elem = 2 if w.bf16 else 4
            rows = w.batch * w.heads * w.n
            by = rows * (2 * w.d * elem + (12 if name != "bwd_preprocess_D" else 4))
            if name == "tc_bwd_preprocess" and "tc_bwd_fused" in kernel_ms:
                by += rows * w.d * 4   # the same pass clears the fp32 dQ accumulator of the fused backward
            avg = sum(kernel_ms[name]) / len(kernel_ms[name])
            gbs = by / (avg * 1e-3) / 1e9
            roofline_hbm = {"bound": "hbm", "kernel": name, "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                            "frac": gbs / peaks["hbm_gbs"], "avg_launch_ms": avg, "bytes_per_launch": by,
                            "peak_source": peaks["source"]}
            break
    # the paper's I/O bound (Theorem 1.1 / 1.2, constant 1, elements -> bytes) at this configuration's on-chip size
    elem = 2 if w.bf16 else 4
    M = attn.attn_cfg_onchip_elems(w.d, dt_code, cfg, True)
    if inputs.is_block_mask(w.mask):
        bound_el = attn.attn_io_bound_sparse_elems(w.n * w.d, kept_entries(w, bmask), M) if M else None
    else:
        bound_el = attn.attn_io_bound_elems(w.n, w.d, M, True) * (0.5 if w.mask == inputs.MASK_CAUSAL else 1.0) if M else None
    comp = (8 * w.n * w.d * elem + 2 * 4 * w.n) * w.batch * w.heads
    io = {"backward_compulsory_bytes": comp, "onchip_elems_M": M,
          # Theorem 1.2: Z_input^2 / Z_QK is the cache size at which the two terms of the sparse bound meet
          "sparse_dividing_M": (float(w.n * w.d) ** 2 / kept_entries(w, bmask)) if inputs.is_block_mask(w.mask) else None,
          "kept_entries_per_head": kept_entries(w, bmask),
          "paper_bound_bytes_at_M": bound_el * elem * w.batch * w.heads if bound_el else None,
          "dram_bytes_from_profile_dominant_kernel": traffic_of(max(tot, key=tot.get), w.name) if tot else None}
    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": step_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if w.bf16 else "f32", "data": "synthetic",
        "config": {"workload": workload_name(w), "algo": args.algo, "tile_q": args.tile_q, "tile_k": args.tile_k,
                   "tile_d": args.tile_d, "deterministic": args.deterministic,
                   "step": "forward (O, LSE) + backward (D, dQ, dK, dV); value counts the backward only",
                   "l2": "inputs (5 x %d MiB) larger than L2; no flush" % (w.batch * w.heads * w.n * w.d * 2 >> 20),
                   "per_rank_batch": w.batch},
        "fwd_tflops": ff_all * args.steps / (fwd_ms * 1e-3) / 1e12,
        "fwd_ms": fwd_ms / args.steps, "bwd_ms": bwd_ms / args.steps, "wall_ms_per_step": wall_ms / args.steps,
        "bwd_ms_median": bwd_each[len(bwd_each) // 2], "bwd_ms_min": bwd_each[0],
        "fwd_ms_median": fwd_each[len(fwd_each) // 2], "fwd_ms_min": fwd_each[0],
        "frac_of_sustained_peak": value / world / peaks["bf16_tflops_sustained"],
        "frac_of_burst_peak": value / world / peaks["bf16_tflops"],
        "clocks": clocks, "gpu_launches": int(launches_all),
        "roofline": roofline, "roofline_hbm": roofline_hbm, "io": io,
    }
    if not args.no_e2e:
        elem = 2 if w.bf16 else 4
        per = w.batch * w.heads * w.n * w.d * elem
        line["e2e"] = {"value": fb_all / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s",
                       "h2d_bytes_per_step": 4 * per, "d2h_bytes_per_step": 3 * per, "ms_per_step": e2e_ms,
                       "serial_ms_per_step": e2e_serial_ms, "calls_per_step": e2e_chunks,
                       "note": "backward FLOPs / (H2D of Q,K,V,dO + forward + backward + D2H of dQ,dK,dV); "
                               "calls_per_step > 1: the API is called on that many chunks of (batch, head) units, "
                               "copies and kernels on three streams; serial_ms_per_step: one call, one stream"}
    if world == 1 and not args.no_weights:
        line["weights"] = weights_leg(attn, torch, w, dev, peaks, phase2=(O, LSE, mask, cfg, dt_code, fb))
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = cpu_baseline(w, bmask)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of a kernel on a workload, taken from
# one ncu capture of a reduced case (fewer heads, same n and d) and scaled by the number of heads (heads are
# independent, the traffic grows in proportion).  Every entry names the source file of the kernel and the
# SHA-1 that file had when the counters were taken: once the file has changed the entry is stale and the
# bench reports null instead.
TRAFFIC: dict = {
    ("tc_bwd_fused", "C3"): {"bytes": 5.916e+08, "src": "attn_tc_bwd.cu", "sha1": "1b0a4a390dd829f7fafd8c47cd68eea024361713",
                 "note": "16 of 32 heads captured, x 2"},
    ("tc_fwd", "C3"): {"bytes": 2.362e+08, "src": "attn_tc_fwd.cu", "sha1": "d8be6effe28394a321c2d3d45e60bf375c4da969",
                 "note": "16 of 32 heads captured, x 2"},
    ("tc_bwd_fused64", "C3"): {"bytes": 5.862e+08, "src": "attn_tc_bwd64.cu", "sha1": "a71a96f8af4e8f387830d7fc92c83e7e4968337e",
                 "note": "16 of 32 heads captured, x 2"},
    ("tc_bwd_dkdv", "C3"): {"bytes": 3.385e+08, "src": "attn_tc_bwd.cu", "sha1": "1b0a4a390dd829f7fafd8c47cd68eea024361713",
                 "note": "16 of 32 heads captured, x 2"},
    ("tc_bwd_fused64", "C4"): {"bytes": 1.038e+08, "src": "attn_tc_bwd64.cu", "sha1": "a71a96f8af4e8f387830d7fc92c83e7e4968337e",
                 "note": "4 of 8 heads captured, x 2; the inputs of either case fit in L2"},
    ("tc_fwd", "C4"): {"bytes": 5.04e+07, "src": "attn_tc_fwd.cu", "sha1": "d8be6effe28394a321c2d3d45e60bf375c4da969",
                 "note": "4 of 8 heads captured, x 2; the inputs of either case fit in L2"},
    ("tc_bwd_fused", "C2"): {"bytes": 1.250e+08, "src": "attn_tc_bwd.cu", "sha1": "1b0a4a390dd829f7fafd8c47cd68eea024361713",
                 "note": "the whole workload captured"},
    ("tc_bwd_fused", "C5"): {"bytes": 3.249e+09, "src": "attn_tc_bwd.cu", "sha1": "1b0a4a390dd829f7fafd8c47cd68eea024361713",
                 "note": "8 of 32 heads captured, x 4"},
}


def traffic_of(kernel: str, workload: str):
    import hashlib
    ent = TRAFFIC.get((kernel, workload))
    if ent is None:
        return None
    path = os.path.join(ROOT, "paper_2410_09397_b200", "csrc", ent["src"])
    try:
        with open(path, "rb") as f:
            sha = hashlib.sha1(f.read()).hexdigest()
    except OSError:
        return None
    return ent["bytes"] if sha == ent["sha1"] else None


if __name__ == "__main__":
    main()
