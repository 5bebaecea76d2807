#!/usr/bin/env python
"""Benchmark of the SPD block library: decode tokens/s of a stack of TP/SPD decoder blocks
whose T shards are emulated on one B200 (the paper's Sec. 4.1.1 block, masks as Algorithm 1
produces them), with the HBM-roofline fraction of the weight-streaming kernels.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl native|reference]
                  [--workload c2] [--mask config|sync|spd]

One "step" is one decode step of the whole stack (every row of the hot path) for the whole
batch.  Prints ONE JSON line on rank 0.
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

import spd_inputs as si  # noqa: E402

METRIC = "decode tokens/s and HBM-roofline fraction (1 B200), sync vs SPD masks"
GEMM_KINDS = ("gemm_qkv", "gemm_o_proj", "gemm_gate_up", "gemm_down")
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the projection GEMM (average of the four
# launches of a block), from the ncu capture summarised in profiles/dram_decode_kernels_c2.md.  Valid for
# that workload with automatic tuning only; set to None when the kernel changes until it is captured again.
NCU_TRAFFIC_PER_LAUNCH = {"c2": 101.86e6}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), float(d["bf16_tflops"]), "measured"
    return 6650.0, 1590.0, "fallback"


def pick_mask(w: si.Workload, which: str):
    if which == "sync":
        return (1,) * w.n_layers
    if which == "spd":
        return (0,) * w.n_layers
    return tuple(w.mask)


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def replica_plan(w, rank: int, world: int):
    """Replicas only: every rank holds a whole emulated stack (its own seed) and its own batch;
    nothing crosses ranks on the data path.  Returns what rank `rank` runs and what the job counts."""
    return {"seed": rank, "batch": w.batch, "tokens_per_step_job": w.batch * world, "scaling": "weak"}


class ClockSampler:
    """nvidia-smi clocks / throttle reasons while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            time.sleep(0.15)
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self):
        sm = [float(r[1]) for r in self.rows if len(r) >= 9 and r[1].replace(".", "").isdigit()]
        mx = [float(r[2]) for r in self.rows if len(r) >= 9 and r[2].replace(".", "").isdigit()]
        reasons = set()
        for r in self.rows:
            if len(r) < 9:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def decode_bytes(w: si.Workload, B: int, ctx: float):
    """Algorithmic HBM bytes of one decode step: every weight once + the cached K/V of every
    sequence + the new token's K/V."""
    es = 2 if w.dtype == "bf16" else 4
    weights = w.n_layers * w.params_per_layer() * es
    kv = w.n_layers * B * ctx * 2 * w.n_kv_heads * w.head_dim * es
    return weights, kv


def gemm_weight_bytes(w: si.Workload):
    es = 2 if w.dtype == "bf16" else 4
    H, qd, kd, F = w.hidden, w.n_q_heads * w.head_dim, w.n_kv_heads * w.head_dim, w.ffn
    fc1 = (1 if w.block == "opt" else 2) * F * H * es  # fc1 alone, or gate and up
    return {"gemm_qkv": (qd + 2 * kd) * H * es, "gemm_o_proj": H * qd * es, "gemm_gate_up": fc1, "gemm_down": H * F * es}


def prefill_flops(w: si.Workload, B: int, S: int):
    gemm = 2.0 * sum(gemm_weight_bytes(w).values()) / (2 if w.dtype == "bf16" else 4) * B * S
    attn = 2.0 * S * S * w.n_q_heads * w.head_dim * B  # causal: half of 4 S^2 nq d
    return w.n_layers * (gemm + attn)


# ----------------------------------------------------------------------------------------
def run_native(args, rank, world):
    import paper_2502_20727_b200 as spd
    from paper_2502_20727_b200 import build as spd_build
    dev = torch.device(f"cuda:{int(os.environ.get('LOCAL_RANK', 0))}")
    torch.cuda.set_device(dev)
    torch.cuda.set_stream(torch.cuda.Stream(device=dev))  # capturable, unlike the legacy default stream
    if rank == 0:
        spd_build.build()
    if world > 1:
        torch.distributed.barrier()
    w = si.WORKLOADS[args.workload]
    mask = pick_mask(w, args.mask)
    B, S = w.batch, w.prompt
    K, W = args.steps, args.warmup
    max_len = S + W + K + 1
    plan = replica_plan(w, rank, world)
    layers = si.make_stack(w, dev, seed=plan["seed"])
    stack = spd.stack_from_workload(w, layers, sync_mask=mask, max_batch=B, max_seq_len=max_len,
                                    max_prefill_tokens=min(B * S, args.prefill_chunk), device=dev)
    pages_per_seq = (max_len + w.kv_block - 1) // w.kv_block
    bt = si.make_block_table(B, pages_per_seq, stack.n_pages, rank).to(dev)
    if args.tune:
        stack.set_tuning(**{kv.split("=")[0]: int(kv.split("=")[1]) for kv in args.tune.split(",")})

    # ---- prefill (reported, not the headline step) -----------------------------------
    xp = si.make_hidden(w, (B, S, w.hidden), dev, rank, 0)
    outp = torch.empty_like(xp)
    stack.prefill(xp, bt, outp)
    torch.cuda.synchronize()
    pre_ms = []
    for _ in range(args.prefill_reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        stack.prefill(xp, bt, outp)
        e1.record()
        torch.cuda.synchronize()
        pre_ms.append(e0.elapsed_time(e1))
    prefill_ms = float(np.median(pre_ms)) if pre_ms else None
    del xp, outp

    # ---- decode ----------------------------------------------------------------------
    n_total = W + K
    xs = si.make_hidden(w, (n_total, B, w.hidden), dev, rank, 1)
    seq_all = (torch.arange(n_total, dtype=torch.int32, device=dev)[:, None] + S).expand(n_total, B).contiguous()
    out = torch.empty((B, w.hidden), dtype=xs.dtype, device=dev)

    # fixed input buffers, as in a serving loop (the library replays a captured graph while the
    # pointers stay the same); refreshing them each step is part of the timed step
    x_in = torch.empty_like(xs[0])
    seq_in = torch.empty_like(seq_all[0])

    if args.rank_mode:
        # every rank of a T-GPU group executed on this GPU: shard sums as exchanges through global memory
        stack.tp_attach_local()
        out_ranks = torch.empty((w.T, B, w.hidden), dtype=xs.dtype, device=dev)
        out = out_ranks[0]

    def step(t, x_ready=False):
        if not x_ready:
            x_in.copy_(xs[t])
        seq_in.copy_(seq_all[t])
        if args.rank_mode:
            stack.tp_decode_step(x_in, seq_in, bt, S + t + 1, out_ranks)
        else:
            stack.decode_step(x_in, seq_in, bt, S + t + 1, out)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
            torch.cuda.synchronize()

    for t in range(W):
        step(t)
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(dev.index or 0) as clk:
        e0.record()
        for t in range(W, W + K):
            step(t)
        e1.record()
        barrier()
    dev_ms = e0.elapsed_time(e1)
    launches = stack.launches_last_call() * K
    if stack.device_error() != 0:
        raise RuntimeError("device error flag set during the timed region")

    # ---- end to end: host buffers, copies inside the timed region, result read every step
    x_host = xs[W:].cpu().pin_memory()
    out_host = torch.empty((K, B, w.hidden), dtype=xs.dtype).pin_memory()
    for t in range(W):
        step(t)
    barrier()
    t0 = time.perf_counter()
    for i in range(K):
        x_in.copy_(x_host[i], non_blocking=True)
        step(W + i, x_ready=True)
        out_host[i].copy_(out, non_blocking=True)
        torch.cuda.current_stream().synchronize()
    e2e_s = time.perf_counter() - t0
    barrier()

    # ---- per-kernel-kind timing of the same steps (events around every launch) ---------
    for t in range(min(W, 3)):
        step(t)
    torch.cuda.synchronize()
    stack.profile_begin()
    for t in range(W, W + K):
        step(t)
    prof = stack.profile_end()

    dev_ms, e2e_s = max_over_ranks([dev_ms, e2e_s], dev)
    if rank != 0:
        return None

    hbm_peak, tf_peak, peak_kind = measured_peaks()
    mid_ctx = S + W + (K + 1) / 2.0
    wbytes, kvbytes = decode_bytes(w, B, mid_ctx)
    ms_per_step = dev_ms / K
    gw = gemm_weight_bytes(w)
    gemm_ms = sum(prof[k]["ms"] for k in GEMM_KINDS)
    gemm_launches = sum(prof[k]["launches"] for k in GEMM_KINDS)
    gemm_bytes_step = w.n_layers * sum(gw.values())
    gemm_gbs = gemm_bytes_step * K / (gemm_ms * 1e-3) / 1e9 if gemm_ms > 0 else None
    es = xs.element_size()
    res = {
        "metric": METRIC, "value": B * world * K / (dev_ms * 1e-3), "unit": "tokens/s", "n_gpus": world,
        "steps": K, "warmup": W, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": f"{w.name}: {w.n_layers} layers, hidden {w.hidden}, {w.n_q_heads}/{w.n_kv_heads} heads x "
                               f"{w.head_dim}, FFN {w.ffn}, T={w.T}, batch {B}, prompt {S}, decode",
                   "block": w.block, "rank_mode": bool(args.rank_mode), "mask": list(mask), "mask_name": args.mask, "l2": "weights per step exceed L2 (inputs larger than L2)",
                   "context_mid": mid_ctx, "multi_gpu": "replicas only" if world > 1 else "single"},
        "e2e": {"value": B * world * K / e2e_s, "unit": "tokens/s", "h2d_bytes_per_step": B * w.hidden * es,
                "d2h_bytes_per_step": B * w.hidden * es},
        "gpu_launches": launches,
        "clocks": clk.summary(),
        "step_roofline": {"bytes_per_step": wbytes + kvbytes, "achieved_gbs": (wbytes + kvbytes) / (ms_per_step * 1e-3) / 1e9,
                          "frac": (wbytes + kvbytes) / (ms_per_step * 1e-3) / 1e9 / hbm_peak, "peak": hbm_peak,
                          "peak_kind": peak_kind},
        "roofline": {"bound": "hbm", "kernel": "weight-streaming projection GEMM (qkv, o_proj, gate/up, down)",
                     "achieved": gemm_gbs, "peak": hbm_peak, "unit": "GB/s",
                     "frac": (gemm_gbs / hbm_peak) if gemm_gbs else None,
                     "traffic": NCU_TRAFFIC_PER_LAUNCH.get(w.name) if not (args.tune or args.rank_mode) else None,
                     "algorithmic_bytes_per_launch": gemm_bytes_step / max(gemm_launches / K, 1), "peak_kind": peak_kind,
                     "launches_per_step": gemm_launches / K, "avg_launch_us": gemm_ms * 1e3 / max(gemm_launches, 1),
                     "bytes_per_step": gemm_bytes_step},
        "kernel_ms_per_step": {k: v["ms"] / K for k, v in prof.items()},
        "prefill": {"ms": prefill_ms, "tokens": B * S,
                    "tflops": prefill_flops(w, B, S) / (prefill_ms * 1e-3) / 1e12 if prefill_ms else None,
                    "frac_of_bf16_peak": prefill_flops(w, B, S) / (prefill_ms * 1e-3) / 1e12 / tf_peak if prefill_ms else None},
    }
    if world == 1 and not args.no_cpu_baseline:
        res["cpu_baseline"] = cpu_baseline(w, mask, B, S, budget_s=args.cpu_budget)
    return res


# ----------------------------------------------------------------------------------------
def oracle_decode_setup(w, mask, B, ctx0, seed=0):
    import oracle
    layers = si.to_oracle_layers(si.make_stack(w, "cpu", seed))
    if w.block == "opt":  # same call shape for both block kinds
        fwd = oracle.bias_stack_forward
        oracle = type("O", (), {"stack_forward": staticmethod(lambda d, m, l, x, p, c: fwd(d, m, l, x, p, c) + (None,)),
                                "Dims": oracle.Dims, "Cache": oracle.Cache})
    dims = oracle.Dims(w.n_layers, w.hidden, w.n_q_heads, w.n_kv_heads, w.head_dim, w.ffn, w.T, w.rms_eps, w.rope_base)
    cache = oracle.Cache(dims, B, ctx0 + 4096)
    rng = np.random.default_rng(seed)
    cache.k[:, :, :ctx0] = rng.standard_normal(cache.k[:, :, :ctx0].shape)
    cache.v[:, :, :ctx0] = rng.standard_normal(cache.v[:, :, :ctx0].shape)
    return oracle, dims, layers, cache


def cpu_baseline(w, mask, B, S, budget_s=15.0):
    """The oracle, as it stands, on the host cores: whole decode steps of the same workload
    (all layers, whole batch) at the prompt's context, the cache holding seeded stand-in values."""
    oracle, dims, layers, cache = oracle_decode_setup(w, mask, B, S)
    n, t_total = 0, 0.0
    while t_total < budget_s and n < 64:
        x = si.make_hidden(w, (B, 1, w.hidden), "cpu", 0, 1 + n).double().numpy()
        t0 = time.perf_counter()
        oracle.stack_forward(dims, list(mask), layers, x, np.full(B, S + n, np.int32), cache)
        t_total += time.perf_counter() - t0
        n += 1
    return {"value": B * n / t_total, "unit": "tokens/s", "cores": os.cpu_count(), "kind": "oracle",
            "sample": f"{n} whole decode steps (all {w.n_layers} layers, batch {B}) at context {S}+, "
                      f"KV cache pre-filled with seeded values instead of an oracle prefill; {t_total:.1f} s"}


def run_reference(args):
    w = si.WORKLOADS[args.workload]
    mask = pick_mask(w, args.mask)
    B, S, K, W = w.batch, w.prompt, args.steps, args.warmup
    oracle, dims, layers, cache = oracle_decode_setup(w, mask, B, S)
    times = []
    for t in range(W + K):
        x = si.make_hidden(w, (B, 1, w.hidden), "cpu", 0, 1 + t).double().numpy()
        t0 = time.perf_counter()
        oracle.stack_forward(dims, list(mask), layers, x, np.full(B, S + t, np.int32), cache)
        if t >= W:
            times.append(time.perf_counter() - t0)
    total = float(sum(times))
    val = B * K / total
    sample = (f"each step = one whole decode step (all {w.n_layers} layers, batch {B}) at context {S}+t; "
              "KV cache pre-filled with seeded values instead of an oracle prefill")
    return {"impl": "reference", "metric": METRIC, "value": val, "unit": "tokens/s", "n_gpus": args.gpus, "steps": K,
            "warmup": W, "ms_per_step": total / K * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{w.name} (CPU oracle)", "mask": list(mask), "mask_name": args.mask},
            "cpu_baseline": {"value": val, "unit": "tokens/s", "kind": "oracle", "cores": os.cpu_count(), "sample": sample},
            "e2e": {"value": val, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--workload", default="c2", choices=sorted(si.WORKLOADS))
    ap.add_argument("--mask", default="config", choices=["config", "sync", "spd"])
    ap.add_argument("--prefill-chunk", type=int, default=8192)
    ap.add_argument("--prefill-reps", type=int, default=3)
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--rank-mode", action="store_true",
                    help="decode through spd_tp_decode_step: all T ranks of a tensor-parallel group executed on this GPU")
    ap.add_argument("--tune", default="", help="decode tuning knobs, e.g. qkv_splits=4,l2_prefetch_blocks=8 (see spd_set_tuning)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.impl == "reference":
        args.steps = args.steps if args.steps is not None else 16
        args.warmup = args.warmup if args.warmup is not None else 1
        if rank == 0:
            print(json.dumps(run_reference(args)), flush=True)
        return
    args.steps = args.steps if args.steps is not None else 128
    args.warmup = max(args.warmup if args.warmup is not None else 5, 3)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.distributed.init_process_group("nccl", device_id=torch.device(f"cuda:{int(os.environ.get('LOCAL_RANK', 0))}"))
    res = run_native(args, rank, world)
    if rank == 0:
        print(json.dumps(res), flush=True)
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
