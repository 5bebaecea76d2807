#!/usr/bin/env python
"""Benchmark of the SPD block library: decode tokens/s of a stack of TP/SPD decoder blocks
whose T shards are emulated on one B200 (the paper's Sec. 4.1.1 block, masks as Algorithm 1
produces them), with the HBM-roofline fraction of the weight-streaming kernels, for the
synchronous mask and the SPD masks.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl native|reference]
                  [--workload c5] [--mask config|sync|spd] [--configs all|none|c2,c4_b1,...]

One "step" is one decode step of the whole stack (every row of the hot path) for the whole
batch.  The headline is the largest listed configuration (c5: 40 blocks of the 70B shape, batch
64, its seeded 25 %-sync mask); `per_config` carries every listed configuration with the
synchronous mask, the all-SPD mask and - where it is a mix - its own mask: decode step time,
tokens/s, HBM-roofline fraction, and the prompt phase with its tensor-core fraction.
Prints ONE JSON line on rank 0.  With --gpus N and no launcher around it, starts the N ranks itself.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import socket
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
PER_CONFIG = ("c2", "c3_t4", "c3_t8", "c4_b1", "c4_b32", "c5")
DECODE_GEMM_SOURCE = os.path.join(ROOT, "paper_2502_20727_b200", "csrc", "gemm_decode.cu")
TRAFFIC_NOTE = os.path.join(ROOT, "profiles", "dram_decode_gemm.md")


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), float(d["bf16_tflops"]), "measured"
    return 6650.0, 1590.0, "fallback"


def masks_of(w: si.Workload):
    """The masks a configuration is run with: synchronous, all-SPD, and its own where that is a mix."""
    out = {"sync": (1,) * w.n_layers, "spd": (0,) * w.n_layers}
    if 0 < sum(w.mask) < w.n_layers:
        out["config"] = tuple(w.mask)
    return out


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


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(n: int, cmd, env=None, timeout=None):
    """Start `cmd` n times as ranks 0..n-1 of one local job (RANK / LOCAL_RANK / WORLD_SIZE / MASTER_* set as a
    launcher would), wait for all, return the largest exit code.  Output goes where the parent's goes."""
    base = dict(os.environ if env is None else env)
    base.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(free_port()), WORLD_SIZE=str(n), LOCAL_WORLD_SIZE=str(n))
    procs = [subprocess.Popen(cmd, env=dict(base, RANK=str(r), LOCAL_RANK=str(r))) for r in range(n)]
    rcs = []
    deadline = None if timeout is None else time.time() + timeout
    for p in procs:
        try:
            rcs.append(p.wait(timeout=None if deadline is None else max(1.0, deadline - time.time())))
        except subprocess.TimeoutExpired:
            p.kill()
            rcs.append(124)
    return max(abs(rc) for rc in rcs)


class ClockSampler:
    """SM clock, power and throttle reasons of one GPU, sampled every few milliseconds by a thread for as long as
    the benchmark runs (NVML queries only: nothing is set).  window(t0, t1) summarises the samples of a timed region."""
    REASONS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20), ("sw_power_cap", 0x4))

    def __init__(self, index: int, period_s: float = 0.004):
        self.index, self.period, self.rows, self.stop_flag, self.thread, self.h = index, period_s, [], False, None, None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(self._physical_index(index))
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.h = None

    @staticmethod
    def _physical_index(index):
        vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
        ids = [v for v in vis.split(",") if v.strip() != ""]
        if ids and all(v.strip().isdigit() for v in ids) and index < len(ids):
            return int(ids[index])
        return index

    def __enter__(self):
        if self.h is not None:
            self.thread = threading.Thread(target=self._run, daemon=True)
            self.thread.start()
        return self

    def _run(self):
        nv = self.nv
        while not self.stop_flag:
            try:
                mhz = float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                reasons = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)) if hasattr(nv, "nvmlDeviceGetCurrentClocksEventReasons") \
                    else int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                watts = nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0
                self.rows.append((time.perf_counter(), mhz, reasons, watts))
            except Exception:
                pass
            time.sleep(self.period)

    def __exit__(self, *a):
        self.stop_flag = True
        if self.thread:
            self.thread.join(timeout=2)

    def window(self, t0=None, t1=None):
        rows = [r for r in self.rows if (t0 is None or r[0] >= t0) and (t1 is None or r[0] <= t1)]
        if not rows and self.rows and t0 is not None:  # region shorter than the sampling period: the nearest sample
            rows = [min(self.rows, key=lambda r: abs(r[0] - 0.5 * (t0 + t1)))]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": getattr(self, "max_mhz", None), "reasons": [], "samples": 0}
        bits = 0
        for r in rows:
            bits |= r[2]
        return {"sm_mhz": float(np.median([r[1] for r in rows])), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(n for n, b in self.REASONS if bits & b), "samples": len(rows),
                "power_w_max": max(r[3] for r in rows)}


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


def captured_traffic(w: si.Workload):
    """DRAM bytes per launch of the decode projection GEMM from the committed ncu summary - valid only for the shape
    it was captured at and while the kernel source is the one that was captured (its hash is kept beside the figure)."""
    try:
        text = open(TRAFFIC_NOTE).read()
        sha = hashlib.sha256(open(DECODE_GEMM_SOURCE, "rb").read()).hexdigest()[:16]
    except OSError:
        return None
    for m in re.finditer(r"bench_traffic:\s*shape=(\S+)\s+bytes_per_launch=([0-9.eE+]+)\s+source_sha=(\w+)", text):
        shape = f"{w.hidden}x{w.n_q_heads}x{w.n_kv_heads}x{w.ffn}xT{w.T}xB{w.batch}"
        if m.group(1) == shape and m.group(3) == sha:
            return float(m.group(2))
    return None


# ----------------------------------------------------------------------------------------
class Run:
    """One configuration resident on the device: weights, stack, block tables."""

    def __init__(self, w: si.Workload, dev, seed: int, K: int, W: int, args, spd):
        self.w, self.dev, self.K, self.W, self.args = w, dev, K, W, args
        self.Bd = w.batch
        self.Bp, self.Sp = (w.prefill_batch or w.batch), (w.prefill_len or w.prompt)
        # the timed decode steps sit in the middle of the configuration's decode run
        self.ctx0 = w.prompt + max(0, (w.decode_steps - (W + K)) // 2)
        steps_room = 3 * (W + K) + 33  # timed, end-to-end and timeline passes advance no further than this
        self.max_len = max(self.Sp, self.ctx0 + steps_room)
        pages_d = (self.ctx0 + steps_room + w.kv_block - 1) // w.kv_block
        pages_p = (self.Sp + w.kv_block - 1) // w.kv_block
        n_pages = max(self.Bd * pages_d, self.Bp * pages_p)
        self.layers = si.make_stack(w, dev, seed=seed)
        self.stack = spd.stack_from_workload(w, self.layers, sync_mask=(0,) * w.n_layers, max_batch=max(self.Bd, self.Bp),
                                             max_seq_len=self.max_len, n_pages=n_pages,
                                             max_prefill_tokens=min(max(self.Bp * self.Sp, self.Bd), args.prefill_chunk), device=dev)
        self.bt_d = si.make_block_table(self.Bd, pages_d, n_pages, seed).to(dev)
        self.bt_p = si.make_block_table(self.Bp, pages_p, n_pages, seed + 1).to(dev)
        if args.tune:
            self.stack.set_tuning(**{kv.split("=")[0]: int(kv.split("=")[1]) for kv in args.tune.split(",")})
        n_total = steps_room - 1
        self.xs = si.make_hidden(w, (W + K, self.Bd, w.hidden), dev, seed, 1)
        self.x_in = torch.empty_like(self.xs[0])
        self.seq_in = torch.empty(self.Bd, dtype=torch.int32, device=dev)
        self.seq_all = (torch.arange(n_total, dtype=torch.int32, device=dev)[:, None] + self.ctx0).expand(n_total, self.Bd).contiguous()
        self.out = torch.empty((self.Bd, w.hidden), dtype=self.xs.dtype, device=dev)
        self.rank_mode = bool(args.rank_mode)
        if self.rank_mode:
            self.stack.tp_attach_local()
            self.out_ranks = torch.empty((w.T, self.Bd, w.hidden), dtype=self.xs.dtype, device=dev)
            self.out = self.out_ranks[0]
        self.filled = False

    def close(self):
        self.stack.close()
        self.layers = self.stack = self.xs = None
        torch.cuda.empty_cache()

    # one decode step; t counts steps since ctx0 (contexts grow by one token per step, as in a decode run)
    def step(self, t, x_ready=False):
        if not x_ready:
            self.x_in.copy_(self.xs[t % (self.W + self.K)])
        self.seq_in.copy_(self.seq_all[t])
        if self.rank_mode:
            self.stack.tp_decode_step(self.x_in, self.seq_in, self.bt_d, self.ctx0 + t + 1, self.out_ranks)
        else:
            self.stack.decode_step(self.x_in, self.seq_in, self.bt_d, self.ctx0 + t + 1, self.out)

    def prefill_ms(self, reps):
        """The configuration's prompt phase (Bp prompts of Sp tokens), median of `reps` after one warm-up."""
        w = self.w
        xp = si.make_hidden(w, (self.Bp, self.Sp, w.hidden), self.dev, 0, 0)
        if self.rank_mode:  # every rank's copy of the output; prompts through the two-shot exchanges
            outp = torch.empty((w.T,) + tuple(xp.shape), dtype=xp.dtype, device=self.dev)
            prefill = self.stack.tp_prefill
        else:
            outp = torch.empty_like(xp)
            prefill = self.stack.prefill
        prefill(xp, self.bt_p, outp)
        torch.cuda.synchronize()
        ms = []
        for _ in range(reps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            prefill(xp, self.bt_p, outp)
            e1.record()
            torch.cuda.synchronize()
            ms.append(e0.elapsed_time(e1))
        self.filled = False  # the prompt pages may overlap the decode rows
        return float(np.median(ms)) if ms else None

    def fill_cache(self):
        """K/V of ctx0 tokens for every sequence of the decode batch (untimed): a prefill of seeded hidden states."""
        if self.filled:
            return
        w = self.w
        per = max(1, min(self.Bd, (1 << 16) // self.ctx0))  # bounded host-side tensor
        for b0 in range(0, self.Bd, per):
            nb = min(per, self.Bd - b0)
            x = si.make_hidden(w, (nb, self.ctx0, w.hidden), self.dev, 1, 100 + b0)
            self.stack.prefill(x, self.bt_d[b0:b0 + nb].contiguous(), torch.empty_like(x))
        torch.cuda.synchronize()
        self.filled = True

    def settle(self, seconds):
        """Untimed decode steps at the starting context until the GPU has been under THIS load for `seconds`: the prompt
        phase before it runs the chip into its power cap, and the clocks need a moment to find the decode level."""
        t0 = time.perf_counter()
        while time.perf_counter() - t0 < seconds:
            for _ in range(self.W):
                self.step(0)
            torch.cuda.synchronize()

    def decode_ms(self, barrier, base=0, stamped=False):
        """Settling, W warm-up steps, then K timed steps between two events: (ms, host window).  stamped: the kernels
        record their start / end and a fold kernel ends every step (see SpdStack.timeline_begin), so that the region
        that gives the step time also gives every kernel's share of it."""
        if stamped:
            self.stack.timeline_begin()
        self.settle(self.args.settle_s)
        for t in range(self.W):
            self.step(base + t)
        barrier()
        if stamped:
            self.stack.timeline_begin()  # clear the totals of the settling and warm-up steps
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0 = time.perf_counter()
        e0.record()
        for t in range(self.W, self.W + self.K):
            self.step(base + t)
        e1.record()
        barrier()
        h1 = time.perf_counter()
        if self.stack.device_error() != 0:
            raise RuntimeError("device error flag set during the timed region")
        return e0.elapsed_time(e1), (h0, h1)

    def timeline_totals(self):
        """Every launch's own share of a step (ms), the steps' mean span and the launches per kind, from the stamps of
        the K steps of the last decode_ms(stamped=True); ends the stamping."""
        per_launch, span_ns, calls = self.stack.timeline_read()
        self.stack.timeline_end()
        if calls != self.K:
            raise RuntimeError(f"timeline folded {calls} calls, expected {self.K}")
        own_ms, launches = {}, {}
        for kind, ns in per_launch:
            own_ms[kind] = own_ms.get(kind, 0.0) + ns / calls * 1e-6
            launches[kind] = launches.get(kind, 0) + 1
        return own_ms, span_ns / calls * 1e-6, launches

def run_tp(args, rank, world):
    """ONE model over the ranks of the job (Sec. 3: shard r on GPU r), decode steps only: --tp fused runs the rank mode
    (shard sums exchanged inside the projection tails over peer-mapped memory), --tp baseline the same shards with
    an NCCL all-reduce between kernels at every sync-point the mask keeps.  The workload's T becomes the world size.
    Strong scaling: the batch is the workload's, whatever the number of ranks."""
    import paper_2502_20727_b200 as spd
    from paper_2502_20727_b200 import build as spd_build
    import torch.distributed as dist
    dev = torch.device(f"cuda:{int(os.environ.get('LOCAL_RANK', 0))}")
    torch.cuda.set_device(dev)
    torch.cuda.set_stream(torch.cuda.Stream(device=dev))
    if rank == 0:
        spd_build.build()
    dist.barrier()
    T, K, W = world, args.steps, args.warmup
    w0 = si.WORKLOADS[args.workload]
    if args.layers:
        w0 = w0.with_(n_layers=args.layers, mask=tuple(w0.mask[:args.layers]))
    w = w0.with_(T=T)
    mask = pick_mask(w, args.mask)
    B, ctx0 = w.batch, w.prompt + max(0, (w.decode_steps - (W + K)) // 2)
    one = w.with_(n_q_heads=w.n_q_heads // T, n_kv_heads=w.n_kv_heads // T, ffn=w.ffn // T, T=1)
    shard = []
    for l in range(w.n_layers):  # every rank draws the same layer (same seed) and keeps its own rows / columns
        shard.append(spd.shard_layer(si.make_layer(w, l, dev, 0), rank, T))
    max_len = ctx0 + W + K + 2
    pages = (max_len + w.kv_block - 1) // w.kv_block
    stack = spd.stack_from_workload(one, shard, sync_mask=mask, max_batch=B, max_seq_len=max_len, n_pages=B * pages,
                                    max_prefill_tokens=min(B * ctx0, args.prefill_chunk), device=dev)
    bt = si.make_block_table(B, pages, B * pages, 0).to(dev)
    xs = si.make_hidden(w, (W + K, B, w.hidden), dev, 0, 1)
    x_in, seq_in = torch.empty_like(xs[0]), torch.empty(B, dtype=torch.int32, device=dev)
    collective = spd.CollectiveAllReduce()
    if args.tp == "fused":
        if T > 1:
            stack.tp_attach_symmetric(rank, T)
        else:
            stack.tp_attach(1, 0, [_one_region(stack, dev)], stack.tp_region_bytes(1))
        out = torch.empty((1, B, w.hidden), dtype=xs.dtype, device=dev)
    else:
        out = torch.empty((B, w.hidden), dtype=xs.dtype, device=dev)

    def step(t):
        x_in.copy_(xs[t])
        seq_in.fill_(ctx0 + t)
        if args.tp == "fused":
            stack.tp_decode_step(x_in, seq_in, bt, ctx0 + t + 1, out)
        else:
            stack.tp_baseline_decode_step(x_in, seq_in, bt, ctx0 + t + 1, collective, out)

    def barrier():
        torch.cuda.synchronize()
        dist.barrier()
        torch.cuda.synchronize()

    with ClockSampler(dev.index or 0) as clk:
        for t in range(W):
            step(t)
        barrier()
        calls0 = collective.calls
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        h0 = time.perf_counter()
        e0.record()
        for t in range(W, W + K):
            step(t)
        e1.record()
        barrier()
        h1 = time.perf_counter()
        if stack.device_error() != 0:
            raise RuntimeError("device error flag set during the timed region")
        dev_ms, = max_over_ranks([e0.elapsed_time(e1)], dev)
        clocks = clk.window(h0, h1)
    if rank != 0:
        return None
    hbm_peak, _, peak_kind = measured_peaks()
    mid_ctx = ctx0 + W + (K + 1) / 2.0
    wbytes, kvbytes = decode_bytes(w, B, mid_ctx)
    per_rank = (wbytes + kvbytes) / T  # every rank streams its own shard of the weights and of the K/V
    sync_points = sum(2 if m else 1 for m in mask)
    return {"metric": METRIC, "value": B * K / (dev_ms * 1e-3), "unit": "tokens/s", "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": dev_ms / K, "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": w.dtype,
            "data": "synthetic",
            "config": {"workload": f"{w.name}: {w.n_layers} layers over {T} ranks (one shard per GPU), batch {B}, context {ctx0}+",
                       "rank_mode": "fused exchange in the projection tails" if args.tp == "fused" else "NCCL all-reduce between kernels",
                       "mask": list(mask), "mask_name": args.mask, "sync_points_per_step": sync_points,
                       "all_reduce_calls_per_step": (collective.calls - calls0) / K if args.tp == "baseline" else None,
                       "exchange_bytes_per_rank_per_step": sync_points * B * w.hidden * 4 * (T - 1),
                       "l2": "weights per step exceed L2 (inputs larger than L2)" if wbytes / T > 126e6 else "rank's shard fits L2",
                       "multi_gpu": "tensor parallel"},
            "gpu_launches": stack.launches_last_call() * K, "clocks": clocks,
            "step_roofline": {"bytes_per_step_per_rank": per_rank, "achieved_gbs_per_rank": per_rank / (dev_ms / K * 1e-3) / 1e9,
                              "frac": per_rank / (dev_ms / K * 1e-3) / 1e9 / hbm_peak, "peak": hbm_peak, "peak_kind": peak_kind}}


def _one_region(stack, dev):
    n = (stack.tp_region_bytes(1) + 1023) // 1024 * 1024
    stack._tp_regions = torch.empty(n + 1024, dtype=torch.uint8, device=dev)
    return (stack._tp_regions.data_ptr() + 1023) // 1024 * 1024


def roofline_entry(w, B, mid_ctx, ms_per_step, hbm_peak, peak_kind):
    wbytes, kvbytes = decode_bytes(w, B, mid_ctx)
    gbs = (wbytes + kvbytes) / (ms_per_step * 1e-3) / 1e9
    return {"bytes_per_step": wbytes + kvbytes, "achieved_gbs": gbs, "frac": gbs / hbm_peak, "peak": hbm_peak, "peak_kind": peak_kind}


def prefill_entry(w, Bp, Sp, ms, tf_peak):
    if not ms:
        return None
    tf = prefill_flops(w, Bp, Sp) / (ms * 1e-3) / 1e12
    return {"ms": ms, "tokens": Bp * Sp, "batch": Bp, "prompt": Sp, "tflops": tf, "frac_of_bf16_peak": tf / tf_peak}


def measure_config(run: Run, mask_names, clk, barrier, peaks, reps):
    """sync / spd / config entries of one configuration: prompt phase, then decode on the filled caches."""
    hbm_peak, tf_peak, peak_kind = peaks
    w = run.w
    masks = masks_of(w)
    out = {}
    pre = {}
    for name in mask_names:
        run.stack.set_mask(masks[name])
        pre[name] = run.prefill_ms(reps)
    run.fill_cache()
    mid_ctx = run.ctx0 + run.W + (run.K + 1) / 2.0
    for name in mask_names:
        run.stack.set_mask(masks[name])
        ms, (h0, h1) = run.decode_ms(barrier)
        per_step = ms / run.K
        out[name] = {"mask": "".join(map(str, masks[name])), "ms_per_step": per_step, "tokens_per_s": run.Bd * run.K / (ms * 1e-3),
                     "steps": run.K, "context_mid": mid_ctx,
                     "step_roofline": roofline_entry(w, run.Bd, mid_ctx, per_step, hbm_peak, peak_kind),
                     "prefill": prefill_entry(w, run.Bp, run.Sp, pre[name], tf_peak), "clocks": clk.window(h0, h1)}
    return out


def describe(w: si.Workload, run: Run):
    return (f"{w.name}: {w.n_layers} layers, hidden {w.hidden}, {w.n_q_heads}/{w.n_kv_heads} heads x {w.head_dim}, FFN {w.ffn}, "
            f"T={w.T}, decode batch {run.Bd} at context {run.ctx0}+ (prompt {w.prompt}, {w.decode_steps} decode steps), "
            f"prefill {run.Bp} x {run.Sp}")


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
    peaks = measured_peaks()
    hbm_peak, tf_peak, peak_kind = peaks
    K, W = args.steps, args.warmup

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
            torch.cuda.synchronize()

    w = si.WORKLOADS[args.workload]
    if args.layers:
        w = w.with_(n_layers=args.layers, mask=tuple(w.mask[:args.layers]))
    mask = pick_mask(w, args.mask)
    plan = replica_plan(w, rank, world)
    with ClockSampler(dev.index or 0) as clk:
        run = Run(w, dev, plan["seed"], K, W, args, spd)
        B = run.Bd
        # bf16 stacks of either block kind run the five fused kernels per block, whose launches carry stamps
        fused = w.dtype == "bf16" and not args.rank_mode and "bias_fused=0" not in (args.tune or "")
        run.stack.set_mask(mask)
        pre_ms = run.prefill_ms(args.prefill_reps) if args.prefill_reps > 0 else None
        run.fill_cache()

        # ---- headline: K decode steps, device-timed --------------------------------------
        # (fused path: with the kernels' own start / end stamps on, so that the same region gives the step time and
        # every kernel's share of it; the unstamped region after it shows what the stamps cost)
        dev_ms, (h0, h1) = run.decode_ms(barrier, stamped=fused)
        launches = run.stack.launches_last_call() * K
        clocks = clk.window(h0, h1)
        if fused:
            kind_ms, span_ms, kind_launches = run.timeline_totals()
            plain_ms, _ = run.decode_ms(barrier, base=2 * (W + K))
            plain_ms /= K
            how = ("kernel start/end stamps (two atomics per thread block) folded on the device by a small kernel at the end of "
                   "every graph-replayed step, taken over the K steps of the timed region itself; a launch's share = its end "
                   "minus the later of its start and the latest end before it, so the shares add up to at most the step; "
                   "ms_per_step_unstamped is the same K steps timed again without stamps")

        # ---- end to end: host buffers, copies inside the timed region, result read every step
        x_host = run.xs[W:].cpu().pin_memory()
        out_host = torch.empty((K, B, w.hidden), dtype=run.xs.dtype).pin_memory()
        for t in range(W):
            run.step(W + K + t)
        barrier()
        t0 = time.perf_counter()
        for i in range(K):
            run.x_in.copy_(x_host[i], non_blocking=True)
            run.step(W + K + W + i, x_ready=True)
            out_host[i].copy_(run.out, non_blocking=True)
            torch.cuda.current_stream().synchronize()
        e2e_s = time.perf_counter() - t0
        barrier()

        # ---- where the step's time goes, for the paths whose kernels carry no stamps -------------
        if not fused:
            for t in range(3):
                run.step(2 * (W + K) + t)
            torch.cuda.synchronize()
            run.stack.profile_begin()
            n_prof = min(K, 16)
            for t in range(n_prof):
                run.step(2 * (W + K) + 3 + t)
            prof = run.stack.profile_end()
            kind_ms = {k: v["ms"] / n_prof for k, v in prof.items()}
            kind_launches = {k: v["launches"] // n_prof for k, v in prof.items()}
            span_ms = plain_ms = None
            how = "events around every launch: serialised (no overlap between launches), a lower bound of what the kernels reach in the step"

        dev_ms, e2e_s = max_over_ranks([dev_ms, e2e_s], dev)
        res = None
        if rank == 0:
            mid_ctx = run.ctx0 + W + (K + 1) / 2.0
            ms_per_step = dev_ms / K
            gw = gemm_weight_bytes(w)
            gemm_ms = sum(kind_ms.get(k, 0.0) for k in GEMM_KINDS)
            gemm_launches = sum(kind_launches.get(k, 0) for k in GEMM_KINDS)
            gemm_bytes_step = w.n_layers * sum(gw.values())
            gemm_gbs = gemm_bytes_step / (gemm_ms * 1e-3) / 1e9 if gemm_ms > 0 else None
            es = run.xs.element_size()
            by_kind = {k: {"bytes_per_launch": gw[k], "us_per_launch": kind_ms.get(k, 0.0) * 1e3 / max(kind_launches.get(k, 0), 1),
                           "gbs": gw[k] * kind_launches.get(k, 0) / (kind_ms[k] * 1e-3) / 1e9 if kind_ms.get(k) else None}
                       for k in GEMM_KINDS}
            for v in by_kind.values():
                v["frac"] = v["gbs"] / hbm_peak if v["gbs"] else None
            res = {
                "metric": METRIC, "value": B * world * K / (dev_ms * 1e-3), "unit": "tokens/s", "n_gpus": world,
                "steps": K, "warmup": W, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
                "config": {"workload": describe(w, run), "block": w.block, "rank_mode": bool(args.rank_mode), "mask": list(mask),
                           "mask_name": args.mask, "sync_blocks": [i for i, m in enumerate(mask) if m],
                           "l2": "weights per step exceed L2 (inputs larger than L2)", "context_mid": mid_ctx,
                           "multi_gpu": "replicas only" if world > 1 else "single"},
                "e2e": {"value": B * world * K / e2e_s, "unit": "tokens/s", "h2d_bytes_per_step": B * w.hidden * es,
                        "d2h_bytes_per_step": B * w.hidden * es},
                "gpu_launches": launches,
                "clocks": clocks,
                "step_roofline": roofline_entry(w, B, mid_ctx, ms_per_step, hbm_peak, peak_kind),
                "roofline": {"bound": "hbm", "kernel": "weight-streaming projection GEMM (qkv, o_proj, gate/up, down)",
                             "achieved": gemm_gbs, "peak": hbm_peak, "unit": "GB/s",
                             "frac": (gemm_gbs / hbm_peak) if gemm_gbs else None,
                             "traffic": captured_traffic(w) if not (args.tune or args.rank_mode) else None,
                             "algorithmic_bytes_per_launch": gemm_bytes_step / max(gemm_launches, 1), "peak_kind": peak_kind,
                             "launches_per_step": gemm_launches, "avg_launch_us": gemm_ms * 1e3 / max(gemm_launches, 1),
                             "bytes_per_step": gemm_bytes_step, "how": how, "by_kind": by_kind},
                "kernel_ms_per_step": kind_ms, "sum_kernel_ms": sum(kind_ms.values()), "timeline_span_ms": span_ms,
                "ms_per_step_unstamped": plain_ms,
                "prefill": prefill_entry(w, run.Bp, run.Sp, pre_ms, tf_peak),
            }

        # ---- every listed configuration with the synchronous and the SPD masks --------------
        per_config = None
        want = [] if (world > 1 or args.configs == "none" or args.rank_mode or w.block != "llama" or args.layers) else \
            (list(PER_CONFIG) if args.configs == "all" else [c for c in args.configs.split(",") if c])
        if want:
            per_config = {}
            # the resident headline configuration first, then it makes room for the others
            for name in ([w.name] if w.name in want else []) + [n for n in want if n != w.name]:
                r2 = None
                try:
                    if name == w.name:
                        r2 = run
                    else:
                        if run is not None:
                            run.close()
                            run = None
                        r2 = Run(si.WORKLOADS[name], dev, plan["seed"], K, W, args, spd)
                    entry = measure_config(r2, list(masks_of(r2.w)), clk, barrier, peaks, max(1, args.prefill_reps))
                    entry["workload"] = describe(r2.w, r2)
                    per_config[name] = entry
                except Exception as e:  # one configuration failing must not lose the line
                    per_config[name] = {"error": f"{type(e).__name__}: {e}"}
                finally:
                    if r2 is not None and r2 is not run:
                        r2.close()
        if res is not None:
            res["per_config"] = per_config
    if res is not None and world == 1 and not args.no_cpu_baseline:
        res["cpu_baseline"] = cpu_baseline(w, mask, budget_s=args.cpu_budget)
    return res


# ----------------------------------------------------------------------------------------
def oracle_sample(w: si.Workload, mask):
    """A bounded sample of the workload's decode step for the CPU oracle: the whole stack and batch where one step
    takes seconds, else a slice of the batch through a few blocks chosen with the mask's share of TP blocks; `scale`
    turns the slice's tokens/s into whole-stack tokens/s."""
    gflop_per_token_layer = 2.0 * w.params_per_layer() / 1e9
    full = gflop_per_token_layer * w.n_layers * w.batch
    if full <= 60.0:  # ~2 s per step on a 16-core host
        return list(range(w.n_layers)), w.batch, 1.0
    n_sync = sum(mask)
    n_lay = min(w.n_layers, 4)
    k_sync = min(n_sync, max(1 if n_sync else 0, round(n_lay * n_sync / w.n_layers)))
    k_sync = max(k_sync, n_lay - (w.n_layers - n_sync))  # not more SPD blocks than the mask has
    sync_ids = [i for i, m in enumerate(mask) if m][:k_sync]
    spd_ids = [i for i, m in enumerate(mask) if not m][:n_lay - k_sync]
    layers = sorted(sync_ids + spd_ids)
    B = max(1, min(w.batch, int(60.0 / (gflop_per_token_layer * len(layers)))))
    return layers, B, len(layers) / w.n_layers


def oracle_decode_setup(w, mask, ctx0, seed=0):
    import oracle
    layer_ids, B, scale = oracle_sample(w, mask)
    gen_dev = "cuda" if (torch.cuda.is_available() and w.params_per_layer() > 10 ** 8) else "cpu"
    make = si.make_bias_layer if w.block == "opt" else si.make_layer
    layers = si.to_oracle_layers([{n: t.cpu() for n, t in make(w, l, gen_dev, seed).items()} for l in layer_ids])
    sub_mask = [mask[l] for l in layer_ids]
    if w.block == "opt":  # same call shape for both block kinds
        fwd = oracle.bias_stack_forward
        forward = lambda d, m, l, x, p, c: fwd(d, m, l, x, p, c) + (None,)  # noqa: E731
    else:
        forward = oracle.stack_forward
    dims = oracle.Dims(len(layer_ids), w.hidden, w.n_q_heads, w.n_kv_heads, w.head_dim, w.ffn, w.T, w.rms_eps, w.rope_base)
    cache = oracle.Cache(dims, B, ctx0 + 128)
    rng = np.random.default_rng(seed)
    cache.k[:, :, :ctx0] = rng.standard_normal(cache.k[:, :, :ctx0].shape)
    cache.v[:, :, :ctx0] = rng.standard_normal(cache.v[:, :, :ctx0].shape)
    what = (f"all {w.n_layers} blocks, whole batch {w.batch}" if scale == 1.0 and B == w.batch else
            f"{B} of the {w.batch} sequences through {len(layer_ids)} of the {w.n_layers} blocks ({sum(sub_mask)} TP + "
            f"{len(sub_mask) - sum(sub_mask)} SPD, blocks {layer_ids}); tokens/s = {B} / (step time x {w.n_layers}/{len(layer_ids)})")
    return forward, dims, layers, sub_mask, cache, B, scale, what


def cpu_baseline(w, mask, budget_s=15.0):
    """The oracle, as it stands, on the host cores: decode steps of a bounded sample of the same workload at the
    mid-run context, the cache holding seeded stand-in values."""
    ctx0 = w.prompt + w.decode_steps // 2
    forward, dims, layers, sub_mask, cache, B, scale, what = oracle_decode_setup(w, mask, ctx0)
    n, t_total = 0, 0.0
    while t_total < budget_s and n < 64:
        x = si.make_hidden(w, (B, 1, w.hidden), "cpu", 0, 1 + n).double().numpy()
        t0 = time.perf_counter()
        forward(dims, sub_mask, layers, x, np.full(B, ctx0 + n, np.int32), cache)
        t_total += time.perf_counter() - t0
        n += 1
    return {"value": B * n / t_total * scale, "unit": "tokens/s", "cores": os.cpu_count(), "kind": "oracle",
            "sample": f"{n} decode steps at context {ctx0}+: {what}; KV cache pre-filled with seeded values instead of an "
                      f"oracle prefill; {t_total:.1f} s"}


def run_reference(args):
    w = si.WORKLOADS[args.workload]
    mask = pick_mask(w, args.mask)
    K, W = args.steps, args.warmup
    ctx0 = w.prompt + w.decode_steps // 2
    forward, dims, layers, sub_mask, cache, B, scale, what = oracle_decode_setup(w, mask, ctx0)
    times = []
    for t in range(W + K):
        x = si.make_hidden(w, (B, 1, w.hidden), "cpu", 0, 1 + t).double().numpy()
        t0 = time.perf_counter()
        forward(dims, sub_mask, layers, x, np.full(B, ctx0 + t, np.int32), cache)
        if t >= W:
            times.append(time.perf_counter() - t0)
    total = float(sum(times))
    val = B * K / total * scale
    sample = f"each step = one decode step at context {ctx0}+t: {what}; KV cache pre-filled with seeded values instead of an oracle prefill"
    return {"impl": "reference", "metric": METRIC, "value": val, "unit": "tokens/s", "n_gpus": args.gpus, "steps": K,
            "warmup": W, "ms_per_step": total / K * 1e3 / scale * (w.batch / B), "higher_is_better": True, "scaling": "weak",
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
    ap.add_argument("--workload", default="c5", choices=sorted(si.WORKLOADS))
    ap.add_argument("--mask", default="config", choices=["config", "sync", "spd"])
    ap.add_argument("--configs", default="all", help="per_config entries: all, none, or a comma-separated list of workloads")
    ap.add_argument("--layers", type=int, default=0, help="run only the first N blocks of the workload (small profiler captures)")
    ap.add_argument("--prefill-chunk", type=int, default=8192)
    ap.add_argument("--prefill-reps", type=int, default=3)
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    ap.add_argument("--settle-s", type=float, default=0.5, help="seconds of untimed decode steps before every timed decode region")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--rank-mode", action="store_true",
                    help="decode through spd_tp_decode_step: all T ranks of a tensor-parallel group executed on this GPU")
    ap.add_argument("--tp", default="", choices=["", "fused", "baseline"],
                    help="ONE model over the job's ranks, shard r on rank r (launch under torchrun with as many ranks as shards): "
                         "fused = exchanges inside the projection tails (rank mode), baseline = NCCL all-reduce between kernels")
    ap.add_argument("--tune", default="", help="decode tuning knobs, e.g. qkv_splits=4,l2_prefetch_blocks=8 (see spd_set_tuning)")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # no launcher around us: be the launcher (one rank per GPU of this node)
        sys.exit(spawn_ranks(args.gpus, [sys.executable, os.path.abspath(__file__)] + sys.argv[1:]))
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))
    if args.impl == "reference":
        args.steps = args.steps if args.steps is not None else 16
        args.warmup = args.warmup if args.warmup is not None else 1
        if rank == 0:
            print(json.dumps(run_reference(args)), flush=True)
        return
    args.steps = args.steps if args.steps is not None else 32
    args.warmup = max(args.warmup if args.warmup is not None else 5, 3)
    if world > 1 or args.tp:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", str(free_port()))
        os.environ.setdefault("RANK", "0")
        os.environ.setdefault("WORLD_SIZE", "1")
        torch.distributed.init_process_group("nccl", device_id=torch.device(f"cuda:{int(os.environ.get('LOCAL_RANK', 0))}"))
    res = run_tp(args, rank, world) if args.tp else run_native(args, rank, world)
    if rank == 0:
        print(json.dumps(res), flush=True)
    if world > 1 or args.tp:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()
