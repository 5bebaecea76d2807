"""Worker of the tensor-parallel CPU test (gloo ranks): rank r holds shard r of one block as
paper_2502_20727_b200.shard_layer cuts it, computes its part with the CPU oracle run as a one-shard
block, and exchanges partial sums with a gloo all-reduce exactly where the rank-mode GPU step
exchanges them: twice in a TP block (Y_r after o_proj, Z_r after down), once in an SPD block
(Y_r + Z_r after down, X added after the sum)."""
import json
import os
import sys

import numpy as np
import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
import paper_2502_20727_b200 as spd  # noqa: E402
import spd_inputs as si  # noqa: E402


def all_reduce(a, collective):
    """Through the same helper the GPU baseline arm hands to spd_tp_baseline_* (there over NCCL, here over gloo)."""
    t = torch.from_numpy(np.ascontiguousarray(a))
    collective(t)
    return t.numpy()


def main():
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    dist.init_process_group("gloo")
    rank, T = dist.get_rank(), dist.get_world_size()
    w = si.Workload("tp_cpu", "fp32", 1, 64, 4, 2, 16, 96, T, (0,), 2, 5, 0)
    full = si.make_layer(w, 0, "cpu", 0)
    mine = spd.shard_layer(full, rank, T)
    dims = oracle.Dims(1, w.hidden, w.n_q_heads, w.n_kv_heads, w.head_dim, w.ffn, T, w.rms_eps, w.rope_base)
    one = oracle.Dims(1, w.hidden, w.n_q_heads // T, w.n_kv_heads // T, w.head_dim, w.ffn // T, 1, w.rms_eps, w.rope_base)
    B, S = 2, 5
    x = si.make_hidden(w, (B, S, w.hidden), "cpu", 0, 0).double().numpy()
    pos0 = np.zeros(B, dtype=np.int32)
    to_np = lambda lw: si.to_oracle_layers([lw])[0]
    res = {}
    for mode, name in ((0, "spd"), (1, "sync")):
        ref, _, ref_syncs = oracle.block_forward(dims, to_np(full), mode, x, pos0, oracle.Cache(dims, B, S))
        n = spd.CollectiveAllReduce()
        if mode == 0:
            # R_r = X + Y_r stays on the rank; one exchange of Y_r + Z_r; X joins after the sum
            out_r, _, _ = oracle.block_forward(one, to_np(mine), 0, x, pos0, oracle.Cache(one, B, S))
            out = x + all_reduce(out_r - x, n)
        else:
            no_mlp = dict(mine, w_down=torch.zeros_like(mine["w_down"]))
            y_r, _, _ = oracle.block_forward(one, to_np(no_mlp), 1, x, pos0, oracle.Cache(one, B, S))
            r = x + all_reduce(y_r - x, n)
            no_attn = dict(mine, wo=torch.zeros_like(mine["wo"]))
            z_r, _, _ = oracle.block_forward(one, to_np(no_attn), 1, r, pos0, oracle.Cache(one, B, S))
            out = r + all_reduce(z_r - r, n)
        res[name] = {"err": float(np.max(np.abs(out - ref)) / np.max(np.abs(ref))), "exchanges": n.calls, "syncs": int(ref_syncs)}
    gathered = [None] * T
    dist.all_gather_object(gathered, res)
    if rank == 0:
        print("WORKER " + json.dumps({"world": T, "ranks": gathered}), flush=True)
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
