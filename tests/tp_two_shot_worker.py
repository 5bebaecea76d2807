"""Worker of the CPU test of the rank mode's prompt exchange (gloo ranks): every rank holds a partial [M, H] matrix;
shot one sends the rows of each 128-token tile to the tile's owner (paper_2502_20727_b200.tp_tile_owner: the mapping the
CUDA kernels use), the owner adds the T planes in rank order, shot two sends the finished rows to every rank."""
import json
import os
import sys

import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

import paper_2502_20727_b200 as spd  # noqa: E402


def main():
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    dist.init_process_group("gloo")
    rank, T = dist.get_rank(), dist.get_world_size()
    M, H = 600, 16                                    # five 128-token tiles, the last with 88 rows
    tiles = (M + 127) // 128
    g = torch.Generator().manual_seed(100 + rank)
    part = torch.randn(M, H, generator=g, dtype=torch.float64)
    rows = lambda i: slice(i * 128, min(M, (i + 1) * 128))
    # shot one: my rows of tile i go to its owner's plane [source = me][slot]
    planes = {}                                       # (source, slot) -> rows, on the owner
    for i in range(tiles):
        owner, slot = spd.tp_tile_owner(i, T)
        for src in range(T):
            if src == owner:
                if rank == owner:
                    planes[(src, slot)] = part[rows(i)].clone()
                continue
            if rank == src:
                dist.send(part[rows(i)].contiguous(), dst=owner, tag=i)
            elif rank == owner:
                buf = torch.empty_like(part[rows(i)])
                dist.recv(buf, src=src, tag=i)
                planes[(src, slot)] = buf
    # the owner adds its T planes in rank order; shot two: finished rows to everyone
    total = torch.zeros(M, H, dtype=torch.float64)
    owned = 0
    for i in range(tiles):
        owner, slot = spd.tp_tile_owner(i, T)
        if rank == owner:
            acc = planes[(0, slot)].clone()
            for src in range(1, T):
                acc += planes[(src, slot)]
            total[rows(i)] = acc
            owned += 1
        dist.broadcast(total[rows(i)], src=owner)
    ref = part.clone()
    dist.all_reduce(ref)
    # the all-reduce may add in another order: compare with the rank-ordered sum computed from gathered partials
    gathered = [torch.empty_like(part) for _ in range(T)]
    dist.all_gather(gathered, part)
    ordered = gathered[0].clone()
    for src in range(1, T):
        ordered += gathered[src]
    stats = [None] * T
    dist.all_gather_object(stats, {"owned": owned, "planes": len(planes), "err": float((total - ordered).abs().max()),
                                   "close_to_all_reduce": bool(torch.allclose(total, ref))})
    if rank == 0:
        assert all(s["close_to_all_reduce"] for s in stats)
        print("WORKER " + json.dumps({"world": T, "tiles": tiles, "max_err": max(s["err"] for s in stats),
                                      "owned": [s["owned"] for s in stats], "planes_received": [s["planes"] for s in stats]}), flush=True)
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
