"""N > 1 on CPU: two gloo ranks run the rank plumbing of bench.py (replicas only: no collective on the
data path, timing = max over ranks, rank 0 prints the one line), and the shard / exchange logic of
tensor parallelism across ranks (one shard per rank, partial sums exchanged where the block keeps
its sync-points)."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def torchrun(script_and_args, n=2):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(free_port())] + script_and_args
    env = dict(os.environ, OMP_NUM_THREADS="2")
    r = subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    return r.stdout


def test_two_ranks_replica_plan_and_max_timing():
    out = torchrun([os.path.join(ROOT, "tests", "rank_worker.py")])
    lines = [l for l in out.splitlines() if l.startswith("WORKER ")]
    assert len(lines) == 1
    res = json.loads(lines[0][7:])
    assert res["world"] == 2 and res["seeds"] == [0, 1]
    assert res["t_max"] == 2.0 and res["t_same"] == 5.0        # slowest rank decides
    assert res["job_tokens"] == 2                               # c1: batch 1 per rank, weak scaling
    assert res["distinct_weights"] == 2                         # independent replicas


def test_reference_arm_prints_one_line_under_torchrun():
    out = torchrun([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1", "--gpus", "2", "--steps", "2",
                    "--warmup", "1"])
    lines = [l for l in out.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    res = json.loads(lines[0])
    assert res["impl"] == "reference" and res["n_gpus"] == 2 and res["value"] > 0
    assert res["cpu_baseline"]["kind"] == "oracle" and res["e2e"]["h2d_bytes_per_step"] == 0


def test_two_ranks_hold_one_shard_each_and_exchange_partial_sums():
    """Sec. 3 / Sec. 4.1.1 across real ranks: shard r from shard_layer, the block's kept sync-points as
    all-reduces - the result equals the oracle's sharded block, with 2 exchanges (TP) or 1 (SPD)."""
    out = torchrun([os.path.join(ROOT, "tests", "tp_rank_worker.py")])
    lines = [l for l in out.splitlines() if l.startswith("WORKER ")]
    assert len(lines) == 1
    res = json.loads(lines[0][7:])
    assert res["world"] == 2
    for r in res["ranks"]:
        assert r["spd"]["err"] < 1e-12 and r["sync"]["err"] < 1e-12
        assert r["spd"]["exchanges"] == 1 == r["spd"]["syncs"]
        assert r["sync"]["exchanges"] == 2 == r["sync"]["syncs"]


def test_bench_starts_its_own_ranks_when_no_launcher_did():
    """`bench.py --gpus 2` without torchrun around it: the process becomes the launcher (one child per rank with RANK /
    WORLD_SIZE / MASTER_* set), and still exactly one line comes out, from rank 0, saying n_gpus 2."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    env["OMP_NUM_THREADS"] = "2"
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c1", "--gpus", "2",
                        "--steps", "2", "--warmup", "1"], cwd=ROOT, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    res = json.loads(lines[0])
    assert res["impl"] == "reference" and res["n_gpus"] == 2 and res["value"] > 0


def test_spawned_ranks_form_a_group_and_a_failing_rank_fails_the_job():
    """spawn_ranks gives every child its rank and a common rendezvous: two gloo ranks find each other through it
    (the worker checks world size, seeds and the max-over-ranks timing), and a non-zero exit of any rank is returned."""
    sys.path.insert(0, ROOT)
    import bench
    env = dict(os.environ, OMP_NUM_THREADS="2")
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        env.pop(k, None)
    assert bench.spawn_ranks(2, [sys.executable, os.path.join(ROOT, "tests", "rank_worker.py")], env=env, timeout=600) == 0
    assert bench.spawn_ranks(2, [sys.executable, "-c", "import os, sys; sys.exit(3 if os.environ['RANK'] == '1' else 0)"], env=env) == 3


def test_two_shot_exchange_index_logic_over_gloo_ranks():
    """The prompt exchange of the rank mode on CPU ranks: 128-token tiles dealt round-robin (tile i -> rank i % T, slot
    i // T), partial rows sent to the owner, summed there in rank order, finished rows sent to everyone.  The result is
    the all-reduce, every (owner, slot) is hit exactly once, and the owner's receive planes hold (tiles it owns) x T
    source planes - the counts the device-side flags are sized by."""
    out = torchrun([os.path.join(ROOT, "tests", "tp_two_shot_worker.py")], n=3)
    lines = [l for l in out.splitlines() if l.startswith("WORKER ")]
    assert len(lines) == 1
    res = json.loads(lines[0][7:])
    assert res["world"] == 3 and res["tiles"] == 5
    assert res["max_err"] == 0.0                      # same sums in the same (rank) order on every rank
    assert res["owned"] == [2, 2, 1]                  # tiles 0,3 | 1,4 | 2
    assert res["planes_received"] == [6, 6, 3]        # owned tiles x T sources
