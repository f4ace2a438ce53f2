"""The N>1 path on CPU: two gloo ranks shard one candidate stream, solve their slices (with the
CPU oracle standing in for the device here), and agree on max-over-ranks timing; the union of the
shards must equal the unsharded batch."""
import json
import os
import socket
import subprocess

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2201_13096_b200 import sharding, workloads as W


def test_shard_range_partitions_exactly():
    for n in (0, 1, 7, 4096, 65537):
        for world in (1, 2, 3, 8):
            spans = [sharding.shard_range(n, r, world) for r in range(world)]
            assert spans[0][0] == 0 and sum(c for _, c in spans) == n
            for (s0, c0), (s1, _) in zip(spans, spans[1:]):
                assert s0 + c0 == s1
            assert max(c for _, c in spans) - min(c for _, c in spans) <= 1


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, n_total, out_dir):
    import oracle

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    start, count = sharding.shard_range(n_total, rank, world)
    wl = W.make_workload(1, N=count, start=start)
    p, c, t = oracle.solve_batch(wl.errors, wl.times, wl.B, threads=2)
    np.savez(os.path.join(out_dir, f"r{rank}.npz"), p=p, c=c, t=t, start=start, count=count)
    mine = 1.0 + rank  # pretend timings
    worst = sharding.max_over_ranks(mine)
    dist.barrier()
    assert worst == float(world)
    rate = sharding.whole_job_rate(count, world, worst)
    gathered = [None] * world
    dist.all_gather_object(gathered, rate)
    assert all(abs(g - gathered[0]) < 1e-9 for g in gathered) or n_total % world != 0
    dist.destroy_process_group()


def test_two_gloo_ranks_cover_the_batch(tmp_path):
    import oracle

    oracle.build()
    world, n_total = 2, 10
    mp.spawn(_worker, args=(world, _free_port(), n_total, str(tmp_path)), nprocs=world, join=True)
    full = W.make_workload(1, N=n_total)
    rp, rc, rt = oracle.solve_batch(full.errors, full.times, full.B, threads=4)
    got_p = np.concatenate([np.load(tmp_path / f"r{r}.npz")["p"] for r in range(world)])
    got_c = np.concatenate([np.load(tmp_path / f"r{r}.npz")["c"] for r in range(world)])
    got_t = np.concatenate([np.load(tmp_path / f"r{r}.npz")["t"] for r in range(world)])
    assert np.array_equal(got_p, rp) and got_c.tobytes() == rc.tobytes() and np.array_equal(got_t, rt)


def test_max_over_ranks_without_a_process_group():
    assert sharding.max_over_ranks(3.5) == 3.5
    assert sharding.whole_job_rate(100, 4, 2.0) == 200.0


def test_local_launcher_starts_the_ranks_itself():
    """The launch path `bench.py --gpus N` takes when no launcher started it: N ranks on this node with
    a 127.0.0.1 rendezvous, rank 0 printing the line.  Here with two gloo ranks on CPU."""
    script = os.path.join(os.path.dirname(os.path.abspath(__file__)), "rank_probe.py")
    cmd = sharding.launch_command(script, ["11"], 2)
    assert "--master-addr" in cmd and cmd[cmd.index("--master-addr") + 1] == "127.0.0.1"
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    out = subprocess.run(cmd, env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads([ln for ln in out.stdout.splitlines() if ln.startswith("{")][-1])
    assert line["n_gpus"] == 2 and line["worst"] == 2.0
    assert line["shards"] == [[0, 6], [6, 5]]
    assert not sharding.under_launcher() or "WORLD_SIZE" in os.environ
    with __import__("pytest").raises(ValueError):
        sharding.launch_command(script, [], 0)
