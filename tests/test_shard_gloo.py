"""The N > 1 plumbing on CPU: two gloo ranks, no GPU.  (batch, head) pairs are independent, so ranks
share nothing but a barrier and the max / sum of their timings; each rank's shard is its own seeded
batch (weak scaling) or a slice of one batch (strong scaling), and the union of the slices is the batch."""
import os
import socket

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2511_21016_b200 import shard, synth


def _free_port() -> int:
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      LOCAL_RANK=str(rank), WORLD_SIZE=str(world))
    assert shard.env_rank_world() == (rank, rank, world)
    shard.init_process_group("gloo")
    cfg = synth.GkaConfig("gloo", B=3, heads=2, T=64, d=8, chunk=64, n_iter=3, io_dtype="f32", seed=5)
    # strong scaling: slice one global batch; every sequence is owned by exactly one rank
    lo, hi = shard.batch_slice(cfg.B, rank, world)
    full = synth.make_inputs(cfg)
    mine = {n: a[lo:hi] for n, a in full.items()}
    res = oracle.fwd(mine["q"], mine["k"], mine["v"], mine["gate"], mine["lam"], cfg.n_iter, threads=1)
    np.save(os.path.join(out_dir, f"out_{rank}.npy"), res["out"])
    np.save(os.path.join(out_dir, f"range_{rank}.npy"), np.array([lo, hi]))
    # weak scaling: per-rank seeds differ
    assert shard.shard_seed(cfg.seed, rank) == cfg.seed + 1000 * rank
    shard.barrier()
    # the job's time is its slowest rank's; counts add up
    t = shard.max_over_ranks(1.0 + rank)
    n = shard.sum_over_ranks(float(hi - lo))
    assert t == float(world) and n == float(cfg.B)
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_without_collectives(tmp_path):
    world = 2
    port = _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    cfg = synth.GkaConfig("gloo", B=3, heads=2, T=64, d=8, chunk=64, n_iter=3, io_dtype="f32", seed=5)
    full = synth.make_inputs(cfg)
    ref = oracle.fwd(full["q"], full["k"], full["v"], full["gate"], full["lam"], cfg.n_iter, threads=1)["out"]
    ranges = [np.load(tmp_path / f"range_{r}.npy") for r in range(world)]
    assert ranges[0][0] == 0 and ranges[-1][1] == cfg.B and ranges[0][1] == ranges[1][0]
    got = np.concatenate([np.load(tmp_path / f"out_{r}.npy") for r in range(world)], axis=0)
    assert np.array_equal(got, ref)       # shards are bit-identical to the unsharded run


def test_batch_slices_cover_without_overlap():
    for total in (1, 5, 8, 64):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                lo, hi = shard.batch_slice(total, r, world)
                seen.extend(range(lo, hi))
            assert seen == list(range(total))


def test_local_launcher_starts_ranks_with_the_torchrun_environment(tmp_path):
    """`bench.py --gpus N` without torchrun starts N ranks itself; here the same environment is given to two CPU
    processes that meet in a gloo barrier and take the max of their ranks."""
    import subprocess
    import sys
    code = (
        "import os, sys; sys.path.insert(0, os.environ['GKA_ROOT'])\n"
        "from paper_2511_21016_b200 import shard\n"
        "r, lr, w = shard.env_rank_world(); assert lr == r and w == 2\n"
        "shard.init_process_group('gloo'); shard.barrier()\n"
        "m = shard.max_over_ranks(float(r))\n"
        "open(os.path.join(os.environ['GKA_OUT'], f'rank{r}.txt'), 'w').write(str(m))\n"
        "import torch.distributed as dist; dist.destroy_process_group()\n")
    port = shard.free_port()
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    procs = []
    for r in range(2):
        env = shard.rank_env(r, 2, port)
        env.update(GKA_ROOT=root, GKA_OUT=str(tmp_path))
        assert env["MASTER_ADDR"] == "127.0.0.1" and env["WORLD_SIZE"] == "2" and env["LOCAL_RANK"] == str(r)
        procs.append(subprocess.Popen([sys.executable, "-c", code], env=env))
    assert [p.wait(timeout=120) for p in procs] == [0, 0]
    assert [open(tmp_path / f"rank{r}.txt").read() for r in range(2)] == ["1.0", "1.0"]
