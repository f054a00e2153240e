"""Multi-rank host logic on CPU (gloo, world_size 2): the parameter axis is split into
64-aligned contiguous ranges, one per rank, all M replicas of an index on the same rank, and
no step of the path crosses ranks.  Each rank runs its shard (here through the CPU oracle,
which stands in for the per-rank kernel launch), the shards are gathered, and the result must
equal the unsharded run bit for bit; timings reduce with MAX as bench.py does."""
import os
import socket
import sys
from pathlib import Path

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent
sys.path.insert(0, str(ROOT))


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def make_state(M, P, seed):
    from paper_2502_12996_b200 import inputs
    st = inputs.make_outer_state(M, P, seed, device="cpu")
    return {k: st[k].numpy() for k in ("theta", "start", "delta_prev_local", "delta_prev_avg", "outer_mom")}, st["stride"]


def worker(rank, world, port, M, P, seed, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from bench import shard_bounds
    full, stride = make_state(M, P, seed)                    # same seed on every rank -> same tensors
    lo, hi = shard_bounds(P, world, rank)
    n = hi - lo
    part = {k: np.ascontiguousarray(v[..., lo:hi]) for k, v in full.items()}
    for _ in range(2):
        oracle.outer_step(oracle.EAGER, M=M, P=n, stride=n, eta=0.7, mu=0.9, theta=part["theta"], start=part["start"],
                          outer_mom=part["outer_mom"], delta_prev_local=part["delta_prev_local"],
                          delta_prev_avg=part["delta_prev_avg"])
        part["theta"] += np.float32(1e-3) * (part["start"] != 0)           # a deterministic "inner phase"
    # bench.py's timing reduction: every rank reports its own time, the job's time is the max
    t = torch.tensor([1.0 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    assert float(t) == float(world)
    bounds = [None] * world
    dist.all_gather_object(bounds, (lo, hi))
    np.savez(Path(out_dir) / f"rank{rank}.npz", lo=lo, hi=hi, bounds=np.array(bounds), **part)
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("P", [100_003, 64 * 7, 130])
def test_two_ranks_reproduce_the_unsharded_step(tmp_path, oracle, P):
    M, seed, world = 4, 77, 2
    mp.spawn(worker, args=(world, free_port(), M, P, seed, str(tmp_path)), nprocs=world, join=True)
    full, stride = make_state(M, P, seed)
    for _ in range(2):
        oracle.outer_step(oracle.EAGER, M=M, P=P, stride=stride, eta=0.7, mu=0.9, theta=full["theta"],
                          start=full["start"], outer_mom=full["outer_mom"],
                          delta_prev_local=full["delta_prev_local"], delta_prev_avg=full["delta_prev_avg"])
        full["theta"][:, :P] += np.float32(1e-3) * (full["start"][:, :P] != 0)
    covered = 0
    for r in range(world):
        z = np.load(tmp_path / f"rank{r}.npz")
        lo, hi = int(z["lo"]), int(z["hi"])
        assert lo % 64 == 0 and lo == covered
        covered = hi
        for k in full:
            np.testing.assert_array_equal(z[k], full[k][..., lo:hi])
    assert covered == P


def test_shard_bounds_cover_and_align():
    from bench import shard_bounds
    for P in (1, 63, 64, 65, 35_000_000, 2_400_000_000):
        for world in (1, 2, 3, 8):
            prev = 0
            for r in range(world):
                lo, hi = shard_bounds(P, world, r)
                assert lo == prev and lo % 64 == 0 and hi >= lo
                prev = hi
            assert prev == P
