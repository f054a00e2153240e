"""The Worker class's plumbing on CPU, two gloo ranks: ring of D + 1 exchange buffers,
asynchronous all-reduce started after each outer step and awaited D steps later, blocking
all-reduce for standard DiLoCo.  The CUDA state is replaced by a stand-in that performs one
worker's share of the step in numpy (fp32, same operation order as the kernels); the ranks'
results must equal the fused CPU oracle bit for bit (two-term sums have only one order)."""
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


class NumpyWorkerState:
    """What binding.State does for one replica, on CPU tensors (shared memory with numpy)."""

    def __init__(self, *, M, P, stride, theta, start, outer_mom, delta_prev_local=None, have_prev=0, overlap_steps=1,
                 outer_lr=0.7, outer_momentum=0.9, **_):
        assert M == 1
        self.P, self.D = P, overlap_steps
        self.theta, self.start, self.mom = theta.numpy(), start.numpy(), outer_mom.numpy()
        self.dpl = None if delta_prev_local is None else delta_prev_local.numpy()
        self.have, self.k = have_prev, 0
        self.eta, self.mu = np.float32(outer_lr), np.float32(outer_momentum)

    def worker_outer_send(self, send):
        send.numpy()[:self.P] = self.start[:self.P] - self.theta[:self.P]

    def worker_outer_apply(self, variant, world, recv, send):
        P, f = self.P, np.float32
        slot = self.k % self.D
        s, x = self.start[:P], self.theta[:P]
        first = variant != 0 and self.have < self.D
        if variant != 0:
            d = (s - x).astype(f)
            send.numpy()[:P] = d
        if first:
            self.start[:P] = x
            if variant == 2:
                self.dpl[slot, :P] = d
        else:
            mean = (recv.numpy()[:P] / f(world)).astype(f)
            if variant == 2:
                g = (((d - self.dpl[slot, :P]).astype(f) / f(world)).astype(f) + mean).astype(f)
            else:
                g = mean
            b = ((self.mu * self.mom[:P]).astype(f) + g).astype(f)
            u = (self.eta * (g + (self.mu * b).astype(f)).astype(f)).astype(f)
            n = (s - u).astype(f)
            self.mom[:P], self.start[:P], self.theta[:P] = b, n, n
            if variant == 2:
                self.dpl[slot, :P] = d
        if variant != 0 and self.have < self.D:
            self.have += 1
        self.k += 1

    def close(self):
        pass


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def draw(world, P, seed):
    rng = np.random.default_rng(seed)
    s0 = rng.normal(0, 0.02, P).astype(np.float32)
    start = np.tile(s0, (world, 1))
    theta = (start + rng.normal(0, 1e-3, (world, P))).astype(np.float32)
    moves = rng.normal(0, 1e-3, (8, world, P)).astype(np.float32)
    return start, theta, moves


def rank_main(rank, world, port, variant, D, P, steps, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2502_12996_b200 import worker
    start, theta, moves = draw(world, P, 5)
    t = dict(theta=torch.from_numpy(theta[rank].copy()), start=torch.from_numpy(start[rank].copy()),
             outer_mom=torch.zeros(P), delta_prev_local=torch.zeros((D, P)))
    w = worker.Worker(t, P=P, stride=P, world_replicas=world, variant=variant, overlap_steps=D, have_prev=0,
                      state_factory=NumpyWorkerState)
    for k in range(steps):
        if k:
            t["theta"].copy_(t["start"] + torch.from_numpy(moves[k - 1, rank]))
        w.outer_step()
    w.finish()
    np.savez(Path(out_dir) / f"rank{rank}.npz", **{k: v.numpy() for k, v in t.items()})
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("variant,D", [(2, 1), (2, 2), (1, 1), (0, 1)])
def test_worker_ring_on_two_gloo_ranks(oracle, tmp_path, variant, D):
    world, P, steps = 2, 1000, 2 * D + 3
    mp.spawn(rank_main, args=(world, free_port(), variant, D, P, steps, str(tmp_path)), nprocs=world, join=True)
    start, theta, moves = draw(world, P, 5)
    h = dict(start=start.copy(), theta=theta.copy(), outer_mom=np.zeros((world, P), np.float32),
             delta_prev_local=np.zeros((D, world, P), np.float32), delta_prev_avg=np.zeros((D, P), np.float32))
    have = 0
    for k in range(steps):
        if k:
            h["theta"] = (h["start"] + moves[k - 1]).astype(np.float32)
        have = oracle.outer_step_overlap(variant, k, have, M=world, P=P, stride=P, eta=0.7, mu=0.9, **h)
    for r in range(world):
        z = np.load(tmp_path / f"rank{r}.npz")
        np.testing.assert_array_equal(z["theta"], h["theta"][r])
        np.testing.assert_array_equal(z["start"], h["start"][r])
        np.testing.assert_array_equal(z["outer_mom"], h["outer_mom"][r])
        if variant == 2:
            np.testing.assert_array_equal(z["delta_prev_local"], h["delta_prev_local"][:, r])
