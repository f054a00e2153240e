"""The worker form (one replica per worker, outer gradients exchanged by an all-reduce).

(1) Emulation in one process: M one-replica states, the all-reduce replaced by an ordered
    torch sum of the workers' send buffers; every buffer must equal the fused M-replica
    oracle's bit for bit (same arithmetic, sum in the order m = 0..M-1).
(2) Two real processes with torch.distributed (gloo; both ranks on this GPU, no rank's kernel
    waits on another's): the Worker class with its asynchronous all-reduce ring against the
    oracle, bit-exact because a two-term sum has only one order.
"""
import os
import socket
import sys
from pathlib import Path

import numpy as np
import pytest
import torch

from paper_2502_12996_b200 import binding, inputs
from gpu_util import assert_state_equal, host_copy, to_numpy

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
ROOT = Path(__file__).resolve().parent.parent


def row(t, m):
    return None if t is None else t[m]


@pytest.mark.parametrize("variant", [0, 1, 2])
@pytest.mark.parametrize("M,P,theta_kind,D,have", [(2, 100_003, 0, 1, 0), (4, 70_001, 0, 1, 1), (3, 30_001, 1, 1, 0),
                                                   (4, 50_002, 2, 2, 0), (8, 20_001, 0, 2, 2), (1, 5_001, 0, 1, 0)])
def test_workers_with_ordered_sum_equal_the_fused_oracle(oracle, variant, M, P, theta_kind, D, have):
    st = inputs.make_outer_state(M, P, 2100 + M + D, device=DEV, theta_kind=theta_kind, overlap_steps=D)
    stride = st["stride"]
    h = host_copy(st)
    dpl = st["delta_prev_local"].view(D, M, stride)
    dpa = st["delta_prev_avg"].view(D, stride)
    states = []
    for m in range(M):
        states.append(binding.State(M=1, P=P, stride=stride, theta=st["theta"][m], master=row(st["master"], m),
                                    start=st["start"][m], outer_mom=st["outer_mom"][m],
                                    delta_prev_local=dpl[:, m].contiguous() if variant == 2 else None,
                                    theta_kind=theta_kind, have_prev=have, overlap_steps=D))
    # each worker's own stale gradients live in its private ring (a copy, as on a real worker)
    own = [s.tensors["delta_prev_local"] for s in states]
    sends = [torch.zeros(stride, device=DEV) for _ in range(M)]
    # the sums "in flight": generation g of the seeded state is the mean times M
    sums = [(dpa[g] * float(M)).clone() for g in range(D)]
    hv = have
    for k in range(2 * D + 2):
        if k:
            inputs.inner_phase_standin(st)
            h["theta"], h["master"] = to_numpy(st["theta"]), to_numpy(st["master"])
        slot = k % D
        if variant == 0:
            for m in range(M):
                states[m].worker_outer_send(sends[m])
        else:
            for m in range(M):
                states[m].worker_outer_apply(variant, M, sums[slot] if hv >= D else None, sends[m])
        total = sends[0].clone()                         # the all-reduce, in worker order
        for m in range(1, M):
            total += sends[m]
        if variant == 0:
            for m in range(M):
                states[m].worker_outer_apply(0, M, total, None)
        else:
            sums[slot] = total
        hv = oracle.outer_step_overlap(variant, k, hv, M=M, P=P, stride=stride, eta=0.7, mu=0.9, theta=h["theta"],
                                       master=h["master"], start=h["start"], outer_mom=h["outer_mom"],
                                       delta_prev_local=h["delta_prev_local"].reshape(D, M, stride),
                                       delta_prev_avg=h["delta_prev_avg"].reshape(D, stride), theta_kind=theta_kind)
        torch.cuda.synchronize()
        got = dict(theta=st["theta"], master=st["master"], start=st["start"], outer_mom=st["outer_mom"])
        assert_state_equal(got, h, keys=tuple(got), what=f"worker form variant {variant} M={M} D={D} step {k + 1}")
        if variant != 0:
            # the fused state keeps the mean; the workers keep the sum
            mean = sums[slot].cpu().numpy() / np.float32(M)   # (torch multiplies by 1/M on the GPU)
            np.testing.assert_array_equal(mean[:P], h["delta_prev_avg"].reshape(D, stride)[slot][:P])
        if variant == 2:
            for m in range(M):
                np.testing.assert_array_equal(own[m].view(D, stride)[slot].cpu().numpy()[:P],
                                              h["delta_prev_local"].reshape(D, M, stride)[slot, m][:P])
    for s in states:
        s.close()


@pytest.mark.parametrize("fmt", [(4, 3), (2, 1), (3, 0), (5, 2), (3, 2)])
@pytest.mark.parametrize("variant,M,P,theta_kind,D", [(2, 4, 70_001, 0, 1), (2, 3, 30_002, 1, 2), (1, 2, 20_003, 0, 1),
                                                      (0, 5, 10_001, 2, 1), (2, 1, 999, 0, 1)])
def test_quantised_wire_workers_equal_the_fused_quantised_oracle(oracle, fmt, variant, M, P, theta_kind, D):
    """Each worker sends EXMY codes + its maximum, gathers everyone's, and forms the mean itself:
    bit-identical to the fused quantised oracle for ANY M (a gather keeps the worker order), and
    the bytes on the wire equal the oracle's encoding."""
    X, Y = fmt
    st = inputs.make_outer_state(M, P, 2300 + M + D, device=DEV, theta_kind=theta_kind, overlap_steps=D)
    stride = st["stride"]
    h = host_copy(st)
    dpl = st["delta_prev_local"].view(D, M, stride)
    states = [binding.State(M=1, P=P, stride=stride, theta=st["theta"][m], master=row(st["master"], m),
                            start=st["start"][m], outer_mom=st["outer_mom"][m],
                            delta_prev_local=dpl[:, m].contiguous() if variant == 2 else None,
                            theta_kind=theta_kind, have_prev=0, overlap_steps=D) for m in range(M)]
    nbytes = (binding.wire_payload_bytes(P, X, Y) + 15) // 16 * 16
    ring = [dict(gathered=torch.zeros((M, nbytes), dtype=torch.uint8, device=DEV),
                 amaxes=torch.zeros(M, dtype=torch.int32, device=DEV)) for _ in range(D)]
    h["delta_prev_local"] = h["delta_prev_local"].reshape(D, M, stride)
    h["delta_prev_avg"] = h["delta_prev_avg"].reshape(D, stride)
    hv = 0
    for k in range(2 * D + 2):
        if k:
            inputs.inner_phase_standin(st)
            h["theta"], h["master"] = to_numpy(st["theta"]), to_numpy(st["master"])
        slot = ring[k % D]
        new = dict(gathered=torch.zeros_like(slot["gathered"]), amaxes=torch.zeros_like(slot["amaxes"]))
        d_before = h["start"] - (h["master"] if theta_kind == 2 else
                                 (h["theta"] if theta_kind == 0 else
                                  torch.tensor(h["theta"].view(np.int16)).view(torch.bfloat16).float().numpy()))
        for m in range(M):                                  # "send" phase of every worker
            if variant == 0:
                states[m].worker_quantized_send(X, Y, new["gathered"][m], new["amaxes"][m:m + 1])
            else:
                states[m].worker_quantized_apply(variant, M, X, Y, slot["gathered"] if hv >= D else None,
                                                 slot["amaxes"] if hv >= D else None, new["gathered"][m],
                                                 new["amaxes"][m:m + 1])
        if variant == 0:
            for m in range(M):
                states[m].worker_quantized_apply(0, M, X, Y, new["gathered"], new["amaxes"], None, None)
        ring[k % D] = new
        torch.cuda.synchronize()
        # wire bytes against the oracle's encoder
        for m in range(M):
            want, amax = oracle.wire_encode(np.ascontiguousarray(d_before[m, :P]), X, Y)
            got = new["gathered"][m].cpu().numpy()
            np.testing.assert_array_equal(got[:len(want)], want)
            assert new["amaxes"][m].cpu().numpy().view(np.float32) == np.float32(amax)
        hv = oracle.outer_step_overlap(variant, k, hv, M=M, P=P, stride=stride, eta=0.7, mu=0.9, theta=h["theta"],
                                       master=h["master"], start=h["start"], outer_mom=h["outer_mom"],
                                       delta_prev_local=h["delta_prev_local"], delta_prev_avg=h["delta_prev_avg"],
                                       theta_kind=theta_kind, comm=oracle.COMM_EXMY, exp_bits=X, man_bits=Y)
        got = dict(theta=st["theta"], master=st["master"], start=st["start"], outer_mom=st["outer_mom"])
        assert_state_equal(got, h, keys=tuple(got), what=f"quantised wire {fmt} variant {variant} M={M} step {k + 1}")
    for s_ in states:
        s_.close()


def test_worker_argument_checks():
    st = inputs.make_outer_state(2, 1000, 1, device=DEV)
    two = binding.State.from_dict(st)
    buf = torch.zeros(st["stride"], device=DEV)
    with pytest.raises(binding.DilocoError) as e:
        two.worker_outer_apply(2, 2, buf, buf)
    assert e.value.status == binding.ERR_BAD_STATE            # the worker form wants one replica per state
    one = binding.State(M=1, P=1000, stride=st["stride"], theta=st["theta"][0], start=st["start"][0],
                        outer_mom=st["outer_mom"][0], delta_prev_local=st["delta_prev_local"][0])
    with pytest.raises(binding.DilocoError) as e:
        one.worker_outer_apply(2, 2, None, buf)               # have_prev = 1: a sum is due
    assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.DilocoError) as e:
        one.worker_outer_apply(2, 0, buf, buf)
    assert e.value.status == binding.ERR_INVALID_ARG
    with pytest.raises(binding.DilocoError) as e:
        one.worker_outer_apply(2, 2, buf, None)
    assert e.value.status == binding.ERR_INVALID_ARG
    torch.cuda.synchronize()


# ------------------------------------------------------------------ two processes, real all-reduce
def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, variant, D, P, H, phases, theta_kind, out_dir, wire=None, backend="gloo"):
    import torch.distributed as dist
    sys.path.insert(0, str(ROOT))
    from paper_2502_12996_b200 import inputs as inp, worker
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    torch.cuda.set_device(0)
    if backend == "nccl":
        os.environ["NCCL_NVLS_ENABLE"] = "0"
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=torch.device("cuda", 0))
    else:
        dist.init_process_group("gloo", rank=rank, world_size=world)
    # every rank draws the same M-replica state from the same seed and keeps its own replica
    st = inp.make_outer_state(world, P, 777, device="cuda:0", theta_kind=theta_kind, with_adam=True, overlap_steps=D)
    stride = st["stride"]
    mine = dict(theta=st["theta"][rank].clone(), start=st["start"][rank].clone(), outer_mom=st["outer_mom"][rank].clone(),
                master=None if st["master"] is None else st["master"][rank].clone(),
                adam_m=st["adam_m"][rank].clone(), adam_v=st["adam_v"][rank].clone(),
                delta_prev_local=torch.zeros((D, stride), device="cuda:0"))
    w = worker.Worker(mine, P=P, stride=stride, world_replicas=world, variant=variant, overlap_steps=D, have_prev=0,
                      theta_kind=theta_kind, grad_kind=theta_kind and 1, H=H, wire=wire)
    gdt = torch.bfloat16 if theta_kind else torch.float32
    for ph in range(phases):
        for _ in range(H):
            g = inp.make_grads(world, P, stride, st["gen"], "cuda:0", 1 if theta_kind else 0)   # same draws on every rank
            w.inner_adamw(g[rank].contiguous().view(1, -1), 4e-4)
        w.outer_step()
    w.finish()
    torch.cuda.synchronize()
    np.savez(Path(out_dir) / f"rank{rank}.npz", **{k: to_numpy(v) for k, v in mine.items() if v is not None})
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("variant,D,theta_kind,wire,world,backend",
                         [(2, 1, 0, None, 2, "gloo"), (2, 2, 1, None, 2, "gloo"), (1, 1, 0, None, 2, "gloo"),
                          (0, 1, 0, None, 2, "gloo"), (2, 1, 0, (4, 3), 2, "gloo"), (2, 2, 1, (2, 1), 2, "gloo"),
                          (0, 1, 0, (3, 0), 2, "gloo"),
                          # one rank over NCCL: the collectives are trivial, but the Worker's asynchronous
                          # all-reduce / all-gather handles and their stream ordering are NCCL's
                          (2, 1, 0, None, 1, "nccl"), (2, 2, 0, (4, 3), 1, "nccl"), (0, 1, 1, None, 1, "nccl")])
def test_worker_processes_with_async_collectives(oracle, tmp_path, variant, D, theta_kind, wire, world, backend):
    import torch.multiprocessing as mp
    P, H, phases = 60_001, 3, 2 * D + 2
    mp.spawn(_rank_main, args=(world, _free_port(), variant, D, P, H, phases, theta_kind, str(tmp_path), wire, backend),
             nprocs=world, join=True)
    comm_kw = {} if wire is None else dict(comm=oracle.COMM_EXMY, exp_bits=wire[0], man_bits=wire[1])
    # the same run through the fused oracle
    st = inputs.make_outer_state(world, P, 777, device=DEV, theta_kind=theta_kind, with_adam=True, overlap_steps=D)
    stride = st["stride"]
    h = host_copy(st)
    h["delta_prev_local"] = np.zeros((D, world, stride), np.float32)
    h["delta_prev_avg"] = np.zeros((D, stride), np.float32)
    hp = dict(lr=4e-4, beta1=0.9, beta2=0.95, eps=1e-8, wd=0.1)
    have, k = 0, 0
    for ph in range(phases):
        for _ in range(H):
            k += 1
            g = inputs.make_grads(world, P, stride, st["gen"], DEV, 1 if theta_kind else 0)
            oracle.inner_adamw(M=world, P=P, stride=stride, gstride=stride, k=k, theta=h["theta"], grads=to_numpy(g),
                               adam_m=h["adam_m"], adam_v=h["adam_v"], master=h["master"], theta_kind=theta_kind,
                               grad_kind=1 if theta_kind else 0, **hp)
        have = oracle.outer_step_overlap(variant, ph, have, M=world, P=P, stride=stride, eta=0.7, mu=0.9,
                                         theta=h["theta"], master=h["master"], start=h["start"], outer_mom=h["outer_mom"],
                                         delta_prev_local=h["delta_prev_local"], delta_prev_avg=h["delta_prev_avg"],
                                         theta_kind=theta_kind, **comm_kw)
    for r in range(world):
        z = np.load(tmp_path / f"rank{r}.npz")
        for key in ("theta", "start", "outer_mom", "adam_m", "adam_v"):
            want = h[key][r]
            assert (z[key].view(np.uint32 if z[key].dtype == np.float32 else np.uint16) ==
                    want.view(np.uint32 if want.dtype == np.float32 else np.uint16)).all(), (r, key)
