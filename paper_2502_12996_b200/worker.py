"""One DiLoCo worker per process and GPU: the deployment form of Algorithms 1-3.

Each worker holds ONE replica and runs ``diloco_worker_outer_apply`` on it; the only thing
exchanged is the local outer gradient Delta_m, summed over the workers by an all-reduce
(``torch.distributed``; NCCL over NVLink between GPUs of a node).  With the delayed and eager
variants the all-reduce is started asynchronously right after the outer step and is given the
whole next inner phase (H AdamW steps), or ``overlap_steps`` phases, to finish: its result is
consumed ``overlap_steps`` outer steps later, which is the point of the method.  This module
is plumbing (buffers, handles, ordering); all arithmetic runs in the library's kernels.
"""
from __future__ import annotations

from typing import Dict, List, Optional

import torch
import torch.distributed as dist

from . import binding


class Worker:
    """State, communication ring and step bookkeeping of one worker.

    tensors: theta [stride] (fp32 or bf16), start, outer_mom [stride] fp32, master (optional),
    delta_prev_local [overlap_steps, stride] (eager), adam_m / adam_v (optional), all on this
    worker's GPU.  ``initial_sums``: for a run that starts with ``have_prev`` generations already
    recorded, the all-reduced SUMS of those generations, oldest first.
    """

    def __init__(self, tensors: Dict[str, torch.Tensor], *, P: int, stride: int, world_replicas: int,
                 variant: int = binding.EAGER, overlap_steps: int = 1, have_prev: int = 0,
                 initial_sums: Optional[List[torch.Tensor]] = None, process_group=None,
                 state_factory=binding.State, wire: Optional[tuple] = None, **hyper):
        self.variant, self.D, self.M = variant, int(overlap_steps), int(world_replicas)
        self.group = process_group
        self.have = int(have_prev)
        self.k = 0
        dev = tensors["start"].device
        # state_factory exists so that the plumbing below can be exercised without a GPU
        # (a stand-in with the same worker_outer_send / worker_outer_apply / inner_adamw methods)
        self.state = state_factory(M=1, P=P, stride=stride, theta=tensors["theta"], master=tensors.get("master"),
                                   start=tensors["start"], outer_mom=tensors["outer_mom"],
                                   delta_prev_local=tensors.get("delta_prev_local"), adam_m=tensors.get("adam_m"),
                                   adam_v=tensors.get("adam_v"), have_prev=self.have, overlap_steps=self.D, **hyper)
        # slot k mod (D+1) carries outer step k's Delta: filled by the kernel, summed in place by
        # the all-reduce, read D steps later; D+1 slots so that the slot being filled is never
        # the one being read
        self.ring = [torch.zeros(stride, dtype=torch.float32, device=dev) for _ in range(self.D + 1)]
        self.pending: Dict[int, object] = {}
        # quantised wire (exp_bits, man_bits): the workers exchange EXMY codes + one fp32 word
        # by all-gather; slot k keeps what this worker sent and everything it gathered
        self.wire = wire
        if wire is not None:
            if self.have:
                raise ValueError("a quantised run starts with have_prev = 0")
            nbytes = (binding.wire_payload_bytes(P, *wire) + 15) // 16 * 16
            u8, i32 = dict(dtype=torch.uint8, device=dev), dict(dtype=torch.int32, device=dev)
            self.qring = [dict(send=torch.zeros(nbytes, **u8), amax=torch.zeros(1, **i32),
                               gathered=torch.zeros((self.M, nbytes), **u8), amaxes=torch.zeros(self.M, **i32))
                          for _ in range(self.D + 1)]
        if self.have:
            if initial_sums is None or len(initial_sums) != self.have:
                raise ValueError("have_prev generations need their all-reduced sums")
            for j, t in enumerate(initial_sums):            # generation of outer step (j - have)
                self.ring[(j - self.have) % (self.D + 1)].copy_(t)

    def inner_adamw(self, grads: torch.Tensor, lr: float) -> None:
        self.state.inner_adamw(grads, lr, grad_stride=grads.shape[-1])

    def _all_reduce(self, t: torch.Tensor, async_op: bool):
        return dist.all_reduce(t, op=dist.ReduceOp.SUM, group=self.group, async_op=async_op)

    def _all_gather(self, slot: dict, async_op: bool):
        works = [dist.all_gather_into_tensor(slot["gathered"].view(-1), slot["send"], group=self.group, async_op=async_op),
                 dist.all_gather_into_tensor(slot["amaxes"], slot["amax"], group=self.group, async_op=async_op)]
        return works if async_op else None

    def _outer_step_quantized(self) -> None:
        k, D, (X, Y) = self.k, self.D, self.wire
        if self.variant == binding.STANDARD:
            slot = self.qring[0]
            self.state.worker_quantized_send(X, Y, slot["send"], slot["amax"])
            self._all_gather(slot, async_op=False)
            self.state.worker_quantized_apply(binding.STANDARD, self.M, X, Y, slot["gathered"], slot["amaxes"], None, None)
        else:
            mine = self.qring[k % (D + 1)]
            due = None
            if self.have >= D:
                for work in self.pending.pop(k - D, ()):
                    work.wait()
                due = self.qring[(k - D) % (D + 1)]
            self.state.worker_quantized_apply(self.variant, self.M, X, Y, None if due is None else due["gathered"],
                                              None if due is None else due["amaxes"], mine["send"], mine["amax"])
            self.pending[k] = self._all_gather(mine, async_op=True)
            self.have = min(D, self.have + 1)
        self.k += 1

    def outer_step(self) -> None:
        if self.wire is not None:
            return self._outer_step_quantized()
        k, D = self.k, self.D
        if self.variant == binding.STANDARD:
            # Algorithm 1: send, block on the all-reduce (line 9), apply
            buf = self.ring[0]
            self.state.worker_outer_send(buf)
            self._all_reduce(buf, async_op=False)
            self.state.worker_outer_apply(binding.STANDARD, self.M, buf, None)
        else:
            send = self.ring[k % (D + 1)]
            recv = None
            if self.have >= D:
                work = self.pending.pop(k - D, None)
                if work is not None:
                    work.wait()                               # block-receive of Delta^(t-DH)
                recv = self.ring[(k - D) % (D + 1)]
            self.state.worker_outer_apply(self.variant, self.M, recv, send)
            self.pending[k] = self._all_reduce(send, async_op=True)   # async-send, hidden behind the next phase
            self.have = min(D, self.have + 1)
        self.k += 1

    def finish(self) -> None:
        """Wait for the all-reduces still in flight (end of training)."""
        for work in self.pending.values():
            for w in (work if isinstance(work, (list, tuple)) else (work,)):
                w.wait()
        self.pending.clear()

    def close(self) -> None:
        self.finish()
        self.state.close()
