"""Data-parallel QODA across processes (Algorithm 1 lines 12-18 with a real exchange step).

Every rank owns a contiguous range of the K workers: it encodes their dual vectors with the worker-range form of
lq_quantize_pack, the messages (packed words and norms) and the per-(worker, layer) side data travel by
all-gather, and every rank then decodes all K messages and updates its replica of the iterate.  The random numbers
are keyed on the workers' global indices, so the result is bit-identical to one process that holds all K workers.

This module is plumbing only (buffers, torch.distributed calls, call order): every arithmetic step runs in the
library's kernels through the plan's methods.
"""
from __future__ import annotations

from typing import Optional, Tuple

import torch
import torch.distributed as dist


def worker_range(rank: int, world: int, num_workers: int) -> Tuple[int, int]:
    """(first worker, count) of `rank`: equal contiguous shares (all-gather needs equal shares)."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError(f"rank {rank} outside world {world}")
    if num_workers % world != 0:
        raise ValueError(f"{num_workers} workers do not divide evenly over {world} ranks")
    count = num_workers // world
    return rank * count, count


class ExchangeStep:
    """One rank's side of the K-worker iteration.  `plan` is a paper_2505_14371_b200.Plan for all K workers."""

    def __init__(self, plan, rank: int, world: int, group=None, device="cuda"):
        self.plan, self.rank, self.world, self.group = plan, rank, world, group
        self.first, self.count = worker_range(rank, world, plan.num_workers)
        plan.lq_set_worker_range(self.first, self.count)
        self.packed = [plan.empty_packed(device), plan.empty_packed(device)]
        self.norms = [plan.empty_norms(device), plan.empty_norms(device)]
        for t in self.packed + self.norms:
            t.zero_()
        K, L = plan.num_workers, max(plan.num_layers, 1)
        self.sq_diff = torch.zeros((K, L), dtype=torch.float64, device=device)
        self.layer_weight = torch.zeros((K, L), dtype=torch.float32, device=device)
        self.flags = torch.zeros((K, L), dtype=torch.int32, device=device)
        self.have_prev = False
        self.cur = 0

    # -- the exchange: own rows of a [K][...] buffer out, everybody's rows in -------------------------
    def all_gather_rows(self, full: torch.Tensor) -> None:
        if self.world == 1:
            return
        own = full[self.first: self.first + self.count]
        in_place = dist.get_backend(self.group) == "nccl"       # NCCL gathers in place when the input is the
        src = own if in_place else own.clone()                  # rank's own slice of the output
        try:
            dist.all_gather_into_tensor(full, src, group=self.group)
        except (NotImplementedError, RuntimeError):
            if in_place:
                raise
            parts = list(full.chunk(self.world, dim=0))         # views of `full`: the gather lands in place
            dist.all_gather(parts, src, group=self.group)

    def encode(self, local_grads: torch.Tensor, step: int, hist: Optional[torch.Tensor] = None) -> int:
        """ENCODE this rank's workers (local_grads [count][D_pad]) and exchange; returns the buffer index of
        the complete message."""
        if local_grads.shape[0] != self.count:
            raise ValueError(f"expected {self.count} rows of gradients, got {local_grads.shape[0]}")
        c = 1 - self.cur if self.have_prev else self.cur
        p = self.cur
        self.plan.lq_quantize_pack(local_grads, step, self.packed[c], self.norms[c], hist=hist,
                                   prev_packed=self.packed[p] if self.have_prev else None,
                                   prev_norms=self.norms[p] if self.have_prev else None)
        self.plan.lq_side_data_export(self.sq_diff, self.layer_weight, self.flags)
        for buf in (self.packed[c], self.norms[c], self.sq_diff, self.layer_weight, self.flags):
            self.all_gather_rows(buf)
        if hist is not None:
            self.all_gather_rows(hist)
        self.plan.lq_side_data_import(self.sq_diff, self.layer_weight, self.flags)
        self.cur, self.have_prev = c, True
        return c

    def step(self, local_grads: torch.Tensor, step: int, X1, Y, Xhalf, X=None, gbar=None,
             hist: Optional[torch.Tensor] = None) -> None:
        """One iteration: encode + exchange, then DECODE, mean and the QODA update on this replica."""
        c = self.encode(local_grads, step, hist)
        self.plan.qoda_step(self.packed[c], self.norms[c], X1, Y, Xhalf, X, gbar)

    def fit_levels(self, hist: torch.Tensor) -> None:
        """Level update (Algorithm 1 lines 2-7) from the gathered histograms of the last encode; every rank
        computes the same levels."""
        self.plan.lq_fit_levels(hist, self.norms[self.cur], self.plan.num_workers)
