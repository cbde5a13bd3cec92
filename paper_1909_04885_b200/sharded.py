"""One CoCoA job over several ranks: the partitions spread over the ranks, the shared vector replicated.

Paper Sec. 4.2 ("Trainer and solver") and the Appendix's example application: every iteration each solver hands its
model update to the trainer, which merges them and broadcasts the model; Sec. 4.3: the exchange is one model-sized
vector per task and iteration. Here every rank holds a handle over the same data with the same partition (same K and
seed on every rank, so the owner map is the one a single rank would compute) and

    round:  rank g runs the local solvers of the partitions {k : k mod G = g}, all others sit the round out;
            the ranks all-gather their summed updates (dim floats each);
            every rank adds the G vectors to its v in rank order with an fp64 accumulator
            (the same vectors in the same order on every rank: the replicas of v stay equal bit for bit);
    state:  a coordinate's alpha is current only on the rank that owns its partition; before the duality gap, a read of
            alpha or a new partition the ranks sum their owned parts (one non-zero term per coordinate: exact).

This module is host-side policy only (who owns what, what is exchanged, in which order); every arithmetic step runs
behind the `backend` object: `GlmBackend` (the CUDA library through its C ABI, tensors on the GPU, NCCL) in
production. The collective is `torch.distributed`'s; no kernel of the library ever reads another GPU's memory.
"""
from __future__ import annotations

from typing import Optional

import numpy as np


def owned_partitions(K: int, rank: int, world: int) -> np.ndarray:
    """Flags of the partitions that `rank` runs: k mod world == rank."""
    if not (0 <= rank < world):
        raise ValueError("rank must lie in [0, world)")
    return (np.arange(K) % world == rank).astype(np.uint8)


def shard_budgets(sizes, rank: int, world: int, H: int = 0, steps=None) -> np.ndarray:
    """Step budgets of one round on `rank`: what the partition would take on a single rank (its size for H = 0, else
    min(H, size); or steps[k]) for the partitions the rank owns, 0 for the others."""
    sizes = np.asarray(sizes, np.int64)
    if steps is not None:
        want = np.asarray(steps, np.int64)
        if want.size != sizes.size:
            raise ValueError("steps must have K entries")
    elif H == 0:
        want = sizes
    else:
        if H > sizes.min():
            raise ValueError("a sharded round takes at most one local epoch: H must not exceed the smallest partition")
        want = np.full_like(sizes, H)
    return np.where(owned_partitions(sizes.size, rank, world) != 0, want, 0).astype(np.int64)


class Comm:
    """The two collectives the job needs, over a torch.distributed process group (None: a single rank)."""

    def __init__(self, dist=None, group=None):
        self.dist, self.group = dist, group
        self.world = 1 if dist is None else dist.get_world_size(group)
        self.rank = 0 if dist is None else dist.get_rank(group)

    def all_gather(self, t):
        """A (world, len) tensor holding every rank's `t`, rank order."""
        import torch
        out = torch.empty((self.world, t.numel()), dtype=t.dtype, device=t.device)
        if self.dist is None:
            out[0].copy_(t)
        else:
            self.dist.all_gather_into_tensor(out.view(-1), t.contiguous().view(-1), group=self.group)
        return out

    def all_reduce_sum(self, t):
        if self.dist is not None:
            self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM, group=self.group)
        return t


class GlmBackend:
    """The CUDA library as the compute side of a sharded job: a `binding.Glm` plus device buffers for the exchange."""

    def __init__(self, glm):
        import torch
        self.glm = glm
        self.device = torch.device("cuda", glm.device)
        self.last_stats = None
        self._delta = torch.empty(glm.dim, dtype=torch.float32, device=self.device)
        self._state = torch.empty(glm.n_coord, dtype=torch.float32, device=self.device)

    def partition(self, K: int, seed: int):
        self.glm.partition(K, seed)

    def partition_sizes(self) -> np.ndarray:
        return np.bincount(self.glm.get_partition(), minlength=self.glm.K).astype(np.int64)

    def round_delta(self, budgets, sigma_prime: float, stats: bool = False):
        self.last_stats = self.glm.cocoa_round_delta(budgets, sigma_prime, self._delta, stats=stats)
        return self._delta

    def apply_deltas(self, stacked):
        self.glm.apply_deltas(stacked)

    def export_state_of(self, keep):
        self.glm.export_state_of(keep, self._state)
        return self._state

    def import_state(self, state):
        self.glm.import_state(state)

    def duality_gap(self):
        return self.glm.duality_gap()

    def sync(self):
        """The library's calls are enqueued on the handle's stream; the collective runs on torch's: order them."""
        import torch
        torch.cuda.synchronize(self.device)


class ShardedGlm:
    """The job as one rank sees it. `backend` does the arithmetic (see GlmBackend for the methods it needs); `comm`
    is a `Comm`. All ranks make the same calls in the same order."""

    def __init__(self, backend, comm: Optional[Comm] = None):
        self.backend = backend
        self.comm = comm or Comm()
        self.rank, self.world = self.comm.rank, self.comm.world
        self.K = 0
        self.sizes = None
        self._state_current = True  # every rank holds the whole per-coordinate state

    def partition(self, K: int, seed: int):
        """A new partition (elastic K between rounds): the state is collected first, because ownership changes."""
        self.sync_state()
        self.backend.partition(K, seed)
        self.K = K
        self.sizes = self.backend.partition_sizes()

    def cocoa_round(self, H: int = 0, sigma_prime: Optional[float] = None, steps=None, stats: bool = False):
        """One round of the whole job. `stats`: returns this rank's round statistics (a backend that keeps them)."""
        if self.K <= 0:
            raise RuntimeError("partition first")
        sp = float(self.K if sigma_prime is None else sigma_prime)
        budgets = shard_budgets(self.sizes, self.rank, self.world, H, steps)
        delta = self.backend.round_delta(budgets, sp, stats=True) if stats else self.backend.round_delta(budgets, sp)
        self.backend.sync()
        stacked = self.comm.all_gather(delta)
        self.backend.apply_deltas(stacked)
        self.backend.sync()  # `stacked` must outlive the kernel that reads it
        self._state_current = self.world == 1
        return getattr(self.backend, "last_stats", None) if stats else None

    def sync_state(self):
        """Every rank receives the per-coordinate state of the coordinates it does not own."""
        if self._state_current or self.K <= 0:
            return
        mine = self.backend.export_state_of(owned_partitions(self.K, self.rank, self.world))
        self.backend.sync()
        whole = self.comm.all_reduce_sum(mine)
        self.backend.import_state(whole)
        self.backend.sync()
        self._state_current = True

    def duality_gap(self):
        """The gap of the whole job, computed by every rank from its replica (the same value on all ranks)."""
        self.sync_state()
        return self.backend.duality_gap()
