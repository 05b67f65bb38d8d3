"""Host-side plan of the sharded (one process per GPU) layout of the SAT epoch: who owns what, who sends what to whom.

Partition-parallel training places the M subgraphs on G GPUs (Preliminaries, "Distributed Training for GNNs"; Algorithm 1
"for m in parallel").  The layout planned here:

  partition m         -> rank m mod G
  cache slot s        -> the rank that owns the partition of the node behind s (every boundary node is an inner node of
                         exactly one partition, so every slot has one owner, which is also the rank that pushes it)
  pull (per epoch and cached layer)   rank r needs the slots its partitions read: the slots of their halo nodes; the slots
                         among them owned by another rank q are one exchange list q -> r (Eq. "communication complexity":
                         the term  sum_m |U N(v) \\ V_m| L d  counts exactly these rows)
  weight gradients    -> all-reduced over the G ranks (the  M L d^2  term)

Only integer bookkeeping lives here: ownership maps and exchange lists, built from the partition lists (as numpy arrays,
e.g. what sat_part_lists / sat_slot_map return) and agreed between the ranks over a torch.distributed process group (any
backend).  On the data path the rows of an exchange list are brought into the reading GPU's own memory first (plain peer
loads or copies, or an all-to-all), and only then read by the kernels: no kernel and no library routine is handed a
pointer into another GPU's memory, and no TMA load uses cluster multicast.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


def owner_of_partition(m: int, world: int) -> int:
    return m % world


@dataclass
class ShardPlan:
    rank: int
    world: int
    parts: list                      # partitions of this rank, ascending
    slot_owner: np.ndarray           # int32 [n_slots]: rank that owns (and pushes) every cache slot
    owned_slots: np.ndarray          # int32: slots owned by this rank, ascending
    need_slots: np.ndarray           # int32: slots this rank's partitions pull (their halo nodes), ascending, unique
    recv: dict = field(default_factory=dict)   # q -> slots this rank receives from rank q (ascending); q != rank
    send: dict = field(default_factory=dict)   # q -> slots this rank sends to rank q (ascending); q != rank

    def pull_rows(self) -> int:
        """Rows that cross between GPUs into this rank per cached layer and epoch."""
        return int(sum(v.shape[0] for v in self.recv.values()))


def local_plan(rank: int, world: int, M: int, part: np.ndarray, slot: np.ndarray, halo_gid_of) -> ShardPlan:
    """What a rank can derive on its own.  part / slot: int32 [n] (partition and cache slot of every node, slot -1 for
    interior nodes); halo_gid_of(m): the halo node ids of partition m (called for this rank's partitions only)."""
    part = np.asarray(part)
    slot = np.asarray(slot)
    n_slots = int(slot.max()) + 1 if slot.size and slot.max() >= 0 else 0
    cached = np.nonzero(slot >= 0)[0]
    slot_owner = np.empty(n_slots, dtype=np.int32)
    slot_owner[slot[cached]] = (part[cached] % world).astype(np.int32)
    parts = [m for m in range(M) if owner_of_partition(m, world) == rank]
    need = [slot[np.asarray(halo_gid_of(m))] for m in parts]
    need_slots = np.unique(np.concatenate(need)).astype(np.int32) if need else np.empty(0, dtype=np.int32)
    plan = ShardPlan(rank=rank, world=world, parts=parts, slot_owner=slot_owner,
                     owned_slots=np.nonzero(slot_owner == rank)[0].astype(np.int32), need_slots=need_slots)
    for q in range(world):
        if q != rank:
            plan.recv[q] = need_slots[slot_owner[need_slots] == q]
    return plan


def exchange_plan(plan: ShardPlan, dist) -> ShardPlan:
    """Tells every owner what this rank needs from it (one all-gather of the request lists over the process group) and
    fills plan.send: the slots this rank owns that rank q pulls.  Collective: every rank of the group must call it."""
    requests = [None] * plan.world
    dist.all_gather_object(requests, {q: v.tolist() for q, v in plan.recv.items()})
    for q in range(plan.world):
        if q != plan.rank:
            want = np.asarray(requests[q].get(plan.rank, []), dtype=np.int32)
            if want.size and not np.all(plan.slot_owner[want] == plan.rank):
                raise ValueError(f"rank {q} asks rank {plan.rank} for slots it does not own")
            plan.send[q] = want
    return plan
