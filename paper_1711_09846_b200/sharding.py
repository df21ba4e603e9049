"""A population sharded over several GPUs, one process and one library handle per GPU.

Members are independent between ready points (Algorithm 1: every member steps on its own record), so a shard
trains its members with no communication at all.  A ready point needs two exchanges, and they take the place of the
shared store through which the paper's workers publish their performance and fetch each other's checkpoints
(Appendix A.1):

  1. the fitness vector p[N] and the hyperparameters h[N][nh] are all-gathered (a few KB); every shard then runs
     the same selection / explore kernel on the whole population's vectors and reaches the same copy map src[N];
  2. a recipient whose donor lives on another shard receives the donor's slabs (weights, optimiser state, shadow,
     Adam's running products) straight into its own slabs in its own GPU's memory, by point-to-point send / receive;
     recipients whose donor is local are copied by the shard's own slab-copy kernel.

Everything drawn per member is keyed by the member's index in the whole population, so the sharded run takes the
steps, decisions and copies of the unsharded one, bit for bit.

This module is host logic only: the partition, the copy plan, and the two exchanges over `torch.distributed`
(NCCL between GPUs, gloo between CPU processes in the tests).  No kernel ever reads another GPU's memory.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, Dict, List, Sequence, Tuple

import numpy as np


# ----------------------------------------------------------------------------------------------------------------
# partition
# ----------------------------------------------------------------------------------------------------------------
def member_range(rank: int, world: int, n: int) -> Tuple[int, int]:
    """[first, last) of the members rank `rank` holds: contiguous blocks, the first n % world ranks one longer."""
    assert 0 <= rank < world and n >= 0
    q, r = divmod(n, world)
    first = rank * q + min(rank, r)
    return first, first + q + (1 if rank < r else 0)


def owner_of(member: int, world: int, n: int) -> int:
    q, r = divmod(n, world)
    cut = r * (q + 1)
    if member < cut:
        return member // (q + 1)
    return r + (member - cut) // q if q else world - 1


# ----------------------------------------------------------------------------------------------------------------
# copy plan
# ----------------------------------------------------------------------------------------------------------------
@dataclass
class CopyPlan:
    """What each rank does with a copy map src[N] (src[b] == b: member b keeps its record), pass by pass.

    A recipient's `level` is its copy pass: under truncation selection every recipient has level 0; under the
    tournament rule a donor that is itself a recipient has a higher level than the members that read it, so going
    through the levels in order makes every copy read the donor's record as it was before the ready point.
    Entries are (recipient, donor) in population indices, sorted by recipient, so that the send list of one rank and
    the receive list of its peer enumerate the same transfers in the same order."""
    world: int
    n: int
    n_levels: int
    local: Dict[Tuple[int, int], List[Tuple[int, int]]] = field(default_factory=dict)   # (rank, level) -> pairs
    send: Dict[Tuple[int, int], List[Tuple[int, int]]] = field(default_factory=dict)    # on the donor's rank
    recv: Dict[Tuple[int, int], List[Tuple[int, int]]] = field(default_factory=dict)    # on the recipient's rank

    @staticmethod
    def from_copy_map(src: Sequence[int], level: Sequence[int], world: int) -> "CopyPlan":
        n = len(src)
        pairs = [(b, int(src[b]), int(level[b])) for b in range(n) if int(src[b]) != b]
        plan = CopyPlan(world=world, n=n, n_levels=(max(l for _, _, l in pairs) + 1) if pairs else 0)
        for b, d, l in pairs:                                        # already sorted by recipient
            assert 0 <= d < n and l >= 0
            rb, rd = owner_of(b, world, n), owner_of(d, world, n)
            if rb == rd:
                plan.local.setdefault((rb, l), []).append((b, d))
            else:
                plan.send.setdefault((rd, l), []).append((b, d))
                plan.recv.setdefault((rb, l), []).append((b, d))
        # within a pass nobody is overwritten and read at once
        for l in range(plan.n_levels):
            rec = {b for b, _, ll in pairs if ll == l}
            don = {d for _, d, ll in pairs if ll == l}
            assert not (rec & don), "a member is donor and recipient in the same copy pass"
        return plan

    def crossing(self) -> int:
        """Number of records that cross shards."""
        return sum(len(v) for v in self.send.values())


# ----------------------------------------------------------------------------------------------------------------
# exchanges
# ----------------------------------------------------------------------------------------------------------------
def all_gather_rows(local, world: int, n: int, group=None):
    """Concatenation over ranks of each rank's rows (rank r contributes the rows of member_range(r)): the same
    array on every rank.  `local` is a torch tensor [n_local, ...]; ranks may hold different numbers of rows."""
    import torch
    import torch.distributed as dist
    if world == 1:
        return local.clone()
    longest = member_range(0, world, n)[1] - member_range(0, world, n)[0]
    pad = torch.zeros((longest,) + tuple(local.shape[1:]), dtype=local.dtype, device=local.device)
    pad[:local.shape[0]] = local
    parts = [torch.empty_like(pad) for _ in range(world)]
    dist.all_gather(parts, pad, group=group)
    out = []
    for r in range(world):
        a, b = member_range(r, world, n)
        out.append(parts[r][:b - a])
    return torch.cat(out, dim=0)


def exchange_level(plan: CopyPlan, rank: int, level: int, slabs_of: Callable[[int], list], group=None) -> int:
    """The transfers of one copy pass that involve `rank`: sends the arrays of its donors, receives into the arrays
    of its recipients (in place: within a pass no recipient is read by anybody).  slabs_of(member) returns the list
    of tensors of a local member's record (population index in, same order on every rank).  Returns the number of
    point-to-point operations posted; they are complete when the call returns."""
    import torch.distributed as dist
    ops = []
    sends = plan.send.get((rank, level), [])
    recvs = plan.recv.get((rank, level), [])
    # one global order (by recipient) on both sides of every pair of ranks
    todo = sorted([(b, d, "s") for b, d in sends] + [(b, d, "r") for b, d in recvs])
    for b, d, kind in todo:
        if kind == "s":
            peer = owner_of(b, plan.world, plan.n)
            ops += [dist.P2POp(dist.isend, t, peer, group=group) for t in slabs_of(d)]
        else:
            peer = owner_of(d, plan.world, plan.n)
            ops += [dist.P2POp(dist.irecv, t, peer, group=group) for t in slabs_of(b)]
    if ops:
        for req in dist.batch_isend_irecv(ops):
            req.wait()
    return len(ops)


# ----------------------------------------------------------------------------------------------------------------
# the sharded population
# ----------------------------------------------------------------------------------------------------------------
class ShardedPopulation:
    """One rank's view of a population of cfg.n_members members sharded over `world` ranks.

    step() and eval() are local.  ready_point() all-gathers p and h, lets the library decide for the whole
    population, and carries out the copy map pass by pass.  `transport` does the two exchanges: the default goes
    through torch.distributed; tests on one GPU pass an in-process transport that serves several shards."""

    def __init__(self, pkg, cfg, inputs, rank: int, world: int, device: str = "cuda:0", transport=None, **kw):
        self.cfg, self.rank, self.world = cfg, rank, world
        self.first, self.last = member_range(rank, world, cfg.n_members)
        self.local = pkg.Population(cfg.replace(n_members=self.last - self.first), inputs, device=device,
                                    member_base=self.first, n_global=cfg.n_members, **kw)
        self.transport = transport if transport is not None else DistTransport(rank, world, cfg.n_members)
        self.last_plan = None

    def step(self, k: int = 1):
        self.local.step(k)

    def eval(self):
        self.local.eval()

    def slabs_of(self, member: int):
        return self.local.member_slabs(member - self.first)

    def decide(self, fitness_all, hparams_all, ready=None, history_all=None) -> CopyPlan:
        """Selection and explore for the whole population on this shard (every shard gets the same answer); the
        rows of this shard's members are applied to its own records.  history_all = (scores [N][10], counts [N]) of
        the whole population, needed by t-test selection.  Returns the copy plan."""
        n = self.cfg.n_members
        if history_all is not None:
            self.local.set_global_history(np.asarray(history_all[0]).reshape(n, -1), np.asarray(history_all[1]).reshape(n))
        src, level, n_levels, _, _ = self.local.exploit_explore_global(
            np.asarray(fitness_all, dtype=np.float64).reshape(n), np.asarray(hparams_all, dtype=np.float64).reshape(n, -1), ready)
        self.last_src = src
        self.last_plan = CopyPlan.from_copy_map(src, level, self.world)
        assert self.last_plan.n_levels <= n_levels
        return self.last_plan

    def ready_point(self, ready=None) -> np.ndarray:
        """eval must have been called.  Returns the copy map of the whole population."""
        import torch
        f = self.transport.all_gather(self, torch.from_numpy(self.local.fitness()))
        h = self.transport.all_gather(self, torch.from_numpy(self.local.hparams()))
        hist = None
        if getattr(self.cfg, "exploit", "truncation") == "ttest":
            hs, hc = self.local.history()
            hist = (self.transport.all_gather(self, torch.from_numpy(hs)).numpy(),
                    self.transport.all_gather(self, torch.from_numpy(hc)).numpy())
        plan = self.decide(f.numpy(), h.numpy(), ready, hist)
        for lv in range(plan.n_levels):
            self.local.copy_members_level(lv)            # local copies of this pass (enqueued on the shard's stream)
            self.transport.exchange(self, plan, lv)      # records that cross shards land in the recipients' slabs
        return self.last_src

    def close(self):
        self.local.close()


class DistTransport:
    """The exchanges over torch.distributed (one process per GPU; NCCL for device tensors, gloo for host tensors)."""

    def __init__(self, rank, world, n, group=None):
        self.rank, self.world, self.n, self.group = rank, world, n, group

    def all_gather(self, shard, local_rows):
        import torch
        dev = shard.local.device if self._device_collectives() else "cpu"
        out = all_gather_rows(local_rows.to(dev), self.world, self.n, self.group)
        return out.cpu()

    def _device_collectives(self) -> bool:
        import torch.distributed as dist
        return self.world > 1 and dist.get_backend(self.group) == "nccl"

    def exchange(self, shard, plan, level):
        import torch
        # the point-to-point kernels must run after the library's kernels already in the shard's stream and before
        # the ones enqueued next: issue them on that stream
        with torch.cuda.stream(shard.local.stream):
            exchange_level(plan, self.rank, level, shard.slabs_of, self.group)


def ready_point_in_process(shards: Sequence[ShardedPopulation], ready=None) -> np.ndarray:
    """The same ready point for shards that are all driven by ONE process (several GPUs, or several shards on one
    GPU): no process group is needed, the vectors are concatenated on the host and a record that crosses shards is
    one device-to-device copy per array from the donor's slab into the recipient's (a peer copy when the shards
    sit on different GPUs).  The passes are taken in order across all shards, so that every copy reads the donor's
    record as it was before the ready point."""
    import torch
    f = np.concatenate([s.local.fitness() for s in shards])
    h = np.concatenate([s.local.hparams() for s in shards], axis=0)
    hist = None
    if getattr(shards[0].cfg, "exploit", "truncation") == "ttest":
        parts = [s.local.history() for s in shards]
        hist = (np.concatenate([p[0] for p in parts], axis=0), np.concatenate([p[1] for p in parts]))
    plans = [s.decide(f, h, ready, hist) for s in shards]
    assert all(np.array_equal(s.last_src, shards[0].last_src) for s in shards), "the shards disagree on the copy map"
    n, world = shards[0].cfg.n_members, len(shards)
    for lv in range(max(p.n_levels for p in plans)):
        for s in shards:
            s.local.synchronize()                        # reads of the previous pass are complete everywhere
        for s in shards:
            s.local.copy_members_level(lv)
            with torch.cuda.stream(s.local.stream):
                for b, d in plans[s.rank].recv.get((s.rank, lv), []):
                    donor = shards[owner_of(d, world, n)]
                    for dst, src_t in zip(s.slabs_of(b), donor.slabs_of(d)):
                        dst.copy_(src_t, non_blocking=True)
    for s in shards:
        s.local.synchronize()
    return shards[0].last_src
