"""Time-sharded multigrid cycle: the host-side schedule of the paper's distribution (Fig. "Parallel distribution of
work in parallel-in-time training"; Section "Multi-grid in Time": every processor owns a contiguous piece of the time
axis, the coarsest level is propagated serially).

What is here is the partition and the hand-off schedule only -- which rank owns which points of which level, and when
one [B, H] slab crosses a rank boundary -- written over two injected callables:

  step(l, j, u_prev) -> values at the level-l points j (global indices) from their predecessors' states,
  comm: an object with ``rank``, ``world``, ``send_right(tensor)``, ``recv_left(like)``  (torch.distributed
        send/recv in `TorchComm`; NCCL on GPUs, gloo on CPUs).

No arithmetic of the method lives in this module.  `DeviceSteps` supplies the two callables on a GPU through the
library's row-wise calls (gru_step_rows / gru_adjoint_step_rows), so that each rank advances its own points on its own
device and `TorchComm` moves the slabs over NCCL.  Only one device is available per run here, so the schedule is
exercised with two and three CPU ranks over gloo (tests/test_time_shard_gloo.py) and the device steps with one rank on
one GPU against the library's own single-device solve (tests/test_gpu_time_shard.py).

Ownership: level l has points 0..N_l and intervals of c_f points.  Rank r owns a contiguous block of whole intervals,
i.e. the F-points of those intervals and the C-point that ENDS each of them; point 0 (the fixed end) and, for r > 0,
the C-point ending the left neighbour's last interval are kept as a read-only halo in local slot 0.  F-relaxation,
residual evaluation, restriction and the FAS right-hand side then need no communication; exactly one slab goes to the
right neighbour whenever a rank's last C-point has changed (after a C-relaxation and after the correction), and the
coarsest level is swept rank after rank, each waiting for its left neighbour's last value (a pipeline: the serial
cost of that level, as in the paper).
"""
from __future__ import annotations

from dataclasses import dataclass

import torch


class TorchComm:
    """Neighbour hand-off over torch.distributed (process group initialised by the caller)."""

    def __init__(self):
        import torch.distributed as dist
        self.dist = dist
        self.rank, self.world = dist.get_rank(), dist.get_world_size()
        self.slabs_sent = 0

    def send_right(self, t: torch.Tensor) -> None:
        if self.rank + 1 < self.world:
            self.dist.send(t.contiguous(), dst=self.rank + 1)
            self.slabs_sent += 1

    def recv_left(self, like: torch.Tensor) -> torch.Tensor | None:
        if self.rank == 0:
            return None
        buf = torch.empty_like(like)
        self.dist.recv(buf, src=self.rank - 1)
        return buf


class LocalComm:
    """world = 1: nothing to hand off."""
    rank, world, slabs_sent = 0, 1, 0

    def send_right(self, t):
        pass

    def recv_left(self, like):
        return None


class DeviceSteps:
    """The two step callables of `sharded_cycle` on this rank's GPU (argument marshalling around the C-ABI calls).

    gi: [T, B, 3H] input projection (device); hfull: [T + 1, B, H] = [h_0; h], the states the adjoint is linearised at
    (needed for `adj` only).  Level l advances with gamma = cf^l * dt and uses the input of the fine step that arrives at
    the same time."""

    def __init__(self, binding, cfg, params, gi, hfull=None):
        self.B, self.cfg, self.p, self.gi, self.hfull = binding, cfg, params, gi, hfull

    def fwd(self, l, j, u_prev):
        m = self.cfg.cf ** l
        rows = self.gi[(m * j - 1).to(self.gi.device)].contiguous()
        return self.B.gru_step_rows(self.cfg, self.p, float(m) * self.cfg.dt, rows, u_prev.contiguous())

    def adj(self, l, s, mu_prev):
        # reversed point s of level l: the forward step that arrives at fine time t = T - m (s - 1) and leaves t - m
        m, T = self.cfg.cf ** l, self.cfg.T
        t = (T - m * (s - 1)).to(self.gi.device)
        return self.B.gru_adjoint_step_rows(self.cfg, self.p, float(m) * self.cfg.dt, self.gi[t - 1].contiguous(),
                                            self.hfull[t - m].contiguous(), mu_prev.contiguous())


@dataclass
class LevelPart:
    """Rank-local view of one level: owned global points first+1 .. last (first = global index held in slot 0)."""
    N: int          # global number of points after point 0
    first: int      # global index of local slot 0 (the halo / fixed end)
    last: int       # global index of the last owned point

    @property
    def n_local(self) -> int:
        return self.last - self.first


def partition(T: int, cf: int, levels: int, rank: int, world: int) -> list[LevelPart]:
    """Contiguous blocks of whole intervals per rank on every level, nested: a rank's coarse points are the C-points it
    owns on the level above.  Needs T divisible by cf^(levels-1) and at least one coarsest point per rank (the paper
    finds no gain below a few time steps per processor either)."""
    if T % (cf ** (levels - 1)) != 0:
        raise ValueError("T must be divisible by cf^(levels-1)")
    if T // cf ** (levels - 1) < world:
        raise ValueError("fewer coarsest-level points than ranks")
    parts = []
    # split the COARSEST level's points evenly, then refine: a rank owns on level l exactly the points that coarsen
    # into its points of level l+1 (cf per coarse point)
    Nc = T // cf ** (levels - 1)
    lo, hi = (rank * Nc) // world, ((rank + 1) * Nc) // world
    for l in range(levels - 1, -1, -1):
        parts.append(LevelPart(T // cf ** l, lo, hi))
        lo, hi = lo * cf, hi * cf
    return parts[::-1]


def sharded_cycle(step, cf: int, relax: list[int], parts: list[LevelPart], u: list, g: list, comm, l: int = 0, res2: list | None = None):
    """One V-cycle (Algorithm "MGProp" with the recursive coarse solve) on this rank's share of level l and below.

    u[l], g[l]: local tensors [n_local + 1, ...], slot i = global point parts[l].first + i; slot 0 is the halo.
    res2: if given, this rank's share of the squared level-0 residual norm is appended (sum over ranks = the norm^2).
    """
    P, ul, gl = parts[l], u[l], g[l]
    n = P.n_local
    gidx = lambda i: P.first + i          # global index of local slot i

    def refresh_halo():
        # my last owned point has changed: the right neighbour's slot 0 must follow
        if n > 0:
            comm.send_right(ul[n])
        got = comm.recv_left(ul[0])          # every rank owns points on every level (partition() checks it)
        if got is not None:
            ul[0] = got

    if l == len(parts) - 1:
        # coarsest level: serial propagation, rank after rank
        got = comm.recv_left(ul[0])
        if got is not None:
            ul[0] = got
        for i in range(1, n + 1):
            ul[i] = step(l, torch.tensor([gidx(i)]), ul[i - 1:i])[0] + gl[i]
        comm.send_right(ul[n])
        return

    nint = n // cf                         # owned intervals

    def f_relax():
        for s in range(1, cf):
            i = torch.arange(0, n, cf) + s
            if len(i):
                ul[i] = step(l, i + P.first, ul[i - 1]) + gl[i]

    def c_relax():
        i = cf * torch.arange(1, nint + 1)
        if len(i):
            ul[i] = step(l, i + P.first, ul[i - 1]) + gl[i]
        refresh_halo()

    f_relax()
    for _ in range(relax[l]):
        c_relax()
        f_relax()
    ic = cf * torch.arange(1, nint + 1)
    if len(ic):
        v = step(l, ic + P.first, ul[ic - 1]) + gl[ic]
        r = ul[ic] - v
        if res2 is not None and l == 0:
            res2.append(float((r * r).sum()))
    elif res2 is not None and l == 0:
        res2.append(0.0)
    # restriction by injection; the coarse halo is the fine halo (both are the left neighbour's last C-point)
    Pc = parts[l + 1]
    Uc = torch.cat([ul[0:1], ul[ic]], dim=0) if len(ic) else ul[0:1].clone()
    Gc = torch.zeros_like(Uc)
    if len(ic):
        kc = torch.arange(1, nint + 1)
        Gc[kc] = v - step(l + 1, kc + Pc.first, Uc[kc - 1])
    u[l + 1], g[l + 1] = Uc, Gc
    sharded_cycle(step, cf, relax, parts, u, g, comm, l + 1, res2)
    if len(ic):
        ul[ic] = u[l + 1][1:]
    refresh_halo()                         # the correction changed every C-point, the rank's last one included
    f_relax()
