"""The time-sharded cycle schedule on CPU: two (and three) gloo ranks, each owning a contiguous piece of the time
axis, exchange one [B, H] slab per hand-off; the assembled result must equal the single-process oracle cycle to
rounding, forward and adjoint, F- and FCF-relaxation, two and three levels.  The step functions are the oracle's
(injected: the schedule itself holds no arithmetic)."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _problem(T, B=2, I=3, H=5):
    rng = np.random.default_rng(77)
    k = 1.0 / np.sqrt(H)
    P = (rng.uniform(-k, k, (3 * H, I)), rng.uniform(-k, k, (3 * H, H)), rng.uniform(-k, k, 3 * H), rng.uniform(-k, k, 3 * H))
    return P, rng.standard_normal((T, B, I)), rng.standard_normal((B, H)) * 0.4, rng.standard_normal((T, B, H))


def _worker(rank, world, port, case, out):
    sys.path.insert(0, ROOT)
    from oracle import mgrit_gru_oracle as O
    from paper_2203_04738_b200.time_shard import TorchComm, partition, sharded_cycle
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    T, cf, levels, relax, iters = case
    P, x, h0, seed = _problem(T)
    gi = x @ P[0].T + P[2]
    hs = O.serial_forward(*P, x, h0)
    hfull = np.concatenate([h0[None], hs], 0)
    comm = TorchComm()
    parts = partition(T, cf, levels, rank, world)

    def fwd_step(l, j, u_prev):
        m = cf ** l
        return torch.from_numpy(O.phi(P[1], P[3], gi[m * j.numpy() - 1], u_prev.numpy(), float(m), O.CELL_IMPLICIT))

    def adj_step(l, s, mu_prev):
        m = cf ** l
        res = []
        for q, sq in enumerate(s.numpy()):
            t = T - m * (int(sq) - 1)
            a, c_r, c_z, c_n, _ = O.adjoint_coefficients(P[1], P[3], gi[t - 1], hfull[t - m], float(m), O.CELL_IMPLICIT)
            mp_ = mu_prev[q].numpy()
            res.append(a * mp_ + np.concatenate([c_r * mp_, c_z * mp_, c_n * mp_], -1) @ P[1])
        return torch.from_numpy(np.stack(res))

    results = {}
    for name, step in (("fwd", fwd_step), ("adj", adj_step)):
        p0 = parts[0]
        u = [torch.zeros((p0.n_local + 1,) + h0.shape, dtype=torch.float64)] + [None] * (levels - 1)
        g = [torch.zeros_like(u[0])] + [None] * (levels - 1)
        if name == "fwd":
            if rank == 0:
                u[0][0] = torch.from_numpy(h0)
        else:
            if rank == 0:
                u[0][0] = torch.from_numpy(seed[T - 1])
            for i in range(1, p0.n_local + 1):                  # source at reversed point s = first + i: dh_seed[T - s - 1]
                sg = p0.first + i
                if sg < T:
                    g[0][i] = torch.from_numpy(seed[T - sg - 1])
        res2 = []
        for _ in range(iters):
            sharded_cycle(step, cf, [relax] * levels, parts, u, g, comm, 0, res2)
        own = u[0][1:].numpy()
        gathered = [None] * world
        dist.all_gather_object(gathered, (own, res2))
        results[name] = (np.concatenate([o for o, _ in gathered], 0), np.sqrt(np.sum([r for _, r in gathered], axis=0)))
    out[rank] = (results, comm.slabs_sent)
    dist.destroy_process_group()


@pytest.mark.parametrize("world,case", [(2, (32, 4, 2, 0, 2)), (2, (32, 2, 3, 1, 2)), (3, (48, 4, 2, 1, 1)), (2, (64, 4, 3, 2, 2))])
def test_sharded_cycle_equals_single_process_cycle(world, case):
    sys.path.insert(0, ROOT)
    from oracle import mgrit_gru_oracle as O
    T, cf, levels, relax, iters = case
    port = _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, case, out), nprocs=world, join=True)
        res = dict(out)
    P, x, h0, seed = _problem(T)
    kw = dict(cf=cf, levels=levels, iters=iters, relax_fine=relax, relax_coarse=relax)
    href, rref = O.mgrit_forward(*P, x, h0, **kw)
    hs = O.serial_forward(*P, x, h0)
    lam, lam0, _, rref_a = O.mgrit_adjoint(*P, x, h0, hs, seed, **kw)
    mu_ref = np.concatenate([lam[::-1][1:], lam0[None]], 0)          # mu_1 .. mu_T
    for r in range(world):
        results, _ = res[r]
        assert np.max(np.abs(results["fwd"][0] - href)) < 1e-14
        assert np.max(np.abs(results["fwd"][1] - np.array(rref))) < 1e-13
        assert np.max(np.abs(results["adj"][0] - mu_ref)) < 1e-13
        assert np.max(np.abs(results["adj"][1] - np.array(rref_a))) < 1e-12
    # hand-offs: per cycle and non-coarsest level one slab after every C-relaxation and one after the correction, plus
    # one for the coarsest sweep; the last rank sends none
    per_cycle = (levels - 1) * (relax + 1) + 1
    assert res[0][1] == 2 * iters * per_cycle and res[world - 1][1] == 0


def test_partition_is_nested_and_complete():
    sys.path.insert(0, ROOT)
    from paper_2203_04738_b200.time_shard import partition
    T, cf, levels, world = 128, 4, 3, 4
    for l in range(levels):
        blocks = [partition(T, cf, levels, r, world)[l] for r in range(world)]
        assert blocks[0].first == 0 and blocks[-1].last == T // cf ** l
        assert all(a.last == b.first for a, b in zip(blocks, blocks[1:]))
        assert all(b.n_local % cf == 0 or l == levels - 1 for b in blocks)
    with pytest.raises(ValueError):
        partition(128, 4, 3, 0, 16)          # 8 coarsest points for 16 ranks
