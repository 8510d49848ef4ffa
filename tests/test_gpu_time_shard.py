"""The time-sharded schedule with its steps on the GPU (library calls gru_step_rows / gru_adjoint_step_rows), one rank:
the cycles it drives must reproduce the library's own single-device solve (fp32 engine, same arithmetic per element) and
the fp64 oracle; the row-wise calls themselves are compared with the oracle's cell and its transposed Jacobian."""
import numpy as np
import pytest
import torch

from oracle import mgrit_gru_oracle as O
from paper_2203_04738_b200.synthetic import Workload, make_inputs
from tests.gpu_util import max_abs, oracle_params, rel_inf, to_dev, upload

pytestmark = pytest.mark.gpu


def test_row_calls_against_the_oracle_cell():
    from paper_2203_04738_b200 import binding as B
    rng = np.random.default_rng(3)
    n, Bz, H = 7, 3, 40
    k = 1.0 / np.sqrt(H)
    W_hh, b_hh = rng.uniform(-k, k, (3 * H, H)), rng.uniform(-k, k, 3 * H)
    gi, u, mu = rng.standard_normal((n, Bz, 3 * H)), rng.standard_normal((n, Bz, H)) * 0.5, rng.standard_normal((n, Bz, H))
    p = dict(W_ih=to_dev(np.zeros((3 * H, 8), np.float32)), W_hh=to_dev(W_hh.astype(np.float32)), b_ih=to_dev(np.zeros(3 * H, np.float32)),
             b_hh=to_dev(b_hh.astype(np.float32)))
    f32 = lambda a: to_dev(a.astype(np.float32))
    for cell in (0, 1):
        for gamma in (1.0, 4.0):
            cfg = B.make_cfg(8, Bz, 8, H, cf=2, levels=1, cell=cell)
            out = B.gru_step_rows(cfg, p, gamma, f32(gi), f32(u))
            assert max_abs(out.cpu().numpy(), O.phi(W_hh, b_hh, gi, u, gamma, cell)) < 1e-5
            a, c_r, c_z, c_n, _ = O.adjoint_coefficients(W_hh, b_hh, gi, u, gamma, cell)
            ref = a * mu + np.concatenate([c_r * mu, c_z * mu, c_n * mu], -1) @ W_hh
            got = B.gru_adjoint_step_rows(cfg, p, gamma, f32(gi), f32(u), f32(mu))
            assert rel_inf(got.cpu().numpy(), ref) < 1e-5
    assert B.last_device_status() == 0


@pytest.mark.parametrize("cf,levels,relax", [(4, 2, 0), (2, 3, 1), (4, 3, 2)])
def test_sharded_cycles_on_one_gpu_equal_the_library_solve(cf, levels, relax):
    from paper_2203_04738_b200 import binding as B
    from paper_2203_04738_b200.time_shard import DeviceSteps, LocalComm, partition, sharded_cycle
    w = Workload("shard", T=64, B=3, I=16, H=32, cf=cf, levels=levels, iters_fwd=2, iters_adj=2, relax_fine=relax, relax_coarse=relax,
                 operands=0, classes=8, relu=True, seed=61)
    d = make_inputs(w)
    p, x, h0 = upload(d)
    P = oracle_params(d)
    cfg = B.make_cfg(w.T, w.B, w.I, w.H, cf=cf, levels=levels, iters=2, relax_fine=relax, relax_coarse=relax, operands=B.OPERANDS_FP32)
    h, gi, rn = B.mgrit_gru_forward(cfg, p, x, h0, want_resnorm=True)
    hfull = torch.cat([h0[None], h], 0)
    seed = torch.from_numpy((np.random.default_rng(5).standard_normal((w.T, w.B, w.H)) * 0.1).astype(np.float32)).cuda()
    r = B.mgrit_gru_adjoint(cfg, p, x, h0, gi, h, dh_seed=seed, want_resnorm=True)
    steps = DeviceSteps(B, cfg, p, gi, hfull)
    parts = partition(w.T, cf, levels, 0, 1)
    comm = LocalComm()
    # forward
    u = [torch.zeros((w.T + 1, w.B, w.H), device="cuda")] + [None] * (levels - 1)
    g = [torch.zeros_like(u[0])] + [None] * (levels - 1)
    u[0][0] = h0
    res2 = []
    for _ in range(2):
        sharded_cycle(steps.fwd, cf, [relax] * levels, parts, u, g, comm, 0, res2)
    assert max_abs(u[0][1:].cpu().numpy(), h.cpu().numpy()) < 2e-6
    assert np.allclose(np.sqrt(res2), rn, rtol=1e-4)
    href, _ = O.mgrit_forward(*P, d["x"].astype(np.float64), d["h0"].astype(np.float64), cf=cf, levels=levels, iters=2, relax_fine=relax,
                              relax_coarse=relax)
    assert max_abs(u[0][1:].cpu().numpy(), href) < 1e-4
    # adjoint on the reversed index: mu_0 = seed at T, source at reversed point s = seed[T - s - 1]
    u = [torch.zeros((w.T + 1, w.B, w.H), device="cuda")] + [None] * (levels - 1)
    g = [torch.zeros_like(u[0])] + [None] * (levels - 1)
    u[0][0] = seed[w.T - 1]
    g[0][1:w.T] = torch.flip(seed[: w.T - 1], dims=[0])
    res2 = []
    for _ in range(2):
        sharded_cycle(steps.adj, cf, [relax] * levels, parts, u, g, comm, 0, res2)
    mu = u[0]
    dh = torch.flip(mu[:w.T], dims=[0])                  # dh[k] = lambda_{k+1} = mu_{T-1-k}
    assert rel_inf(dh.cpu().numpy(), r.dh.cpu().numpy()) < 1e-5
    assert rel_inf(mu[w.T].cpu().numpy(), r.dh0.cpu().numpy()) < 1e-4
    assert np.allclose(np.sqrt(res2), r.resnorm, rtol=1e-4)
    assert B.last_device_status() == 0
