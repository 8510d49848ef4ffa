"""GPU parity of the cycle variants against the fp64 oracle at the same cycle count: relaxation F(CF)^n, F-cycles and
sequence lengths that are not a multiple of c_f^(levels-1) (forward grids anchored at t = 0, the adjoint's reversed
grids at t = T), in both operand modes, forward and adjoint with all gradients."""
import numpy as np
import pytest
import torch

from oracle import mgrit_gru_oracle as O
from paper_2203_04738_b200.synthetic import Workload, make_inputs
from tests.gpu_util import max_abs, oracle_params, rel_inf, to_dev, upload

pytestmark = pytest.mark.gpu

CASES = [
    # T, B, I, H, cf, levels, relax_fine, relax_coarse, f_cycle, ragged, operands
    dict(T=64, B=2, I=16, H=32, cf=4, levels=2, rf=2, rc=1, fc=0, rag=0, op=0),      # FCFCF on the fine level
    dict(T=64, B=3, I=16, H=32, cf=2, levels=4, rf=0, rc=2, fc=0, rag=0, op=0),      # FCFCF on inner levels
    dict(T=64, B=2, I=16, H=32, cf=4, levels=3, rf=0, rc=1, fc=1, rag=0, op=0),      # F-cycle, three levels
    dict(T=32, B=2, I=16, H=32, cf=2, levels=4, rf=1, rc=1, fc=1, rag=0, op=0),      # F-cycle, four levels
    dict(T=23, B=2, I=16, H=32, cf=4, levels=2, rf=0, rc=1, fc=0, rag=1, op=0),      # ragged, two levels
    dict(T=50, B=3, I=16, H=32, cf=3, levels=3, rf=1, rc=1, fc=0, rag=1, op=0),      # ragged on both coarsenings
    dict(T=37, B=2, I=16, H=32, cf=2, levels=4, rf=0, rc=2, fc=1, rag=1, op=0),      # everything at once
    dict(T=64, B=8, I=64, H=128, cf=4, levels=3, rf=2, rc=1, fc=1, rag=0, op=2),     # tensor-core engine
    dict(T=100, B=8, I=64, H=128, cf=4, levels=3, rf=0, rc=1, fc=0, rag=1, op=2),    # ragged, chains of 6 coarse steps
    dict(T=77, B=24, I=48, H=192, cf=3, levels=3, rf=1, rc=1, fc=1, rag=1, op=2),    # batch that does not divide the tile
]


@pytest.mark.parametrize("c", CASES, ids=lambda c: "T{T}B{B}H{H}cf{cf}L{levels}r{rf}{rc}f{fc}g{rag}o{op}".format(**c))
def test_cycle_variant(c):
    from paper_2203_04738_b200 import binding as B
    w = Workload("var", T=c["T"], B=c["B"], I=c["I"], H=c["H"], cf=c["cf"], levels=c["levels"], iters_fwd=2, iters_adj=2,
                 relax_fine=c["rf"], relax_coarse=c["rc"], operands=c["op"], classes=8, relu=True, seed=300 + c["T"])
    d = make_inputs(w)
    p, x, h0 = upload(d)
    P = oracle_params(d)
    xr, h0r = d["x"].astype(np.float64), d["h0"].astype(np.float64)
    flags = (B.FLAG_F_CYCLE if c["fc"] else 0) | (B.FLAG_RAGGED_T if c["rag"] else 0)
    cfg = B.make_cfg(w.T, w.B, w.I, w.H, cf=w.cf, levels=w.levels, iters=2, relax_fine=w.relax_fine, relax_coarse=w.relax_coarse,
                     operands=c["op"], flags=flags)
    kw = dict(cf=w.cf, levels=w.levels, iters=2, relax_fine=w.relax_fine, relax_coarse=w.relax_coarse,
              cycle=O.CYCLE_F if c["fc"] else O.CYCLE_V, ragged=bool(c["rag"]))
    fp32 = c["op"] == 0
    h, gi, rn = B.mgrit_gru_forward(cfg, p, x, h0, want_resnorm=True)
    href, rref = O.mgrit_forward(*P, xr, h0r, **kw)
    if fp32:
        assert max_abs(h.cpu().numpy(), href) < 1e-4
    else:
        assert rel_inf(h.cpu().numpy(), href) < 2e-2
    for a, b in zip(rn, rref):
        assert abs(a - b) <= (1e-3 * b + 1e-5 if fp32 else 1e-3 * b + 1e-3 * rref[0])
    # the same with the duplicate F-relaxation skipped: identical bits
    cfg2 = B.make_cfg(w.T, w.B, w.I, w.H, cf=w.cf, levels=w.levels, iters=2, relax_fine=w.relax_fine, relax_coarse=w.relax_coarse,
                      operands=c["op"], flags=flags | B.FLAG_SKIP_DUPLICATE_FRELAX)
    h2, _, _ = B.mgrit_gru_forward(cfg2, p, x, h0)
    assert torch.equal(h, h2)
    # adjoint at the GPU's states, seeded at every time
    hn = h.cpu().numpy().astype(np.float64)
    seed = (np.random.default_rng(5).standard_normal(hn.shape) * 0.05).astype(np.float32)
    r = B.mgrit_gru_adjoint(cfg, p, x, h0, gi, h, dh_seed=to_dev(seed), want_resnorm=True)
    lam, lam0, g, rref = O.mgrit_adjoint(*P, xr, h0r, hn, seed.astype(np.float64), **kw)
    tol = 1e-3 if fp32 else 2e-2
    assert rel_inf(r.dh.cpu().numpy(), lam) < tol
    assert max_abs(r.dh0.cpu().numpy(), lam0) / np.max(np.abs(lam)) < tol
    for k in ("dx", "dW_ih", "dW_hh", "db_ih", "db_hh"):
        assert rel_inf(getattr(r, k).cpu().numpy(), g[k]) < tol, k
    for a, b in zip(r.resnorm, rref):
        assert abs(a - b) <= (1e-3 * b + 1e-7 if fp32 else 1e-3 * b + 1e-3 * rref[0])
    assert B.last_device_status() == 0


def test_ragged_needs_the_flag_and_enough_points():
    from paper_2203_04738_b200 import binding as B
    with pytest.raises(B.MgritError) as e:
        B.workspace_bytes(B.make_cfg(23, 2, 16, 32, cf=4, levels=2))
    assert e.value.code == -2
    B.workspace_bytes(B.make_cfg(23, 2, 16, 32, cf=4, levels=2, flags=B.FLAG_RAGGED_T))
    with pytest.raises(B.MgritError) as e:
        B.workspace_bytes(B.make_cfg(7, 2, 16, 32, cf=4, levels=3, flags=B.FLAG_RAGGED_T))       # level 2 would be empty
    assert e.value.code == -2
