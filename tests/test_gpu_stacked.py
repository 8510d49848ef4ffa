"""GPU parity of the stacked-layer solve (all layers in one state, one MGRIT cycle for the stack) against the fp64
oracle at the same cycle count, both operand modes: forward states, adjoint sensitivities and every layer's
gradients; plus the serial sweep of the stack (levels = 1)."""
import numpy as np
import pytest
import torch

from oracle import mgrit_gru_oracle as O
from paper_2203_04738_b200.synthetic import Workload, make_inputs
from tests.gpu_util import NAMES, max_abs, rel_inf, to_dev

pytestmark = pytest.mark.gpu

CASES = [
    dict(T=64, B=2, I=16, H=32, cf=4, levels=3, nl=2, rf=0, rc=1, flags=0, op=0),
    dict(T=32, B=3, I=16, H=32, cf=2, levels=3, nl=3, rf=1, rc=1, flags=2, op=0),        # three layers, F-cycle
    dict(T=37, B=2, I=16, H=32, cf=3, levels=3, nl=2, rf=0, rc=2, flags=4, op=0),        # ragged T, FCFCF inside
    dict(T=24, B=2, I=16, H=32, cf=4, levels=1, nl=2, rf=0, rc=0, flags=0, op=0),        # serial sweep of the stack
    dict(T=64, B=8, I=64, H=128, cf=4, levels=3, nl=2, rf=0, rc=1, flags=0, op=2),       # tensor-core engine
    dict(T=50, B=24, I=48, H=192, cf=3, levels=2, nl=2, rf=1, rc=1, flags=4, op=2),      # ragged, awkward batch
]


@pytest.mark.parametrize("c", CASES, ids=lambda c: "T{T}B{B}H{H}cf{cf}L{levels}nl{nl}r{rf}{rc}f{flags}o{op}".format(**c))
def test_stacked_solve(c):
    from paper_2203_04738_b200 import binding as B
    w = Workload("stk", T=c["T"], B=c["B"], I=c["I"], H=c["H"], cf=c["cf"], levels=c["levels"], iters_fwd=2, iters_adj=2,
                 relax_fine=c["rf"], relax_coarse=c["rc"], operands=c["op"], classes=8, relu=True, seed=500 + c["T"], layers=c["nl"])
    d = make_inputs(w)
    nl = c["nl"]
    layers_dev = [{n: to_dev(l[n]) for n in NAMES} for l in d["layers"]]
    layers_ref = [tuple(l[n].astype(np.float64) for n in NAMES) for l in d["layers"]]
    rng = np.random.default_rng(3)
    h0 = (rng.standard_normal((nl, w.B, w.H)) * 0.3).astype(np.float32)
    x = to_dev(d["x"])
    cfg = B.make_cfg(w.T, w.B, w.I, w.H, cf=w.cf, levels=w.levels, iters=2, relax_fine=w.relax_fine, relax_coarse=w.relax_coarse,
                     operands=c["op"], flags=c["flags"])
    kw = dict(cf=w.cf, levels=w.levels, iters=2, relax_fine=w.relax_fine, relax_coarse=w.relax_coarse,
              cycle=O.CYCLE_F if c["flags"] & 2 else O.CYCLE_V, ragged=bool(c["flags"] & 4))
    fp32 = c["op"] == 0
    tol = 1e-3 if fp32 else 2e-2
    xr, h0r = d["x"].astype(np.float64), h0.astype(np.float64)
    h, gi0, rn = B.mgrit_gru_stack_forward(cfg, layers_dev, x, to_dev(h0), want_resnorm=w.levels > 1)
    href, rref = O.stacked_mgrit_forward(layers_ref, xr, h0r, **kw)
    if fp32:
        assert max_abs(h.cpu().numpy(), href) < 1e-4
    else:
        assert rel_inf(h.cpu().numpy(), href) < tol
    if w.levels > 1:
        for a, b in zip(rn, rref):
            assert abs(a - b) <= (1e-3 * b + 1e-5 if fp32 else 1e-3 * b + 1e-3 * rref[0])
    else:   # levels = 1: the exact serial sweep of the stacked network
        assert (max_abs(h.cpu().numpy(), O.stacked_serial_forward(layers_ref, xr, h0r)) < 1e-4 if fp32 else True)
    # adjoint at the GPU's states: loss derivative on the top layer's last state plus small seeds everywhere
    hn = h.cpu().numpy().astype(np.float64)
    seed = (rng.standard_normal(hn.shape) * 0.02).astype(np.float32)
    dhT = rng.standard_normal((w.B, w.H)).astype(np.float32)
    dh, dh0, dx, gr, rna = B.mgrit_gru_stack_adjoint(cfg, layers_dev, x, to_dev(h0), gi0, h, dh_seed=to_dev(seed), dhT=to_dev(dhT),
                                                     want_resnorm=w.levels > 1)
    seed64 = seed.astype(np.float64)
    seed64[-1, nl - 1] += dhT
    if w.levels > 1:
        lam, lam0, g, rref = O.stacked_mgrit_adjoint(layers_ref, xr, h0r, hn, seed64, **kw)
        for a, b in zip(rna, rref):
            assert abs(a - b) <= (1e-3 * b + 1e-7 if fp32 else 1e-3 * b + 1e-3 * rref[0])
    else:
        lam, lam0, g = O.stacked_serial_backward(layers_ref, xr, h0r, hn, seed64)
    assert rel_inf(dh.cpu().numpy(), lam) < tol
    assert max_abs(dh0.cpu().numpy(), lam0) / np.max(np.abs(lam)) < tol
    assert rel_inf(dx.cpu().numpy(), g[0]["dx"]) < tol
    for k in range(nl):
        for key in ("dW_ih", "dW_hh", "db_ih", "db_hh"):
            assert rel_inf(getattr(gr[k], key).cpu().numpy(), g[k][key]) < tol, (k, key)
    assert B.last_device_status() == 0
