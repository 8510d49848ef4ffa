"""GPU parity on a seeded sweep of small, awkward shapes (bf16 tensor-core engine and fp32 engine): batch sizes that
do and do not divide the 128-row tile, hidden sizes with one to four unit tiles, input widths with a K tail, two
to four levels, F and FCF relaxation, both cells.  Every case compares the forward states, the adjoint and all
gradients with the fp64 oracle at the same cycle count."""
import numpy as np
import pytest
import torch

from oracle import mgrit_gru_oracle as O
from paper_2203_04738_b200.synthetic import Workload, make_inputs
from tests.gpu_util import oracle_params, rel_inf, to_dev, upload

pytestmark = pytest.mark.gpu


def _cases():
    # the tensor-core engine needs H % 64 == 0, I % 16 == 0 and (T*B) % 8 == 0 (other shapes: MGRIT_UNSUPPORTED)
    rng = np.random.default_rng(2203)
    out = []
    for i in range(14):
        cf = int(rng.choice([2, 4]))
        levels = int(rng.choice([2, 3, 4])) if cf == 2 else int(rng.choice([2, 3]))
        B = int(rng.choice([1, 3, 8, 16, 24, 33, 40]))
        k = int(rng.choice([1, 2, 3, 5]))
        if B % 8 != 0:
            k = 8 if B % 2 else 4
        T = cf ** (levels - 1) * k
        out.append(dict(T=T, B=B, I=int(rng.choice([16, 48, 80, 144])),
                        H=int(rng.choice([64, 128, 192, 256])), cf=cf, levels=levels,
                        # the explicit cell only where its coarse step (gamma = 2) is still stable
                        cell=int(rng.choice([0, 1])) if (cf == 2 and levels == 2) else 1,
                        relax_fine=int(rng.choice([0, 1])), relax_coarse=int(rng.choice([0, 1])),
                        operands=2 if i % 7 != 6 else 0, seed=100 + i))
    return out


@pytest.mark.parametrize("c", _cases(), ids=lambda c: "T{T}B{B}I{I}H{H}cf{cf}L{levels}c{cell}r{relax_fine}{relax_coarse}o{operands}".format(**c))
def test_random_shape(c):
    from paper_2203_04738_b200 import binding as B
    w = Workload("rnd", T=c["T"], B=c["B"], I=c["I"], H=c["H"], cf=c["cf"], levels=c["levels"], iters_fwd=2, iters_adj=2,
                 relax_fine=c["relax_fine"], relax_coarse=c["relax_coarse"], operands=c["operands"], classes=8, relu=True,
                 seed=c["seed"], cell=c["cell"])
    d = make_inputs(w)
    p, x, h0 = upload(d)
    P = oracle_params(d)
    xr, h0r = d["x"].astype(np.float64), d["h0"].astype(np.float64)
    kw = dict(cf=w.cf, levels=w.levels, relax_fine=w.relax_fine, relax_coarse=w.relax_coarse, cell=w.cell)
    cfg = B.make_cfg(w.T, w.B, w.I, w.H, iters=2, operands=w.operands, **kw)
    tol = 2e-2 if w.operands == 2 else 1e-3
    h, gi, _ = B.mgrit_gru_forward(cfg, p, x, h0, want_resnorm=True)
    href, _ = O.mgrit_forward(*P, xr, h0r, iters=2, **kw)
    assert rel_inf(h.cpu().numpy(), href) < tol
    hn = h.cpu().numpy().astype(np.float64)
    rng = np.random.default_rng(c["seed"])
    seed = rng.standard_normal(hn.shape).astype(np.float32)
    r = B.mgrit_gru_adjoint(cfg, p, x, h0, gi, h, dh_seed=to_dev(seed))
    lam, lam0, g, _ = O.mgrit_adjoint(*P, xr, h0r, hn, seed.astype(np.float64), iters=2, **kw)
    assert rel_inf(r.dh.cpu().numpy(), lam) < tol
    for k in ("dx", "dW_ih", "dW_hh", "db_ih", "db_hh"):
        assert rel_inf(getattr(r, k).cpu().numpy(), g[k]) < tol, k
    assert B.last_device_status() == 0
