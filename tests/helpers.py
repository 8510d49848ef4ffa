"""Small helpers for the tests: float64 views of the seeded inputs."""
import numpy as np

from paper_2203_04738_b200.synthetic import Workload, make_inputs


def tiny_workload(**kw):
    base = dict(name="t", T=64, B=2, I=16, H=32, cf=4, levels=2, iters_fwd=2, iters_adj=2,
                relax_fine=0, relax_coarse=1, operands=0, classes=8, relu=False, seed=0)
    base.update(kw)
    return Workload(**base)


def f64_inputs(w, **kw):
    d = make_inputs(w, **kw)
    lay = d["layers"][0]
    P = [lay[n].astype(np.float64) for n in ("W_ih", "W_hh", "b_ih", "b_hh")]
    return P, d["x"].astype(np.float64), d["h0"].astype(np.float64), d
