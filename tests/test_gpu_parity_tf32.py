"""GPU parity of the tf32 tensor-core operand modes against the fp64 oracle at the same cycle count.

OPERANDS_TF32 (every product as the three-term split x_hi w_hi + x_lo w_hi + x_hi w_lo) is held to the fp32
tolerances: max-abs 1e-4 on h, 1e-3 norm-relative on gradients, 1e-3 relative on residual norms.
OPERANDS_TF32_1PASS (operands rounded to tf32 once, 10 mantissa bits) is held to 5e-3 norm-relative; it must also be
measurably less exact than the split form, otherwise the split would not be doing anything.
"""
import numpy as np
import pytest

from oracle import mgrit_gru_oracle as O
from paper_2203_04738_b200.synthetic import WORKLOADS, Workload, make_inputs
from tests.gpu_util import max_abs, oracle_params, rel_inf, upload
from tests.test_gpu_parity_fp32 import TOL_G, TOL_H, _adjoint_case

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_2203_04738_b200 import binding
    return binding


def _cfg(B, w, iters, operands=None, cell=1, flags=0):
    return B.make_cfg(w.T, w.B, w.I, w.H, cf=w.cf, levels=w.levels, iters=iters, cell=cell, relax_fine=w.relax_fine,
                      relax_coarse=w.relax_coarse, operands=B.OPERANDS_TF32 if operands is None else operands, flags=flags)


def _forward_case(B, w, cfg, cell=1, tol=TOL_H, rtol=1e-3):
    d = make_inputs(w)
    p, x, h0 = upload(d)
    P = oracle_params(d)
    xr, h0r = d["x"].astype(np.float64), d["h0"].astype(np.float64)
    gi = B.gru_input_projection(cfg, p, x)
    assert max_abs(gi.cpu().numpy(), O.input_projection(P[0], P[2], xr)) < tol
    h, _, rn = B.mgrit_gru_forward(cfg, p, x, h0, want_resnorm=True)
    ref, rref = O.mgrit_forward(*P, xr, h0r, cf=w.cf, levels=w.levels, iters=cfg.iters, relax_fine=w.relax_fine,
                                relax_coarse=w.relax_coarse, cell=cell, ragged=bool(cfg.flags & B.FLAG_RAGGED_T))
    err = max_abs(h.cpu().numpy(), ref)
    assert err < tol, err
    for a, b in zip(rn, rref):
        assert abs(a - b) <= rtol * b + rtol * 1e-2 * rref[0]
    return d, err


def test_clip_forward_and_adjoint_split(B):
    w = WORKLOADS["clip"]
    cfg = _cfg(B, w, w.iters_fwd)
    d, _ = _forward_case(B, w, cfg)
    _adjoint_case(B, w, d, cfg, w.iters_adj, seed_all=True)


def test_three_levels_ragged_rows_and_tiles(B):
    # B = 5: 128-row tiles straddle intervals and end in a partial tile; H = 192: three gate tiles of 64 units; I = 48;
    # (T*B) % 4 == 0 is needed by the gradient operands: 320 rows
    w = Workload("tf32-a", T=64, B=5, I=48, H=192, cf=4, levels=3, iters_fwd=2, iters_adj=2, relax_fine=1, relax_coarse=1,
                 operands=1, classes=8, relu=True, seed=21)
    cfg = _cfg(B, w, 2)
    d, _ = _forward_case(B, w, cfg)
    _adjoint_case(B, w, d, cfg, 2, seed_all=True)


@pytest.mark.parametrize("cell", [0, 1])
def test_serial_sweep_and_bptt_split(B, cell):
    w = Workload("tf32-s", T=24, B=4, I=32, H=64, cf=4, levels=2, iters_fwd=1, iters_adj=1, relax_fine=0, relax_coarse=1,
                 operands=1, classes=8, relu=True, seed=22)
    d = make_inputs(w)
    p, x, h0 = upload(d)
    cfg = _cfg(B, w, 1, cell=cell)
    h, _ = B.gru_serial_forward(cfg, p, x, h0)
    ref = O.serial_forward(*oracle_params(d), d["x"].astype(np.float64), d["h0"].astype(np.float64), cell=cell)
    assert max_abs(h.cpu().numpy(), ref) < TOL_H
    if cell == 1:
        _adjoint_case(B, w, d, cfg, 1, serial=True, seed_all=True)


def test_ragged_T_and_f_cycle_split(B):
    w = Workload("tf32-r", T=52, B=8, I=32, H=128, cf=4, levels=3, iters_fwd=2, iters_adj=2, relax_fine=2, relax_coarse=1,
                 operands=1, classes=8, relu=True, seed=23)
    cfg = _cfg(B, w, 2, flags=B.FLAG_RAGGED_T)
    _forward_case(B, w, cfg)


def test_single_pass_is_close_but_less_exact_than_the_split(B):
    w = WORKLOADS["clip"]
    _, e3 = _forward_case(B, w, _cfg(B, w, w.iters_fwd))
    _, e1 = _forward_case(B, w, _cfg(B, w, w.iters_fwd, operands=B.OPERANDS_TF32_1PASS), tol=5e-3, rtol=2e-2)
    print(f"clip forward max|dh|: tf32 split {e3:.3e}, single pass {e1:.3e}")
    assert e1 > 4 * e3


def test_unsupported_shapes_and_entry_points(B):
    w = WORKLOADS["tiny"]                 # H = 32 is not a multiple of 64
    with pytest.raises(B.MgritError) as e:
        B.workspace_bytes(_cfg(B, w, 2))
    assert e.value.code == -4
    w2 = Workload("tf32-u", T=16, B=4, I=32, H=64, cf=4, levels=2, iters_fwd=1, iters_adj=1, relax_fine=0, relax_coarse=1,
                  operands=1, classes=8, relu=True, seed=1)
    with pytest.raises(B.MgritError) as e:
        B.stack_workspace_bytes(_cfg(B, w2, 1), 2)
    assert e.value.code == -4


def test_medium_full_size_split_keeps_the_fp32_tolerances():
    # third configuration's sizes (I = 1024, H = 512, B = 32, T = 1024, three levels) in the tf32 split mode: reductions of
    # 1024 and 1536 products per output, 1024 time steps -- every element against the oracle, forward and adjoint
    import dataclasses
    from paper_2203_04738_b200 import binding as B
    w = dataclasses.replace(WORKLOADS["medium"], operands=1)
    cfg = _cfg(B, w, w.iters_fwd)
    d, err = _forward_case(B, w, cfg)
    print(f"medium forward max|dh| in the tf32 split mode: {err:.3e}")
    _adjoint_case(B, w, d, cfg, w.iters_adj, seed_all=True)
