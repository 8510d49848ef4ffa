"""GPU parity of the Implicit LSTM solved by MGRIT against the fp64 oracle at the same cycle count, on the fp32 engine
and on the tensor cores (tf32 three-term split at the fp32 tolerances; bf16 operands at 2e-2 norm-relative; four-gate
tiles of 64 hidden units): states (c, h), adjoint sensitivities, all gradients; cycle variants; the serial sweep and
exact BPTT (levels = 1)."""
import numpy as np
import pytest
import torch

from oracle import mgrit_gru_oracle as O
from tests.gpu_util import max_abs, rel_inf, to_dev

pytestmark = pytest.mark.gpu

CASES = [
    dict(T=64, B=2, I=16, H=32, cf=4, levels=2, rf=0, rc=1, flags=0, cell=1),
    dict(T=64, B=3, I=24, H=40, cf=2, levels=4, rf=1, rc=1, flags=0, cell=1),
    dict(T=50, B=2, I=16, H=32, cf=3, levels=3, rf=0, rc=2, flags=2 | 4, cell=1),     # F-cycle, ragged T, FCFCF inside
    dict(T=32, B=2, I=16, H=32, cf=2, levels=2, rf=0, rc=1, flags=0, cell=0),         # explicit (classic) cell, gamma <= 2
    dict(T=40, B=4, I=16, H=32, cf=4, levels=1, rf=0, rc=0, flags=0, cell=1),         # serial sweep + exact BPTT
    # tensor cores (operands = 1: tf32 split): H a multiple of 64, rows that end in a partial 128-row tile
    dict(T=64, B=5, I=48, H=128, cf=4, levels=3, rf=0, rc=1, flags=0, cell=1, op=1),
    dict(T=52, B=4, I=32, H=64, cf=4, levels=2, rf=1, rc=1, flags=2 | 4, cell=1, op=1),   # F-cycle, ragged T
    dict(T=24, B=4, I=32, H=192, cf=4, levels=1, rf=0, rc=0, flags=0, cell=1, op=1),      # serial sweep + exact BPTT
    # bf16 operands
    dict(T=64, B=5, I=48, H=128, cf=4, levels=3, rf=0, rc=1, flags=0, cell=1, op=2),
    dict(T=256, B=16, I=64, H=256, cf=4, levels=3, rf=1, rc=1, flags=0, cell=1, op=2),
    dict(T=24, B=8, I=32, H=64, cf=4, levels=1, rf=0, rc=0, flags=0, cell=1, op=2),       # serial sweep + exact BPTT
    # bf16 operands on the persistent chain kernels (H a multiple of 128): the whole serial sweep / the coarsest level in
    # one launch; two row groups with a partial one; the widest shapes (weights of the adjoint chain held in registers)
    dict(T=48, B=20, I=32, H=128, cf=4, levels=1, rf=0, rc=0, flags=0, cell=1, op=2),
    dict(T=64, B=32, I=64, H=512, cf=4, levels=2, rf=0, rc=1, flags=0, cell=1, op=2),
    dict(T=32, B=32, I=64, H=1024, cf=4, levels=2, rf=0, rc=1, flags=0, cell=1, op=2),
    dict(T=24, B=16, I=64, H=1024, cf=4, levels=1, rf=0, rc=0, flags=0, cell=0, op=2),    # classic cell, serial sweep
]


@pytest.mark.parametrize("c", CASES, ids=lambda c: "T{T}B{B}H{H}cf{cf}L{levels}r{rf}{rc}f{flags}c{cell}".format(**c) + f"o{c.get('op', 0)}")
def test_lstm_solve(c):
    from paper_2203_04738_b200 import binding as B
    rng = np.random.default_rng(700 + c["T"])
    T, Bn, I, H = c["T"], c["B"], c["I"], c["H"]
    k = 1.0 / np.sqrt(H)
    P32 = [rng.uniform(-k, k, s).astype(np.float32) for s in ((4 * H, I), (4 * H, H), (4 * H,), (4 * H,))]
    x32 = np.maximum(rng.standard_normal((T, Bn, I)), 0).astype(np.float32)
    u032 = (rng.standard_normal((2, Bn, H)) * 0.3).astype(np.float32)
    P = [a.astype(np.float64) for a in P32]
    p = dict(zip(("W_ih", "W_hh", "b_ih", "b_hh"), [to_dev(a) for a in P32]))
    cfg = B.make_cfg(T, Bn, I, H, cf=c["cf"], levels=c["levels"], iters=2, cell=c["cell"], relax_fine=c["rf"], relax_coarse=c["rc"],
                     operands=c.get("op", B.OPERANDS_FP32), flags=c["flags"])
    kw = dict(cf=c["cf"], levels=c["levels"], iters=2, cell=c["cell"], relax_fine=c["rf"], relax_coarse=c["rc"],
              cycle=O.CYCLE_F if c["flags"] & 2 else O.CYCLE_V, ragged=bool(c["flags"] & 4))
    multi = c["levels"] > 1
    bf = c.get("op", 0) == 2
    tol_g = 2e-2 if bf else 1e-3
    close = (lambda a, b: rel_inf(a, b) < 2e-2) if bf else (lambda a, b: max_abs(a, b) < 1e-4)
    u, gi, rn = B.mgrit_lstm_forward(cfg, p, to_dev(x32), to_dev(u032), want_resnorm=multi)
    uref, rref = O.lstm_mgrit_forward(*P, x32.astype(np.float64), u032.astype(np.float64), **kw)
    assert close(u.cpu().numpy(), uref)
    if multi:
        for a, b in zip(rn, rref):
            assert abs(a - b) <= 1e-3 * b + (1e-3 * rref[0] if bf else 1e-5)
    else:
        assert close(u.cpu().numpy(), O.lstm_serial_forward(*P, x32.astype(np.float64), u032.astype(np.float64), cell=c["cell"]))
    un = u.cpu().numpy().astype(np.float64)
    seed = (rng.standard_normal(un.shape) * 0.05).astype(np.float32)
    dhT = rng.standard_normal((Bn, H)).astype(np.float32)
    du, du0, r, rna = B.mgrit_lstm_adjoint(cfg, p, to_dev(x32), to_dev(u032), gi, u, du_seed=to_dev(seed), dhT=to_dev(dhT), want_resnorm=multi)
    seed64 = seed.astype(np.float64)
    seed64[-1, 1] += dhT
    if multi:
        lam, lam0, g, rref = O.lstm_mgrit_adjoint(*P, x32.astype(np.float64), u032.astype(np.float64), un, seed64, **kw)
        for a, b in zip(rna, rref):
            assert abs(a - b) <= 1e-3 * b + (1e-3 * rref[0] if bf else 1e-7)
    else:
        lam, lam0, g = O.lstm_serial_backward(*P, x32.astype(np.float64), u032.astype(np.float64), un, seed64, cell=c["cell"])
    assert rel_inf(du.cpu().numpy(), lam) < tol_g
    assert max_abs(du0.cpu().numpy(), lam0) / np.max(np.abs(lam)) < tol_g
    for key in ("dx", "dW_ih", "dW_hh", "db_ih", "db_hh"):
        assert rel_inf(getattr(r, key).cpu().numpy(), g[key]) < tol_g, key
    assert B.last_device_status() == 0


def test_lstm_tensor_core_modes_reject_unsupported_shapes():
    from paper_2203_04738_b200 import binding as B
    for op in (B.OPERANDS_BF16, B.OPERANDS_TF32):
        with pytest.raises(B.MgritError) as e:
            B.lstm_workspace_bytes(B.make_cfg(64, 8, 64, 32, cf=4, levels=2, operands=op))       # H = 32 is not a multiple of 64
        assert e.value.code == -4
        assert B.lstm_workspace_bytes(B.make_cfg(64, 8, 64, 128, cf=4, levels=2, operands=op))[0] > 0


def test_lstm_full_size_sampled_row_and_gradients():
    """One Implicit-LSTM layer at the shape and in the launch configuration that `bench.py --lstm` times (the default
    workload's T, B, I, H, levels and cycle counts; bf16 operands; chain kernels on the coarsest level).  Batch rows do
    not interact in the recurrence, so the oracle solves the full-length problem for one sampled row (states, adjoint
    sensitivities, dx); the weight gradients sum over ALL (t, b): one time-parallel fp64 pass of the oracle over the
    full batch, fed the GPU's states and sensitivities, checks exactly the gradient kernels."""
    from paper_2203_04738_b200 import binding as B
    from paper_2203_04738_b200.synthetic import WORKLOADS
    w = WORKLOADS["train"]
    T, Bn, I, H = w.T, w.B, w.I, w.H
    rng = np.random.default_rng(811)
    k = 1.0 / np.sqrt(H)
    P32 = [rng.uniform(-k, k, s).astype(np.float32) for s in ((4 * H, I), (4 * H, H), (4 * H,), (4 * H,))]
    x32 = np.maximum(rng.standard_normal((T, Bn, I)), 0).astype(np.float32)
    u032 = (rng.standard_normal((2, Bn, H)) * 0.3).astype(np.float32)
    dhT = rng.standard_normal((Bn, H)).astype(np.float32)
    p = dict(zip(("W_ih", "W_hh", "b_ih", "b_hh"), [to_dev(a) for a in P32]))
    kwc = dict(cf=w.cf, levels=w.levels, relax_fine=w.relax_fine, relax_coarse=w.relax_coarse, operands=B.OPERANDS_BF16)
    cfg_f = B.make_cfg(T, Bn, I, H, iters=w.iters_fwd, **kwc)
    cfg_a = B.make_cfg(T, Bn, I, H, iters=w.iters_adj, **kwc)
    xd, u0d = to_dev(x32), to_dev(u032)
    n0 = B.kernel_launches()
    u, gi, rn = B.mgrit_lstm_forward(cfg_f, p, xd, u0d, want_resnorm=True)
    du, du0, r, rna = B.mgrit_lstm_adjoint(cfg_a, p, xd, u0d, gi, u, dhT=to_dev(dhT), want_resnorm=True)
    # the coarsest level ran as chains: far fewer launches than one per dependent step (128 steps, 4 cycles in all)
    # (MGRIT_GRU_CHAIN_LL=0, an A/B switch of the library, turns those kernels off)
    import os
    assert B.kernel_launches() - n0 < 400 or os.environ.get("MGRIT_GRU_CHAIN_LL") == "0"
    assert B.last_device_status() == 0
    assert all(a > b for a, b in zip(rn, rn[1:])) and all(a > b for a, b in zip(rna, rna[1:]))
    P = [a.astype(np.float64) for a in P32]
    kw = dict(cf=w.cf, levels=w.levels, cell=1, relax_fine=w.relax_fine, relax_coarse=w.relax_coarse)
    rows = [11]
    xr, u0r = x32[:, rows].astype(np.float64), u032[:, rows].astype(np.float64)
    uref, _ = O.lstm_mgrit_forward(*P, xr, u0r, iters=w.iters_fwd, **kw)
    ug = u[:, :, rows].cpu().numpy().astype(np.float64)
    assert rel_inf(ug, uref) < 2e-2
    seed = np.zeros_like(ug)
    seed[-1, 1] = dhT[rows]
    lam, lam0, g, _ = O.lstm_mgrit_adjoint(*P, xr, u0r, ug, seed, iters=w.iters_adj, **kw)
    assert rel_inf(du[:, :, rows].cpu().numpy(), lam) < 2e-2
    assert max_abs(du0[:, rows].cpu().numpy(), lam0) / np.max(np.abs(lam)) < 2e-2
    assert rel_inf(r.dx[:, rows].cpu().numpy(), g["dx"]) < 2e-2
    del g, lam, uref
    gw = O.lstm_weight_gradients(*P, x32.astype(np.float64), u032.astype(np.float64), u.cpu().numpy().astype(np.float64),
                                 du.cpu().numpy().astype(np.float64), want_dx=False)
    for key in ("dW_ih", "dW_hh", "db_ih", "db_hh"):
        assert rel_inf(getattr(r, key).cpu().numpy(), gw[key]) < 2e-2, key
