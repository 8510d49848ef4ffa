"""GPU parity, fp32 operand mode: the CUDA path through the C ABI against the fp64 oracle,
element by element, at the same cycle count.  Tolerances: max-abs 1e-4 on h, 1e-3 norm-relative
on gradients, 1e-3 relative on residual norms."""
import numpy as np
import pytest
import torch

from oracle import mgrit_gru_oracle as O
from paper_2203_04738_b200.synthetic import WORKLOADS, Workload, make_inputs
from tests.gpu_util import max_abs, oracle_params, rel_inf, to_dev, upload

pytestmark = pytest.mark.gpu

TOL_H = 1e-4
TOL_G = 1e-3


@pytest.fixture(scope="module")
def B():
    from paper_2203_04738_b200 import binding
    return binding


def _cfg(B, w, iters, levels=None, cf=None, relax_fine=None, relax_coarse=None, T=None, cell=1, flags=0):
    return B.make_cfg(T or w.T, w.B, w.I, w.H, cf=cf or w.cf, levels=levels or w.levels, iters=iters, cell=cell,
                      relax_fine=w.relax_fine if relax_fine is None else relax_fine,
                      relax_coarse=w.relax_coarse if relax_coarse is None else relax_coarse,
                      operands=B.OPERANDS_FP32, flags=flags)


def test_projection(B):
    w = WORKLOADS["tiny"]
    d = make_inputs(w)
    p, x, h0 = upload(d)
    gi = B.gru_input_projection(_cfg(B, w, 1), p, x)
    P = oracle_params(d)
    ref = O.input_projection(P[0], P[2], d["x"].astype(np.float64))
    assert max_abs(gi.cpu().numpy(), ref) < 1e-5


@pytest.mark.parametrize("cell", [0, 1])
def test_serial_forward(B, cell):
    w = WORKLOADS["tiny"]
    d = make_inputs(w)
    p, x, h0 = upload(d)
    h, _ = B.gru_serial_forward(_cfg(B, w, 1, cell=cell), p, x, h0)
    ref = O.serial_forward(*oracle_params(d), d["x"].astype(np.float64), d["h0"].astype(np.float64), cell=cell)
    assert max_abs(h.cpu().numpy(), ref) < TOL_H


@pytest.mark.parametrize("iters", [1, 2, 16])
@pytest.mark.parametrize("relax_fine", [0, 1])
def test_tiny_forward_two_level(B, iters, relax_fine):
    w = WORKLOADS["tiny"]
    d = make_inputs(w)
    p, x, h0 = upload(d)
    cfg = _cfg(B, w, iters, relax_fine=relax_fine)
    h, gi, rn = B.mgrit_gru_forward(cfg, p, x, h0, want_resnorm=True)
    P = oracle_params(d)
    xr, h0r = d["x"].astype(np.float64), d["h0"].astype(np.float64)
    ref, rref = O.mgrit_forward(*P, xr, h0r, cf=w.cf, levels=2, iters=iters, relax_fine=relax_fine)
    assert max_abs(h.cpu().numpy(), ref) < TOL_H
    for a, b in zip(rn, rref):
        assert abs(a - b) <= 1e-3 * b + 1e-5
    if iters == 16:  # T / cf cycles: the two-level method has become the serial sweep
        hs, _ = B.gru_serial_forward(cfg, p, x, h0)
        assert max_abs(h.cpu().numpy(), hs.cpu().numpy()) < 1e-5
        assert max_abs(h.cpu().numpy(), O.serial_forward(*P, xr, h0r)) < TOL_H


@pytest.mark.parametrize("levels,cf,T,rf,rc", [(3, 4, 64, 0, 1), (3, 2, 64, 1, 1), (4, 2, 48, 0, 0), (2, 8, 64, 0, 1), (3, 4, 80, 1, 0),
                                                 (3, 4, 16, 0, 1), (4, 2, 8, 1, 1)])   # the last two: one-point coarsest level
def test_tiny_forward_multilevel_and_ragged(B, levels, cf, T, rf, rc):
    w = WORKLOADS["tiny"]
    d = make_inputs(w, T=T, B=3)
    p, x, h0 = upload(d)
    w3 = Workload(**{**w.__dict__, "B": 3})
    cfg = _cfg(B, w3, 3, levels=levels, cf=cf, relax_fine=rf, relax_coarse=rc, T=T)
    h, _, rn = B.mgrit_gru_forward(cfg, p, x, h0, want_resnorm=True)
    ref, rref = O.mgrit_forward(*oracle_params(d), d["x"].astype(np.float64), d["h0"].astype(np.float64), cf=cf,
                                levels=levels, iters=3, relax_fine=rf, relax_coarse=rc)
    assert max_abs(h.cpu().numpy(), ref) < TOL_H
    for a, b in zip(rn, rref):
        assert abs(a - b) <= 1e-3 * b + 1e-5


def test_skip_duplicate_frelax_is_identical(B):
    w = WORKLOADS["tiny"]
    d = make_inputs(w)
    p, x, h0 = upload(d)
    h1, _, _ = B.mgrit_gru_forward(_cfg(B, w, 3, levels=3), p, x, h0)
    h2, _, _ = B.mgrit_gru_forward(_cfg(B, w, 3, levels=3, flags=B.FLAG_SKIP_DUPLICATE_FRELAX), p, x, h0)
    assert torch.equal(h1, h2)


def _adjoint_case(B, w, d, cfg, iters, serial=False, seed_all=False, cf=None, levels=None, rf=None, rc=None):
    p, x, h0 = upload(d)
    P = oracle_params(d)
    xr, h0r = d["x"].astype(np.float64), d["h0"].astype(np.float64)
    Wc, bc, lab = d["W_c"].astype(np.float64), d["b_c"].astype(np.float64), d["labels"]
    cf = cf or w.cf; levels = levels or w.levels
    rf = w.relax_fine if rf is None else rf; rc = w.relax_coarse if rc is None else rc
    # forward on the GPU, loss head on the GPU
    if serial:
        h, gi = B.gru_serial_forward(cfg, p, x, h0)
    else:
        h, gi, _ = B.mgrit_gru_forward(cfg, p, x, h0)
    loss, dhT, dWc, dbc = B.xent_head_fwd_bwd(h[-1].contiguous(), to_dev(d["W_c"]), to_dev(d["b_c"]), to_dev(lab))
    # the oracle is fed the GPU's forward states (fp32 values) so that only the adjoint path is compared
    h_np = h.cpu().numpy().astype(np.float64)
    loss_r, dhT_r, dWc_r, dbc_r = O.xent_head(h_np[-1], Wc, bc, lab)
    assert abs(loss.item() - loss_r) < 1e-5
    assert rel_inf(dhT.cpu().numpy(), dhT_r) < TOL_G and rel_inf(dWc.cpu().numpy(), dWc_r) < TOL_G
    assert rel_inf(dbc.cpu().numpy(), dbc_r) < TOL_G
    seed = np.zeros_like(h_np)
    seed_dev = None
    if seed_all:
        seed = np.random.default_rng(5).standard_normal(h_np.shape).astype(np.float32).astype(np.float64) * 0.01
        seed_dev = to_dev(seed.astype(np.float32))
    seed[-1] += dhT.cpu().numpy().astype(np.float64)
    if serial:
        r = B.gru_serial_backward(cfg, p, x, h0, gi, h, dh_seed=seed_dev, dhT=dhT)
        lam, lam0, g = O.serial_backward(*P, xr, h0r, h_np, seed)
    else:
        r = B.mgrit_gru_adjoint(cfg, p, x, h0, gi, h, dh_seed=seed_dev, dhT=dhT, want_resnorm=True)
        lam, lam0, g, rref = O.mgrit_adjoint(*P, xr, h0r, h_np, seed, cf=cf, levels=levels, iters=iters, relax_fine=rf,
                                             relax_coarse=rc)
        for a, b in zip(r.resnorm, rref):
            assert abs(a - b) <= 1e-3 * b + 1e-7
    errs = {
        "dh": rel_inf(r.dh.cpu().numpy(), lam), "dh0": rel_inf(r.dh0.cpu().numpy(), lam0),
        "dx": rel_inf(r.dx.cpu().numpy(), g["dx"]), "dW_ih": rel_inf(r.dW_ih.cpu().numpy(), g["dW_ih"]),
        "dW_hh": rel_inf(r.dW_hh.cpu().numpy(), g["dW_hh"]), "db_ih": rel_inf(r.db_ih.cpu().numpy(), g["db_ih"]),
        "db_hh": rel_inf(r.db_hh.cpu().numpy(), g["db_hh"]),
    }
    for k, v in errs.items():
        # dh0 of a long sequence underflows towards zero: compare it on the scale of dh
        if k == "dh0":
            v = max_abs(r.dh0.cpu().numpy(), lam0) / max(np.max(np.abs(lam)), 1e-30)
        assert v < TOL_G, (k, v)


@pytest.mark.parametrize("iters", [2, 16])
@pytest.mark.parametrize("seed_all", [False, True])
def test_tiny_adjoint_two_level(B, iters, seed_all):
    w = WORKLOADS["tiny"]
    d = make_inputs(w)
    _adjoint_case(B, w, d, _cfg(B, w, iters), iters, seed_all=seed_all)


def test_tiny_adjoint_three_level_fcf(B):
    w = WORKLOADS["tiny"]
    d = make_inputs(w)
    _adjoint_case(B, w, d, _cfg(B, w, 2, levels=3, cf=2, relax_fine=1), 2, seed_all=True, cf=2, levels=3, rf=1)


def test_whole_chain_against_the_oracles_own_forward(B):
    # Forward, loss head, adjoint and gradients on the GPU against the same chain run by the oracle alone (its
    # adjoint linearised at its OWN forward states): nothing of the GPU's output enters the reference.
    w = WORKLOADS["tiny"]
    d = make_inputs(w)
    p, x, h0 = upload(d)
    P = oracle_params(d)
    xr, h0r = d["x"].astype(np.float64), d["h0"].astype(np.float64)
    for levels, cf, rf in ((2, 4, 0), (3, 2, 1)):
        cfg = _cfg(B, w, 2, levels=levels, cf=cf, relax_fine=rf)
        kw = dict(cf=cf, levels=levels, relax_fine=rf, relax_coarse=w.relax_coarse, iters=2)
        h, gi, _ = B.mgrit_gru_forward(cfg, p, x, h0)
        loss, dhT, dWc, dbc = B.xent_head_fwd_bwd(h[-1].contiguous(), to_dev(d["W_c"]), to_dev(d["b_c"]), to_dev(d["labels"]))
        r = B.mgrit_gru_adjoint(cfg, p, x, h0, gi, h, dhT=dhT)
        href, _ = O.mgrit_forward(*P, xr, h0r, **kw)
        loss_r, dhT_r, dWc_r, dbc_r = O.xent_head(href[-1], d["W_c"].astype(np.float64), d["b_c"].astype(np.float64), d["labels"])
        seed = np.zeros_like(href)
        seed[-1] = dhT_r
        lam, lam0, g, _ = O.mgrit_adjoint(*P, xr, h0r, href, seed, **kw)
        assert abs(loss.item() - loss_r) < 1e-5
        assert rel_inf(dWc.cpu().numpy(), dWc_r) < TOL_G and rel_inf(dbc.cpu().numpy(), dbc_r) < TOL_G
        assert rel_inf(r.dh.cpu().numpy(), lam) < TOL_G
        for k in ("dx", "dW_ih", "dW_hh", "db_ih", "db_hh"):
            assert rel_inf(getattr(r, k).cpu().numpy(), g[k]) < TOL_G, (k, levels)
        # dh is an optional output: without it everything else is unchanged, bit for bit
        r2 = B.mgrit_gru_adjoint(cfg, p, x, h0, gi, h, dhT=dhT, want_dh=False)
        assert r2.dh is None
        for k in ("dh0", "dx", "dW_ih", "dW_hh", "db_ih", "db_hh"):
            assert torch.equal(getattr(r, k), getattr(r2, k)), k


def test_tiny_serial_backward(B):
    w = WORKLOADS["tiny"]
    d = make_inputs(w)
    _adjoint_case(B, w, d, _cfg(B, w, 1), 1, serial=True, seed_all=True)


def test_clip_forward_and_adjoint(B):
    # second configuration: I=512, H=256, B=16, T=128, two levels, FCF everywhere, 2 cycles, 51 classes
    w = WORKLOADS["clip"]
    d = make_inputs(w)
    p, x, h0 = upload(d)
    cfg = _cfg(B, w, w.iters_fwd)
    h, _, rn = B.mgrit_gru_forward(cfg, p, x, h0, want_resnorm=True)
    ref, rref = O.mgrit_forward(*oracle_params(d), d["x"].astype(np.float64), d["h0"].astype(np.float64), cf=w.cf,
                                levels=w.levels, iters=w.iters_fwd, relax_fine=w.relax_fine, relax_coarse=w.relax_coarse)
    assert max_abs(h.cpu().numpy(), ref) < TOL_H
    for a, b in zip(rn, rref):
        assert abs(a - b) <= 1e-3 * b
    _adjoint_case(B, w, d, cfg, w.iters_adj)


def test_sgd_update(B):
    rng = np.random.default_rng(0)
    for n in (1, 7, 1024, 4099):
        pv = rng.standard_normal(n).astype(np.float32); gv = rng.standard_normal(n).astype(np.float32)
        out = B.sgd_update(to_dev(pv), to_dev(gv), 1e-3)
        assert max_abs(out.cpu().numpy(), O.sgd_update(pv.astype(np.float64), gv.astype(np.float64), 1e-3)) < 1e-6


def test_error_codes(B):
    w = WORKLOADS["tiny"]
    d = make_inputs(w)
    p, x, h0 = upload(d)
    with pytest.raises(B.MgritError) as e:
        B.workspace_bytes(B.make_cfg(100, 2, 16, 32, cf=8, levels=3))
    assert e.value.code == -2
    cfg = _cfg(B, w, 2)
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    import ctypes
    rc = B.lib.mgrit_gru_forward(ctypes.byref(cfg), ctypes.byref(B._params(p)), x.data_ptr(), h0.data_ptr(),
                                 torch.empty(w.T, w.B, 3 * w.H, device="cuda").data_ptr(),
                                 torch.empty(w.T, w.B, w.H, device="cuda").data_ptr(), None, small.data_ptr(), 256, None)
    assert rc == -3
    rc = B.lib.mgrit_gru_forward(ctypes.byref(cfg), ctypes.byref(B._params(p)), None, h0.data_ptr(), None, None, None,
                                 small.data_ptr(), 256, None)
    assert rc == -1
    assert B.last_device_status() == 0


def test_misaligned_pointer_is_rejected(B):
    """Data pointers must be 32-byte aligned (the kernels move whole 32-byte sectors per thread)."""
    import ctypes
    w = WORKLOADS["tiny"]
    d = make_inputs(w)
    p, x, h0 = upload(d)
    cfg = _cfg(B, w, 2)
    nb = B.workspace_bytes(cfg)[0]
    ws = torch.empty(nb, dtype=torch.uint8, device="cuda")
    gi = torch.empty(w.T * w.B * 3 * w.H + 8, device="cuda")
    h = torch.empty(w.T, w.B, w.H, device="cuda")
    args = lambda gi_ptr: (ctypes.byref(cfg), ctypes.byref(B._params(p)), x.data_ptr(), h0.data_ptr(), gi_ptr, h.data_ptr(),
                           None, ws.data_ptr(), nb, None)
    assert B.lib.mgrit_gru_forward(*args(gi.data_ptr())) == 0
    assert B.lib.mgrit_gru_forward(*args(gi.data_ptr() + 16)) == -1      # 16-byte aligned only
    torch.cuda.synchronize()


def test_workspace_content_is_irrelevant(B):
    # only the C-points of the initial guess are cleared by the library: nothing else of the workspace may be read before it
    # is written, whatever it held (NaN patterns here), forward and adjoint, V- and F-cycles, ragged T
    w = WORKLOADS["tiny"]
    d = make_inputs(w)
    p, x, h0 = upload(d)
    for flags, T, levels, cf in ((0, w.T, 2, 4), (B.FLAG_F_CYCLE, w.T, 3, 2), (B.FLAG_RAGGED_T, 61, 3, 4)):
        d2 = make_inputs(w, T=T)
        p, x, h0 = upload(d2)
        cfg = _cfg(B, w, 2, levels=levels, cf=cf, T=T, flags=flags)
        nf, na = B.workspace_bytes(cfg)
        outs = []
        for fill in (0x00, 0xFF):
            ws = torch.full((nf,), fill, dtype=torch.uint8, device="cuda")
            h, gi, _ = B.mgrit_gru_forward(cfg, p, x, h0, ws=ws)
            wa = torch.full((na,), fill, dtype=torch.uint8, device="cuda")
            r = B.mgrit_gru_adjoint(cfg, p, x, h0, gi, h, dhT=h[-1].contiguous(), ws=wa)
            outs.append([t.clone() for t in (h, r.dh, r.dh0, r.dx, r.dW_hh, r.dW_ih)])
        for a, b in zip(*outs):
            assert torch.equal(a, b) and bool(torch.isfinite(a).all())
