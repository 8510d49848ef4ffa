"""Pins for the oracle's cell, serial sweep, BPTT and loss head (CPU only)."""
import numpy as np
import pytest
import torch

from oracle import mgrit_gru_oracle as O
from tests.helpers import f64_inputs, tiny_workload


def _torch_gru(P, I, H):
    gru = torch.nn.GRU(I, H, num_layers=1).double()
    with torch.no_grad():
        gru.weight_ih_l0.copy_(torch.from_numpy(P[0]))
        gru.weight_hh_l0.copy_(torch.from_numpy(P[1]))
        gru.bias_ih_l0.copy_(torch.from_numpy(P[2]))
        gru.bias_hh_l0.copy_(torch.from_numpy(P[3]))
    return gru


def test_classic_serial_equals_library_gru():
    # Eq. "gru" is the textbook GRU: the classic propagator with gamma = 1 must reproduce
    # torch.nn.GRU in float64 (gate order r|z|n, both biases, r applied to W_hn h + b_hn).
    w = tiny_workload(T=12, B=3, I=5, H=7)
    P, x, h0, _ = f64_inputs(w)
    h0 = np.random.default_rng(5).standard_normal(h0.shape)
    h = O.serial_forward(*P, x, h0, cell=O.CELL_CLASSIC, dt=1.0)
    gru = _torch_gru(P, w.I, w.H)
    out, _ = gru(torch.from_numpy(x), torch.from_numpy(h0)[None])
    assert np.max(np.abs(out.detach().numpy() - h)) < 1e-13


def test_classic_bptt_equals_library_autograd():
    w = tiny_workload(T=9, B=2, I=4, H=6)
    P, x, h0, _ = f64_inputs(w)
    rng = np.random.default_rng(7)
    h0 = rng.standard_normal(h0.shape)
    seed = rng.standard_normal((w.T, w.B, w.H))       # a loss touching every h_t
    h = O.serial_forward(*P, x, h0, cell=O.CELL_CLASSIC)
    lam, lam0, g = O.serial_backward(*P, x, h0, h, seed, cell=O.CELL_CLASSIC)
    gru = _torch_gru(P, w.I, w.H)
    xt = torch.from_numpy(x).requires_grad_(True)
    h0t = torch.from_numpy(h0).requires_grad_(True)
    out, _ = gru(xt, h0t[None])
    (out * torch.from_numpy(seed)).sum().backward()
    tol = 1e-12
    assert np.max(np.abs(g["dW_ih"] - gru.weight_ih_l0.grad.numpy())) < tol
    assert np.max(np.abs(g["dW_hh"] - gru.weight_hh_l0.grad.numpy())) < tol
    assert np.max(np.abs(g["db_ih"] - gru.bias_ih_l0.grad.numpy())) < tol
    assert np.max(np.abs(g["db_hh"] - gru.bias_hh_l0.grad.numpy())) < tol
    assert np.max(np.abs(g["dx"] - xt.grad.numpy())) < tol
    assert np.max(np.abs(lam0 - h0t.grad.numpy())) < tol


@pytest.mark.parametrize("gamma", [0.5, 1.0, 4.0, 64.0])
def test_implicit_cell_satisfies_its_defining_equation(gamma):
    # Eq. "gru-implicit": (1 + dt(1-z)) h_t = h_{t-1} + dt (1-z) n, z and n at (x_t, h_{t-1}).
    rng = np.random.default_rng(1)
    H = 9
    W_hh = rng.standard_normal((3 * H, H)) * 0.4
    b_hh = rng.standard_normal(3 * H) * 0.1
    gi = rng.standard_normal((4, 3 * H))
    hp = rng.standard_normal((4, H))
    r, z, n, _ = O.gates(W_hh, b_hh, gi, hp)
    hn = O.phi(W_hh, b_hh, gi, hp, gamma, O.CELL_IMPLICIT)
    assert np.max(np.abs((1 + gamma * (1 - z)) * hn - hp - gamma * (1 - z) * n)) < 1e-13
    # difference to the explicit propagator: -q^2 (n-h)/(1+q)
    he = O.phi(W_hh, b_hh, gi, hp, gamma, O.CELL_CLASSIC)
    q = gamma * (1 - z)
    assert np.max(np.abs((hn - he) + q * q * (n - hp) / (1 + q))) < 1e-11 * max(1.0, gamma ** 2)
    # each component is a convex combination of h_{t-1} and n: no growth for any step size
    lo, hi = np.minimum(hp, n), np.maximum(hp, n)
    assert np.all(hn >= lo - 1e-14) and np.all(hn <= hi + 1e-14)


def test_cell_limits():
    rng = np.random.default_rng(2)
    H = 5
    W_hh = rng.standard_normal((3 * H, H)) * 0.3
    b_hh = np.zeros(3 * H)
    hp = rng.standard_normal((2, H))
    gi = rng.standard_normal((2, 3 * H))
    for cell in (O.CELL_CLASSIC, O.CELL_IMPLICIT):
        # gamma -> 0: identity
        assert np.max(np.abs(O.phi(W_hh, b_hh, gi, hp, 0.0, cell) - hp)) == 0.0
        # z -> 1 (huge update-gate pre-activation): state is kept
        g2 = gi.copy()
        g2[:, H:2 * H] = 60.0
        assert np.max(np.abs(O.phi(W_hh, b_hh, g2, hp, 8.0, cell) - hp)) < 1e-12


def test_model_problem_stability():
    # Section "Coarse Grid Propagators": with z fixed and n = 0 the explicit step multiplies h
    # by 1 - dt(1-z) (unstable for dt > 2 when z = 0), the implicit one by 1/(1 + dt(1-z)) <= 1.
    H = 3
    W_hh = np.zeros((3 * H, H))
    b_hh = np.zeros(3 * H)
    gi = np.zeros((1, 3 * H))
    gi[:, H:2 * H] = -50.0            # z ~ 0
    hp = np.ones((1, H))
    for dt in (1.0, 2.0, 4.0, 16.0):
        e = O.phi(W_hh, b_hh, gi, hp, dt, O.CELL_CLASSIC)
        i = O.phi(W_hh, b_hh, gi, hp, dt, O.CELL_IMPLICIT)
        assert np.allclose(e, 1 - dt, atol=1e-12)
        assert np.allclose(i, 1 / (1 + dt), atol=1e-12)
    assert abs(1 - 4.0) > 1            # explicit amplification beyond dt = 2


@pytest.mark.parametrize("cell", [O.CELL_CLASSIC, O.CELL_IMPLICIT])
@pytest.mark.parametrize("gamma", [1.0, 4.0])
def test_adjoint_coefficients_vs_finite_differences(cell, gamma):
    rng = np.random.default_rng(3)
    H, Bn = 6, 2
    W_hh = rng.standard_normal((3 * H, H)) * 0.5
    b_hh = rng.standard_normal(3 * H) * 0.2
    gi = rng.standard_normal((Bn, 3 * H))
    hp = rng.standard_normal((Bn, H))
    lam = rng.standard_normal((Bn, H))
    a, c_r, c_z, c_n, c_np = O.adjoint_coefficients(W_hh, b_hh, gi, hp, gamma, cell)
    dA_h = np.concatenate([c_r * lam, c_z * lam, c_n * lam], -1)
    dA_i = np.concatenate([c_r * lam, c_z * lam, c_np * lam], -1)
    lam_prev = a * lam + dA_h @ W_hh
    F = lambda W, b, g, h: np.sum(lam * O.phi(W, b, g, h, gamma, cell))
    eps = 1e-6

    def fd(arr, setter):
        out = np.zeros_like(arr)
        it = np.nditer(arr, flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            p = arr.copy(); p[idx] += eps
            m = arr.copy(); m[idx] -= eps
            out[idx] = (setter(p) - setter(m)) / (2 * eps)
        return out

    assert np.max(np.abs(fd(hp, lambda v: F(W_hh, b_hh, gi, v)) - lam_prev)) < 1e-8
    assert np.max(np.abs(fd(gi, lambda v: F(W_hh, b_hh, v, hp)) - dA_i)) < 1e-8
    assert np.max(np.abs(fd(b_hh, lambda v: F(W_hh, v, gi, hp)) - dA_h.sum(0))) < 1e-8
    assert np.max(np.abs(fd(W_hh, lambda v: F(v, b_hh, gi, hp)) - dA_h.T @ hp)) < 1e-8


def test_implicit_bptt_vs_finite_differences_of_the_loss():
    w = tiny_workload(T=6, B=2, I=3, H=4, classes=3)
    P, x, h0, d = f64_inputs(w)
    rng = np.random.default_rng(11)
    h0 = rng.standard_normal(h0.shape) * 0.3
    Wc, bc, lab = d["W_c"].astype(np.float64), d["b_c"].astype(np.float64), d["labels"]

    def loss(Pv, xv, h0v):
        h = O.serial_forward(*Pv, xv, h0v)
        return O.xent_head(h[-1], Wc, bc, lab)[0]

    h = O.serial_forward(*P, x, h0)
    _, dhT, _, _ = O.xent_head(h[-1], Wc, bc, lab)
    seed = np.zeros_like(h); seed[-1] = dhT
    lam, lam0, g = O.serial_backward(*P, x, h0, h, seed)
    eps = 1e-6
    names = ["dW_ih", "dW_hh", "db_ih", "db_hh"]
    for pi, nm in enumerate(names):
        ref = np.zeros_like(P[pi])
        it = np.nditer(P[pi], flags=["multi_index"])
        for _ in it:
            idx = it.multi_index
            Pp = [a.copy() for a in P]; Pp[pi][idx] += eps
            Pm = [a.copy() for a in P]; Pm[pi][idx] -= eps
            ref[idx] = (loss(Pp, x, h0) - loss(Pm, x, h0)) / (2 * eps)
        assert np.max(np.abs(ref - g[nm])) < 1e-8 * max(1.0, np.max(np.abs(ref))), nm
    refx = np.zeros_like(x)
    it = np.nditer(x, flags=["multi_index"])
    for _ in it:
        idx = it.multi_index
        xp = x.copy(); xp[idx] += eps
        xm = x.copy(); xm[idx] -= eps
        refx[idx] = (loss(P, xp, h0) - loss(P, xm, h0)) / (2 * eps)
    assert np.max(np.abs(refx - g["dx"])) < 1e-8
    refh = np.zeros_like(h0)
    it = np.nditer(h0, flags=["multi_index"])
    for _ in it:
        idx = it.multi_index
        hp_ = h0.copy(); hp_[idx] += eps
        hm_ = h0.copy(); hm_[idx] -= eps
        refh[idx] = (loss(P, x, hp_) - loss(P, x, hm_)) / (2 * eps)
    assert np.max(np.abs(refh - lam0)) < 1e-8


def test_xent_head_equals_library():
    rng = np.random.default_rng(4)
    Bn, H, C = 5, 7, 4
    hT = rng.standard_normal((Bn, H)); Wc = rng.standard_normal((C, H)); bc = rng.standard_normal(C)
    lab = rng.integers(0, C, Bn)
    loss, dh, dW, db = O.xent_head(hT, Wc, bc, lab)
    ht = torch.from_numpy(hT).requires_grad_(True)
    Wt = torch.from_numpy(Wc).requires_grad_(True)
    bt = torch.from_numpy(bc).requires_grad_(True)
    L = torch.nn.functional.cross_entropy(ht @ Wt.T + bt, torch.from_numpy(lab).long())
    L.backward()
    assert abs(L.item() - loss) < 1e-13
    assert np.max(np.abs(ht.grad.numpy() - dh)) < 1e-13
    assert np.max(np.abs(Wt.grad.numpy() - dW)) < 1e-13
    assert np.max(np.abs(bt.grad.numpy() - db)) < 1e-13
    assert np.allclose(O.sgd_update(Wc, dW, 0.5), Wc - 0.5 * dW)


def test_adam_equals_library():
    rng = np.random.default_rng(6)
    p0 = rng.standard_normal(17)
    pt = torch.from_numpy(p0.copy()).requires_grad_(True)
    opt = torch.optim.Adam([pt], lr=1e-2)
    p, m, v = p0.copy(), np.zeros(17), np.zeros(17)
    for step in range(1, 6):
        g = rng.standard_normal(17)
        pt.grad = torch.from_numpy(g.copy())
        opt.step()
        p, m, v = O.adam_update(p, g, m, v, 1e-2, step)
        assert np.max(np.abs(p - pt.detach().numpy())) < 1e-12
