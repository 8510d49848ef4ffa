"""Pins for the oracle's Implicit LSTM (CPU only).

The paper names the LSTM as a cell its implicit treatment carries over to; the reading taken (cell state as a
forward-Euler step of c' = -(1-f) c + i g, decay term implicit, h re-evaluated from the new c) is pinned by: the
explicit cell with unit step IS torch.nn.LSTM (float64, forward and autograd); the defining identity and the limits
of the implicit step; the model-problem amplification factors; finite differences for the adjoint; and the same
MGRIT facts as for the GRU (fixed point, exactness count, monotone residual, limit = serial sweep)."""
import numpy as np
import pytest
import torch

from oracle import mgrit_gru_oracle as O


def _setup(T=16, B=2, I=3, H=5, seed=0):
    rng = np.random.default_rng(seed)
    k = 1.0 / np.sqrt(H)
    P = (rng.uniform(-k, k, (4 * H, I)), rng.uniform(-k, k, (4 * H, H)), rng.uniform(-k, k, 4 * H), rng.uniform(-k, k, 4 * H))
    return P, rng.standard_normal((T, B, I)), rng.standard_normal((2, B, H)) * 0.4, rng


def test_classic_lstm_is_torch_lstm_forward_and_backward():
    P, x, u0, rng = _setup(T=12)
    T, B, I = x.shape
    H = u0.shape[-1]
    u = O.lstm_serial_forward(*P, x, u0, cell=O.CELL_CLASSIC)
    lstm = torch.nn.LSTM(I, H).double()
    with torch.no_grad():
        for name, arr in zip(("weight_ih_l0", "weight_hh_l0", "bias_ih_l0", "bias_hh_l0"), P):
            getattr(lstm, name).copy_(torch.from_numpy(arr))
    xt = torch.from_numpy(x).requires_grad_(True)
    c0 = torch.from_numpy(u0[0:1]).requires_grad_(True)
    h0 = torch.from_numpy(u0[1:2]).requires_grad_(True)
    out, (hn, cn) = lstm(xt, (h0, c0))
    assert np.max(np.abs(out.detach().numpy() - u[:, 1])) < 1e-14
    assert np.max(np.abs(cn.detach().numpy()[0] - u[-1, 0])) < 1e-14
    wgt = torch.from_numpy(rng.standard_normal(out.shape))
    wc = torch.from_numpy(rng.standard_normal(cn.shape))
    ((out * wgt).sum() + (cn * wc).sum()).backward()
    seed = np.zeros_like(u)
    seed[:, 1] = wgt.numpy()
    seed[-1, 0] = wc.numpy()[0]
    lam, lam0, g = O.lstm_serial_backward(*P, x, u0, u, seed, cell=O.CELL_CLASSIC)
    assert np.max(np.abs(c0.grad.numpy()[0] - lam0[0])) < 1e-13 and np.max(np.abs(h0.grad.numpy()[0] - lam0[1])) < 1e-13
    assert np.max(np.abs(xt.grad.numpy() - g["dx"])) < 1e-13
    for name, key in (("weight_ih_l0", "dW_ih"), ("weight_hh_l0", "dW_hh"), ("bias_ih_l0", "db_ih"), ("bias_hh_l0", "db_hh")):
        assert np.max(np.abs(getattr(lstm, name).grad.numpy() - g[key])) < 1e-12, key


def test_implicit_lstm_identity_limits_and_stability():
    P, x, u0, rng = _setup()
    gi = x[0] @ P[0].T + P[2]
    i, f, g, o = O.lstm_gates(P[1], P[3], gi, u0[1])
    for gamma in (0.5, 1.0, 4.0, 16.0):
        u = O.lstm_phi(P[1], P[3], gi, u0, gamma, O.CELL_IMPLICIT)
        # defining relation of the implicit step, and h re-evaluated from the new cell state
        assert np.max(np.abs((1 + gamma * (1 - f)) * u[0] - u0[0] - gamma * i * g)) < 1e-14
        assert np.max(np.abs(u[1] - o * np.tanh(u[0]))) < 1e-15
        # convex combination of the old cell state and the gate target i g / (1 - f): never leaves their hull
        tgt = i * g / (1 - f)
        lo, hi = np.minimum(u0[0], tgt), np.maximum(u0[0], tgt)
        assert np.all(u[0] >= lo - 1e-12) and np.all(u[0] <= hi + 1e-12)
        # difference to the explicit step: -q^2 (target - c) / (1 + q) with q = gamma (1 - f)
        ue = O.lstm_phi(P[1], P[3], gi, u0, gamma, O.CELL_CLASSIC)
        q = gamma * (1 - f)
        assert np.max(np.abs((u[0] - ue[0]) - (-q * q * (tgt - u0[0]) / (1 + q)))) < 1e-12
    # gamma -> 0: the cell state does not move
    u = O.lstm_phi(P[1], P[3], gi, u0, 1e-12, O.CELL_IMPLICIT)
    assert np.max(np.abs(u[0] - u0[0])) < 1e-11
    # model problem (i = 0): explicit amplification 1 - gamma (1 - f) leaves [-1, 1] for large steps, implicit 1 / (1 + gamma (1 - f)) never
    assert np.all(1.0 / (1 + 16.0 * (1 - f)) <= 1.0) and np.any(np.abs(1 - 16.0 * (1 - f)) > 1.0)


@pytest.mark.parametrize("cell", [O.CELL_CLASSIC, O.CELL_IMPLICIT])
def test_lstm_adjoint_against_finite_differences(cell):
    P, x, u0, rng = _setup(T=9)
    u = O.lstm_serial_forward(*P, x, u0, cell=cell, dt=1.5)
    seed = rng.standard_normal(u.shape)
    lam, lam0, g = O.lstm_serial_backward(*P, x, u0, u, seed, cell=cell, dt=1.5)
    loss = lambda PP, xx, uu0: float(np.sum(seed * O.lstm_serial_forward(*PP, xx, uu0, cell=cell, dt=1.5)))
    eps = 1e-6
    for idx, key in ((0, "dW_ih"), (1, "dW_hh"), (2, "db_ih"), (3, "db_hh")):
        for _ in range(3):
            pos = tuple(int(v) for v in rng.integers(0, np.array(P[idx].shape)))
            def pert(d):
                PP = [a.copy() for a in P]
                PP[idx][pos] += d
                return PP
            fd = (loss(pert(eps), x, u0) - loss(pert(-eps), x, u0)) / (2 * eps)
            assert abs(fd - g[key][pos]) < 1e-7 * max(1.0, abs(fd)), key
    for arr, grad in ((u0, lam0), (x, g["dx"])):
        d = rng.standard_normal(arr.shape)
        if arr is u0:
            fd = (loss(P, x, u0 + eps * d) - loss(P, x, u0 - eps * d)) / (2 * eps)
        else:
            fd = (loss(P, x + eps * d, u0) - loss(P, x - eps * d, u0)) / (2 * eps)
        assert abs(fd - np.sum(grad * d)) < 1e-7 * max(1.0, abs(fd))


def test_lstm_mgrit_fixed_point_exactness_and_limit():
    P, x, u0, rng = _setup(T=32)
    us = O.lstm_serial_forward(*P, x, u0)
    u, res = O.lstm_mgrit_forward(*P, x, u0, cf=4, levels=2, iters=1, u_init=us)
    assert np.max(np.abs(u - us)) < 1e-14 and res[0] < 1e-13
    u, _ = O.lstm_mgrit_forward(*P, x, u0, cf=4, levels=2, iters=8, relax_fine=O.RELAX_F)
    assert np.max(np.abs(u - us)) < 1e-13
    u, _ = O.lstm_mgrit_forward(*P, x, u0, cf=4, levels=2, iters=6, relax_fine=O.RELAX_F)
    assert np.max(np.abs(u - us)) > 1e-10
    u, res = O.lstm_mgrit_forward(*P, x, u0, cf=2, levels=4, iters=10)
    res = [r for r in res if r > 1e-13]
    assert all(b < a for a, b in zip(res, res[1:])) and np.max(np.abs(u - us)) < 1e-5
    seed = rng.standard_normal(us.shape)
    lam_s, lam0_s, g_s = O.lstm_serial_backward(*P, x, u0, us, seed)
    lam, lam0, g, _ = O.lstm_mgrit_adjoint(*P, x, u0, us, seed, cf=4, levels=2, iters=8, relax_fine=O.RELAX_F)
    assert np.max(np.abs(lam - lam_s)) < 1e-13 and np.max(np.abs(lam0 - lam0_s)) < 1e-13
    for k in g_s:
        assert np.max(np.abs(g[k] - g_s[k])) < 1e-12, k
    # ragged length, three levels: converges to the same limits
    P, x, u0, rng = _setup(T=27, seed=3)
    us = O.lstm_serial_forward(*P, x, u0)
    u, _ = O.lstm_mgrit_forward(*P, x, u0, cf=2, levels=3, iters=14, ragged=True)
    assert np.max(np.abs(u - us)) < 1e-6
    seed = rng.standard_normal(us.shape)
    lam_s, _, _ = O.lstm_serial_backward(*P, x, u0, us, seed)
    lam, _, _, _ = O.lstm_mgrit_adjoint(*P, x, u0, us, seed, cf=2, levels=3, iters=14, ragged=True)
    assert np.max(np.abs(lam - lam_s)) < 1e-6 * max(1.0, np.max(np.abs(lam_s)))
