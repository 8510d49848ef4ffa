"""Pins for the oracle's stacked-layer functions (CPU only): all layers in one state, one cycle for the stack.

The paper's experiments use a 2-layer GRU; the stacked state (layer k's input at a step = layer k-1's new state of
that step) with the classic cell and unit time step is the textbook multi-layer GRU, which pins the step, the serial
sweep and the exact back-propagation against torch.nn.GRU(num_layers=2) in float64.  The MGRIT solves are pinned
through the same facts as the single-layer ones: the serial solution is a fixed point, two-level F-relaxation is
exact after T/c_f cycles (forward and adjoint), residuals fall monotonically, and with one layer every function
reduces to its single-layer counterpart."""
import numpy as np
import pytest
import torch

from oracle import mgrit_gru_oracle as O


def _layers(rng, I, H, nl):
    out = []
    k = 1.0 / np.sqrt(H)
    for q in range(nl):
        Iq = I if q == 0 else H
        out.append((rng.uniform(-k, k, (3 * H, Iq)), rng.uniform(-k, k, (3 * H, H)), rng.uniform(-k, k, 3 * H), rng.uniform(-k, k, 3 * H)))
    return out


def _setup(T=16, B=2, I=3, H=5, nl=2, seed=0):
    rng = np.random.default_rng(seed)
    layers = _layers(rng, I, H, nl)
    return layers, rng.standard_normal((T, B, I)), rng.standard_normal((nl, B, H)) * 0.3, rng


def test_classic_stack_is_torch_multilayer_gru_forward_and_backward():
    layers, x, h0, rng = _setup(T=12)
    T, B, I = x.shape
    H = h0.shape[-1]
    h = O.stacked_serial_forward(layers, x, h0, cell=O.CELL_CLASSIC)
    gru = torch.nn.GRU(I, H, num_layers=2).double()
    with torch.no_grad():
        for k in range(2):
            for name, arr in zip(("weight_ih", "weight_hh", "bias_ih", "bias_hh"), layers[k]):
                getattr(gru, f"{name}_l{k}").copy_(torch.from_numpy(arr))
    xt = torch.from_numpy(x).requires_grad_(True)
    h0t = torch.from_numpy(h0).requires_grad_(True)
    out, hn = gru(xt, h0t)
    assert np.max(np.abs(out.detach().numpy() - h[:, 1])) < 1e-14
    assert np.max(np.abs(hn.detach().numpy() - h[-1])) < 1e-14
    wgt = torch.from_numpy(rng.standard_normal(out.shape))
    (out * wgt).sum().backward()
    seed = np.zeros_like(h)
    seed[:, 1] = wgt.numpy()
    lam, lam0, grads = O.stacked_serial_backward(layers, x, h0, h, seed, cell=O.CELL_CLASSIC)
    assert np.max(np.abs(h0t.grad.numpy() - lam0)) < 1e-13
    assert np.max(np.abs(xt.grad.numpy() - grads[0]["dx"])) < 1e-13
    for k in range(2):
        for name, key in (("weight_ih", "dW_ih"), ("weight_hh", "dW_hh"), ("bias_ih", "db_ih"), ("bias_hh", "db_hh")):
            assert np.max(np.abs(getattr(gru, f"{name}_l{k}").grad.numpy() - grads[k][key])) < 1e-12, (k, key)


def test_one_layer_stack_reduces_to_the_single_layer_functions():
    layers, x, h0, rng = _setup(T=16, nl=1)
    P = layers[0]
    kw = dict(cf=2, levels=3, iters=2, relax_fine=1, relax_coarse=1)
    h, res = O.stacked_mgrit_forward(layers, x, h0, **kw)
    h1, res1 = O.mgrit_forward(*P, x, h0[0], **kw)
    assert np.max(np.abs(h[:, 0] - h1)) < 1e-15 and np.max(np.abs(np.array(res) - np.array(res1))) < 1e-14
    seed = rng.standard_normal(h.shape)
    lam, lam0, g, _ = O.stacked_mgrit_adjoint(layers, x, h0, h, seed, **kw)
    lam1, lam01, g1, _ = O.mgrit_adjoint(*P, x, h0[0], h1, seed[:, 0], **kw)
    assert np.max(np.abs(lam[:, 0] - lam1)) < 1e-14 and np.max(np.abs(lam0[0] - lam01)) < 1e-14
    for k in g1:
        assert np.max(np.abs(g[0][k] - g1[k])) < 1e-13, k


def test_stacked_mgrit_fixed_point_exactness_and_monotone_residual():
    layers, x, h0, rng = _setup(T=32)
    hs = O.stacked_serial_forward(layers, x, h0)
    h, res = O.stacked_mgrit_forward(layers, x, h0, cf=4, levels=2, iters=1, h_init=hs)
    assert np.max(np.abs(h - hs)) < 1e-14 and res[0] < 1e-13
    h, _ = O.stacked_mgrit_forward(layers, x, h0, cf=4, levels=2, iters=8, relax_fine=O.RELAX_F)      # T / cf cycles
    assert np.max(np.abs(h - hs)) < 1e-13
    h, _ = O.stacked_mgrit_forward(layers, x, h0, cf=4, levels=2, iters=6, relax_fine=O.RELAX_F)
    assert np.max(np.abs(h - hs)) > 1e-10
    h, res = O.stacked_mgrit_forward(layers, x, h0, cf=2, levels=4, iters=10)
    res = [r for r in res if r > 1e-13]
    assert all(b < a for a, b in zip(res, res[1:])) and np.max(np.abs(h - hs)) < 1e-5
    # prefix exactness: after k cycles the first k*cf states of every layer are the serial ones
    h, _ = O.stacked_mgrit_forward(layers, x, h0, cf=4, levels=3, iters=2)
    assert np.max(np.abs(h[:8] - hs[:8])) < 1e-14 and np.max(np.abs(h - hs)) > 1e-6


@pytest.mark.parametrize("ragged", [False, True])
def test_stacked_adjoint_exact_after_enough_cycles_and_against_finite_differences(ragged):
    T = 19 if ragged else 16
    layers, x, h0, rng = _setup(T=T)
    hs = O.stacked_serial_forward(layers, x, h0)
    seed = rng.standard_normal(hs.shape)
    lam_s, lam0_s, g_s = O.stacked_serial_backward(layers, x, h0, hs, seed)
    need = T // 4 + 1
    lam, lam0, g, res = O.stacked_mgrit_adjoint(layers, x, h0, hs, seed, cf=4, levels=2, iters=need, relax_fine=O.RELAX_F, ragged=ragged)
    assert np.max(np.abs(lam - lam_s)) < 1e-13 and np.max(np.abs(lam0 - lam0_s)) < 1e-13
    for k in range(2):
        for key in g_s[k]:
            assert np.max(np.abs(g[k][key] - g_s[k][key])) < 1e-12, (k, key)
    # the serial gradients against central finite differences of  L = sum(seed * h)  (implicit cell, fp64)
    def loss(ls, xx, hh0):
        return float(np.sum(seed * O.stacked_serial_forward(ls, xx, hh0)))
    eps = 1e-6
    for k, idx, key in ((0, 1, "dW_hh"), (1, 0, "dW_ih"), (1, 3, "db_hh")):
        arr = layers[k][idx]
        pos = tuple(int(v) for v in rng.integers(0, np.array(arr.shape)))
        def pert(d):
            ls = [list(l) for l in layers]
            a2 = arr.copy(); a2[pos] += d
            ls[k][idx] = a2
            return [tuple(l) for l in ls]
        fd = (loss(pert(eps), x, h0) - loss(pert(-eps), x, h0)) / (2 * eps)
        assert abs(fd - g_s[k][key][pos]) < 1e-7 * max(1.0, abs(fd)), (k, key)
    d = rng.standard_normal(h0.shape)
    fd = (loss(layers, x, h0 + eps * d) - loss(layers, x, h0 - eps * d)) / (2 * eps)
    assert abs(fd - np.sum(lam0_s * d)) < 1e-7 * max(1.0, abs(fd))
