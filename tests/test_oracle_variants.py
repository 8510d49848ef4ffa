"""Pins for the oracle's cycle variants (CPU only): relaxation F(CF)^n, F-cycles, and sequence lengths that are not
a multiple of c_f^(levels-1).

The paper defines F- and FCF-relaxation (Eq. "fcf-relax") and uses T = 128 throughout; the variants here are the
readings recorded for them: FCFCF composes the C and F sweeps once more; an F-cycle follows the correction of every
level by one more V-cycle from that level down; for a ragged T the C-points of a level are its points 0, c_f,
2 c_f, ... and whatever follows the last one is a shorter interval of F-points (forward grids anchored at t = 0,
the adjoint's reversed grids at t = T).  Each is pinned against what the mathematics fixes: exactness counts,
identities between cycle types, the serial sweep as the limit, and cycles written out statement by statement.
"""
import numpy as np
import pytest

from oracle import mgrit_gru_oracle as O
from tests.helpers import f64_inputs, tiny_workload


def _setup(T, B=2, I=3, H=5, seed=21):
    w = tiny_workload(T=T, B=B, I=I, H=H)
    P, x, h0, _ = f64_inputs(w)
    h0 = np.random.default_rng(seed).standard_normal(h0.shape) * 0.5
    return P, x, h0


# ------------------------------------------------------------------------------------------ FCFCF
def test_fcfcf_two_level_exactness_count():
    # every CF pair carries exact values one interval further: F(CF)^n is exact after ceil((T/cf) / (n+1)) cycles
    P, x, h0 = _setup(64)
    hs = O.serial_forward(*P, x, h0)
    for n, need in ((1, 8), (2, 6), (3, 4)):
        h, _ = O.mgrit_forward(*P, x, h0, cf=4, levels=2, iters=need, relax_fine=n)
        assert np.max(np.abs(h - hs)) < 1e-13, n
        h, _ = O.mgrit_forward(*P, x, h0, cf=4, levels=2, iters=need - 1, relax_fine=n)
        assert np.max(np.abs(h - hs)) > 1e-10, n


def test_fcfcf_equals_fcf_followed_by_one_more_cf_sweep():
    # written out on two levels: relax = 2 is the FCF cycle with one more C sweep and F sweep before the residual
    T, cf = 12, 3
    P, x, h0 = _setup(T)
    gi = x @ P[0].T + P[2]
    f = lambda j, prev: O.phi(P[1], P[3], gi[j - 1], prev, 1.0, O.CELL_IMPLICIT)
    c = lambda k, prev: O.phi(P[1], P[3], gi[cf * k - 1], prev, float(cf), O.CELL_IMPLICIT)
    u = np.zeros((T + 1,) + h0.shape)
    u[0] = h0
    F = lambda: [u.__setitem__(j, f(j, u[j - 1])) for k in range(T // cf) for j in range(k * cf + 1, k * cf + cf)]
    C = lambda: [u.__setitem__(k * cf, f(k * cf, u[k * cf - 1])) for k in range(1, T // cf + 1)]
    F(); C(); F(); C(); F()
    v = [f(k * cf, u[k * cf - 1]) for k in range(1, T // cf + 1)]
    U = [u[0]] + [u[k * cf].copy() for k in range(1, T // cf + 1)]
    G = [None] + [v[k - 1] - c(k, U[k - 1]) for k in range(1, T // cf + 1)]
    for k in range(1, T // cf + 1):
        U[k] = c(k, U[k - 1]) + G[k]
        u[k * cf] = U[k]
    F()
    h, _ = O.mgrit_forward(*P, x, h0, cf=cf, levels=2, iters=1, relax_fine=O.RELAX_FCFCF)
    assert np.max(np.abs(h - u[1:])) < 1e-14


# ------------------------------------------------------------------------------------------ F-cycle
def test_f_cycle_on_two_levels_is_two_v_cycles():
    P, x, h0 = _setup(32)
    for k in (1, 2):
        hF, rF = O.mgrit_forward(*P, x, h0, cf=4, levels=2, iters=k, cycle=O.CYCLE_F)
        hV, rV = O.mgrit_forward(*P, x, h0, cf=4, levels=2, iters=2 * k)
        assert np.max(np.abs(hF - hV)) < 1e-14
        assert np.max(np.abs(np.array(rF) - np.array(rV[0::2]))) < 1e-13     # only the first residual of a cycle is recorded


def test_f_cycle_three_levels_written_out():
    # F(0) = [relax, restrict, F(1), correct, F-relax] then V(0);  F(1) on the last two levels = two V(1).
    # The level-1 pieces are run through the oracle's own two-level machinery (pinned elsewhere) on the level-1
    # system with its FAS term; what is pinned here is the ORDER in which an F-cycle visits the levels.
    T, cf = 16, 2
    P, x, h0 = _setup(T)
    hs = O.serial_forward(*P, x, h0)
    gi = x @ P[0].T + P[2]

    def step(l, j, prev):
        m = cf ** l
        return O.phi(P[1], P[3], gi[m * j - 1], prev, float(m), O.CELL_IMPLICIT)

    N = [16, 8, 4]
    relax = [O.RELAX_F, O.RELAX_FCF, O.RELAX_FCF]
    u = [np.zeros((T + 1,) + h0.shape), None, None]
    g = [np.zeros_like(u[0]), None, None]
    u[0][0] = h0

    def F0():
        for s in range(1, cf):
            j = np.arange(0, N[0], cf) + s
            u[0][j] = step(0, j, u[0][j - 1])

    # ---- down-leg on level 0
    F0()
    jc = np.arange(cf, N[0] + 1, cf)
    v = step(0, jc, u[0][jc - 1])
    u[1] = np.concatenate([u[0][0:1], u[0][jc]], 0)
    g[1] = np.zeros_like(u[1])
    g[1][1:] = v - step(1, np.arange(1, N[1] + 1), u[1][:-1])
    # ---- F(1): two V-cycles of the (level 1, level 2) pair
    O.fas_vcycle(step, N, cf, relax, u, g, 1, None, O.CYCLE_V)
    O.fas_vcycle(step, N, cf, relax, u, g, 1, None, O.CYCLE_V)
    # ---- up-leg on level 0, then V(0)
    u[0][jc] = u[1][1:]
    F0()
    O.fas_vcycle(step, N, cf, relax, u, g, 0, None, O.CYCLE_V)
    h, _ = O.mgrit_forward(*P, x, h0, cf=cf, levels=3, iters=1, cycle=O.CYCLE_F)
    assert np.max(np.abs(h - u[0][1:])) < 1e-14
    # and an F-cycle reduces the error at least as much as a V-cycle
    hV, _ = O.mgrit_forward(*P, x, h0, cf=cf, levels=3, iters=1)
    assert np.max(np.abs(h - hs)) < np.max(np.abs(hV - hs))


def test_f_cycle_adjoint_two_levels_is_two_v_cycles():
    P, x, h0 = _setup(32)
    h = O.serial_forward(*P, x, h0)
    seed = np.random.default_rng(2).standard_normal(h.shape)
    lF, l0F, gF, _ = O.mgrit_adjoint(*P, x, h0, h, seed, cf=4, levels=2, iters=1, cycle=O.CYCLE_F)
    lV, l0V, gV, _ = O.mgrit_adjoint(*P, x, h0, h, seed, cf=4, levels=2, iters=2)
    assert np.max(np.abs(lF - lV)) < 1e-14 and np.max(np.abs(l0F - l0V)) < 1e-14


# ------------------------------------------------------------------------------------------ ragged T
def test_ragged_level_sizes():
    assert O.level_sizes(100, 8, 3, ragged=True) == [100, 12, 1]
    assert O.level_sizes(128, 4, 3, ragged=True) == [128, 32, 8]
    with pytest.raises(ValueError):
        O.level_sizes(7, 4, 3, ragged=True)


def test_ragged_forward_T7_cf2_statement_by_statement():
    # T = 7, c_f = 2: fine points 0..7, C-points 0, 2, 4, 6, and the last point 7 is an F-point of a one-point interval
    P, x, h0 = _setup(7, B=1)
    gi = x @ P[0].T + P[2]
    a = lambda t, hp: O.phi(P[1], P[3], gi[t - 1], hp, 1.0, O.CELL_IMPLICIT)
    c = lambda t, hp: O.phi(P[1], P[3], gi[t - 1], hp, 2.0, O.CELL_IMPLICIT)
    z = np.zeros_like(h0)
    u0, u2, u4, u6 = h0, z, z, z
    u1 = a(1, u0); u3 = a(3, u2); u5 = a(5, u4); u7 = a(7, u6)          # F-relaxation, the tail point included
    v2 = a(2, u1); v4 = a(4, u3); v6 = a(6, u5)                          # three C-points
    r = [u2 - v2, u4 - v4, u6 - v6]
    G2 = v2 - c(2, u0); G4 = v4 - c(4, u2); G6 = v6 - c(6, u4)
    U2 = c(2, u0) + G2; U4 = c(4, U2) + G4; U6 = c(6, U4) + G6
    u2, u4, u6 = U2, U4, U6
    u1 = a(1, u0); u3 = a(3, u2); u5 = a(5, u4); u7 = a(7, u6)
    h, res = O.mgrit_forward(*P, x, h0, cf=2, levels=2, iters=1, ragged=True)
    assert np.max(np.abs(h - np.stack([u1, u2, u3, u4, u5, u6, u7]))) < 1e-15
    assert abs(res[0] - np.sqrt(sum(np.sum(q * q) for q in r))) < 1e-14


@pytest.mark.parametrize("T,cf,levels", [(23, 4, 2), (50, 3, 3), (37, 2, 4)])
def test_ragged_forward_and_adjoint_converge_to_the_serial_sweep(T, cf, levels):
    P, x, h0 = _setup(T)
    hs = O.serial_forward(*P, x, h0)
    seed = np.random.default_rng(8).standard_normal(hs.shape)
    lam_s, lam0_s, g_s = O.serial_backward(*P, x, h0, hs, seed)
    # the serial solution is a fixed point
    h, res = O.mgrit_forward(*P, x, h0, cf=cf, levels=levels, iters=1, ragged=True, h_init=hs)
    assert np.max(np.abs(h - hs)) < 1e-14 and res[0] < 1e-13
    # two-level F-relaxation: exact once the exact prefix has crossed all floor(T/cf) + 1 intervals
    need = T // cf + 1
    h, _ = O.mgrit_forward(*P, x, h0, cf=cf, levels=2, iters=need, ragged=True, relax_fine=O.RELAX_F)
    assert np.max(np.abs(h - hs)) < 1e-13
    lam, lam0, g, _ = O.mgrit_adjoint(*P, x, h0, hs, seed, cf=cf, levels=2, iters=need, ragged=True, relax_fine=O.RELAX_F)
    assert np.max(np.abs(lam - lam_s)) < 1e-12 and np.max(np.abs(lam0 - lam0_s)) < 1e-12
    for k in g_s:
        assert np.max(np.abs(g[k] - g_s[k])) < 1e-11, k
    # multilevel: monotone residual, limit = serial
    h, res = O.mgrit_forward(*P, x, h0, cf=cf, levels=levels, iters=12, ragged=True)
    res = [r for r in res if r > 1e-13]
    assert all(b < a for a, b in zip(res, res[1:]))
    assert np.max(np.abs(h - hs)) < 1e-5
    lam, _, _, res = O.mgrit_adjoint(*P, x, h0, hs, seed, cf=cf, levels=levels, iters=12, ragged=True)
    assert np.max(np.abs(lam - lam_s)) < 1e-5 * max(1.0, np.max(np.abs(lam_s)))


def test_ragged_adjoint_T5_cf2_statement_by_statement():
    # T = 5, c_f = 2, two levels.  Reversed points s = 0..5 sit at fine times 5, 4, 3, 2, 1, 0; the reversed C-points
    # s = 2, 4 at fine times 3 and 1 (anchored at T), s = 5 (time 0) is the tail F-point.  The coarse step into
    # reversed C-point k transposes the forward step of time step 2 that arrives at fine time 5 - 2(k-1).
    H = 5
    P, x, h0 = _setup(5, B=1, H=H)
    W_hh, b_hh = P[1], P[3]
    gi = x @ P[0].T + P[2]
    h = O.serial_forward(*P, x, h0)
    hfull = np.concatenate([h0[None], h], 0)
    seed = np.random.default_rng(4).standard_normal(h.shape)

    def JT(t_arrive, m):
        a, c_r, c_z, c_n, _ = O.adjoint_coefficients(W_hh, b_hh, gi[t_arrive - 1], hfull[t_arrive - m], float(m), O.CELL_IMPLICIT)
        M = np.diag(a[0])
        for gate, cg in enumerate((c_r, c_z, c_n)):
            M = M + W_hh[gate * H:(gate + 1) * H].T @ np.diag(cg[0])
        return M

    f = lambda s, mu: mu @ JT(5 - (s - 1), 1).T          # fine reversed step into s
    c = lambda k, mu: mu @ JT(5 - 2 * (k - 1), 2).T      # coarse reversed step into coarse point k (fine s = 2k)
    src = lambda s: seed[5 - s - 1] if s < 5 else 0.0    # direct loss derivative at fine time 5 - s
    z = np.zeros((1, H))
    m0, m2, m4 = seed[4], z, z
    m1 = f(1, m0) + src(1); m3 = f(3, m2) + src(3); m5 = f(5, m4) + src(5)      # F-relaxation with the tail point s = 5
    v2 = f(2, m1) + src(2); v4 = f(4, m3) + src(4)
    G2 = v2 - c(1, m0); G4 = v4 - c(2, m2)
    U2 = c(1, m0) + G2; U4 = c(2, U2) + G4
    m2, m4 = U2, U4
    m1 = f(1, m0) + src(1); m3 = f(3, m2) + src(3); m5 = f(5, m4) + src(5)
    lam, lam0, _, _ = O.mgrit_adjoint(*P, x, h0, h, seed, cf=2, levels=2, iters=1, ragged=True, relax_fine=O.RELAX_F)
    want = np.stack([m4, m3, m2, m1, m0])                 # lam[k] = dL/dh_{k+1} = mu at fine time k+1 = mu_{5-(k+1)}
    assert np.max(np.abs(lam - want)) < 1e-14 and np.max(np.abs(lam0 - m5)) < 1e-14
