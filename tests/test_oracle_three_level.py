"""Pins for the oracle's multilevel recursion (CPU only): a THREE-level cycle written out level by level.

Remark "Beyond Two-Level" says the coarse equation of Algorithm "MGProp" is itself solved by MGProp, and Section
"Coarse Grid Propagators" fixes the coarse time step ("on coarse grids the time step is equal to c_f^l"), while
Eq. "restrict" injects the coarse input sequence x_{c_f t}.  So on level l the step into point j is
Phi with gamma = c_f^l and the input of fine step c_f^l j (array row c_f^l j - 1), and the level-1 system carries
the FAS term of the level-0 residual.  None of the two-level pins can see those three facts; the cases below do:
every level is spelled out with its own propagator, no recursion, no shared step function, and the level-2
propagator is never built from a formula in l.  Sizes are chosen so that c_f^2 != 2 c_f (c_f = 3, 4) next to the
T = 8, c_f = 2 case, which is written out statement by statement, and so that level 2 has three points (with two,
FCF-relaxation on level 1 makes the level-2 solve independent of its propagator).
"""
import numpy as np
import pytest

from oracle import mgrit_gru_oracle as O
from tests.helpers import f64_inputs, tiny_workload


def _three_level_cycle(cf, N0, f0, f1, f2, u, g0, relax0, relax1):
    """One cycle of Algorithm "MGProp" on level 0 whose coarse solve is one MGProp on levels 1 and 2 and whose
    level 2 is swept serially.  f0/f1/f2(j, prev): the three levels' propagators into their point j.
    u: level-0 unknowns [N0+1, ...] (u[0] fixed), g0: level-0 source.  Returns (new u, residual norm)."""
    u = u.copy()
    N1, N2 = N0 // cf, N0 // (cf * cf)

    # ---------------- level 0: relaxation
    def F0():
        for k in range(N1):
            for j in range(k * cf + 1, k * cf + cf):
                u[j] = f0(j, u[j - 1]) + g0[j]

    def C0():
        for k in range(1, N1 + 1):
            u[k * cf] = f0(k * cf, u[k * cf - 1]) + g0[k * cf]

    F0()
    if relax0 == O.RELAX_FCF:
        C0()
        F0()
    # residual at the level-0 C-points, restriction by injection
    v = {k: f0(k * cf, u[k * cf - 1]) + g0[k * cf] for k in range(1, N1 + 1)}
    rnorm = np.sqrt(sum(np.sum((u[k * cf] - v[k]) ** 2) for k in v))
    W = np.stack([u[k * cf] for k in range(N1 + 1)])            # level-1 unknowns, initial guess = restricted state
    G1 = np.zeros_like(W)
    for k in range(1, N1 + 1):
        G1[k] = v[k] - f1(k, W[k - 1])                          # FAS right-hand side of level 1

    # ---------------- level 1: the same algorithm on  W_k = f1(k, W_{k-1}) + G1_k
    def F1():
        for m in range(N2):
            for k in range(m * cf + 1, m * cf + cf):
                W[k] = f1(k, W[k - 1]) + G1[k]

    def C1():
        for m in range(1, N2 + 1):
            W[m * cf] = f1(m * cf, W[m * cf - 1]) + G1[m * cf]

    F1()
    if relax1 == O.RELAX_FCF:
        C1()
        F1()
    V = {m: f1(m * cf, W[m * cf - 1]) + G1[m * cf] for m in range(1, N2 + 1)}
    Z = np.stack([W[m * cf] for m in range(N2 + 1)])
    G2 = np.zeros_like(Z)
    for m in range(1, N2 + 1):
        G2[m] = V[m] - f2(m, Z[m - 1])
    # ---------------- level 2: serial
    for m in range(1, N2 + 1):
        Z[m] = f2(m, Z[m - 1]) + G2[m]
    # ---------------- back up: correct level 1, final F; correct level 0, final F
    for m in range(1, N2 + 1):
        W[m * cf] = Z[m]
    F1()
    for k in range(1, N1 + 1):
        u[k * cf] = W[k]
    F0()
    return u, rnorm


@pytest.mark.parametrize("cf,T", [(2, 12), (3, 27), (4, 48)])
@pytest.mark.parametrize("relax0,relax1", [(O.RELAX_F, O.RELAX_F), (O.RELAX_F, O.RELAX_FCF), (O.RELAX_FCF, O.RELAX_FCF)])
def test_forward_three_levels_written_out(cf, T, relax0, relax1):
    w = tiny_workload(T=T, B=2, I=3, H=5)
    P, x, h0, _ = f64_inputs(w)
    h0 = np.random.default_rng(5).standard_normal(h0.shape) * 0.5
    W_hh, b_hh = P[1], P[3]
    gi = x @ P[0].T + P[2]
    # level l, point j: time step c_f^l, input of fine step c_f^l * j  (0-based row c_f^l * j - 1)
    f0 = lambda j, prev: O.phi(W_hh, b_hh, gi[j - 1], prev, 1.0, O.CELL_IMPLICIT)
    f1 = lambda j, prev: O.phi(W_hh, b_hh, gi[cf * j - 1], prev, float(cf), O.CELL_IMPLICIT)
    f2 = lambda j, prev: O.phi(W_hh, b_hh, gi[cf * cf * j - 1], prev, float(cf * cf), O.CELL_IMPLICIT)
    u = np.zeros((T + 1,) + h0.shape)
    u[0] = h0
    g0 = np.zeros_like(u)
    want_res = []
    for it in range(2):                                   # the second cycle starts from a non-trivial iterate
        u, rn = _three_level_cycle(cf, T, f0, f1, f2, u, g0, relax0, relax1)
        want_res.append(rn)
        h, res = O.mgrit_forward(*P, x, h0, cf=cf, levels=3, iters=it + 1, relax_fine=relax0, relax_coarse=relax1)
        assert np.max(np.abs(h - u[1:])) < 1e-14
        assert np.max(np.abs(np.array(res) - np.array(want_res))) < 1e-13
        if it == 0:
            assert np.max(np.abs(u[1:] - O.serial_forward(*P, x, h0))) > 1e-6      # not vacuous: not converged yet


def test_forward_T8_cf2_statement_by_statement():
    # T = 8, c_f = 2, levels 8 / 4 / 2, F-relaxation on both non-coarsest levels, zero initial guess: every
    # assignment of the cycle written as its own statement.
    w = tiny_workload(T=8, B=1, I=3, H=5)
    P, x, h0, _ = f64_inputs(w)
    h0 = np.random.default_rng(6).standard_normal(h0.shape) * 0.5
    gi = x @ P[0].T + P[2]
    a = lambda t, hp: O.phi(P[1], P[3], gi[t - 1], hp, 1.0, O.CELL_IMPLICIT)   # level 0: step 1, into fine point t
    b = lambda t, hp: O.phi(P[1], P[3], gi[t - 1], hp, 2.0, O.CELL_IMPLICIT)   # level 1: step 2, into fine point t
    c = lambda t, hp: O.phi(P[1], P[3], gi[t - 1], hp, 4.0, O.CELL_IMPLICIT)   # level 2: step 4, into fine point t
    z = np.zeros_like(h0)
    u0, u2, u4, u6, u8 = h0, z, z, z, z
    u1 = a(1, u0); u3 = a(3, u2); u5 = a(5, u4); u7 = a(7, u6)                 # level 0 F-relaxation
    v2 = a(2, u1); v4 = a(4, u3); v6 = a(6, u5); v8 = a(8, u7)                 # level 0 residual points
    r = [u2 - v2, u4 - v4, u6 - v6, u8 - v8]
    W0, W1, W2, W3, W4 = u0, u2, u4, u6, u8                                    # level 1 = fine points 0,2,4,6,8
    G1 = v2 - b(2, W0); G2 = v4 - b(4, W1); G3 = v6 - b(6, W2); G4 = v8 - b(8, W3)
    W1 = b(2, W0) + G1; W3 = b(6, W2) + G3                                     # level 1 F-relaxation
    V2 = b(4, W1) + G2; V4 = b(8, W3) + G4                                     # level 1 residual points
    Z0, Z1, Z2 = W0, W2, W4                                                    # level 2 = fine points 0,4,8
    K1 = V2 - c(4, Z0); K2 = V4 - c(8, Z1)
    Z1 = c(4, Z0) + K1; Z2 = c(8, Z1) + K2                                     # serial coarsest solve
    W2, W4 = Z1, Z2                                                            # correct level 1
    W1 = b(2, W0) + G1; W3 = b(6, W2) + G3                                     # final F on level 1
    u2, u4, u6, u8 = W1, W2, W3, W4                                            # correct level 0
    u1 = a(1, u0); u3 = a(3, u2); u5 = a(5, u4); u7 = a(7, u6)                 # final F on level 0
    h, res = O.mgrit_forward(*P, x, h0, cf=2, levels=3, iters=1, relax_fine=O.RELAX_F, relax_coarse=O.RELAX_F)
    assert np.max(np.abs(h - np.stack([u1, u2, u3, u4, u5, u6, u7, u8]))) < 1e-15
    assert abs(res[0] - np.sqrt(sum(np.sum(q * q) for q in r))) < 1e-14


@pytest.mark.parametrize("cf,T", [(2, 12), (3, 27), (4, 48)])
@pytest.mark.parametrize("relax0,relax1", [(O.RELAX_F, O.RELAX_F), (O.RELAX_F, O.RELAX_FCF), (O.RELAX_FCF, O.RELAX_FCF)])
def test_adjoint_three_levels_written_out(cf, T, relax0, relax1):
    # The adjoint recurrence is linear: its level-l step is a matrix, built here densely from the transposed
    # Jacobian of the level's own forward step (time step c_f^l, input and state of fine step c_f^l j).  The
    # cycle written out above is run with those matrices on the reversed index.
    H = 5
    w = tiny_workload(T=T, B=1, I=3, H=H)
    P, x, h0, _ = f64_inputs(w)
    rng = np.random.default_rng(11)
    h0 = rng.standard_normal(h0.shape) * 0.4
    W_hh, b_hh = P[1], P[3]
    gi = x @ P[0].T + P[2]
    h = O.serial_forward(*P, x, h0)
    hfull = np.concatenate([h0[None], h], 0)
    seed = rng.standard_normal(h.shape)                   # direct loss derivative at every t (stacked-layer case)

    def jac_T(t_arrive, stride):
        # transposed Jacobian of the forward step that arrives at fine point t_arrive with time step `stride`,
        # leaving from fine point t_arrive - stride
        a, c_r, c_z, c_n, _ = O.adjoint_coefficients(W_hh, b_hh, gi[t_arrive - 1], hfull[t_arrive - stride], float(stride),
                                                     O.CELL_IMPLICIT)
        M = np.diag(a[0])
        for gate, cg in enumerate((c_r, c_z, c_n)):
            M = M + W_hh[gate * H:(gate + 1) * H].T @ np.diag(cg[0])
        return M

    # reversed point s of level l sits at fine time T - c_f^l s; the step arriving there undoes the forward step
    # that arrives at fine time T - c_f^l (s - 1)
    mat = lambda stride: (lambda s, prev: prev @ jac_T(T - stride * (s - 1), stride).T)
    u = np.zeros((T + 1, 1, H))
    u[0] = seed[T - 1]
    g0 = np.zeros_like(u)
    for s in range(1, T):
        g0[s] = seed[T - s - 1]
    want_res = []
    for it in range(2):
        u, rn = _three_level_cycle(cf, T, mat(1), mat(cf), mat(cf * cf), u, g0, relax0, relax1)
        want_res.append(rn)
        lam, lam0, _, res = O.mgrit_adjoint(*P, x, h0, h, seed, cf=cf, levels=3, iters=it + 1, relax_fine=relax0,
                                            relax_coarse=relax1)
        assert np.max(np.abs(lam - u[0:T][::-1])) < 1e-13
        assert np.max(np.abs(lam0 - u[T])) < 1e-13
        assert np.max(np.abs(np.array(res) - np.array(want_res))) < 1e-12
        if it == 0:
            lam_s, _, _ = O.serial_backward(*P, x, h0, h, seed)
            assert np.max(np.abs(lam - lam_s)) > 1e-7             # not vacuous
