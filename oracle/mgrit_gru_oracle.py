"""fp64 CPU oracle for the MGRIT solve of the GRU recurrence (forward and adjoint).

THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, NumPy float64
restatement of the method, written from the paper's equations and algorithms in
their own order and notation, so that it can be checked against the paper by eye.
It shares no code with the CUDA path and must never be imported by it; only the
tests, the smoke check and the benchmark's CPU-baseline leg call it.

What pins each function (see tests/test_oracle_*.py):
  * classic cell / serial sweep / BPTT ........ torch.nn.GRU in float64 (Eq. "gru")
  * implicit cell ............................. algebraic identity of Eq. "gru-implicit",
                                                limits z->1 and gamma->0, model-problem decay
  * adjoint step coefficients ................. central finite differences
  * MGRIT cycle (forward and adjoint) ......... fixed point, exactness after T/c_f (F) and
                                                T/(2 c_f) (FCF) two-level cycles, prefix
                                                exactness, monotone residual, hand-unrolled
                                                brute force on T=8, dense two-level error
                                                propagator for the linear adjoint problem,
                                                hierarchy sizes quoted in the paper
  * multilevel recursion (time step c_f^l, input
    row c_f^l j - 1, FAS term of inner levels) .. three-level cycles written out level by level
                                                with each level's own propagator, forward and
                                                adjoint, c_f = 2, 3, 4 (tests/test_oracle_three_level.py)
  * loss head ................................. torch.nn.functional.cross_entropy float64
  * Adam ...................................... torch.optim.Adam float64
  * values after a FEW cycles (2-3) ........... parity unpinned by the paper (an iteration's
                                                intermediate iterates have no closed form);
                                                they are covered only indirectly by the pins
                                                above, which any wrong step of the cycle breaks.

Array conventions (row-major, time-major): x[T,B,I], gi[T,B,3H], h[T,B,H] with h[k] the
paper's h_{k+1}; h_0 is passed separately.  Gate order along 3H is r | z | n.
"""
from __future__ import annotations

import numpy as np

CELL_CLASSIC = 0   # explicit Euler propagator, Eq. "gru-classic"
CELL_IMPLICIT = 1  # Implicit GRU propagator, Eq. "gru-imap"
RELAX_F = 0        # F-relaxation
RELAX_FCF = 1      # F, then C, then F (Eq. "fcf-relax")
RELAX_FCFCF = 2    # ... and C, F once more; in general relax = n means F (CF)^n
CYCLE_V = 0        # Algorithm "MGProp" with one recursive coarse solve per level (remark "Beyond Two-Level")
CYCLE_F = 1        # F-cycle: after the correction of a level, one more V-cycle from that level down


# --------------------------------------------------------------------------- cell
def sigmoid(a):
    return 1.0 / (1.0 + np.exp(-a))


def input_projection(W_ih, b_ih, x):
    """gi_t = W_i x_t + b_i for every t (input half of Eq. "gru"); computed once on the
    fine grid and reused by every level and by the adjoint (Appendix, feature reuse)."""
    return x @ W_ih.T + b_ih


def gates(W_hh, b_hh, gi, h_prev):
    """r, z, n of Eq. "gru" from the pre-computed input part gi and the previous state.
    Also returns gh_n = W_hn h + b_hn, which the adjoint needs."""
    H = h_prev.shape[-1]
    gh = h_prev @ W_hh.T + b_hh
    r = sigmoid(gi[..., 0:H] + gh[..., 0:H])
    z = sigmoid(gi[..., H:2 * H] + gh[..., H:2 * H])
    n = np.tanh(gi[..., 2 * H:3 * H] + r * gh[..., 2 * H:3 * H])
    return r, z, n, gh[..., 2 * H:3 * H]


def phi(W_hh, b_hh, gi, h_prev, gamma, cell):
    """Propagator Phi_gamma(x_t, h_{t-1}).

    classic  (Eq. "gru-classic"): h + gamma * ( -(1-z) h + (1-z) n )
    implicit (Eq. "gru-imap")   : (1 + gamma (1-z))^-1 * ( h + gamma (1-z) n )
    """
    r, z, n, _ = gates(W_hh, b_hh, gi, h_prev)
    q = gamma * (1.0 - z)
    if cell == CELL_CLASSIC:
        return h_prev + q * (n - h_prev)
    if cell == CELL_IMPLICIT:
        return (h_prev + q * n) / (1.0 + q)
    raise ValueError("cell")


def adjoint_coefficients(W_hh, b_hh, gi, h_prev, gamma, cell):
    """Entries of the transposed Jacobian of one Phi_gamma step (discrete adjoint of
    Eq. "gru-imap" / "gru-classic").  With lambda the sensitivity of the step's output:

        lambda_prev = a*lambda + [c_r*lambda | c_z*lambda | c_n*lambda] W_hh
        d(gi)       =            [c_r*lambda | c_z*lambda | c_np*lambda]

    Returns a, c_r, c_z, c_n, c_np  (c_n = c_np * r: the n-gate path seen through gh_n).
    """
    r, z, n, gh_n = gates(W_hh, b_hh, gi, h_prev)
    q = gamma * (1.0 - z)
    if cell == CELL_IMPLICIT:
        D = 1.0 + q
        a = 1.0 / D
        dPhi_dn = q / D
        dPhi_dz = -gamma * (n - h_prev) / (D * D)
    elif cell == CELL_CLASSIC:
        a = 1.0 - q
        dPhi_dn = q
        dPhi_dz = -gamma * (n - h_prev)
    else:
        raise ValueError("cell")
    c_np = dPhi_dn * (1.0 - n * n)
    c_n = c_np * r
    c_r = c_np * gh_n * r * (1.0 - r)
    c_z = dPhi_dz * z * (1.0 - z)
    return a, c_r, c_z, c_n, c_np


# --------------------------------------------------------------------------- serial sweep
def serial_forward(W_ih, W_hh, b_ih, b_hh, x, h0, cell=CELL_IMPLICIT, dt=1.0):
    """h_t = Phi_dt(x_t, h_{t-1}), t = 1..T: the solution of f(h) = 0 (Eq. "fine-res")."""
    T = x.shape[0]
    gi = input_projection(W_ih, b_ih, x)
    h = np.empty((T,) + h0.shape)
    prev = h0
    for t in range(T):
        prev = phi(W_hh, b_hh, gi[t], prev, dt, cell)
        h[t] = prev
    return h


def weight_gradients(W_ih, W_hh, b_ih, b_hh, x, h0, h, lam, cell=CELL_IMPLICIT, dt=1.0, want_dx=True):
    """g_i = w_i d(h_i)/d(Theta) for every fine step (Algorithm "MGRITTraining", gradient
    line): one time-parallel pass with given states h and sensitivities lam (lam[k] = dL/dh_{k+1})."""
    T = x.shape[0]
    gi = input_projection(W_ih, b_ih, x)
    hprev = np.concatenate([h0[None], h[:-1]], axis=0)           # h_{t-1} for t = 1..T
    a, c_r, c_z, c_n, c_np = adjoint_coefficients(W_hh, b_hh, gi, hprev, dt, cell)
    dA_h = np.concatenate([c_r * lam, c_z * lam, c_n * lam], axis=-1)    # [T,B,3H]
    dA_i = np.concatenate([c_r * lam, c_z * lam, c_np * lam], axis=-1)
    G3 = dA_h.shape[-1]
    out = {
        "dW_hh": dA_h.reshape(-1, G3).T @ hprev.reshape(-1, hprev.shape[-1]),
        "dW_ih": dA_i.reshape(-1, G3).T @ x.reshape(-1, x.shape[-1]),
        "db_hh": dA_h.reshape(-1, G3).sum(axis=0),
        "db_ih": dA_i.reshape(-1, G3).sum(axis=0),
    }
    if want_dx:
        out["dx"] = dA_i @ W_ih
    return out


def serial_backward(W_ih, W_hh, b_ih, b_hh, x, h0, h, dh_seed, cell=CELL_IMPLICIT, dt=1.0):
    """Exact back-propagation through time for the serial sweep.

    dh_seed[k] is the direct derivative of the loss with respect to h_{k+1} (zero except the
    last slice for a loss on h_T).  Returns the total sensitivities lam[k] = dL/dh_{k+1},
    lam0 = dL/dh_0 and the parameter / input gradients."""
    T = x.shape[0]
    gi = input_projection(W_ih, b_ih, x)
    lam = np.empty_like(h)
    cur = dh_seed[T - 1].copy()
    for t in range(T, 0, -1):                       # paper index t: step h_{t-1} -> h_t
        lam[t - 1] = cur
        hprev = h[t - 2] if t >= 2 else h0
        a, c_r, c_z, c_n, _ = adjoint_coefficients(W_hh, b_hh, gi[t - 1], hprev, dt, cell)
        back = a * cur + np.concatenate([c_r * cur, c_z * cur, c_n * cur], axis=-1) @ W_hh
        cur = back + (dh_seed[t - 2] if t >= 2 else 0.0)
    lam0 = cur
    grads = weight_gradients(W_ih, W_hh, b_ih, b_hh, x, h0, h, lam, cell, dt)
    return lam, lam0, grads


# --------------------------------------------------------------------------- MGRIT cycle
def level_sizes(T, cf, levels, ragged=False):
    """N_l = T / c_f^l (e.g. 128/32/8 for c_f = 4 and three levels).

    ragged=True admits any T: the C-points of a level are its points 0, c_f, 2 c_f, ...; what follows the last of
    them is a shorter last interval of F-points only, so N_{l+1} = floor(N_l / c_f) (at least one point per level)."""
    if cf < 2 or levels < 1:
        raise ValueError("cf >= 2 and levels >= 1 required")
    if not ragged:
        if T % (cf ** (levels - 1)) != 0:
            raise ValueError("T must be divisible by cf^(levels-1)")
        return [T // cf ** l for l in range(levels)]
    N = [T]
    for _ in range(levels - 1):
        N.append(N[-1] // cf)
    if N[-1] < 1:
        raise ValueError("too many levels for this T")
    return N


def fas_vcycle(step, N, cf, relax, u, g, l=0, resnorm=None, cycle=CYCLE_V):
    """One multigrid cycle on level l (Algorithm "MGProp" with the recursive coarse solve of
    the remark "Beyond Two-Level"), for the level-l system

        u_j = step(l, j, u_{j-1}) + g_j ,  j = 1..N_l ,   u_0 fixed.

    step(l, j, u_prev): j is an integer array of target points, u_prev their predecessors'
    states; all entries are independent (the "ParallelFor" of Algorithm "F-relaxation").
    u[l], g[l]: arrays [N_l+1, ...].  relax[l] = n means F (CF)^n.  Modifies u in place.
    N_l need not be a multiple of c_f: points after the last C-point form a shorter last interval of F-points.
    cycle = CYCLE_F: when the correction has been spread (the cycle below is complete) one more V-cycle is run
    from this level down, as in the F-cycle of multigrid; on the last two levels that is simply two V-cycles.
    """
    Nl = N[l]
    ul, gl = u[l], g[l]
    L = len(N)
    if l == L - 1:
        # coarsest level: serial propagation resolves the level's system exactly
        for j in range(1, Nl + 1):
            ul[j] = step(l, np.array([j]), ul[j - 1:j])[0] + gl[j]
        return
    Nc = N[l + 1]                                 # number of C-points after point 0 (= floor(N_l / c_f))

    def f_relax():
        # from every C-point fill the F-points up to the next C-point, exclusive (or to the end of the level)
        for s in range(1, cf):
            j = np.arange(0, Nl + 1, cf) + s
            j = j[j <= Nl]
            ul[j] = step(l, j, ul[j - 1]) + gl[j]

    def c_relax():
        # one more step from the last F-point of each interval onto the next C-point
        j = cf * np.arange(1, Nc + 1)
        ul[j] = step(l, j, ul[j - 1]) + gl[j]

    # relax the current guess
    f_relax()
    for _ in range(relax[l]):
        c_relax()
        f_relax()

    # residual at the C-points, restricted by injection:  r_c = R(f(h')),  h'_c = R(h')
    jc = cf * np.arange(1, Nc + 1)
    v = step(l, jc, ul[jc - 1]) + gl[jc]
    r_c = ul[jc] - v
    if resnorm is not None and l == 0:
        resnorm.append(float(np.sqrt(np.sum(r_c * r_c))))
    Uc = np.concatenate([ul[0:1], ul[jc]], axis=0)            # U'_0 .. U'_{N_{l+1}}

    # coarse equation f_c(h_c*) = f_c(h'_c) - r_c, i.e.  U_k = step(l+1,k,U_{k-1}) + G_k  with
    # G_k = U'_k - step(l+1,k,U'_{k-1}) - r_k = v_k - step(l+1,k,U'_{k-1})
    k = np.arange(1, Nc + 1)
    G = np.zeros_like(Uc)
    G[k] = v - step(l + 1, k, Uc[k - 1])
    u[l + 1] = Uc.copy()                                       # initial guess = restricted state
    g[l + 1] = G
    fas_vcycle(step, N, cf, relax, u, g, l + 1, resnorm, cycle)

    # h'' = h' + P(h_c* - h'_c): only the C-point values are read afterwards
    ul[jc] = u[l + 1][1:]
    # final F-relaxation spreads the correction over the F-points
    f_relax()
    if cycle == CYCLE_F:
        # F-cycle: one V-cycle from this level down on the corrected state (its level-0 residual is not recorded again)
        fas_vcycle(step, N, cf, relax, u, g, l, None, CYCLE_V)


def _relax_list(levels, relax_fine, relax_coarse):
    return [relax_fine] + [relax_coarse] * (levels - 1)


def mgrit_forward(W_ih, W_hh, b_ih, b_hh, x, h0, cf, levels, iters, cell=CELL_IMPLICIT,
                  relax_fine=RELAX_F, relax_coarse=RELAX_FCF, dt=1.0, h_init=None, cycle=CYCLE_V, ragged=False):
    """Forward propagation by `iters` MGRIT cycles from the zero initial guess
    (Algorithm "MGRITTraining", forward block).  Level l uses the same cell with time step
    gamma = c_f^l * dt and, for its point j, the input of fine step c_f^l * j.

    Returns h[T,B,H] and the list of level-0 C-point residual 2-norms, one per cycle, each
    measured after that cycle's pre-relaxation."""
    T = x.shape[0]
    N = level_sizes(T, cf, levels, ragged)
    gi = input_projection(W_ih, b_ih, x)

    def step(l, j, u_prev):
        m = cf ** l
        return phi(W_hh, b_hh, gi[m * j - 1], u_prev, m * dt, cell)

    u = [None] * levels
    g = [None] * levels
    u[0] = np.zeros((T + 1,) + h0.shape)
    u[0][0] = h0
    if h_init is not None:
        u[0][1:] = h_init
    g[0] = np.zeros_like(u[0])
    relax = _relax_list(levels, relax_fine, relax_coarse)
    resnorm = []
    if levels == 1:
        fas_vcycle(step, N, cf, relax, u, g, 0, None)
        return u[0][1:].copy(), resnorm
    for _ in range(iters):
        fas_vcycle(step, N, cf, relax, u, g, 0, resnorm, cycle)
    return u[0][1:].copy(), resnorm


def mgrit_adjoint(W_ih, W_hh, b_ih, b_hh, x, h0, h, dh_seed, cf, levels, iters, cell=CELL_IMPLICIT,
                  relax_fine=RELAX_F, relax_coarse=RELAX_FCF, dt=1.0, want_dx=True, cycle=CYCLE_V, ragged=False):
    """Backward propagation by MGRIT on the adjoint recurrence, time reversed
    (Algorithm "MGRITTraining", backward block; Appendix "Training With MGRIT").

    Reversed index: the level-l unknown mu_s approximates lambda at fine time T - c_f^l s.
    mu_0 = lambda_T is fixed; the step arriving at s applies the transposed Jacobian of the
    level-l forward step (gamma = c_f^l dt) that ARRIVES at fine time T - c_f^l (s-1), i.e. with
    that time's input and linearised at the GIVEN state c_f^l fine steps earlier (restriction by
    injection).  For T divisible by c_f^(levels-1) this is forward step j = N_l - s + 1 of the
    level; otherwise the reversed coarse grids are anchored at T, not at 0.  The fine-level
    source is the direct loss derivative dh_seed at that time.  Zero initial guess.

    Returns lam[T,B,H] (lam[k] = dL/dh_{k+1}), lam0, gradients (one time-parallel pass with
    the final lam and h) and the residual norms."""
    T = x.shape[0]
    N = level_sizes(T, cf, levels, ragged)
    gi = input_projection(W_ih, b_ih, x)
    hfull = np.concatenate([h0[None], h], axis=0)                 # h_0 .. h_T

    def step(l, s, mu_prev):
        m = cf ** l
        t_arrive = T - m * (s - 1)                                # fine time the transposed forward step arrives at
        a, c_r, c_z, c_n, _ = adjoint_coefficients(W_hh, b_hh, gi[t_arrive - 1], hfull[t_arrive - m],
                                                   m * dt, cell)
        return a * mu_prev + np.concatenate([c_r * mu_prev, c_z * mu_prev, c_n * mu_prev], axis=-1) @ W_hh

    u = [None] * levels
    g = [None] * levels
    u[0] = np.zeros((T + 1,) + h0.shape)
    u[0][0] = dh_seed[T - 1]
    g[0] = np.zeros_like(u[0])
    for s in range(1, T):
        g[0][s] = dh_seed[T - s - 1]                               # seed at forward point T-s
    relax = _relax_list(levels, relax_fine, relax_coarse)
    resnorm = []
    if levels == 1:
        fas_vcycle(step, N, cf, relax, u, g, 0, None)
    else:
        for _ in range(iters):
            fas_vcycle(step, N, cf, relax, u, g, 0, resnorm, cycle)
    lam = np.ascontiguousarray(u[0][0:T][::-1])                    # lam[k] = mu_{T-1-k}
    lam0 = u[0][T].copy()
    grads = weight_gradients(W_ih, W_hh, b_ih, b_hh, x, h0, h, lam, cell, dt, want_dx)
    return lam, lam0, grads, resnorm


# --------------------------------------------------------------------------- head / update
def xent_head(hT, W_c, b_c, labels):
    """Linear classifier on h_T with mean softmax cross-entropy; returns the loss and
    w_T = grad_{h_T} L (the seed of the backward block) plus the head's own gradients."""
    B = hT.shape[0]
    logits = hT @ W_c.T + b_c
    m = logits.max(axis=1, keepdims=True)
    e = np.exp(logits - m)
    p = e / e.sum(axis=1, keepdims=True)
    logp = (logits - m) - np.log(e.sum(axis=1, keepdims=True))
    loss = -np.mean(logp[np.arange(B), labels])
    dlogits = p.copy()
    dlogits[np.arange(B), labels] -= 1.0
    dlogits /= B
    return loss, dlogits @ W_c, dlogits.T @ hT, dlogits.sum(axis=0)


def sgd_update(p, g, lr):
    """Theta <- Theta - l_r g (last line of Algorithm "MGRITTraining")."""
    return p - lr * g


def adam_update(p, g, m, v, lr, step, beta1=0.9, beta2=0.999, eps=1e-8):
    """Adam step with bias correction (the optimiser of the paper's experiments); returns new (p, m, v)."""
    m = beta1 * m + (1.0 - beta1) * g
    v = beta2 * v + (1.0 - beta2) * g * g
    mhat = m / (1.0 - beta1 ** step)
    vhat = v / (1.0 - beta2 ** step)
    return p - lr * mhat / (np.sqrt(vhat) + eps), m, v


# --------------------------------------------------------------------------- stacked layers in one state
# A multi-layer GRU advanced one TIME step at a time: the state of a time point is the stack of all layers' hidden
# states, and layer k's input at a step is layer k-1's NEW state of the same step (layer 0 reads x).  MGRIT then
# runs ONE cycle for the whole stack (the paper's experiments use two layers); on level l every layer uses the same
# cell with time step c_f^l and layer 0 the input of fine step c_f^l j.
# layers: list of (W_ih, W_hh, b_ih, b_hh); states are arrays [..., n_layers, B, H].

def stacked_phi(layers, gi0, u_prev, gamma, cell):
    """One step of the stack.  gi0 = W_i x + b_i of layer 0 for this step; u_prev[..., k, :, :] the layers' states."""
    out = []
    gik = gi0
    for k, (W_ih, W_hh, b_ih, b_hh) in enumerate(layers):
        if k > 0:
            gik = out[-1] @ W_ih.T + b_ih          # input projection of the layer below's new state
        out.append(phi(W_hh, b_hh, gik, u_prev[..., k, :, :], gamma, cell))
    return np.stack(out, axis=-3)


def stacked_serial_forward(layers, x, h0, cell=CELL_IMPLICIT, dt=1.0):
    """h0: [n_layers, B, H] -> h[T, n_layers, B, H]; with the classic cell and dt = 1 this is the usual stacked GRU."""
    T = x.shape[0]
    gi0 = input_projection(layers[0][0], layers[0][2], x)
    h = np.empty((T,) + h0.shape)
    prev = h0
    for t in range(T):
        prev = stacked_phi(layers, gi0[t], prev, dt, cell)
        h[t] = prev
    return h


def stacked_mgrit_forward(layers, x, h0, cf, levels, iters, cell=CELL_IMPLICIT, relax_fine=RELAX_F, relax_coarse=RELAX_FCF,
                          dt=1.0, cycle=CYCLE_V, ragged=False, h_init=None):
    """`iters` MGRIT cycles on the stacked state from the zero initial guess; returns h[T, n_layers, B, H] and the
    level-0 C-point residual norms (over all layers)."""
    T = x.shape[0]
    N = level_sizes(T, cf, levels, ragged)
    gi0 = input_projection(layers[0][0], layers[0][2], x)

    def step(l, j, u_prev):
        m = cf ** l
        return stacked_phi(layers, gi0[m * j - 1], u_prev, m * dt, cell)

    u = [None] * levels
    g = [None] * levels
    u[0] = np.zeros((T + 1,) + h0.shape)
    u[0][0] = h0
    if h_init is not None:
        u[0][1:] = h_init
    g[0] = np.zeros_like(u[0])
    relax = _relax_list(levels, relax_fine, relax_coarse)
    resnorm = []
    if levels == 1:
        fas_vcycle(step, N, cf, relax, u, g, 0, None)
    else:
        for _ in range(iters):
            fas_vcycle(step, N, cf, relax, u, g, 0, resnorm, cycle)
    return u[0][1:].copy(), resnorm


def stacked_adjoint_step(layers, coefs, lam_out):
    """Transposed Jacobian of one step of the stack applied to lam_out[..., k, :, :] (sensitivities of the step's
    outputs).  coefs[k] = (a, c_r, c_z, c_n, c_np) of layer k at the step's linearisation point.  Works from the top
    layer down: what layer k+1 sends to its input joins layer k's own output sensitivity.
    Returns (sensitivities of the step's input states, the per-layer TOTAL output sensitivities used on the way --
    the ones the parameter gradients of that step need)."""
    nl = len(layers)
    lam_in = [None] * nl
    lam_tot = [None] * nl
    from_above = 0.0
    for k in range(nl - 1, -1, -1):
        W_ih, W_hh, _, _ = layers[k]
        a, c_r, c_z, c_n, c_np = coefs[k]
        lt = lam_out[..., k, :, :] + from_above
        lam_tot[k] = lt
        lam_in[k] = a * lt + np.concatenate([c_r * lt, c_z * lt, c_n * lt], axis=-1) @ W_hh
        from_above = np.concatenate([c_r * lt, c_z * lt, c_np * lt], axis=-1) @ W_ih if k > 0 else 0.0
    return np.stack(lam_in, axis=-3), np.stack(lam_tot, axis=-3)


def _stacked_inputs(layers, x, h):
    """Layer k's input sequence given the states h[T, nl, B, H]: x for layer 0, the layer below's states otherwise."""
    return [x if k == 0 else h[:, k - 1] for k in range(len(layers))]


def stacked_serial_backward(layers, x, h0, h, dh_seed, cell=CELL_IMPLICIT, dt=1.0):
    """Exact back-propagation through time of the stacked sweep.  dh_seed[T, nl, B, H]: direct loss derivatives.
    Returns lam[T, nl, B, H] (sensitivity of every state as a step OUTPUT, before the within-step coupling),
    lam0[nl, B, H] and per-layer gradient dicts."""
    T = x.shape[0]
    nl = len(layers)
    hfull = np.concatenate([h0[None], h], axis=0)
    inps = _stacked_inputs(layers, x, h)
    gis = [input_projection(layers[k][0], layers[k][2], inps[k]) for k in range(nl)]
    lam = np.empty_like(h)
    lam_tot = np.empty_like(h)
    cur = dh_seed[T - 1].copy()
    for t in range(T, 0, -1):
        lam[t - 1] = cur
        coefs = [adjoint_coefficients(layers[k][1], layers[k][3], gis[k][t - 1], hfull[t - 1, k], dt, cell) for k in range(nl)]
        back, tot = stacked_adjoint_step(layers, coefs, cur)
        lam_tot[t - 1] = tot
        cur = back + (dh_seed[t - 2] if t >= 2 else 0.0)
    grads = [weight_gradients(*layers[k], inps[k], h0[k], h[:, k], lam_tot[:, k], cell, dt, want_dx=(k == 0)) for k in range(nl)]
    return lam, cur, grads


def stacked_mgrit_adjoint(layers, x, h0, h, dh_seed, cf, levels, iters, cell=CELL_IMPLICIT, relax_fine=RELAX_F,
                          relax_coarse=RELAX_FCF, dt=1.0, cycle=CYCLE_V, ragged=False):
    """MGRIT on the adjoint of the stacked recurrence, time reversed, linearised at the GIVEN states h[T, nl, B, H].
    The level-l step arriving at reversed point s transposes the level's forward step (time step c_f^l) that arrives
    at fine time t = T - c_f^l (s-1): every layer is linearised at its given state c_f^l fine steps earlier, with the
    input that the given states provide at time t (x_t for layer 0, the layer below's given state at t otherwise:
    restriction by injection for the inputs as for the states).  Gradients: one time-parallel pass with the final
    sensitivities, top layer first (its input gradient joins the layer below's sensitivity)."""
    T = x.shape[0]
    nl = len(layers)
    N = level_sizes(T, cf, levels, ragged)
    hfull = np.concatenate([h0[None], h], axis=0)
    inps = _stacked_inputs(layers, x, h)
    gis = [input_projection(layers[k][0], layers[k][2], inps[k]) for k in range(nl)]

    def coefs_at(t_arrive, m):
        return [adjoint_coefficients(layers[k][1], layers[k][3], gis[k][t_arrive - 1], hfull[t_arrive - m][..., k, :, :], m * dt, cell)
                for k in range(nl)]

    def step(l, s, mu_prev):
        m = cf ** l
        out = np.empty_like(mu_prev)
        for q, sq in enumerate(np.atleast_1d(s)):
            out[q], _ = stacked_adjoint_step(layers, coefs_at(T - m * (int(sq) - 1), m), mu_prev[q])
        return out

    u = [None] * levels
    g = [None] * levels
    u[0] = np.zeros((T + 1,) + h0.shape)
    u[0][0] = dh_seed[T - 1]
    g[0] = np.zeros_like(u[0])
    for s in range(1, T):
        g[0][s] = dh_seed[T - s - 1]
    relax = _relax_list(levels, relax_fine, relax_coarse)
    resnorm = []
    if levels == 1:
        fas_vcycle(step, N, cf, relax, u, g, 0, None)
    else:
        for _ in range(iters):
            fas_vcycle(step, N, cf, relax, u, g, 0, resnorm, cycle)
    lam = np.ascontiguousarray(u[0][0:T][::-1])
    lam0 = u[0][T].copy()
    # total output sensitivities of every fine step (the within-step coupling added), then the gradient pass
    lam_tot = np.empty_like(lam)
    for t in range(1, T + 1):
        _, lam_tot[t - 1] = stacked_adjoint_step(layers, coefs_at(t, 1), lam[t - 1])
    grads = [weight_gradients(*layers[k], inps[k], h0[k], h[:, k], lam_tot[:, k], cell, dt, want_dx=(k == 0)) for k in range(nl)]
    return lam, lam0, grads, resnorm


# --------------------------------------------------------------------------- Implicit LSTM
# The paper's conclusion names the LSTM as a cell the same treatment applies to.  Reading taken here: the LSTM cell
# state obeys  c_t = f c_{t-1} + i g = c_{t-1} + [ -(1-f) c_{t-1} + i g ], a unit-step forward-Euler update of
# c' = -(1-f) c + i g, exactly as Eq. "gru-classic" reads the GRU; the stiff decay term -(1-f) c is taken implicitly
# as in Eq. "gru-implicit":  (1 + gamma (1-f)) c_t = c_{t-1} + gamma i g.  The hidden state h_t = o tanh(c_t) has no
# dynamics of its own and is re-evaluated from the new cell state.  gamma = 1 explicit is the textbook LSTM.
# Gate order along 4H is i | f | g | o (the usual library order); the state of a time point is (c, h), stored as
# [..., 2, B, H] with part 0 = c and part 1 = h.

def lstm_gates(W_hh, b_hh, gi, h_prev):
    H = h_prev.shape[-1]
    pre = gi + h_prev @ W_hh.T + b_hh
    return sigmoid(pre[..., 0:H]), sigmoid(pre[..., H:2 * H]), np.tanh(pre[..., 2 * H:3 * H]), sigmoid(pre[..., 3 * H:4 * H])


def lstm_phi(W_hh, b_hh, gi, u_prev, gamma, cell):
    """One LSTM step on the state u_prev[..., 0] = c, u_prev[..., 1] = h with the pre-computed input part gi."""
    c_prev, h_prev = u_prev[..., 0, :, :], u_prev[..., 1, :, :]
    i, f, g, o = lstm_gates(W_hh, b_hh, gi, h_prev)
    q = gamma * (1.0 - f)
    if cell == CELL_CLASSIC:
        c = c_prev - q * c_prev + gamma * i * g
    elif cell == CELL_IMPLICIT:
        c = (c_prev + gamma * i * g) / (1.0 + q)
    else:
        raise ValueError("cell")
    return np.stack([c, o * np.tanh(c)], axis=-3)


def lstm_adjoint_coefficients(W_hh, b_hh, gi, u_prev, gamma, cell):
    """Entries of the transposed Jacobian of one LSTM step.  With (L_c, L_h) the sensitivities of the step's outputs:

        dc      = L_c + p * L_h                       total sensitivity of the new cell state
        dA      = [ c_i*dc | c_f*dc | c_g*dc | c_o*L_h ]      = d(pre-activations) = d(gi)
        L_c_in  = a * dc ,   L_h_in = dA W_hh

    Returns a, p, c_i, c_f, c_g, c_o."""
    c_prev, h_prev = u_prev[..., 0, :, :], u_prev[..., 1, :, :]
    i, f, g, o = lstm_gates(W_hh, b_hh, gi, h_prev)
    q = gamma * (1.0 - f)
    if cell == CELL_IMPLICIT:
        D = 1.0 + q
        c = (c_prev + gamma * i * g) / D
        a, dci, dcg, dcf = 1.0 / D, gamma * g / D, gamma * i / D, gamma * c / D
    elif cell == CELL_CLASSIC:
        c = c_prev - q * c_prev + gamma * i * g
        a, dci, dcg, dcf = 1.0 - q, gamma * g, gamma * i, gamma * c_prev
    else:
        raise ValueError("cell")
    th = np.tanh(c)
    return a, o * (1.0 - th * th), dci * i * (1.0 - i), dcf * f * (1.0 - f), dcg * (1.0 - g * g), th * o * (1.0 - o)


def lstm_adjoint_step(W_hh, coefs, lam_out):
    """Applies the transposed Jacobian: lam_out[..., 0] = L_c, lam_out[..., 1] = L_h -> (input sensitivities, dA)."""
    a, p, c_i, c_f, c_g, c_o = coefs
    Lc, Lh = lam_out[..., 0, :, :], lam_out[..., 1, :, :]
    dc = Lc + p * Lh
    dA = np.concatenate([c_i * dc, c_f * dc, c_g * dc, c_o * Lh], axis=-1)
    return np.stack([a * dc, dA @ W_hh], axis=-3), dA


def lstm_serial_forward(W_ih, W_hh, b_ih, b_hh, x, u0, cell=CELL_IMPLICIT, dt=1.0):
    """u0[2, B, H] = (c_0, h_0) -> u[T, 2, B, H]."""
    T = x.shape[0]
    gi = input_projection(W_ih, b_ih, x)
    u = np.empty((T,) + u0.shape)
    prev = u0
    for t in range(T):
        prev = lstm_phi(W_hh, b_hh, gi[t], prev, dt, cell)
        u[t] = prev
    return u


def lstm_weight_gradients(W_ih, W_hh, b_ih, b_hh, x, u0, u, lam, cell=CELL_IMPLICIT, dt=1.0, want_dx=True):
    """Time-parallel gradient pass: dA_t from the step-output sensitivities lam[T, 2, B, H] and the given states."""
    gi = input_projection(W_ih, b_ih, x)
    uprev = np.concatenate([u0[None], u[:-1]], axis=0)
    coefs = lstm_adjoint_coefficients(W_hh, b_hh, gi, uprev, dt, cell)
    _, dA = lstm_adjoint_step(W_hh, coefs, lam)
    G4 = dA.shape[-1]
    hprev = uprev[:, 1]
    out = {"dW_hh": dA.reshape(-1, G4).T @ hprev.reshape(-1, hprev.shape[-1]), "dW_ih": dA.reshape(-1, G4).T @ x.reshape(-1, x.shape[-1]),
           "db_hh": dA.reshape(-1, G4).sum(axis=0), "db_ih": dA.reshape(-1, G4).sum(axis=0)}
    if want_dx:
        out["dx"] = dA @ W_ih
    return out


def lstm_serial_backward(W_ih, W_hh, b_ih, b_hh, x, u0, u, du_seed, cell=CELL_IMPLICIT, dt=1.0):
    """Exact BPTT.  du_seed[T, 2, B, H]: direct loss derivatives w.r.t. (c_t, h_t).  Returns lam, lam0, gradients."""
    T = x.shape[0]
    gi = input_projection(W_ih, b_ih, x)
    ufull = np.concatenate([u0[None], u], axis=0)
    lam = np.empty_like(u)
    cur = du_seed[T - 1].copy()
    for t in range(T, 0, -1):
        lam[t - 1] = cur
        back, _ = lstm_adjoint_step(W_hh, lstm_adjoint_coefficients(W_hh, b_hh, gi[t - 1], ufull[t - 1], dt, cell), cur)
        cur = back + (du_seed[t - 2] if t >= 2 else 0.0)
    return lam, cur, lstm_weight_gradients(W_ih, W_hh, b_ih, b_hh, x, u0, u, lam, cell, dt)


def lstm_mgrit_forward(W_ih, W_hh, b_ih, b_hh, x, u0, cf, levels, iters, cell=CELL_IMPLICIT, relax_fine=RELAX_F,
                       relax_coarse=RELAX_FCF, dt=1.0, cycle=CYCLE_V, ragged=False, u_init=None):
    """MGRIT on the LSTM recurrence of the state (c, h); level l uses time step c_f^l and the input of fine step c_f^l j."""
    T = x.shape[0]
    N = level_sizes(T, cf, levels, ragged)
    gi = input_projection(W_ih, b_ih, x)

    def step(l, j, u_prev):
        m = cf ** l
        return lstm_phi(W_hh, b_hh, gi[m * j - 1], u_prev, m * dt, cell)

    u = [None] * levels
    g = [None] * levels
    u[0] = np.zeros((T + 1,) + u0.shape)
    u[0][0] = u0
    if u_init is not None:
        u[0][1:] = u_init
    g[0] = np.zeros_like(u[0])
    relax = _relax_list(levels, relax_fine, relax_coarse)
    resnorm = []
    if levels == 1:
        fas_vcycle(step, N, cf, relax, u, g, 0, None)
    else:
        for _ in range(iters):
            fas_vcycle(step, N, cf, relax, u, g, 0, resnorm, cycle)
    return u[0][1:].copy(), resnorm


def lstm_mgrit_adjoint(W_ih, W_hh, b_ih, b_hh, x, u0, u, du_seed, cf, levels, iters, cell=CELL_IMPLICIT, relax_fine=RELAX_F,
                       relax_coarse=RELAX_FCF, dt=1.0, cycle=CYCLE_V, ragged=False, want_dx=True):
    """MGRIT on the adjoint LSTM recurrence, time reversed, linearised at the GIVEN states (as mgrit_adjoint)."""
    T = x.shape[0]
    N = level_sizes(T, cf, levels, ragged)
    gi = input_projection(W_ih, b_ih, x)
    ufull = np.concatenate([u0[None], u], axis=0)

    def step(l, s, mu_prev):
        m = cf ** l
        t_arrive = T - m * (s - 1)
        back, _ = lstm_adjoint_step(W_hh, lstm_adjoint_coefficients(W_hh, b_hh, gi[t_arrive - 1], ufull[t_arrive - m], m * dt, cell), mu_prev)
        return back

    v = [None] * levels
    g = [None] * levels
    v[0] = np.zeros((T + 1,) + u0.shape)
    v[0][0] = du_seed[T - 1]
    g[0] = np.zeros_like(v[0])
    for s in range(1, T):
        g[0][s] = du_seed[T - s - 1]
    relax = _relax_list(levels, relax_fine, relax_coarse)
    resnorm = []
    if levels == 1:
        fas_vcycle(step, N, cf, relax, v, g, 0, None)
    else:
        for _ in range(iters):
            fas_vcycle(step, N, cf, relax, v, g, 0, resnorm, cycle)
    lam = np.ascontiguousarray(v[0][0:T][::-1])
    lam0 = v[0][T].copy()
    return lam, lam0, lstm_weight_gradients(W_ih, W_hh, b_ih, b_hh, x, u0, u, lam, cell, dt, want_dx), resnorm
