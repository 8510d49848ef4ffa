"""GPU parity, bf16 tensor-core operand mode (tcgen05 GEMMs, fp32 accumulation, fp32 state), against the
fp64 oracle at the same cycle count.  Tolerance: 2e-2 norm-relative (||a-b||_inf / ||b||_inf) on h, on
every gradient and on dh; residual norms within 1e-3 of their own size plus 1e-3 of the first cycle's residual.
(A late residual is a difference of nearly equal bf16-perturbed states, so its error has a floor that scales with the
state error, i.e. with the first residual r_0.  Measured over these workloads at up to five cycles: the mismatch is
at most 7e-4 of the residual while the residual is above 1e-2 r_0, and never above 3.1e-4 r_0; the fastest-converging
variant case, F-cycles with FCFCF relaxation, reaches its floor in the second cycle with a mismatch of 6.6e-4 r_0.)

Small shapes are compared element by element over everything.  The full-size configurations are compared
on sampled batch rows (rows of a batch never interact in the forward or adjoint recurrences, so the oracle
can compute a few rows exactly as the full problem would) in the launch configuration the benchmark times; their
weight gradients, sums over all T*B rows, are compared in full with the oracle's time-parallel gradient pass in
fp64 fed the GPU's states and sensitivities.
"""
import numpy as np
import pytest
import torch

from oracle import mgrit_gru_oracle as O
from paper_2203_04738_b200.synthetic import WORKLOADS, Workload, make_inputs
from tests.gpu_util import NAMES, max_abs, oracle_params, rel_inf, to_dev, upload

pytestmark = pytest.mark.gpu
TOL = 2e-2


@pytest.fixture(scope="module")
def B():
    from paper_2203_04738_b200 import binding
    return binding


def _cfg(B, w, iters, T=None, Bsz=None, flags=0):
    return B.make_cfg(T or w.T, Bsz or w.B, w.I, w.H, cf=w.cf, levels=w.levels, iters=iters, cell=w.cell,
                      relax_fine=w.relax_fine, relax_coarse=w.relax_coarse, operands=B.OPERANDS_BF16, flags=flags)


def _full_case(B, w, check_grads=True):
    d = make_inputs(w)
    p, x, h0 = upload(d)
    P = oracle_params(d)
    xr, h0r = d["x"].astype(np.float64), d["h0"].astype(np.float64)
    kw = dict(cf=w.cf, levels=w.levels, relax_fine=w.relax_fine, relax_coarse=w.relax_coarse)
    cfg = _cfg(B, w, w.iters_fwd)
    h, gi, rn = B.mgrit_gru_forward(cfg, p, x, h0, want_resnorm=True)
    href, rref = O.mgrit_forward(*P, xr, h0r, iters=w.iters_fwd, **kw)
    assert rel_inf(gi.cpu().numpy(), O.input_projection(P[0], P[2], xr)) < TOL
    assert rel_inf(h.cpu().numpy(), href) < TOL
    for a, b in zip(rn, rref):
        assert abs(a - b) <= 1e-3 * b + 1e-3 * rref[0]   # floor: bf16 noise of the states, a fraction of the first residual
    hs, _ = B.gru_serial_forward(cfg, p, x, h0)
    assert rel_inf(hs.cpu().numpy(), O.serial_forward(*P, xr, h0r)) < TOL
    if not check_grads:
        return
    loss, dhT, dWc, dbc = B.xent_head_fwd_bwd(h[-1].contiguous(), to_dev(d["W_c"]), to_dev(d["b_c"]), to_dev(d["labels"]))
    hn = h.cpu().numpy().astype(np.float64)
    rng = np.random.default_rng(3)
    seed = (rng.standard_normal(hn.shape) * 1e-3).astype(np.float32)
    seed64 = seed.astype(np.float64)
    seed64[-1] += dhT.cpu().numpy()
    cfga = _cfg(B, w, w.iters_adj)
    r = B.mgrit_gru_adjoint(cfga, p, x, h0, gi, h, dh_seed=to_dev(seed), dhT=dhT, want_resnorm=True)
    gi64 = None
    lam, lam0, g, rref = O.mgrit_adjoint(*P, xr, h0r, hn, seed64, iters=w.iters_adj, **kw)
    for a, b in zip(r.resnorm, rref):
        assert abs(a - b) <= 1e-3 * b + 1e-3 * rref[0]   # floor: bf16 noise of the states, a fraction of the first residual
    assert rel_inf(r.dh.cpu().numpy(), lam) < TOL
    assert max_abs(r.dh0.cpu().numpy(), lam0) / np.max(np.abs(lam)) < TOL
    for k in ("dx", "dW_ih", "dW_hh", "db_ih", "db_hh"):
        assert rel_inf(getattr(r, k).cpu().numpy(), g[k]) < TOL, k
    # exact BPTT of the serial sweep
    rs = B.gru_serial_backward(cfga, p, x, h0, gi, h, dh_seed=to_dev(seed), dhT=dhT)
    lam_s, lam0_s, g_s = O.serial_backward(*P, xr, h0r, hn, seed64)
    assert rel_inf(rs.dh.cpu().numpy(), lam_s) < TOL
    for k in ("dx", "dW_ih", "dW_hh", "db_ih", "db_hh"):
        assert rel_inf(getattr(rs, k).cpu().numpy(), g_s[k]) < TOL, k


def test_small_two_level(B):
    _full_case(B, Workload("s2", T=64, B=8, I=128, H=128, cf=4, levels=2, iters_fwd=2, iters_adj=2, relax_fine=0, relax_coarse=1,
                           operands=2, classes=8, relu=True, seed=7))


def test_small_ragged_three_level_fcf(B):
    # rows per step 48*24 = 1152 (nine 128-row tiles, batch rows straddling tiles), H = 192 (three unit tiles,
    # one partial 256-column tile in the adjoint GEMM), I = 80 (K tail of 16 in the projection)
    _full_case(B, Workload("s3", T=96, B=24, I=80, H=192, cf=2, levels=3, iters_fwd=2, iters_adj=3, relax_fine=1, relax_coarse=1,
                           operands=2, classes=8, relu=True, seed=8))


def test_small_single_level_and_tiny_batch(B):
    _full_case(B, Workload("s1", T=24, B=8, I=16, H=64, cf=2, levels=4, iters_fwd=3, iters_adj=1, relax_fine=0, relax_coarse=0,
                           operands=2, classes=8, relu=False, seed=9))


def test_small_four_level_one_point_coarsest(B):
    # level sizes 64/16/4/1: the persistent chain of the coarsest level has a single step
    _full_case(B, Workload("s4", T=64, B=8, I=64, H=128, cf=4, levels=4, iters_fwd=2, iters_adj=2, relax_fine=0, relax_coarse=1,
                           operands=2, classes=8, relu=True, seed=10))


def test_whole_chain_against_the_oracles_own_forward(B):
    # Forward, loss head, adjoint and gradients on the GPU against the same chain run by the oracle alone: the
    # oracle's adjoint is linearised at the ORACLE's forward states, so nothing of the GPU's output enters the reference.
    w = Workload("chain", T=96, B=16, I=64, H=128, cf=4, levels=3, iters_fwd=2, iters_adj=2, relax_fine=0, relax_coarse=1,
                 operands=2, classes=8, relu=True, seed=12)
    d = make_inputs(w, T=96)
    p, x, h0 = upload(d)
    P = oracle_params(d)
    xr, h0r = d["x"].astype(np.float64), d["h0"].astype(np.float64)
    kw = dict(cf=4, levels=2, relax_fine=0, relax_coarse=1)       # 96 = 4 * 24: two levels
    cfg = B.make_cfg(96, w.B, w.I, w.H, cf=4, levels=2, iters=2, operands=B.OPERANDS_BF16)
    h, gi, _ = B.mgrit_gru_forward(cfg, p, x, h0)
    loss, dhT, dWc, dbc = B.xent_head_fwd_bwd(h[-1].contiguous(), to_dev(d["W_c"]), to_dev(d["b_c"]), to_dev(d["labels"]))
    r = B.mgrit_gru_adjoint(cfg, p, x, h0, gi, h, dhT=dhT)
    href, _ = O.mgrit_forward(*P, xr, h0r, iters=2, **kw)
    loss_r, dhT_r, dWc_r, dbc_r = O.xent_head(href[-1], d["W_c"].astype(np.float64), d["b_c"].astype(np.float64), d["labels"])
    seed = np.zeros_like(href)
    seed[-1] = dhT_r
    lam, lam0, g, _ = O.mgrit_adjoint(*P, xr, h0r, href, seed, iters=2, **kw)
    assert abs(loss.item() - loss_r) < TOL * abs(loss_r)
    assert rel_inf(dWc.cpu().numpy(), dWc_r) < TOL and rel_inf(dbc.cpu().numpy(), dbc_r) < TOL
    assert rel_inf(r.dh.cpu().numpy(), lam) < TOL
    for k in ("dx", "dW_ih", "dW_hh", "db_ih", "db_hh"):
        assert rel_inf(getattr(r, k).cpu().numpy(), g[k]) < TOL, k


def test_medium_full(B):
    # third configuration, everything compared: I=1024 H=512 B=32 T=1024, cf=4, 3 levels, 2 + 2 cycles
    _full_case(B, WORKLOADS["medium"])


def _sampled_rows_case(B, w, rows):
    """Full-size run on the GPU; the oracle recomputes the batch rows `rows` of every layer."""
    from paper_2203_04738_b200.train_step import alloc_buffers, training_step
    d = make_inputs(w)
    dev = torch.device("cuda")
    layers = [{n: to_dev(l[n]) for n in NAMES} for l in d["layers"]]
    W_c, b_c, labels, h0, x = to_dev(d["W_c"]), to_dev(d["b_c"]), to_dev(d["labels"]), to_dev(d["h0"]), to_dev(d["x"])
    buf = alloc_buffers(w, w.T, w.B, dev, flags=B.FLAG_SKIP_DUPLICATE_FRELAX, want_dh=True)   # as the benchmark runs it (+ dh)
    training_step(w, layers, W_c, b_c, x, h0, labels, buf, update=False)
    torch.cuda.synchronize()
    assert B.last_device_status() == 0
    kw = dict(cf=w.cf, levels=w.levels, relax_fine=w.relax_fine, relax_coarse=w.relax_coarse)
    inp = d["x"][:, rows].astype(np.float64)
    h0r = d["h0"][rows].astype(np.float64)
    hs_gpu = []
    for l in range(w.layers):
        P = oracle_params(d, l)
        href, _ = O.mgrit_forward(*P, inp, h0r, iters=w.iters_fwd, **kw)
        hg = buf.h[l][:, rows].cpu().numpy()
        assert rel_inf(hg, href) < TOL, ("h", l)
        hs_gpu.append(hg.astype(np.float64))
        inp = hs_gpu[-1]          # the next layer is fed what the GPU fed it
    # adjoint of the sampled rows, linearised at the GPU's states, seeded with the GPU's loss gradient
    # (which couples the rows through the batch mean only by a constant factor already inside dhT)
    loss, dhT, dWc, dbc = B.xent_head_fwd_bwd(buf.h[-1][-1], W_c, b_c, labels)
    lr, dh_r, _, _ = O.xent_head(buf.h[-1][-1].cpu().numpy().astype(np.float64), d["W_c"].astype(np.float64),
                                 d["b_c"].astype(np.float64), d["labels"])
    assert abs(loss.item() - lr) < 1e-4 and rel_inf(dhT.cpu().numpy(), dh_r) < 1e-3
    seed = np.zeros_like(hs_gpu[-1])
    seed[-1] = dhT[rows].cpu().numpy()
    for l in range(w.layers - 1, -1, -1):
        P = oracle_params(d, l)
        inp = d["x"][:, rows].astype(np.float64) if l == 0 else hs_gpu[l - 1]
        lam, lam0, g, _ = O.mgrit_adjoint(*P, inp, h0r, hs_gpu[l], seed, iters=w.iters_adj, want_dx=l > 0, **kw)
        assert rel_inf(buf.adj[l].dh[:, rows].cpu().numpy(), lam) < TOL, ("dh", l)
        if l > 0:
            dxg = buf.adj[l].dx[:, rows].cpu().numpy()
            assert rel_inf(dxg, g["dx"]) < TOL, ("dx", l)
            seed = dxg.astype(np.float64)
    # Weight gradients: g = sum over ALL (t, b) of w_t dh_t/dTheta (Algorithm "MGRITTraining", gradient line) -- one
    # time-parallel pass of the oracle in fp64 over the full batch, fed the GPU's states and sensitivities, so that
    # exactly the gradient kernels (operand forming, split reduction GEMMs with K = T*B, bias sums) are compared.
    h0f = d["h0"].astype(np.float64)
    for l in range(w.layers):
        P = oracle_params(d, l)
        inp = (d["x"] if l == 0 else buf.h[l - 1].cpu().numpy()).astype(np.float64)
        g = O.weight_gradients(*P, inp, h0f, buf.h[l].cpu().numpy().astype(np.float64),
                               buf.adj[l].dh.cpu().numpy().astype(np.float64), want_dx=False)
        del inp
        for k in ("dW_ih", "dW_hh", "db_ih", "db_hh"):
            assert rel_inf(getattr(buf.adj[l], k).cpu().numpy(), g[k]) < TOL, (k, l)
        del g


def test_long_sampled_rows(B):
    # fourth configuration at full size: I=2048 H=1024 B=8 T=4096, cf=8, 4 levels, 3 + 3 cycles
    _sampled_rows_case(B, WORKLOADS["long"], [0, 5])


def test_train_sampled_rows(B):
    # fifth configuration at full size: 2 stacked layers, I=2048 H=1024 B=32 T=2048, cf=4, 3 levels, 2 + 2 cycles
    _sampled_rows_case(B, WORKLOADS["train"], [3])


def test_prefix_exactness_and_convergence_at_full_size(B):
    # properties that hold at any size: after k cycles the first k*cf states equal the serial sweep, the residual
    # falls from cycle to cycle, and more cycles approach the GPU's own serial sweep
    w = WORKLOADS["long"]
    d = make_inputs(w, T=1024)
    p, x, h0 = upload(d)
    cfg = _cfg(B, w, 3, T=1024)
    h, gi, rn = B.mgrit_gru_forward(cfg, p, x, h0, want_resnorm=True)
    hs, _ = B.gru_serial_forward(cfg, p, x, h0)
    k = 3 * w.cf
    assert rel_inf(h[:k].cpu().numpy(), hs[:k].cpu().numpy()) < 1e-2
    assert rn[0] > rn[1] > rn[2]
    e3 = rel_inf(h.cpu().numpy(), hs.cpu().numpy())
    h8, _, _ = B.mgrit_gru_forward(_cfg(B, w, 8, T=1024), p, x, h0)
    e8 = rel_inf(h8.cpu().numpy(), hs.cpu().numpy())
    assert e8 < e3 and e8 < 2e-2
    h_dup, _, _ = B.mgrit_gru_forward(_cfg(B, w, 3, T=1024, flags=B.FLAG_SKIP_DUPLICATE_FRELAX), p, x, h0)
    assert torch.equal(h, h_dup)


def test_run_to_run_bit_identical_and_workspace_content_irrelevant(B):
    # The result must not depend on scheduling (many tiles per CTA, three levels, additive terms on the inner
    # level) nor on what the caller's workspace held before the call.
    w = Workload("det", T=1024, B=32, I=64, H=512, cf=4, levels=3, iters_fwd=2, iters_adj=2, relax_fine=0, relax_coarse=1,
                 operands=2, classes=8, relu=True, seed=7)
    d = make_inputs(w)
    p, x, h0 = upload(d)
    cfg = _cfg(B, w, 2)
    nf, na = B.workspace_bytes(cfg)
    outs = []
    for fill in (0x00, 0x7F, 0x00, 0xFF):
        ws = torch.full((nf,), fill, dtype=torch.uint8, device="cuda")
        h, gi, _ = B.mgrit_gru_forward(cfg, p, x, h0, ws=ws)
        wa = torch.full((na,), fill, dtype=torch.uint8, device="cuda")
        r = B.mgrit_gru_adjoint(cfg, p, x, h0, gi, h, dhT=h[-1].contiguous(), ws=wa)
        loss, dhT, dWc, dbc = B.xent_head_fwd_bwd(h[-1].contiguous(), to_dev(d["W_c"]), to_dev(d["b_c"]), to_dev(d["labels"]))
        outs.append([t.clone() for t in (h, r.dh, r.dh0, r.dx, r.dW_hh, r.dW_ih, r.db_hh, r.db_ih, loss, dhT, dWc, dbc)])
    for o in outs[1:]:
        for a, b in zip(o, outs[0]):
            assert torch.equal(a, b)      # every reduction (split GEMMs, bias sums, loss) runs in a fixed order
    assert B.last_device_status() == 0


def test_copies_carried_behind_gi_change_nothing_but_rounding(B):
    # FLAG_GI_CARRIES_COPIES moves where the bf16 copies of x, [h_0; h] and gi live: the forward outputs keep their bits
    # (also with the larger buffer poisoned beforehand); the adjoint then linearises at the bf16 copy of gi, the values the
    # forward solve itself used, instead of the fp32 projection, so its outputs move by that rounding and no more.  A case
    # without state copies (B does not divide 128) ignores the flag and keeps every bit.
    for Bsz in (32, 24):
        w = Workload("carry", T=256, B=Bsz, I=64, H=256, cf=4, levels=3, iters_fwd=2, iters_adj=2, relax_fine=0, relax_coarse=1,
                     operands=2, classes=8, relu=True, seed=11)
        d = make_inputs(w)
        p, x, h0 = upload(d)
        plain, carry = _cfg(B, w, 2), _cfg(B, w, 2, flags=B.FLAG_GI_CARRIES_COPIES)
        h, gi, _ = B.mgrit_gru_forward(plain, p, x, h0)
        r = B.mgrit_gru_adjoint(plain, p, x, h0, gi, h, dhT=h[-1].contiguous())
        buf = B.alloc_gi(carry, x.device)
        assert buf.numel() * 4 == B.lib.mgrit_gru_gi_bytes(carry) > gi.numel() * 4 + 2 * (x.numel() + h.numel())
        buf.fill_(float("nan"))
        h2, gi2, _ = B.mgrit_gru_forward(carry, p, x, h0, gi=buf)
        assert gi2 is buf and torch.equal(B.gi_view(carry, buf), gi) and torch.equal(h2, h)
        r2 = B.mgrit_gru_adjoint(carry, p, x, h0, buf, h2, dhT=h2[-1].contiguous())
        for k in ("dh", "dh0", "dx", "dW_ih", "dW_hh", "db_ih", "db_hh"):
            a, b = getattr(r, k), getattr(r2, k)
            if Bsz == 24:
                assert torch.equal(a, b), k
            else:
                # (dh0 has decayed by orders of magnitude over the sequence: compared on the scale of dh)
                scale = float(r.dh.abs().max()) if k == "dh0" else float(a.abs().max())
                assert float((a - b).abs().max()) <= 5e-3 * scale, k
    assert B.last_device_status() == 0


def test_unwritten_fp32_projection_changes_no_bit(B):
    # FLAG_GI_F32_UNUSED: the forward call writes only the bf16 copy of the projection (the chain of the coarsest level
    # then reads that copy instead of rounding the fp32 values itself) and leaves the fp32 part of the buffer alone --
    # every output of the forward and of the adjoint call must keep its bits, and the poison must still be there.
    # Where the copies do not exist (B does not divide 128) the flag is ignored and the projection is written.
    for Bsz in (32, 8, 24):
        w = Workload("nof32", T=256, B=Bsz, I=64, H=256, cf=4, levels=3, iters_fwd=2, iters_adj=2, relax_fine=0, relax_coarse=1,
                     operands=2, classes=8, relu=True, seed=17)
        d = make_inputs(w)
        p, x, h0 = upload(d)
        carry = _cfg(B, w, 2, flags=B.FLAG_GI_CARRIES_COPIES)
        skip = _cfg(B, w, 2, flags=B.FLAG_GI_CARRIES_COPIES | B.FLAG_GI_F32_UNUSED)
        b1, b2 = B.alloc_gi(carry, x.device), B.alloc_gi(skip, x.device)
        assert b1.numel() == b2.numel()
        b2.fill_(float("nan"))
        h, _, rn = B.mgrit_gru_forward(carry, p, x, h0, gi=b1, want_resnorm=True)
        h2, _, rn2 = B.mgrit_gru_forward(skip, p, x, h0, gi=b2, want_resnorm=True)
        assert torch.equal(h, h2) and rn == rn2
        written = not bool(torch.isnan(B.gi_view(skip, b2)).all())
        import os
        assert written == (Bsz == 24 or os.environ.get("MGRIT_GRU_GI_BF16") == "0")      # (that A/B switch removes the bf16 copy)
        if written:
            assert torch.equal(B.gi_view(skip, b2), B.gi_view(carry, b1))
        r = B.mgrit_gru_adjoint(carry, p, x, h0, b1, h, dhT=h[-1].contiguous())
        r2 = B.mgrit_gru_adjoint(skip, p, x, h0, b2, h2, dhT=h2[-1].contiguous())
        for k in ("dh", "dh0", "dx", "dW_ih", "dW_hh", "db_ih", "db_hh"):
            assert torch.equal(getattr(r, k), getattr(r2, k)), k
    assert B.last_device_status() == 0


def test_state_array_with_a_leading_slot_keeps_every_bit(B):
    # FLAG_H_LEADS_WITH_H0: the level-0 unknowns live in the caller's [T+1,B,H] array (slot 0 = h_0) and the final copy is
    # saved; h must keep its bits, for the multigrid solve and the serial sweep, on the tensor-core and the FFMA engine.
    for operands in (B.OPERANDS_BF16, B.OPERANDS_FP32):
        w = Workload("lead", T=128, B=16, I=64, H=128, cf=4, levels=3, iters_fwd=2, iters_adj=2, relax_fine=0, relax_coarse=1,
                     operands=operands, classes=8, relu=True, seed=19)
        d = make_inputs(w)
        d["h0"] = (np.random.default_rng(3).standard_normal(d["h0"].shape) * 0.3).astype(np.float32)
        p, x, h0 = upload(d)
        kw = dict(cf=w.cf, levels=w.levels, iters=2, relax_fine=w.relax_fine, relax_coarse=w.relax_coarse, operands=operands)
        plain = B.make_cfg(w.T, w.B, w.I, w.H, **kw)
        lead = B.make_cfg(w.T, w.B, w.I, w.H, flags=B.FLAG_H_LEADS_WITH_H0, **kw)
        h, gi, _ = B.mgrit_gru_forward(plain, p, x, h0)
        full = torch.full((w.T + 1, w.B, w.H), float("nan"), device="cuda")
        h2, _, _ = B.mgrit_gru_forward(lead, p, x, h0, h=full)
        assert h2.data_ptr() == full[1:].data_ptr() and torch.equal(h2, h) and torch.equal(full[0], h0)
        # the adjoint given h_0 in the slot in front of h (one linearisation launch per level instead of two) changes no bit
        seed = to_dev((np.random.default_rng(4).standard_normal((w.T, w.B, w.H)) * 0.1).astype(np.float32))
        pad = torch.zeros(3, w.B, w.H, device="cuda")      # an h_0 that certainly does not sit in front of h
        pad[1].copy_(h0)
        n0 = B.kernel_launches()
        r = B.mgrit_gru_adjoint(plain, p, x, pad[1], gi, h, dh_seed=seed)
        n1 = B.kernel_launches()
        r2 = B.mgrit_gru_adjoint(plain, p, x, full[0], gi, h2, dh_seed=seed)
        n2 = B.kernel_launches()
        for k in ("dh", "dh0", "dx", "dW_ih", "dW_hh", "db_ih", "db_hh"):
            assert torch.equal(getattr(r, k), getattr(r2, k)), k
        if operands == B.OPERANDS_BF16:
            assert n2 - n1 < n1 - n0
        hs, _ = B.gru_serial_forward(plain, p, x, h0)
        full.fill_(float("nan"))
        hs2, _ = B.gru_serial_forward(lead, p, x, h0, h=full)
        assert torch.equal(hs2, hs) and torch.equal(full[0], h0)
    assert B.last_device_status() == 0


def test_long_sweeps_repeat_bit_for_bit(B):
    # Sixteen dependent steps per launch (cf = 8, FCF on both non-coarsest levels), single-CTA and pair geometry, tiles of a
    # later step waiting on counters of the earlier one: a missed dependency would show as a run that differs.
    for Bsz, T in ((8, 2048), (32, 1024)):
        w = Workload("rep", T=T, B=Bsz, I=64, H=512, cf=8, levels=3, iters_fwd=2, iters_adj=2, relax_fine=1, relax_coarse=1,
                     operands=2, classes=8, relu=True, seed=13)
        d = make_inputs(w)
        p, x, h0 = upload(d)
        cfg = _cfg(B, w, 2)
        first = None
        for _ in range(12):
            h, _, rn = B.mgrit_gru_forward(cfg, p, x, h0, want_resnorm=True)
            if first is None:
                first = h.clone()
            assert torch.equal(h, first)
    assert B.last_device_status() == 0
