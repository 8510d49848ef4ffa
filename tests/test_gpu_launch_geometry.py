"""The same solve on two launch geometries: the tensor-core products on CTA pairs (plain products: 256 x 256 tiles;
fused recurrent product + cell: 256 x 240 tiles of 80 hidden units; two CTAs per MMA) and on single CTAs (128 x 256
and 128 x 192 tiles).  Each output element is accumulated over the same k-blocks in the
same order either way, so the results may differ by rounding of the accumulation inside the tensor core at most:
every output must agree to 1e-5 of its largest magnitude (bf16-operand noise is 100 times that).  The shape makes
the projection (40960 x 1536), the level-0 adjoint steps (10240 x 512) and the input gradient (40960 x 256) multi-wave
products, i.e. the ones that run on pairs.  The switch is read once per process, so each geometry runs in a child
process."""
import os
import subprocess
import sys

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

CHILD = r"""
import sys, numpy as np, torch
from paper_2203_04738_b200 import binding as B
from paper_2203_04738_b200.synthetic import Workload, make_inputs
w = Workload("geo", T=1280, B=32, I=256, H=512, cf=4, levels=3, iters_fwd=2, iters_adj=2, relax_fine=0, relax_coarse=1,
             operands=2, classes=8, relu=True, seed=31)
d = make_inputs(w)
names = ("W_ih", "W_hh", "b_ih", "b_hh")
p = {n: torch.from_numpy(d["layers"][0][n]).cuda() for n in names}
x, h0 = torch.from_numpy(d["x"]).cuda(), torch.from_numpy(d["h0"]).cuda()
cfg = B.make_cfg(w.T, w.B, w.I, w.H, cf=w.cf, levels=w.levels, iters=2, operands=B.OPERANDS_BF16)
h, gi, _ = B.mgrit_gru_forward(cfg, p, x, h0, want_resnorm=True)
seed = torch.from_numpy(np.random.default_rng(5).standard_normal(tuple(h.shape)).astype(np.float32)).cuda()
r = B.mgrit_gru_adjoint(cfg, p, x, h0, gi, h, dh_seed=seed)
torch.cuda.synchronize()
assert B.last_device_status() == 0
np.savez(sys.argv[1], gi=gi.cpu().numpy(), h=h.cpu().numpy(), dh=r.dh.cpu().numpy(), dx=r.dx.cpu().numpy(),
         dW_ih=r.dW_ih.cpu().numpy(), dW_hh=r.dW_hh.cpu().numpy())
"""


def test_pair_and_single_cta_products_agree(tmp_path):
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    outs = []
    for flag in ("1", "0"):
        out = str(tmp_path / f"geo{flag}.npz")
        env = dict(os.environ, MGRIT_GRU_GEMM_PAIR=flag, MGRIT_GRU_CELL_PAIR=flag, PYTHONPATH=root)
        subprocess.run([sys.executable, "-c", CHILD, out], check=True, env=env, cwd=root, timeout=600)
        outs.append(np.load(out))
    a, b = outs
    differ = 0
    for k in a.files:
        scale = np.max(np.abs(a[k]))
        err = np.max(np.abs(a[k] - b[k]))
        assert err <= 1e-5 * scale, (k, err, scale)
        differ += int(err > 0)
    print("outputs that differ at all:", differ, "of", len(a.files))


CHILD_SWEEP = r"""
import sys, numpy as np, torch
from paper_2203_04738_b200 import binding as B
from paper_2203_04738_b200.synthetic import Workload, make_inputs
out = {}
# (cf, levels, relax_fine, relax_coarse, B, T, flags): FCF and FCFCF sweeps with C-steps, pair and single-CTA geometry,
# a row count that ends in a partial tile, F-cycles
cases = [(4, 3, 0, 1, 32, 1024, 0), (4, 3, 1, 2, 16, 512, 0), (2, 4, 1, 1, 8, 272, 0), (8, 2, 1, 1, 32, 512, B.FLAG_F_CYCLE),
         (4, 2, 2, 0, 4, 96, 0)]
for i, (cf, L, rf, rc, Bz, T, fl) in enumerate(cases):
    w = Workload("sweep", T=T, B=Bz, I=64, H=512, cf=cf, levels=L, iters_fwd=2, iters_adj=2, relax_fine=rf, relax_coarse=rc,
                 operands=2, classes=8, relu=True, seed=40 + i)
    d = make_inputs(w)
    p = {n: torch.from_numpy(d["layers"][0][n]).cuda() for n in ("W_ih", "W_hh", "b_ih", "b_hh")}
    x, h0 = torch.from_numpy(d["x"]).cuda(), torch.from_numpy(d["h0"]).cuda()
    cfg = B.make_cfg(T, Bz, w.I, w.H, cf=cf, levels=L, iters=2, relax_fine=rf, relax_coarse=rc, operands=B.OPERANDS_BF16, flags=fl)
    n0 = B.kernel_launches()
    h, gi, rn = B.mgrit_gru_forward(cfg, p, x, h0, want_resnorm=True)
    out[f"launches{i}"] = np.array([B.kernel_launches() - n0])
    out[f"h{i}"] = h.cpu().numpy(); out[f"rn{i}"] = np.array(rn)
torch.cuda.synchronize()
assert B.last_device_status() == 0
np.savez(sys.argv[1], **out)
"""


def test_relaxation_sweeps_in_one_launch_give_the_same_bits(tmp_path):
    """A relaxation sweep F (CF)^n [+ the evaluation of v] as ONE launch of the fused kernel, tiles of later steps
    waiting on the row tiles they read, against one launch per step: the arithmetic of every element is the same, so
    the states must be bit-identical (the residual norms are sums of atomics and agree to rounding); and the sweeps
    must really have replaced launches."""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    outs = []
    for flag in ("1", "0"):
        out = str(tmp_path / f"sweep{flag}.npz")
        env = dict(os.environ, MGRIT_GRU_SWEEP=flag, PYTHONPATH=root)
        subprocess.run([sys.executable, "-c", CHILD_SWEEP, out], check=True, env=env, cwd=root, timeout=600)
        outs.append(np.load(out))
    a, b = outs
    for k in a.files:
        if k.startswith("h"):
            assert np.array_equal(a[k], b[k]), k
        elif k.startswith("rn"):
            assert np.allclose(a[k], b[k], rtol=1e-5), k
        else:
            assert a[k][0] < b[k][0], (k, a[k], b[k])


def test_staged_and_global_load_adjoint_epilogues_agree(tmp_path):
    """The adjoint product with TMA-staged epilogue operands (reversed coefficient rows, pair and single-CTA geometry,
    with and without a source term) against the plain GEMM whose epilogue loads the same operands from global memory:
    the same sums in the same order, up to how the compiler contracts one multiply-add."""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    outs = []
    for flag in ("1", "0"):
        out = str(tmp_path / f"adj{flag}.npz")
        env = dict(os.environ, MGRIT_GRU_ADJ_STAGED=flag, PYTHONPATH=root)
        subprocess.run([sys.executable, "-c", CHILD, out], check=True, env=env, cwd=root, timeout=600)
        outs.append(np.load(out))
    a, b = outs
    for k in a.files:
        scale = np.max(np.abs(a[k]))
        assert np.max(np.abs(a[k] - b[k])) <= 1e-6 * scale, k


CHILD_CHAIN = r"""
import sys, numpy as np, torch
from paper_2203_04738_b200 import binding as B
from paper_2203_04738_b200.synthetic import Workload, make_inputs
out = {}
# (T, B, H, levels): the serial sweep as one chain (8 units per CTA), and a coarsest level of 16 steps at the widest shape
# (16 units per CTA, two row groups, one of them partial)
for i, (T, Bz, H, L) in enumerate([(48, 8, 512, 1), (64, 24, 1024, 2)]):
    w = Workload("chainw", T=T, B=Bz, I=64, H=H, cf=4, levels=L, iters_fwd=2, iters_adj=2, relax_fine=0, relax_coarse=1,
                 operands=2, classes=8, relu=True, seed=70 + i)
    d = make_inputs(w)
    p = {n: torch.from_numpy(d["layers"][0][n]).cuda() for n in ("W_ih", "W_hh", "b_ih", "b_hh")}
    x, h0 = torch.from_numpy(d["x"]).cuda(), torch.from_numpy(d["h0"]).cuda()
    cfg = B.make_cfg(T, Bz, w.I, H, cf=4, levels=L, iters=2, operands=B.OPERANDS_BF16)
    if L == 1:
        h, gi = B.gru_serial_forward(cfg, p, x, h0)
    else:
        h, gi, _ = B.mgrit_gru_forward(cfg, p, x, h0)
    seed = torch.from_numpy(np.random.default_rng(5 + i).standard_normal(tuple(h.shape)).astype(np.float32)).cuda()
    r = B.gru_serial_backward(cfg, p, x, h0, gi, h, dh_seed=seed) if L == 1 else B.mgrit_gru_adjoint(cfg, p, x, h0, gi, h, dh_seed=seed)
    out[f"h{i}"] = h.cpu().numpy(); out[f"dh{i}"] = r.dh.cpu().numpy(); out[f"dW_hh{i}"] = r.dW_hh.cpu().numpy()
torch.cuda.synchronize()
assert B.last_device_status() == 0
np.savez(sys.argv[1], **out)
"""


def test_chain_weights_in_registers_give_the_same_bits(tmp_path):
    """The persistent chain kernels with their weight fragments in registers issue the same products in the same order
    as with the weights in shared memory: every output must be bit-identical."""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    outs = []
    for flag in ("1", "0"):
        out = str(tmp_path / f"chainw{flag}.npz")
        env = dict(os.environ, MGRIT_GRU_CHAIN_WREG=flag, PYTHONPATH=root)
        subprocess.run([sys.executable, "-c", CHILD_CHAIN, out], check=True, env=env, cwd=root, timeout=600)
        outs.append(np.load(out))
    a, b = outs
    for k in a.files:
        assert np.array_equal(a[k], b[k]), k
