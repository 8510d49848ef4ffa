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
