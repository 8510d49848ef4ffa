"""Error paths of the C ABI that need a device but provoke no fault on it.

A launch that cannot be PREPARED (the tensor-map encoder is unavailable, an encode fails) must surface as
MGRIT_CUDA_ERROR from the entry point, not as MGRIT_OK with stale outputs.  The library reads
MGRIT_GRU_TEST_FAIL_ENCODE once per process and then refuses to prepare any tensor-core launch, so the path is
exercised from the host: the kernels concerned are simply never launched.  Each case runs in a child process."""
import os
import subprocess
import sys

import pytest

pytestmark = pytest.mark.gpu

CHILD = r"""
import ctypes, sys, torch
from paper_2203_04738_b200 import binding as B
from paper_2203_04738_b200.synthetic import Workload, make_inputs
w = Workload("err", T=64, B=8, I=64, H=128, cf=4, levels=2, iters_fwd=2, iters_adj=2, relax_fine=0, relax_coarse=1,
             operands=2, classes=8, relu=True, seed=3)
d = make_inputs(w)
names = ("W_ih", "W_hh", "b_ih", "b_hh")
p = {n: torch.from_numpy(d["layers"][0][n]).cuda() for n in names}
x, h0 = torch.from_numpy(d["x"]).cuda(), torch.from_numpy(d["h0"]).cuda()
codes = []
for operands in (B.OPERANDS_BF16, B.OPERANDS_FP32):
    cfg = B.make_cfg(w.T, w.B, w.I, w.H, cf=w.cf, levels=w.levels, iters=2, operands=operands)
    try:
        h, gi, _ = B.mgrit_gru_forward(cfg, p, x, h0)
        codes.append(0)
    except B.MgritError as e:
        codes.append(e.code)
    try:
        h, gi = B.gru_serial_forward(cfg, p, x, h0)
        codes.append(0)
    except B.MgritError as e:
        codes.append(e.code)
torch.cuda.synchronize()
assert B.last_device_status() == 0          # nothing hung, nothing faulted: the context is still usable
print("CODES", *codes)
"""


def _run(env_extra):
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, PYTHONPATH=root, **env_extra)
    r = subprocess.run([sys.executable, "-c", CHILD], check=True, env=env, cwd=root, timeout=600, capture_output=True, text=True)
    line = [l for l in r.stdout.splitlines() if l.startswith("CODES")][0]
    return [int(v) for v in line.split()[1:]]


def test_failed_launch_preparation_is_reported():
    # bf16 engine: every entry point that needs a tensor map reports MGRIT_CUDA_ERROR (-5); the fp32 engine needs none
    assert _run({"MGRIT_GRU_TEST_FAIL_ENCODE": "1"}) == [-5, -5, 0, 0]
    assert _run({}) == [0, 0, 0, 0]
