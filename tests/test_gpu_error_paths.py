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


# A bounded device-side wait that runs out: the library's self-test kernel waits 20 ms, with the same wait routine as
# the tensor-core kernels, on a barrier nothing signals, records the timeout and RETURNS (no trap, no fault).  The
# condition must show up in the status query and in the next synchronising entry point, stay until it is cleared, and
# leave the context fully usable: the same solve before and after gives the same bits.
TIMEOUT_CHILD = r"""
import time, torch
from paper_2203_04738_b200 import binding as B
from paper_2203_04738_b200.synthetic import Workload, make_inputs
w = Workload("err", T=64, B=8, I=64, H=128, cf=4, levels=2, iters_fwd=2, iters_adj=2, relax_fine=0, relax_coarse=1,
             operands=2, classes=8, relu=True, seed=3)
d = make_inputs(w)
p = {n: torch.from_numpy(d["layers"][0][n]).cuda() for n in ("W_ih", "W_hh", "b_ih", "b_hh")}
x, h0 = torch.from_numpy(d["x"]).cuda(), torch.from_numpy(d["h0"]).cuda()
cfg = B.make_cfg(w.T, w.B, w.I, w.H, cf=w.cf, levels=w.levels, iters=2, operands=B.OPERANDS_BF16)
h_before, _, rn_before = B.mgrit_gru_forward(cfg, p, x, h0, want_resnorm=True)
assert B.last_device_status() == 0
t0 = time.time()
B.selftest_bounded_wait(20)
st = B.last_device_status()                      # synchronises: returns once the wait has run out
dt = time.time() - t0
sync_code = 0
try:
    B.mgrit_gru_forward(cfg, p, x, h0, want_resnorm=True)
except B.MgritError as e:
    sync_code = e.code
still = B.last_device_status()
B.clear_device_status()
cleared = B.last_device_status()
h_after, _, rn_after = B.mgrit_gru_forward(cfg, p, x, h0, want_resnorm=True)
same = bool(torch.equal(h_before, h_after)) and rn_before == rn_after
print("RESULT", st, sync_code, still, cleared, int(same), int(0.015 < dt < 5.0), B.last_device_status())
"""


def test_bounded_wait_that_runs_out_is_reported_and_recoverable():
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, PYTHONPATH=root)
    r = subprocess.run([sys.executable, "-c", TIMEOUT_CHILD], check=True, env=env, cwd=root, timeout=600,
                       capture_output=True, text=True)
    line = [l for l in r.stdout.splitlines() if l.startswith("RESULT")][0]
    st, sync_code, still, cleared, same, in_time, final = (int(v) for v in line.split()[1:])
    assert st == -6 and sync_code == -6 and still == -6      # MGRIT_DEVICE_TIMEOUT, sticky
    assert cleared == 0 and final == 0
    assert same == 1 and in_time == 1
