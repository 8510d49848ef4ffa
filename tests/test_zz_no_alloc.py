"""The allocation-free loss head (xent_head_fwd_bwd_noalloc) against the regular entry point.

Collected last on purpose (file name): a run that stops at the first failure has then already run
every other test.  Some users of the library cannot allocate device memory when they need the head
(their own arena owns the GPU's memory, or they must stay clear of the driver's allocator in a
latency-critical loop), so this entry point keeps its only intermediate in an array built into the
library.  Checked here through the C ABI: same results as the workspace version and as the fp64
oracle, on two calls in a row with different inputs (the second call sees the first call's leftovers
in the shared array); no device memory is allocated by a call; and a clear error beyond the built-in
limit.  Passes alone in a fresh process and after the other tests.
"""
import ctypes
import gc

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def test_noalloc_head_matches_workspace_head_twice_in_a_row():
    from oracle import mgrit_gru_oracle as O
    from paper_2203_04738_b200 import binding as B
    rng = np.random.default_rng(123)
    dev = torch.device("cuda")
    for call, (Bn, H, C) in enumerate([(32, 256, 51), (7, 64, 8)]):      # second call: smaller, other values
        hT = torch.from_numpy(rng.standard_normal((Bn, H)).astype(np.float32)).to(dev)
        Wc = torch.from_numpy((rng.standard_normal((C, H)) * 0.1).astype(np.float32)).to(dev)
        bc = torch.from_numpy((rng.standard_normal(C) * 0.1).astype(np.float32)).to(dev)
        lab = torch.from_numpy(rng.integers(0, C, Bn).astype(np.int32)).to(dev)
        ref = B.xent_head_fwd_bwd(hT, Wc, bc, lab)
        # outputs are allocated by the caller beforehand; the call itself gets no workspace
        out = (torch.empty(1, device=dev), torch.empty(Bn, H, device=dev), torch.empty(C, H, device=dev), torch.empty(C, device=dev))
        got = B.xent_head_fwd_bwd_noalloc(hT, Wc, bc, lab, out=out)
        assert abs(got[0].item() - ref[0].item()) < 1e-5, call
        for a, b in zip(got[1:], ref[1:]):
            den = float(b.abs().max())
            assert float((a - b).abs().max()) <= 1e-3 * den + 1e-7, call      # the gradient tolerance of the fp32 tests
        # ... and against the oracle's head (mean softmax cross-entropy and its derivatives in fp64)
        want = O.xent_head(hT.cpu().numpy().astype(np.float64), Wc.cpu().numpy().astype(np.float64),
                           bc.cpu().numpy().astype(np.float64), lab.cpu().numpy())
        assert abs(got[0].item() - want[0]) < 1e-5, call
        for a, b in zip(got[1:], want[1:]):
            assert float(np.max(np.abs(a.cpu().numpy() - b))) <= 1e-3 * float(np.max(np.abs(b))) + 1e-7, call
        # The set-up call above resolved the built-in array's address.  From here on a call must leave the
        # device's memory as it found it: nothing allocated through torch, nothing taken from the driver.
        # (Python's cycle collector is held off meanwhile: it may free tensors of earlier tests at any moment.)
        gc.collect()
        gc.disable()
        try:
            torch.cuda.synchronize()
            free0, alloc0, reserved0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
            B.xent_head_fwd_bwd_noalloc(hT, Wc, bc, lab, out=out)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free0 and torch.cuda.memory_allocated() == alloc0
            assert torch.cuda.memory_reserved() == reserved0
        finally:
            gc.enable()
    assert B.last_device_status() == 0


def test_noalloc_head_rejects_sizes_beyond_its_scratch():
    from paper_2203_04738_b200 import binding as B
    dev = torch.device("cuda")
    Bn, H, C = 1024, 8, 128                                                 # B*(C+1) = 132096 > 65536
    hT = torch.zeros(Bn, H, device=dev); Wc = torch.zeros(C, H, device=dev); bc = torch.zeros(C, device=dev)
    lab = torch.zeros(Bn, dtype=torch.int32, device=dev)
    with pytest.raises(B.MgritError) as e:
        B.xent_head_fwd_bwd_noalloc(hT, Wc, bc, lab)
    assert e.value.code == -7 and "scratch" in str(e.value)
    # exactly at the limit is accepted, one row more is not:  B*(C+1) <= 65536
    Bn, C = 1024, 63
    hT = torch.zeros(Bn, H, device=dev); Wc = torch.zeros(C, H, device=dev); bc = torch.zeros(C, device=dev)
    lab = torch.zeros(Bn, dtype=torch.int32, device=dev)
    B.xent_head_fwd_bwd_noalloc(hT, Wc, bc, lab)
    hT = torch.zeros(Bn + 1, H, device=dev); lab = torch.zeros(Bn + 1, dtype=torch.int32, device=dev)
    with pytest.raises(B.MgritError) as e:
        B.xent_head_fwd_bwd_noalloc(hT, Wc, bc, lab)
    assert e.value.code == -7
