"""The C-ABI library loads without a GPU and exports every function that include/mgrit_gru.h declares;
host-side argument checks answer without touching a device."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADER = os.path.join(ROOT, "include", "mgrit_gru.h")


@pytest.fixture(scope="module")
def lib():
    from paper_2203_04738_b200.build import build
    return ctypes.CDLL(build())


def declared_functions():
    src = open(HEADER).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    names = re.findall(r"\b([a-z_0-9]+)\s*\(", src)
    return sorted({n for n in names if n not in ("defined",)})


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert "mgrit_gru_forward" in names and "mgrit_gru_adjoint" in names and "gru_serial_backward" in names
    assert "xent_head_fwd_bwd_noalloc" in names and len(names) >= 14
    for n in names:
        assert hasattr(lib, n), n


def test_host_side_validation_without_a_device(lib):
    from paper_2203_04738_b200.binding import Cfg, make_cfg
    f, a = ctypes.c_size_t(0), ctypes.c_size_t(0)
    fn = lib.mgrit_gru_workspace_bytes
    fn.argtypes = [ctypes.POINTER(Cfg), ctypes.POINTER(ctypes.c_size_t), ctypes.POINTER(ctypes.c_size_t)]
    assert fn(ctypes.byref(make_cfg(128, 4, 16, 32, cf=4, levels=3)), ctypes.byref(f), ctypes.byref(a)) == 0
    assert f.value > 0 and a.value > f.value
    assert fn(ctypes.byref(make_cfg(100, 4, 16, 32, cf=8, levels=3)), ctypes.byref(f), ctypes.byref(a)) == -2   # not divisible
    assert fn(ctypes.byref(make_cfg(128, 4, 16, 32, cf=1, levels=2)), ctypes.byref(f), ctypes.byref(a)) == -1   # cf < 2
    assert fn(ctypes.byref(make_cfg(128, 4, 16, 36, cf=4, levels=2)), ctypes.byref(f), ctypes.byref(a)) == -4   # H % 8
    assert fn(ctypes.byref(make_cfg(128, 4, 16, 32, cf=4, levels=2, operands=2)), ctypes.byref(f), ctypes.byref(a)) == -4  # bf16 needs H % 64
    assert fn(None, ctypes.byref(f), ctypes.byref(a)) == -1
    lib.mgrit_gru_strerror.restype = ctypes.c_char_p
    assert b"divisible" in lib.mgrit_gru_strerror(-2)
    lib.xent_head_workspace_bytes.restype = ctypes.c_size_t
    assert lib.xent_head_workspace_bytes(32, 51) >= 32 * 51 * 4


def test_sizes_beyond_32_bit_row_counts_are_rejected(lib):
    from paper_2203_04738_b200.binding import Cfg, make_cfg
    f = ctypes.c_size_t(0)
    fn = lib.mgrit_gru_workspace_bytes
    fn.argtypes = [ctypes.POINTER(Cfg), ctypes.POINTER(ctypes.c_size_t), ctypes.POINTER(ctypes.c_size_t)]
    # (T + 1) * B just above 2^31: row counts are 32-bit inside the kernels
    assert fn(ctypes.byref(make_cfg(1 << 26, 32, 16, 64, cf=4, levels=2)), ctypes.byref(f), None) == -4
    assert fn(ctypes.byref(make_cfg(1 << 25, 32, 16, 64, cf=4, levels=2)), ctypes.byref(f), None) == 0
    assert f.value > (1 << 25) * 32 * 64 * 4          # the size itself is computed in 64 bits


def test_status_calls_answer_without_a_device(lib):
    # no device: nothing to wait for and nothing recorded -- the calls must return an error code, never crash
    lib.mgrit_gru_last_device_status.restype = ctypes.c_int
    lib.mgrit_gru_clear_device_status.restype = ctypes.c_int
    import torch
    if torch.cuda.is_available():
        assert lib.mgrit_gru_clear_device_status() == 0 and lib.mgrit_gru_last_device_status() == 0
    else:
        assert lib.mgrit_gru_last_device_status() == -5 and lib.mgrit_gru_clear_device_status() == -5
        assert lib.mgrit_gru_selftest_bounded_wait(20, None) == -5        # no device to run the self-test on
    assert lib.mgrit_gru_selftest_bounded_wait(0, None) == -1 and lib.mgrit_gru_selftest_bounded_wait(5000, None) == -1


def test_cycle_variant_flags_are_validated_on_the_host(lib):
    from paper_2203_04738_b200.binding import Cfg, FLAG_F_CYCLE, FLAG_RAGGED_T, make_cfg
    f, a = ctypes.c_size_t(0), ctypes.c_size_t(0)
    fn = lib.mgrit_gru_workspace_bytes
    fn.argtypes = [ctypes.POINTER(Cfg), ctypes.POINTER(ctypes.c_size_t), ctypes.POINTER(ctypes.c_size_t)]
    assert fn(ctypes.byref(make_cfg(23, 2, 16, 32, cf=4, levels=2)), ctypes.byref(f), ctypes.byref(a)) == -2
    assert fn(ctypes.byref(make_cfg(23, 2, 16, 32, cf=4, levels=2, flags=FLAG_RAGGED_T)), ctypes.byref(f), ctypes.byref(a)) == 0
    assert fn(ctypes.byref(make_cfg(7, 2, 16, 32, cf=4, levels=3, flags=FLAG_RAGGED_T)), ctypes.byref(f), ctypes.byref(a)) == -2
    assert fn(ctypes.byref(make_cfg(64, 2, 16, 32, cf=4, levels=3, relax_fine=2, relax_coarse=3, flags=FLAG_F_CYCLE)),
              ctypes.byref(f), ctypes.byref(a)) == 0
    assert fn(ctypes.byref(make_cfg(64, 2, 16, 32, cf=4, levels=3, relax_fine=9)), ctypes.byref(f), ctypes.byref(a)) == -1


def test_gi_buffer_size_with_and_without_carried_copies(lib):
    from paper_2203_04738_b200.binding import Cfg, FLAG_GI_CARRIES_COPIES, make_cfg
    fn = lib.mgrit_gru_gi_bytes
    fn.argtypes, fn.restype = [ctypes.POINTER(Cfg)], ctypes.c_size_t
    T, Bz, I, H = 128, 4, 16, 64
    assert fn(ctypes.byref(make_cfg(T, Bz, I, H, cf=4, levels=3))) == T * Bz * 3 * H * 4
    n = fn(ctypes.byref(make_cfg(T, Bz, I, H, cf=4, levels=3, flags=FLAG_GI_CARRIES_COPIES)))
    # the projection, then the bf16 copies of x, of [h_0; h] and of the projection itself, each padded to 256 bytes
    need = T * Bz * 3 * H * 4 + T * Bz * I * 2 + (T + 1) * Bz * H * 2 + T * Bz * 3 * H * 2
    assert need <= n <= need + 4 * 256 and n % 256 == 0
    assert fn(ctypes.byref(make_cfg(100, Bz, I, H, cf=8, levels=3))) == 0       # a bad cfg has no size
