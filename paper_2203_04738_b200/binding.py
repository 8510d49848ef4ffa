"""Thin ctypes binding of the C ABI in include/mgrit_gru.h: argument marshalling only.

Tensors are torch CUDA tensors (fp32, contiguous); outputs and the workspace are allocated with
torch; work is enqueued on torch's current stream.  Every step of the path runs in the
library's kernels -- if the library has not been built, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmgrit_gru.so")
if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2203_04738_b200.build` "
                      "(there is no CPU or PyTorch fallback)")
lib = ctypes.CDLL(LIB_PATH)

OK = 0
CELL_CLASSIC, CELL_IMPLICIT = 0, 1
RELAX_F, RELAX_FCF, RELAX_FCFCF = 0, 1, 2
OPERANDS_FP32, OPERANDS_TF32, OPERANDS_BF16, OPERANDS_TF32_1PASS = 0, 1, 2, 3
FLAG_SKIP_DUPLICATE_FRELAX, FLAG_F_CYCLE, FLAG_RAGGED_T, FLAG_GI_CARRIES_COPIES, FLAG_GI_F32_UNUSED = 1, 2, 4, 8, 16
FLAG_H_LEADS_WITH_H0 = 32


class Cfg(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("T", "B", "I", "H", "cf", "levels", "iters", "cell", "relax_fine", "relax_coarse", "operands", "flags")] + \
               [("dt", ctypes.c_float)]


class _Params(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("W_ih", "W_hh", "b_ih", "b_hh")]


class _Grads(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("dW_ih", "dW_hh", "db_ih", "db_hh")]


_vp, _sz, _i32 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int32
lib.mgrit_gru_workspace_bytes.argtypes = [ctypes.POINTER(Cfg), ctypes.POINTER(_sz), ctypes.POINTER(_sz)]
lib.mgrit_gru_gi_bytes.argtypes = [ctypes.POINTER(Cfg)]
lib.mgrit_gru_gi_bytes.restype = _sz
lib.gru_input_projection.argtypes = [ctypes.POINTER(Cfg), ctypes.POINTER(_Params), _vp, _vp, _vp, _sz, _vp]
lib.mgrit_gru_forward.argtypes = [ctypes.POINTER(Cfg), ctypes.POINTER(_Params), _vp, _vp, _vp, _vp,
                                  ctypes.POINTER(ctypes.c_float), _vp, _sz, _vp]
lib.gru_serial_forward.argtypes = [ctypes.POINTER(Cfg), ctypes.POINTER(_Params), _vp, _vp, _vp, _vp, _vp, _sz, _vp]
lib.mgrit_gru_adjoint.argtypes = [ctypes.POINTER(Cfg), ctypes.POINTER(_Params), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp,
                                  ctypes.POINTER(_Grads), ctypes.POINTER(ctypes.c_float), _vp, _sz, _vp]
lib.gru_serial_backward.argtypes = [ctypes.POINTER(Cfg), ctypes.POINTER(_Params), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp,
                                    ctypes.POINTER(_Grads), _vp, _sz, _vp]
lib.mgrit_gru_stack_workspace_bytes.argtypes = [ctypes.POINTER(Cfg), _i32, ctypes.POINTER(_sz), ctypes.POINTER(_sz)]
lib.mgrit_gru_stack_forward.argtypes = [ctypes.POINTER(Cfg), _i32, ctypes.POINTER(_Params), _vp, _vp, _vp, _vp,
                                        ctypes.POINTER(ctypes.c_float), _vp, _sz, _vp]
lib.mgrit_gru_stack_adjoint.argtypes = [ctypes.POINTER(Cfg), _i32, ctypes.POINTER(_Params), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp,
                                        ctypes.POINTER(_Grads), ctypes.POINTER(ctypes.c_float), _vp, _sz, _vp]
lib.mgrit_lstm_workspace_bytes.argtypes = [ctypes.POINTER(Cfg), ctypes.POINTER(_sz), ctypes.POINTER(_sz)]
lib.mgrit_lstm_forward.argtypes = [ctypes.POINTER(Cfg), ctypes.POINTER(_Params), _vp, _vp, _vp, _vp, ctypes.POINTER(ctypes.c_float), _vp, _sz, _vp]
lib.mgrit_lstm_adjoint.argtypes = [ctypes.POINTER(Cfg), ctypes.POINTER(_Params), _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp,
                                   ctypes.POINTER(_Grads), ctypes.POINTER(ctypes.c_float), _vp, _sz, _vp]
lib.gru_step_rows.argtypes = [ctypes.POINTER(Cfg), ctypes.POINTER(_Params), _i32, ctypes.c_float, _vp, _vp, _vp, _vp]
lib.gru_adjoint_step_rows.argtypes = [ctypes.POINTER(Cfg), ctypes.POINTER(_Params), _i32, ctypes.c_float, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
lib.xent_head_workspace_bytes.argtypes = [_i32, _i32]
lib.xent_head_workspace_bytes.restype = _sz
lib.xent_head_fwd_bwd.argtypes = [_i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _sz, _vp]
lib.xent_head_fwd_bwd_noalloc.argtypes = [_i32, _i32, _i32, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp]
lib.sgd_update.argtypes = [_vp, _vp, _sz, ctypes.c_float, _vp]
lib.adam_update.argtypes = [_vp, _vp, _vp, _vp, _sz, ctypes.c_float, ctypes.c_float, ctypes.c_float, ctypes.c_float, _i32, _vp]
lib.mgrit_gru_selftest_bounded_wait.argtypes = [_i32, _vp]
lib.mgrit_gru_last_device_status.restype = ctypes.c_int
lib.mgrit_gru_clear_device_status.restype = ctypes.c_int
lib.mgrit_gru_kernel_launches.restype = ctypes.c_ulonglong
lib.mgrit_gru_profile_enable.argtypes = [ctypes.c_int]
lib.mgrit_gru_profile_read.argtypes = [ctypes.c_int, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_ulonglong),
                                       ctypes.POINTER(ctypes.c_double)]
lib.mgrit_gru_profile_records.argtypes = [ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double),
                                          ctypes.POINTER(ctypes.c_int32), _sz, ctypes.POINTER(_sz)]
lib.mgrit_gru_strerror.argtypes = [ctypes.c_int]
lib.mgrit_gru_strerror.restype = ctypes.c_char_p


class MgritError(RuntimeError):
    def __init__(self, code):
        self.code = code
        super().__init__(f"mgrit_gru error {code}: {lib.mgrit_gru_strerror(code).decode()}")


def _check(rc):
    if rc != OK:
        raise MgritError(rc)


def make_cfg(T, B, I, H, cf=4, levels=2, iters=2, cell=CELL_IMPLICIT, relax_fine=RELAX_F, relax_coarse=RELAX_FCF,
             operands=OPERANDS_FP32, flags=0, dt=1.0) -> Cfg:
    return Cfg(T, B, I, H, cf, levels, iters, cell, relax_fine, relax_coarse, operands, flags, dt)


def _ptr(t):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "CUDA contiguous tensor required"
    return ctypes.c_void_p(t.data_ptr())


def _f32(t):
    assert t is None or t.dtype == torch.float32
    return _ptr(t)


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _params(p):
    return _Params(*[p[n].data_ptr() for n in ("W_ih", "W_hh", "b_ih", "b_hh")])


def workspace_bytes(cfg: Cfg):
    f, a = _sz(0), _sz(0)
    _check(lib.mgrit_gru_workspace_bytes(ctypes.byref(cfg), ctypes.byref(f), ctypes.byref(a)))
    return f.value, a.value


def alloc_gi(cfg: Cfg, device) -> torch.Tensor:
    """The gi buffer for cfg as a flat fp32 tensor: gi[T,B,3H] first, then (with FLAG_GI_CARRIES_COPIES) room for the
    bf16 copies that travel from the forward call to the adjoint call.  `gi_view(cfg, buf)` is the projection itself."""
    nbytes = lib.mgrit_gru_gi_bytes(ctypes.byref(cfg))
    if nbytes == 0:
        raise MgritError(-1)
    return torch.empty((nbytes + 3) // 4, dtype=torch.float32, device=device)


def gi_view(cfg: Cfg, buf: torch.Tensor) -> torch.Tensor:
    return buf[: cfg.T * cfg.B * 3 * cfg.H].view(cfg.T, cfg.B, 3 * cfg.H)


def _ws(nbytes, ws, dev):
    if ws is None or ws.numel() < nbytes:
        ws = torch.empty(nbytes, dtype=torch.uint8, device=dev)
    return ws


def gru_input_projection(cfg, p, x, gi=None, ws=None):
    gi = torch.empty(cfg.T, cfg.B, 3 * cfg.H, device=x.device) if gi is None else gi
    ws = _ws(workspace_bytes(cfg)[0], ws, x.device)
    _check(lib.gru_input_projection(ctypes.byref(cfg), ctypes.byref(_params(p)), _f32(x), _f32(gi), _ptr(ws), ws.numel(), _stream()))
    return gi


def _h_array(cfg, h, dev):
    """The state array of a forward call and the number of leading slots that are not part of h[T,B,H]."""
    lead = 1 if cfg.flags & FLAG_H_LEADS_WITH_H0 else 0
    if h is None:
        h = torch.empty(cfg.T + lead, cfg.B, cfg.H, device=dev)
    assert h.shape[0] == cfg.T + lead and h.is_contiguous()
    return h, lead


def mgrit_gru_forward(cfg, p, x, h0, want_resnorm=False, gi=None, h=None, ws=None):
    """-> (h[T,B,H], gi[T,B,3H], resnorm list or None).  With FLAG_H_LEADS_WITH_H0 the array passed as `h` (or allocated
    here) has T + 1 slots, slot 0 receives h_0, and the returned h is the view of its slots 1..T."""
    dev = x.device
    gi = alloc_gi(cfg, dev) if gi is None else gi       # (a flat buffer when the copies flag is set, else viewed as [T,B,3H])
    if gi.dim() == 1 and not (cfg.flags & FLAG_GI_CARRIES_COPIES):
        gi = gi_view(cfg, gi)
    h, lead = _h_array(cfg, h, dev)
    ws = _ws(workspace_bytes(cfg)[0], ws, dev)
    rn = (ctypes.c_float * max(cfg.iters, 1))() if want_resnorm else None
    _check(lib.mgrit_gru_forward(ctypes.byref(cfg), ctypes.byref(_params(p)), _f32(x), _f32(h0), _f32(gi), _f32(h), rn,
                                 _ptr(ws), ws.numel(), _stream()))
    return h[lead:], gi, (list(rn)[:cfg.iters] if want_resnorm else None)


def gru_serial_forward(cfg, p, x, h0, gi=None, h=None, ws=None):
    dev = x.device
    gi = torch.empty(cfg.T, cfg.B, 3 * cfg.H, device=dev) if gi is None else gi
    h, lead = _h_array(cfg, h, dev)
    ws = _ws(workspace_bytes(cfg)[0], ws, dev)
    _check(lib.gru_serial_forward(ctypes.byref(cfg), ctypes.byref(_params(p)), _f32(x), _f32(h0), _f32(gi), _f32(h),
                                  _ptr(ws), ws.numel(), _stream()))
    return h[lead:], gi


@dataclass
class AdjointResult:
    dh: torch.Tensor | None
    dh0: torch.Tensor
    dx: torch.Tensor | None
    dW_ih: torch.Tensor
    dW_hh: torch.Tensor
    db_ih: torch.Tensor
    db_hh: torch.Tensor
    resnorm: list | None = None


def _adjoint(fn, serial, cfg, p, x, h0, gi, h, dh_seed, dhT, want_dx, want_resnorm, ws, out, want_dh=True):
    dev = x.device
    o = out or AdjointResult(
        dh=torch.empty(cfg.T, cfg.B, cfg.H, device=dev) if want_dh else None, dh0=torch.empty(cfg.B, cfg.H, device=dev),
        dx=torch.empty(cfg.T, cfg.B, cfg.I, device=dev) if want_dx else None,
        dW_ih=torch.empty(3 * cfg.H, cfg.I, device=dev), dW_hh=torch.empty(3 * cfg.H, cfg.H, device=dev),
        db_ih=torch.empty(3 * cfg.H, device=dev), db_hh=torch.empty(3 * cfg.H, device=dev))
    ws = _ws(workspace_bytes(cfg)[1], ws, dev)
    g = _Grads(o.dW_ih.data_ptr(), o.dW_hh.data_ptr(), o.db_ih.data_ptr(), o.db_hh.data_ptr())
    args = [ctypes.byref(cfg), ctypes.byref(_params(p)), _f32(x), _f32(h0), _f32(gi), _f32(h), _f32(dh_seed), _f32(dhT),
            _f32(o.dh), _f32(o.dh0), _f32(o.dx), ctypes.byref(g)]
    if not serial:
        rn = (ctypes.c_float * max(cfg.iters, 1))() if want_resnorm else None
        args.append(rn)
    args += [_ptr(ws), ws.numel(), _stream()]
    _check(fn(*args))
    if not serial and want_resnorm:
        o.resnorm = list(rn)[:cfg.iters]
    return o


def mgrit_gru_adjoint(cfg, p, x, h0, gi, h, dh_seed=None, dhT=None, want_dx=True, want_resnorm=False, ws=None, out=None,
                      want_dh=True):
    return _adjoint(lib.mgrit_gru_adjoint, False, cfg, p, x, h0, gi, h, dh_seed, dhT, want_dx, want_resnorm, ws, out, want_dh)


def gru_serial_backward(cfg, p, x, h0, gi, h, dh_seed=None, dhT=None, want_dx=True, ws=None, out=None, want_dh=True):
    return _adjoint(lib.gru_serial_backward, True, cfg, p, x, h0, gi, h, dh_seed, dhT, want_dx, False, ws, out, want_dh)


def gru_step_rows(cfg, p, gamma, gi_rows, u_prev, out=None):
    """out[n,B,H] = Phi_gamma(gi_rows[n,B,3H], u_prev[n,B,H]): one cell evaluation for n*B independent rows (fp32 engine)."""
    n = u_prev.shape[0]
    out = torch.empty_like(u_prev) if out is None else out
    _check(lib.gru_step_rows(ctypes.byref(cfg), ctypes.byref(_params(p)), n, float(gamma), _f32(gi_rows), _f32(u_prev), _f32(out),
                             _stream()))
    return out


def gru_adjoint_step_rows(cfg, p, gamma, gi_rows, h_lin, mu, out=None, ws=None):
    """out[n,B,H] = (dPhi_gamma/dh at (gi_rows, h_lin))^T mu: the adjoint of gru_step_rows, row by row."""
    n = mu.shape[0]
    out = torch.empty_like(mu) if out is None else out
    ws = _ws(5 * n * cfg.B * cfg.H * 4 + 5 * 256, ws, mu.device)
    _check(lib.gru_adjoint_step_rows(ctypes.byref(cfg), ctypes.byref(_params(p)), n, float(gamma), _f32(gi_rows), _f32(h_lin),
                                     _f32(mu), _f32(out), _ptr(ws), ws.numel(), _stream()))
    return out


def stack_workspace_bytes(cfg: Cfg, n_layers: int):
    f, a = _sz(0), _sz(0)
    _check(lib.mgrit_gru_stack_workspace_bytes(ctypes.byref(cfg), n_layers, ctypes.byref(f), ctypes.byref(a)))
    return f.value, a.value


def _param_array(layers):
    arr = (_Params * len(layers))()
    for k, p in enumerate(layers):
        arr[k] = _params(p)
    return arr


def mgrit_gru_stack_forward(cfg, layers, x, h0, want_resnorm=False, ws=None):
    """All layers in one state, one MGRIT cycle for the stack.  layers: list of parameter dicts; h0[n_layers,B,H].
    -> (h[T,n_layers,B,H], gi0[T,B,3H], resnorm list or None)"""
    dev, nl = x.device, len(layers)
    gi0 = torch.empty(cfg.T, cfg.B, 3 * cfg.H, device=dev)
    h = torch.empty(cfg.T, nl, cfg.B, cfg.H, device=dev)
    ws = _ws(stack_workspace_bytes(cfg, nl)[0], ws, dev)
    rn = (ctypes.c_float * max(cfg.iters, 1))() if want_resnorm else None
    _check(lib.mgrit_gru_stack_forward(ctypes.byref(cfg), nl, _param_array(layers), _f32(x), _f32(h0), _f32(gi0), _f32(h), rn,
                                       _ptr(ws), ws.numel(), _stream()))
    return h, gi0, (list(rn)[:cfg.iters] if want_resnorm else None)


def mgrit_gru_stack_adjoint(cfg, layers, x, h0, gi0, h, dh_seed=None, dhT=None, want_dx=True, want_dh=True, want_resnorm=False, ws=None):
    """-> (dh[T,n_layers,B,H] or None, dh0[n_layers,B,H], dx or None, list of per-layer AdjointResult (gradients only), resnorm)"""
    dev, nl = x.device, len(layers)
    dh = torch.empty(cfg.T, nl, cfg.B, cfg.H, device=dev) if want_dh else None
    dh0 = torch.empty(nl, cfg.B, cfg.H, device=dev)
    dx = torch.empty(cfg.T, cfg.B, cfg.I, device=dev) if want_dx else None
    outs, garr = [], (_Grads * nl)()
    for k in range(nl):
        Ik = cfg.I if k == 0 else cfg.H
        o = AdjointResult(dh=None, dh0=None, dx=None, dW_ih=torch.empty(3 * cfg.H, Ik, device=dev), dW_hh=torch.empty(3 * cfg.H, cfg.H, device=dev),
                          db_ih=torch.empty(3 * cfg.H, device=dev), db_hh=torch.empty(3 * cfg.H, device=dev))
        garr[k] = _Grads(o.dW_ih.data_ptr(), o.dW_hh.data_ptr(), o.db_ih.data_ptr(), o.db_hh.data_ptr())
        outs.append(o)
    ws = _ws(stack_workspace_bytes(cfg, nl)[1], ws, dev)
    rn = (ctypes.c_float * max(cfg.iters, 1))() if want_resnorm else None
    _check(lib.mgrit_gru_stack_adjoint(ctypes.byref(cfg), nl, _param_array(layers), _f32(x), _f32(h0), _f32(gi0), _f32(h), _f32(dh_seed),
                                       _f32(dhT), _f32(dh), _f32(dh0), _f32(dx), garr, rn, _ptr(ws), ws.numel(), _stream()))
    return dh, dh0, dx, outs, (list(rn)[:cfg.iters] if want_resnorm else None)


def lstm_workspace_bytes(cfg: Cfg):
    f, a = _sz(0), _sz(0)
    _check(lib.mgrit_lstm_workspace_bytes(ctypes.byref(cfg), ctypes.byref(f), ctypes.byref(a)))
    return f.value, a.value


def mgrit_lstm_forward(cfg, p, x, u0, want_resnorm=False, ws=None):
    """Implicit LSTM by MGRIT.  p: dict W_ih[4H,I], W_hh[4H,H], b_ih, b_hh; u0[2,B,H] = (c_0, h_0).
    -> (u[T,2,B,H], gi[T,B,4H], resnorm list or None)"""
    dev = x.device
    gi = torch.empty(cfg.T, cfg.B, 4 * cfg.H, device=dev)
    u = torch.empty(cfg.T, 2, cfg.B, cfg.H, device=dev)
    ws = _ws(lstm_workspace_bytes(cfg)[0], ws, dev)
    rn = (ctypes.c_float * max(cfg.iters, 1))() if want_resnorm else None
    _check(lib.mgrit_lstm_forward(ctypes.byref(cfg), ctypes.byref(_params(p)), _f32(x), _f32(u0), _f32(gi), _f32(u), rn, _ptr(ws),
                                  ws.numel(), _stream()))
    return u, gi, (list(rn)[:cfg.iters] if want_resnorm else None)


def mgrit_lstm_adjoint(cfg, p, x, u0, gi, u, du_seed=None, dhT=None, want_dx=True, want_du=True, want_resnorm=False, ws=None):
    """-> (du[T,2,B,H] or None, du0[2,B,H], AdjointResult with dx and the 4H-row gradients, resnorm)"""
    dev = x.device
    du = torch.empty(cfg.T, 2, cfg.B, cfg.H, device=dev) if want_du else None
    du0 = torch.empty(2, cfg.B, cfg.H, device=dev)
    o = AdjointResult(dh=None, dh0=None, dx=torch.empty(cfg.T, cfg.B, cfg.I, device=dev) if want_dx else None,
                      dW_ih=torch.empty(4 * cfg.H, cfg.I, device=dev), dW_hh=torch.empty(4 * cfg.H, cfg.H, device=dev),
                      db_ih=torch.empty(4 * cfg.H, device=dev), db_hh=torch.empty(4 * cfg.H, device=dev))
    g = _Grads(o.dW_ih.data_ptr(), o.dW_hh.data_ptr(), o.db_ih.data_ptr(), o.db_hh.data_ptr())
    ws = _ws(lstm_workspace_bytes(cfg)[1], ws, dev)
    rn = (ctypes.c_float * max(cfg.iters, 1))() if want_resnorm else None
    _check(lib.mgrit_lstm_adjoint(ctypes.byref(cfg), ctypes.byref(_params(p)), _f32(x), _f32(u0), _f32(gi), _f32(u), _f32(du_seed),
                                  _f32(dhT), _f32(du), _f32(du0), _f32(o.dx), ctypes.byref(g), rn, _ptr(ws), ws.numel(), _stream()))
    return du, du0, o, (list(rn)[:cfg.iters] if want_resnorm else None)


def xent_head_fwd_bwd(hT, Wc, bc, labels, ws=None):
    """-> (loss[1], dhT[B,H], dWc[C,H], dbc[C]) device tensors"""
    B, H = hT.shape
    C = Wc.shape[0]
    dev = hT.device
    assert labels.dtype == torch.int32
    loss = torch.empty(1, device=dev)
    dhT, dWc, dbc = torch.empty(B, H, device=dev), torch.empty(C, H, device=dev), torch.empty(C, device=dev)
    ws = _ws(lib.xent_head_workspace_bytes(B, C), ws, dev)
    _check(lib.xent_head_fwd_bwd(B, H, C, _f32(hT), _f32(Wc), _f32(bc), _ptr(labels), _f32(loss), _f32(dhT), _f32(dWc),
                                 _f32(dbc), _ptr(ws), ws.numel(), _stream()))
    return loss, dhT, dWc, dbc


def xent_head_fwd_bwd_noalloc(hT, Wc, bc, labels, out=None):
    """Loss head for callers that must not allocate device memory inside the call: the library's built-in
    scratch replaces the workspace (B*C <= 65536).  `out` = (loss[1], dhT[B,H], dWc[C,H], dbc[C]) preallocated
    by the caller; when omitted this convenience wrapper allocates the four outputs with torch before the call.
    Calls share one scratch array: do not overlap them on the GPU."""
    B, H = hT.shape
    C = Wc.shape[0]
    dev = hT.device
    assert labels.dtype == torch.int32
    if out is None:
        out = (torch.empty(1, device=dev), torch.empty(B, H, device=dev), torch.empty(C, H, device=dev), torch.empty(C, device=dev))
    loss, dhT, dWc, dbc = out
    _check(lib.xent_head_fwd_bwd_noalloc(B, H, C, _f32(hT), _f32(Wc), _f32(bc), _ptr(labels), _f32(loss), _f32(dhT), _f32(dWc),
                                         _f32(dbc), _stream()))
    return loss, dhT, dWc, dbc


def sgd_update(p, g, lr):
    _check(lib.sgd_update(_f32(p), _f32(g), p.numel(), ctypes.c_float(lr), _stream()))
    return p


def adam_update(p, g, m, v, lr, step, beta1=0.9, beta2=0.999, eps=1e-8):
    _check(lib.adam_update(_f32(p), _f32(g), _f32(m), _f32(v), p.numel(), ctypes.c_float(lr), ctypes.c_float(beta1),
                           ctypes.c_float(beta2), ctypes.c_float(eps), int(step), _stream()))
    return p


def last_device_status() -> int:
    return lib.mgrit_gru_last_device_status()


def clear_device_status() -> None:
    _check(lib.mgrit_gru_clear_device_status())


def selftest_bounded_wait(limit_ms: int = 20) -> None:
    """Launch the library's wait self-test: a bounded wait that runs out and records MGRIT_DEVICE_TIMEOUT."""
    _check(lib.mgrit_gru_selftest_bounded_wait(limit_ms, _stream()))


def kernel_launches() -> int:
    return int(lib.mgrit_gru_kernel_launches())


KERNEL_CLASSES = ("input_projection", "forward_step", "adjoint_linearise", "adjoint_step", "gradient_gemms",
                  "forward_serial_chain", "adjoint_serial_chain")


def profile_enable(on: bool) -> None:
    _check(lib.mgrit_gru_profile_enable(1 if on else 0))


def profile_records():
    """-> list of (class name, ms, flops) per recorded launch, in launch order."""
    n = _sz(0)
    _check(lib.mgrit_gru_profile_records(None, None, None, 0, ctypes.byref(n)))
    cap = n.value
    ms, fl, kc = (ctypes.c_double * cap)(), (ctypes.c_double * cap)(), (ctypes.c_int32 * cap)()
    _check(lib.mgrit_gru_profile_records(ms, fl, kc, cap, ctypes.byref(n)))
    return [(KERNEL_CLASSES[kc[i]], ms[i], fl[i]) for i in range(cap)]


def profile_read():
    """-> {class name: (total ms, launches, algorithmic flops)} for the launches recorded since profile_enable(True)."""
    out = {}
    for i, name in enumerate(KERNEL_CLASSES):
        ms, n, fl = ctypes.c_double(0), ctypes.c_ulonglong(0), ctypes.c_double(0)
        _check(lib.mgrit_gru_profile_read(i, ctypes.byref(ms), ctypes.byref(n), ctypes.byref(fl)))
        out[name] = (ms.value, int(n.value), fl.value)
    return out
