"""One training step of a stacked GRU whose layers are each solved by MGRIT: a fixed sequence
of C-ABI calls (no arithmetic here).  Layer l+1 reads layer l's (inexact) hidden states; in the
backward direction layer l+1's input gradient is layer l's direct loss derivative dh_seed."""
from __future__ import annotations

from dataclasses import dataclass, field

import torch

from . import binding as B
from .synthetic import Workload


@dataclass
class StepBuffers:
    """Device buffers reused across steps (allocated once; the library itself never allocates)."""
    cfgs_fwd: list
    cfgs_adj: list
    ws_fwd: torch.Tensor
    ws_adj: torch.Tensor
    ws_head: torch.Tensor
    gi: list
    h: list            # h[l]: [T,B,H] view of slots 1..T of h_full[l]
    adj: list
    serial: bool = False
    h_full: list = None    # h_full[l]: [T+1,B,H], slot 0 = h_0 (written by the forward call: MGRIT_FLAG_H_LEADS_WITH_H0)


def make_cfgs(w: Workload, T: int, Bsz: int, serial: bool = False, flags: int = 0):
    fw, ad = [], []
    for l in range(w.layers):
        I = w.I if l == 0 else w.H
        kw = dict(cf=w.cf, levels=1 if serial else w.levels, cell=w.cell, relax_fine=w.relax_fine,
                  relax_coarse=w.relax_coarse, operands=w.operands, flags=flags | B.FLAG_GI_CARRIES_COPIES | B.FLAG_GI_F32_UNUSED)      # (nothing here reads the fp32 projection)
        # the forward calls write the level-0 unknowns straight into the buffers' state arrays (one leading slot for h_0)
        fw.append(B.make_cfg(T, Bsz, I, w.H, iters=w.iters_fwd, **dict(kw, flags=kw["flags"] | B.FLAG_H_LEADS_WITH_H0)))
        ad.append(B.make_cfg(T, Bsz, I, w.H, iters=w.iters_adj, **kw))
    return fw, ad


def alloc_buffers(w: Workload, T: int, Bsz: int, device, serial: bool = False, flags: int = 0, want_dh: bool = False) -> StepBuffers:
    fw, ad = make_cfgs(w, T, Bsz, serial, flags)
    nf = max(B.workspace_bytes(c)[0] for c in fw)
    na = max(B.workspace_bytes(c)[1] for c in ad)
    mk = lambda *s: torch.empty(*s, device=device)
    adj = []
    for l, c in enumerate(ad):
        # dh (dL/dh_t for every t) is not an input of anything in a training step: only written when asked for
        adj.append(B.AdjointResult(dh=mk(T, Bsz, w.H) if want_dh else None, dh0=mk(Bsz, w.H), dx=mk(T, Bsz, c.I) if l > 0 else None,
                                   dW_ih=mk(3 * w.H, c.I), dW_hh=mk(3 * w.H, w.H), db_ih=mk(3 * w.H), db_hh=mk(3 * w.H)))
    h_full = [mk(T + 1, Bsz, w.H) for _ in fw]
    return StepBuffers(fw, ad, torch.empty(nf, dtype=torch.uint8, device=device), torch.empty(na, dtype=torch.uint8, device=device),
                       torch.empty(B.lib.xent_head_workspace_bytes(Bsz, w.classes), dtype=torch.uint8, device=device),
                       [B.alloc_gi(c, device) for c in fw], [t[1:] for t in h_full], adj, serial, h_full)


class HostInputPipeline:
    """Double-buffered staging of each step's input from pinned host memory.

    The copy of step k+1's input runs on a side stream while step k computes, so an end-to-end step costs
    max(copy, compute) instead of their sum.  Usage per step: ``x = acquire()`` (the compute stream waits
    for that buffer's copy), optionally ``submit(next_host_input)``, run the step on ``x``, ``release()``.
    No arithmetic here: two device buffers, one stream, four events."""

    def __init__(self, shape, dtype, device):
        self.bufs = [torch.empty(shape, dtype=dtype, device=device) for _ in range(2)]
        self.stream = torch.cuda.Stream(device=device)
        self.ready = [torch.cuda.Event() for _ in range(2)]
        self.free = [None, None]
        self.n_sub = 0
        self.n_acq = 0

    def submit(self, x_host: torch.Tensor) -> None:
        i = self.n_sub % 2
        self.n_sub += 1
        if self.free[i] is not None:
            self.stream.wait_event(self.free[i])      # the step that read this buffer has finished
        with torch.cuda.stream(self.stream):
            self.bufs[i].copy_(x_host, non_blocking=True)
            self.ready[i].record(self.stream)

    def acquire(self) -> torch.Tensor:
        if self.n_acq >= self.n_sub:
            raise RuntimeError("HostInputPipeline.acquire() without a submitted input")
        i = self.n_acq % 2
        torch.cuda.current_stream().wait_event(self.ready[i])
        return self.bufs[i]

    def release(self) -> None:
        i = self.n_acq % 2
        self.n_acq += 1
        ev = torch.cuda.Event()
        ev.record(torch.cuda.current_stream())
        self.free[i] = ev


class AdamState:
    """Moment buffers of the Adam optimiser (the optimiser of the paper's experiments), one pair per parameter."""

    def __init__(self, params):
        self.m = [torch.zeros_like(p) for p in params]
        self.v = [torch.zeros_like(p) for p in params]
        self.step = 0


def all_params(layers, W_c, b_c):
    out = []
    for p in layers:
        out += [p["W_ih"], p["W_hh"], p["b_ih"], p["b_hh"]]
    return out + [W_c, b_c]


def forward_pass(layers, x, h0, buf: StepBuffers):
    """Input projection + forward solve of every layer (MGRIT, or the serial sweep when the buffers say so); returns
    the top layer's states (device, owned by buf)."""
    inp = x
    for l, p in enumerate(layers):
        fn = B.gru_serial_forward if buf.serial else B.mgrit_gru_forward
        fn(buf.cfgs_fwd[l], p, inp, h0, gi=buf.gi[l], h=buf.h_full[l], ws=buf.ws_fwd)
        inp = buf.h[l]
    return inp


def training_step(w: Workload, layers, W_c, b_c, x, h0, labels, buf: StepBuffers, lr: float = 1e-3, update: bool = True,
                  adam: AdamState | None = None):
    """Forward (all layers) -> loss head -> adjoint (top layer first) -> weight gradients -> SGD (or Adam when an
    AdamState is given).  layers: list of dicts W_ih, W_hh, b_ih, b_hh (device fp32).  Returns the loss (device)."""
    forward_pass(layers, x, h0, buf)
    loss, dhT, dWc, dbc = B.xent_head_fwd_bwd(buf.h[-1][-1], W_c, b_c, labels, ws=buf.ws_head)
    seed = None
    for l in range(len(layers) - 1, -1, -1):
        inp = x if l == 0 else buf.h[l - 1]
        fn = B.gru_serial_backward if buf.serial else B.mgrit_gru_adjoint
        # (h_0 as the forward call left it in slot 0 of the state array: contiguous with h, one linearisation launch per level)
        fn(buf.cfgs_adj[l], layers[l], inp, buf.h_full[l][0], buf.gi[l], buf.h[l], dh_seed=seed, dhT=dhT if seed is None else None,
           want_dx=l > 0, ws=buf.ws_adj, out=buf.adj[l])
        seed = buf.adj[l].dx
    if update and adam is not None:
        grads = []
        for l in range(len(layers)):
            a = buf.adj[l]
            grads += [a.dW_ih, a.dW_hh, a.db_ih, a.db_hh]
        grads += [dWc, dbc]
        adam.step += 1
        for p_, g_, m_, v_ in zip(all_params(layers, W_c, b_c), grads, adam.m, adam.v):
            B.adam_update(p_, g_, m_, v_, lr, adam.step)
    elif update:
        for l, p in enumerate(layers):
            a = buf.adj[l]
            for name, g in (("W_ih", a.dW_ih), ("W_hh", a.dW_hh), ("b_ih", a.db_ih), ("b_hh", a.db_hh)):
                B.sgd_update(p[name], g, lr)
        B.sgd_update(W_c, dWc, lr)
        B.sgd_update(b_c, dbc, lr)
    return loss


class GraphedTrainingStep:
    """One training step captured once into a CUDA graph and replayed: the step is a fixed sequence of a few hundred
    dependent launches (cooperative chain launches and programmatic dependent launches included), so replaying it
    removes the per-launch CPU work and shortens the gaps between launches.  All pointers are baked in: the
    tensors passed here must stay alive and keep their addresses; new data is copied INTO them.  ``launches`` is
    the number of library kernels one replay runs."""

    def __init__(self, w: Workload, layers, W_c, b_c, x, h0, labels, buf: StepBuffers, step_fn=None, **kw):
        args = (w, layers, W_c, b_c, x, h0, labels, buf)
        fn = (lambda: training_step(*args, **kw)) if step_fn is None else step_fn     # step_fn: any fixed sequence of library calls
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):               # first use of every kernel outside the capture (attribute set-up)
            fn()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        n0 = B.kernel_launches()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            self.loss = fn()
        self.launches = B.kernel_launches() - n0
        self._keep = args

    def __call__(self):
        self.graph.replay()
        return self.loss



def stacked_training_step(w: Workload, layers, W_c, b_c, x, h0s, labels, ws_fwd=None, ws_adj=None, ws_head=None, lr: float = 1e-3,
                          update: bool = True, flags: int = 0):
    """The same training step with ALL layers in one time-step state and ONE MGRIT cycle for the stack
    (mgrit_gru_stack_forward / mgrit_gru_stack_adjoint): forward -> loss head on the top layer's last state -> adjoint ->
    per-layer gradients -> SGD.  h0s[n_layers,B,H].  Returns (loss, forward residual norms or None)."""
    T, Bsz = x.shape[0], x.shape[1]
    kw = dict(cf=w.cf, levels=w.levels, cell=w.cell, relax_fine=w.relax_fine, relax_coarse=w.relax_coarse, operands=w.operands, flags=flags)
    cf_ = B.make_cfg(T, Bsz, w.I, w.H, iters=w.iters_fwd, **kw)
    ca_ = B.make_cfg(T, Bsz, w.I, w.H, iters=w.iters_adj, **kw)
    h, gi0, _ = B.mgrit_gru_stack_forward(cf_, layers, x, h0s, ws=ws_fwd)
    loss, dhT, dWc, dbc = B.xent_head_fwd_bwd(h[-1, -1], W_c, b_c, labels, ws=ws_head)
    _, _, _, grads, _ = B.mgrit_gru_stack_adjoint(ca_, layers, x, h0s, gi0, h, dhT=dhT, want_dx=False, want_dh=False, ws=ws_adj)
    if update:
        for p, g in zip(layers, grads):
            for name, gg in (("W_ih", g.dW_ih), ("W_hh", g.dW_hh), ("b_ih", g.db_ih), ("b_hh", g.db_hh)):
                B.sgd_update(p[name], gg, lr)
        B.sgd_update(W_c, dWc, lr)
        B.sgd_update(b_c, dbc, lr)
    return loss
