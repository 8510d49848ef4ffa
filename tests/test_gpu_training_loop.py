"""Training with MGRIT as in Algorithm "MGRITTraining" with the paper's settings (2 forward cycles, 1 backward
cycle, Adam): (1) the loss trajectory of the CUDA path equals the fp64 oracle's running the same algorithm,
(2) on a learnable synthetic task the loss falls as it does with exact serial propagation, and the trained
network gives the same predictions whether it is evaluated serially or in parallel (the paper's remark on
serial vs. parallel inference)."""
import numpy as np
import pytest
import torch

from oracle import mgrit_gru_oracle as O
from paper_2203_04738_b200.synthetic import Workload, make_inputs
from tests.gpu_util import NAMES, to_dev

pytestmark = pytest.mark.gpu


def _oracle_training(w, d, steps, lr):
    f64 = lambda a: a.astype(np.float64)
    P = [f64(d["layers"][0][n]) for n in NAMES]
    Wc, bc = f64(d["W_c"]), f64(d["b_c"])
    x, h0, lab = f64(d["x"]), f64(d["h0"]), d["labels"]
    params = P + [Wc, bc]
    m = [np.zeros_like(p) for p in params]
    v = [np.zeros_like(p) for p in params]
    kw = dict(cf=w.cf, levels=w.levels, relax_fine=w.relax_fine, relax_coarse=w.relax_coarse)
    losses = []
    for step in range(1, steps + 1):
        h, _ = O.mgrit_forward(*params[:4], x, h0, iters=w.iters_fwd, **kw)
        loss, dhT, dWc, dbc = O.xent_head(h[-1], params[4], params[5], lab)
        seed = np.zeros_like(h)
        seed[-1] = dhT
        _, _, g, _ = O.mgrit_adjoint(*params[:4], x, h0, h, seed, iters=w.iters_adj, want_dx=False, **kw)
        grads = [g["dW_ih"], g["dW_hh"], g["db_ih"], g["db_hh"], dWc, dbc]
        for i in range(6):
            params[i], m[i], v[i] = O.adam_update(params[i], grads[i], m[i], v[i], lr, step)
        losses.append(loss)
    return losses


def test_adam_update_matches_oracle():
    from paper_2203_04738_b200 import binding as B
    rng = np.random.default_rng(2)
    n = 4099
    p = rng.standard_normal(n).astype(np.float32); m = np.zeros(n); v = np.zeros(n)
    pd, md, vd = to_dev(p), torch.zeros(n, device="cuda"), torch.zeros(n, device="cuda")
    pr = p.astype(np.float64)
    for step in range(1, 5):
        g = rng.standard_normal(n).astype(np.float32)
        B.adam_update(pd, to_dev(g), md, vd, 1e-3, step)
        pr, m, v = O.adam_update(pr, g.astype(np.float64), m, v, 1e-3, step)
        assert np.max(np.abs(pd.cpu().numpy() - pr)) < 1e-5


def test_loss_trajectory_matches_oracle():
    from paper_2203_04738_b200 import binding as B
    from paper_2203_04738_b200.train_step import AdamState, all_params, alloc_buffers, training_step
    w = Workload("tl", T=64, B=4, I=16, H=32, cf=4, levels=3, iters_fwd=2, iters_adj=1, relax_fine=0, relax_coarse=1,
                 operands=0, classes=8, relu=False, seed=11)
    d = make_inputs(w)
    layers = [{n: to_dev(d["layers"][0][n]) for n in NAMES}]
    W_c, b_c, labels, h0, x = to_dev(d["W_c"]), to_dev(d["b_c"]), to_dev(d["labels"]), to_dev(d["h0"]), to_dev(d["x"])
    buf = alloc_buffers(w, w.T, w.B, torch.device("cuda"))
    adam = AdamState(all_params(layers, W_c, b_c))
    lr, steps = 1e-2, 6
    got = [training_step(w, layers, W_c, b_c, x, h0, labels, buf, lr=lr, adam=adam).item() for _ in range(steps)]
    want = _oracle_training(w, d, steps, lr)
    assert want[-1] < want[0]
    for a, b in zip(got, want):
        assert abs(a - b) < 1e-4 * max(1.0, abs(b)), (got, want)


def _task_batch(rng, T, Bn, I, C):
    """Learnable synthetic sequence classification: the class is the input channel (among the first C) with the
    largest mean over the second half of the sequence."""
    x = rng.standard_normal((T, Bn, I)).astype(np.float32)
    lab = rng.integers(0, C, Bn)
    x[T // 2:, np.arange(Bn), lab] += 1.0
    return x, lab.astype(np.int32)


def test_training_with_mgrit_learns_like_serial_and_inference_agrees():
    from paper_2203_04738_b200 import binding as B
    from paper_2203_04738_b200.train_step import AdamState, all_params, alloc_buffers, training_step
    T, Bn, I, H, C = 64, 32, 16, 64, 4
    w = Workload("task", T=T, B=Bn, I=I, H=H, cf=4, levels=3, iters_fwd=2, iters_adj=1, relax_fine=0, relax_coarse=1,
                 operands=2, classes=C, relu=False, seed=12)
    dev = torch.device("cuda")
    finals, nets = {}, {}
    for mode in ("mgrit", "serial"):
        d = make_inputs(w)
        layers = [{n: to_dev(d["layers"][0][n]) for n in NAMES}]
        W_c, b_c, h0 = to_dev(d["W_c"]), to_dev(d["b_c"]), to_dev(d["h0"])
        buf = alloc_buffers(w, T, Bn, dev, serial=(mode == "serial"))
        adam = AdamState(all_params(layers, W_c, b_c))
        rng = np.random.default_rng(100)
        losses = []
        for _ in range(200):
            x, lab = _task_batch(rng, T, Bn, I, C)
            losses.append(training_step(w, layers, W_c, b_c, to_dev(x), h0, to_dev(lab), buf, lr=5e-3, adam=adam).item())
        finals[mode] = (np.mean(losses[:10]), np.mean(losses[-20:]))
        nets[mode] = (layers, W_c, b_c, h0)
    for mode, (first, last) in finals.items():
        assert last < 0.6 * first, (mode, first, last)
    assert abs(finals["mgrit"][1] - finals["serial"][1]) < 0.35 * finals["serial"][0], finals
    # serial vs parallel inference of the MGRIT-trained network on held-out data
    layers, W_c, b_c, h0 = nets["mgrit"]
    rng = np.random.default_rng(999)
    agree = correct = total = 0
    cfg = B.make_cfg(T, Bn, I, H, cf=4, levels=3, iters=2, operands=B.OPERANDS_BF16)
    for _ in range(8):
        x, lab = _task_batch(rng, T, Bn, I, C)
        xd = to_dev(x)
        hp, _, _ = B.mgrit_gru_forward(cfg, layers[0], xd, h0)
        hs, _ = B.gru_serial_forward(cfg, layers[0], xd, h0)
        pp = (hp[-1] @ W_c.T + b_c).argmax(1).cpu().numpy()
        ps = (hs[-1] @ W_c.T + b_c).argmax(1).cpu().numpy()
        agree += int((pp == ps).sum()); correct += int((ps == lab).sum()); total += Bn
    assert agree >= 0.9 * total, (agree, total)
    assert correct >= 0.5 * total, (correct, total)       # chance is 0.25
    assert B.last_device_status() == 0


def test_host_input_pipeline_feeds_the_right_inputs():
    """Three steps with three DIFFERENT host inputs through the double-buffered pipeline give the same losses
    as the same steps run on plainly copied inputs (no update, so the steps are independent)."""
    from paper_2203_04738_b200.train_step import HostInputPipeline, alloc_buffers, training_step
    w = Workload("hp", T=64, B=4, I=16, H=32, cf=4, levels=3, iters_fwd=2, iters_adj=1, relax_fine=0, relax_coarse=1,
                 operands=0, classes=8, relu=False, seed=5)
    d = make_inputs(w)
    layers = [{n: to_dev(d["layers"][0][n]) for n in NAMES}]
    W_c, b_c, h0, labels = to_dev(d["W_c"]), to_dev(d["b_c"]), to_dev(d["h0"]), to_dev(d["labels"])
    buf = alloc_buffers(w, w.T, w.B, torch.device("cuda"))
    rng = np.random.default_rng(9)
    hosts = [torch.from_numpy(rng.standard_normal(d["x"].shape).astype(np.float32)).pin_memory() for _ in range(3)]
    want = [float(training_step(w, layers, W_c, b_c, xh.cuda(), h0, labels, buf, update=False)) for xh in hosts]
    pipe = HostInputPipeline(hosts[0].shape, hosts[0].dtype, torch.device("cuda"))
    got = []
    pipe.submit(hosts[0])
    for k in range(3):
        xk = pipe.acquire()
        if k + 1 < 3:
            pipe.submit(hosts[k + 1])
        loss = training_step(w, layers, W_c, b_c, xk, h0, labels, buf, update=False)
        pipe.release()
        got.append(float(loss))
    # the loss is a sum over batch rows accumulated with atomics, so equal inputs agree to rounding, not bitwise
    assert np.max(np.abs(np.array(got) - np.array(want))) < 1e-5
    assert min(abs(want[0] - want[1]), abs(want[1] - want[2]), abs(want[0] - want[2])) > 5e-5


def test_graph_replay_equals_host_launches():
    """The captured step replays the same kernels on the same buffers: with the update switched off two replays and
    a host-launched step give the same loss (to the rounding of the loss's atomic batch sum) and the same gradients."""
    from paper_2203_04738_b200.train_step import GraphedTrainingStep, alloc_buffers, training_step
    w = Workload("gr", T=64, B=8, I=128, H=128, cf=4, levels=3, iters_fwd=2, iters_adj=2, relax_fine=0, relax_coarse=1,
                 operands=2, classes=8, relu=True, seed=21)
    d = make_inputs(w)
    layers = [{n: to_dev(d["layers"][0][n]) for n in NAMES}]
    W_c, b_c, h0, labels, x = to_dev(d["W_c"]), to_dev(d["b_c"]), to_dev(d["h0"]), to_dev(d["labels"]), to_dev(d["x"])
    buf = alloc_buffers(w, w.T, w.B, torch.device("cuda"))
    want = float(training_step(w, layers, W_c, b_c, x, h0, labels, buf, update=False))
    g_want = buf.adj[0].dW_hh.clone()
    g = GraphedTrainingStep(w, layers, W_c, b_c, x, h0, labels, buf, update=False)
    assert g.launches > 50
    for _ in range(2):
        buf.adj[0].dW_hh.zero_()
        got = float(g())
        assert abs(got - want) < 1e-5
        assert torch.equal(buf.adj[0].dW_hh, g_want)
    # new data goes INTO the captured input tensor
    x.mul_(0.5)
    got = float(g())
    ref = float(training_step(w, layers, W_c, b_c, x, h0, labels, buf, update=False))
    assert abs(got - ref) < 1e-5 and abs(got - want) > 1e-4
