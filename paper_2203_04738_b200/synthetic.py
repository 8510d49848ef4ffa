"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA path.

This module holds no arithmetic of the method: it only draws parameters and sequences.
The sequences stand in for per-frame CNN feature sequences of video clips (non-negative,
about half zeros, unstructured), which the paper's experiments feed to the GRU.

Draw order (NumPy PCG64, float64, rounded once to float32): per layer W_ih[3H,I_l],
W_hh[3H,H], b_ih[3H], b_hh[3H] ~ U(-k,k), k = 1/sqrt(H) -- layer 0 first, then x[T,B,I]
~ N(0,1) (ReLU'd when `relu`), then the further layers' parameters, then W_c[C,H], b_c[C]
~ U(-k,k) and labels[B] uniform over C classes.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np


@dataclass(frozen=True)
class Workload:
    name: str
    T: int
    B: int
    I: int
    H: int
    cf: int
    levels: int
    iters_fwd: int
    iters_adj: int
    relax_fine: int          # 0 = F, 1 = FCF
    relax_coarse: int
    operands: int            # 0 = fp32 FFMA, 1 = tf32 three-term split, 2 = bf16, 3 = tf32 single pass (tensor-core operands)
    classes: int
    relu: bool
    layers: int = 1
    seed: int = 0
    cell: int = 1            # implicit GRU on every level


# The five configurations of the benchmark spec.  Index = position in that list.
WORKLOADS = {
    "tiny": Workload("tiny", T=64, B=2, I=16, H=32, cf=4, levels=2, iters_fwd=2, iters_adj=2,
                     relax_fine=0, relax_coarse=1, operands=0, classes=8, relu=False, seed=0),
    # fp32 state at fp32 tolerances; the products run on the tensor cores as three-term tf32 splits (operands = 1)
    "clip": Workload("clip", T=128, B=16, I=512, H=256, cf=4, levels=2, iters_fwd=2, iters_adj=2,
                     relax_fine=1, relax_coarse=1, operands=1, classes=51, relu=True, seed=1),
    "medium": Workload("medium", T=1024, B=32, I=1024, H=512, cf=4, levels=3, iters_fwd=2, iters_adj=2,
                       relax_fine=0, relax_coarse=1, operands=2, classes=51, relu=True, seed=2),
    "long": Workload("long", T=4096, B=8, I=2048, H=1024, cf=8, levels=4, iters_fwd=3, iters_adj=3,
                     relax_fine=0, relax_coarse=1, operands=2, classes=51, relu=True, seed=3),
    "train": Workload("train", T=2048, B=32, I=2048, H=1024, cf=4, levels=3, iters_fwd=2, iters_adj=2,
                      relax_fine=0, relax_coarse=1, operands=2, classes=51, relu=True, layers=2, seed=4),
}


def _uniform(rng, shape, k):
    return rng.uniform(-k, k, size=shape)


def make_inputs(w: Workload, T: int | None = None, B: int | None = None, dtype=np.float32):
    """Returns a dict of float32 arrays: layers (list of dicts W_ih, W_hh, b_ih, b_hh), x, h0,
    W_c, b_c, labels(int32).  T / B override the workload's (for sweeps and CPU samples)."""
    T = w.T if T is None else T
    B = w.B if B is None else B
    rng = np.random.default_rng(w.seed)
    k = 1.0 / np.sqrt(w.H)

    def layer(I):
        return {
            "W_ih": _uniform(rng, (3 * w.H, I), k),
            "W_hh": _uniform(rng, (3 * w.H, w.H), k),
            "b_ih": _uniform(rng, (3 * w.H,), k),
            "b_hh": _uniform(rng, (3 * w.H,), k),
        }

    layers = [layer(w.I)]
    x = rng.standard_normal((T, B, w.I))
    if w.relu:
        x = np.maximum(x, 0.0)
    for _ in range(1, w.layers):
        layers.append(layer(w.H))
    W_c = _uniform(rng, (w.classes, w.H), k)
    b_c = _uniform(rng, (w.classes,), k)
    labels = rng.integers(0, w.classes, size=(B,)).astype(np.int32)
    cast = lambda a: np.ascontiguousarray(a.astype(dtype))
    return {
        "layers": [{n: cast(v) for n, v in lay.items()} for lay in layers],
        "x": cast(x),
        "h0": np.zeros((B, w.H), dtype=dtype),
        "W_c": cast(W_c),
        "b_c": cast(b_c),
        "labels": labels,
    }
