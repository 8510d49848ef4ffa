"""Helpers of the GPU parity tests: upload seeded inputs, run the oracle on the same fp32-rounded values."""
import numpy as np
import torch

from oracle import mgrit_gru_oracle as O
from paper_2203_04738_b200.synthetic import make_inputs

NAMES = ("W_ih", "W_hh", "b_ih", "b_hh")


def to_dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def upload(d, layer=0):
    p = {n: to_dev(d["layers"][layer][n]) for n in NAMES}
    return p, to_dev(d["x"]), to_dev(d["h0"])


def oracle_params(d, layer=0):
    return [d["layers"][layer][n].astype(np.float64) for n in NAMES]


def max_abs(a, b):
    return float(np.max(np.abs(np.asarray(a, dtype=np.float64) - np.asarray(b, dtype=np.float64))))


def rel_inf(a, b):
    """||a - b||_inf / ||b||_inf : the gradient metric (norm-wise, never element-relative)."""
    b = np.asarray(b, dtype=np.float64)
    den = float(np.max(np.abs(b)))
    return max_abs(a, b) / (den if den > 0 else 1.0)
