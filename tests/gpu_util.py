"""Shared helpers of the GPU parity tests."""
import numpy as np
import torch

from oracle import snlp_oracle as O
from paper_2605_17842_b200 import synth


def make_model(cfg, W, max_rows, max_batch=1, max_ctx=None):
    from paper_2605_17842_b200 import snlp
    m = snlp.Model(cfg, max_rows=max_rows, max_batch=max_batch, max_ctx=max_ctx)
    m.load_weights(W)
    return m


def layer_relerr(got, want):
    """max over layers of ||got[l] - want[l]||_2 / ||want[l]||_2 (the tolerance metric)."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    worst = 0.0
    for l in range(want.shape[0]):
        den = np.linalg.norm(want[l])
        worst = max(worst, np.linalg.norm(got[l] - want[l]) / max(den, 1e-300))
    return worst


def dev(x, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(x))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


TOL = {"fp32": 1e-4, "bf16": 2e-2}
