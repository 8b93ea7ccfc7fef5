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


def row_relerr(got, want):
    """max over layers and rows of the relative L2 error of one row's state (its n streams x d features)."""
    want = np.asarray(want, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64).reshape(want.shape)
    L1 = want.shape[0]
    nd = want.shape[-2] * want.shape[-1]
    w = want.reshape(L1, -1, nd)
    g = got.reshape(L1, -1, nd)
    den = np.maximum(np.linalg.norm(w, axis=-1), 1e-300)
    return float(np.max(np.linalg.norm(g - w, axis=-1) / den))


def trace_err(got, want, tol):
    """The tolerance metric (per-layer relative L2 <= tol) with a per-row guard beside it: at thousands of rows a
    wholly wrong row, or a wrong run of columns in one row, hardly moves a layer's norm, so every single row must
    also be within 5 x tol of the oracle's.  Returns the layer error; raises if a row is off."""
    rows = row_relerr(got, want)
    assert rows <= 5.0 * tol, f"worst single row off by {rows:.3e} (limit {5.0 * tol:.1e})"
    return layer_relerr(got, want)


def dev(x, dtype=None):
    t = torch.from_numpy(np.ascontiguousarray(x))
    if dtype is not None:
        t = t.to(dtype)
    return t.cuda()


TOL = {"fp32": 1e-4, "bf16": 2e-2}
