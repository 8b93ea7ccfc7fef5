"""Plain CPU oracle for SNLP (Structured Newton Layer Parallelism).

TEST INFRASTRUCTURE ONLY.  This module is the slow, obviously-correct statement of
what the CUDA library computes.  It is written with numpy in fp64 (``dtype`` may be
set to ``np.float32`` for the timed CPU baseline), shares no code with the CUDA path
and imports nothing from the product package.  Only the tests, the smoke check and
the benchmark's CPU-baseline leg may call it; the product never does.

Index convention (0-based): hidden states ``h_0 .. h_L``; block ``l`` (0 <= l < L)
maps ``h_l -> h_{l+1} = F_l(h_l)``.  The paper numbers states the same way but its
layer maps from 1 (``h_l = f_l(h_{l-1})``, Sec. 3.1); ``F_l`` here is its ``f_{l+1}``.

What follows the paper literally:
  * ``forward_sequential``      -- Algorithm 1.
  * ``forward_snlp``            -- Algorithm 2 with prefix length S = 0 and ``h0``
                                   initialisation; the correction line is Eq. (5)
                                   (the SNLP update) with A = I (IDN, Eqs. 6-7),
                                   A = H_res_mlp @ H_res_attn (HCN, Eq. 8) or A = 0
                                   (naive fixed point, Sec. 3.2 "Effect of the
                                   correction"), written exactly as
                                   ``h~ + A (h_new_prev - h_old_prev)``.
  * ``residual_norms``          -- Eq. (2), G_l(h) = h_l - f_l(h_{l-1}).
  * ``mhc_block``               -- the two mHC sub-layer equations of App. C.2.
  * ``ssd_ideal_speedup``       -- the self-speculative-decoding estimate of Sec. 5.1.

  * ``fused_chunk`` / ``forward_chunked`` -- fused cross-layer chunks of App. C.3 and the chunkwise update,
                                   Eq. (11) (``snlp-iterative``), with the identity chunk surrogate.

What the paper leaves open and this file fixes by definition (parity unpinned for
these constants; they are definitions shared with the CUDA library, not checks):
  RMSNorm without weights, eps inside the square root; rotary pairs (i, i+hd/2) with
  angle pos * base^(-2i/hd), rotation by +angle; rotary before QK-norm; softmax scale
  1/sqrt(hd); no biases; ReLU^2 MLP; untied lm head; final RMSNorm before the head;
  mHC: branch input = RMSNorm(H_pre . x), entry replicates the embedding into all n
  streams, exit sums the streams; greedy argmax ties go to the lowest index.

Finite-K values of the SNLP iterate are "parity unpinned" by the paper (it prints no
worked example with weights); they are pinned by the invariants in tests/ (finite-step
exactness, K=1 closed form, prefix-sum identity, HCN->IDN reduction, zero-branch
identity, staircase without correction) and by a brute-force scalar implementation.
"""
from __future__ import annotations

import math
from types import SimpleNamespace

import numpy as np

MODE_IDN = 0
MODE_HCN = 1
MODE_NOCORR = 2


# --------------------------------------------------------------------------- #
# elementary pieces
# --------------------------------------------------------------------------- #
def rmsnorm(x, eps):
    """Weight-free RMSNorm over the last axis: x / sqrt(mean(x^2) + eps)."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x / np.sqrt(ms + eps)


def rotary(x, pos, base):
    """Rotary position embedding (RoFormer) on x[..., T, H, hd] at integer positions pos[T].

    Element i (< hd/2) is paired with element i + hd/2 and the pair is rotated by
    angle pos * base**(-2 i / hd).
    """
    hd = x.shape[-1]
    half = hd // 2
    i = np.arange(half, dtype=np.float64)
    inv_freq = base ** (-2.0 * i / hd)
    ang = np.asarray(pos, dtype=np.float64)[:, None] * inv_freq[None, :]  # [T, half]
    cos = np.cos(ang).astype(x.dtype)[:, None, :]
    sin = np.sin(ang).astype(x.dtype)[:, None, :]
    x1 = x[..., :half]
    x2 = x[..., half:]
    return np.concatenate([x1 * cos - x2 * sin, x1 * sin + x2 * cos], axis=-1)


def softmax_lastaxis(s):
    s = s - np.max(s, axis=-1, keepdims=True)
    e = np.exp(s)
    return e / np.sum(e, axis=-1, keepdims=True)


class LayerKV:
    """Per-layer key/value store of one model: k[l], v[l] have shape [B, ctx, H, hd]."""

    def __init__(self, n_layer, B, max_ctx, n_head, head_dim, dtype=np.float64):
        self.k = np.zeros((n_layer, B, max_ctx, n_head, head_dim), dtype=dtype)
        self.v = np.zeros((n_layer, B, max_ctx, n_head, head_dim), dtype=dtype)
        self.len = 0

    def copy(self):
        o = LayerKV.__new__(LayerKV)
        o.k = self.k.copy()
        o.v = self.v.copy()
        o.len = self.len
        return o


def attention_branch(cfg, W, l, xin, kv, pos0, dtype):
    """Attention branch of block l on its (un-normalised) input xin[B, T, d].

    Writes this call's keys/values into kv slots pos0 .. pos0+T-1 of layer l, then lets
    query t attend causally over slots 0 .. pos0+t of that same layer.
    Returns a[B, T, d] = Wo . Attn(...).
    """
    B, T, d = xin.shape
    H, hd = cfg.n_head, cfg.head_dim
    x = rmsnorm(xin, cfg.rms_eps)
    wqkv = W.wqkv[l].astype(dtype)
    q = (x @ wqkv[0:d].T).reshape(B, T, H, hd)
    k = (x @ wqkv[d:2 * d].T).reshape(B, T, H, hd)
    v = (x @ wqkv[2 * d:3 * d].T).reshape(B, T, H, hd)
    pos = np.arange(pos0, pos0 + T)
    q = rmsnorm(rotary(q, pos, cfg.rope_base), cfg.rms_eps)
    k = rmsnorm(rotary(k, pos, cfg.rope_base), cfg.rms_eps)
    kv.k[l, :, pos0:pos0 + T] = k
    kv.v[l, :, pos0:pos0 + T] = v
    Tk = pos0 + T
    kk = kv.k[l, :, :Tk]  # [B, Tk, H, hd]
    vv = kv.v[l, :, :Tk]
    s = np.einsum("bthe,bshe->bhts", q, kk) / math.sqrt(hd)
    key_pos = np.arange(Tk)[None, :]
    qry_pos = pos[:, None]
    s = np.where(key_pos <= qry_pos, s, -np.inf)
    p = softmax_lastaxis(s)
    o = np.einsum("bhts,bshe->bthe", p, vv).reshape(B, T, d)
    return o @ W.wo[l].astype(dtype).T


def mlp_branch(cfg, W, l, uin, dtype):
    """MLP branch of block l on its (un-normalised) input uin[B, T, d]: Wdn . relu(Wup . norm(u))^2."""
    y = rmsnorm(uin, cfg.rms_eps) @ W.wup[l].astype(dtype).T
    z = np.maximum(y, 0.0) ** 2
    return z @ W.wdn[l].astype(dtype).T


# --------------------------------------------------------------------------- #
# blocks
# --------------------------------------------------------------------------- #
def residual_block(cfg, W, l, h, kv, pos0, dtype):
    """Residual Transformer block F_l(h) = u + MLP(u), u = h + Attn(h)  (f(x) = x + g(x), App. C.1).

    h: [B, T, 1, d].  Returns (F_l(h), a, m) with a, m the two branch outputs [B, T, d].
    """
    x = h[:, :, 0, :]
    a = attention_branch(cfg, W, l, x, kv, pos0, dtype)
    u = x + a
    m = mlp_branch(cfg, W, l, u, dtype)
    return (u + m)[:, :, None, :], a, m


def mhc_block(cfg, W, l, x, kv, pos0, dtype):
    """mHC block on the stream tensor x[B, T, n, d] (App. C.2):

        x'      = Hres_attn x + Hpost_attn * Attn(Hpre_attn x)
        x_next  = Hres_mlp x' + Hpost_mlp  * MLP (Hpre_mlp  x')

    Hres: [n, n] acting on the stream axis; Hpre: [n] (a 1 x n row); Hpost: [n] (an n x 1 column).
    """
    Ra = W.hc_res_attn[l].astype(dtype)
    Rm = W.hc_res_mlp[l].astype(dtype)
    Pa = W.hc_pre_attn[l].astype(dtype)
    Pm = W.hc_pre_mlp[l].astype(dtype)
    Qa = W.hc_post_attn[l].astype(dtype)
    Qm = W.hc_post_mlp[l].astype(dtype)
    a = attention_branch(cfg, W, l, np.einsum("s,btsd->btd", Pa, x), kv, pos0, dtype)
    xp = np.einsum("rs,btsd->btrd", Ra, x) + Qa[None, None, :, None] * a[:, :, None, :]
    m = mlp_branch(cfg, W, l, np.einsum("s,btsd->btd", Pm, xp), dtype)
    xn = np.einsum("rs,btsd->btrd", Rm, xp) + Qm[None, None, :, None] * m[:, :, None, :]
    return xn, a, m


def block(cfg, W, l, h, kv, pos0, dtype):
    if cfg.n_streams == 1:
        return residual_block(cfg, W, l, h, kv, pos0, dtype)[0]
    return mhc_block(cfg, W, l, h, kv, pos0, dtype)[0]


def surrogate(cfg, W, l, mode, dtype):
    """The n x n surrogate A_l of Eq. (5): I (IDN), Hres_mlp Hres_attn (HCN, Eq. 8), 0 (no correction)."""
    n = cfg.n_streams
    if mode == MODE_IDN:
        return np.eye(n, dtype=dtype)
    if mode == MODE_HCN:
        if n == 1:
            return np.eye(1, dtype=dtype)
        return W.hc_res_mlp[l].astype(dtype) @ W.hc_res_attn[l].astype(dtype)
    if mode == MODE_NOCORR:
        return np.zeros((n, n), dtype=dtype)
    raise ValueError("unknown mode")


# --------------------------------------------------------------------------- #
# model entry / exit
# --------------------------------------------------------------------------- #
def embed(cfg, W, ids, dtype=np.float64):
    """h_0 = Embed(x): ids[B, T] -> [B, T, n, d]; the embedding row is copied into every stream."""
    e = W.embed[np.asarray(ids)].astype(dtype)  # [B, T, d]
    return np.repeat(e[:, :, None, :], cfg.n_streams, axis=2)


def lm_head(cfg, W, hL, dtype=np.float64):
    """LMHead(h_L): sum the streams, RMSNorm, project: [B, T, n, d] -> logits [B, T, V]."""
    x = rmsnorm(np.sum(hL, axis=2), cfg.rms_eps)
    return x @ W.lm_head.astype(dtype).T


def greedy(logits):
    """argmax over the vocabulary, ties to the lowest index."""
    return np.argmax(logits, axis=-1).astype(np.int32)


# --------------------------------------------------------------------------- #
# Algorithm 1 and Algorithm 2
# --------------------------------------------------------------------------- #
def _scratch_kv(cfg, B, T, dtype):
    return LayerKV(cfg.n_layer, B, T, cfg.n_head, cfg.head_dim, dtype)


def forward_sequential(cfg, W, h0, kv=None, pos0=0, dtype=np.float64):
    """Algorithm 1.  h0: [B, T, n, d].  Returns the trace [L+1, B, T, n, d]."""
    h0 = np.asarray(h0, dtype=dtype)
    B, T = h0.shape[:2]
    if kv is None:
        kv = _scratch_kv(cfg, B, T, dtype)
    L = cfg.n_layer
    trace = np.empty((L + 1,) + h0.shape, dtype=dtype)
    trace[0] = h0
    for l in range(L):
        trace[l + 1] = block(cfg, W, l, trace[l], kv, pos0, dtype)
    return trace


def residual_norms(cfg, W, trace, kv=None, pos0=0, dtype=np.float64):
    """Eq. (2) evaluated on a trace: per layer (sum |F_l(h_l) - h_{l+1}|^2, sum |h_{l+1}|^2)."""
    L = cfg.n_layer
    B, T = trace.shape[1:3]
    if kv is None:
        kv = _scratch_kv(cfg, B, T, dtype)
    out = np.zeros((L, 2), dtype=np.float64)
    for l in range(L):
        r = block(cfg, W, l, trace[l], kv, pos0, dtype) - trace[l + 1]
        out[l, 0] = np.sum(r.astype(np.float64) ** 2)
        out[l, 1] = np.sum(trace[l + 1].astype(np.float64) ** 2)
    return out


INIT_H0 = 0   # suffix states start at the prefix state h_S          (Alg. 2 line 5)
INIT_FWD = 1  # suffix states start at a one-shot parallel forward f_l(h_S)   (Sec. 3.5, Sec. 5 "fwd")


def forward_snlp(cfg, W, h0, K, mode, kv=None, pos0=0, dtype=np.float64, all_sweeps=False, S=0, init=INIT_H0):
    """Algorithm 2: sequential prefix of S layers, then K sweeps over the suffix S..L-1.

    init = INIT_H0: every suffix state starts at h_S (Alg. 2 line 5).  init = INIT_FWD: suffix state l+1
    starts at F_l(h_S), one batched evaluation of every suffix block on the prefix state (Sec. 3.5).
    Returns (trace after K sweeps [L+1, B, T, n, d], resnorm [K, L, 2]) where, for suffix layers,
    resnorm[k, l] = (sum |F_l(h_l^k) - h_{l+1}^k|^2, sum |h_{l+1}^k|^2): the residual of Eq. (2)
    at the trace that ENTERS sweep k (prefix layers: zeros).  With all_sweeps=True also returns the list of
    traces h^0 .. h^K.  K = 0 is allowed when S > 0 or init = INIT_FWD (prefix / one-shot forward only).
    """
    L = cfg.n_layer
    if K < 0 or not (0 <= S <= L):
        raise ValueError("K must be >= 0 and 0 <= S <= L")
    h0 = np.asarray(h0, dtype=dtype)
    B, T = h0.shape[:2]
    if kv is None:
        kv = _scratch_kv(cfg, B, T, dtype)
    old = np.empty((L + 1,) + h0.shape, dtype=dtype)
    old[0] = h0
    for l in range(S):  # sequential prefix (Alg. 2 lines 2-4)
        old[l + 1] = block(cfg, W, l, old[l], kv, pos0, dtype)
    hS = old[S].copy()
    for l in range(S, L):
        old[l + 1] = hS if init == INIT_H0 else block(cfg, W, l, hS, kv, pos0, dtype)
    res = np.zeros((K, L, 2), dtype=np.float64)
    history = [old.copy()]
    for k in range(K):
        # parallel for: every suffix block on its own current input
        tilde = np.empty_like(old)
        for l in range(S, L):
            tilde[l + 1] = block(cfg, W, l, old[l], kv, pos0, dtype)
            r = (tilde[l + 1] - old[l + 1]).astype(np.float64)
            res[k, l, 0] = np.sum(r * r)
            res[k, l, 1] = np.sum(old[l + 1].astype(np.float64) ** 2)
        # sequential structured correction, Eq. (5); h_S^(k+1) = h_S
        new = old.copy()
        for l in range(S, L):
            A = surrogate(cfg, W, l, mode, dtype)
            delta = new[l] - old[l]
            new[l + 1] = tilde[l + 1] + np.einsum("rs,btsd->btrd", A, delta)
        old = new
        history.append(old.copy())
    if all_sweeps:
        return old, res, history
    return old, res


# --------------------------------------------------------------------------- #
# fused chunks (App. C.3) and the chunkwise update, Eq. (11)
# --------------------------------------------------------------------------- #
def fused_chunk(cfg, W, layers, h, kv, pos0, dtype):
    """One fused chunk of residual blocks that all read the same input h[B, T, 1, d] (App. C.3):

        a_C = sum_{l in C} O_l Attn_l(Q_l h, K_l h, V_l h)
        u_C = h + a_C
        m_C = sum_{l in C} P_l phi(W_l Norm(u_C))
        F_C = u_C + m_C

    Returns (F_C(h), a_C, m_C).  Every layer of the chunk keeps its own keys/values.
    """
    x = h[:, :, 0, :]
    a = np.zeros_like(x)
    for l in layers:
        a = a + attention_branch(cfg, W, l, x, kv, pos0, dtype)
    u = x + a
    m = np.zeros_like(x)
    for l in layers:
        m = m + mlp_branch(cfg, W, l, u, dtype)
    return (u + m)[:, :, None, :], a, m


def forward_chunked(cfg, W, h0, K, fuse, kv=None, pos0=0, dtype=np.float64, S=0, init=INIT_H0, correct=True):
    """Chunkwise SNLP with fused layers ("NxFM" configurations, Sec. 3.5): a sequential prefix of S layers, then
    the suffix split into N = (L - S) / fuse chunks of `fuse` fused layers; K sweeps of Eq. (11) with the identity
    chunk surrogate.  K = 0 with init = INIT_H0 is not meaningful; K = None runs the fused model sequentially
    (chunk after chunk), the reference the paper compares fused-weight variants with.

    Returns the list of chunk-boundary states [h_S, h_{S+fuse}, ..., h_L] (each [B, T, 1, d]).
    """
    if cfg.n_streams != 1:
        raise ValueError("fused chunks are defined for residual (single-stream) blocks")
    L = cfg.n_layer
    if (L - S) % fuse:
        raise ValueError("suffix length must be a multiple of the chunk size")
    h0 = np.asarray(h0, dtype=dtype)
    B, T = h0.shape[:2]
    if kv is None:
        kv = _scratch_kv(cfg, B, T, dtype)
    h = h0
    for l in range(S):
        h = block(cfg, W, l, h, kv, pos0, dtype)
    chunks = [list(range(S + c * fuse, S + (c + 1) * fuse)) for c in range((L - S) // fuse)]
    N = len(chunks)
    if K is None:  # sequential execution of the fused model
        states = [h]
        for C in chunks:
            states.append(fused_chunk(cfg, W, C, states[-1], kv, pos0, dtype)[0])
        return states
    old = [h] + [h if init == INIT_H0 else fused_chunk(cfg, W, C, h, kv, pos0, dtype)[0] for C in chunks]
    for _ in range(K):
        tilde = [None] + [fused_chunk(cfg, W, chunks[c], old[c], kv, pos0, dtype)[0] for c in range(N)]
        new = [h]
        for c in range(N):
            corr = (new[c] - old[c]) if correct else 0.0
            new.append(tilde[c + 1] + corr)
        old = new
    return old


# --------------------------------------------------------------------------- #
# KV-cached decoding and greedy self-speculative decoding
# --------------------------------------------------------------------------- #
def prefill(cfg, W, ids, kv, dtype=np.float64):
    """Sequential forward over ids[B, T] starting at kv.len; fills the cache.  Returns last-row logits."""
    ids = np.asarray(ids)
    h0 = embed(cfg, W, ids, dtype)
    tr = forward_sequential(cfg, W, h0, kv, kv.len, dtype)
    kv.len += ids.shape[1]
    return lm_head(cfg, W, tr[-1][:, -1:], dtype)[:, 0]


def decode_step(cfg, W, kv, tok_in, K, mode, dtype=np.float64):
    """One decode step at position kv.len.  K = 0: sequential; K >= 1: K SNLP sweeps.

    Every sweep recomputes the new position's keys/values from the current iterate and overwrites
    the cache slot, so the cache keeps the last sweep's values.  Returns (tok_out[B], logits[B, V]).
    """
    ids = np.asarray(tok_in).reshape(-1, 1)
    h0 = embed(cfg, W, ids, dtype)
    if K == 0:
        hL = forward_sequential(cfg, W, h0, kv, kv.len, dtype)[-1]
    else:
        hL = forward_snlp(cfg, W, h0, K, mode, kv, kv.len, dtype)[0][-1]
    kv.len += 1
    logits = lm_head(cfg, W, hL, dtype)[:, 0]
    return greedy(logits), logits


def draft_and_verify(cfg, W, kv, last_tok, block_size, K, mode, dtype=np.float64):
    """One round of greedy self-speculative decoding, batch 1 (Sec. 5.1).

    Drafter: block_size SNLP(K) decode steps from last_tok -> x_1..x_B.
    Verifier: one sequential forward over [last_tok, x_1..x_B] at the round's first position
    -> y_0..y_B (its keys/values overwrite the drafter's).  Accept the longest prefix with
    x_i == y_{i-1}; emit x_1..x_n, y_n; the cache is cut back to len_before + n + 1.
    Returns (emitted list, n_accepted, next last_tok).
    """
    len0 = kv.len
    drafts = []
    t = int(last_tok)
    for _ in range(block_size):
        t = int(decode_step(cfg, W, kv, [t], K, mode, dtype)[0][0])
        drafts.append(t)
    kv.len = len0
    ids = np.array([[int(last_tok)] + drafts])
    h0 = embed(cfg, W, ids, dtype)
    tr = forward_sequential(cfg, W, h0, kv, len0, dtype)
    y = greedy(lm_head(cfg, W, tr[-1], dtype))[0]  # [B+1]
    n = 0
    while n < block_size and drafts[n] == int(y[n]):
        n += 1
    emitted = drafts[:n] + [int(y[n])]
    kv.len = len0 + n + 1
    return emitted, n, int(y[n])


def ssd_ideal_speedup(alpha, block_size, s):
    """Ideal self-speculative speed-up ((1 - a^(B+1)) / (1 - a)) / (B / s + 1)  (Sec. 5.1)."""
    if alpha >= 1.0:
        num = block_size + 1.0
    else:
        num = (1.0 - alpha ** (block_size + 1)) / (1.0 - alpha)
    return num / (block_size / s + 1.0)


def make_config(**kw):
    """Plain attribute bag with the fields the oracle reads (the oracle never imports the product's config)."""
    d = dict(n_layer=4, d_model=64, n_head=2, head_dim=32, d_ff=256, vocab=256, n_streams=1,
             rms_eps=1e-6, rope_base=10000.0)
    d.update(kw)
    return SimpleNamespace(**d)
