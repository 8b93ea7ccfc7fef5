"""CPU-only pins of the oracle against what the paper and the mathematics fix.

Each test is chosen so that a plausible mistake in oracle/snlp_oracle.py (dropped term, wrong
sign or index, transposed operand) fails at least one of them.
"""
import math
import os

import numpy as np
import pytest

from oracle import snlp_oracle as O
from paper_2605_17842_b200 import synth
from tests.naive_ref import NaiveModel

HERE = os.path.dirname(os.path.abspath(__file__))


def small_cfg(n_streams=1, L=3):
    return synth.ModelConfig(n_layer=L, d_model=16, n_head=2, head_dim=8, d_ff=24, vocab=50,
                             n_streams=n_streams, dtype="fp32")


def big_weights(cfg, seed=11):
    # std large enough that the branches matter (far from the J ~ I regime)
    return synth.make_weights(cfg, seed=seed, std=0.3, embed_std=1.0)


def to_lists(x):  # [1, T, n, d] -> list[t][s][j]
    return x[0].astype(np.float64).tolist()


def relerr(a, b):
    return np.linalg.norm(np.asarray(a, dtype=np.float64) - np.asarray(b, dtype=np.float64)) / (
        np.linalg.norm(np.asarray(b, dtype=np.float64)) + 1e-300)


# ------------------------------------------------------------------ elementary pieces
def test_rotary_pos0_is_identity_and_norm_preserving():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((1, 5, 2, 8))
    y = O.rotary(x, np.arange(5), 10000.0)
    assert np.allclose(y[:, 0], x[:, 0], atol=0, rtol=0)
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-13)


def test_rotary_is_relative():
    # textbook RoPE property: <R_m q, R_n k> depends only on m - n
    rng = np.random.default_rng(1)
    q = rng.standard_normal((1, 1, 1, 8))
    k = rng.standard_normal((1, 1, 1, 8))
    def dot(m, n):
        return float(np.sum(O.rotary(q, [m], 10000.0) * O.rotary(k, [n], 10000.0)))
    assert abs(dot(7, 3) - dot(11, 7)) < 1e-12
    assert abs(dot(7, 3) - dot(3, 7)) > 1e-6  # and it is not symmetric


def test_rotary_first_pair_is_plain_rotation():
    # i = 0 has frequency 1: the pair (x0, x_{hd/2}) turns by `pos` radians, counter-clockwise
    x = np.zeros((1, 1, 1, 8)); x[..., 0] = 1.0
    y = O.rotary(x, [2], 10000.0)[0, 0, 0]
    assert abs(y[0] - math.cos(2.0)) < 1e-15 and abs(y[4] - math.sin(2.0)) < 1e-15


def test_rmsnorm_closed_form():
    x = np.array([[3.0, 4.0, 0.0, 0.0]])
    y = O.rmsnorm(x, 0.0)
    assert np.allclose(y, x / math.sqrt(25.0 / 4.0))
    assert np.allclose(np.mean(O.rmsnorm(np.random.default_rng(2).standard_normal((7, 33)), 0.0) ** 2, -1), 1.0)


# ------------------------------------------------------------------ brute force
@pytest.mark.parametrize("n_streams", [1, 3])
def test_block_and_sequential_match_scalar_brute_force(n_streams):
    cfg = small_cfg(n_streams)
    W = big_weights(cfg)
    h0 = synth.make_hidden(cfg, 1, 5, seed=3).astype(np.float64)
    tr = O.forward_sequential(cfg, W, h0)
    nv = NaiveModel(cfg, W).sequential(to_lists(h0))
    for l in range(cfg.n_layer + 1):
        assert relerr(tr[l][0], np.array(nv[l])) < 1e-12, l


@pytest.mark.parametrize("n_streams,mode", [(1, O.MODE_IDN), (3, O.MODE_HCN), (3, O.MODE_IDN), (1, O.MODE_NOCORR)])
@pytest.mark.parametrize("K", [1, 2])
def test_snlp_matches_scalar_brute_force(n_streams, mode, K):
    cfg = small_cfg(n_streams)
    W = big_weights(cfg)
    h0 = synth.make_hidden(cfg, 1, 4, seed=4).astype(np.float64)
    tr, _ = O.forward_snlp(cfg, W, h0, K, mode)
    nv = NaiveModel(cfg, W).snlp(to_lists(h0), K, mode)
    for l in range(cfg.n_layer + 1):
        assert relerr(tr[l][0], np.array(nv[l])) < 1e-12, l


def test_tiny_config_sequential_matches_scalar_brute_force():
    cfg = synth.CONFIGS["tiny"]
    W = synth.make_weights(cfg, seed=1234)
    ids = synth.make_ids(cfg, 1, 6, seed=1)
    h0 = O.embed(cfg, W, ids)
    tr = O.forward_sequential(cfg, W, h0)
    nv = NaiveModel(cfg, W).sequential(to_lists(h0))
    assert relerr(tr[-1][0], np.array(nv[-1])) < 1e-12


# ------------------------------------------------------------------ structure of the block
def test_attention_is_causal_and_rows_independent_of_future():
    cfg = small_cfg()
    W = big_weights(cfg)
    h0 = synth.make_hidden(cfg, 2, 6, seed=5).astype(np.float64)
    tr = O.forward_sequential(cfg, W, h0)
    h1 = h0.copy()
    h1[:, 4:] += 1.0  # perturb positions >= 4
    tr1 = O.forward_sequential(cfg, W, h1)
    assert np.array_equal(tr[:, :, :4], tr1[:, :, :4])
    assert not np.allclose(tr[-1][:, 4:], tr1[-1][:, 4:])
    # batch rows do not interact
    h2 = h0.copy(); h2[1] += 1.0
    assert np.array_equal(O.forward_sequential(cfg, W, h2)[:, 0], tr[:, 0])


def test_single_token_attention_returns_value_projection():
    # with one key the softmax weight is 1, so a = Wo Wv norm(x) exactly
    cfg = small_cfg()
    W = big_weights(cfg)
    d = cfg.d_model
    x = synth.make_hidden(cfg, 1, 1, seed=6).astype(np.float64)[:, :, 0]
    kv = O.LayerKV(cfg.n_layer, 1, 1, cfg.n_head, cfg.head_dim)
    a = O.attention_branch(cfg, W, 1, x, kv, 0, np.float64)
    xn = x / np.sqrt(np.mean(x * x, -1, keepdims=True) + cfg.rms_eps)
    want = (xn @ W.wqkv[1][2 * d:3 * d].astype(np.float64).T) @ W.wo[1].astype(np.float64).T
    assert relerr(a, want) < 1e-13


def test_uniform_attention_when_keys_equal():
    # if all inputs in a sequence are equal and rotary is switched off (base -> inf makes every
    # frequency except i=0 vanish; use a 2-dim head to keep only ... ) -- instead use zero Wq:
    # zero queries give uniform softmax, so o_t is the running mean of the values.
    cfg = small_cfg()
    W = big_weights(cfg)
    d = cfg.d_model
    W.wqkv = W.wqkv.copy(); W.wqkv[:, 0:d] = 0.0
    x = synth.make_hidden(cfg, 1, 5, seed=8).astype(np.float64)[:, :, 0]
    kv = O.LayerKV(cfg.n_layer, 1, 5, cfg.n_head, cfg.head_dim)
    a = O.attention_branch(cfg, W, 0, x, kv, 0, np.float64)
    v = (O.rmsnorm(x, cfg.rms_eps) @ W.wqkv[0][2 * d:].astype(np.float64).T)
    run_mean = np.cumsum(v, axis=1) / np.arange(1, 6)[None, :, None]
    assert relerr(a, run_mean @ W.wo[0].astype(np.float64).T) < 1e-12


def test_mlp_is_relu_squared():
    cfg = small_cfg()
    W = big_weights(cfg)
    u = synth.make_hidden(cfg, 1, 3, seed=9).astype(np.float64)[:, :, 0]
    y = O.rmsnorm(u, cfg.rms_eps) @ W.wup[2].astype(np.float64).T
    want = (np.where(y > 0, y * y, 0.0)) @ W.wdn[2].astype(np.float64).T
    assert relerr(O.mlp_branch(cfg, W, 2, u, np.float64), want) < 1e-13
    assert np.any(y < 0) and np.any(y > 0)


# ------------------------------------------------------------------ SNLP invariants
@pytest.mark.parametrize("n_streams,mode", [(1, O.MODE_IDN), (4, O.MODE_HCN), (4, O.MODE_IDN), (1, O.MODE_NOCORR), (4, O.MODE_NOCORR)])
def test_finite_step_exactness(n_streams, mode):
    """After k sweeps from the h0 initialisation, states 0..k equal the sequential trace for any
    surrogate (Newton on a block lower-bidiagonal system); K = L recovers it; K > L changes nothing."""
    cfg = small_cfg(n_streams, L=4)
    W = big_weights(cfg)
    h0 = synth.make_hidden(cfg, 2, 5, seed=10).astype(np.float64)
    seq = O.forward_sequential(cfg, W, h0)
    _, res, hist = O.forward_snlp(cfg, W, h0, cfg.n_layer + 2, mode, all_sweeps=True)
    for k in range(cfg.n_layer + 3):
        for l in range(min(k, cfg.n_layer) + 1):
            assert relerr(hist[k][l], seq[l]) < 1e-12, (k, l)
        if 0 < k < cfg.n_layer:
            # and the iterate is NOT yet converged further down (the test has teeth)
            assert relerr(hist[k][-1], seq[-1]) > 1e-6
    # residuals of already-exact layers vanish: res[k, l] == 0 for l < k
    for k in range(res.shape[0]):
        for l in range(min(k, cfg.n_layer)):
            assert res[k, l, 0] <= 1e-20 * max(res[k, l, 1], 1.0), (k, l)


def test_idn_one_step_closed_form():
    """K = 1 IDN from h0: h_L = h_0 + sum_l g_l(h_0)  (App. C.1)."""
    cfg = small_cfg(1, L=4)
    W = big_weights(cfg)
    h0 = synth.make_hidden(cfg, 1, 5, seed=12).astype(np.float64)
    tr, _ = O.forward_snlp(cfg, W, h0, 1, O.MODE_IDN)
    kv = O.LayerKV(cfg.n_layer, 1, 5, cfg.n_head, cfg.head_dim)
    acc = h0.copy()
    for l in range(cfg.n_layer):
        _, a, m = O.residual_block(cfg, W, l, h0, kv, 0, np.float64)
        acc = acc + (a + m)[:, :, None, :]
        assert relerr(tr[l + 1], acc) < 1e-13


def test_idn_prefix_sum_identity():
    """h_{l+1}^{k+1} = h_0 + sum_{j<=l} g_j(h_j^k), g = F - id  (Eq. 7 telescoped)."""
    cfg = small_cfg(1, L=4)
    W = big_weights(cfg)
    h0 = synth.make_hidden(cfg, 1, 4, seed=13).astype(np.float64)
    _, _, hist = O.forward_snlp(cfg, W, h0, 3, O.MODE_IDN, all_sweeps=True)
    kv = O.LayerKV(cfg.n_layer, 1, 4, cfg.n_head, cfg.head_dim)
    for k in range(3):
        acc = h0.copy()
        for l in range(cfg.n_layer):
            acc = acc + (O.block(cfg, W, l, hist[k][l], kv, 0, np.float64) - hist[k][l])
            assert relerr(hist[k + 1][l + 1], acc) < 1e-12


def test_idn_residual_identity():
    """For IDN and k >= 1 the residual entering sweep k is g_l(h_l^k) - g_l(h_l^{k-1})."""
    cfg = small_cfg(1, L=4)
    W = big_weights(cfg)
    h0 = synth.make_hidden(cfg, 1, 4, seed=14).astype(np.float64)
    _, res, hist = O.forward_snlp(cfg, W, h0, 3, O.MODE_IDN, all_sweeps=True)
    kv = O.LayerKV(cfg.n_layer, 1, 4, cfg.n_head, cfg.head_dim)
    g = lambda l, h: O.block(cfg, W, l, h, kv, 0, np.float64) - h
    for l in range(cfg.n_layer):
        assert abs(res[0, l, 0] - np.sum(g(l, h0) ** 2)) < 1e-10 * res[0, l, 0]
        assert abs(res[0, l, 1] - np.sum(h0 ** 2)) < 1e-10 * res[0, l, 1]
    for k in (1, 2):
        for l in range(k, cfg.n_layer):
            want = np.sum((g(l, hist[k][l]) - g(l, hist[k - 1][l])) ** 2)
            assert abs(res[k, l, 0] - want) < 1e-9 * max(want, 1e-30)


def test_residual_norms_function_agrees_and_vanishes_on_sequential_trace():
    cfg = small_cfg(1, L=3)
    W = big_weights(cfg)
    h0 = synth.make_hidden(cfg, 1, 4, seed=15).astype(np.float64)
    seq = O.forward_sequential(cfg, W, h0)
    assert np.all(O.residual_norms(cfg, W, seq)[:, 0] == 0.0)
    _, res, hist = O.forward_snlp(cfg, W, h0, 2, O.MODE_IDN, all_sweeps=True)
    assert np.allclose(O.residual_norms(cfg, W, hist[1]), res[1], rtol=1e-12)


def test_hcn_reduces_to_idn():
    """n = 1 with all maps 1 is the residual block; n = 4 with identity mixing and unit maps runs
    IDN on every stream (IDN is the degenerate residual case of the HC template, App. C.2)."""
    cfg1 = small_cfg(1)
    W = big_weights(cfg1)
    h0 = synth.make_hidden(cfg1, 1, 4, seed=16).astype(np.float64)
    ref, res_ref = O.forward_snlp(cfg1, W, h0, 2, O.MODE_IDN)
    # (a) HCN mode on a single-stream model is IDN, bit for bit
    got, res = O.forward_snlp(cfg1, W, h0, 2, O.MODE_HCN)
    assert np.array_equal(got, ref) and np.array_equal(res, res_ref)
    # (b) mHC block with n=1 and H = 1 equals the residual block
    L = cfg1.n_layer
    W.hc_res_attn = np.ones((L, 1, 1), np.float32); W.hc_res_mlp = np.ones((L, 1, 1), np.float32)
    for nm in ("hc_pre_attn", "hc_pre_mlp", "hc_post_attn", "hc_post_mlp"):
        setattr(W, nm, np.ones((L, 1), np.float32))
    kv = O.LayerKV(L, 1, 4, cfg1.n_head, cfg1.head_dim)
    assert relerr(O.mhc_block(cfg1, W, 1, h0, kv, 0, np.float64)[0],
                  O.residual_block(cfg1, W, 1, h0, kv, 0, np.float64)[0]) < 1e-14
    # (c) n = 2, R = I, pre = e_0 (read stream 0), post = e_0: stream 0 runs the residual model
    #     with IDN, stream 1 is carried unchanged
    cfg2 = small_cfg(2)
    W.hc_res_attn = np.tile(np.eye(2, dtype=np.float32), (L, 1, 1)); W.hc_res_mlp = W.hc_res_attn.copy()
    e0 = np.tile(np.array([1.0, 0.0], np.float32), (L, 1))
    for nm in ("hc_pre_attn", "hc_pre_mlp", "hc_post_attn", "hc_post_mlp"):
        setattr(W, nm, e0.copy())
    x0 = np.concatenate([h0, 5.0 + h0], axis=2)
    got2, _ = O.forward_snlp(cfg2, W, x0, 2, O.MODE_HCN)
    assert relerr(got2[:, :, :, 0:1], ref) < 1e-13
    assert np.array_equal(got2[:, :, :, 1:2], np.broadcast_to(x0[:, :, 1:2], got2[:, :, :, 1:2].shape))


def test_hcn_surrogate_is_doubly_stochastic_product_in_the_right_order():
    cfg = small_cfg(4)
    W = big_weights(cfg)
    for l in range(cfg.n_layer):
        A = O.surrogate(cfg, W, l, O.MODE_HCN, np.float64)
        assert np.allclose(A.sum(0), 1.0, atol=1e-6) and np.allclose(A.sum(1), 1.0, atol=1e-6)
        # A is the Jacobian of the block w.r.t. its input when both branches are switched off
        Wz = synth.make_weights(cfg, seed=11, std=0.3)
        Wz.wo = np.zeros_like(Wz.wo); Wz.wdn = np.zeros_like(Wz.wdn)
        x = synth.make_hidden(cfg, 1, 2, seed=17).astype(np.float64)
        kv = O.LayerKV(cfg.n_layer, 1, 2, cfg.n_head, cfg.head_dim)
        y = O.mhc_block(cfg, Wz, l, x, kv, 0, np.float64)[0]
        assert relerr(y, np.einsum("rs,btsd->btrd", A, x)) < 1e-13
        assert not np.allclose(A, A.T)  # order of the product matters


def test_zero_branch_gives_identity_trace():
    cfg = small_cfg(1)
    W = big_weights(cfg)
    W.wo = np.zeros_like(W.wo); W.wdn = np.zeros_like(W.wdn)
    h0 = synth.make_hidden(cfg, 1, 4, seed=18).astype(np.float64)
    tr, res = O.forward_snlp(cfg, W, h0, 2, O.MODE_IDN)
    assert all(np.array_equal(tr[l], h0) for l in range(cfg.n_layer + 1))
    assert np.all(res[:, :, 0] == 0.0)


def test_staircase_without_correction():
    """A = 0: after k sweeps h_L depends only on the last k blocks; with the IDN correction every
    block already moves h_L at K = 1 (Sec. 3.2, appendix 'Correction Propagation')."""
    cfg = small_cfg(1, L=4)
    W = big_weights(cfg)
    W2 = big_weights(cfg)
    W2.wup = W2.wup.copy(); W2.wup[0] *= -1.3; W2.wup[1] *= 0.4  # perturb blocks 0 and 1
    h0 = synth.make_hidden(cfg, 1, 4, seed=19).astype(np.float64)
    for K in (1, 2):
        a = O.forward_snlp(cfg, W, h0, K, O.MODE_NOCORR)[0][-1]
        b = O.forward_snlp(cfg, W2, h0, K, O.MODE_NOCORR)[0][-1]
        assert np.array_equal(a, b)
    a = O.forward_snlp(cfg, W, h0, 3, O.MODE_NOCORR)[0][-1]
    b = O.forward_snlp(cfg, W2, h0, 3, O.MODE_NOCORR)[0][-1]
    assert relerr(a, b) > 1e-6  # block 1 is reached at K = 3
    a = O.forward_snlp(cfg, W, h0, 1, O.MODE_IDN)[0][-1]
    b = O.forward_snlp(cfg, W2, h0, 1, O.MODE_IDN)[0][-1]
    assert relerr(a, b) > 1e-6
    # closed form: after k sweeps without correction h_L = F_{L-1} o ... o F_{L-k}(h_0)
    kv = O.LayerKV(cfg.n_layer, 1, 4, cfg.n_head, cfg.head_dim)
    h = h0
    for l in (2, 3):
        h = O.block(cfg, W, l, h, kv, 0, np.float64)
    assert relerr(O.forward_snlp(cfg, W, h0, 2, O.MODE_NOCORR)[0][-1], h) < 1e-13


def test_hcn_stream_sum_conservation():
    """Column sums of A_l are 1, so the stream-sum of the correction term is carried unchanged:
    sum_r [A (dx)]_r = sum_s dx_s."""
    cfg = small_cfg(4)
    W = big_weights(cfg)
    rng = np.random.default_rng(3)
    dx = rng.standard_normal((1, 2, 4, cfg.d_model))
    A = O.surrogate(cfg, W, 0, O.MODE_HCN, np.float64)
    assert np.allclose(np.einsum("rs,btsd->btrd", A, dx).sum(2), dx.sum(2), atol=1e-5)


# ------------------------------------------------------------------ decoding
@pytest.mark.parametrize("n_streams", [1, 4])
def test_decode_equals_prefill_and_KL_equals_sequential(n_streams):
    cfg = small_cfg(n_streams, L=3)
    W = big_weights(cfg)
    ids = synth.make_ids(cfg, 2, 7, seed=20)
    kv_a = O.LayerKV(cfg.n_layer, 2, 16, cfg.n_head, cfg.head_dim)
    logits_a = O.prefill(cfg, W, ids, kv_a)
    # token-by-token sequential decode fills the same cache and gives the same last logits
    kv_b = O.LayerKV(cfg.n_layer, 2, 16, cfg.n_head, cfg.head_dim)
    for t in range(7):
        _, logits_b = O.decode_step(cfg, W, kv_b, ids[:, t], 0, O.MODE_IDN)
    assert relerr(logits_b, logits_a) < 1e-12
    assert relerr(kv_b.k[:, :, :7], kv_a.k[:, :, :7]) < 1e-12 and kv_b.len == 7
    # K = L sweeps reproduce the sequential step (token, logits and the cache it leaves)
    mode = O.MODE_HCN if n_streams > 1 else O.MODE_IDN
    kv_c, kv_d = kv_a.copy(), kv_a.copy()
    tok_c, log_c = O.decode_step(cfg, W, kv_c, ids[:, 0], 0, mode)
    tok_d, log_d = O.decode_step(cfg, W, kv_d, ids[:, 0], cfg.n_layer, mode)
    assert np.array_equal(tok_c, tok_d) and relerr(log_d, log_c) < 1e-12
    assert relerr(kv_d.v[:, :, :8], kv_c.v[:, :, :8]) < 1e-12
    # K = 1 differs (the solver bias is real) but layer 0's cache entry is already exact
    kv_e = kv_a.copy()
    _, log_e = O.decode_step(cfg, W, kv_e, ids[:, 0], 1, mode)
    assert relerr(log_e, log_c) > 1e-8
    assert relerr(kv_e.k[0, :, 7], kv_c.k[0, :, 7]) < 1e-13


def test_draft_and_verify_reproduces_sequential_greedy():
    cfg = small_cfg(1, L=3)
    W = big_weights(cfg)
    ids = synth.make_ids(cfg, 1, 5, seed=21)
    kv = O.LayerKV(cfg.n_layer, 1, 64, cfg.n_head, cfg.head_dim)
    first = int(O.greedy(O.prefill(cfg, W, ids, kv))[0])
    kv_seq = kv.copy()
    # reference stream: plain sequential greedy decoding
    want, t = [], first
    for _ in range(20):
        t = int(O.decode_step(cfg, W, kv_seq, [t], 0, O.MODE_IDN)[0][0])
        want.append(t)
    got, last, n_acc_total, rounds = [], first, 0, 0
    while len(got) < 20:
        emitted, n_acc, last = O.draft_and_verify(cfg, W, kv, last, 4, 1, O.MODE_IDN)
        assert 1 <= len(emitted) <= 5 and len(emitted) == n_acc + 1
        got += emitted
        n_acc_total += n_acc
        rounds += 1
    assert got[:20] == want
    assert kv.len == 5 + len(got)
    # with K = L the drafter is exact, so every draft is accepted
    kv2 = O.LayerKV(cfg.n_layer, 1, 64, cfg.n_head, cfg.head_dim)
    f2 = int(O.greedy(O.prefill(cfg, W, ids, kv2))[0])
    emitted, n_acc, _ = O.draft_and_verify(cfg, W, kv2, f2, 4, cfg.n_layer, O.MODE_IDN)
    assert n_acc == 4 and emitted == want[:5]


def test_ssd_estimator_reproduces_the_papers_table():
    rows = [l.split() for l in open(os.path.join(HERE, "golden", "ssd_table.txt")) if l.strip() and l[0] != "#"]
    assert len(rows) == 18
    for s, B, alpha, _tok, speed in rows:
        est = O.ssd_ideal_speedup(float(alpha), int(B), float(s))
        assert abs(est - float(speed)) < 0.02, (s, B, alpha, est, speed)
    assert O.ssd_ideal_speedup(1.0, 4, 2.0) == pytest.approx(5.0 / 3.0)


def test_greedy_ties_go_to_lowest_index():
    assert O.greedy(np.array([[1.0, 3.0, 3.0, 2.0]]))[0] == 1


def test_fp32_instantiation_close_to_fp64():
    cfg = small_cfg(1)
    W = big_weights(cfg)
    h0 = synth.make_hidden(cfg, 1, 4, seed=22)
    a = O.forward_snlp(cfg, W, h0, 2, O.MODE_IDN, dtype=np.float32)[0]
    b = O.forward_snlp(cfg, W, h0, 2, O.MODE_IDN)[0]
    assert a.dtype == np.float32 and relerr(a, b) < 1e-4


# ------------------------------------------------------------------ prefix S, fwd initialisation, fused chunks
@pytest.mark.parametrize("n_streams,mode", [(1, O.MODE_IDN), (4, O.MODE_HCN)])
def test_prefix_and_fwd_init(n_streams, mode):
    cfg = small_cfg(n_streams, L=5)
    W = big_weights(cfg)
    h0 = synth.make_hidden(cfg, 1, 4, seed=30).astype(np.float64)
    seq = O.forward_sequential(cfg, W, h0)
    L = cfg.n_layer
    # S = L is the sequential forward; S = 0 / h0 init is the plain algorithm
    assert relerr(O.forward_snlp(cfg, W, h0, 0, mode, S=L)[0], seq) < 1e-13
    for S in (0, 2):
        for init in (O.INIT_H0, O.INIT_FWD):
            _, _, hist = O.forward_snlp(cfg, W, h0, 3, mode, S=S, init=init, all_sweeps=True)
            extra = 1 if init == O.INIT_FWD else 0   # the one-shot forward already makes state S+1 exact
            for k in range(4):
                exact_upto = min(L, S + k + extra)
                for l in range(exact_upto + 1):
                    assert relerr(hist[k][l], seq[l]) < 1e-12, (S, init, k, l)
                if exact_upto + 1 <= L:
                    assert relerr(hist[k][exact_upto + 1], seq[exact_upto + 1]) > 1e-8, (S, init, k)
    # fwd initialisation is one evaluation of every suffix block on the prefix state
    tr = O.forward_snlp(cfg, W, h0, 0, mode, S=2, init=O.INIT_FWD)[0]
    kv = O.LayerKV(L, 1, 4, cfg.n_head, cfg.head_dim)
    for l in range(2, L):
        assert relerr(tr[l + 1], O.block(cfg, W, l, seq[2], kv, 0, np.float64)) < 1e-13
    # with a prefix the h0-initialised K = 1 closed form starts from h_S (App. C.1)
    if n_streams == 1:
        tr = O.forward_snlp(cfg, W, h0, 1, O.MODE_IDN, S=2)[0]
        acc = seq[2].copy()
        for l in range(2, L):
            _, a, m = O.residual_block(cfg, W, l, seq[2], kv, 0, np.float64)
            acc = acc + (a + m)[:, :, None, :]
        assert relerr(tr[L], acc) < 1e-13


def test_fused_chunks():
    cfg = small_cfg(1, L=4)
    W = big_weights(cfg)
    h0 = synth.make_hidden(cfg, 1, 4, seed=31).astype(np.float64)
    L = cfg.n_layer
    # fuse = 1 is the unfused algorithm
    st = O.forward_chunked(cfg, W, h0, 2, 1)
    ref = O.forward_snlp(cfg, W, h0, 2, O.MODE_IDN)[0]
    for l in range(L + 1):
        assert relerr(st[l], ref[l]) < 1e-13
    # sequential execution of the fuse = 1 model is Algorithm 1
    seq = O.forward_sequential(cfg, W, h0)
    st = O.forward_chunked(cfg, W, h0, None, 1)
    assert relerr(st[-1], seq[-1]) < 1e-13
    # brute force: one fused chunk of 2 layers against the scalar implementation's branches
    from tests.naive_ref import NaiveModel
    nv = NaiveModel(cfg, W)
    xs = h0[0, :, 0, :].tolist()
    a_sum = np.zeros((4, cfg.d_model))
    for l in (1, 2):
        a_sum += np.array(nv.attn(l, xs))
    u = np.array(xs) + a_sum
    m_sum = np.zeros_like(u)
    for l in (1, 2):
        m_sum += np.array(nv.mlp(l, u.tolist()))
    kv = O.LayerKV(L, 1, 4, cfg.n_head, cfg.head_dim)
    F, a, m = O.fused_chunk(cfg, W, [1, 2], h0, kv, 0, np.float64)
    assert relerr(a[0], a_sum) < 1e-12 and relerr(m[0], m_sum) < 1e-12 and relerr(F[0, :, 0], u + m_sum) < 1e-12
    # cross-layer coupling (App. C.3): fused minus "independent branches summed" is exactly the coupling term, and it
    # vanishes when the attention out-projections are zero (every MLP branch then sees the same input h)
    def independent(Wx):
        out = h0.copy()
        for l in (1, 2):
            _, a_l, m_l = O.residual_block(cfg, Wx, l, h0, kv, 0, np.float64)
            out = out + (a_l + m_l)[:, :, None, :]
        return out
    assert relerr(F, independent(W)) > 1e-6
    Wz = big_weights(cfg)
    Wz.wo = np.zeros_like(Wz.wo)
    Fz = O.fused_chunk(cfg, Wz, [1, 2], h0, kv, 0, np.float64)[0]
    assert relerr(Fz, independent(Wz)) < 1e-13
    # chunkwise finite-step exactness against sequential execution of the SAME fused model
    fseq = O.forward_chunked(cfg, W, h0, None, 2)
    for K in (1, 2):
        st = O.forward_chunked(cfg, W, h0, K, 2)
        for c in range(K + 1):
            assert relerr(st[c], fseq[c]) < 1e-12
    assert relerr(O.forward_chunked(cfg, W, h0, 1, 2)[-1], fseq[-1]) > 1e-8
    # one chunk holding the whole suffix (the "1xF4" shape): K = 1 from h0 equals its sequential execution
    assert relerr(O.forward_chunked(cfg, W, h0, 1, 4)[-1], O.forward_chunked(cfg, W, h0, None, 4)[-1]) < 1e-13
    # without correction information moves one chunk per sweep
    a = O.forward_chunked(cfg, W, h0, 1, 2, correct=False)
    assert relerr(a[-1], O.fused_chunk(cfg, W, [2, 3], h0, kv, 0, np.float64)[0]) < 1e-13


# ------------------------------------------------------------------ model entry / exit (Alg. 1 lines 1 and 5)
@pytest.mark.parametrize("n_streams", [1, 3])
def test_embed_and_lm_head_match_scalar_brute_force(n_streams):
    cfg = small_cfg(n_streams)
    W = big_weights(cfg)
    ids = synth.make_ids(cfg, 1, 6, seed=40)
    nv = NaiveModel(cfg, W)
    h0 = O.embed(cfg, W, ids)
    assert h0.shape == (1, 6, n_streams, cfg.d_model)
    assert np.array_equal(h0[0], np.array(nv.embed(ids[0].tolist())))
    # every stream carries the token's own embedding row (not a scaled or split copy)
    for s in range(n_streams):
        assert np.array_equal(h0[0, :, s, :], W.embed[ids[0]].astype(np.float64))
    hL = synth.make_hidden(cfg, 1, 6, seed=41).astype(np.float64)   # streams differ from one another
    want = np.array(nv.lm_head(to_lists(hL)))
    got = O.lm_head(cfg, W, hL)
    assert got.shape == (1, 6, cfg.vocab)
    assert relerr(got[0], want) < 1e-13


def test_lm_head_closed_forms():
    # a one-hot row of the head reads one feature of the normalised stream sum: logit = sum_s h[s][j] / rms(sum_s h[s])
    cfg = small_cfg(3)
    W = big_weights(cfg)
    W.lm_head = np.zeros_like(W.lm_head)
    W.lm_head[7, 5] = 1.0
    W.lm_head[9, 2] = -2.0
    hL = synth.make_hidden(cfg, 1, 4, seed=42).astype(np.float64)
    s = hL.sum(axis=2)                                   # [1, T, d]
    rms = np.sqrt((s * s).mean(-1) + cfg.rms_eps)
    lg = O.lm_head(cfg, W, hL)
    assert np.allclose(lg[..., 7], s[..., 5] / rms, rtol=1e-14, atol=0)
    assert np.allclose(lg[..., 9], -2.0 * s[..., 2] / rms, rtol=1e-14, atol=0)
    assert np.count_nonzero(np.delete(lg, [7, 9], axis=-1)) == 0
    # the final norm makes the logits invariant to the scale of h_L (up to eps) ...
    assert relerr(O.lm_head(cfg, W, 3.0 * hL), lg) < 1e-6
    # ... and the streams enter through their SUM: a mean would not change the logits either, but moving mass
    # between streams must not, while changing one stream alone must
    moved = hL.copy(); moved[:, :, 0] += 0.25; moved[:, :, 1] -= 0.25
    assert relerr(O.lm_head(cfg, W, moved), lg) < 1e-12
    bumped = hL.copy(); bumped[:, :, 2, 5] += 1.0
    assert relerr(O.lm_head(cfg, W, bumped), lg) > 1e-3


# ------------------------------------------------------------------ chunkwise form with a prefix / fwd initialisation
@pytest.mark.parametrize("init", [O.INIT_H0, O.INIT_FWD])
def test_forward_chunked_prefix_and_fwd(init):
    cfg = small_cfg(1, L=6)
    W = big_weights(cfg)
    h0 = synth.make_hidden(cfg, 1, 4, seed=43).astype(np.float64)
    L = cfg.n_layer
    extra = 1 if init == O.INIT_FWD else 0
    # fuse = 1 is Algorithm 2 with the same prefix and initialisation, state for state
    for S in (0, 2):
        for K in (0, 1, 2) if (init == O.INIT_FWD or S > 0) else (1, 2):
            st = O.forward_chunked(cfg, W, h0, K, 1, S=S, init=init)
            ref = O.forward_snlp(cfg, W, h0, K, O.MODE_IDN, S=S, init=init)[0]
            assert len(st) == L - S + 1
            for i, l in enumerate(range(S, L + 1)):
                assert relerr(st[i], ref[l]) < 1e-13, (S, K, l)
    # fuse = 2 behind a prefix of 2: chunkwise finite-step exactness against sequential execution of the SAME fused
    # model -- after K sweeps the first K (+1 with fwd) chunk outputs are final and the next one is not
    S, F = 2, 2
    fseq = O.forward_chunked(cfg, W, h0, None, F, S=S)
    seq = O.forward_sequential(cfg, W, h0)
    assert relerr(fseq[0], seq[S]) < 1e-13          # the prefix is Algorithm 1 up to h_S
    N = (L - S) // F
    for K in (0, 1) if init == O.INIT_FWD else (1,):
        st = O.forward_chunked(cfg, W, h0, K, F, S=S, init=init)
        assert len(st) == N + 1
        exact = min(N, K + extra)
        for c in range(exact + 1):
            assert relerr(st[c], fseq[c]) < 1e-12, (K, c)
        if exact + 1 <= N:
            assert relerr(st[exact + 1], fseq[exact + 1]) > 1e-8, (K, exact)
    # fwd initialisation alone (K = 0) is one evaluation of every chunk on the prefix state
    if init == O.INIT_FWD:
        st = O.forward_chunked(cfg, W, h0, 0, F, S=S, init=O.INIT_FWD)
        kv = O.LayerKV(L, 1, 4, cfg.n_head, cfg.head_dim)
        for c in range(N):
            layers = [S + c * F, S + c * F + 1]
            assert relerr(st[c + 1], O.fused_chunk(cfg, W, layers, seq[S], kv, 0, np.float64)[0]) < 1e-13
    else:
        # h0 initialisation, K = 1: h_S plus every chunk's branches evaluated on h_S (App. C.1 form, chunkwise)
        st = O.forward_chunked(cfg, W, h0, 1, F, S=S)
        kv = O.LayerKV(L, 1, 4, cfg.n_head, cfg.head_dim)
        acc = seq[S].copy()
        for c in range(N):
            _, a, m = O.fused_chunk(cfg, W, [S + c * F, S + c * F + 1], seq[S], kv, 0, np.float64)
            acc = acc + (a + m)[:, :, None, :]
            assert relerr(st[c + 1], acc) < 1e-13
