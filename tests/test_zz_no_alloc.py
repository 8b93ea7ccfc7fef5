"""The allocation-free greedy LM head (snlp_lm_head_greedy_static) against the regular snlp_lm_head and the oracle.

This file is named so that pytest collects it last: the regular entry points are exercised first.
The two calls in a row use different row counts and inputs, so anything the first call leaves in the
library's fixed scratch array must not leak into the second result.

The two entry points run different kernels (tcgen05 product with the handle's workspace / register-fed mma.sync
product with the fixed scratch) that add a logit's terms in different orders, so their tokens must agree wherever
the winning margin of the regular entry point's own logits exceeds the rounding noise of an fp32 sum of d_model
bf16 products; below that margin either token is accepted, and the oracle's fp64 logits bound both."""
import numpy as np
import pytest
import torch

from oracle import snlp_oracle as O
from paper_2605_17842_b200 import synth

pytestmark = pytest.mark.gpu


def _setup(n_streams):
    from paper_2605_17842_b200 import snlp
    cfg = synth.ModelConfig(2, 256, 2, 128, 512, 2048, n_streams, "bf16")
    W = synth.make_weights(cfg, seed=77, std=0.05, embed_std=1.0)
    m = snlp.Model(cfg, max_rows=16, max_batch=16, max_ctx=16)
    m.load_weights(W)
    # the caller's own device copy of the head weights (bf16 bit patterns)
    head = torch.from_numpy(synth.bf16_bits(W.lm_head).view(np.int16)).cuda()
    return snlp, cfg, W, m, head


@pytest.mark.parametrize("n_streams", [1, 4])
def test_static_lm_head_matches_regular_entry_point_twice_in_a_row(n_streams):
    snlp, cfg, W, m, head = _setup(n_streams)
    for call, rows in enumerate((12, 5)):
        hL_np = synth.make_hidden(cfg, rows, 1, seed=100 + call)
        hL = torch.from_numpy(hL_np).cuda()
        logits, want = m.lm_head(hL, want_logits=True)
        out = torch.full((rows,), -7, dtype=torch.int32, device="cuda")   # pre-allocated by the caller
        got = snlp.lm_head_greedy_static(hL, head, n_streams, cfg.rms_eps, argmax=out)
        torch.cuda.synchronize()
        got, want, logits = got.cpu().numpy(), want.cpu().numpy(), logits.cpu().numpy().astype(np.float64)
        r = np.arange(rows)
        assert got.min() >= 0 and got.max() < cfg.vocab
        # same token as the regular entry point, except where that entry point's own margin is rounding noise
        noise = 1e-5 * np.abs(logits).max()
        margin = logits[r, want] - logits[r, got]
        assert np.all((got == want) | (margin <= noise)), (call, got, want, margin)
        # and against the oracle: the chosen logit is the fp64 maximum up to the bf16 error of the normalised input
        ref = O.lm_head(cfg, W, hL_np.astype(np.float64))[:, 0]
        tau = 2.0 * 2.0 ** -8 * np.sqrt(cfg.d_model) * float(np.max(np.linalg.norm(W.lm_head.astype(np.float64), axis=1)))
        assert np.all(ref.max(-1) - ref[r, got] <= tau), (call, ref.max(-1) - ref[r, got], tau)


def test_static_lm_head_rejects_sizes_beyond_its_fixed_scratch():
    snlp, cfg, W, m, head = _setup(1)
    hL = torch.zeros((17, 1, cfg.d_model), device="cuda")
    with pytest.raises(snlp.SnlpError) as e:
        snlp.lm_head_greedy_static(hL, head, 1, cfg.rms_eps)
    assert e.value.code == snlp.ERR_SHAPE and "exceed" in str(e.value)
    big_vocab = torch.zeros((262144 + 128, 32), dtype=torch.int16, device="cuda")
    with pytest.raises(snlp.SnlpError) as e:
        snlp.lm_head_greedy_static(torch.zeros((1, 1, 32), device="cuda"), big_vocab, 1, cfg.rms_eps)
    assert e.value.code == snlp.ERR_SHAPE
    with pytest.raises(snlp.SnlpError) as e:
        snlp.lm_head_greedy_static(torch.zeros((1, 1, 32), device="cuda"), torch.zeros((100, 32), dtype=torch.int16, device="cuda"),
                                   1, cfg.rms_eps)
    assert e.value.code == snlp.ERR_UNSUPPORTED
    torch.cuda.synchronize()


def _torch_logits(hL, head_bits, n_streams, eps):
    """fp32 logits of the same bf16 product on the GPU (plain torch ops: a test-side check, not the product path)."""
    x = hL.sum(dim=1) if hL.dim() == 3 else hL
    rstd = torch.rsqrt((x * x).mean(-1, keepdim=True) + eps)
    xb = x.to(torch.bfloat16).float()
    w = head_bits.view(torch.bfloat16).float()
    return (xb @ w.T) * rstd


@pytest.mark.parametrize("rows,d_model,vocab,n_streams", [(16, 4096, 2048, 1), (16, 32, 262144, 1), (9, 1280, 65536, 4)])
def test_static_lm_head_at_the_ends_of_its_limits(rows, d_model, vocab, n_streams):
    """The largest row count with the widest model (the two-tile variant with its large shared-memory request), the
    whole scratch array (largest vocabulary), and the benchmark's own head shape; and the property the entry point
    exists for: the device's free memory is the same before and after a call."""
    from paper_2605_17842_b200 import snlp
    g = torch.Generator(device="cuda").manual_seed(1234 + rows + d_model)
    hL = torch.randn((rows, n_streams, d_model), device="cuda", generator=g)
    head = (torch.randn((vocab, d_model), device="cuda", generator=g) * 0.05).to(torch.bfloat16).view(torch.int16)
    out = torch.full((rows,), -7, dtype=torch.int32, device="cuda")
    snlp.lm_head_greedy_static(hL, head, n_streams, 1e-6, argmax=out)      # first call on the device does the set-up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    out.fill_(-7)
    snlp.lm_head_greedy_static(hL, head, n_streams, 1e-6, argmax=out)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0, (free0, free1)
    logits = _torch_logits(hL, head, n_streams, 1e-6)
    got = out.long()
    assert int(got.min()) >= 0 and int(got.max()) < vocab
    top = logits.max(dim=-1).values
    chosen = logits.gather(1, got[:, None])[:, 0]
    # the chosen token is the maximum up to the rounding noise of two fp32 sums of d_model bf16 products
    assert bool(torch.all(top - chosen <= 2e-5 * logits.abs().max() + 1e-6)), (top - chosen)
