"""The allocation-free greedy LM head (snlp_lm_head_greedy_static) against the regular snlp_lm_head.

This file is named so that pytest collects it last: the regular entry points are exercised first.
The two calls in a row use different row counts and inputs, so anything the first call leaves in the
library's fixed scratch array must not leak into the second result."""
import numpy as np
import pytest
import torch

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
    return snlp, cfg, m, head


@pytest.mark.parametrize("n_streams", [1, 4])
def test_static_lm_head_matches_regular_entry_point_twice_in_a_row(n_streams):
    snlp, cfg, m, head = _setup(n_streams)
    for call, rows in enumerate((12, 5)):
        hL = torch.from_numpy(synth.make_hidden(cfg, rows, 1, seed=100 + call)).cuda()
        _, want = m.lm_head(hL, want_logits=False)
        out = torch.full((rows,), -7, dtype=torch.int32, device="cuda")   # pre-allocated by the caller
        got = snlp.lm_head_greedy_static(hL, head, n_streams, cfg.rms_eps, argmax=out)
        torch.cuda.synchronize()
        assert torch.equal(got, want), (call, got, want)     # integer outputs: exact
        assert got.min().item() >= 0


def test_static_lm_head_rejects_sizes_beyond_its_fixed_scratch():
    snlp, cfg, m, head = _setup(1)
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
