"""Error behaviour of the C ABI (called through ctypes exactly as a C caller would)."""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2605_17842_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    from paper_2605_17842_b200 import snlp
    cfg = synth.CONFIGS["tiny"]
    W = synth.make_weights(cfg)
    return snlp, cfg, W


def test_error_codes(env):
    snlp, cfg, W = env
    lib = snlp.raw_library()
    # bad configs
    h = C.c_void_p()
    bad = snlp.Config(4, 64, 3, 32, 256, 256, 1, 0, 16, 1, 16, 1e-6, 10000.0)   # 3*32 != 64
    assert lib.snlp_create(C.byref(bad), C.byref(h)) == snlp.ERR_ARG
    assert b"n_head" in lib.snlp_last_error()
    assert lib.snlp_create(None, C.byref(h)) == snlp.ERR_ARG
    # calls before load_weights
    m = snlp.Model(cfg, max_rows=16, max_batch=1, max_ctx=16)
    h0 = torch.zeros((1, 16, 1, 64), device="cuda")
    with pytest.raises(snlp.SnlpError) as e:
        m.forward_sequential(h0)
    assert e.value.code == snlp.ERR_STATE
    # missing hc arrays for a multi-stream model
    cfg4 = synth.ModelConfig(2, 64, 2, 32, 128, 64, 4, "fp32")
    m4 = snlp.Model(cfg4, max_rows=4)
    with pytest.raises(snlp.SnlpError) as e:
        m4.load_weights(W)   # W has hc_* = None
    assert e.value.code == snlp.ERR_ARG
    m.load_weights(W)
    # K < 1, unknown mode, NULL h0
    for K, mode, code in ((0, 0, snlp.ERR_ARG), (-1, 0, snlp.ERR_ARG), (1, 7, snlp.ERR_ARG)):
        with pytest.raises(snlp.SnlpError) as e:
            m.forward_parallel(h0, K, mode)
        assert e.value.code == code
    assert lib.snlp_forward_parallel(m._h, None, 1, 16, 1, 0, None, None, None) == snlp.ERR_ARG
    # shape limits
    big = torch.zeros((1, 17, 1, 64), device="cuda")
    with pytest.raises(snlp.SnlpError) as e:
        m.forward_sequential(big)
    assert e.value.code == snlp.ERR_SHAPE
    with pytest.raises(snlp.SnlpError) as e:
        m.kv_cache(2, 16)            # B > max_batch
    assert e.value.code == snlp.ERR_SHAPE
    with pytest.raises(snlp.SnlpError) as e:
        m.kv_cache(1, 17)            # ctx > max_ctx
    assert e.value.code == snlp.ERR_SHAPE
    kv = m.kv_cache(1, 16)
    ids = torch.zeros((1, 16), dtype=torch.int32, device="cuda")
    m.prefill(kv, ids)
    assert len(kv) == 16
    with pytest.raises(snlp.SnlpError) as e:
        m.decode_step(kv, ids[:, 0].contiguous(), 0)     # cache full
    assert e.value.code == snlp.ERR_SHAPE
    with pytest.raises(snlp.SnlpError) as e:
        kv.truncate(17)
    assert e.value.code == snlp.ERR_ARG
    kv.truncate(4)
    with pytest.raises(snlp.SnlpError) as e:
        m.draft_and_verify(kv, ids[0, :1].contiguous(), 0, 1)   # block < 1
    assert e.value.code == snlp.ERR_ARG
    with pytest.raises(snlp.SnlpError) as e:
        m.draft_and_verify(kv, ids[0, :1].contiguous(), 12, 1)  # 4 + 13 > 16
    assert e.value.code == snlp.ERR_SHAPE
    # K > L is allowed
    tr, _ = m.forward_parallel(h0, cfg.n_layer + 3, 0)
    assert torch.isfinite(tr).all()
    # the context is still healthy after all the refused calls
    torch.cuda.synchronize()


def test_cache_may_outlive_its_model(env):
    snlp, cfg, W = env
    m = snlp.Model(cfg, max_rows=16, max_batch=1, max_ctx=16)
    m.load_weights(W)
    kv = m.kv_cache(1, 16)
    ids = torch.zeros((1, 4), dtype=torch.int32, device="cuda")
    t = m.prefill(kv, ids)
    m.decode_step(kv, t, 2)          # leaves a captured graph that refers to the cache
    torch.cuda.synchronize()
    m.close()                        # model first ...
    with pytest.raises(snlp.SnlpError) as e:
        kv.truncate(1)
    assert e.value.code == snlp.ERR_STATE
    kv.close()                       # ... then the cache: must not touch the freed model
