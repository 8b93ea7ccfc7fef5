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


def test_injected_device_error_is_reported_once(env):
    """Failure detection without a GPU fault: the host writes the error word that a kernel raises when a bounded
    wait expires; snlp_device_status must report SNLP_ERR_TIMEOUT for it exactly once and the handle keeps working."""
    snlp, cfg, W = env
    m = snlp.Model(cfg, max_rows=16, max_batch=1, max_ctx=16)
    m.load_weights(W)
    h0 = torch.from_numpy(synth.make_hidden(cfg, 1, 16, seed=3)).cuda()
    before = m.forward_sequential(h0)
    m.device_status()                       # healthy
    m.set_flag(3, 1)                        # inject
    with pytest.raises(snlp.SnlpError) as e:
        m.device_status()
    assert e.value.code == snlp.ERR_TIMEOUT and "bounded wait" in str(e.value)
    m.device_status()                       # cleared by the report
    m.set_flag(3, 1)
    m.set_flag(3, 0)                        # the hook can also take it back
    m.device_status()
    after = m.forward_sequential(h0)
    assert torch.equal(before, after)
    m.close()


def test_misaligned_pointers_are_rejected_on_the_host(env):
    snlp, cfg, W = env
    lib = snlp.raw_library()
    m = snlp.Model(cfg, max_rows=16, max_batch=1, max_ctx=16)
    m.load_weights(W)
    buf = torch.zeros((16 * 64 + 8,), device="cuda")
    tr = torch.zeros((5 * 16 * 64 + 8,), device="cuda")
    odd = C.c_void_p(buf.data_ptr() + 4)    # 4-byte aligned only
    ok = C.c_void_p(buf.data_ptr())
    assert lib.snlp_forward_sequential(m._h, odd, 1, 16, None, None) == snlp.ERR_ARG
    assert b"aligned" in lib.snlp_last_error()
    assert lib.snlp_forward_sequential(m._h, ok, 1, 16, C.c_void_p(tr.data_ptr() + 8), None) == snlp.ERR_ARG
    assert lib.snlp_forward_parallel(m._h, odd, 1, 16, 1, 0, None, None, None) == snlp.ERR_ARG
    assert lib.snlp_lm_head(m._h, odd, 1, None, ok, None) == snlp.ERR_ARG
    ids = torch.zeros((8,), dtype=torch.int32, device="cuda")
    kv = m.kv_cache(1, 16)
    assert lib.snlp_decode_step(m._h, kv._h, C.c_void_p(ids.data_ptr() + 2), 0, 0, C.c_void_p(ids.data_ptr()), None, None) == snlp.ERR_ARG
    assert lib.snlp_copy_trace(m._h, 1, None, None) == snlp.ERR_ARG
    assert lib.snlp_copy_trace(m._h, 1, ok, None) == snlp.ERR_STATE       # nothing has run on this handle yet
    m.forward_sequential(buf[:16 * 64].view(1, 16, 1, 64))
    assert lib.snlp_copy_trace(m._h, 3, C.c_void_p(tr.data_ptr()), None) == snlp.ERR_SHAPE
    assert lib.snlp_copy_trace(m._h, 16, C.c_void_p(tr.data_ptr()), None) == snlp.OK
    lm = torch.zeros((128 * 32 + 8,), dtype=torch.int16, device="cuda")
    out = torch.zeros((4,), dtype=torch.int32, device="cuda")
    rc = lib.snlp_lm_head_greedy_static(C.c_void_p(buf.data_ptr() + 4), C.c_void_p(lm.data_ptr()), 1, 1, 32, 128, C.c_float(1e-6),
                                        C.c_void_p(out.data_ptr()), None)
    assert rc == snlp.ERR_ARG
    rc = lib.snlp_lm_head_greedy_static(C.c_void_p(buf.data_ptr()), C.c_void_p(lm.data_ptr() + 2), 1, 1, 32, 128, C.c_float(1e-6),
                                        C.c_void_p(out.data_ptr()), None)
    assert rc == snlp.ERR_ARG
    torch.cuda.synchronize()
    kv.close()
    m.close()


def test_decode_graphs_are_not_keyed_on_the_token_buffers():
    """300 steps, each with a fresh output tensor (what a plain caller of the binding does): one captured graph per
    attention grid size, not one per step, and the same tokens as with one fixed buffer."""
    from paper_2605_17842_b200 import snlp
    cfg = synth.ModelConfig(2, 256, 2, 128, 512, 1024, 1, "bf16")
    W = synth.make_weights(cfg, seed=1234, std=0.05, embed_std=1.0)
    m = snlp.Model(cfg, max_rows=16, max_batch=1, max_ctx=400)
    m.load_weights(W)
    ids = torch.from_numpy(synth.make_ids(cfg, 1, 16, seed=2)).cuda()
    kv = m.kv_cache(1, 400)
    t0 = m.prefill(kv, ids)
    keep = []                                # hold every tensor so the allocator must hand out new addresses
    t = t0
    for _ in range(300):
        t = m.decode_step(kv, t, 2)
        keep.append(t)
    torch.cuda.synchronize()
    assert len({x.data_ptr() for x in keep}) == 300
    chunks = (16 + 300 - 1) // 256 + 1       # 256-key chunks of the split-KV attention (2 heads x 1 sequence)
    assert m.graph_count() == chunks, m.graph_count()
    fresh = torch.stack(keep).flatten().tolist()
    kv.truncate(16)
    t = t0.clone()
    fixed = []
    for _ in range(300):
        m.decode_step(kv, t, 2, tok_out=t)
        fixed.append(int(t.item()))
    assert m.graph_count() == chunks
    assert fresh == fixed
    m.device_status()
    m.close()
