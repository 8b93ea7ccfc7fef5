"""GPU parity of the general solver options: sequential prefix S and the fwd initialisation (Alg. 2 general
form), against the oracle and against the library's own sequential forward."""
import numpy as np
import pytest
import torch

from oracle import snlp_oracle as O
from paper_2605_17842_b200 import synth
from tests.gpu_util import TOL, dev, layer_relerr, make_model, trace_err

pytestmark = pytest.mark.gpu

CASES = {
    "f32": (synth.ModelConfig(5, 64, 2, 32, 128, 128, 1, "fp32"), 2, 9),
    "f32_hc": (synth.ModelConfig(4, 64, 2, 32, 128, 128, 3, "fp32"), 1, 7),
    "bf16_decode": (synth.ModelConfig(5, 256, 2, 128, 512, 1024, 1, "bf16"), 2, 5),
    "bf16_prefill": (synth.ModelConfig(4, 256, 2, 128, 512, 1024, 1, "bf16"), 1, 140),
}


@pytest.mark.parametrize("name", list(CASES))
def test_prefix_and_fwd_init_match_oracle(name):
    from paper_2605_17842_b200 import snlp
    cfg, B, T = CASES[name]
    W = synth.make_weights(cfg, seed=1234, std=0.05, embed_std=1.0)
    h0 = synth.make_hidden(cfg, B, T, seed=7)
    m = make_model(cfg, W, max_rows=B * T, max_batch=B)
    mode = O.MODE_HCN if cfg.n_streams > 1 else O.MODE_IDN
    seq = m.forward_sequential(dev(h0))
    for S, init, K in [(2, O.INIT_H0, 1), (2, O.INIT_FWD, 1), (0, O.INIT_FWD, 2), (3, O.INIT_H0, 2), (0, O.INIT_FWD, 0)]:
        want, want_res = O.forward_snlp(cfg, W, h0.astype(np.float64), K, mode, S=S, init=init)
        tr, rn = m.forward_solver(dev(h0), snlp.Solver(K=K, mode=mode, prefix=S, init=init))
        assert trace_err(tr.cpu().numpy(), want, TOL[cfg.dtype]) <= TOL[cfg.dtype], (S, init, K)
        if K > 0:
            gr, wr = np.sqrt(rn.cpu().numpy()[:K, :, 0]), np.sqrt(want_res[..., 0])
            scale = np.sqrt(want_res[..., 1]).max() + 1e-30
            assert np.max(np.abs(gr - wr)) / scale <= 2 * TOL[cfg.dtype], (S, init, K)
        # finite-step exactness on the GPU, bit for bit: states 0 .. S + K (+1 with fwd) equal the sequential trace
        exact = min(cfg.n_layer, S + K + (1 if init == O.INIT_FWD else 0))
        assert torch.equal(tr[:exact + 1], seq[:exact + 1]), (S, init, K)
    # prefix = L and the sequential mode are Algorithm 1
    tr, _ = m.forward_solver(dev(h0), snlp.Solver(K=0, mode=mode, prefix=cfg.n_layer))
    assert torch.equal(tr, seq)
    tr, _ = m.forward_solver(dev(h0), snlp.Solver(K=3, mode=snlp.MODE_SEQUENTIAL))
    assert torch.equal(tr, seq)
    m.device_status()


def test_solver_argument_errors():
    from paper_2605_17842_b200 import snlp
    cfg, B, T = CASES["f32"]
    W = synth.make_weights(cfg, seed=1234)
    m = make_model(cfg, W, max_rows=B * T, max_batch=B)
    h0 = dev(synth.make_hidden(cfg, B, T, seed=7))
    for bad in (snlp.Solver(K=-1), snlp.Solver(K=1, prefix=6), snlp.Solver(K=1, init=2), snlp.Solver(K=1, fuse=0),
                snlp.Solver(K=1, mode=9), snlp.Solver(K=1, fuse=2, prefix=0)):   # 5 layers are not a multiple of 2
        with pytest.raises(snlp.SnlpError) as e:
            m.forward_solver(h0, bad)
        assert e.value.code == snlp.ERR_ARG


@pytest.mark.parametrize("name", list(CASES))
def test_zero_sweeps_return_the_initialisation(name):
    """K = 0 with the h0 initialisation: states 0..S are the sequential ones and every later state is a copy of h_S
    (Alg. 2 line 5 with nothing after it).  The tensor-core path does not write those copies when a sweep follows, so
    this is the one call in which it has to."""
    from paper_2605_17842_b200 import snlp
    cfg, B, T = CASES[name]
    W = synth.make_weights(cfg, seed=1234, std=0.05, embed_std=1.0)
    h0 = synth.make_hidden(cfg, B, T, seed=7)
    m = make_model(cfg, W, max_rows=B * T, max_batch=B)
    mode = O.MODE_HCN if cfg.n_streams > 1 else O.MODE_IDN
    seq = m.forward_sequential(dev(h0))
    m.forward_solver(dev(h0), snlp.Solver(K=2, mode=mode))     # leave other values in the trace first
    for S in (0, 2):
        tr, _ = m.forward_solver(dev(h0), snlp.Solver(K=0, mode=mode, prefix=S))
        assert torch.equal(tr[: S + 1], seq[: S + 1])
        for l in range(S + 1, cfg.n_layer + 1):
            assert torch.equal(tr[l], tr[S]), (S, l)
    m.device_status()


def test_decode_step_with_prefix_and_fwd_init():
    from paper_2605_17842_b200 import snlp
    cfg = synth.ModelConfig(5, 256, 2, 128, 512, 1024, 1, "bf16")
    W = synth.make_weights(cfg, seed=1234, std=0.05, embed_std=1.0)
    m = make_model(cfg, W, max_rows=32, max_batch=2, max_ctx=64)
    ids = dev(synth.make_ids(cfg, 2, 20, seed=5))
    kv = m.kv_cache(2, 64)
    first = m.prefill(kv, ids)
    ref = [m.decode_step(kv, first, 0).clone()]
    ref.append(m.decode_step(kv, ref[-1], 0).clone())
    # prefix 3 + 2 sweeps covers the 2 suffix layers exactly; fwd init + 1 sweep + prefix 3 as well
    for sol in (snlp.Solver(K=2, prefix=3), snlp.Solver(K=1, prefix=3, init=snlp.INIT_FWD), snlp.Solver(K=0, prefix=5)):
        kv.truncate(20)
        a = m.decode_step_solver(kv, first, sol).clone()
        b = m.decode_step_solver(kv, a, sol).clone()
        assert torch.equal(a, ref[0]) and torch.equal(b, ref[1])
    assert len(kv) == 22


FUSED = {
    "f32": (synth.ModelConfig(6, 64, 2, 32, 128, 128, 1, "fp32"), 2, 9),
    "bf16_decode": (synth.ModelConfig(6, 256, 2, 128, 512, 1024, 1, "bf16"), 2, 5),
    "bf16_prefill": (synth.ModelConfig(6, 256, 2, 128, 640, 1024, 1, "bf16"), 1, 140),
}


@pytest.mark.parametrize("name", list(FUSED))
def test_fused_chunks_match_oracle(name):
    """Chunkwise SNLP with fused layers (NxFM): the chunk-boundary states against the oracle's forward_chunked."""
    from paper_2605_17842_b200 import snlp
    cfg, B, T = FUSED[name]
    W = synth.make_weights(cfg, seed=1234, std=0.05, embed_std=1.0)
    h0 = synth.make_hidden(cfg, B, T, seed=7)
    m = make_model(cfg, W, max_rows=B * T, max_batch=B)
    L = cfg.n_layer
    for S, F, K, init in [(0, 2, 1, O.INIT_H0), (0, 2, 2, O.INIT_H0), (0, 3, 1, O.INIT_FWD), (2, 2, 1, O.INIT_H0), (0, 6, 1, O.INIT_H0)]:
        want = O.forward_chunked(cfg, W, h0.astype(np.float64), K, F, S=S, init=init)
        tr, _ = m.forward_solver(dev(h0), snlp.Solver(K=K, mode=O.MODE_IDN, prefix=S, init=init, fuse=F))
        got = tr.cpu().numpy()[S::F]
        assert got.shape[0] == len(want)
        assert trace_err(got, np.stack(want), TOL[cfg.dtype]) <= TOL[cfg.dtype], (S, F, K, init)
        # sequential execution of the same fused model, and chunkwise finite-step exactness against it (bit for bit)
        fseq_want = O.forward_chunked(cfg, W, h0.astype(np.float64), None, F, S=S)
        fseq, _ = m.forward_solver(dev(h0), snlp.Solver(K=0, mode=snlp.MODE_SEQUENTIAL, prefix=S, fuse=F))
        assert trace_err(fseq.cpu().numpy()[S::F], np.stack(fseq_want), TOL[cfg.dtype]) <= TOL[cfg.dtype], (S, F)
        nexact = min((L - S) // F, K + (1 if init == O.INIT_FWD else 0))
        assert torch.equal(tr[S::F][:nexact + 1], fseq[S::F][:nexact + 1]), (S, F, K, init)
    # fuse = 1 through the same entry point is the unfused algorithm
    a, _ = m.forward_solver(dev(h0), snlp.Solver(K=2, mode=O.MODE_IDN, fuse=1))
    b, _ = m.forward_parallel(dev(h0), 2, O.MODE_IDN)
    assert torch.equal(a, b)
    # without correction (A = 0) information moves one chunk per sweep
    want = O.forward_chunked(cfg, W, h0.astype(np.float64), 1, 2, correct=False)
    tr, _ = m.forward_solver(dev(h0), snlp.Solver(K=1, mode=O.MODE_NOCORR, fuse=2))
    assert trace_err(tr.cpu().numpy()[0::2], np.stack(want), TOL[cfg.dtype]) <= TOL[cfg.dtype]
    m.device_status()


def test_fused_decode_steps_are_consistent():
    """Decoding with fused chunks: enough sweeps reproduce sequential execution of the fused model, token for token."""
    from paper_2605_17842_b200 import snlp
    cfg = synth.ModelConfig(6, 256, 2, 128, 512, 1024, 1, "bf16")
    W = synth.make_weights(cfg, seed=1234, std=0.05, embed_std=1.0)
    m = make_model(cfg, W, max_rows=32, max_batch=2, max_ctx=64)
    ids = dev(synth.make_ids(cfg, 2, 20, seed=5))
    kv = m.kv_cache(2, 64)
    first = m.prefill(kv, ids)
    seq = snlp.Solver(K=0, mode=snlp.MODE_SEQUENTIAL, fuse=2)
    ref = [m.decode_step_solver(kv, first, seq).clone()]
    ref.append(m.decode_step_solver(kv, ref[-1], seq).clone())
    kv.truncate(20)
    sol = snlp.Solver(K=3, mode=O.MODE_IDN, fuse=2)     # 3 chunks, 3 sweeps: exact
    a = m.decode_step_solver(kv, first, sol).clone()
    b = m.decode_step_solver(kv, a, sol).clone()
    assert torch.equal(a, ref[0]) and torch.equal(b, ref[1])
    with pytest.raises(snlp.SnlpError) as e:
        m.decode_step_solver(kv, first, snlp.Solver(K=1, mode=O.MODE_HCN, fuse=2))
    assert e.value.code == snlp.ERR_ARG
