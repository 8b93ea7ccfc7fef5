"""Thin ctypes binding over libsnlp.so (argument marshalling only; every step runs in the CUDA library).

Importing this module loads the library and raises if it is missing: there is no fallback path.
Device memory is held in torch tensors; the current torch CUDA stream is passed to every call.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsnlp.so")

OK = 0
ERR_ARG, ERR_SHAPE, ERR_STATE, ERR_OOM, ERR_CUDA, ERR_TIMEOUT, ERR_UNSUPPORTED = -1, -2, -3, -4, -5, -6, -7
DTYPE_FP32, DTYPE_BF16 = 0, 1
MODE_IDN, MODE_HCN, MODE_NOCORR, MODE_SEQUENTIAL = 0, 1, 2, 3
INIT_H0, INIT_FWD = 0, 1

EXPORTS = [
    "snlp_create", "snlp_destroy", "snlp_load_weights", "snlp_embed", "snlp_forward_sequential",
    "snlp_forward_parallel", "snlp_forward_solver", "snlp_decode_step_solver", "snlp_lm_head", "snlp_kv_create", "snlp_kv_destroy", "snlp_kv_len",
    "snlp_kv_truncate", "snlp_prefill", "snlp_decode_step", "snlp_decode_step_host", "snlp_draft_and_verify", "snlp_set_flag",
    "snlp_launch_count", "snlp_kernel_times", "snlp_device_status", "snlp_lm_head_greedy_static", "snlp_last_error",
    "snlp_copy_trace", "snlp_draft_and_verify_async", "snlp_graph_count",
]


class Config(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layer", "d_model", "n_head", "head_dim", "d_ff", "vocab", "n_streams",
                                         "dtype", "max_rows", "max_batch", "max_ctx")] + \
               [("rms_eps", C.c_float), ("rope_base", C.c_float)]


class Solver(C.Structure):
    """snlp_solver: K sweeps, mode, sequential prefix S, initialisation, fused layers per chunk."""
    _fields_ = [(n, C.c_int32) for n in ("K", "mode", "prefix", "init", "fuse")]

    def __init__(self, K=1, mode=0, prefix=0, init=0, fuse=1):
        super().__init__(K, mode, prefix, init, fuse)


class Weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("embed", "lm_head", "wqkv", "wo", "wup", "wdn", "hc_res_attn", "hc_res_mlp",
                                          "hc_pre_attn", "hc_pre_mlp", "hc_post_attn", "hc_post_mlp")]


class SnlpError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"libsnlp error {code}: {msg}")
        self.code = code


def load_library(path: str = LIB_PATH) -> C.CDLL:
    if not os.path.exists(path):
        raise ImportError(f"{path} is missing: build it with `python -m paper_2605_17842_b200.build` "
                          "(there is no CPU or PyTorch fallback)")
    lib = C.CDLL(path)
    for name in EXPORTS:
        getattr(lib, name)  # AttributeError if a declared symbol is not exported
    lib.snlp_last_error.restype = C.c_char_p
    for name in EXPORTS:
        if name != "snlp_last_error":
            getattr(lib, name).restype = C.c_int
    return lib


_lib = load_library()


def _check(rc):
    if rc != OK:
        raise SnlpError(rc, _lib.snlp_last_error().decode())


def _ptr(t):
    if t is None:
        return C.c_void_p(0)
    assert t.is_cuda and t.is_contiguous()
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _bf16_bits(x: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    return (u >> 16).astype(np.uint16)


class KVCache:
    def __init__(self, model: "Model", B: int, max_ctx: int):
        self.model = model
        self.B = B
        self.max_ctx = max_ctx
        self._h = C.c_void_p()
        _check(_lib.snlp_kv_create(model._h, C.c_int(B), C.c_int(max_ctx), C.byref(self._h)))

    def __len__(self):
        n = C.c_int32()
        _check(_lib.snlp_kv_len(self._h, C.byref(n)))
        return n.value

    def truncate(self, new_len: int):
        _check(_lib.snlp_kv_truncate(self._h, C.c_int(new_len), _stream()))

    def close(self):
        if self._h:
            _lib.snlp_kv_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Model:
    """One model handle: snlp_create + snlp_load_weights, then the forward / decode entry points."""

    def __init__(self, cfg, max_rows: int, max_batch: int = 1, max_ctx: int | None = None):
        self.cfg = cfg
        self.n_layer, self.d_model, self.n_streams, self.vocab = cfg.n_layer, cfg.d_model, cfg.n_streams, cfg.vocab
        c = Config(cfg.n_layer, cfg.d_model, cfg.n_head, cfg.head_dim, cfg.d_ff, cfg.vocab, cfg.n_streams,
                   DTYPE_BF16 if cfg.dtype == "bf16" else DTYPE_FP32, max_rows, max_batch,
                   max_ctx if max_ctx is not None else max_rows, cfg.rms_eps, cfg.rope_base)
        self._h = C.c_void_p()
        _check(_lib.snlp_create(C.byref(c), C.byref(self._h)))

    def load_weights(self, W):
        """W: attribute bag of float32 numpy arrays (bf16-representable values when the model is bf16)."""
        keep = []

        def conv(a):
            if a is None:
                return C.c_void_p(0)
            a = _bf16_bits(a) if self.cfg.dtype == "bf16" else np.ascontiguousarray(a, dtype=np.float32)
            keep.append(a)
            return C.c_void_p(a.ctypes.data)

        def f32(a):
            if a is None:
                return C.c_void_p(0)
            a = np.ascontiguousarray(a, dtype=np.float32)
            keep.append(a)
            return C.c_void_p(a.ctypes.data)

        w = Weights(conv(W.embed), conv(W.lm_head), conv(W.wqkv), conv(W.wo), conv(W.wup), conv(W.wdn),
                    f32(getattr(W, "hc_res_attn", None)), f32(getattr(W, "hc_res_mlp", None)),
                    f32(getattr(W, "hc_pre_attn", None)), f32(getattr(W, "hc_pre_mlp", None)),
                    f32(getattr(W, "hc_post_attn", None)), f32(getattr(W, "hc_post_mlp", None)))
        _check(_lib.snlp_load_weights(self._h, C.byref(w)))

    # -- forward passes ---------------------------------------------------------------------------
    def embed(self, ids: torch.Tensor) -> torch.Tensor:
        B, T = ids.shape
        h0 = torch.empty((B, T, self.n_streams, self.d_model), dtype=torch.float32, device=ids.device)
        _check(_lib.snlp_embed(self._h, _ptr(ids), C.c_int(B), C.c_int(T), _ptr(h0), _stream()))
        return h0

    def _trace(self, h0):
        B, T = h0.shape[:2]
        return torch.empty((self.n_layer + 1, B, T, self.n_streams, self.d_model), dtype=torch.float32, device=h0.device)

    def forward_sequential(self, h0: torch.Tensor, want_trace: bool = True):
        B, T = h0.shape[:2]
        tr = self._trace(h0) if want_trace else None
        _check(_lib.snlp_forward_sequential(self._h, _ptr(h0), C.c_int(B), C.c_int(T), _ptr(tr), _stream()))
        return tr

    def forward_parallel(self, h0: torch.Tensor, K: int, mode: int = MODE_IDN, want_trace: bool = True,
                         want_resnorm: bool = True):
        B, T = h0.shape[:2]
        tr = self._trace(h0) if want_trace else None
        rn = torch.zeros((max(K, 1), self.n_layer, 2), dtype=torch.float32, device=h0.device) if want_resnorm else None
        _check(_lib.snlp_forward_parallel(self._h, _ptr(h0), C.c_int(B), C.c_int(T), C.c_int(K), C.c_int(mode),
                                          _ptr(tr), _ptr(rn), _stream()))
        return tr, rn

    def forward_solver(self, h0: torch.Tensor, solver: "Solver", want_trace: bool = True, want_resnorm: bool = True):
        B, T = h0.shape[:2]
        tr = self._trace(h0) if want_trace else None
        rn = torch.zeros((max(solver.K, 1), self.n_layer, 2), dtype=torch.float32, device=h0.device) if want_resnorm else None
        _check(_lib.snlp_forward_solver(self._h, _ptr(h0), C.c_int(B), C.c_int(T), C.byref(solver), _ptr(tr), _ptr(rn), _stream()))
        return tr, rn

    def decode_step_solver(self, kv: "KVCache", tok_in: torch.Tensor, solver: "Solver", tok_out: torch.Tensor | None = None):
        if tok_out is None:
            tok_out = torch.empty_like(tok_in)
        _check(_lib.snlp_decode_step_solver(self._h, kv._h, _ptr(tok_in), C.byref(solver), _ptr(tok_out), C.c_void_p(0), _stream()))
        return tok_out

    def lm_head(self, hL: torch.Tensor, want_logits: bool = True):
        rows = hL.numel() // (self.n_streams * self.d_model)
        logits = torch.empty((rows, self.vocab), dtype=torch.float32, device=hL.device) if want_logits else None
        arg = torch.empty((rows,), dtype=torch.int32, device=hL.device)
        _check(_lib.snlp_lm_head(self._h, _ptr(hL), C.c_int(rows), _ptr(logits), _ptr(arg), _stream()))
        return logits, arg

    # -- decoding ---------------------------------------------------------------------------------
    def kv_cache(self, B: int, max_ctx: int) -> KVCache:
        return KVCache(self, B, max_ctx)

    def prefill(self, kv: KVCache, ids: torch.Tensor) -> torch.Tensor:
        B, T = ids.shape
        out = torch.empty((B,), dtype=torch.int32, device=ids.device)
        _check(_lib.snlp_prefill(self._h, kv._h, _ptr(ids), C.c_int(B), C.c_int(T), _ptr(out), _stream()))
        return out

    def decode_step(self, kv: KVCache, tok_in: torch.Tensor, K: int, mode: int = MODE_IDN,
                    tok_out: torch.Tensor | None = None, resnorm: torch.Tensor | None = None) -> torch.Tensor:
        if tok_out is None:
            tok_out = torch.empty_like(tok_in)
        _check(_lib.snlp_decode_step(self._h, kv._h, _ptr(tok_in), C.c_int(K), C.c_int(mode), _ptr(tok_out),
                                     _ptr(resnorm), _stream()))
        return tok_out

    def decode_step_host(self, kv: KVCache, tok_in, K: int, mode: int = MODE_IDN, tok_out=None):
        """decode_step on HOST int32 tensors (CPU, pinned or not): copies in, step, copies out, synchronises."""
        if tok_out is None:
            tok_out = torch.empty_like(tok_in)
        assert tok_in.device.type == "cpu" and tok_out.device.type == "cpu" and tok_in.dtype == torch.int32 and tok_out.dtype == torch.int32
        _check(_lib.snlp_decode_step_host(self._h, kv._h, C.c_void_p(tok_in.data_ptr()), C.c_int(K), C.c_int(mode),
                                          C.c_void_p(tok_out.data_ptr()), _stream()))
        return tok_out

    def draft_and_verify(self, kv: KVCache, last_tok: torch.Tensor, block: int, K: int, mode: int = MODE_IDN):
        """Returns (emitted list, n_accepted); last_tok is updated in place."""
        dev = last_tok.device
        emitted = torch.empty((block + 1,), dtype=torch.int32, device=dev)
        counts = torch.zeros((2,), dtype=torch.int32, device=dev)
        _check(_lib.snlp_draft_and_verify(self._h, kv._h, _ptr(last_tok), C.c_int(block), C.c_int(K), C.c_int(mode),
                                          _ptr(emitted), C.c_void_p(counts.data_ptr()), C.c_void_p(counts.data_ptr() + 4),
                                          _stream()))
        n_emit, n_acc = counts.tolist()
        return emitted[:n_emit].tolist(), n_acc

    def draft_and_verify_async(self, kv: KVCache, last_tok: torch.Tensor, block: int, K: int, mode: int = MODE_IDN,
                               emitted: torch.Tensor | None = None, counts: torch.Tensor | None = None):
        """One round with no host synchronisation.  Returns (emitted [block+1] int32, counts [2] int32 =
        (n_emitted, n_accepted)), both still on the device; last_tok is updated in place."""
        dev = last_tok.device
        if emitted is None:
            emitted = torch.empty((block + 1,), dtype=torch.int32, device=dev)
        if counts is None:
            counts = torch.zeros((2,), dtype=torch.int32, device=dev)
        _check(_lib.snlp_draft_and_verify_async(self._h, kv._h, _ptr(last_tok), C.c_int(block), C.c_int(K), C.c_int(mode),
                                                _ptr(emitted), C.c_void_p(counts.data_ptr()), C.c_void_p(counts.data_ptr() + 4),
                                                _stream()))
        return emitted, counts

    def copy_trace(self, rows: int) -> torch.Tensor:
        """The states [L+1, rows, n, d] of the handle's last forward / prefill chunk / decode step / verify block."""
        tr = torch.empty((self.n_layer + 1, rows, self.n_streams, self.d_model), dtype=torch.float32, device="cuda")
        _check(_lib.snlp_copy_trace(self._h, C.c_int(rows), _ptr(tr), _stream()))
        return tr

    def graph_count(self) -> int:
        n = C.c_int64()
        _check(_lib.snlp_graph_count(self._h, C.byref(n)))
        return n.value

    # -- misc -------------------------------------------------------------------------------------
    def set_flag(self, flag: int, value: int):
        _check(_lib.snlp_set_flag(self._h, C.c_int(flag), C.c_int(value)))

    def device_status(self):
        """Synchronise and raise SnlpError(ERR_TIMEOUT) if a kernel gave up on a bounded device-side wait."""
        _check(_lib.snlp_device_status(self._h, _stream()))

    def launch_count(self) -> int:
        n = C.c_int64()
        _check(_lib.snlp_launch_count(self._h, C.byref(n)))
        return n.value

    KERNEL_CLASSES = ("qkv", "attention", "out_proj", "mlp_up", "mlp_down", "correction", "lm_head", "other")

    def kernel_times(self, reset: bool = True):
        """{class: (milliseconds, launches)} of the launches timed since set_flag(2, 1)."""
        ms = (C.c_double * 8)()
        n = (C.c_int64 * 8)()
        _check(_lib.snlp_kernel_times(self._h, ms, n, C.c_int(1 if reset else 0)))
        return {k: (ms[i], n[i]) for i, k in enumerate(self.KERNEL_CLASSES)}

    def close(self):
        if self._h:
            _lib.snlp_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def lm_head_greedy_static(hL: torch.Tensor, lm_head_bf16: torch.Tensor, n_streams: int, rms_eps: float,
                          argmax: torch.Tensor | None = None) -> torch.Tensor:
    """Greedy LM head through the entry point that allocates nothing inside the library.

    hL: cuda fp32 [rows, n_streams, d]; lm_head_bf16: cuda bf16 (or int16/uint16 bit patterns) [vocab, d].
    Pass a pre-allocated int32 `argmax` tensor to keep the whole call free of allocations."""
    vocab, d = lm_head_bf16.shape
    rows = hL.numel() // (n_streams * d)
    if argmax is None:
        argmax = torch.empty((rows,), dtype=torch.int32, device=hL.device)
    _check(_lib.snlp_lm_head_greedy_static(_ptr(hL), _ptr(lm_head_bf16), C.c_int(rows), C.c_int(n_streams), C.c_int(d),
                                           C.c_int(vocab), C.c_float(rms_eps), _ptr(argmax), _stream()))
    return argmax


def raw_library() -> C.CDLL:
    """The ctypes handle itself, for tests of the C ABI's error paths."""
    return _lib
