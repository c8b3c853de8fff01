"""Thin ctypes binding over the C ABI declared in include/ssd.h.

Argument marshalling only: every step of the verify path runs in the CUDA library.  torch is used
for device memory and streams.  There is no CPU fallback: if the library is missing or no CUDA
device is present, calls raise.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence, Tuple

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libssd_b200.so")
_lib = None

EXPORTS = [
    "ssd_model_arena_bytes", "ssd_model_create", "ssd_model_destroy", "ssd_kv_bytes",
    "ssd_workspace_bytes", "ssd_streams_create", "ssd_streams_destroy", "ssd_streams_set_path",
    "ssd_streams_set_activation_split",
    "ssd_streams_set_attention_kernel",
    "ssd_streams_set_trace", "ssd_forward", "ssd_fast_plan_host",
    "ssd_fast_pack_roundtrip_host", "ssd_kv_truncate",
    "ssd_streams_get_state", "ssd_prefill", "ssd_draft_step", "ssd_verify", "ssd_verify_host",
    "ssd_kv_commit", "ssd_kv_restore", "ssd_accept_noalloc", "ssd_streams_inject_failure",
    "ssd_tc_gemm_scratch_bytes", "ssd_tc_gemm_check", "ssd_iteration", "ssd_paged_kv_bytes",
    "ssd_paged_workspace_bytes", "ssd_streams_create_paged", "ssd_paged_state",
    "ssd_model_create_inherited", "ssd_model_inherited_arena_bytes",
    "ssd_kernel_launch_count",
    "ssd_last_status", "ssd_last_cuda_error", "ssd_strerror",
]


class ModelConfig(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("n_layers", "d_model", "n_q_heads", "n_kv_heads", "head_dim", "d_ffn",
                 "vocab_out", "vocab_text")] + \
               [("rope_theta", ctypes.c_float), ("rms_eps", ctypes.c_float),
                ("weight_dtype", ctypes.c_int32), ("qkv_bias", ctypes.c_int32)]


class VerifyParams(ctypes.Structure):
    _fields_ = [("gamma", ctypes.c_int32), ("temperature", ctypes.c_float),
                ("top_k", ctypes.c_int32), ("beta", ctypes.c_float), ("top_p", ctypes.c_float),
                ("ras_window", ctypes.c_int32), ("ras_tau", ctypes.c_float),
                ("dev_recent_tokens", ctypes.c_void_p)]


class LoopIo(ctypes.Structure):
    """ssd_loop_io of include/ssd.h: device pointers of the device-resident SSD iteration."""
    _fields_ = [("dev_uniform_pool", ctypes.c_void_p), ("n_iterations", ctypes.c_int32),
                ("dev_iteration", ctypes.c_void_p), ("dev_in_ids", ctypes.c_void_p),
                ("dev_draft_tokens", ctypes.c_void_p), ("dev_draft_probs", ctypes.c_void_p),
                ("dev_accepted_len", ctypes.c_void_p), ("dev_next_token", ctypes.c_void_p),
                ("dev_out_tokens", ctypes.c_void_p), ("out_capacity", ctypes.c_int32),
                ("dev_out_count", ctypes.c_void_p), ("dev_accept_log", ctypes.c_void_p)]


class SsdError(RuntimeError):
    pass


def lib() -> ctypes.CDLL:
    """Loads libssd_b200.so (built in-tree by `python -m paper_2505_15380_b200.build`)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise SsdError(f"{LIB_PATH} is missing: build it with `python -m paper_2505_15380_b200.build`")
    L = ctypes.CDLL(LIB_PATH)
    vp, sz, i32 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int32
    cfgp, parp = ctypes.POINTER(ModelConfig), ctypes.POINTER(VerifyParams)
    L.ssd_model_arena_bytes.restype = sz
    L.ssd_model_arena_bytes.argtypes = [cfgp]
    L.ssd_model_create.argtypes = [cfgp, vp, sz, vp, sz, ctypes.POINTER(vp)]
    L.ssd_model_create_inherited.argtypes = [vp, vp, i32, vp, sz, ctypes.POINTER(vp)]
    L.ssd_model_inherited_arena_bytes.restype = sz
    L.ssd_model_inherited_arena_bytes.argtypes = [vp, i32]
    L.ssd_model_destroy.restype = None
    L.ssd_model_destroy.argtypes = [vp]
    L.ssd_kv_bytes.restype = sz
    L.ssd_kv_bytes.argtypes = [cfgp, i32, i32]
    L.ssd_workspace_bytes.restype = sz
    L.ssd_workspace_bytes.argtypes = [cfgp, i32, i32, i32]
    L.ssd_streams_create.argtypes = [vp, i32, i32, i32, vp, sz, vp, sz, ctypes.POINTER(vp)]
    L.ssd_streams_destroy.restype = None
    L.ssd_streams_destroy.argtypes = [vp]
    L.ssd_streams_set_path.argtypes = [vp, i32]
    L.ssd_streams_set_activation_split.argtypes = [vp, i32]
    L.ssd_streams_set_attention_kernel.argtypes = [vp, i32]
    L.ssd_streams_set_trace.argtypes = [vp, vp, i32, i32]
    L.ssd_forward.argtypes = [vp, vp, vp, i32, vp, vp]
    L.ssd_fast_plan_host.argtypes = [cfgp, i32, ctypes.POINTER(ctypes.c_int64)]
    L.ssd_fast_pack_roundtrip_host.argtypes = [cfgp, i32, vp, sz, vp, ctypes.POINTER(ctypes.c_int64)]
    L.ssd_kv_truncate.argtypes = [vp, vp, vp, vp]
    L.ssd_streams_get_state.argtypes = [vp, vp, vp, vp]
    L.ssd_prefill.argtypes = [vp, vp, vp, vp, vp]
    L.ssd_draft_step.argtypes = [vp, vp, vp, i32, vp, parp, vp, vp, vp]
    L.ssd_verify.argtypes = [vp, vp, vp, vp, vp, parp, vp, vp, vp, vp]
    L.ssd_verify_host.argtypes = [vp, vp, vp, vp, vp, parp, vp, vp, vp]
    L.ssd_kv_commit.argtypes = [vp, vp, vp, vp]
    L.ssd_kv_restore.argtypes = [vp, vp, vp, vp]
    L.ssd_accept_noalloc.argtypes = [vp, vp, vp, vp, parp, i32, i32, vp, vp, vp]
    L.ssd_streams_inject_failure.argtypes = [vp, vp]
    L.ssd_iteration.argtypes = [vp, vp, vp, vp, parp, ctypes.POINTER(LoopIo), vp]
    L.ssd_paged_kv_bytes.restype = sz
    L.ssd_paged_kv_bytes.argtypes = [cfgp, i32]
    L.ssd_paged_workspace_bytes.restype = sz
    L.ssd_paged_workspace_bytes.argtypes = [cfgp, i32, i32, i32, i32]
    L.ssd_streams_create_paged.argtypes = [vp, i32, i32, i32, i32, vp, sz, vp, sz, ctypes.POINTER(vp)]
    L.ssd_paged_state.argtypes = [vp, vp, vp, vp, vp]
    L.ssd_tc_gemm_scratch_bytes.restype = sz
    L.ssd_tc_gemm_scratch_bytes.argtypes = [i32, i32, i32]
    L.ssd_tc_gemm_check.argtypes = [vp, vp, i32, i32, i32, i32, i32, vp, sz, vp, vp, vp]
    L.ssd_kernel_launch_count.restype = ctypes.c_uint64
    L.ssd_kernel_launch_count.argtypes = []
    L.ssd_last_status.argtypes = [vp, ctypes.POINTER(i32), vp]
    L.ssd_last_cuda_error.restype = ctypes.c_char_p
    L.ssd_strerror.restype = ctypes.c_char_p
    L.ssd_strerror.argtypes = [ctypes.c_int]
    _lib = L
    return L


def check(rc: int) -> None:
    if rc != 0:
        L = lib()
        msg = L.ssd_strerror(rc).decode()
        detail = L.ssd_last_cuda_error().decode()
        raise SsdError(f"ssd error {rc}: {msg}" + (f" ({detail})" if detail and rc == -7 else ""))


def _require_cuda() -> None:
    if not torch.cuda.is_available():
        raise SsdError("no CUDA device: the SSD verify path has no CPU fallback")


def make_config(shape) -> ModelConfig:
    """ModelConfig from any object with the fields of synth.ModelShape."""
    return ModelConfig(shape.n_layers, shape.d_model, shape.n_q_heads, shape.n_kv_heads,
                       shape.head_dim, shape.d_ffn, shape.vocab_out, shape.vocab_text,
                       shape.rope_theta, shape.rms_eps, shape.weight_dtype, shape.qkv_bias)


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _alloc(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


class Model:
    """ssd_model handle plus the torch tensor that owns its device arena."""

    def __init__(self, shape, blob: np.ndarray, device="cuda:0"):
        _require_cuda()
        L = lib()
        self.shape = shape
        self.cfg = make_config(shape)
        self.device = torch.device(device)
        nbytes = L.ssd_model_arena_bytes(ctypes.byref(self.cfg))
        if nbytes == 0:
            raise SsdError("unsupported model configuration")
        with torch.cuda.device(self.device):
            self.arena = _alloc(nbytes, self.device)
            blob = np.ascontiguousarray(blob)
            h = ctypes.c_void_p()
            check(L.ssd_model_create(ctypes.byref(self.cfg), blob.ctypes.data, blob.nbytes,
                                     self.arena.data_ptr(), nbytes, ctypes.byref(h)))
        self.handle = h

    def __del__(self):
        if getattr(self, "handle", None) is not None and _lib is not None:
            _lib.ssd_model_destroy(self.handle)
            self.handle = None


class InheritedModel(Model):
    """A model made of some of another model's layers (ssd_model_create_inherited): no weights are
    copied.  `shape` is the source's shape with the new number of layers."""

    def __init__(self, source: Model, layer_map: Sequence[int]):
        import dataclasses
        L = lib()
        self.source = source                      # keeps the source's arena alive
        self.layer_map = [int(x) for x in layer_map]
        self.shape = dataclasses.replace(source.shape, n_layers=len(self.layer_map))
        self.cfg = make_config(self.shape)
        self.device = source.device
        m = np.ascontiguousarray(self.layer_map, dtype=np.int32)
        with torch.cuda.device(self.device):
            self.arena = _alloc(L.ssd_model_inherited_arena_bytes(source.handle, len(m)), self.device)
            h = ctypes.c_void_p()
            check(L.ssd_model_create_inherited(source.handle, m.ctypes.data, len(m), self.arena.data_ptr(),
                                               self.arena.numel(), ctypes.byref(h)))
        self.handle = h


class Streams:
    """ssd_streams handle plus the torch tensors that own the KV cache and the workspace."""

    def __init__(self, model: Model, batch: int, capacity: int, max_gamma: int):
        L = lib()
        self.model, self.B, self.capacity, self.max_gamma = model, batch, capacity, max_gamma
        cfg = model.cfg
        dev = model.device
        kvb = L.ssd_kv_bytes(ctypes.byref(cfg), batch, capacity)
        wsb = L.ssd_workspace_bytes(ctypes.byref(cfg), batch, max_gamma, capacity)
        if kvb == 0 or wsb == 0:
            raise SsdError("unsupported stream configuration")
        with torch.cuda.device(dev):
            self.kv_raw = _alloc(kvb, dev)
            self.ws = _alloc(wsb, dev)
            h = ctypes.c_void_p()
            check(L.ssd_streams_create(model.handle, batch, capacity, max_gamma,
                                       self.kv_raw.data_ptr(), kvb, self.ws.data_ptr(), wsb,
                                       ctypes.byref(h)))
        self.handle = h
        s = model.shape
        dt = torch.float32 if s.weight_dtype == 0 else torch.bfloat16
        self.kv = self.kv_raw[:kvb].view(dt).view(s.n_layers, batch, 2, s.n_kv_heads, capacity,
                                                  s.head_dim)

    def __del__(self):
        if getattr(self, "handle", None) is not None and _lib is not None:
            _lib.ssd_streams_destroy(self.handle)
            self.handle = None

    def set_path(self, path: int) -> None:
        """0: persistent small-batch kernel where the forward fits it (default); 1: generic kernels."""
        check(lib().ssd_streams_set_path(self.handle, path))

    def set_attention_kernel(self, which: int) -> None:
        """Batched forward: 0 picks the attention kernel by the key range per CTA (default), 1 the
        warp-level tensor-core kernel always, 2 the tcgen05 kernel wherever the head size allows."""
        check(lib().ssd_streams_set_attention_kernel(self.handle, which))

    def set_activation_split(self, on: bool) -> None:
        """Persistent kernel: True (default) feeds activations to the tensor cores as bf16 leading
        part + remainder (near-fp32 inputs), False rounds them to bf16."""
        check(lib().ssd_streams_set_activation_split(self.handle, 1 if on else 0))

    def set_trace(self, buf: Optional[torch.Tensor]) -> None:
        """buf: int64 CUDA tensor [ctas >= 256, events_per_cta] that receives the persistent
        kernel's phase-boundary clocks, or None to turn the trace off."""
        if buf is None:
            check(lib().ssd_streams_set_trace(self.handle, None, 0, 0))
        else:
            assert buf.dtype == torch.int64 and buf.is_cuda and buf.is_contiguous() and buf.dim() == 2
            check(lib().ssd_streams_set_trace(self.handle, buf.data_ptr(), buf.shape[0], buf.shape[1]))
        self._trace = buf

    # -- state ------------------------------------------------------------------------------
    def kv_truncate(self, lens: Sequence[int], pending: Sequence[int], stream=None) -> None:
        a = np.ascontiguousarray(lens, dtype=np.int32)
        p = np.ascontiguousarray(pending, dtype=np.int32)
        assert a.shape == (self.B,) and p.shape == (self.B,)
        check(lib().ssd_kv_truncate(self.handle, a.ctypes.data, p.ctypes.data, _stream_ptr(stream)))

    def kv_restore(self, dev_len: torch.Tensor, dev_pending: torch.Tensor, stream=None) -> None:
        assert dev_len.dtype == torch.int32 and dev_pending.dtype == torch.int32
        assert dev_len.is_cuda and dev_len.numel() == self.B and dev_pending.numel() == self.B
        check(lib().ssd_kv_restore(self.handle, dev_len.data_ptr(), dev_pending.data_ptr(),
                                   _stream_ptr(stream)))

    def get_state(self, stream=None) -> Tuple[np.ndarray, np.ndarray]:
        a = np.zeros(self.B, np.int32)
        p = np.zeros(self.B, np.int32)
        check(lib().ssd_streams_get_state(self.handle, a.ctypes.data, p.ctypes.data,
                                          _stream_ptr(stream)))
        return a, p

    def inject_failure(self, stream=None) -> None:
        """Marks the streams object as failed, as a timed-out wait in the persistent kernel would."""
        check(lib().ssd_streams_inject_failure(self.handle, _stream_ptr(stream)))

    def last_status(self, stream=None) -> int:
        v = ctypes.c_int32(0)
        check(lib().ssd_last_status(self.handle, ctypes.byref(v), _stream_ptr(stream)))
        return v.value

    # -- the calls --------------------------------------------------------------------------
    def prefill(self, prefixes: Sequence[np.ndarray], stream=None) -> None:
        assert len(prefixes) == self.B
        offs = np.zeros(self.B + 1, np.int32)
        offs[1:] = np.cumsum([len(p) for p in prefixes])
        ids = torch.from_numpy(np.concatenate(prefixes).astype(np.int32)).to(self.model.device)
        check(lib().ssd_prefill(self.model.handle, self.handle, ids.data_ptr(), offs.ctypes.data,
                                _stream_ptr(stream)))
        torch.cuda.current_stream().synchronize() if stream is None else stream.synchronize()

    def verify(self, draft_tokens: torch.Tensor, draft_probs: torch.Tensor,
               uniforms: torch.Tensor, params: VerifyParams, accepted_len: torch.Tensor,
               next_token: torch.Tensor, logits: Optional[torch.Tensor] = None,
               stream=None) -> None:
        g = params.gamma
        assert draft_tokens.dtype == torch.int32 and draft_tokens.numel() == self.B * g
        assert draft_probs.dtype == torch.float32 and \
            draft_probs.numel() == self.B * g * self.model.shape.vocab_out
        assert uniforms.dtype == torch.float32 and uniforms.numel() == self.B * (g + 1) * 2
        assert accepted_len.dtype == torch.int32 and next_token.dtype == torch.int32
        for t in (draft_tokens, draft_probs, uniforms, accepted_len, next_token):
            assert t.is_cuda and t.is_contiguous()
        if logits is not None:
            assert logits.dtype == torch.float32 and logits.is_contiguous() and \
                logits.numel() == self.B * (g + 1) * self.model.shape.vocab_out
        check(lib().ssd_verify(self.model.handle, self.handle, draft_tokens.data_ptr(),
                               draft_probs.data_ptr(), uniforms.data_ptr(), ctypes.byref(params),
                               accepted_len.data_ptr(), next_token.data_ptr(), _ptr(logits),
                               _stream_ptr(stream)))

    def forward(self, draft_tokens: torch.Tensor, gamma: int, logits: torch.Tensor, stream=None) -> None:
        """ssd_forward: the decoder forward alone (logits [B, gamma+1, V]), no acceptance step."""
        assert draft_tokens.dtype == torch.int32 and draft_tokens.numel() == self.B * gamma
        assert logits.dtype == torch.float32 and logits.is_contiguous() and \
            logits.numel() == self.B * (gamma + 1) * self.model.shape.vocab_out
        check(lib().ssd_forward(self.model.handle, self.handle, draft_tokens.data_ptr(), gamma,
                                logits.data_ptr(), _stream_ptr(stream)))

    def verify_host(self, draft_tokens: torch.Tensor, draft_probs: torch.Tensor,
                    uniforms: torch.Tensor, params: VerifyParams, accepted_len: torch.Tensor,
                    next_token: torch.Tensor, stream=None) -> None:
        """Host-buffer variant (pinned CPU tensors); includes the commit and a stream sync."""
        for t in (draft_tokens, draft_probs, uniforms, accepted_len, next_token):
            assert not t.is_cuda and t.is_contiguous()
        check(lib().ssd_verify_host(self.model.handle, self.handle, draft_tokens.data_ptr(),
                                    draft_probs.data_ptr(), uniforms.data_ptr(),
                                    ctypes.byref(params), accepted_len.data_ptr(),
                                    next_token.data_ptr(), _stream_ptr(stream)))

    def kv_commit(self, accepted_len: torch.Tensor, next_token: torch.Tensor, stream=None) -> None:
        check(lib().ssd_kv_commit(self.handle, accepted_len.data_ptr(), next_token.data_ptr(),
                                  _stream_ptr(stream)))

    def draft_step(self, in_ids: torch.Tensor, n_in: int, uniform: torch.Tensor,
                   params: VerifyParams, out_token: torch.Tensor, out_prob_row: torch.Tensor,
                   stream=None) -> None:
        assert in_ids.dtype == torch.int32 and in_ids.numel() == self.B * n_in
        assert uniform.dtype == torch.float32 and uniform.numel() == self.B
        assert out_prob_row.dtype == torch.float32 and \
            out_prob_row.numel() == self.B * self.model.shape.vocab_out
        check(lib().ssd_draft_step(self.model.handle, self.handle, in_ids.data_ptr(), n_in,
                                   uniform.data_ptr(), ctypes.byref(params), out_token.data_ptr(),
                                   out_prob_row.data_ptr(), _stream_ptr(stream)))


class PagedStreams(Streams):
    """Streams whose K/V live in 64-token pages drawn from one pool (ssd_streams_create_paged)."""

    PAGE_TOKENS = 64

    def __init__(self, model: Model, batch: int, n_pages: int, max_pages_per_stream: int, max_gamma: int):
        L = lib()
        self.model, self.B, self.max_gamma = model, batch, max_gamma
        self.n_pages, self.max_pages = n_pages, max_pages_per_stream
        self.capacity = max_pages_per_stream * self.PAGE_TOKENS
        cfg, dev = model.cfg, model.device
        kvb = L.ssd_paged_kv_bytes(ctypes.byref(cfg), n_pages)
        wsb = L.ssd_paged_workspace_bytes(ctypes.byref(cfg), batch, max_gamma, n_pages, max_pages_per_stream)
        if kvb == 0 or wsb == 0:
            raise SsdError("unsupported paged stream configuration")
        with torch.cuda.device(dev):
            self.kv_raw = _alloc(kvb, dev)
            self.ws = _alloc(wsb, dev)
            h = ctypes.c_void_p()
            check(L.ssd_streams_create_paged(model.handle, batch, n_pages, max_pages_per_stream, max_gamma,
                                             self.kv_raw.data_ptr(), kvb, self.ws.data_ptr(), wsb,
                                             ctypes.byref(h)))
        self.handle = h
        s = model.shape
        self.kv = self.kv_raw[:kvb].view(torch.bfloat16).view(s.n_layers, n_pages, 2, s.n_kv_heads,
                                                              self.PAGE_TOKENS, s.head_dim)

    def paged_state(self, stream=None):
        """(pages held by each stream, free pages, block tables [B, max_pages] with -1 = none)."""
        used = np.zeros(self.B, np.int32)
        free = np.zeros(1, np.int32)
        table = np.zeros((self.B, self.max_pages), np.int32)
        check(lib().ssd_paged_state(self.handle, used.ctypes.data, free.ctypes.data, table.ctypes.data,
                                    _stream_ptr(stream)))
        return used, int(free[0]), table

    def prefill_some(self, prefixes: Sequence[Optional[np.ndarray]], stream=None) -> None:
        """Prefill only the streams whose entry is not None (the others keep their state)."""
        self.prefill([p if p is not None else np.zeros(0, np.int32) for p in prefixes], stream)


def accept_noalloc(logits: torch.Tensor, draft_tokens: torch.Tensor, draft_probs: torch.Tensor,
                   uniforms: torch.Tensor, params: VerifyParams, accepted_len: torch.Tensor,
                   next_token: torch.Tensor, stream=None) -> None:
    """ssd_accept_noalloc: the acceptance step on caller-held logits [B, gamma+1, V], for callers
    that cannot allocate device memory (the kernel's scratch is a fixed array in the library).
    Limits: at most 256 streams, gamma + 1 <= 16.  Calls share that array, so calls that overlap
    on the GPU race; make the first call on a device outside any stream capture."""
    B, R, V = logits.shape
    assert logits.dtype == torch.float32 and logits.is_cuda and logits.is_contiguous()
    assert R == params.gamma + 1 and draft_tokens.numel() == B * params.gamma
    assert draft_probs.numel() == B * params.gamma * V and uniforms.numel() == B * R * 2
    with torch.cuda.device(logits.device):
        check(lib().ssd_accept_noalloc(logits.data_ptr(), draft_tokens.data_ptr(),
                                       draft_probs.data_ptr(), uniforms.data_ptr(),
                                       ctypes.byref(params), B, V, accepted_len.data_ptr(),
                                       next_token.data_ptr(), _stream_ptr(stream)))


def tc_gemm_check(w: torch.Tensor, x: torch.Tensor, ksplit: int, epilogue: int, stream=None):
    """ssd_tc_gemm_check: one tensor-core projection on caller data.  w bf16 [n_rows, K], x float32
    [M, K], both CUDA.  Returns (raw output tensor, status word): float32 [ksplit, Mpad, ld] partial
    sums (epilogue 0), float32 [M, n_rows] (1), or the packed SiLU(gate) * up operand as uint8 (2)."""
    _require_cuda()
    L = lib()
    assert w.dtype == torch.bfloat16 and x.dtype == torch.float32 and w.is_cuda and x.is_cuda
    assert w.is_contiguous() and x.is_contiguous() and w.shape[1] == x.shape[1]
    n_rows, K = w.shape
    M = x.shape[0]
    Mpad, ld = (M + 15) // 16 * 16, (n_rows + 127) // 128 * 128
    need = L.ssd_tc_gemm_scratch_bytes(M, n_rows, K)
    if need == 0:
        raise SsdError("sizes outside the range of the tensor-core projection")
    with torch.cuda.device(w.device):
        scratch = torch.zeros(need, dtype=torch.uint8, device=w.device)
        status = torch.zeros(1, dtype=torch.int32, device=w.device)
        if epilogue == 0:
            out = torch.zeros((ksplit, Mpad, ld), dtype=torch.float32, device=w.device)
        elif epilogue == 1:
            out = torch.zeros((M, n_rows), dtype=torch.float32, device=w.device)
        else:
            chunks = 1 if Mpad <= 256 else (Mpad + 255) // 256
            mc = Mpad if chunks == 1 else ((Mpad + chunks - 1) // chunks + 15) // 16 * 16
            out = torch.zeros(((n_rows // 2 + 15) // 16) * chunks * mc * 64, dtype=torch.uint8, device=w.device)
        check(L.ssd_tc_gemm_check(w.data_ptr(), x.data_ptr(), M, n_rows, K, ksplit, epilogue,
                                  scratch.data_ptr(), need, out.data_ptr(), status.data_ptr(),
                                  _stream_ptr(stream)))
    return out, status


class Loop:
    """Buffers of the device-resident SSD iteration (ssd_iteration) and the call itself.

    Both stream sets must already hold the same prefixes (prefill both models); this object rolls
    the draft streams back by one token and keeps the last two prefix ids, as the call expects."""

    def __init__(self, target: Streams, draft: Streams, prefixes: Sequence[np.ndarray], gamma: int,
                 uniform_pool: np.ndarray, out_capacity: int, ras_window: int = 0):
        B, V = target.B, target.model.shape.vocab_out
        assert draft.B == B and len(prefixes) == B and all(len(p) >= 2 for p in prefixes)
        per = gamma + 2 * (gamma + 1)
        assert uniform_pool.dtype == np.float32 and uniform_pool.shape[1:] == (B, per)
        dev = target.model.device
        self.target, self.draft, self.gamma = target, draft, gamma
        self.pool = torch.from_numpy(np.ascontiguousarray(uniform_pool)).to(dev)
        self.iteration = torch.zeros(1, dtype=torch.int32, device=dev)
        self.in_ids = torch.from_numpy(np.stack([np.asarray(p[-2:], np.int32) for p in prefixes])).to(dev)
        self.draft_tokens = torch.zeros((B, gamma), dtype=torch.int32, device=dev)
        self.draft_probs = torch.zeros((B, gamma, V), dtype=torch.float32, device=dev)
        self.accepted_len = torch.zeros(B, dtype=torch.int32, device=dev)
        self.next_token = torch.zeros(B, dtype=torch.int32, device=dev)
        self.out_tokens = torch.zeros((B, out_capacity), dtype=torch.int32, device=dev)
        self.out_count = torch.zeros(B, dtype=torch.int32, device=dev)
        self.accept_log = torch.full((uniform_pool.shape[0], B), -9, dtype=torch.int32, device=dev)
        # window of the repetition-aware sampler: the last tokens of each prefix, pending token last
        self.recent = None
        if ras_window > 0:
            rec = np.full((B, ras_window), -1, dtype=np.int32)
            for b, p in enumerate(prefixes):
                tail = np.asarray(p[-ras_window:], np.int32)
                rec[b, ras_window - len(tail):] = tail
            self.recent = torch.from_numpy(rec).to(dev)
        lens, pend = draft.get_state()
        draft.kv_truncate(lens - 1, pend)
        self.io = LoopIo(self.pool.data_ptr(), uniform_pool.shape[0], self.iteration.data_ptr(),
                         self.in_ids.data_ptr(), self.draft_tokens.data_ptr(), self.draft_probs.data_ptr(),
                         self.accepted_len.data_ptr(), self.next_token.data_ptr(),
                         self.out_tokens.data_ptr(), out_capacity, self.out_count.data_ptr(),
                         self.accept_log.data_ptr())

    def iterate(self, params: VerifyParams, stream=None) -> None:
        assert params.gamma == self.gamma
        check(lib().ssd_iteration(self.target.model.handle, self.target.handle, self.draft.model.handle,
                                  self.draft.handle, ctypes.byref(params), ctypes.byref(self.io),
                                  _stream_ptr(stream)))
