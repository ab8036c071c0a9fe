"""Thin ctypes binding of the C ABI in ``include/pmkvq.h`` (same call names, argument
marshalling only).  PyTorch supplies device memory (the arena, inputs, outputs) and the stream;
every step of the path runs inside ``libpmkvq.so``.  There is no fallback: if the library is
missing it is built with nvcc, and if that fails the import raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np
import torch

from . import build as _build

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libpmkvq.so")

STATUS_NAMES = ["OK", "INVALID_ARG", "ARENA_TOO_SMALL", "BUDGET_FULL", "AT_FBIT", "CAPACITY", "CUDA", "STATE",
                "SCRATCH_LIMIT", "DEVICE_WAIT"]
(OK, INVALID_ARG, ARENA_TOO_SMALL, BUDGET_FULL, AT_FBIT, CAPACITY, CUDA_ERROR, STATE, SCRATCH_LIMIT,
 DEVICE_WAIT) = range(10)


class PmkvqError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__(f"{what}: {STATUS_NAMES[status] if 0 <= status < len(STATUS_NAMES) else status}")
        self.status = status


class _Config(ctypes.Structure):
    _fields_ = [
        ("layers", ctypes.c_int32), ("q_heads", ctypes.c_int32), ("kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32), ("batch", ctypes.c_int32), ("max_tokens", ctypes.c_int32),
        ("fbit", ctypes.POINTER(ctypes.c_uint8)), ("budget_bytes", ctypes.POINTER(ctypes.c_uint64)),
        ("lam", ctypes.POINTER(ctypes.c_float)),
        ("n_sink", ctypes.c_int32), ("window", ctypes.c_int32), ("evict_chunk", ctypes.c_int32),
        ("count_metadata", ctypes.c_int32), ("auto_reduce", ctypes.c_int32), ("sm_scale", ctypes.c_float),
        ("d_arena", ctypes.c_void_p), ("arena_bytes", ctypes.c_size_t), ("shift_variant", ctypes.c_int32),
        ("attention_path", ctypes.c_int32),
    ]


def load_library() -> ctypes.CDLL:
    if _build.needs_build():
        _build.build()
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i32, u64p, i32p = ctypes.c_void_p, ctypes.c_int32, ctypes.POINTER(ctypes.c_uint64), ctypes.POINTER(ctypes.c_int32)
    lib.pmkvq_arena_bytes_required.restype = ctypes.c_size_t
    lib.pmkvq_arena_bytes_required.argtypes = [ctypes.POINTER(_Config)]
    lib.pmkvq_cache_create.restype = i32
    lib.pmkvq_cache_create.argtypes = [ctypes.POINTER(_Config), ctypes.POINTER(vp)]
    lib.pmkvq_cache_destroy.restype = None
    lib.pmkvq_cache_destroy.argtypes = [vp]
    lib.pmkvq_append.restype = i32
    lib.pmkvq_append.argtypes = [vp, i32, vp, vp, i32, vp]
    lib.pmkvq_progressive_reduce.restype = i32
    lib.pmkvq_progressive_reduce.argtypes = [vp, i32, vp]
    lib.pmkvq_decode_attention.restype = i32
    lib.pmkvq_decode_attention.argtypes = [vp, i32, vp, vp, vp]
    lib.pmkvq_decode_attention_static.restype = i32
    lib.pmkvq_decode_attention_static.argtypes = [vp, i32, vp, vp, vp]
    lib.pmkvq_decode_step.restype = i32
    lib.pmkvq_decode_step.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.pmkvq_decode_attention_all.restype = i32
    lib.pmkvq_decode_attention_all.argtypes = [vp, vp, vp, vp]
    lib.pmkvq_device_status.restype = i32
    lib.pmkvq_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.pmkvq_selftest_bounded_wait.restype = i32
    lib.pmkvq_selftest_bounded_wait.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.pmkvq_restore_layer_state.restype = i32
    lib.pmkvq_restore_layer_state.argtypes = [vp, i32, i32, i32]
    lib.pmkvq_arena_layout.restype = i32
    lib.pmkvq_arena_layout.argtypes = [vp, i32, u64p]
    lib.pmkvq_set_attention_ctas.restype = i32
    lib.pmkvq_set_attention_ctas.argtypes = [vp, i32]
    lib.pmkvq_layer_state.restype = i32
    lib.pmkvq_layer_state.argtypes = [vp, i32, i32p, i32p, u64p, u64p]
    lib.pmkvq_launch_count.restype = ctypes.c_uint64
    lib.pmkvq_launch_count.argtypes = [vp]
    lib.pmkvq_attention_bytes.restype = ctypes.c_uint64
    lib.pmkvq_attention_bytes.argtypes = [vp, i32]
    lib.pmkvq_export_slice.restype = i32
    lib.pmkvq_export_slice.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.pmkvq_calibrate_lambda.restype = i32
    lib.pmkvq_calibrate_lambda.argtypes = [vp, i32, i32, i32, ctypes.c_double, ctypes.c_double, ctypes.c_float,
                                           ctypes.c_float, vp, vp]
    lib.pmkvq_alpha_grid_workspace_bytes.restype = ctypes.c_uint64
    lib.pmkvq_alpha_grid_workspace_bytes.argtypes = [i32, i32, i32, i32]
    lib.pmkvq_alpha_grid_search.restype = i32
    lib.pmkvq_alpha_grid_search.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, vp, i32, ctypes.c_double, ctypes.c_double,
                                            ctypes.c_float, vp, vp, vp, vp]
    lib.pmkvq_allocate_bits.restype = i32
    lib.pmkvq_allocate_bits.argtypes = [i32, i32, vp, vp, vp, ctypes.c_uint64, vp, vp]
    lib.pmkvq_status_string.restype = ctypes.c_char_p
    lib.pmkvq_status_string.argtypes = [i32]
    return lib


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = load_library()
    return _lib


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


def calibrate_lambda(k_pre: torch.Tensor, pos_scale: float = 1.0, theta: float = 10000.0, alpha: float = 0.5,
                     floor_value: float = 1e-5, stream=None) -> torch.Tensor:
    """Eq. 10-12 on the device.  k_pre: CUDA bf16 [n_tokens, n_seq, kv_heads, 128] pre-RoPE Keys, token t at
    position t -> lambda fp32 [kv_heads, 128] (CUDA)."""
    if not (k_pre.is_cuda and k_pre.is_contiguous() and k_pre.dtype == torch.bfloat16 and k_pre.dim() == 4
            and k_pre.shape[3] == 128):
        raise ValueError("k_pre must be a contiguous CUDA bf16 tensor [n_tokens, n_seq, kv_heads, 128]")
    n_tokens, n_seq, kv_heads, _ = k_pre.shape
    lam = torch.empty(kv_heads, 128, dtype=torch.float32, device=k_pre.device)
    st = lib().pmkvq_calibrate_lambda(k_pre.data_ptr(), n_tokens, n_seq, kv_heads, float(pos_scale), float(theta),
                                      float(alpha), float(floor_value), lam.data_ptr(), _stream_ptr(stream))
    if st != OK:
        raise PmkvqError(st, "pmkvq_calibrate_lambda")
    return lam


def alpha_grid_search(k_pre: torch.Tensor, q_pre: torch.Tensor, v: torch.Tensor, bits: int, alphas=None,
                      pos_scale: float = 1.0, theta: float = 10000.0, floor_value: float = 1e-5, stream=None):
    """alpha of Eq. 10 by grid search on the attention reconstruction loss (Sec. 4.1.1), on the device.
    k_pre, v: CUDA bf16 [n_tokens, n_seq, kv_heads, 128]; q_pre: [n_tokens, n_seq, kv_heads * group, 128];
    alphas: the grid (default j / 20, j = 0..19).  Returns (best alpha, losses as a float64 array)."""
    for t in (k_pre, q_pre, v):
        if not (t.is_cuda and t.is_contiguous() and t.dtype == torch.bfloat16 and t.dim() == 4 and t.shape[3] == 128):
            raise ValueError("k_pre, q_pre, v must be contiguous CUDA bf16 tensors [n_tokens, n_seq, heads, 128]")
    n_tokens, n_seq, kv_heads, _ = k_pre.shape
    if v.shape != k_pre.shape or q_pre.shape[:2] != k_pre.shape[:2] or q_pre.shape[2] % kv_heads:
        raise ValueError("shapes of k_pre, q_pre, v do not fit together")
    group = q_pre.shape[2] // kv_heads
    a = np.ascontiguousarray(np.arange(20) / 20.0 if alphas is None else alphas, dtype=np.float32)
    ws = torch.empty(int(lib().pmkvq_alpha_grid_workspace_bytes(n_tokens, n_seq, kv_heads, group)), dtype=torch.uint8, device=k_pre.device)
    losses = np.zeros(len(a), np.float64)
    best = ctypes.c_int32()
    st = lib().pmkvq_alpha_grid_search(k_pre.data_ptr(), q_pre.data_ptr(), v.data_ptr(), n_tokens, n_seq, kv_heads, group,
                                       int(bits), a.ctypes.data, len(a), float(pos_scale), float(theta), float(floor_value),
                                       ws.data_ptr(), losses.ctypes.data, ctypes.addressof(best), _stream_ptr(stream))
    if st != OK:
        raise PmkvqError(st, "pmkvq_alpha_grid_search")
    return float(a[best.value]), losses


def allocate_bits(widths, sensitivity, mem_bytes, budget_bytes):
    """Block-wise bit allocation (Eq. 6-8): widths [C], sensitivity and mem_bytes [layers, C] ->
    (fbit per block as a list, minimal summed sensitivity).  Host only."""
    sens = np.ascontiguousarray(sensitivity, dtype=np.float64)
    mem = np.ascontiguousarray(mem_bytes, dtype=np.uint64)
    w = np.ascontiguousarray(widths, dtype=np.uint8)
    layers, c = sens.shape
    if mem.shape != sens.shape or w.shape != (c,):
        raise ValueError("bad shapes")
    out = np.zeros(layers, np.uint8)
    cost = ctypes.c_double()
    st = lib().pmkvq_allocate_bits(layers, c, w.ctypes.data, sens.ctypes.data, mem.ctypes.data, int(budget_bytes),
                                   out.ctypes.data, ctypes.addressof(cost))
    if st != OK:
        raise PmkvqError(st, "pmkvq_allocate_bits")
    return out.tolist(), cost.value


class Cache:
    """A PM-KVQ cache of ``layers`` transformer blocks living in one torch-owned device arena."""

    def __init__(self, layers: int, q_heads: int, kv_heads: int, batch: int, max_tokens: int,
                 fbit: Sequence[int], budget_bytes: Optional[Sequence[int]] = None,
                 lam: Optional[np.ndarray] = None, n_sink: int = 1, window: int = 128, evict_chunk: int = 1,
                 count_metadata: bool = True, auto_reduce: bool = True, sm_scale: float = 0.0,
                 device: str = "cuda:0", shift_variant: int = 0, attention_path: int = 0, slack_bytes: int = 0,
                 fill_byte: Optional[int] = None):
        self._h = None
        self.layers, self.q_heads, self.kv_heads, self.batch = layers, q_heads, kv_heads, batch
        self._fbit = (ctypes.c_uint8 * layers)(*[int(b) for b in fbit])
        self._budget = None if budget_bytes is None else (ctypes.c_uint64 * layers)(*[int(b) for b in budget_bytes])
        self._lam = None
        if lam is not None:
            self._lam = np.ascontiguousarray(lam, dtype=np.float32).reshape(layers, kv_heads, 128)
        cfg = _Config()
        cfg.layers, cfg.q_heads, cfg.kv_heads, cfg.head_dim = layers, q_heads, kv_heads, 128
        cfg.batch, cfg.max_tokens = batch, max_tokens
        cfg.fbit = ctypes.cast(self._fbit, ctypes.POINTER(ctypes.c_uint8))
        cfg.budget_bytes = None if self._budget is None else ctypes.cast(self._budget, ctypes.POINTER(ctypes.c_uint64))
        cfg.lam = None if self._lam is None else self._lam.ctypes.data_as(ctypes.POINTER(ctypes.c_float))
        cfg.n_sink, cfg.window, cfg.evict_chunk = n_sink, window, evict_chunk
        cfg.count_metadata, cfg.auto_reduce, cfg.sm_scale = int(count_metadata), int(auto_reduce), float(sm_scale)
        cfg.shift_variant = int(shift_variant)
        cfg.attention_path = int(attention_path)
        need = lib().pmkvq_arena_bytes_required(ctypes.byref(cfg))
        if need == 0:
            raise PmkvqError(INVALID_ARG, "pmkvq_arena_bytes_required")
        self.arena_bytes = need
        self.device = torch.device(device)
        with torch.cuda.device(self.device):
            self.arena = torch.empty(need + 256 + int(slack_bytes), dtype=torch.uint8, device=self.device)
            if fill_byte is not None:       # tests that watch the bytes no kernel may touch
                self.arena.fill_(int(fill_byte))
            base = self.arena.data_ptr()
            self.arena_offset = (base + 255) // 256 * 256 - base
            cfg.d_arena = (base + 255) // 256 * 256
            cfg.arena_bytes = need
            h = ctypes.c_void_p()
            st = lib().pmkvq_cache_create(ctypes.byref(cfg), ctypes.byref(h))
        if st != OK:
            raise PmkvqError(st, "pmkvq_cache_create")
        self._h = h

    def close(self):
        if self._h is not None:
            lib().pmkvq_cache_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @staticmethod
    def _check(t: torch.Tensor, dtype, what):
        if not (t.is_cuda and t.is_contiguous() and t.dtype == dtype):
            raise ValueError(f"{what} must be a contiguous CUDA tensor of {dtype}")

    def append(self, layer: int, k: torch.Tensor, v: torch.Tensor, stream=None, check: bool = True) -> int:
        """k, v: bf16 [n_new, batch, kv_heads, 128] (or [batch, kv_heads, 128] for one token)."""
        self._check(k, torch.bfloat16, "k"); self._check(v, torch.bfloat16, "v")
        n_new = 1 if k.dim() == 3 else k.shape[0]
        if k.numel() != n_new * self.batch * self.kv_heads * 128 or v.numel() != k.numel():
            raise ValueError("bad K/V shape")
        st = lib().pmkvq_append(self._h, layer, k.data_ptr(), v.data_ptr(), n_new, _stream_ptr(stream))
        if check and st != OK:
            raise PmkvqError(st, "pmkvq_append")
        return st

    def progressive_reduce(self, layer: int, stream=None, check: bool = True) -> int:
        st = lib().pmkvq_progressive_reduce(self._h, layer, _stream_ptr(stream))
        if check and st != OK:
            raise PmkvqError(st, "pmkvq_progressive_reduce")
        return st

    def decode_attention(self, layer: int, q: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None):
        """q: bf16 [batch, q_heads, 128] -> fp32 [batch, q_heads, 128]."""
        self._check(q, torch.bfloat16, "q")
        if q.numel() != self.batch * self.q_heads * 128:
            raise ValueError("bad Q shape")
        if out is None:
            out = torch.empty(self.batch, self.q_heads, 128, dtype=torch.float32, device=q.device)
        self._check(out, torch.float32, "out")
        st = lib().pmkvq_decode_attention(self._h, layer, q.data_ptr(), out.data_ptr(), _stream_ptr(stream))
        if st != OK:
            raise PmkvqError(st, "pmkvq_decode_attention")
        return out

    def decode_attention_static(self, layer: int, q: torch.Tensor, out: torch.Tensor, stream=None, check: bool = True):
        """pmkvq_decode_attention_static: same result as decode_attention, split-K workspace inside the
        library image instead of the arena.  `out` must be supplied (nothing is allocated here either)."""
        self._check(q, torch.bfloat16, "q"); self._check(out, torch.float32, "out")
        if q.numel() != self.batch * self.q_heads * 128 or out.numel() != q.numel():
            raise ValueError("bad Q / out shape")
        st = lib().pmkvq_decode_attention_static(self._h, layer, q.data_ptr(), out.data_ptr(), _stream_ptr(stream))
        if check and st != OK:
            raise PmkvqError(st, "pmkvq_decode_attention_static")
        return st

    def decode_step(self, k: torch.Tensor, v: torch.Tensor, q: torch.Tensor, out: Optional[torch.Tensor] = None,
                    stream=None):
        """One decode step over all blocks.  k, v: bf16 [layers, batch, kv_heads, 128]; q: bf16
        [layers, batch, q_heads, 128] -> fp32 [layers, batch, q_heads, 128]."""
        self._check(k, torch.bfloat16, "k"); self._check(v, torch.bfloat16, "v"); self._check(q, torch.bfloat16, "q")
        if (k.numel() != self.layers * self.batch * self.kv_heads * 128 or v.numel() != k.numel()
                or q.numel() != self.layers * self.batch * self.q_heads * 128):
            raise ValueError("bad K/V/Q shape")
        if out is None:
            out = torch.empty(self.layers, self.batch, self.q_heads, 128, dtype=torch.float32, device=q.device)
        self._check(out, torch.float32, "out")
        if out.numel() != q.numel():
            raise ValueError("bad out shape")
        st = lib().pmkvq_decode_step(self._h, k.data_ptr(), v.data_ptr(), q.data_ptr(), out.data_ptr(), _stream_ptr(stream))
        if st != OK:
            raise PmkvqError(st, "pmkvq_decode_step")
        return out

    def decode_attention_all(self, q: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None):
        """Attention of all blocks in one launch, nothing appended.  q: bf16 [layers, batch, q_heads, 128]
        -> fp32 [layers, batch, q_heads, 128]."""
        self._check(q, torch.bfloat16, "q")
        if q.numel() != self.layers * self.batch * self.q_heads * 128:
            raise ValueError("bad Q shape")
        if out is None:
            out = torch.empty(self.layers, self.batch, self.q_heads, 128, dtype=torch.float32, device=q.device)
        self._check(out, torch.float32, "out")
        if out.numel() != q.numel():
            raise ValueError("bad out shape")
        st = lib().pmkvq_decode_attention_all(self._h, q.data_ptr(), out.data_ptr(), _stream_ptr(stream))
        if st != OK:
            raise PmkvqError(st, "pmkvq_decode_attention_all")
        return out

    def device_status(self, check: bool = True) -> int:
        """Synchronises; returns the word of device-side waits that ran out (0 = none)."""
        word = ctypes.c_uint32()
        st = lib().pmkvq_device_status(self._h, ctypes.byref(word))
        if check and st != OK:
            raise PmkvqError(st, f"pmkvq_device_status (bits {word.value:#x})")
        return int(word.value)

    def selftest_bounded_wait(self, stream=None) -> int:
        """1 if the deliberately unsatisfiable wait gave up as designed."""
        got = ctypes.c_uint32()
        st = lib().pmkvq_selftest_bounded_wait(self._h, _stream_ptr(stream), ctypes.byref(got))
        if st != OK:
            raise PmkvqError(st, "pmkvq_selftest_bounded_wait")
        return int(got.value)

    def restore_layer_state(self, layer: int, n_tokens: int, cur_bits: int):
        st = lib().pmkvq_restore_layer_state(self._h, layer, int(n_tokens), int(cur_bits))
        if st != OK:
            raise PmkvqError(st, "pmkvq_restore_layer_state")

    def arena_layout(self, layer: int):
        out = (ctypes.c_uint64 * 10)()
        st = lib().pmkvq_arena_layout(self._h, layer, out)
        if st != OK:
            raise PmkvqError(st, "pmkvq_arena_layout")
        keys = ("arena_bytes", "offset", "slice_stride", "ring_off", "body_off", "stream_stride", "ring_tokens",
                "partials_off", "partials_bytes", "partial_slot_bytes")
        return dict(zip(keys, [int(x) for x in out]))

    def set_attention_ctas(self, n_ctas: int):
        st = lib().pmkvq_set_attention_ctas(self._h, n_ctas)
        if st != OK:
            raise PmkvqError(st, "pmkvq_set_attention_ctas")

    def layer_state(self, layer: int):
        n, b = ctypes.c_int32(), ctypes.c_int32()
        used, budget = ctypes.c_uint64(), ctypes.c_uint64()
        st = lib().pmkvq_layer_state(self._h, layer, ctypes.byref(n), ctypes.byref(b), ctypes.byref(used), ctypes.byref(budget))
        if st != OK:
            raise PmkvqError(st, "pmkvq_layer_state")
        return {"n_tokens": n.value, "cur_bits": b.value, "bytes_used": used.value, "budget_bytes": budget.value}

    def launch_count(self) -> int:
        return int(lib().pmkvq_launch_count(self._h))

    def attention_bytes(self, layer: int) -> int:
        return int(lib().pmkvq_attention_bytes(self._h, layer))

    def export_slice(self, layer: int, batch_idx: int, kv_head: int, is_value: bool, packed: bool = False):
        n = self.layer_state(layer)["n_tokens"]
        codes = np.zeros((n, 128), np.uint16)
        scale, zero, bits = np.zeros(n, np.float32), np.zeros(n, np.float32), np.zeros(n, np.uint8)
        pk = np.zeros(n * 256, np.uint8) if packed else None
        st = lib().pmkvq_export_slice(self._h, layer, batch_idx, kv_head, int(is_value), codes.ctypes.data,
                                      scale.ctypes.data, zero.ctypes.data, bits.ctypes.data,
                                      None if pk is None else pk.ctypes.data)
        if st != OK:
            raise PmkvqError(st, "pmkvq_export_slice")
        if packed:
            return codes, scale, zero, bits, pk[: int(bits.astype(np.int64).sum()) * 16]
        return codes, scale, zero, bits
