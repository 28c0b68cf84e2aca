"""Thin ctypes binding of the GLIDE C ABI (include/glide.h): argument marshalling only.

Every step of the path runs in the CUDA kernels of libglide.so.  torch is used for
device memory and streams.  There is no fallback: if the library has not been built
(python -m paper_2607_24788_b200.build) loading raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libglide.so")

GLIDE_F32, GLIDE_BF16 = 0, 1
GLIDE_PHI_SOFTMAX, GLIDE_PHI_PROJ_SOFTMAX2 = 0, 1
GLIDE_MERGE_SHARED, GLIDE_MERGE_SUM_EVICTED, GLIDE_MERGE_SUM_ALL = 0, 1, 2
GLIDE_DECODE_AUTO, GLIDE_DECODE_MMA, GLIDE_DECODE_FMA, GLIDE_DECODE_STREAM = 0, 1, 2, 3
GLIDE_PREFILL_AUTO, GLIDE_PREFILL_MMA_SYNC, GLIDE_PREFILL_TCGEN05, GLIDE_PREFILL_FMA = 0, 1, 2, 3

GLIDE_OK = 0
GLIDE_ERR_INVALID_ARG = 1
GLIDE_ERR_UNSUPPORTED = 2
GLIDE_ERR_WORKSPACE_TOO_SMALL = 3
GLIDE_ERR_CAPACITY = 4
GLIDE_ERR_STATE = 5
GLIDE_ERR_CUDA = 6
GLIDE_ERR_SCRATCH_LIMIT = 7


class GlideError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {strerror(code)} (status {code})")


class glide_config(ctypes.Structure):
    _fields_ = [
        ("n_layers", ctypes.c_int32), ("batch", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
        ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("io_dtype", ctypes.c_int32),
        ("phi", ctypes.c_int32), ("merge", ctypes.c_int32),
        ("windows", ctypes.POINTER(ctypes.c_int64)), ("q_to_kv", ctypes.POINTER(ctypes.c_int32)),
        ("max_tokens", ctypes.c_int64), ("softmax_scale", ctypes.c_float), ("prefill_chunk", ctypes.c_int32),
        ("decode_chunk", ctypes.c_int32), ("decode_state_splits", ctypes.c_int32), ("decode_impl", ctypes.c_int32),
        ("prefill_impl", ctypes.c_int32),
        ("phi_wq", ctypes.c_void_p), ("phi_wk", ctypes.c_void_p), ("gated", ctypes.c_int32), ("reserved_", ctypes.c_int32),
    ]


class glide_layer_info_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int64) for n in ("window", "capacity", "n", "count", "head_slot", "n_evicted")]


_lib = None


def load_library() -> ctypes.CDLL:
    """dlopen libglide.so and declare the prototypes. Raises if the library is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} not built: run `python -m paper_2607_24788_b200.build` "
                           "(there is no CPU or PyTorch fallback for the GLIDE kernels)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    cfgp = ctypes.POINTER(glide_config)
    lib.glide_workspace_bytes.argtypes = [cfgp, ctypes.POINTER(ctypes.c_size_t)]
    lib.glide_create.argtypes = [cfgp, vp, ctypes.c_size_t, vp, ctypes.POINTER(vp)]
    lib.glide_prefill.argtypes = [vp, i32, i32, i64, vp, vp, vp, vp, vp]
    lib.glide_decode_step.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.glide_decode_step_noalloc.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.glide_prefill_gated.argtypes = [vp, i32, i32, i64, vp, vp, vp, vp, vp, vp]
    lib.glide_decode_step_gated.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.glide_export_gates.argtypes = [vp, i32, vp, vp]
    lib.glide_import_gates.argtypes = [vp, i32, vp, vp]
    lib.glide_decode_step_layers.argtypes = [vp, i32, i32, vp, vp, vp, vp, vp]
    lib.glide_reset_seq.argtypes = [vp, i32, vp]
    lib.glide_park_seq.argtypes = [vp, i32, vp]
    lib.glide_prefill_seq.argtypes = [vp, i32, i64, vp, vp, vp, vp, vp]
    lib.glide_seq_tokens.argtypes = [vp, i32, ctypes.POINTER(i64)]
    lib.glide_seq_layer_info.argtypes = [vp, i32, i32, vp, ctypes.POINTER(glide_layer_info_t)]
    lib.glide_destroy.argtypes = [vp]
    lib.glide_layer_info.argtypes = [vp, i32, vp, ctypes.POINTER(glide_layer_info_t)]
    lib.glide_export_state.argtypes = [vp, i32, vp, vp, vp, vp, vp]
    lib.glide_import_state.argtypes = [vp, i32, i64, vp, vp, vp, vp, vp]
    lib.glide_reset.argtypes = [vp, vp]
    lib.glide_device_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
    lib.glide_decode_launch_info.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32)]
    lib.glide_stream_schedule.argtypes = [cfgp, i32, i64, ctypes.POINTER(i32), i32, ctypes.POINTER(i32)]
    lib.glide_stream_schedule.restype = ctypes.c_int
    lib.glide_strerror.argtypes = [ctypes.c_int]
    lib.glide_strerror.restype = ctypes.c_char_p
    for name in ("glide_workspace_bytes", "glide_create", "glide_prefill", "glide_decode_step", "glide_destroy",
                 "glide_decode_step_noalloc", "glide_decode_step_layers", "glide_prefill_gated",
                 "glide_decode_step_gated", "glide_export_gates", "glide_import_gates",
                 "glide_layer_info", "glide_export_state", "glide_import_state", "glide_reset",
                 "glide_device_status", "glide_decode_launch_info"):
        getattr(lib, name).restype = ctypes.c_int
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load_library().glide_strerror(int(code)).decode()


def glide_stream_schedule(cfg, n_sms: int = 148, smem_limit: int = 232448):
    """The streaming decode kernel's all-layer schedule for `cfg` (host only): an int32 array [segments][12], see
    include/glide.h."""
    import numpy as np
    lib = load_library()
    n = ctypes.c_int32(0)
    _check(lib.glide_stream_schedule(ctypes.byref(cfg), n_sms, smem_limit, None, 0, ctypes.byref(n)), "glide_stream_schedule")
    rows = np.zeros((n.value, 12), dtype=np.int32)
    if n.value:
        _check(lib.glide_stream_schedule(ctypes.byref(cfg), n_sms, smem_limit,
                                         rows.ctypes.data_as(ctypes.POINTER(ctypes.c_int32)), n.value, ctypes.byref(n)),
               "glide_stream_schedule")
    return rows


def _check(code: int, where: str):
    if code != GLIDE_OK:
        raise GlideError(code, where)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device buffers must be contiguous CUDA tensors"
    return t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> Optional[int]:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream or None


def make_config(windows: Sequence[int], batch: int, n_q_heads: int, n_kv_heads: int, head_dim: int, max_tokens: int,
                dtype: torch.dtype = torch.bfloat16, q_to_kv: Optional[Sequence[int]] = None,
                softmax_scale: float = 0.0, prefill_chunk: int = 0, decode_chunk: int = 0,
                decode_state_splits: int = 0, decode_impl: int = 0, prefill_impl: int = 0, merge: int = 0,
                phi: int = GLIDE_PHI_SOFTMAX, phi_wq: Optional[torch.Tensor] = None,
                phi_wk: Optional[torch.Tensor] = None, gated: bool = False):
    """Returns (glide_config, keepalive) -- keepalive holds the host arrays the struct points to.
    phi = GLIDE_PHI_PROJ_SOFTMAX2 takes the projections phi_wq [L][H][d][d], phi_wk [L][Hkv][d][d] (device tensors of
    the I/O dtype; the library borrows them)."""
    win = (ctypes.c_int64 * len(windows))(*[int(w) for w in windows])
    qmap = (ctypes.c_int32 * len(q_to_kv))(*[int(x) for x in q_to_kv]) if q_to_kv is not None else None
    cfg = glide_config()
    cfg.n_layers, cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim = len(windows), batch, n_q_heads, n_kv_heads, head_dim
    cfg.io_dtype = {torch.float32: GLIDE_F32, torch.bfloat16: GLIDE_BF16}[dtype]
    cfg.phi, cfg.merge = int(phi), int(merge)
    if phi_wq is not None or phi_wk is not None:
        L = len(windows)
        assert phi_wq.shape == (L, n_q_heads, head_dim, head_dim) and phi_wk.shape == (L, n_kv_heads, head_dim, head_dim)
        assert phi_wq.dtype == dtype and phi_wk.dtype == dtype
    cfg.phi_wq, cfg.phi_wk = _ptr(phi_wq), _ptr(phi_wk)
    cfg.gated, cfg.reserved_ = int(bool(gated)), 0
    cfg.windows = ctypes.cast(win, ctypes.POINTER(ctypes.c_int64))
    cfg.q_to_kv = ctypes.cast(qmap, ctypes.POINTER(ctypes.c_int32)) if qmap is not None else None
    cfg.max_tokens = int(max_tokens)
    cfg.softmax_scale = float(softmax_scale)
    cfg.prefill_chunk, cfg.decode_chunk, cfg.decode_state_splits = int(prefill_chunk), int(decode_chunk), int(decode_state_splits)
    cfg.decode_impl = int(decode_impl)
    cfg.prefill_impl = int(prefill_impl)
    return cfg, (win, qmap, phi_wq, phi_wk)


def glide_workspace_bytes(cfg: glide_config) -> int:
    out = ctypes.c_size_t(0)
    _check(load_library().glide_workspace_bytes(ctypes.byref(cfg), ctypes.byref(out)), "glide_workspace_bytes")
    return int(out.value)


class Glide:
    """Owns a torch workspace and a glide_ctx; methods carry the C ABI's names."""

    def __init__(self, windows: Sequence[int], batch: int, n_q_heads: int, n_kv_heads: int, head_dim: int,
                 max_tokens: int, dtype: torch.dtype = torch.bfloat16, device="cuda", **kw):
        self.lib = load_library()
        self.device = torch.device(device)
        self.dtype = dtype
        self.L, self.B, self.H, self.Hkv, self.d = len(windows), batch, n_q_heads, n_kv_heads, head_dim
        self.windows = [int(w) for w in windows]
        self.max_tokens = int(max_tokens)
        self.dp = 2 * head_dim if kw.get("phi", GLIDE_PHI_SOFTMAX) == GLIDE_PHI_PROJ_SOFTMAX2 else head_dim
        self.gated = bool(kw.get("gated", False))
        self.cfg, self._keep = make_config(windows, batch, n_q_heads, n_kv_heads, head_dim, max_tokens, dtype, **kw)
        self.workspace_bytes = glide_workspace_bytes(self.cfg)
        with torch.cuda.device(self.device):
            # 256-byte alignment is required; 2 MiB keeps the library's own 2 MiB-aligned offsets of the streamed
            # arrays aligned in device memory as well
            align = 2 << 20
            self.workspace = torch.empty(self.workspace_bytes + align, dtype=torch.uint8, device=self.device)
            base = self.workspace.data_ptr()
            self._ws_ptr = (base + align - 1) // align * align
            handle = ctypes.c_void_p()
            _check(self.lib.glide_create(ctypes.byref(self.cfg), self._ws_ptr, self.workspace_bytes, _stream(None),
                                         ctypes.byref(handle)), "glide_create")
        self._h = handle

    # -- the four calls of the hot path ---------------------------------------------------------
    def glide_prefill(self, q: Optional[torch.Tensor], k: torch.Tensor, v: torch.Tensor,
                      out: Optional[torch.Tensor] = None, layer_begin: int = 0, layer_count: Optional[int] = None,
                      stream=None) -> None:
        lc = self.L - layer_begin if layer_count is None else layer_count
        T = k.shape[2]
        assert k.shape == (lc, self.B, T, self.Hkv, self.d) and v.shape == k.shape and k.dtype == self.dtype
        if out is not None:
            assert q is not None and q.shape == (lc, self.B, T, self.H, self.d) and out.shape == q.shape
        _check(self.lib.glide_prefill(self._h, layer_begin, lc, T, _ptr(q), _ptr(k), _ptr(v), _ptr(out),
                                      _stream(stream)), "glide_prefill")

    def glide_decode_step(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: torch.Tensor,
                          stream=None) -> None:
        assert q.shape == (self.L, self.B, self.H, self.d) and out.shape == q.shape
        assert k.shape == (self.L, self.B, self.Hkv, self.d) and v.shape == k.shape
        assert q.dtype == k.dtype == v.dtype == out.dtype == self.dtype
        _check(self.lib.glide_decode_step(self._h, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _stream(stream)),
               "glide_decode_step")

    def glide_prefill_gated(self, q: Optional[torch.Tensor], k: torch.Tensor, v: torch.Tensor,
                            gate: Optional[torch.Tensor], out: Optional[torch.Tensor] = None, layer_begin: int = 0,
                            layer_count: Optional[int] = None, stream=None) -> None:
        """glide_prefill of a gated context: gate fp32 [layer_count][B][T][H_kv] in (0, 1], or None for gates of 1."""
        lc = self.L - layer_begin if layer_count is None else layer_count
        T = k.shape[2]
        assert k.shape == (lc, self.B, T, self.Hkv, self.d) and v.shape == k.shape and k.dtype == self.dtype
        assert gate is None or (gate.shape == (lc, self.B, T, self.Hkv) and gate.dtype == torch.float32)
        if out is not None:
            assert q is not None and q.shape == (lc, self.B, T, self.H, self.d) and out.shape == q.shape
        _check(self.lib.glide_prefill_gated(self._h, layer_begin, lc, T, _ptr(q), _ptr(k), _ptr(v), _ptr(gate), _ptr(out),
                                            _stream(stream)), "glide_prefill_gated")

    def glide_decode_step_gated(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, gate: Optional[torch.Tensor],
                                out: torch.Tensor, stream=None) -> None:
        """glide_decode_step of a gated context: gate fp32 [L][B][H_kv] in (0, 1], or None for gates of 1."""
        assert q.shape == (self.L, self.B, self.H, self.d) and out.shape == q.shape
        assert k.shape == (self.L, self.B, self.Hkv, self.d) and v.shape == k.shape
        assert q.dtype == k.dtype == v.dtype == out.dtype == self.dtype
        assert gate is None or (gate.shape == (self.L, self.B, self.Hkv) and gate.dtype == torch.float32)
        _check(self.lib.glide_decode_step_gated(self._h, _ptr(q), _ptr(k), _ptr(v), _ptr(gate), _ptr(out),
                                                _stream(stream)), "glide_decode_step_gated")

    def glide_decode_step_layers(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: torch.Tensor,
                                 layer_begin: int, layer_count: int, stream=None) -> None:
        """glide_decode_step for the layers [layer_begin, layer_begin + layer_count); tensors are the range's."""
        assert q.shape == (layer_count, self.B, self.H, self.d) and out.shape == q.shape
        assert k.shape == (layer_count, self.B, self.Hkv, self.d) and v.shape == k.shape
        assert q.dtype == k.dtype == v.dtype == out.dtype == self.dtype
        _check(self.lib.glide_decode_step_layers(self._h, int(layer_begin), int(layer_count), _ptr(q), _ptr(k), _ptr(v),
                                                 _ptr(out), _stream(stream)), "glide_decode_step_layers")

    def glide_decode_step_noalloc(self, q: torch.Tensor, k: torch.Tensor, v: torch.Tensor, out: torch.Tensor,
                                  stream=None) -> None:
        """glide_decode_step for callers that must not allocate: the step's split-K scratch lives in a static
        buffer inside the library instead of the workspace (see include/glide.h for the limits)."""
        assert q.shape == (self.L, self.B, self.H, self.d) and out.shape == q.shape
        assert k.shape == (self.L, self.B, self.Hkv, self.d) and v.shape == k.shape
        assert q.dtype == k.dtype == v.dtype == out.dtype == self.dtype
        _check(self.lib.glide_decode_step_noalloc(self._h, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _stream(stream)),
               "glide_decode_step_noalloc")

    # -- sequences of different lengths: every slot of the batch has its own position ---------------
    def glide_reset_seq(self, b: int, stream=None) -> None:
        """Slot b starts an empty sequence; the other slots are untouched."""
        _check(self.lib.glide_reset_seq(self._h, int(b), _stream(stream)), "glide_reset_seq")

    def glide_park_seq(self, b: int, stream=None) -> None:
        """Slot b holds no sequence: decode steps skip it until glide_reset_seq starts a new one there."""
        _check(self.lib.glide_park_seq(self._h, int(b), _stream(stream)), "glide_park_seq")

    def glide_prefill_seq(self, b: int, q: Optional[torch.Tensor], k: torch.Tensor, v: torch.Tensor,
                          out: Optional[torch.Tensor] = None, stream=None) -> None:
        """glide_prefill for slot b alone, all layers: q, out [L][T][H][d]; k, v [L][T][H_kv][d]."""
        T = k.shape[1]
        assert k.shape == (self.L, T, self.Hkv, self.d) and v.shape == k.shape and k.dtype == self.dtype
        if out is not None:
            assert q is not None and q.shape == (self.L, T, self.H, self.d) and out.shape == q.shape
        _check(self.lib.glide_prefill_seq(self._h, int(b), T, _ptr(q), _ptr(k), _ptr(v), _ptr(out), _stream(stream)),
               "glide_prefill_seq")

    def glide_seq_tokens(self, b: int) -> int:
        n = ctypes.c_int64(0)
        _check(self.lib.glide_seq_tokens(self._h, int(b), ctypes.byref(n)), "glide_seq_tokens")
        return int(n.value)

    def glide_seq_layer_info(self, layer: int, b: int) -> dict:
        info = glide_layer_info_t()
        _check(self.lib.glide_seq_layer_info(self._h, layer, int(b), _stream(None), ctypes.byref(info)),
               "glide_seq_layer_info")
        return {n: int(getattr(info, n)) for n, _ in glide_layer_info_t._fields_}

    def glide_destroy(self) -> None:
        if getattr(self, "_h", None):
            self.lib.glide_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.glide_destroy()
        except Exception:
            pass

    # -- support ----------------------------------------------------------------------------------
    def glide_layer_info(self, layer: int) -> dict:
        info = glide_layer_info_t()
        _check(self.lib.glide_layer_info(self._h, layer, _stream(None), ctypes.byref(info)), "glide_layer_info")
        return {n: int(getattr(info, n)) for n, _ in glide_layer_info_t._fields_}

    def capacity(self, layer: int) -> int:
        return min(self.windows[layer], self.max_tokens)

    def glide_export_state(self, layer: int):
        cap = self.capacity(layer)
        rk = torch.empty((self.B, self.Hkv, cap, self.d), dtype=self.dtype, device=self.device)
        rv = torch.empty_like(rk)
        S = torch.empty((self.B, self.Hkv, self.dp, self.d), dtype=torch.float32, device=self.device)
        z = torch.empty((self.B, self.Hkv, self.dp), dtype=torch.float32, device=self.device)
        _check(self.lib.glide_export_state(self._h, layer, _ptr(rk) if cap else None, _ptr(rv) if cap else None,
                                           _ptr(S), _ptr(z), _stream(None)), "glide_export_state")
        return rk, rv, S, z

    def glide_import_state(self, layer: int, n: int, ringK=None, ringV=None, S=None, z=None) -> None:
        _check(self.lib.glide_import_state(self._h, layer, int(n), _ptr(ringK), _ptr(ringV), _ptr(S), _ptr(z),
                                           _stream(None)), "glide_import_state")

    def glide_export_gates(self, layer: int) -> torch.Tensor:
        """[B][H_kv][capacity] fp32: the gates of the ring's tokens (gated contexts)."""
        gates = torch.empty((self.B, self.Hkv, self.capacity(layer)), dtype=torch.float32, device=self.device)
        _check(self.lib.glide_export_gates(self._h, layer, _ptr(gates), _stream(None)), "glide_export_gates")
        return gates

    def glide_import_gates(self, layer: int, gates: torch.Tensor) -> None:
        assert gates.shape == (self.B, self.Hkv, self.capacity(layer)) and gates.dtype == torch.float32
        _check(self.lib.glide_import_gates(self._h, layer, _ptr(gates), _stream(None)), "glide_import_gates")

    def glide_reset(self) -> None:
        _check(self.lib.glide_reset(self._h, _stream(None)), "glide_reset")

    def glide_device_status(self) -> int:
        out = ctypes.c_int32(0)
        _check(self.lib.glide_device_status(self._h, _stream(None), ctypes.byref(out)), "glide_device_status")
        return int(out.value)

    def glide_decode_launch_info(self) -> dict:
        a, b, c = ctypes.c_int32(0), ctypes.c_int32(0), ctypes.c_int32(0)
        _check(self.lib.glide_decode_launch_info(self._h, ctypes.byref(a), ctypes.byref(b), ctypes.byref(c)),
               "glide_decode_launch_info")
        return dict(launches=a.value, work_items=b.value, grid=c.value)
