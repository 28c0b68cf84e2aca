"""ctypes wrapper around the plain-C fp64 oracle (test infrastructure only).

The C file holds every bit of arithmetic; this module only builds it with gcc,
marshals numpy float64 arrays, and loops cells over (layer, sequence).
Used by tests, the smoke check and the benchmark's CPU-baseline leg -- never by
the product path.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "glide_oracle.c")
_LIB = os.path.join(_HERE, "libglide_oracle.so")
_lib = None

_f64p = ctypes.POINTER(ctypes.c_double)
_i64p = ctypes.POINTER(ctypes.c_int64)
_i32p = ctypes.POINTER(ctypes.c_int32)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (building the checker is not using it)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is not None:
        return _lib
    lib = ctypes.CDLL(build())
    lib.glide_oracle_bruteforce.argtypes = [
        ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int64, ctypes.c_double, ctypes.c_int,
        _i32p, _f64p, _f64p, _f64p, ctypes.c_int64, _i64p, _f64p]
    lib.glide_oracle_bruteforce.restype = None
    lib.glide_oracle_cell_new.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int64,
                                          ctypes.c_double, ctypes.c_int, _i32p]
    lib.glide_oracle_cell_new.restype = ctypes.c_void_p
    lib.glide_oracle_cell_free.argtypes = [ctypes.c_void_p]
    lib.glide_oracle_cell_free.restype = None
    lib.glide_oracle_cell_reset.argtypes = [ctypes.c_void_p]
    lib.glide_oracle_cell_reset.restype = None
    lib.glide_oracle_cell_decode.argtypes = [ctypes.c_void_p, _f64p, _f64p, _f64p, _f64p]
    lib.glide_oracle_cell_decode.restype = None
    lib.glide_oracle_stack_decode.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.c_int64,
                                              _f64p, _f64p, _f64p, _f64p, ctypes.c_int]
    lib.glide_oracle_stack_decode.restype = ctypes.c_int
    lib.glide_oracle_cell_prefill.argtypes = [ctypes.c_void_p, ctypes.c_int64, _f64p, _f64p, _f64p,
                                              ctypes.c_int64, _i64p, _f64p]
    lib.glide_oracle_cell_prefill.restype = None
    lib.glide_oracle_cell_info.argtypes = [ctypes.c_void_p, _i64p, _i64p, _i64p, _i64p]
    lib.glide_oracle_cell_info.restype = None
    lib.glide_oracle_cell_slot_tokens.argtypes = [ctypes.c_void_p, _i64p]
    lib.glide_oracle_cell_slot_tokens.restype = None
    lib.glide_oracle_cell_export.argtypes = [ctypes.c_void_p, _f64p, _f64p, _f64p, _f64p]
    lib.glide_oracle_cell_export.restype = None
    lib.glide_oracle_bruteforce_ex.argtypes = lib.glide_oracle_bruteforce.argtypes + [ctypes.c_int, _f64p, _f64p, _f64p]
    lib.glide_oracle_bruteforce_ex.restype = None
    lib.glide_oracle_cell_set_phi.argtypes = [ctypes.c_void_p, ctypes.c_int, _f64p, _f64p]
    lib.glide_oracle_cell_set_phi.restype = None
    lib.glide_oracle_cell_decode_ex.argtypes = [ctypes.c_void_p, _f64p, _f64p, _f64p, _f64p, _f64p]
    lib.glide_oracle_cell_decode_ex.restype = None
    lib.glide_oracle_stack_decode_ex.argtypes = [ctypes.POINTER(ctypes.c_void_p), ctypes.c_int64,
                                                 _f64p, _f64p, _f64p, _f64p, _f64p, ctypes.c_int]
    lib.glide_oracle_stack_decode_ex.restype = ctypes.c_int
    lib.glide_oracle_cell_prefill_ex.argtypes = [ctypes.c_void_p, ctypes.c_int64, _f64p, _f64p, _f64p, _f64p,
                                                 ctypes.c_int64, _i64p, _f64p]
    lib.glide_oracle_cell_prefill_ex.restype = None
    lib.glide_oracle_cell_export_gates.argtypes = [ctypes.c_void_p, _f64p]
    lib.glide_oracle_cell_export_gates.restype = None
    lib.glide_oracle_max_threads.argtypes = []
    lib.glide_oracle_max_threads.restype = ctypes.c_int
    _lib = lib
    return lib


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _ptr(a: Optional[np.ndarray], typ=_f64p):
    return None if a is None else a.ctypes.data_as(typ)


def default_q_to_kv(H: int, Hkv: int) -> np.ndarray:
    """Contiguous GQA groups (Llama/Mistral convention): head h reads KV head h // (H/Hkv)."""
    assert H % Hkv == 0
    return (np.arange(H, dtype=np.int32) // (H // Hkv)).astype(np.int32)


def max_threads() -> int:
    return int(_load().glide_oracle_max_threads())


def bruteforce(q, k, v, w: int, scale: float, q_to_kv=None, sel: Optional[Sequence[int]] = None,
               merge: int = 0, phi: int = 0, wq=None, wk=None, gate=None) -> np.ndarray:
    """Form B: the defining sums over the full history (merge: 0 shared normaliser, 1 / 2 the appendix' sums of
    two separately normalised terms with the evicted-token / all-token state).

    q [T][H][d], k,v [T][Hkv][d] -> out [T or len(sel)][H][d] (float64).
    phi 1: the learned feature map with wq [H][d][d], wk [Hkv][d][d]; gate [T][Hkv]: the decay each token brings."""
    lib = _load()
    q, k, v = _f64(q), _f64(k), _f64(v)
    T, H, d = q.shape
    Hkv = k.shape[1]
    m = default_q_to_kv(H, Hkv) if q_to_kv is None else np.ascontiguousarray(q_to_kv, dtype=np.int32)
    wq = None if wq is None else _f64(wq)
    wk = None if wk is None else _f64(wk)
    gate = None if gate is None else _f64(gate)
    assert (phi == 0) == (wq is None) == (wk is None)
    if phi:
        assert wq.shape == (H, d, d) and wk.shape == (Hkv, d, d)
    if gate is not None:
        assert gate.shape == (T, Hkv)
    if sel is None:
        out = np.empty((T, H, d), dtype=np.float64)
        lib.glide_oracle_bruteforce_ex(T, H, Hkv, d, int(w), float(scale), int(merge), _ptr(m, _i32p), _ptr(q), _ptr(k),
                                       _ptr(v), 0, None, _ptr(out), int(phi), _ptr(wq), _ptr(wk), _ptr(gate))
    else:
        s = np.ascontiguousarray(sel, dtype=np.int64)
        out = np.empty((len(s), H, d), dtype=np.float64)
        lib.glide_oracle_bruteforce_ex(T, H, Hkv, d, int(w), float(scale), int(merge), _ptr(m, _i32p), _ptr(q), _ptr(k),
                                       _ptr(v), len(s), _ptr(s, _i64p), _ptr(out), int(phi), _ptr(wq), _ptr(wk),
                                       _ptr(gate))
    return out


class Cell:
    """Form A for one (layer, sequence): ring of the last w tokens + S/z state."""

    def __init__(self, H: int, Hkv: int, d: int, w: int, scale: float, q_to_kv=None, merge: int = 0, phi: int = 0,
                 wq=None, wk=None):
        self._lib = _load()
        self.merge = int(merge)
        self.H, self.Hkv, self.d, self.w, self.scale = H, Hkv, d, int(w), float(scale)
        self.q_to_kv = default_q_to_kv(H, Hkv) if q_to_kv is None else np.ascontiguousarray(q_to_kv, dtype=np.int32)
        self._h = ctypes.c_void_p(self._lib.glide_oracle_cell_new(H, Hkv, d, int(w), float(scale), int(merge),
                                                                   _ptr(self.q_to_kv, _i32p)))
        self.phi, self.dp = int(phi), (2 * d if phi else d)
        if phi:
            wq, wk = _f64(wq), _f64(wk)
            assert wq.shape == (H, d, d) and wk.shape == (Hkv, d, d)
            self._lib.glide_oracle_cell_set_phi(self._h, int(phi), _ptr(wq), _ptr(wk))

    def __del__(self):
        if getattr(self, "_h", None):
            self._lib.glide_oracle_cell_free(self._h)
            self._h = None

    def reset(self):
        self._lib.glide_oracle_cell_reset(self._h)

    def decode(self, q, k, v, gate=None) -> np.ndarray:
        q, k, v = _f64(q), _f64(k), _f64(v)
        assert q.shape == (self.H, self.d) and k.shape == (self.Hkv, self.d) and v.shape == k.shape
        gate = None if gate is None else _f64(gate)
        assert gate is None or gate.shape == (self.Hkv,)
        out = np.empty((self.H, self.d), dtype=np.float64)
        self._lib.glide_oracle_cell_decode_ex(self._h, _ptr(q), _ptr(k), _ptr(v), _ptr(gate), _ptr(out))
        return out

    def prefill(self, q, k, v, sel: Optional[Sequence[int]] = None, outputs: bool = True, gate=None) -> Optional[np.ndarray]:
        """Append T tokens. Outputs for all positions (sel None), for sel, or none (outputs=False)."""
        k, v = _f64(k), _f64(v)
        T = k.shape[0]
        assert k.shape == (T, self.Hkv, self.d) and v.shape == k.shape
        gate = None if gate is None else _f64(gate)
        assert gate is None or gate.shape == (T, self.Hkv)
        if not outputs:
            self._lib.glide_oracle_cell_prefill_ex(self._h, T, None, _ptr(k), _ptr(v), _ptr(gate), 0, None, None)
            return None
        q = _f64(q)
        assert q.shape == (T, self.H, self.d)
        if sel is None:
            out = np.empty((T, self.H, self.d), dtype=np.float64)
            self._lib.glide_oracle_cell_prefill_ex(self._h, T, _ptr(q), _ptr(k), _ptr(v), _ptr(gate), -1, None, _ptr(out))
        else:
            s = np.ascontiguousarray(sel, dtype=np.int64)
            out = np.empty((len(s), self.H, self.d), dtype=np.float64)
            self._lib.glide_oracle_cell_prefill_ex(self._h, T, _ptr(q), _ptr(k), _ptr(v), _ptr(gate), len(s),
                                                   _ptr(s, _i64p), _ptr(out))
        return out

    def info(self) -> dict:
        vals = [ctypes.c_int64() for _ in range(4)]
        self._lib.glide_oracle_cell_info(self._h, *[ctypes.byref(x) for x in vals])
        return dict(n=vals[0].value, count=vals[1].value, head_slot=vals[2].value, n_evicted=vals[3].value)

    def slot_tokens(self) -> np.ndarray:
        tok = np.empty((self.w,), dtype=np.int64)
        if self.w:
            self._lib.glide_oracle_cell_slot_tokens(self._h, _ptr(tok, _i64p))
        return tok

    def export(self):
        """(ringK [Hkv][w][d], ringV, S [Hkv][dp][d], z [Hkv][dp]) as float64 copies (dp: the feature dimension)."""
        rk = np.zeros((self.Hkv, self.w, self.d), dtype=np.float64)
        rv = np.zeros_like(rk)
        S = np.empty((self.Hkv, self.dp, self.d), dtype=np.float64)
        z = np.empty((self.Hkv, self.dp), dtype=np.float64)
        self._lib.glide_oracle_cell_export(self._h, _ptr(rk) if self.w else None, _ptr(rv) if self.w else None,
                                           _ptr(S), _ptr(z))
        return rk, rv, S, z

    def export_gates(self) -> np.ndarray:
        """[Hkv][w]: the gates of the ring's tokens, slot order."""
        gr = np.zeros((self.Hkv, self.w), dtype=np.float64)
        if self.w:
            self._lib.glide_oracle_cell_export_gates(self._h, _ptr(gr))
        return gr


class Stack:
    """[n_layers][batch] grid of cells with the library's decode/prefill tensor layouts.

    decode: q [L][B][H][d], k,v [L][B][Hkv][d] (gate [L][B][Hkv]) -> out [L][B][H][d]
    prefill (layers lb..lb+lc): q [lc][B][T][H][d], k,v [lc][B][T][Hkv][d] (gate [lc][B][T][Hkv]).
    phi 1: wq [L][H][d][d], wk [L][Hkv][d][d]."""

    def __init__(self, windows: Sequence[int], batch: int, H: int, Hkv: int, d: int, scale: float, q_to_kv=None,
                 merge: int = 0, phi: int = 0, wq=None, wk=None):
        self.L, self.B, self.H, self.Hkv, self.d = len(windows), batch, H, Hkv, d
        self.windows = [int(w) for w in windows]
        self.cells = [[Cell(H, Hkv, d, w, scale, q_to_kv, merge, phi, None if wq is None else wq[l],
                            None if wk is None else wk[l]) for _ in range(batch)]
                      for l, w in enumerate(self.windows)]
        flat = [c._h for row in self.cells for c in row]
        self._handles = (ctypes.c_void_p * len(flat))(*flat)
        self._lib = _load()

    def decode(self, q, k, v, threads: int = 0, gate=None) -> np.ndarray:
        q, k, v = _f64(q), _f64(k), _f64(v)
        assert q.shape == (self.L, self.B, self.H, self.d)
        assert k.shape == (self.L, self.B, self.Hkv, self.d) and v.shape == k.shape
        gate = None if gate is None else _f64(gate)
        assert gate is None or gate.shape == (self.L, self.B, self.Hkv)
        out = np.empty_like(q)
        self.threads_used = self._lib.glide_oracle_stack_decode_ex(self._handles, self.L * self.B, _ptr(q), _ptr(k),
                                                                   _ptr(v), _ptr(gate), _ptr(out), int(threads))
        return out

    def prefill(self, q, k, v, layer_begin: int = 0, sel=None, outputs: bool = True, gate=None):
        k, v = _f64(k), _f64(v)
        lc = k.shape[0]
        outs = []
        for li in range(lc):
            row = []
            for b in range(self.B):
                cell = self.cells[layer_begin + li][b]
                row.append(cell.prefill(None if not outputs else q[li][b], k[li][b], v[li][b], sel=sel,
                                        outputs=outputs, gate=None if gate is None else gate[li][b]))
            outs.append(row)
        if not outputs:
            return None
        return np.asarray(outs)  # [lc][B][T or len(sel)][H][d]
