"""Seeded synthetic q/k/v generator shared by the CUDA path's tests, the benchmark and the oracle's tests.

It holds none of the attention arithmetic.  Every element of the logical
tensors q/k/v[layer][batch][token][head][feature] is addressable on its own:

    value = TABLE[ top16( mix64(linear_index + seed * GOLDEN) ) ]

where mix64 is the splitmix64 finaliser (integer only) and TABLE is a
65 536-entry inverse-normal-CDF table (quantiles (i + 1/2)/65536, times a scale,
rounded once to the I/O dtype).  Integer hashing plus a table lookup gives the
same bits on CPU and on the GPU, so a test can regenerate any slice of a
prompt that is far too large to store (the 128K-context workloads hold
hundreds of GB of q/k/v) and hand exactly the same numbers to both sides.
"""
from __future__ import annotations

import math
from typing import Dict, Tuple

import torch

Q, K, V = 0, 1, 2
_T_MAX = 1 << 22          # tokens per sequence the index packing allows
_GOLDEN = -7046029254386353131   # 0x9E3779B97F4A7C15 as int64
_M1 = -4658895280553007687       # 0xBF58476D1CE4E5B9
_M2 = -7723592293110705685       # 0x94D049BB133111EB

_tables: Dict[Tuple[float, torch.dtype, str], torch.Tensor] = {}


def normal_table(scale: float, dtype: torch.dtype, device="cpu") -> torch.Tensor:
    """[65536] values of dtype: Phi^-1((i + 1/2)/65536) * scale, computed in fp64, rounded once."""
    key = (float(scale), dtype, str(device))
    if key not in _tables:
        p = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
        t = (torch.special.ndtri(p) * float(scale)).to(dtype)
        _tables[key] = t.to(device)
    return _tables[key]


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical right shift of int64."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def _mix64(x: torch.Tensor) -> torch.Tensor:
    x = (x ^ _lsr(x, 30)) * _M1
    x = (x ^ _lsr(x, 27)) * _M2
    return x ^ _lsr(x, 31)


def generate(seed: int, tensor: int, layers, batches, tokens, n_heads: int, d: int, *, n_layers: int, batch: int,
             scale: float, dtype: torch.dtype, device="cpu") -> torch.Tensor:
    """Slice [len(layers)][len(batches)][len(tokens)][n_heads][d] of logical tensor `tensor` (Q, K or V).

    layers / batches / tokens are ranges or 1-D integer sequences of absolute
    indices; n_layers and batch are the logical extents used to pack the index
    (they must be the same for every call that addresses one workload)."""
    dev = torch.device(device)
    li = torch.as_tensor(list(layers) if not isinstance(layers, torch.Tensor) else layers, dtype=torch.int64, device=dev)
    bi = torch.as_tensor(list(batches) if not isinstance(batches, torch.Tensor) else batches, dtype=torch.int64, device=dev)
    ti = torch.as_tensor(list(tokens) if not isinstance(tokens, torch.Tensor) else tokens, dtype=torch.int64, device=dev)
    assert int(ti.max()) < _T_MAX if ti.numel() else True
    hi = torch.arange(n_heads, dtype=torch.int64, device=dev)
    ri = torch.arange(d, dtype=torch.int64, device=dev)
    # fixed packing: 64 heads x 256 features per token
    assert n_heads <= 64 and d <= 256
    idx = ((int(tensor) * n_layers + li)[:, None, None, None, None] * batch + bi[None, :, None, None, None])
    idx = (idx * _T_MAX + ti[None, None, :, None, None]) * 64 + hi[None, None, None, :, None]
    idx = idx * 256 + ri[None, None, None, None, :]
    offset = ((int(seed) * _GOLDEN + (1 << 63)) % (1 << 64)) - (1 << 63)   # wrap to int64
    h = _mix64(idx + offset)
    tab = normal_table(scale, dtype, dev)
    return tab[_lsr(h, 48)]


class Workload:
    """Addressable synthetic q/k/v for one configuration."""

    def __init__(self, seed: int, n_layers: int, batch: int, H: int, Hkv: int, d: int, dtype: torch.dtype,
                 scale: float, v_scale: float = None):
        """scale: standard deviation of the q and k entries (and of v unless v_scale gives its own)."""
        self.seed, self.L, self.B, self.H, self.Hkv, self.d = seed, n_layers, batch, H, Hkv, d
        self.dtype, self.scale = dtype, scale
        self.v_scale = scale if v_scale is None else v_scale

    def _gen(self, tensor, layers, batches, tokens, heads, device):
        return generate(self.seed, tensor, layers, batches, tokens, heads, self.d, n_layers=self.L, batch=self.B,
                        scale=self.v_scale if tensor == V else self.scale, dtype=self.dtype, device=device)

    def qkv(self, layers, batches, tokens, device="cpu"):
        """(q [l][b][t][H][d], k [l][b][t][Hkv][d], v likewise)."""
        return (self._gen(Q, layers, batches, tokens, self.H, device),
                self._gen(K, layers, batches, tokens, self.Hkv, device),
                self._gen(V, layers, batches, tokens, self.Hkv, device))

    def kv(self, layers, batches, tokens, device="cpu"):
        return (self._gen(K, layers, batches, tokens, self.Hkv, device),
                self._gen(V, layers, batches, tokens, self.Hkv, device))

    def decode_qkv(self, t: int, device="cpu"):
        """One token for every layer and sequence, in the decode layouts
        q [L][B][H][d], k,v [L][B][Hkv][d]."""
        q, k, v = self.qkv(range(self.L), range(self.B), [t], device)
        return q[:, :, 0].contiguous(), k[:, :, 0].contiguous(), v[:, :, 0].contiguous()


def default_value_scale(d: int, unit_variance: bool) -> float:
    """N(0,1) for the tiny fp32 configuration, N(0,1)/sqrt(d) for the Llama/Mistral-shaped ones."""
    return 1.0 if unit_variance else 1.0 / math.sqrt(d)
