"""The benchmark configurations (shapes, per-layer windows, controls) and the analytic cost model.

Windows follow the layer-wise adaptive policy of the paper (Sec. III-B/III-C):
each layer l has its own effective window w_l = w - delta_l.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from typing import List, Sequence


@dataclass(frozen=True)
class GlideShape:
    name: str
    n_layers: int
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    windows: tuple          # per layer
    context: int            # prompt tokens absorbed before decode
    decode_steps: int
    dtype: str              # "f32" | "bf16"  (q,k,v,out and ring; S,z always fp32)
    unit_variance: bool = False   # q,k,v ~ N(0,1) (True) or N(0,1)/sqrt(d)
    prefill_chunk: int = 0
    seed: int = 0
    value_scales: tuple = None    # (std of q and k entries, std of v entries) when the defaults above are not wanted

    @property
    def max_tokens(self) -> int:
        return self.context + self.decode_steps

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2


def blockwise_windows(w: int, deltas: Sequence[int], split: Sequence[int]) -> List[int]:
    """Block-wise delta allocation (Sec. III-C, Algorithm 1's Split/Assign): layers of block b get
    window w - delta_b."""
    out: List[int] = []
    for delta, n in zip(deltas, split):
        out += [w - delta] * n
    return out


def mistral_decay_windows(n_layers: int = 32) -> List[int]:
    """w_l = 4096 * 2^(-l/4), rounded to the nearest multiple of 16, floored at 32."""
    out = []
    for l in range(n_layers):
        x = 4096.0 * 2.0 ** (-l / 4.0)
        out.append(max(32, int(round(x / 16.0)) * 16))
    return out


_LLAMA = dict(n_layers=32, n_q_heads=32, n_kv_heads=8, head_dim=128, dtype="bf16")
_DEPTH_DECREASING = tuple([4096] * 4 + [1024] * 8 + [256] * 12 + [64] * 8)

C0 = GlideShape("c0_tiny_f32", 1, 1, 4, 4, 64, (64,), 512, 16, "f32", unit_variance=True)
C1 = GlideShape("c1_llama8b_b1_32k", batch=1, windows=_DEPTH_DECREASING, context=32768, decode_steps=256, **_LLAMA)
C2 = GlideShape("c2_llama8b_b16_16k", batch=16, windows=_DEPTH_DECREASING, context=16384, decode_steps=512, **_LLAMA)
C2_UNIFORM = replace(C2, name="c2_control_uniform_w1024", windows=tuple([1024] * 32))
C3 = GlideShape("c3_llama8b_b4_128k", batch=4, windows=tuple([131072] * 2 + [2048] * 6 + [128] * 24),
                context=131072, decode_steps=256, **_LLAMA)
C3_FULLKV = replace(C3, name="c3_control_full_kv", windows=tuple([131072 + 256] * 32))
C4 = GlideShape("c4_mistral7b_b8_8k_chunked", batch=8, windows=tuple(mistral_decay_windows()), context=8192,
                decode_steps=128, prefill_chunk=256, **_LLAMA)
# paper-shaped extra: block-wise (0, w/2, w) at w = 1024 with a 10/12/10 split -> exercises w_l = 0 layers
P1 = GlideShape("p1_blockwise_0_half_w", batch=1, windows=tuple(blockwise_windows(1024, (0, 512, 1024), (10, 12, 10))),
                context=32768, decode_steps=256, **_LLAMA)

ALL = {c.name: c for c in (C0, C1, C2, C2_UNIFORM, C3, C3_FULLKV, C4, P1)}


# ---------------------------------------------------------------------------------------------
# Cost model
# ---------------------------------------------------------------------------------------------
def kv_io_bytes_per_token(windows: Sequence[int], n_kv_heads: int = 8, head_dim: int = 128, elem_bytes: int = 2) -> int:
    """KV-cache bytes read per generated token, the paper's accounting (Fig. 4, Table 1 last column):
    sum over layers of (window tokens) x (K and V rows of every KV head). State I/O counts as zero there."""
    return sum(int(w) for w in windows) * 2 * n_kv_heads * head_dim * elem_bytes


def decode_step_bytes(shape: GlideShape, n: int, feature_mult: int = 1) -> int:
    """Algorithmic bytes one decode step must move when n tokens are already absorbed (all sequences):
    per layer, the window slots read (one of them the token that leaves the window), the recurrent state
    read and written once the layer evicts, the new K/V row written, and q,k,v in / out.
    feature_mult: feature dimension of the linear part over head_dim (2 for the learned map)."""
    H, Hkv, d, eb = shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.elem_bytes
    total = 0
    for w in shape.windows:
        total += 2 * min(w, n + 1) * Hkv * d * eb
        if n >= w:
            total += 2 * feature_mult * (Hkv * d * d + Hkv * d) * 4
        if w > 0:
            total += 2 * Hkv * d * eb
        total += (2 * H + 2 * Hkv) * d * eb
    return total * shape.batch


def decode_step_stream_bytes(shape: GlideShape, n: int, feature_mult: int = 1) -> int:
    """The roofline bytes of one decode step as the task states them: per layer and sequence the window's K and V rows,
    2 w H_kv d elem, plus the recurrent state S, z read and written once the layer evicts (all sequences)."""
    Hkv, d, eb = shape.n_kv_heads, shape.head_dim, shape.elem_bytes
    total = 0
    for w in shape.windows:
        total += 2 * min(w, n + 1) * Hkv * d * eb
        if n >= w:
            total += 2 * feature_mult * (Hkv * d * d + Hkv * d) * 4
    return total * shape.batch


def theoretical_speedup(alpha: float, w: float, d: float) -> float:
    """Per-token speedup of a three-equal-block (0, alpha*w, w) allocation over the (0,0,0) hybrid
    (Sec. III-C): S = 1 + (1 + alpha) / ((2 + 3d/w) - alpha)."""
    return 1.0 + (1.0 + alpha) / ((2.0 + 3.0 * d / w) - alpha)


def blockwise_cost(L: int, w: float, d: float, alpha: float) -> float:
    """Per-token cost of the (0, alpha*w, w) allocation with three equal blocks: Lwd/3 + Lw(1-alpha)d/3 + Ld^2."""
    return L * w * d / 3.0 + L * w * (1.0 - alpha) * d / 3.0 + L * d * d


def three_block_split(n_layers: int) -> List[int]:
    """Split of Algorithm 1: early, middle and last block of contiguous layers, as equal as the layer count allows
    (a remainder goes to the earlier blocks, which keep the larger windows)."""
    base, rem = divmod(n_layers, 3)
    return [base + (1 if b < rem else 0) for b in range(3)]


def blockwise_delta_candidates(w: int) -> List[int]:
    """The search space of Algorithm 1 for the middle block: delta in {0, w/2, 15w/16, w}."""
    return [0, w // 2, (15 * w) // 16, w]


def blockwise_allocate(n_layers: int, w: int, task_acc_eval, split: Sequence[int] = None):
    """Block-wise delta allocation (Algorithm 1).  The early block keeps delta = 0 (window w), the last block gets
    delta = w (window 0: linear attention only); each candidate delta of the middle block is scored by
    `task_acc_eval(windows) -> float` (the caller's task accuracy of the model run with these per-layer windows) and
    the best one is kept.  Among equal scores the larger delta wins: it reads less of the cache for the same accuracy.
    Returns (windows, delta_mid, {delta: score})."""
    split = list(split) if split is not None else three_block_split(n_layers)
    if len(split) != 3 or sum(split) != n_layers or min(split) < 0:
        raise ValueError("split must give three block sizes that add up to n_layers")
    scores = {}
    for delta in blockwise_delta_candidates(w):
        if delta not in scores:
            scores[delta] = float(task_acc_eval(blockwise_windows(w, (0, delta, w), split)))
    best = max(scores, key=lambda dl: (scores[dl], dl))
    return blockwise_windows(w, (0, best, w), split), best, scores
