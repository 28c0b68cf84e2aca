"""Shared helpers of the GPU parity tests: run the CUDA path and the CPU oracle on the same seeded inputs."""
from __future__ import annotations

import math
from typing import Optional, Sequence

import numpy as np
import torch

from oracle import glide_oracle as orc
from paper_2607_24788_b200 import glide, synth

TOL = {torch.float32: dict(max_abs=1e-4, rel_l2=None), torch.bfloat16: dict(max_abs=2e-2, rel_l2=1e-2)}
STATE_REL_L2 = 1e-5
# bf16: the relative-L2 bound also holds for every output row on its own (the d values of one layer, sequence,
# token and head), so that an error confined to one head, one token or one layer with small outputs cannot hide
# behind the rest of the tensor.  Rows whose reference norm is below the floor are left to the max-abs bound: a
# row that small is dominated by the bf16 rounding of outputs near zero, not by the attention arithmetic.
ROW_NORM_FLOOR = 1e-6


def f32_scale(d: int) -> float:
    """1/sqrt(d) as the fp32 value both sides use."""
    return float(np.float32(1.0) / np.sqrt(np.float32(d)))


def to_np(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu", torch.float64).numpy()


def check_outputs(got: torch.Tensor, ref: np.ndarray, dtype: torch.dtype, what: str):
    g = to_np(got)
    assert g.shape == ref.shape, (what, g.shape, ref.shape)
    assert np.isfinite(g).all(), f"{what}: non-finite output"
    tol = TOL[dtype]
    err = np.abs(g - ref).max() if g.size else 0.0
    assert err <= tol["max_abs"], f"{what}: max-abs {err:.3e} > {tol['max_abs']}"
    if tol["rel_l2"] is not None and g.size:
        rel = np.linalg.norm(g - ref) / max(np.linalg.norm(ref), 1e-30)
        assert rel <= tol["rel_l2"], f"{what}: rel-L2 {rel:.3e} > {tol['rel_l2']}"
        row_ref = np.linalg.norm(ref, axis=-1)
        row_err = np.linalg.norm(g - ref, axis=-1)
        live = row_ref >= ROW_NORM_FLOOR
        if live.any():
            row_rel = np.where(live, row_err / np.maximum(row_ref, ROW_NORM_FLOOR), 0.0)
            worst = np.unravel_index(np.argmax(row_rel), row_rel.shape)
            assert row_rel[worst] <= tol["rel_l2"], (f"{what}: row {tuple(int(i) for i in worst)} rel-L2 "
                                                     f"{row_rel[worst]:.3e} > {tol['rel_l2']} (row norm {row_ref[worst]:.3e})")
    return err


def check_state(g: "glide.Glide", stack: orc.Stack, what: str = ""):
    """Bookkeeping bit-exact; ring rows verbatim; S,z within rel-L2 1e-5."""
    for l in range(g.L):
        info = g.glide_layer_info(l)
        for b in range(g.B):
            oi = stack.cells[l][b].info()
            assert (info["n"], info["count"], info["n_evicted"]) == (oi["n"], oi["count"], oi["n_evicted"]), (what, l, info, oi)
            cap = info["capacity"]
            assert cap == min(g.windows[l], g.max_tokens)
            if cap:
                assert info["head_slot"] == oi["n"] % cap
        rk, rv, S, z = g.glide_export_state(l)
        for b in range(g.B):
            cell = stack.cells[l][b]
            ork, orv, oS, oz = cell.export()
            tok = cell.slot_tokens()
            cap = info["capacity"]
            valid = np.nonzero(tok[:cap] >= 0)[0] if cap else np.array([], dtype=np.int64)
            if len(valid):
                np.testing.assert_array_equal(to_np(rk[b])[:, valid], ork[:, valid], err_msg=f"{what} ringK l{l} b{b}")
                np.testing.assert_array_equal(to_np(rv[b])[:, valid], orv[:, valid], err_msg=f"{what} ringV l{l} b{b}")
            for name, a, r in (("S", to_np(S[b]), oS), ("z", to_np(z[b]), oz)):
                assert a.shape == r.shape, (what, name, a.shape, r.shape)
                nr = np.linalg.norm(r)
                if nr == 0:
                    assert np.abs(a).max() == 0, f"{what} {name} l{l} b{b} should be zero"
                else:
                    rel = np.linalg.norm(a - r) / nr
                    assert rel <= STATE_REL_L2, f"{what} {name} l{l} b{b}: rel-L2 {rel:.3e}"
            if getattr(g, "gated", False) and len(valid):   # the ring's gates are copies of the callers' fp32 values
                gr = to_np(g.glide_export_gates(l)[b])
                np.testing.assert_array_equal(gr[:, valid], cell.export_gates()[:, valid], err_msg=f"{what} gates l{l} b{b}")


def learned_phi_weights(L: int, H: int, Hkv: int, d: int, dtype: torch.dtype, seed: int, device="cuda"):
    """The projections of the learned feature map, entries N(0, 1/d) rounded to the I/O dtype: (wq [L][H][d][d],
    wk [L][Hkv][d][d]) on the device; both sides use these rounded values."""
    gen = torch.Generator().manual_seed(1000 + seed)
    wq = (torch.randn((L, H, d, d), generator=gen) / math.sqrt(d)).to(dtype)
    wk = (torch.randn((L, Hkv, d, d), generator=gen) / math.sqrt(d)).to(dtype)
    return wq.to(device), wk.to(device)


def gates_for(shape, seed: int, lo: float = 0.6, device="cuda") -> torch.Tensor:
    """fp32 gates in (lo, 1) of the given shape, seeded."""
    gen = torch.Generator().manual_seed(2000 + seed)
    return (lo + (1.0 - lo) * torch.rand(shape, generator=gen)).to(torch.float32).to(device)


def run_case(windows: Sequence[int], B: int, H: int, Hkv: int, d: int, dtype: torch.dtype, prompt_calls: Sequence[int],
             n_decode: int, amp: float = 1.0, seed: int = 0, q_to_kv: Optional[Sequence[int]] = None,
             max_tokens: Optional[int] = None, check_prefill_outputs: bool = True, state_checks: bool = True,
             phi: int = 0, gated: bool = False, **cfg_kw):
    """prefill (one call per entry of prompt_calls) then n_decode steps on both sides; asserts parity.
    phi = 1: the learned feature map with seeded projections; gated: seeded gates with every call."""
    dev = "cuda"
    L = len(windows)
    total = sum(prompt_calls) + n_decode
    max_tokens = max_tokens or max(total, 1)
    scale = f32_scale(d)
    wl = synth.Workload(seed, L, B, H, Hkv, d, dtype, amp)
    wq = wk = None
    if phi:
        wq, wk = learned_phi_weights(L, H, Hkv, d, dtype, seed)
        cfg_kw = dict(cfg_kw, phi=phi, phi_wq=wq, phi_wk=wk)
    if gated:
        cfg_kw = dict(cfg_kw, gated=True)
    g = glide.Glide(windows, B, H, Hkv, d, max_tokens, dtype=dtype, device=dev, q_to_kv=q_to_kv, softmax_scale=scale,
                    **cfg_kw)
    stack = orc.Stack(windows, B, H, Hkv, d, scale, q_to_kv=None if q_to_kv is None else np.asarray(q_to_kv, np.int32),
                      merge=cfg_kw.get("merge", 0), phi=phi, wq=None if wq is None else to_np(wq),
                      wk=None if wk is None else to_np(wk))
    pos = 0
    worst = 0.0
    for T in prompt_calls:
        q, k, v = wl.qkv(range(L), range(B), range(pos, pos + T), device=dev)
        out = torch.full_like(q, float("nan")) if check_prefill_outputs else None
        gate = gates_for((L, B, T, Hkv), seed * 131 + pos) if gated else None
        if gated:
            g.glide_prefill_gated(q if check_prefill_outputs else None, k, v, gate, out)
        else:
            g.glide_prefill(q if check_prefill_outputs else None, k, v, out)
        ref = stack.prefill(to_np(q), to_np(k), to_np(v), outputs=check_prefill_outputs,
                            gate=None if gate is None else to_np(gate))
        if check_prefill_outputs:
            worst = max(worst, check_outputs(out, ref, dtype, f"prefill@{pos}+{T}"))
        pos += T
        if state_checks:
            check_state(g, stack, f"after prefill to {pos}")
    for s in range(n_decode):
        q, k, v = wl.decode_qkv(pos, device=dev)
        out = torch.full_like(q, float("nan"))
        gate = gates_for((L, B, Hkv), seed * 131 + pos) if gated else None
        if gated:
            g.glide_decode_step_gated(q, k, v, gate, out)
        else:
            g.glide_decode_step(q, k, v, out)
        ref = stack.decode(to_np(q), to_np(k), to_np(v), gate=None if gate is None else to_np(gate))
        worst = max(worst, check_outputs(out, ref, dtype, f"decode step {s} (t={pos})"))
        pos += 1
    if state_checks:
        check_state(g, stack, f"after decode to {pos}")
    assert g.glide_device_status() == 0
    g.glide_destroy()
    return worst
