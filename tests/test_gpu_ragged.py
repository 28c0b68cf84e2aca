"""Sequences of different lengths in one context (continuous batching) against the CPU oracle.

Every slot of the batch holds its own sequence: slots are prefilled one by one with prompts of different lengths,
decoded together, reset and refilled while the others keep going.  The oracle side is one independent cell per
(layer, live sequence), so nothing but the per-sequence definition of the method enters the expected values.
"""
import numpy as np
import pytest
import torch

from oracle import glide_oracle as orc
from paper_2607_24788_b200 import glide, synth
from tests.parity_util import STATE_REL_L2, check_outputs, f32_scale, to_np

pytestmark = pytest.mark.gpu

N_IDS = 64   # logical sequences of the synthetic workload (slots draw fresh ids from it)


class Ragged:
    """The CUDA context and, per slot, the oracle cells of the sequence that lives there."""

    def __init__(self, windows, B, H, Hkv, d, dtype, max_tokens, seed=0, amp=1.0, **cfg_kw):
        self.L, self.B, self.H, self.Hkv, self.d, self.dtype = len(windows), B, H, Hkv, d, dtype
        self.windows, self.merge = list(windows), cfg_kw.get("merge", 0)
        self.scale = f32_scale(d)
        self.wl = synth.Workload(seed, self.L, N_IDS, H, Hkv, d, dtype, amp)
        self.g = glide.Glide(windows, B, H, Hkv, d, max_tokens, dtype=dtype, device="cuda", softmax_scale=self.scale,
                             **cfg_kw)
        self.next_id = 0
        self.ids, self.pos, self.cells = [0] * B, [0] * B, [None] * B
        self.parked = set()
        for b in range(B):
            self.new_sequence(b, reset=False)
        self.worst = 0.0

    def new_sequence(self, b, reset=True):
        self.ids[b], self.pos[b] = self.next_id, 0
        self.next_id += 1
        self.cells[b] = [orc.Cell(self.H, self.Hkv, self.d, w, self.scale, merge=self.merge) for w in self.windows]
        self.parked.discard(b)
        if reset:
            self.g.glide_reset_seq(b)

    def park(self, b):
        self.parked.add(b)
        self.g.glide_park_seq(b)

    def prefill_seq(self, b, T, outputs=True):
        q, k, v = self.wl.qkv(range(self.L), [self.ids[b]], range(self.pos[b], self.pos[b] + T), device="cuda")
        q, k, v = q[:, 0].contiguous(), k[:, 0].contiguous(), v[:, 0].contiguous()
        out = torch.full_like(q, float("nan")) if outputs else None
        self.g.glide_prefill_seq(b, q if outputs else None, k, v, out)
        for l in range(self.L):
            ref = self.cells[b][l].prefill(to_np(q[l]), to_np(k[l]), to_np(v[l]), outputs=outputs)
            if outputs:
                self.worst = max(self.worst, check_outputs(out[l], ref, self.dtype, f"prefill slot {b} layer {l} @{self.pos[b]}+{T}"))
        self.pos[b] += T
        assert self.g.glide_seq_tokens(b) == self.pos[b]

    def _step_inputs(self):
        parts = [self.wl.qkv(range(self.L), [self.ids[b]], [self.pos[b]], device="cuda") for b in range(self.B)]
        return [torch.cat([p[i][:, :, 0] for p in parts], dim=1).contiguous() for i in range(3)]

    def decode(self, steps=1, by_layer=False):
        for _ in range(steps):
            q, k, v = self._step_inputs()
            out = torch.full_like(q, float("nan"))
            if by_layer:
                for l in range(self.L):
                    self.g.glide_decode_step_layers(q[l:l + 1], k[l:l + 1], v[l:l + 1], out[l:l + 1], l, 1)
            else:
                self.g.glide_decode_step(q, k, v, out)
            for b in range(self.B):
                if b in self.parked:
                    assert torch.isnan(out[:, b].float()).all(), "a parked slot's output rows were written"
                    continue
                ref = np.stack([self.cells[b][l].decode(to_np(q[l, b]), to_np(k[l, b]), to_np(v[l, b])) for l in range(self.L)])
                self.worst = max(self.worst, check_outputs(out[:, b], ref, self.dtype, f"decode slot {b} t={self.pos[b]}"))
                self.pos[b] += 1

    def check_state(self, what=""):
        g = self.g
        for l in range(self.L):
            rk, rv, S, z = g.glide_export_state(l)
            for b in range(self.B):
                if b in self.parked:
                    continue
                cell = self.cells[b][l]
                info, oi = g.glide_seq_layer_info(l, b), cell.info()
                assert (info["n"], info["count"], info["n_evicted"]) == (oi["n"], oi["count"], oi["n_evicted"]), (what, l, b, info, oi)
                cap = info["capacity"]
                if cap:
                    assert info["head_slot"] == oi["n"] % cap
                ork, orv, oS, oz = cell.export()
                tok = cell.slot_tokens()
                valid = np.nonzero(tok[:cap] >= 0)[0] if cap else np.array([], dtype=np.int64)
                if len(valid):
                    np.testing.assert_array_equal(to_np(rk[b])[:, valid], ork[:, valid], err_msg=f"{what} ringK l{l} b{b}")
                    np.testing.assert_array_equal(to_np(rv[b])[:, valid], orv[:, valid], err_msg=f"{what} ringV l{l} b{b}")
                for name, a, r in (("S", to_np(S[b]), oS), ("z", to_np(z[b]), oz)):
                    nr = np.linalg.norm(r)
                    if nr == 0:
                        assert np.abs(a).max() == 0, f"{what} {name} l{l} b{b} should be zero"
                    else:
                        assert np.linalg.norm(a - r) / nr <= STATE_REL_L2, f"{what} {name} l{l} b{b}"
        assert g.glide_device_status() == 0


def scenario(r: Ragged, prompts, by_layer=False):
    """prompts of different lengths, joint decode, one slot reset and refilled in two calls, joint decode again"""
    for b, T in enumerate(prompts):
        if T:
            r.prefill_seq(b, T)
    r.check_state("after the prompts")
    r.decode(5, by_layer=by_layer)
    r.check_state("after the first decode steps")
    victim = 1 % r.B
    r.new_sequence(victim)
    r.check_state("after resetting a slot")
    r.prefill_seq(victim, 40)
    r.prefill_seq(victim, 27, outputs=False)
    r.decode(6, by_layer=by_layer)
    # a slot that was never prefilled decodes from position 0 on; another reset right before a step
    r.new_sequence(0)
    r.decode(3, by_layer=by_layer)
    r.check_state("at the end")
    r.g.glide_destroy()
    return r.worst


@pytest.mark.parametrize("merge", [0, 1, 2])
def test_ragged_fp32_cuda_cores(merge):
    r = Ragged([48, 16, 0, 200], 3, 4, 2, 64, torch.float32, 400, seed=3, amp=1.5, merge=merge, prefill_chunk=32)
    scenario(r, [37, 5, 150])


@pytest.mark.parametrize("merge", [0, 1, 2])
def test_ragged_bf16_streaming_and_tcgen05(merge):
    # (the sum of two normalised terms is up to twice as large as one: smaller values keep bf16 output rounding
    # inside the absolute tolerance)
    r = Ragged([64, 16, 0, 300, 128], 4, 8, 2, 128, torch.bfloat16, 600, seed=4, amp=1.0 if merge == 0 else 0.5,
               merge=merge, prefill_chunk=64)
    scenario(r, [130, 0, 333, 17])


def test_ragged_bf16_layer_by_layer():
    r = Ragged([64, 0, 160], 3, 8, 2, 128, torch.bfloat16, 500, seed=5, prefill_chunk=64)
    scenario(r, [100, 7, 261], by_layer=True)


def test_ragged_bf16_per_item_mma_and_mma_sync_prefill():
    r = Ragged([64, 16, 0, 300], 3, 8, 2, 128, torch.bfloat16, 600, seed=6, prefill_chunk=64,
               decode_impl=glide.GLIDE_DECODE_MMA, prefill_impl=glide.GLIDE_PREFILL_MMA_SYNC)
    scenario(r, [130, 2, 333])


def test_ragged_noalloc_step():
    r = Ragged([32, 0, 100], 2, 4, 2, 64, torch.float32, 300, seed=7)
    r.prefill_seq(0, 120)
    r.prefill_seq(1, 9)
    for _ in range(4):
        q, k, v = r._step_inputs()
        out = torch.full_like(q, float("nan"))
        r.g.glide_decode_step_noalloc(q, k, v, out)
        for b in range(r.B):
            ref = np.stack([r.cells[b][l].decode(to_np(q[l, b]), to_np(k[l, b]), to_np(v[l, b])) for l in range(r.L)])
            check_outputs(out[:, b], ref, r.dtype, f"noalloc slot {b}")
            r.pos[b] += 1
    r.check_state("noalloc")
    r.g.glide_destroy()


def test_joint_prefill_needs_level_slots_and_capacity_follows_the_longest_slot():
    L, B, H, Hkv, d = 2, 2, 4, 2, 64
    r = Ragged([16, 0], B, H, Hkv, d, torch.float32, 64, seed=8)
    r.prefill_seq(0, 50)
    q, k, v = r.wl.qkv(range(L), [0, 1], range(0, 4), device="cuda")
    with pytest.raises(glide.GlideError) as e:
        r.g.glide_prefill(q, k, v, torch.empty_like(q))
    assert e.value.code == glide.GLIDE_ERR_STATE
    with pytest.raises(glide.GlideError) as e:
        r.prefill_seq(0, 15)                      # 50 + 15 > 64
    assert e.value.code == glide.GLIDE_ERR_CAPACITY
    r.decode(14)                                   # slot 0 reaches 64 tokens
    q, k, v = r._step_inputs()
    with pytest.raises(glide.GlideError) as e:
        r.g.glide_decode_step(q, k, v, torch.empty_like(q))
    assert e.value.code == glide.GLIDE_ERR_CAPACITY
    # every slot reset: level again (all offsets equal), a joint prefill works and matches fresh sequences
    for b in range(B):
        r.new_sequence(b)
    q, k, v = r.wl.qkv(range(L), r.ids, range(0, 20), device="cuda")
    out = torch.full_like(q, float("nan"))
    r.g.glide_prefill(q, k, v, out)
    for b in range(B):
        for l in range(L):
            ref = r.cells[b][l].prefill(to_np(q[l, b]), to_np(k[l, b]), to_np(v[l, b]))
            check_outputs(out[l, b], ref, r.dtype, "joint prefill after resets")
        r.pos[b] += 20
    r.decode(3)
    r.check_state("after joint prefill")
    r.g.glide_reset()
    assert [r.g.glide_seq_tokens(b) for b in range(B)] == [0, 0]
    r.g.glide_destroy()


@pytest.mark.parametrize("seed", range(8))
def test_ragged_random_schedules(seed):
    """Seeded random configurations and random sequences of per-slot prefills, joint decode steps, resets and
    parked slots."""
    rng = np.random.default_rng(1000 + seed)
    bf16 = bool(rng.integers(0, 2))
    dtype, d = (torch.bfloat16, 128) if bf16 else (torch.float32, int(rng.choice([64, 128])))
    Hkv = int(rng.choice([1, 2, 4]))
    H = Hkv * int(rng.choice([1, 2, 4]))
    B = int(rng.integers(1, 6))
    L = int(rng.integers(1, 5))
    windows = [int(rng.choice([0, 1, 7, 16, 33, 64, 150, 400])) for _ in range(L)]
    merge = int(rng.integers(0, 3))
    kw = dict(merge=merge, prefill_chunk=int(rng.choice([16, 64, 256])))
    if bf16 and rng.integers(0, 3) == 0:
        kw.update(decode_impl=glide.GLIDE_DECODE_FMA, prefill_impl=glide.GLIDE_PREFILL_FMA)
    max_tokens = 700
    r = Ragged(windows, B, H, Hkv, d, dtype, max_tokens, seed=seed, amp=0.5 if merge else 1.0, **kw)
    for _ in range(int(rng.integers(6, 12))):
        op = int(rng.integers(0, 5))
        b = int(rng.integers(0, B))
        if op == 4:
            r.park(b)
        elif op == 0:
            if b in r.parked:
                r.new_sequence(b)
            T = int(rng.choice([1, 3, 17, 64, 130, 260]))
            if r.pos[b] + T <= max_tokens - 40:
                r.prefill_seq(b, T, outputs=bool(rng.integers(0, 4)))
        elif op == 1:
            r.new_sequence(b)
        else:
            r.decode(int(rng.integers(1, 4)), by_layer=bool(rng.integers(0, 4) == 0))
    r.decode(2)
    r.check_state(f"seed {seed}")
    r.g.glide_destroy()


def test_ragged_llama_shape_long_sequences_sampled_layers():
    """Config-1 shapes (32 layers, H = 32, H_kv = 8, d = 128) with four sequences of very different lengths: heavy
    units are cut across CTAs and merged through global records while every sequence sits at its own position.  The oracle
    follows one layer of every window size."""
    from paper_2607_24788_b200 import configs as C
    windows = list(C.C1.windows)
    L, B, H, Hkv, d = len(windows), 4, 32, 8, 128
    lengths = [9000, 4100, 17, 6500]
    layers = [0, 5, 13, 31]                       # windows 4096, 1024, 256, 64
    scale = f32_scale(d)
    wl = synth.Workload(21, L, N_IDS, H, Hkv, d, torch.bfloat16, d ** -0.5 * 4)
    g = glide.Glide(windows, B, H, Hkv, d, 10000, dtype=torch.bfloat16, device="cuda", softmax_scale=scale)
    cells = {(l, b): orc.Cell(H, Hkv, d, windows[l], scale) for l in layers for b in range(B)}
    for b, T in enumerate(lengths):
        pos = 0
        while pos < T:
            n = min(4096, T - pos)
            k, v = wl.kv(range(L), [b], range(pos, pos + n), device="cuda")
            g.glide_prefill_seq(b, None, k[:, 0].contiguous(), v[:, 0].contiguous(), None)
            for l in layers:
                cells[(l, b)].prefill(None, to_np(k[l, 0]), to_np(v[l, 0]), outputs=False)
            pos += n
        assert g.glide_seq_tokens(b) == T
    pos = list(lengths)
    for step in range(3):
        parts = [wl.qkv(range(L), [b], [pos[b]], device="cuda") for b in range(B)]
        q, k, v = [torch.cat([p[i][:, :, 0] for p in parts], dim=1).contiguous() for i in range(3)]
        out = torch.full_like(q, float("nan"))
        g.glide_decode_step(q, k, v, out)
        assert torch.isfinite(out.float()).all()
        for l in layers:
            for b in range(B):
                ref = cells[(l, b)].decode(to_np(q[l, b]), to_np(k[l, b]), to_np(v[l, b]))
                check_outputs(out[l, b], ref, torch.bfloat16, f"step {step} layer {l} slot {b} t={pos[b]}")
        pos = [x + 1 for x in pos]
    for l in layers:
        for b in range(B):
            info, oi = g.glide_seq_layer_info(l, b), cells[(l, b)].info()
            assert (info["n"], info["count"], info["n_evicted"]) == (oi["n"], oi["count"], oi["n_evicted"])
    assert g.glide_device_status() == 0
    g.glide_destroy()


def _snapshot(g, b):
    """ring, S, z of slot b for every layer (device copies)"""
    snap = []
    for l in range(g.L):
        rk, rv, S, z = g.glide_export_state(l)
        snap.append(tuple(x[b].clone() for x in (rk, rv, S, z)))
    return snap


@pytest.mark.parametrize("kind", ["f32", "bf16_stream", "bf16_stream_by_layer", "bf16_mma", "bf16_sum"])
def test_parked_slot_is_skipped(kind):
    """A parked slot is not stepped: its outputs stay as the caller left them, its ring, S, z do not change (bit for
    bit), whatever its input rows hold (NaN here); the other slots are unaffected; a reset starts a new sequence."""
    kw, by_layer = {}, False
    if kind == "f32":
        dtype, d, H, Hkv = torch.float32, 64, 4, 2
    else:
        dtype, d, H, Hkv = torch.bfloat16, 128, 8, 2
        if kind == "bf16_mma":
            kw = dict(decode_impl=glide.GLIDE_DECODE_MMA)
        if kind == "bf16_sum":
            kw = dict(merge=1)
        by_layer = kind == "bf16_stream_by_layer"
    r = Ragged([48, 0, 300, 16], 3, H, Hkv, d, dtype, 600, seed=12, amp=0.5 if kw.get("merge") else 1.0, **kw)
    for b, T in enumerate([200, 350, 31]):
        r.prefill_seq(b, T)
    r.decode(2, by_layer=by_layer)
    victim = 1
    r.g.glide_park_seq(victim)
    assert r.g.glide_seq_tokens(victim) == -1
    before = _snapshot(r.g, victim)
    live = [b for b in range(r.B) if b != victim]
    for _ in range(4):
        q, k, v = r._step_inputs()
        q[:, victim], k[:, victim], v[:, victim] = float("nan"), float("nan"), float("nan")
        out = torch.full_like(q, 7.0)
        if by_layer:
            for l in range(r.L):
                r.g.glide_decode_step_layers(q[l:l + 1], k[l:l + 1], v[l:l + 1], out[l:l + 1], l, 1)
        else:
            r.g.glide_decode_step(q, k, v, out)
        assert (out[:, victim] == 7.0).all()
        for b in live:
            ref = np.stack([r.cells[b][l].decode(to_np(q[l, b]), to_np(k[l, b]), to_np(v[l, b])) for l in range(r.L)])
            check_outputs(out[:, b], ref, r.dtype, f"slot {b} beside a parked slot")
            r.pos[b] += 1
    after = _snapshot(r.g, victim)
    for l in range(r.L):
        for x, y in zip(before[l], after[l]):
            assert torch.equal(x, y)
    with pytest.raises(glide.GlideError) as e:
        r.prefill_seq(victim, 4)
    assert e.value.code == glide.GLIDE_ERR_STATE
    r.new_sequence(victim)          # glide_reset_seq: the slot is live again, at position 0
    r.prefill_seq(victim, 70)
    r.decode(3, by_layer=by_layer)
    r.check_state("after the parked slot was reused")
    r.g.glide_destroy()


def test_parked_slots_do_not_count_for_capacity_and_all_parked_is_a_no_op():
    r = Ragged([16, 0], 2, 4, 2, 64, torch.float32, 40, seed=13)
    r.prefill_seq(0, 39)
    r.g.glide_park_seq(0)
    for _ in range(5):             # slot 0 would be past max_tokens by now
        q, k, v = r._step_inputs()
        out = torch.full_like(q, 3.0)
        r.g.glide_decode_step(q, k, v, out)
        ref = np.stack([r.cells[1][l].decode(to_np(q[l, 1]), to_np(k[l, 1]), to_np(v[l, 1])) for l in range(r.L)])
        check_outputs(out[:, 1], ref, r.dtype, "live slot")
        r.pos[1] += 1
    r.g.glide_park_seq(1)
    q, k, v = r._step_inputs()
    out = torch.full_like(q, 3.0)
    r.g.glide_decode_step_noalloc(q, k, v, out)
    assert (out == 3.0).all() and r.g.glide_device_status() == 0
    r.g.glide_destroy()
