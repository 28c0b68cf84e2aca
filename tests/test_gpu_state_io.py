"""State export / import and run-to-run determinism of the CUDA path, through the C ABI.

glide_import_state is what the benchmark uses to clone the post-prefill state into its rotating copies, so the
steps it times run on imported states: they are checked here against the oracle.  The determinism tests run the
same step sequence on two contexts and compare every output and the whole exported state bit for bit; the
lock-free "last arrival merges" reductions of the decode kernels would show a race as a difference."""
import numpy as np
import pytest
import torch

from oracle import glide_oracle as orc
from paper_2607_24788_b200 import glide, synth
from tests.parity_util import check_outputs, check_state, f32_scale, to_np

pytestmark = pytest.mark.gpu
BF16, F32 = torch.bfloat16, torch.float32


def _decode_against_oracle(g, stack, wl, pos, steps, dtype, what):
    for s in range(steps):
        q, k, v = wl.decode_qkv(pos, device="cuda")
        out = torch.full_like(q, float("nan"))
        g.glide_decode_step(q, k, v, out)
        ref = stack.decode(to_np(q), to_np(k), to_np(v))
        check_outputs(out, ref, dtype, f"{what}: decode step {s} (t={pos})")
        pos += 1
    check_state(g, stack, f"{what}: after decode to {pos}")
    return pos


@pytest.mark.parametrize("dtype,d,windows,kw", [
    (BF16, 128, [96, 16, 0, 4000, 33], {}),                      # streaming kernel; never-evicting and linear-only layers
    (BF16, 64, [40, 7], {}),                                     # per-item tensor-core kernel
    (F32, 64, [64, 5], {}),                                      # CUDA-core kernel
    (BF16, 128, [48, 20], dict(merge=glide.GLIDE_MERGE_SUM_ALL)),
])
def test_import_state_round_trip(dtype, d, windows, kw):
    """export -> import into a fresh context -> decode steps against the oracle (which never saw an export)."""
    B, H, Hkv, T, steps = 2, 8, 2, 150, 6
    L = len(windows)
    scale = f32_scale(d)
    wl = synth.Workload(23, L, B, H, Hkv, d, dtype, 4 * d ** -0.5)
    a = glide.Glide(windows, B, H, Hkv, d, T + steps, dtype=dtype, softmax_scale=scale, **kw)
    stack = orc.Stack(windows, B, H, Hkv, d, scale, merge=kw.get("merge", 0))
    q, k, v = wl.qkv(range(L), range(B), range(T), device="cuda")
    a.glide_prefill(None, k, v, None)
    stack.prefill(None, to_np(k), to_np(v), outputs=False)
    b = glide.Glide(windows, B, H, Hkv, d, T + steps, dtype=dtype, softmax_scale=scale, **kw)
    for l in range(L):
        rk, rv, S, z = a.glide_export_state(l)
        cap = a.capacity(l)
        b.glide_import_state(l, T, rk if cap else None, rv if cap else None, S, z)
        assert b.glide_layer_info(l) == a.glide_layer_info(l)
    check_state(b, stack, "imported copy")
    _decode_against_oracle(b, stack, wl, T, steps, dtype, "imported copy")
    assert b.glide_device_status() == 0


def test_import_of_the_closed_form_state():
    """The state after a prompt written out from its definition (ring = the newest w tokens at slot position mod w,
    S = sum over the older tokens of phi(k) v^T, z = sum of phi(k)), imported without any prefill on the GPU."""
    dtype, d, B, H, Hkv, T, steps = BF16, 128, 2, 8, 2, 200, 5
    windows = [64, 0, 24]
    L = len(windows)
    scale = f32_scale(d)
    wl = synth.Workload(29, L, B, H, Hkv, d, dtype, 4 * d ** -0.5)
    q, k, v = wl.qkv(range(L), range(B), range(T))
    kd, vd = k.double().numpy(), v.double().numpy()          # [L][B][T][Hkv][d]
    g = glide.Glide(windows, B, H, Hkv, d, T + steps, dtype=dtype, softmax_scale=scale)
    stack = orc.Stack(windows, B, H, Hkv, d, scale)
    stack.prefill(None, kd, vd, outputs=False)                # the oracle's own route to the same state
    for l, w in enumerate(windows):
        e = np.exp(kd[l] - kd[l].max(axis=-1, keepdims=True))
        phi = e / e.sum(axis=-1, keepdims=True)               # softmax over the d features
        old = max(0, T - w)                                   # tokens [0, old) have left the window
        S = np.einsum("bthr,bthc->bhrc", phi[:, :old], vd[l][:, :old])
        z = phi[:, :old].sum(axis=1)
        cap = min(w, T + steps)
        rk = torch.zeros((B, Hkv, cap, d), dtype=dtype)
        rv = torch.zeros_like(rk)
        for t in range(old, T):
            rk[:, :, t % w] = k[l][:, t]
            rv[:, :, t % w] = v[l][:, t]
        g.glide_import_state(l, T, rk.cuda() if cap else None, rv.cuda() if cap else None,
                             torch.from_numpy(S).float().cuda().contiguous(), torch.from_numpy(z).float().cuda().contiguous())
    torch.cuda.synchronize()
    check_state(g, stack, "closed-form import")
    _decode_against_oracle(g, stack, wl, T, steps, dtype, "closed-form import")


def _run_sequence(windows, B, H, Hkv, d, dtype, prompt, steps, seed, **kw):
    """prefill with outputs, then decode steps; returns every output and the final exported state."""
    L = len(windows)
    wl = synth.Workload(seed, L, B, H, Hkv, d, dtype, 4 * d ** -0.5)
    g = glide.Glide(windows, B, H, Hkv, d, prompt + steps, dtype=dtype, softmax_scale=f32_scale(d), **kw)
    got = []
    q, k, v = wl.qkv(range(L), range(B), range(prompt), device="cuda")
    out = torch.empty_like(q)
    g.glide_prefill(q, k, v, out)
    got.append(out)
    for s in range(steps):
        q, k, v = wl.decode_qkv(prompt + s, device="cuda")
        out = torch.empty_like(q)
        g.glide_decode_step(q, k, v, out)
        got.append(out)
    for l in range(L):
        got.extend(g.glide_export_state(l))
    torch.cuda.synchronize()
    assert g.glide_device_status() == 0
    return got


@pytest.mark.parametrize("kw", [
    dict(),                                                   # streaming kernel, tcgen05 prefill
    dict(decode_impl=glide.GLIDE_DECODE_MMA, prefill_impl=glide.GLIDE_PREFILL_MMA_SYNC),   # per-item kernel, mma.sync prefill
    dict(decode_impl=glide.GLIDE_DECODE_FMA, prefill_impl=glide.GLIDE_PREFILL_FMA),        # CUDA-core kernels
    dict(merge=glide.GLIDE_MERGE_SUM_EVICTED),
])
def test_same_steps_on_two_contexts_give_the_same_bits(kw):
    """Config 1's window schedule at batch 1 (units heavier than a CTA's share, cut across CTAs and merged from
    their global records; units shared by the warps of a CTA; units inside one warp) with a prompt that fills the windows."""
    windows = [4096] * 2 + [1024] * 3 + [256] * 5 + [64] * 4
    args = (windows, 1, 32, 8, 128, BF16, 4200, 6, 31)
    a = _run_sequence(*args, **kw)
    b = _run_sequence(*args, **kw)
    assert len(a) == len(b)
    for i, (x, y) in enumerate(zip(a, b)):
        assert torch.equal(x.view(torch.uint8), y.view(torch.uint8)), f"tensor {i} differs between two runs"


def test_same_steps_twice_fp32_and_batched():
    a = _run_sequence([64, 200, 0], 4, 8, 4, 64, F32, 300, 5, 37)
    b = _run_sequence([64, 200, 0], 4, 8, 4, 64, F32, 300, 5, 37)
    for i, (x, y) in enumerate(zip(a, b)):
        assert torch.equal(x.view(torch.uint8), y.view(torch.uint8)), f"tensor {i} differs between two runs"


def test_two_contexts_stepping_on_two_streams_at_once():
    """Two contexts of config 1's window schedule decode on two streams with nothing ordering one stream against the
    other, so launches of the streaming kernel may share the SMs.  Each context must produce the bits it produces
    alone, and no bounded wait may have run out (a merge must never wait for a CTA that is not running)."""
    windows = [4096] * 2 + [1024] * 3 + [256] * 5 + [64] * 4
    B, H, Hkv, d, prompt, steps = 1, 32, 8, 128, 4200, 40
    L = len(windows)

    def build(seed):
        wl = synth.Workload(seed, L, B, H, Hkv, d, BF16, 4 * d ** -0.5)
        g = glide.Glide(windows, B, H, Hkv, d, prompt + steps, dtype=BF16, softmax_scale=f32_scale(d))
        _, k, v = wl.qkv(range(L), range(B), range(prompt), device="cuda")
        g.glide_prefill(None, k, v, None)
        inputs = [wl.decode_qkv(prompt + s, device="cuda") for s in range(steps)]
        return g, inputs

    def run(pairs, streams):
        outs = [[torch.empty_like(inp[0][0]) for _ in range(steps)] for _, inp in pairs]
        torch.cuda.synchronize()
        for s in range(steps):
            for i, (g, inp) in enumerate(pairs):
                q, k, v = inp[s]
                g.glide_decode_step(q, k, v, outs[i][s], stream=streams[i])
        torch.cuda.synchronize()
        for g, _ in pairs:
            assert g.glide_device_status() == 0
        return outs

    one = torch.cuda.current_stream()
    alone = run([build(51), build(52)], [one, one])
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    together = run([build(51), build(52)], [s1, s2])
    for a, b in zip(alone, together):
        for x, y in zip(a, b):
            assert torch.equal(x.view(torch.uint8), y.view(torch.uint8))
