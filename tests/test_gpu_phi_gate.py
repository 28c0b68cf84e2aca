"""GPU parity of the learned feature map (phi = GLIDE_PHI_PROJ_SOFTMAX2, feature dimension 2d) and of the gated
recurrence against the CPU oracle, through the C ABI: prefill calls with outputs (several, unaligned), decode steps,
exported S [2d][d] / z [2d], ring rows, gates and counters."""
import pytest
import torch

from paper_2607_24788_b200 import glide
from tests.parity_util import run_case

pytestmark = pytest.mark.gpu
BF16, F32 = torch.bfloat16, torch.float32


def test_config0_tiny_fp32_with_the_learned_map():
    """Config 0 (1 layer, 4 = 4 heads, d = 64, w = 64, 512-token prompt, 16 decode steps, N(0,1) inputs) with the
    d x d projection of N(0, 1/d) weights and 2d features."""
    run_case([64], 1, 4, 4, 64, F32, [512], 16, amp=1.0, phi=1)


@pytest.mark.parametrize("dtype,d,G", [(F32, 64, 1), (F32, 128, 2), (BF16, 64, 4), (BF16, 128, 4), (BF16, 128, 8)])
def test_learned_map_prefill_then_decode(dtype, d, G):
    Hkv = 2
    amp = 1.0 if dtype == F32 else 4 * d ** -0.5
    run_case([24, 0, 100, 5], 2, Hkv * G, Hkv, d, dtype, [37, 1, 50], 6, amp=amp, seed=3 + G, phi=1,
             prefill_chunk=32, max_tokens=100)


@pytest.mark.parametrize("merge", [glide.GLIDE_MERGE_SUM_EVICTED, glide.GLIDE_MERGE_SUM_ALL])
def test_learned_map_with_the_sum_of_terms_merges(merge):
    run_case([16, 0, 40], 2, 8, 2, 128, BF16, [45, 20], 5, amp=4 * 128 ** -0.5, seed=5, phi=1, merge=merge)


def test_learned_map_forced_cuda_core_kernels_bf16():
    run_case([32, 8], 3, 8, 2, 128, BF16, [70], 5, amp=4 * 128 ** -0.5, seed=6, phi=1,
             decode_impl=glide.GLIDE_DECODE_FMA, prefill_impl=glide.GLIDE_PREFILL_FMA)


@pytest.mark.parametrize("dtype,d,phi", [(F32, 64, 0), (BF16, 128, 0), (F32, 64, 1), (BF16, 128, 1)])
def test_gated_recurrence_prefill_then_decode(dtype, d, phi):
    amp = 1.0 if dtype == F32 else 4 * d ** -0.5
    run_case([12, 0, 90, 3], 2, 8, 2, d, dtype, [29, 2, 40], 8, amp=amp, seed=7 + phi, phi=phi, gated=True,
             prefill_chunk=16, max_tokens=90)


def test_gated_context_without_gates_is_the_plain_method():
    """gamma = 1 everywhere: the calls without gates on a gated context, against the ungated oracle."""
    import numpy as np
    from oracle import glide_oracle as orc
    from paper_2607_24788_b200 import synth
    from tests.parity_util import check_outputs, check_state, f32_scale, to_np
    windows, B, H, Hkv, d, T = [10, 0], 2, 4, 2, 64, 33
    wl = synth.Workload(9, len(windows), B, H, Hkv, d, F32, 1.0)
    g = glide.Glide(windows, B, H, Hkv, d, T + 4, dtype=F32, softmax_scale=f32_scale(d), gated=True)
    stack = orc.Stack(windows, B, H, Hkv, d, f32_scale(d))
    q, k, v = wl.qkv(range(len(windows)), range(B), range(T), device="cuda")
    out = torch.empty_like(q)
    g.glide_prefill(q, k, v, out)
    check_outputs(out, stack.prefill(to_np(q), to_np(k), to_np(v)), F32, "prefill")
    for s in range(4):
        q, k, v = wl.decode_qkv(T + s, device="cuda")
        out = torch.empty_like(q)
        g.glide_decode_step(q, k, v, out)
        check_outputs(out, stack.decode(to_np(q), to_np(k), to_np(v)), F32, f"decode {s}")
    check_state(g, stack, "ungated calls on a gated context")


def test_feature_map_and_gate_argument_checks():
    d = 128
    wq = torch.zeros((1, 4, d, d), dtype=BF16, device="cuda")
    wk = torch.zeros((1, 2, d, d), dtype=BF16, device="cuda")
    for kw, code in ((dict(phi=1), glide.GLIDE_ERR_INVALID_ARG),                                  # no weights
                     (dict(phi=0, phi_wq=wq, phi_wk=wk), glide.GLIDE_ERR_INVALID_ARG),            # weights without the map
                     (dict(phi=1, phi_wq=wq, phi_wk=wk, decode_impl=glide.GLIDE_DECODE_MMA), glide.GLIDE_ERR_UNSUPPORTED),
                     (dict(phi=1, phi_wq=wq, phi_wk=wk, prefill_impl=glide.GLIDE_PREFILL_MMA_SYNC), glide.GLIDE_ERR_UNSUPPORTED),
                     (dict(phi=1, phi_wq=wq, phi_wk=wk, prefill_impl=glide.GLIDE_PREFILL_TCGEN05,
                           merge=glide.GLIDE_MERGE_SUM_EVICTED), glide.GLIDE_ERR_UNSUPPORTED),
                     (dict(gated=True, decode_impl=glide.GLIDE_DECODE_MMA), glide.GLIDE_ERR_UNSUPPORTED),
                     (dict(gated=True, prefill_impl=glide.GLIDE_PREFILL_TCGEN05), glide.GLIDE_ERR_UNSUPPORTED)):
        with pytest.raises(glide.GlideError) as e:
            glide.Glide([16], 1, 4, 2, d, 64, dtype=BF16, **kw)
        assert e.value.code == code, kw
    plain = glide.Glide([16], 1, 4, 2, d, 64, dtype=BF16)
    q = torch.zeros((1, 1, 4, d), dtype=BF16, device="cuda")
    k = torch.zeros((1, 1, 2, d), dtype=BF16, device="cuda")
    with pytest.raises(glide.GlideError) as e:   # gated call on a context without gates
        plain.glide_decode_step_gated(q, k, k, None, torch.empty_like(q))
    assert e.value.code == glide.GLIDE_ERR_INVALID_ARG


@pytest.mark.parametrize("merge,G", [(glide.GLIDE_MERGE_SUM_EVICTED, 4), (glide.GLIDE_MERGE_SUM_ALL, 4),
                                     (glide.GLIDE_MERGE_SUM_EVICTED, 8), (glide.GLIDE_MERGE_SUM_ALL, 1)])
def test_learned_map_with_sum_of_terms_merges_on_the_streaming_kernel(merge, G):
    """Both options at once on the streaming decode kernel (records twice as wide, 16 state tiles per unit), with
    units inside one warp, shared by the warps of a CTA and cut across CTAs."""
    Hkv = 2
    run_case([1500, 64, 0, 5000, 300], 1, Hkv * G, Hkv, 128, BF16, [1490, 7], 10, amp=4 * 128 ** -0.5, seed=31 + G,
             phi=1, merge=merge, check_prefill_outputs=False, decode_impl=glide.GLIDE_DECODE_STREAM)


@pytest.mark.parametrize("G,B", [(4, 1), (1, 3), (8, 2)])
def test_learned_map_on_the_streaming_kernel_units_cut_across_ctas(G, B):
    """Windows long enough for units to be cut across warps and CTAs (global records and their merges) with 16 state
    tiles per unit; layers without a ring and layers that never evict; decode steps that cross a ring wrap."""
    Hkv = 2
    run_case([1500, 64, 0, 5000, 300], B, Hkv * G, Hkv, 128, BF16, [1490, 7], 12, amp=4 * 128 ** -0.5, seed=11 + G,
             phi=1, check_prefill_outputs=False, decode_impl=glide.GLIDE_DECODE_STREAM)


@pytest.mark.parametrize("G,chunk,calls", [(4, 0, [144, 130, 61]), (1, 64, [144, 130, 61]), (2, 128, [144, 130, 61]),
                                           (8, 256, [144, 61]), (1, 512, [300, 40])])
def test_learned_map_prefill_on_tcgen05(G, chunk, calls):
    """The learned map's two halves as two linear parts of the tcgen05 prefill kernel: calls that are not multiples of
    anything, several chunks per call, layers without a ring, with short and long windows and one that never evicts;
    outputs at every position, the state after every call, decode steps on top."""
    run_case([0, 16, 100, 128, 304, 1 << 20], 2, 2 * G, 2, 128, BF16, calls, 4, amp=128 ** -0.5 * 4,
             seed=23 + G, phi=1, prefill_chunk=chunk, prefill_impl=glide.GLIDE_PREFILL_TCGEN05)


def test_learned_map_prefill_tcgen05_equals_the_cuda_core_kernel_closely():
    """Same inputs through the tensor-core and the CUDA-core prefill: outputs within the bf16 tolerance of each other,
    and the states they leave (same carry kernel; the keys' features from the tensor cores on one route, from the
    CUDA cores on the other) within the state tolerance."""
    from paper_2607_24788_b200 import synth
    from tests.parity_util import f32_scale, learned_phi_weights
    windows, B, H, Hkv, d, T = [64, 0, 300], 1, 8, 2, 128, 700
    L = len(windows)
    wq, wk = learned_phi_weights(L, H, Hkv, d, BF16, 3)
    wl = synth.Workload(29, L, B, H, Hkv, d, BF16, 4 * d ** -0.5)
    q, k, v = wl.qkv(range(L), range(B), range(T), device="cuda")
    res = []
    for impl in (glide.GLIDE_PREFILL_TCGEN05, glide.GLIDE_PREFILL_FMA):
        g = glide.Glide(windows, B, H, Hkv, d, T, dtype=BF16, softmax_scale=f32_scale(d), phi=1, phi_wq=wq, phi_wk=wk,
                        prefill_impl=impl)
        out = torch.empty_like(q)
        g.glide_prefill(q, k, v, out)
        res.append((out, [g.glide_export_state(l)[2] for l in range(L)]))
        assert g.glide_device_status() == 0
    a, b = res
    err = (a[0].float() - b[0].float()).abs().max().item()
    assert err <= 2e-2, err
    for x, y in zip(a[1], b[1]):
        rel = ((x.double() - y.double()).norm() / y.double().norm().clamp_min(1e-30)).item()
        assert rel <= 1e-5, rel


@pytest.mark.parametrize("phi,G,B", [(0, 4, 1), (0, 8, 2), (1, 4, 1), (0, 1, 3)])
def test_gated_recurrence_on_the_streaming_kernel(phi, G, B):
    """Gates on the bf16 streaming decode kernel: units inside one warp, shared by the warps of a CTA and cut across
    CTAs; a layer without a ring (the current token's gate decays the state), one that never evicts, and decode
    steps that cross a ring wrap (the gate of the leaving token comes from the ring of gates written by earlier
    steps and by the prefill)."""
    Hkv = 2
    run_case([1500, 64, 0, 5000, 300], B, Hkv * G, Hkv, 128, BF16, [1490, 7], 12, amp=4 * 128 ** -0.5, seed=17 + G,
             phi=phi, gated=True, check_prefill_outputs=False, decode_impl=glide.GLIDE_DECODE_STREAM)


def test_gated_streaming_kernel_without_gates_is_bit_identical_to_the_plain_one():
    """A gated context driven without gates multiplies by gamma = 1: the same bits as a context without gates."""
    from paper_2607_24788_b200 import synth
    from tests.parity_util import f32_scale
    windows, B, H, Hkv, d, T = [300, 0, 64], 1, 8, 2, 128, 400
    wl = synth.Workload(19, len(windows), B, H, Hkv, d, BF16, 4 * d ** -0.5)
    outs = []
    for gated in (False, True):
        g = glide.Glide(windows, B, H, Hkv, d, T + 8, dtype=BF16, softmax_scale=f32_scale(d), gated=gated,
                        decode_impl=glide.GLIDE_DECODE_STREAM, prefill_impl=glide.GLIDE_PREFILL_FMA)
        q, k, v = wl.qkv(range(len(windows)), range(B), range(T), device="cuda")
        g.glide_prefill(None, k, v, None)
        got = []
        for s in range(6):
            q, k, v = wl.decode_qkv(T + s, device="cuda")
            out = torch.empty_like(q)
            g.glide_decode_step(q, k, v, out)
            got.append(out)
        got.extend(g.glide_export_state(0)[2:])
        assert g.glide_device_status() == 0
        outs.append(got)
    for x, y in zip(*outs):
        assert torch.equal(x.view(torch.uint8), y.view(torch.uint8))


def test_learned_map_streaming_layer_by_layer_and_ragged_slots():
    """glide_decode_step_layers (one schedule per layer) and slots of different lengths with the learned map."""
    import numpy as np
    from oracle import glide_oracle as orc
    from paper_2607_24788_b200 import synth
    from tests.parity_util import check_outputs, f32_scale, learned_phi_weights, to_np
    windows, B, H, Hkv, d = [40, 0, 200], 2, 8, 2, 128
    L = len(windows)
    wq, wk = learned_phi_weights(L, H, Hkv, d, BF16, 5)
    wl = synth.Workload(13, L, B, H, Hkv, d, BF16, 4 * d ** -0.5)
    g = glide.Glide(windows, B, H, Hkv, d, 400, dtype=BF16, softmax_scale=f32_scale(d), phi=1, phi_wq=wq, phi_wk=wk)
    cells = [[orc.Cell(H, Hkv, d, w, f32_scale(d), phi=1, wq=to_np(wq[l]), wk=to_np(wk[l])) for _ in range(B)]
             for l, w in enumerate(windows)]
    lens = [90, 33]
    for b in range(B):   # slots prefilled one by one to different lengths
        q, k, v = wl.qkv(range(L), [b], range(lens[b]), device="cuda")
        g.glide_reset_seq(b)
        g.glide_prefill_seq(b, None, k[:, 0], v[:, 0], None)
        for l in range(L):
            cells[l][b].prefill(None, to_np(k[l, 0]), to_np(v[l, 0]), outputs=False)
    for s in range(6):
        qs, ks, vs = [], [], []
        for b in range(B):
            q, k, v = wl.qkv(range(L), [b], [lens[b] + s], device="cuda")
            qs.append(q[:, 0, 0]); ks.append(k[:, 0, 0]); vs.append(v[:, 0, 0])
        q, k, v = (torch.stack(x, 1).contiguous() for x in (qs, ks, vs))     # [L][B][heads][d]
        out = torch.full_like(q, float("nan"))
        if s % 2 == 0:
            g.glide_decode_step(q, k, v, out)
        else:
            for l in range(L):
                g.glide_decode_step_layers(q[l:l + 1], k[l:l + 1], v[l:l + 1], out[l:l + 1], l, 1)
        ref = np.stack([[cells[l][b].decode(to_np(q[l, b]), to_np(k[l, b]), to_np(v[l, b])) for b in range(B)]
                        for l in range(L)])
        check_outputs(out, ref, BF16, f"step {s}")
    assert g.glide_device_status() == 0
