"""GPU parity: the CUDA path through the C ABI vs the CPU oracle, element by element, same seeded inputs."""
import pytest
import torch

from paper_2607_24788_b200 import configs as C
from tests.parity_util import run_case

pytestmark = pytest.mark.gpu

F32, BF16 = torch.float32, torch.bfloat16


def test_config0_tiny_fp32():
    c = C.C0
    run_case(c.windows, c.batch, c.n_q_heads, c.n_kv_heads, c.head_dim, F32, [c.context], c.decode_steps, amp=1.0)


@pytest.mark.parametrize("w", [0, 1, 2, 3, 15, 16, 17, 63, 64, 65])
def test_window_edge_sizes_decode_only(w):
    # every token goes through decode: T crosses w, ring wraps several times
    run_case([w], 1, 4, 4, 64, F32, [], 150, amp=1.0, seed=w)


@pytest.mark.parametrize("w", [0, 1, 3, 16, 17, 64, 65, 300])
@pytest.mark.parametrize("calls", [(97,), (16, 16, 65), (1, 50, 3, 43)])
def test_prefill_then_decode_fp32(w, calls):
    run_case([w], 2, 4, 2, 64, F32, list(calls), 12, amp=1.0, seed=w + len(calls), prefill_chunk=32)


@pytest.mark.parametrize("G,Hkv", [(1, 2), (2, 2), (4, 2), (8, 1)])
@pytest.mark.parametrize("d", [64, 128])
@pytest.mark.parametrize("dtype", [F32, BF16])
def test_group_sizes_and_head_dims(G, Hkv, d, dtype):
    amp = 1.0 if dtype == F32 else 0.5
    run_case([0, 5, 40, 1000], 2, G * Hkv, Hkv, d, dtype, [70], 20, amp=amp, prefill_chunk=32, decode_chunk=16)


def test_large_logits_exercise_rescaling():
    # q,k x3: window logits with std ~ 9/sqrt(64)*8 -> running-max rescaling and m* = max(m, 0) matter
    run_case([7, 48], 1, 4, 2, 64, F32, [60], 40, amp=3.0, prefill_chunk=16, decode_chunk=8)


def test_non_contiguous_head_map():
    run_case([6, 20], 1, 4, 2, 64, F32, [30], 10, q_to_kv=[1, 0, 0, 1], prefill_chunk=16)


@pytest.mark.parametrize("impl", [1, 2, 3])   # per-item tensor-core kernel, CUDA-core kernel, streaming tensor-core kernel
def test_multi_layer_split_k_bf16(impl):
    # several split-K items per unit, ragged last item, several state row blocks
    run_case([300, 129, 64, 0], 2, 8, 2, 128, BF16, [400], 40, amp=128 ** -0.5 * 4, decode_chunk=64,
             decode_state_splits=4, decode_impl=impl)


@pytest.mark.parametrize("w", [1, 2, 15, 16, 17, 31, 33, 100])
@pytest.mark.parametrize("d,G", [(128, 4), (64, 2), (64, 8), (128, 1)])
def test_bf16_tensor_core_decode_window_edges(w, d, G):
    # every token through decode: partially filled ring, wrap-around, the slot being evicted inside a tile
    run_case([w], 2, 2 * G, 2, d, BF16, [], 2 * w + 40, amp=d ** -0.5 * 4, seed=w, decode_chunk=16 if w < 64 else 48)


@pytest.mark.parametrize("w", [0, 16, 32, 100])
def test_bf16_stream_many_small_units(w):
    # 256 units over 148 CTAs: units that live inside one CTA and units cut by a CTA boundary
    run_case([w] * 8, 8, 8, 4, 128, BF16, [w + 24], 6, amp=128 ** -0.5 * 4, seed=w, decode_impl=3, state_checks=True)


def test_bf16_stream_mixed_windows_and_batch():
    run_case([700, 300, 64, 16, 0, 0, 48, 1 << 20], 3, 8, 2, 128, BF16, [720], 24, amp=128 ** -0.5 * 4, decode_impl=3,
             max_tokens=760)


def test_bf16_large_logits():
    run_case([40, 200], 1, 8, 2, 128, BF16, [250], 30, amp=128 ** -0.5 * 12)


def test_never_evicting_layer_is_full_softmax():
    run_case([1 << 20, 50], 1, 4, 4, 64, F32, [100], 30, max_tokens=130)


def test_layer_ranges_prefilled_separately():
    import numpy as np
    from oracle import glide_oracle as orc
    from paper_2607_24788_b200 import glide, synth
    from tests.parity_util import check_outputs, check_state, f32_scale, to_np
    windows, B, H, Hkv, d, T = [5, 40, 12], 1, 4, 2, 64, 50
    wl = synth.Workload(3, 3, B, H, Hkv, d, F32, 1.0)
    g = glide.Glide(windows, B, H, Hkv, d, 64, dtype=F32, softmax_scale=f32_scale(d), prefill_chunk=16)
    stack = orc.Stack(windows, B, H, Hkv, d, f32_scale(d))
    for lb, lc in ((1, 2), (0, 1)):
        q, k, v = wl.qkv(range(lb, lb + lc), range(B), range(T), device="cuda")
        out = torch.empty_like(q)
        g.glide_prefill(q, k, v, out, layer_begin=lb, layer_count=lc)
        ref = stack.prefill(to_np(q), to_np(k), to_np(v), layer_begin=lb)
        check_outputs(out, ref, F32, f"layers {lb}..{lb+lc}")
    check_state(g, stack)
    q, k, v = wl.decode_qkv(T, device="cuda")
    out = torch.empty_like(q)
    g.glide_decode_step(q, k, v, out)
    check_outputs(out, stack.decode(to_np(q), to_np(k), to_np(v)), F32, "decode")


def test_errors_and_capacity():
    from paper_2607_24788_b200 import glide
    g = glide.Glide([4, 4], 1, 2, 2, 64, 8, dtype=F32)
    q = torch.zeros((2, 1, 2, 64), device="cuda")
    kv = torch.zeros((2, 1, 2, 64), device="cuda")
    k1 = torch.zeros((1, 1, 3, 2, 64), device="cuda")
    g.glide_prefill(None, k1, k1, None, layer_begin=0, layer_count=1)
    with pytest.raises(glide.GlideError) as e:       # layers at different positions
        g.glide_decode_step(q, kv, kv, torch.empty_like(q))
    assert e.value.code == glide.GLIDE_ERR_STATE
    g.glide_prefill(None, k1, k1, None, layer_begin=1, layer_count=1)
    for _ in range(5):
        g.glide_decode_step(q, kv, kv, torch.empty_like(q))
    with pytest.raises(glide.GlideError) as e:       # 8 tokens absorbed: full
        g.glide_decode_step(q, kv, kv, torch.empty_like(q))
    assert e.value.code == glide.GLIDE_ERR_CAPACITY
    assert g.glide_layer_info(0)["n"] == 8
    g.glide_reset()
    assert g.glide_layer_info(1) == dict(window=4, capacity=4, n=0, count=0, head_slot=0, n_evicted=0)


# prefill outputs: impl 1 mma.sync, 2 tcgen05 + TMEM, 3 CUDA cores
@pytest.mark.parametrize("impl,G,chunk", [(1, 1, 96), (1, 4, 256), (2, 1, 256), (2, 4, 96), (2, 4, 256), (3, 4, 96)])
def test_bf16_prefill_tensor_core_multi_call(impl, G, chunk):
    # several calls, so window tiles mix ring rows with the call's rows; windows below, at and above the
    # 128-key tile, one never-evicting layer, one purely linear layer; ragged last query tile
    run_case([0, 100, 128, 300, 1 << 20], 2, 2 * G, 2, 128, BF16, [130, 257, 61], 4, amp=128 ** -0.5 * 4,
             seed=chunk + G, prefill_chunk=chunk, prefill_impl=impl)


def test_contexts_with_different_schedules_coexist():
    # two live contexts whose streaming schedules need different amounts of shared memory; the one created first
    # must still launch after the second was created
    import numpy as np
    from paper_2607_24788_b200 import glide, synth
    from oracle import glide_oracle as orc
    from tests.parity_util import f32_scale, to_np, check_outputs
    d, B, H, Hkv = 128, 1, 8, 2
    shapes = [[48] * 24, [48]]
    wls = [synth.Workload(5 + i, len(w), B, H, Hkv, d, BF16, d ** -0.5 * 4) for i, w in enumerate(shapes)]
    gs = [glide.Glide(w, B, H, Hkv, d, 64, dtype=BF16, softmax_scale=f32_scale(d)) for w in shapes]
    stacks = [orc.Stack(w, B, H, Hkv, d, f32_scale(d)) for w in shapes]
    for t in range(6):
        for g, wl, st, w in zip(gs, wls, stacks, shapes):
            q, k, v = wl.decode_qkv(t, "cuda")
            out = torch.empty_like(q)
            g.glide_decode_step(q, k, v, out)
            ref = st.decode(to_np(q), to_np(k), to_np(v))
            check_outputs(out, ref, BF16, f"L={len(w)} step {t}")


@pytest.mark.parametrize("G,chunk", [(1, 96), (2, 256), (4, 96), (4, 256), (8, 96)])
def test_bf16_prefill_tcgen05_aligned_calls(G, chunk):
    # the tcgen05 kernel runs when every call starts at a multiple of 16 tokens and wrapping rings are multiples
    # of 16: windows below, at and above the 128-key tile, a ring that wraps several times, a never-evicting
    # layer whose ring size is not a multiple of 16, a purely linear layer; one and two row tiles per CTA
    run_case([0, 16, 64, 128, 304, 1 << 20], 2, 2 * G, 2, 128, BF16, [144, 256, 48, 16], 5, amp=128 ** -0.5 * 4,
             seed=chunk + G, prefill_chunk=chunk, prefill_impl=2)


def test_bf16_prefill_tcgen05_large_logits():
    run_case([48, 208], 1, 8, 2, 128, BF16, [256], 6, amp=128 ** -0.5 * 12, prefill_impl=2)


@pytest.mark.parametrize("merge", [1, 2])   # appendix hybrid equations: evicted-token state / all-token state
@pytest.mark.parametrize("dtype,d,kw", [(F32, 64, {}), (BF16, 128, {}), (BF16, 128, dict(prefill_impl=3, decode_impl=2)),
                                        (BF16, 64, {})])
def test_sum_of_terms_merges(merge, dtype, d, kw):
    # bf16 / d = 128 default: tcgen05 prefill + streaming decode; forced CUDA-core kernels; d = 64; fp32
    amp = 1.0 if dtype == F32 else d ** -0.5 * 4
    run_case([0, 1, 5, 40, 1000], 2, 4, 2, d, dtype, [70, 33], 24, amp=amp, seed=merge, prefill_chunk=32, decode_chunk=16,
             merge=merge, **kw)


@pytest.mark.parametrize("merge", [1, 2])
@pytest.mark.parametrize("G,chunk", [(1, 96), (4, 256), (8, 32)])
def test_sum_of_terms_merges_tcgen05_prefill(merge, G, chunk):
    # several calls (aligned and not), windows below / at / above the key tile, a purely linear and a never-evicting layer
    run_case([0, 16, 100, 128, 304, 1 << 20], 2, 2 * G, 2, 128, BF16, [144, 130, 61], 4, amp=128 ** -0.5 * 4,
             seed=merge + G, prefill_chunk=chunk, prefill_impl=2, merge=merge)


@pytest.mark.parametrize("merge", [1, 2])
@pytest.mark.parametrize("G", [1, 4, 8])
def test_sum_of_terms_merges_streaming_kernel(merge, G):
    # bf16, d = 128: decode on the streaming tensor-core kernel (units inside one warp, shared-memory groups and
    # units cut across CTAs all occur with these windows), prefill on the CUDA-core kernel
    # (prefill outputs of these merges are checked in test_sum_of_terms_merges: here the prompt only builds the state)
    run_case([700, 300, 64, 16, 0, 0, 48, 1 << 20], 2, 2 * G, 2, 128, BF16, [720], 12, amp=128 ** -0.5 * 4, seed=merge + G,
             decode_impl=3, merge=merge, check_prefill_outputs=False)
    run_case([0, 5, 40], 3, 2 * G, 2, 128, BF16, [30], 30, amp=128 ** -0.5 * 8, seed=merge, decode_impl=3, merge=merge)


def test_sum_of_terms_merges_kernel_limits():
    from paper_2607_24788_b200 import glide
    with pytest.raises(glide.GlideError):
        glide.Glide([64], 1, 8, 2, 128, 256, dtype=BF16, merge=1, decode_impl=1)   # per-item tensor-core kernel
    with pytest.raises(glide.GlideError):
        glide.Glide([64], 1, 8, 2, 128, 256, dtype=BF16, merge=2, prefill_impl=1)   # mma.sync prefill kernel


@pytest.mark.parametrize("dtype,d,impl,merge", [(BF16, 128, 0, 0), (BF16, 128, 1, 0), (BF16, 64, 0, 0), (F32, 64, 0, 0),
                                               (BF16, 128, 0, 2), (F32, 64, 0, 1)])
def test_decode_step_layers(dtype, d, impl, merge):
    # layer by layer, in ranges, and for the whole stack, interleaved: every path against the oracle, and the
    # positions of the layers bit-exact afterwards (streaming kernel, per-item tensor-core kernel, CUDA-core kernel)
    import numpy as np
    from paper_2607_24788_b200 import glide, synth
    from oracle import glide_oracle as orc
    from tests.parity_util import f32_scale, to_np, check_outputs, check_state
    windows, B, H, Hkv = [40, 0, 16, 300, 1 << 20], 2, 8, 2
    L = len(windows)
    amp = 1.0 if dtype == F32 else d ** -0.5 * 4
    wl = synth.Workload(3, L, B, H, Hkv, d, dtype, amp)
    g = glide.Glide(windows, B, H, Hkv, d, 128, dtype=dtype, softmax_scale=f32_scale(d), decode_impl=impl, merge=merge)
    stack = orc.Stack(windows, B, H, Hkv, d, f32_scale(d), merge=merge)
    q, k, v = wl.qkv(range(L), range(B), range(0, 50), device="cuda")
    g.glide_prefill(None, k, v, None)
    stack.prefill(None, to_np(k), to_np(v), outputs=False)
    for t in range(50, 62):
        q, k, v = wl.decode_qkv(t, "cuda")
        out = torch.full_like(q, float("nan"))
        ref = stack.decode(to_np(q), to_np(k), to_np(v))
        if t % 3 == 0:
            g.glide_decode_step(q, k, v, out)
        elif t % 3 == 1:
            for l in range(L):
                g.glide_decode_step_layers(q[l:l + 1], k[l:l + 1], v[l:l + 1], out[l:l + 1], l, 1)
        else:
            g.glide_decode_step_layers(q[3:5], k[3:5], v[3:5], out[3:5], 3, 2)
            with pytest.raises(glide.GlideError):      # layers 3, 4 are ahead of the others now
                g.glide_decode_step(q, k, v, out)
            g.glide_decode_step_layers(q[0:3], k[0:3], v[0:3], out[0:3], 0, 3)
        check_outputs(out, ref, dtype, f"step {t}")
    check_state(g, stack, "after mixed steps")
    assert g.glide_device_status() == 0


@pytest.mark.parametrize("merge,G", [(0, 4), (0, 8), (1, 4), (0, 1)])
def test_units_cut_into_many_records(merge, G):
    """One long-window layer at batch 1: its few units are spread over many CTAs (eight or nine records per unit), so
    the merging warp reads them in several batches of 16 / G records (one batch for G = 1), each polled until it
    carries the launch's tag; run as one-layer launches and as a whole-stack launch, for several steps (the tags
    move on)."""
    import numpy as np
    from paper_2607_24788_b200 import glide, synth
    from oracle import glide_oracle as orc
    from tests.parity_util import f32_scale, to_np, check_outputs, check_state
    windows, B, Hkv, d, T = [4096, 64], 1, 2, 128, 4200
    H = Hkv * G
    wl = synth.Workload(41 + G, len(windows), B, H, Hkv, d, BF16, d ** -0.5 * 4)
    g = glide.Glide(windows, B, H, Hkv, d, T + 16, dtype=BF16, softmax_scale=f32_scale(d), merge=merge)
    sched = glide.glide_stream_schedule(g.cfg)   # columns 10, 11: record index of the segment, records of its unit
    assert sched[:, 11].max() >= 6, "the whole-stack schedule should cut the long-window units into many records"
    stack = orc.Stack(windows, B, H, Hkv, d, f32_scale(d), merge=merge)
    q, k, v = wl.qkv(range(2), range(B), range(T), device="cuda")
    g.glide_prefill(None, k, v, None)
    stack.prefill(None, to_np(k), to_np(v), outputs=False)
    for t in range(T, T + 6):
        q, k, v = wl.decode_qkv(t, "cuda")
        out = torch.full_like(q, float("nan"))
        ref = stack.decode(to_np(q), to_np(k), to_np(v))
        if t % 2 == 0:
            for l in range(2):
                g.glide_decode_step_layers(q[l:l + 1], k[l:l + 1], v[l:l + 1], out[l:l + 1], l, 1)
        else:
            g.glide_decode_step(q, k, v, out)
        check_outputs(out, ref, BF16, f"step {t}")
    check_state(g, stack, "after steps with many records per unit")
    assert g.glide_device_status() == 0


def test_bf16_prefill_tcgen05_after_decode_steps():
    # a prompt, a few decode steps, then another prompt (a second turn): the second call starts at a position that
    # is not a multiple of 16 and its first key tiles mix ring rows, wrapped ring rows and the call's rows
    from paper_2607_24788_b200 import glide, synth
    from oracle import glide_oracle as orc
    from tests.parity_util import f32_scale, to_np, check_outputs, check_state
    windows, B, H, Hkv, d = [24, 100, 150, 1 << 20, 0], 2, 8, 2, 128
    L = len(windows)
    wl = synth.Workload(17, L, B, H, Hkv, d, BF16, d ** -0.5 * 4)
    g = glide.Glide(windows, B, H, Hkv, d, 600, dtype=BF16, softmax_scale=f32_scale(d), prefill_impl=2)
    stack = orc.Stack(windows, B, H, Hkv, d, f32_scale(d))
    pos = 0
    for T, n_dec in ((173, 5), (140, 3), (64, 0)):
        q, k, v = wl.qkv(range(L), range(B), range(pos, pos + T), device="cuda")
        out = torch.full_like(q, float("nan"))
        g.glide_prefill(q, k, v, out)
        check_outputs(out, stack.prefill(to_np(q), to_np(k), to_np(v)), BF16, f"prefill@{pos}+{T}")
        pos += T
        for _ in range(n_dec):
            q, k, v = wl.decode_qkv(pos, "cuda")
            out = torch.empty_like(q)
            g.glide_decode_step(q, k, v, out)
            check_outputs(out, stack.decode(to_np(q), to_np(k), to_np(v)), BF16, f"decode@{pos}")
            pos += 1
    check_state(g, stack, "after two turns")
    assert g.glide_device_status() == 0


@pytest.mark.parametrize("dtype,d,kw", [(BF16, 128, {}), (BF16, 128, dict(prefill_impl=1, decode_impl=1)),
                                        (BF16, 128, dict(prefill_impl=3, decode_impl=2)), (F32, 64, {})])
def test_very_negative_window_logits_without_linear_terms(dtype, d, kw):
    # every window logit is about -180 (keys close to the all-ones vector, queries close to minus a multiple of it;
    # values of order one): rows that have no evicted token yet, and layers that never evict, must be normalised
    # against their own maximum, not against the logit 0 of the linear terms, or their window weights underflow to
    # 0 / 0.  Every kernel family, prefill and decode.
    from paper_2607_24788_b200 import glide, synth
    from oracle import glide_oracle as orc
    from tests.parity_util import f32_scale, to_np, check_outputs
    windows, B, H, Hkv = [16, 100, 1 << 20], 2, 8, 2
    L = len(windows)
    wl = synth.Workload(5, L, B, H, Hkv, d, dtype, 1.0)
    qmul = 16.0 if d == 128 else 24.0

    def shaped(q, k, v):
        return (-qmul + 0.25 * q.float()).to(dtype), (1.0 + 0.05 * k.float()).to(dtype), v

    g = glide.Glide(windows, B, H, Hkv, d, 64, dtype=dtype, softmax_scale=f32_scale(d), prefill_chunk=32, **kw)
    stack = orc.Stack(windows, B, H, Hkv, d, f32_scale(d))
    q, k, v = shaped(*wl.qkv(range(L), range(B), range(0, 48), device="cuda"))
    logits = torch.einsum("lbthd,lbshd->lbhts", q.float(), k.float().repeat_interleave(H // Hkv, dim=3)) * f32_scale(d)
    assert logits.max().item() < -150.0      # the case is what it claims to be
    out = torch.full_like(q, float("nan"))
    g.glide_prefill(q, k, v, out)
    check_outputs(out, stack.prefill(to_np(q), to_np(k), to_np(v)), dtype, "prefill")
    for t in range(48, 56):
        q, k, v = shaped(*wl.decode_qkv(t, "cuda"))
        out = torch.empty_like(q)
        g.glide_decode_step(q, k, v, out)
        check_outputs(out, stack.decode(to_np(q), to_np(k), to_np(v)), dtype, f"decode@{t}")


def test_streaming_kernel_with_hundreds_of_units_per_cta():
    # 32 768 small units: the segment table of a CTA takes over most of the shared-memory record pool; the streaming
    # kernel (asked for explicitly) must still apply and agree with the oracle
    run_case([0, 1] * 16, 128, 8, 8, 128, BF16, [], 3, amp=128 ** -0.5 * 4, seed=3, decode_impl=3, state_checks=False)


@pytest.mark.parametrize("impl", [2, 3])
def test_chunk_scan_carry_stays_fp32_accurate_over_a_long_prompt(impl):
    """16 chunks of carry: the tensor-core state kernel (prefill_impl 2: phi(K') split into three bf16 terms, exact
    products, fp32 accumulation) and the CUDA-core one (prefill_impl 3) both stay well inside the 1e-5 state tolerance."""
    import numpy as np
    from oracle import glide_oracle as orc
    from paper_2607_24788_b200 import glide, synth
    from tests.parity_util import f32_scale, to_np
    L, B, H, Hkv, d, T = 2, 1, 8, 2, 128, 4096
    windows = [64, 0]
    wl = synth.Workload(11, L, B, H, Hkv, d, BF16, 2.0)
    g = glide.Glide(windows, B, H, Hkv, d, T + 8, dtype=BF16, softmax_scale=f32_scale(d), prefill_impl=impl)
    stack = orc.Stack(windows, B, H, Hkv, d, f32_scale(d))
    q, k, v = wl.qkv(range(L), range(B), range(T), device="cuda")
    g.glide_prefill(None, k, v, None)
    stack.prefill(to_np(q), to_np(k), to_np(v), outputs=False)
    for l in range(L):
        _, _, S, z = g.glide_export_state(l)
        _, _, oS, oz = stack.cells[l][0].export()
        assert np.linalg.norm(to_np(S[0]) - oS) / np.linalg.norm(oS) <= 3e-6
        assert np.linalg.norm(to_np(z[0]) - oz) / np.linalg.norm(oz) <= 3e-6
    g.glide_destroy()
