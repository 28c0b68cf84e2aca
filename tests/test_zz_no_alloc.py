"""The allocation-free decode entry point against the regular one (collected last on purpose).

glide_decode_step_noalloc serves processes that pre-reserve all device memory and may not call cudaMalloc
afterwards: its split-K scratch is a static buffer inside the library.  Here two contexts are brought to the
same state, then each entry point decodes the same two tokens in a row through the C ABI; outputs, ring rows,
counters and recurrent state must agree (the second call also shows that the shared buffer is re-armed)."""
import pytest
import torch

from tests.parity_util import TOL, f32_scale, to_np

pytestmark = pytest.mark.gpu


def _run(dtype, windows, B, H, Hkv, d, T, amp):
    import numpy as np
    from paper_2607_24788_b200 import glide, synth
    L = len(windows)
    wl = synth.Workload(11, L, B, H, Hkv, d, dtype, amp)
    ctxs = [glide.Glide(windows, B, H, Hkv, d, T + 4, dtype=dtype, softmax_scale=f32_scale(d), decode_chunk=32)
            for _ in range(2)]
    k, v = wl.kv(range(L), range(B), range(T), device="cuda")
    for g in ctxs:
        g.glide_prefill(None, k, v, None)
    tol = TOL[dtype]
    for step in range(2):
        q, k1, v1 = wl.decode_qkv(T + step, device="cuda")
        ref = torch.full_like(q, float("nan"))
        got = torch.full_like(q, float("nan"))
        ctxs[0].glide_decode_step(q, k1, v1, ref)
        ctxs[1].glide_decode_step_noalloc(q, k1, v1, got)
        torch.cuda.synchronize()
        a, b = to_np(got), to_np(ref)
        assert np.isfinite(a).all()
        assert np.abs(a - b).max() <= tol["max_abs"], f"step {step}: max-abs {np.abs(a - b).max():.3e}"
        if tol["rel_l2"] is not None:
            assert np.linalg.norm(a - b) / np.linalg.norm(b) <= tol["rel_l2"]
    for l in range(L):
        assert ctxs[0].glide_layer_info(l) == ctxs[1].glide_layer_info(l)
        for x, y in zip(ctxs[0].glide_export_state(l), ctxs[1].glide_export_state(l)):
            if x.dtype == torch.float32:
                assert torch.allclose(x, y, rtol=1e-5, atol=1e-6)
            else:
                assert torch.equal(x, y)      # ring rows are bit copies of the inputs
    assert ctxs[1].glide_device_status() == 0
    return ctxs


def test_noalloc_matches_decode_step_bf16():
    _run(torch.bfloat16, [200, 48, 0], 2, 8, 2, 128, 230, 128 ** -0.5 * 4)


def test_noalloc_matches_decode_step_fp32():
    _run(torch.float32, [64, 5], 1, 4, 4, 64, 80, 1.0)


def test_noalloc_refuses_configurations_beyond_its_static_buffer():
    from paper_2607_24788_b200 import glide
    # 32 layers x 8 KV heads with 4096-slot windows need ~6 MB of records at 128-slot items; 16-slot items need more
    g = glide.Glide([4096] * 32, 1, 32, 8, 128, 5000, dtype=torch.bfloat16, decode_chunk=16)
    q = torch.zeros((32, 1, 32, 128), dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros((32, 1, 8, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(glide.GlideError) as e:
        g.glide_decode_step_noalloc(q, kv, kv, torch.empty_like(q))
    assert e.value.code == glide.GLIDE_ERR_SCRATCH_LIMIT
    assert g.glide_layer_info(0)["n"] == 0        # a refused call changes nothing
