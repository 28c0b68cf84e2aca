"""Pins for the CPU oracle: checks against things other than itself.

* form B (defining sums) vs a library causal softmax attention when w >= n       (Sec. III-B boundary condition)
* form B with w = 0 vs matrix-form linear attention built from library matmuls    (Sec. II, Eq. 6)
* form B for general w vs a masked-matrix evaluation assembled from library softmax / logsumexp / matmul
  pieces merged by their denominators                                             (the "(+)" operator)
* the q = k = 0 closed form (exact rationals, tests/golden/closed_form_zero_qk.txt)
* convexity (weights positive, sum to one)
* form A (ring + state) vs form B, decode == prefill, bookkeeping arithmetic
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import glide_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rand_qkv(T, H, Hkv, d, seed, amp=1.0):
    rng = np.random.default_rng(seed)
    return (amp * rng.standard_normal((T, H, d)), amp * rng.standard_normal((T, Hkv, d)),
            rng.standard_normal((T, Hkv, d)))


def expand_kv(x, H):
    """[T][Hkv][d] -> [T][H][d] for contiguous GQA groups."""
    return np.repeat(x, H // x.shape[1], axis=1)


# ----------------------------------------------------------------------------------------------
# w >= n  ==>  standard causal softmax attention (library routine)
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("T,H,Hkv,d,w", [(40, 4, 4, 16, 40), (33, 8, 2, 8, 1000), (17, 2, 1, 64, 17)])
def test_full_window_is_causal_softmax(T, H, Hkv, d, w):
    q, k, v = rand_qkv(T, H, Hkv, d, 1)
    scale = 1.0 / math.sqrt(d)
    got = orc.bruteforce(q, k, v, w, scale)
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]                  # [1][H][T][d]
    tk = torch.from_numpy(expand_kv(k, H)).permute(1, 0, 2)[None]
    tv = torch.from_numpy(expand_kv(v, H)).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=scale)
    ref = ref[0].permute(1, 0, 2).numpy()
    np.testing.assert_allclose(got, ref, rtol=1e-11, atol=1e-12)


def test_scale_is_applied_to_window_logits_only():
    # same inputs, two scales: the library routine is re-run with each, so a dropped or misplaced scale fails
    q, k, v = rand_qkv(24, 2, 2, 8, 2, amp=2.0)
    for scale in (1.0, 0.25):
        got = orc.bruteforce(q, k, v, 24, scale)
        tq, tk, tv = (torch.from_numpy(x).permute(1, 0, 2)[None] for x in (q, k, v))
        ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=scale)
        np.testing.assert_allclose(got, ref[0].permute(1, 0, 2).numpy(), rtol=1e-11, atol=1e-12)


# ----------------------------------------------------------------------------------------------
# w = 0  ==>  pure linear attention, phi = softmax over features, inclusive of the current token
# ----------------------------------------------------------------------------------------------
def linear_attention_matrix_form(q, k, v):
    """O = (tril(phi(Q) phi(K)^T) V) / rowsum(tril(...)), per head, with library softmax/matmul."""
    T, H, d = q.shape
    k, v = expand_kv(k, H), expand_kv(v, H)
    out = np.empty_like(q)
    for h in range(H):
        fq = torch.softmax(torch.from_numpy(q[:, h]), dim=-1)
        fk = torch.softmax(torch.from_numpy(k[:, h]), dim=-1)
        A = torch.tril(fq @ fk.T)
        out[:, h] = ((A @ torch.from_numpy(v[:, h])) / A.sum(-1, keepdim=True)).numpy()
    return out


@pytest.mark.parametrize("T,H,Hkv,d", [(30, 2, 2, 8), (21, 4, 1, 16)])
def test_zero_window_is_linear_attention(T, H, Hkv, d):
    q, k, v = rand_qkv(T, H, Hkv, d, 3, amp=1.5)
    got = orc.bruteforce(q, k, v, 0, 1.0 / math.sqrt(d))
    np.testing.assert_allclose(got, linear_attention_matrix_form(q, k, v), rtol=1e-11, atol=1e-12)


# ----------------------------------------------------------------------------------------------
# general w: two separately normalised library pieces merged by their denominators
# ----------------------------------------------------------------------------------------------
def hybrid_matrix_form(q, k, v, w, scale):
    T, H, d = q.shape
    k, v = expand_kv(k, H), expand_kv(v, H)
    i = torch.arange(T)[:, None]
    j = torch.arange(T)[None, :]
    in_window = (j <= i) & (j > i - w)
    evicted = j <= i - w
    out = np.empty_like(q)
    for h in range(H):
        Q, K, V = (torch.from_numpy(x[:, h]) for x in (q, k, v))
        logits = (Q @ K.T) * scale
        neg = torch.full_like(logits, -float("inf"))
        wl = torch.where(in_window, logits, neg)
        if w > 0:
            O_swa = torch.softmax(wl, dim=-1) @ V                  # separately normalised window output
            D_swa = torch.exp(torch.logsumexp(wl, dim=-1))         # its denominator
        else:
            O_swa = torch.zeros_like(V)
            D_swa = torch.zeros(T, dtype=torch.float64)
        A = (torch.softmax(Q, -1) @ torch.softmax(K, -1).T) * evicted
        D_lin = A.sum(-1)
        O_lin = torch.where(D_lin[:, None] > 0, (A @ V) / D_lin.clamp_min(1e-300)[:, None], torch.zeros_like(V))
        o = (D_swa[:, None] * O_swa + D_lin[:, None] * O_lin) / (D_swa + D_lin)[:, None]
        out[:, h] = o.numpy()
    return out


@pytest.mark.parametrize("w", [1, 2, 3, 5, 16, 31])
@pytest.mark.parametrize("amp", [1.0, 3.0])
def test_general_window_matches_denominator_weighted_merge(w, amp):
    T, H, Hkv, d = 48, 4, 2, 8
    q, k, v = rand_qkv(T, H, Hkv, d, 10 + w, amp=amp)
    scale = 1.0 / math.sqrt(d)
    np.testing.assert_allclose(orc.bruteforce(q, k, v, w, scale), hybrid_matrix_form(q, k, v, w, scale),
                               rtol=1e-10, atol=1e-12)


def test_non_contiguous_head_map():
    T, H, Hkv, d, w = 20, 4, 2, 8, 4
    q, k, v = rand_qkv(T, H, Hkv, d, 5)
    m = np.array([1, 0, 0, 1], dtype=np.int32)
    got = orc.bruteforce(q, k, v, w, 0.3, q_to_kv=m)
    ref = hybrid_matrix_form(q, k[:, m], v[:, m], w, 0.3)   # k[:, m] has H heads: groups of size 1
    np.testing.assert_allclose(got, ref, rtol=1e-10, atol=1e-12)


# ----------------------------------------------------------------------------------------------
# closed form with q = k = 0 and v_j[0] = j
# ----------------------------------------------------------------------------------------------
def _closed_form_rows():
    rows = []
    with open(os.path.join(GOLDEN, "closed_form_zero_qk.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                d, w, t, num, den = line.split()
                rows.append((int(d), int(w), int(t), float(num), float(den)))
    return rows


@pytest.mark.parametrize("d,w,t,num,den", _closed_form_rows())
def test_closed_form_zero_qk(d, w, t, num, den):
    T = t + 1
    q = np.zeros((T, 1, d))
    k = np.zeros((T, 1, d))
    v = np.zeros((T, 1, d))
    v[:, 0, 0] = np.arange(T)
    v[:, 0, 1] = 1.0
    out_b = orc.bruteforce(q, k, v, w, 1.0 / math.sqrt(d), sel=[t])[0, 0]
    assert out_b[0] == pytest.approx(num / den, rel=1e-13)
    assert out_b[1] == pytest.approx(1.0, rel=1e-13)
    cell = orc.Cell(1, 1, d, w, 1.0 / math.sqrt(d))
    for i in range(T):
        o = cell.decode(q[i], k[i], v[i])
    assert o[0, 0] == pytest.approx(num / den, rel=1e-12)
    cell2 = orc.Cell(1, 1, d, w, 1.0 / math.sqrt(d))
    o2 = cell2.prefill(q, k, v, sel=[t])
    assert o2[0, 0, 0] == pytest.approx(num / den, rel=1e-12)


# ----------------------------------------------------------------------------------------------
# convexity: positive weights that sum to one
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("w", [0, 1, 7, 100])
def test_convex_combination(w):
    T, H, Hkv, d = 40, 4, 2, 8
    q, k, v = rand_qkv(T, H, Hkv, d, 7, amp=2.0)
    vc = np.full_like(v, 3.25)
    np.testing.assert_allclose(orc.bruteforce(q, k, vc, w, 0.5), 3.25, rtol=1e-13)
    out = orc.bruteforce(q, k, v, w, 0.5)
    vx = expand_kv(v, H)
    for t in range(T):
        assert (out[t] <= vx[: t + 1].max(0) + 1e-12).all() and (out[t] >= vx[: t + 1].min(0) - 1e-12).all()


# ----------------------------------------------------------------------------------------------
# form A (ring + state) vs form B; decode == prefill; chunked prefill; bookkeeping
# ----------------------------------------------------------------------------------------------
@pytest.mark.parametrize("d,H,Hkv", [(2, 1, 1), (4, 4, 2), (64, 4, 4)])
@pytest.mark.parametrize("w", [0, 1, 2, 3, 5, 64])
def test_stateful_decode_matches_bruteforce(d, H, Hkv, w):
    T = 150 if d < 64 else 200
    q, k, v = rand_qkv(T, H, Hkv, d, 100 + w, amp=1.5)
    scale = 1.0 / math.sqrt(d)
    ref = orc.bruteforce(q, k, v, w, scale)
    cell = orc.Cell(H, Hkv, d, w, scale)
    for t in range(T):
        np.testing.assert_allclose(cell.decode(q[t], k[t], v[t]), ref[t], rtol=1e-10, atol=1e-12)
        info = cell.info()
        n = t + 1
        assert info == dict(n=n, count=min(n, w), head_slot=(n % w if w else 0), n_evicted=max(0, n - w))


@pytest.mark.parametrize("w", [0, 1, 3, 16, 64, 1000])
@pytest.mark.parametrize("chunks", [(97,), (16, 16, 65), (1, 50, 3, 43), (64, 33)])
def test_prefill_matches_bruteforce_and_decode(w, chunks):
    H, Hkv, d = 4, 2, 8
    T = sum(chunks)
    q, k, v = rand_qkv(T, H, Hkv, d, 200 + w, amp=1.5)
    scale = 0.4
    ref = orc.bruteforce(q, k, v, w, scale)
    pre = orc.Cell(H, Hkv, d, w, scale)
    dec = orc.Cell(H, Hkv, d, w, scale)
    pos = 0
    for c in chunks:
        out = pre.prefill(q[pos:pos + c], k[pos:pos + c], v[pos:pos + c])
        np.testing.assert_allclose(out, ref[pos:pos + c], rtol=1e-10, atol=1e-12)
        pos += c
    for t in range(T):
        dec.decode(q[t], k[t], v[t])
    assert pre.info() == dec.info()
    np.testing.assert_array_equal(pre.slot_tokens(), dec.slot_tokens())
    for a, b in zip(pre.export(), dec.export()):
        np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-14)
    # ring holds token j at slot j mod w, verbatim
    rk, rv, _, _ = pre.export()
    for s, j in enumerate(pre.slot_tokens()):
        if j >= 0:
            np.testing.assert_array_equal(rk[:, s], k[j])
            np.testing.assert_array_equal(rv[:, s], v[j])
    # decode continues identically from either state
    q2, k2, v2 = rand_qkv(5, H, Hkv, d, 999)
    for t in range(5):
        np.testing.assert_allclose(pre.decode(q2[t], k2[t], v2[t]), dec.decode(q2[t], k2[t], v2[t]), rtol=1e-10)


def test_state_is_sum_over_evicted_tokens():
    H, Hkv, d, w, T = 2, 2, 4, 5, 23
    q, k, v = rand_qkv(T, H, Hkv, d, 42)
    cell = orc.Cell(H, Hkv, d, w, 0.5)
    cell.prefill(None, k, v, outputs=False)
    _, _, S, z = cell.export()
    fk = torch.softmax(torch.from_numpy(k[: T - w]), dim=-1).numpy()       # [E][Hkv][d]
    np.testing.assert_allclose(S, np.einsum("egr,egc->grc", fk, v[: T - w]), rtol=1e-12)
    np.testing.assert_allclose(z, fk.sum(0), rtol=1e-12)


def test_slot_tokens_and_eviction_order():
    cell = orc.Cell(1, 1, 2, 4, 1.0)
    z = np.zeros((1, 2))
    for t in range(10):
        cell.decode(z, z, z)
    # tokens 6..9 live at slots j mod 4
    assert list(cell.slot_tokens()) == [8, 9, 6, 7]
    assert cell.info() == dict(n=10, count=4, head_slot=2, n_evicted=6)


def test_stack_decode_threads_match_serial():
    L, B, H, Hkv, d = 3, 2, 4, 2, 8
    windows = [0, 3, 50]
    rng = np.random.default_rng(0)
    a = orc.Stack(windows, B, H, Hkv, d, 0.5)
    for t in range(12):
        q = rng.standard_normal((L, B, H, d))
        k = rng.standard_normal((L, B, Hkv, d))
        v = rng.standard_normal((L, B, Hkv, d))
        out = a.decode(q, k, v, threads=4)
        for l in range(L):
            for b in range(B):
                pass
        if t == 0:
            hist = [[[] for _ in range(B)] for _ in range(L)]
        for l in range(L):
            for b in range(B):
                hist[l][b].append((q[l, b], k[l, b], v[l, b]))
                qq, kk, vv = (np.stack(x) for x in zip(*hist[l][b]))
                ref = orc.bruteforce(qq, kk, vv, windows[l], 0.5, sel=[t])[0]
                np.testing.assert_allclose(out[l, b], ref, rtol=1e-10, atol=1e-12)
