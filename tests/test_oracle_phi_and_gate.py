"""Pins for the two extensions of the CPU oracle: the learned feature map phi_W(x) = [softmax(W^T x); softmax(-W^T x)]
and the gated recurrence S <- gamma S + phi(k) v^T (checks against things other than the oracle itself).

* closed forms with exact rationals (tests/golden/closed_form_learned_phi_and_gate.txt): W = 0, and constant gates
  with q = k = 0
* w = 0 vs matrix-form (gated) linear attention built from library softmax / matmul / cumsum; W = I and random,
  non-symmetric W per head (a transposed W or a per-layer instead of per-head W fails)
* general w vs a denominator-weighted merge of library pieces
* gamma = 1 reproduces the ungated method bit for bit
* form A (ring + state) vs form B at every position, decode == prefill with chunked calls, state = its defining sum
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import glide_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "closed_form_learned_phi_and_gate.txt")


def rand_case(T, H, Hkv, d, seed, amp=1.0, gates=False, learned=True):
    rng = np.random.default_rng(seed)
    q, k, v = amp * rng.standard_normal((T, H, d)), amp * rng.standard_normal((T, Hkv, d)), rng.standard_normal((T, Hkv, d))
    wq = rng.standard_normal((H, d, d)) / math.sqrt(d) if learned else None
    wk = rng.standard_normal((Hkv, d, d)) / math.sqrt(d) if learned else None
    gate = rng.uniform(0.5, 1.0, size=(T, Hkv)) if gates else None
    return q, k, v, wq, wk, gate


def phi_lib(x, W):
    """[T][d] -> [T][2d] with library softmax: y = x @ W, i.e. y_j = sum_i x_i W[i][j]."""
    y = torch.from_numpy(x) @ torch.from_numpy(W)
    return torch.cat([torch.softmax(y, -1), torch.softmax(-y, -1)], -1)


def linear_matrix_form(q, k, v, wq, wk, gate=None, delay=0):
    """Gated linear attention in matrix form: A_ij = phi(q_i).phi(k_j) * prod_{m=j+1..i-delay} gate_m for
    j <= i - delay; returns (A V, rowsum A) per head, [T][H][d] and [T][H]."""
    T, H, d = q.shape
    Hkv = k.shape[1]
    G = H // Hkv
    num, den = np.zeros((T, H, d)), np.zeros((T, H))
    for h in range(H):
        g = h // G
        fq = phi_lib(q[:, h], wq[h]) if wq is not None else torch.softmax(torch.from_numpy(q[:, h]), -1)
        fk = phi_lib(k[:, g], wk[g]) if wk is not None else torch.softmax(torch.from_numpy(k[:, g]), -1)
        A = fq @ fk.T
        i, j = torch.meshgrid(torch.arange(T), torch.arange(T), indexing="ij")
        mask = j <= i - delay
        if gate is not None:
            cum = torch.cumsum(torch.log(torch.from_numpy(gate[:, g])), 0)       # log of prod_{m<=x} gate_m
            hi = torch.clamp(i - delay, min=0)
            A = A * torch.exp(cum[hi] - cum[j])
        A = torch.where(mask, A, torch.zeros_like(A))
        num[:, h] = (A @ torch.from_numpy(v[:, g])).numpy()
        den[:, h] = A.sum(-1).numpy()
    return num, den


def test_closed_forms_of_the_golden_file():
    rows = [l.split() for l in open(GOLDEN) if l.strip() and not l.startswith("#")]
    assert len(rows) == 6
    for kind, d, w, t, gamma, numer, denom in rows:
        d, w, t, gamma = int(d), int(w), int(t), float(gamma)
        T = t + 1
        q, k = np.zeros((T, 1, d)), np.zeros((T, 1, d))
        v = np.zeros((T, 1, d))
        v[:, 0, 0] = np.arange(T)
        if kind == "phi":
            out = orc.bruteforce(q, k, v, w, 1.0, sel=[t], phi=1, wq=np.zeros((1, d, d)), wk=np.zeros((1, d, d)))
            cell = orc.Cell(1, 1, d, w, 1.0, phi=1, wq=np.zeros((1, d, d)), wk=np.zeros((1, d, d)))
            gate = None
        else:
            gate = np.full((T, 1), gamma)
            out = orc.bruteforce(q, k, v, w, 1.0, sel=[t], gate=gate)
            cell = orc.Cell(1, 1, d, w, 1.0)
        want = float(numer) / float(denom)
        assert abs(out[0, 0, 0] - want) <= 1e-12 * max(1.0, abs(want)), (kind, d, w, t)
        for s in range(T):   # the stateful form, token by token
            o = cell.decode(q[s], k[s], v[s], gate=None if gate is None else gate[s])
        assert abs(o[0, 0] - want) <= 1e-12 * max(1.0, abs(want)), (kind, d, w, t, "form A")


def test_zero_projection_makes_the_linear_weights_independent_of_q_and_k():
    """W = 0: every evicted token weighs 2/d whatever q and k are; the window keeps its softmax weights."""
    T, H, Hkv, d, w = 40, 4, 2, 8, 5
    q, k, v, _, _, _ = rand_case(T, H, Hkv, d, 1)
    out = orc.bruteforce(q, k, v, w, 0.3, phi=1, wq=np.zeros((H, d, d)), wk=np.zeros((Hkv, d, d)))
    G = H // Hkv
    for t in (0, 4, 5, 17, 39):
        for h in range(H):
            g = h // G
            lo = max(0, t - w + 1)
            a = np.exp(0.3 * (k[lo:t + 1, g] @ q[t, h]))
            num = a @ v[lo:t + 1, g] + (2.0 / d) * v[:lo, g].sum(0)
            den = a.sum() + (2.0 / d) * lo
            np.testing.assert_allclose(out[t, h], num / den, rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("identity", [True, False])
@pytest.mark.parametrize("T,H,Hkv,d", [(30, 2, 2, 8), (21, 4, 1, 16), (18, 8, 2, 4)])
def test_zero_window_is_linear_attention_with_the_learned_map(T, H, Hkv, d, identity):
    q, k, v, wq, wk, _ = rand_case(T, H, Hkv, d, 3, amp=1.5)
    if identity:   # W = I: phi(x) = [softmax(x); softmax(-x)]
        wq, wk = np.stack([np.eye(d)] * H), np.stack([np.eye(d)] * Hkv)
    got = orc.bruteforce(q, k, v, 0, 1.0 / math.sqrt(d), phi=1, wq=wq, wk=wk)
    num, den = linear_matrix_form(q, k, v, wq, wk)
    np.testing.assert_allclose(got, num / den[..., None], rtol=1e-10, atol=1e-12)


@pytest.mark.parametrize("learned", [False, True])
@pytest.mark.parametrize("T,H,Hkv,d", [(26, 2, 2, 8), (19, 4, 2, 4)])
def test_zero_window_is_gated_linear_attention(T, H, Hkv, d, learned):
    q, k, v, wq, wk, gate = rand_case(T, H, Hkv, d, 5, gates=True, learned=learned)
    got = orc.bruteforce(q, k, v, 0, 1.0, phi=int(learned), wq=wq, wk=wk, gate=gate)
    num, den = linear_matrix_form(q, k, v, wq, wk, gate)
    np.testing.assert_allclose(got, num / den[..., None], rtol=1e-10, atol=1e-12)


@pytest.mark.parametrize("w", [1, 3, 7, 64])
@pytest.mark.parametrize("gates", [False, True])
def test_general_window_is_the_denominator_weighted_merge_of_library_pieces(w, gates):
    """window part from library softmax / logsumexp, linear part from the matrix form above (delayed by w), merged
    as (D_lin O_lin + D_swa O_swa) / (D_lin + D_swa)."""
    T, H, Hkv, d = 24, 4, 2, 8
    q, k, v, wq, wk, gate = rand_case(T, H, Hkv, d, 7, gates=gates)
    scale = 0.4
    got = orc.bruteforce(q, k, v, w, scale, phi=1, wq=wq, wk=wk, gate=gate)
    num_l, den_l = linear_matrix_form(q, k, v, wq, wk, gate, delay=w)
    G = H // Hkv
    for h in range(H):
        g = h // G
        logits = scale * torch.from_numpy(q[:, h]) @ torch.from_numpy(k[:, g]).T
        i, j = torch.meshgrid(torch.arange(T), torch.arange(T), indexing="ij")
        logits = torch.where((j <= i) & (j > i - w), logits, torch.full_like(logits, -math.inf))
        lse = torch.logsumexp(logits, -1)
        o_swa = (torch.softmax(logits, -1) @ torch.from_numpy(v[:, g])).numpy()
        d_swa = torch.exp(lse).numpy()
        want = (d_swa[:, None] * o_swa + num_l[:, h]) / (d_swa + den_l[:, h])[:, None]
        np.testing.assert_allclose(got[:, h], want, rtol=1e-10, atol=1e-12)


def test_unit_gates_reproduce_the_ungated_method_bit_for_bit():
    T, H, Hkv, d, w = 30, 4, 2, 8, 6
    q, k, v, wq, wk, _ = rand_case(T, H, Hkv, d, 9)
    ones = np.ones((T, Hkv))
    for phi, a, b in ((0, None, None), (1, wq, wk)):
        assert np.array_equal(orc.bruteforce(q, k, v, w, 0.5, phi=phi, wq=a, wk=b),
                              orc.bruteforce(q, k, v, w, 0.5, phi=phi, wq=a, wk=b, gate=ones))
        c0, c1 = orc.Cell(H, Hkv, d, w, 0.5, phi=phi, wq=a, wk=b), orc.Cell(H, Hkv, d, w, 0.5, phi=phi, wq=a, wk=b)
        for t in range(T):
            assert np.array_equal(c0.decode(q[t], k[t], v[t]), c1.decode(q[t], k[t], v[t], gate=ones[t]))
        for x, y in zip(c0.export(), c1.export()):
            assert np.array_equal(x, y)


@pytest.mark.parametrize("phi,gates", [(1, False), (0, True), (1, True)])
@pytest.mark.parametrize("w,merge", [(0, 0), (1, 0), (5, 0), (64, 0), (4, 1), (4, 2)])
def test_form_a_equals_form_b_and_decode_equals_prefill(phi, gates, w, merge):
    T, H, Hkv, d = 37, 4, 2, 8
    q, k, v, wq, wk, gate = rand_case(T, H, Hkv, d, 11 + w, gates=gates, learned=bool(phi))
    scale = 0.35
    ref = orc.bruteforce(q, k, v, w, scale, merge=merge, phi=phi, wq=wq, wk=wk, gate=gate)
    dec = orc.Cell(H, Hkv, d, w, scale, merge=merge, phi=phi, wq=wq, wk=wk)
    for t in range(T):
        o = dec.decode(q[t], k[t], v[t], gate=None if gate is None else gate[t])
        np.testing.assert_allclose(o, ref[t], rtol=1e-10, atol=1e-12, err_msg=f"decode t={t}")
    pre = orc.Cell(H, Hkv, d, w, scale, merge=merge, phi=phi, wq=wq, wk=wk)
    pos = 0
    for n in (1, 9, 0, 20, 7):
        o = pre.prefill(q[pos:pos + n], k[pos:pos + n], v[pos:pos + n], gate=None if gate is None else gate[pos:pos + n])
        np.testing.assert_allclose(o, ref[pos:pos + n], rtol=1e-10, atol=1e-12, err_msg=f"prefill at {pos}")
        pos += n
    assert pos == T and pre.info() == dec.info()
    for x, y in zip(pre.export() + (pre.export_gates(),), dec.export() + (dec.export_gates(),)):
        np.testing.assert_allclose(x, y, rtol=1e-11, atol=1e-13)
    # the state is its defining sum: tokens that have entered it, each with the gates of the later entries
    delay = 0 if merge == 2 else w
    n_in = max(0, T - delay)
    S = dec.export()[2]
    G = H // Hkv
    for g in range(Hkv):
        fk = phi_lib(k[:n_in, g], wk[g]).numpy() if phi else torch.softmax(torch.from_numpy(k[:n_in, g]), -1).numpy()
        wts = np.ones(n_in)
        if gate is not None:
            for j in range(n_in):
                wts[j] = np.prod(gate[j + 1:n_in, g])
        np.testing.assert_allclose(S[g], np.einsum("t,tr,tc->rc", wts, fk, v[:n_in, g]), rtol=1e-10, atol=1e-12)
    assert S.shape == (Hkv, 2 * d if phi else d, d)


def test_gates_wait_in_the_ring_with_their_tokens():
    """The gate that decays the state at step t is the one token t - w brought, not the current token's."""
    H = Hkv = 1
    d, w, T = 4, 3, 9
    rng = np.random.default_rng(2)
    q, k, v = rng.standard_normal((T, 1, d)), rng.standard_normal((T, 1, d)), rng.standard_normal((T, 1, d))
    gate = rng.uniform(0.3, 1.0, size=(T, 1))
    cell = orc.Cell(H, Hkv, d, w, 1.0)
    for t in range(T):
        cell.decode(q[t], k[t], v[t], gate=gate[t])
    z = cell.export()[3][0]
    fk = torch.softmax(torch.from_numpy(k[:, 0]), -1).numpy()
    n_in = T - w
    want = sum(fk[j] * np.prod(gate[j + 1:n_in, 0]) for j in range(n_in))
    np.testing.assert_allclose(z, want, rtol=1e-12)
    np.testing.assert_array_equal(cell.export_gates()[0], [gate[t, 0] for t in (6, 7, 8)])   # slots 6%3, 7%3, 8%3
