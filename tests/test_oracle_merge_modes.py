"""Pins for the oracle's alternative merges (appendix "(b) Retention-based SWA": the two hybrid equations).

merge = 1: O_t = phi(q) S_{t-w} / phi(q) z_{t-w} + window softmax        (state = evicted tokens)
merge = 2: O_t = phi(q) S_t / phi(q) z_t + window softmax                (state = every token up to t)

Each is checked against library routines that do not come from the oracle: a library softmax attention over the
window slice plus matrix-form linear attention over the token set of the state; closed forms for q = k = 0; the
limits in which a term vanishes; and form A (ring + state, decode and prefill) against form B.
"""
import math

import numpy as np
import pytest
import torch

from oracle import glide_oracle as orc
from tests.test_oracle_pins import expand_kv, linear_attention_matrix_form, rand_qkv


def sum_of_terms_matrix_form(q, k, v, w, scale, merge):
    """Window term: library softmax over the masked logits; linear term: tril-masked phi(Q) phi(K)^T, normalised."""
    T, H, d = q.shape
    k, v = expand_kv(k, H), expand_kv(v, H)
    i = torch.arange(T)[:, None]
    j = torch.arange(T)[None, :]
    in_window = (j <= i) & (j > i - w)
    in_state = (j <= i - w) if merge == 1 else (j <= i)
    out = np.empty_like(q)
    for h in range(H):
        Q, K, V = (torch.from_numpy(x[:, h]) for x in (q, k, v))
        o = torch.zeros_like(V)
        if w > 0:
            logits = torch.where(in_window, (Q @ K.T) * scale, torch.full((T, T), -float("inf"), dtype=torch.float64))
            o = o + torch.softmax(logits, dim=-1) @ V
        A = (torch.softmax(Q, -1) @ torch.softmax(K, -1).T) * in_state
        D = A.sum(-1, keepdim=True)
        o = o + torch.where(D > 0, (A @ V) / D.clamp_min(1e-300), torch.zeros_like(V))
        out[:, h] = o.numpy()
    return out


@pytest.mark.parametrize("merge", [1, 2])
@pytest.mark.parametrize("w", [0, 1, 2, 5, 16, 31, 100])
@pytest.mark.parametrize("amp", [1.0, 3.0])
def test_sum_of_separately_normalised_terms(merge, w, amp):
    T, H, Hkv, d = 48, 4, 2, 8
    q, k, v = rand_qkv(T, H, Hkv, d, 20 + w + merge, amp=amp)
    scale = 1.0 / math.sqrt(d)
    np.testing.assert_allclose(orc.bruteforce(q, k, v, w, scale, merge=merge),
                               sum_of_terms_matrix_form(q, k, v, w, scale, merge), rtol=1e-10, atol=1e-12)


def test_evicted_state_sum_is_plain_softmax_until_the_window_fills():
    # merge = 1 with w >= n: the linear term has no tokens, the output is standard causal attention
    T, H, Hkv, d = 30, 4, 2, 16
    q, k, v = rand_qkv(T, H, Hkv, d, 7)
    scale = 1.0 / math.sqrt(d)
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(expand_kv(k, H)).permute(1, 0, 2)[None]
    tv = torch.from_numpy(expand_kv(v, H)).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=scale)[0].permute(1, 0, 2).numpy()
    np.testing.assert_allclose(orc.bruteforce(q, k, v, T, scale, merge=1), ref, rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("merge", [1, 2])
def test_zero_window_is_linear_attention_in_every_mode(merge):
    T, H, Hkv, d = 25, 2, 2, 8
    q, k, v = rand_qkv(T, H, Hkv, d, 8, amp=1.5)
    np.testing.assert_allclose(orc.bruteforce(q, k, v, 0, 0.5, merge=merge), linear_attention_matrix_form(q, k, v),
                               rtol=1e-11, atol=1e-12)


def test_all_token_state_with_full_window_is_softmax_plus_linear():
    # merge = 2, w >= n: both terms run over the whole causal prefix
    T, H, Hkv, d = 20, 2, 1, 8
    q, k, v = rand_qkv(T, H, Hkv, d, 9)
    scale = 0.3
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]
    tk = torch.from_numpy(expand_kv(k, H)).permute(1, 0, 2)[None]
    tv = torch.from_numpy(expand_kv(v, H)).permute(1, 0, 2)[None]
    soft = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=scale)[0].permute(1, 0, 2).numpy()
    np.testing.assert_allclose(orc.bruteforce(q, k, v, T, scale, merge=2), soft + linear_attention_matrix_form(q, k, v),
                               rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("d,w,t", [(4, 3, 10), (64, 64, 511), (8, 5, 4), (8, 0, 6)])
def test_closed_form_zero_qk(d, w, t):
    # q = k = 0: every window weight is 1 and every feature product is 1/d, so each term is a plain mean of its
    # tokens' values; with v_j[0] = j the means are exact rationals
    T = t + 1
    q = np.zeros((T, 1, d))
    k = np.zeros((T, 1, d))
    v = np.zeros((T, 1, d))
    v[:, 0, 0] = np.arange(T)
    win = list(range(max(0, t - w + 1), t + 1)) if w > 0 else []
    mean = lambda xs: sum(xs) / len(xs) if xs else 0.0
    want1 = mean(win) + mean(list(range(0, t - w + 1)))
    want2 = mean(win) + mean(list(range(0, t + 1)))
    got1 = orc.bruteforce(q, k, v, w, 1.0, sel=[t], merge=1)[0, 0, 0]
    got2 = orc.bruteforce(q, k, v, w, 1.0, sel=[t], merge=2)[0, 0, 0]
    assert abs(got1 - want1) <= 1e-12 * max(1.0, abs(want1))
    assert abs(got2 - want2) <= 1e-12 * max(1.0, abs(want2))


@pytest.mark.parametrize("merge", [1, 2])
@pytest.mark.parametrize("w", [0, 1, 3, 16, 64])
@pytest.mark.parametrize("chunks", [(97,), (16, 16, 65), (1, 50, 3, 43)])
def test_stateful_forms_match_bruteforce(merge, w, chunks):
    H, Hkv, d = 4, 2, 8
    T = sum(chunks)
    q, k, v = rand_qkv(T, H, Hkv, d, 300 + w + merge, amp=1.5)
    scale = 0.4
    ref = orc.bruteforce(q, k, v, w, scale, merge=merge)
    pre = orc.Cell(H, Hkv, d, w, scale, merge=merge)
    dec = orc.Cell(H, Hkv, d, w, scale, merge=merge)
    pos = 0
    for c in chunks:
        np.testing.assert_allclose(pre.prefill(q[pos:pos + c], k[pos:pos + c], v[pos:pos + c]), ref[pos:pos + c],
                                   rtol=1e-10, atol=1e-12)
        pos += c
    for t in range(T):
        np.testing.assert_allclose(dec.decode(q[t], k[t], v[t]), ref[t], rtol=1e-10, atol=1e-12)
    assert pre.info() == dec.info()
    np.testing.assert_array_equal(pre.slot_tokens(), dec.slot_tokens())
    for a, b in zip(pre.export(), dec.export()):
        np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-14)


def test_all_token_state_holds_every_token():
    # merge = 2: S, z are sums over ALL tokens so far, whatever the window
    H, Hkv, d, w, T = 2, 2, 4, 5, 23
    q, k, v = rand_qkv(T, H, Hkv, d, 11)
    cell = orc.Cell(H, Hkv, d, w, 0.5, merge=2)
    for t in range(T):
        cell.decode(q[t], k[t], v[t])
    _, _, S, z = cell.export()
    fk = torch.softmax(torch.from_numpy(k), dim=-1).numpy()          # [T][Hkv][d]
    np.testing.assert_allclose(z, fk.sum(0), rtol=1e-12)
    np.testing.assert_allclose(S, np.einsum("tgr,tgc->grc", fk, v), rtol=1e-12)
