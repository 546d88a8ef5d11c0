"""Pins of the fp64 oracle against things other than itself (CPU only).

Each check compares the oracle with an independent statement of the same quantity:
a hand-worked example, a dense N x N brute-force form written with numpy matrix
products, a library routine (torch SDPA, torch elu), a closed form, or an invariant
that a dropped term / wrong sign / wrong index / transposed operand would break.
"""
import json
import math
import os

import numpy as np
import pytest
import torch

import oracle

HERE = os.path.dirname(os.path.abspath(__file__))


def rnd(shape, seed, scale=1.0):
    return np.random.default_rng(seed).standard_normal(shape) * scale


# ----------------------------------------------------------------------------- brute force
def brute_window(q, k, v, w, scale):
    """Full N x N logits, explicit band mask (-inf outside i-w < j <= i), row softmax."""
    B, H, N, d = q.shape
    i = np.arange(N)[:, None]
    j = np.arange(N)[None, :]
    allowed = (j <= i) & (j > i - w)
    out = np.empty_like(q)
    for b in range(B):
        for h in range(H):
            logits = (q[b, h] @ k[b, h].T) * scale
            logits = np.where(allowed, logits, -np.inf)
            logits = logits - logits.max(axis=1, keepdims=True)
            p = np.exp(logits)
            p = p / p.sum(axis=1, keepdims=True)
            out[b, h] = p @ v[b, h]
    return out


def np_phi(x):
    return np.where(x > 0, x + 1.0, np.exp(np.minimum(x, 0.0)))


def brute_linear(q, k, v):
    """Quadratic masked form ((phi(Q) phi(K)^T) * M) V / rowsum."""
    B, H, N, d = q.shape
    M = np.tril(np.ones((N, N)))
    out = np.empty_like(q)
    for b in range(B):
        for h in range(H):
            A = (np_phi(q[b, h]) @ np_phi(k[b, h]).T) * M
            out[b, h] = (A @ v[b, h]) / A.sum(axis=1, keepdims=True)
    return out


# ----------------------------------------------------------------------------- golden
def _golden():
    with open(os.path.join(HERE, "golden", "hand_worked.json")) as f:
        return json.load(f)


def test_golden_window_hand_worked():
    g = _golden()["window"]
    q = np.array(g["q"])[None, None]
    k = np.log(np.array(g["k_log_of"]))[None, None]
    v = np.array(g["v"])[None, None]
    for w, exp in g["expected"].items():
        o = oracle.window_attn(q, k, v, int(w), scale=g["scale"])
        np.testing.assert_allclose(o[0, 0], np.array(exp), rtol=0, atol=1e-14)


def test_golden_linear_hand_worked():
    g = _golden()["linear"]
    fix = lambda rows: np.array([[(-math.log(2.0) if x == "-ln2" else x) for x in r] for r in rows])
    q, k, v = fix(g["q"])[None, None], fix(g["k"])[None, None], fix(g["v"])[None, None]
    S = np.zeros((1, 1, 2, 2))
    z = np.zeros((1, 1, 2))
    o = oracle.causal_linear_attn(q, k, v, S, z)
    np.testing.assert_allclose(o[0, 0], np.array(g["expected"]), atol=1e-14)
    np.testing.assert_allclose(S[0, 0], np.array(g["expected_S"]), atol=1e-14)
    np.testing.assert_allclose(z[0, 0], np.array(g["expected_z"]), atol=1e-14)


# ----------------------------------------------------------------------------- phi
def test_phi_matches_library_elu_plus_one():
    x = np.concatenate([np.linspace(-30, 30, 2001), [0.0, -0.0, 1e-300, -1e-300]])
    ref = (torch.nn.functional.elu(torch.from_numpy(x)) + 1.0).numpy()
    # the library forms (exp(x) - 1) + 1, which carries one rounding at magnitude 1
    np.testing.assert_allclose(oracle.phi(x), ref, rtol=1e-15, atol=2.3e-16)


def test_phi_properties():
    assert oracle.phi(np.array([0.0]))[0] == 1.0
    x = np.linspace(-20, 20, 4001)
    y = oracle.phi(x)
    assert (y > 0).all()
    assert (np.diff(y) > 0).all()
    np.testing.assert_allclose(y[x > 0], x[x > 0] + 1.0, rtol=1e-15)
    np.testing.assert_allclose(y[x <= 0], np.exp(x[x <= 0]), rtol=1e-15)


# ----------------------------------------------------------------------------- window
@pytest.mark.parametrize("N,d", [(1, 4), (7, 3), (33, 8), (64, 16)])
def test_window_equals_bruteforce_band_mask_all_w(N, d):
    q, k, v = rnd((2, 2, N, d), 1), rnd((2, 2, N, d), 2), rnd((2, 2, N, d), 3)
    for w in range(1, N + 3):
        o = oracle.window_attn(q, k, v, w, scale=0.37)
        np.testing.assert_allclose(o, brute_window(q, k, v, w, 0.37), rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("w", [48, 49, 1000])
def test_window_ge_N_is_full_causal_attention_library(w):
    N, d = 48, 16
    q, k, v = rnd((2, 3, N, d), 4), rnd((2, 3, N, d), 5), rnd((2, 3, N, d), 6)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v), is_causal=True).numpy()
    o = oracle.window_attn(q, k, v, w)  # default scale 1/sqrt(d), same as the library's
    np.testing.assert_allclose(o, ref, rtol=1e-12, atol=1e-13)


def test_window_banded_matches_library_with_explicit_mask():
    N, d, w = 40, 8, 7
    q, k, v = rnd((1, 2, N, d), 7), rnd((1, 2, N, d), 8), rnd((1, 2, N, d), 9)
    i = torch.arange(N)[:, None]
    j = torch.arange(N)[None, :]
    mask = (j <= i) & (j > i - w)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v), attn_mask=mask).numpy()
    np.testing.assert_allclose(oracle.window_attn(q, k, v, w), ref, rtol=1e-12, atol=1e-13)


def test_window_one_returns_values():
    q, k, v = rnd((1, 2, 19, 5), 10), rnd((1, 2, 19, 5), 11), rnd((1, 2, 19, 5), 12)
    assert np.array_equal(oracle.window_attn(q, k, v, 1), v)


@pytest.mark.parametrize("zero", ["q", "k", "scale"])
def test_window_uniform_logits_give_sliding_mean(zero):
    N, d, w = 37, 6, 5
    q, k, v = rnd((1, 1, N, d), 13), rnd((1, 1, N, d), 14), rnd((1, 1, N, d), 15)
    scale = None
    if zero == "q":
        q = np.zeros_like(q)
    elif zero == "k":
        k = np.zeros_like(k)
    else:
        scale = 0.0
    o = oracle.window_attn(q, k, v, w, scale=scale)
    for i in range(N):
        lo = max(0, i - w + 1)
        np.testing.assert_allclose(o[0, 0, i], v[0, 0, lo:i + 1].mean(axis=0), rtol=1e-13, atol=1e-14)


def test_window_constant_values_and_key_shift_invariance():
    N, d, w = 50, 8, 9
    q, k, v = rnd((1, 2, N, d), 16), rnd((1, 2, N, d), 17), rnd((1, 2, N, d), 18)
    c = rnd((d,), 19)
    vc = np.broadcast_to(c, v.shape).copy()
    np.testing.assert_allclose(oracle.window_attn(q, k, vc, w), vc, rtol=1e-13)
    u = rnd((d,), 20)
    np.testing.assert_allclose(oracle.window_attn(q, k + u, v, w), oracle.window_attn(q, k, v, w),
                               rtol=1e-10, atol=1e-12)


def test_window_row_depends_only_on_its_window():
    N, d, w = 40, 4, 6
    q, k, v = rnd((1, 1, N, d), 21), rnd((1, 1, N, d), 22), rnd((1, 1, N, d), 23)
    base = oracle.window_attn(q, k, v, w)
    i = 20
    for j in range(N):
        k2, v2 = k.copy(), v.copy()
        k2[0, 0, j] += 1.0
        v2[0, 0, j] -= 2.0
        changed = np.abs(oracle.window_attn(q, k2, v2, w)[0, 0, i] - base[0, 0, i]).max() > 1e-9
        assert changed == (i - w < j <= i), (i, j)


def test_window_needle_at_window_edge():
    # One key with a huge logit: visible to row i exactly while it is inside the window.
    N, d, w = 30, 4, 8
    q = np.zeros((1, 1, N, d)); q[..., 0] = 1.0
    k = np.zeros((1, 1, N, d)); k[0, 0, 5, 0] = 50.0
    v = rnd((1, 1, N, d), 24)
    o = oracle.window_attn(q, k, v, w, scale=1.0)
    for i in range(N):
        lo = max(0, i - w + 1)
        if lo <= 5 <= i:
            np.testing.assert_allclose(o[0, 0, i], v[0, 0, 5], atol=1e-12)
        else:
            np.testing.assert_allclose(o[0, 0, i], v[0, 0, lo:i + 1].mean(axis=0), atol=1e-12)


# ----------------------------------------------------------------------------- linear
@pytest.mark.parametrize("N,d", [(1, 3), (9, 2), (40, 8), (64, 16)])
def test_linear_prefix_sum_equals_quadratic_masked_form(N, d):
    q, k, v = rnd((2, 2, N, d), 30), rnd((2, 2, N, d), 31), rnd((2, 2, N, d), 32)
    np.testing.assert_allclose(oracle.causal_linear_attn(q, k, v), brute_linear(q, k, v),
                               rtol=1e-12, atol=1e-13)


def test_linear_first_row_is_first_value_and_K0_gives_cumulative_mean():
    N, d = 25, 5
    q, k, v = rnd((1, 2, N, d), 33), rnd((1, 2, N, d), 34), rnd((1, 2, N, d), 35)
    o = oracle.causal_linear_attn(q, k, v)
    np.testing.assert_allclose(o[:, :, 0], v[:, :, 0], rtol=1e-14)
    o = oracle.causal_linear_attn(q, np.zeros_like(k), v)  # phi(0) = 1 -> plain running mean
    cm = np.cumsum(v, axis=2) / np.arange(1, N + 1)[None, None, :, None]
    np.testing.assert_allclose(o, cm, rtol=1e-13, atol=1e-14)


def test_linear_constant_values_and_causality():
    N, d = 30, 6
    q, k, v = rnd((1, 1, N, d), 36), rnd((1, 1, N, d), 37), rnd((1, 1, N, d), 38)
    c = rnd((d,), 39)
    vc = np.broadcast_to(c, v.shape).copy()
    np.testing.assert_allclose(oracle.causal_linear_attn(q, k, vc), vc, rtol=1e-13)
    base = oracle.causal_linear_attn(q, k, v)
    i = 12
    for j in range(N):
        k2, v2 = k.copy(), v.copy()
        k2[0, 0, j] += 0.5
        v2[0, 0, j] += 1.0
        changed = np.abs(oracle.causal_linear_attn(q, k2, v2)[0, 0, i] - base[0, 0, i]).max() > 1e-9
        assert changed == (j <= i)


def test_linear_state_is_sum_of_outer_products_and_resumes():
    N, d = 21, 4
    q, k, v = rnd((1, 2, N, d), 40), rnd((1, 2, N, d), 41), rnd((1, 2, N, d), 42)
    S = np.zeros((1, 2, d, d)); z = np.zeros((1, 2, d))
    full = oracle.causal_linear_attn(q, k, v, S, z)
    for h in range(2):
        pk = np_phi(k[0, h])
        np.testing.assert_allclose(S[0, h], pk.T @ v[0, h], rtol=1e-13)  # S[a][c] = sum_i phi(k_i)[a] v_i[c]
        np.testing.assert_allclose(z[0, h], pk.sum(axis=0), rtol=1e-13)
    # Splitting the sequence and carrying (S, z) gives the same rows.
    S2 = np.zeros_like(S); z2 = np.zeros_like(z)
    a = oracle.causal_linear_attn(q[:, :, :8], k[:, :, :8], v[:, :, :8], S2, z2)
    b = oracle.causal_linear_attn(q[:, :, 8:], k[:, :, 8:], v[:, :, 8:], S2, z2)
    np.testing.assert_allclose(np.concatenate([a, b], axis=2), full, rtol=1e-12)
    np.testing.assert_allclose(S2, S, rtol=1e-13)


def test_linear_differs_from_contract_before_cumsum_order():
    # Contracting with phi(q_j) before the cumulative sum (the order in which the paper's
    # PyTorch listing is printed) is a different, non-attention quantity; Algorithm 1 wins.
    N, d = 12, 3
    q, k, v = rnd((1, 1, N, d), 43), rnd((1, 1, N, d), 44), rnd((1, 1, N, d), 45)
    pq, pk = np_phi(q[0, 0]), np_phi(k[0, 0])
    num = np.cumsum(np.einsum("na,na,nc->nc", pq, pk, v[0, 0]), axis=0)
    den = np.cumsum(np.einsum("na,na->n", pq, pk), axis=0)[:, None]
    printed = num / den
    o = oracle.causal_linear_attn(q, k, v)[0, 0]
    assert np.abs(printed - o).max() > 1e-3
    # ... while cumsum-then-contract is Algorithm 1 exactly.
    A = np.cumsum(np.einsum("na,nc->nac", pk, v[0, 0]), axis=0)
    Z = np.cumsum(pk, axis=0)
    np.testing.assert_allclose(np.einsum("na,nac->nc", pq, A) / np.einsum("na,na->n", pq, Z)[:, None],
                               o, rtol=1e-12)


# ----------------------------------------------------------------------------- hybrid
def test_default_head_split():
    assert [oracle.default_h_sparse(H) for H in (2, 12, 16, 32)] == [1, 2, 3, 6]


@pytest.mark.parametrize("h0", [0, 1, 2, 4])
def test_hybrid_is_headwise_merge(h0):
    B, H, N, d, w = 2, 4, 23, 8, 5
    q, k, v = rnd((B, H, N, d), 50), rnd((B, H, N, d), 51), rnd((B, H, N, d), 52)
    o = oracle.hybrid_attn(q, k, v, w, h_sparse=h0)
    if h0 > 0:
        np.testing.assert_array_equal(o[:, :h0], oracle.window_attn(q[:, :h0], k[:, :h0], v[:, :h0], w))
        np.testing.assert_allclose(o[:, :h0], brute_window(q[:, :h0], k[:, :h0], v[:, :h0], w, d ** -0.5),
                                   rtol=1e-12, atol=1e-13)
    if h0 < H:
        np.testing.assert_array_equal(o[:, h0:], oracle.causal_linear_attn(q[:, h0:], k[:, h0:], v[:, h0:]))
        np.testing.assert_allclose(o[:, h0:], brute_linear(q[:, h0:], k[:, h0:], v[:, h0:]),
                                   rtol=1e-12, atol=1e-13)


# ----------------------------------------------------------------------------- decode
@pytest.mark.parametrize("w", [1, 4, 16, 40])
def test_decode_token_by_token_equals_full_sequence_rows(w):
    B, H, N, d, h0 = 2, 3, 33, 4, 1
    q, k, v = rnd((B, H, N, d), 60), rnd((B, H, N, d), 61), rnd((B, H, N, d), 62)
    full_w = brute_window(q[:, :h0], k[:, :h0], v[:, :h0], w, d ** -0.5)
    full_l = brute_linear(q[:, h0:], k[:, h0:], v[:, h0:])
    st = oracle.DecodeState(B, H, d, w, h0)
    for t in range(N):
        o = oracle.decode_step(q[:, :, t], k[:, :, t], v[:, :, t], st)
        np.testing.assert_allclose(o[:, :h0], full_w[:, :, t], rtol=1e-11, atol=1e-12)
        np.testing.assert_allclose(o[:, h0:], full_l[:, :, t], rtol=1e-11, atol=1e-12)
    assert st.t == N


@pytest.mark.parametrize("N0,w", [(5, 8), (8, 8), (21, 8), (30, 7)])
def test_prefill_export_then_decode_equals_one_long_sequence(N0, w):
    B, H, d, h0, steps = 1, 4, 4, 2, 13
    N = N0 + steps
    q, k, v = rnd((B, H, N, d), 63), rnd((B, H, N, d), 64), rnd((B, H, N, d), 65)
    ref = np.concatenate([brute_window(q[:, :h0], k[:, :h0], v[:, :h0], w, d ** -0.5),
                          brute_linear(q[:, h0:], k[:, h0:], v[:, h0:])], axis=1)
    o, st = oracle.hybrid_attn(q[:, :, :N0], k[:, :, :N0], v[:, :, :N0], w, h_sparse=h0, export_state=True)
    np.testing.assert_allclose(o, ref[:, :, :N0], rtol=1e-11, atol=1e-12)
    assert st.t == N0
    # ring placement: token j sits in slot j mod w
    for j in range(max(0, N0 - w), N0):
        np.testing.assert_array_equal(st.k_cache[:, :, j % w], k[:, :h0, j])
        np.testing.assert_array_equal(st.v_cache[:, :, j % w], v[:, :h0, j])
    for t in range(N0, N):
        o = oracle.decode_step(q[:, :, t], k[:, :, t], v[:, :, t], st)
        np.testing.assert_allclose(o, ref[:, :, t], rtol=1e-11, atol=1e-12)


# ----------------------------------------------------------------------------- "self" (bidirectional) layer
# The bidirectional layer's oracle functions and what fixes them.
def test_self_window_covering_the_sequence_is_library_softmax_attention():
    q, k, v = rnd((2, 2, 37, 16), 501), rnd((2, 2, 37, 16), 502), rnd((2, 2, 37, 16), 503)
    for w in (37, 38, 500):  # |i - j| < w holds for every pair: plain Eq. 1, no mask
        got = oracle.window_attn_self(q, k, v, w)
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v)).numpy()
        np.testing.assert_allclose(got, ref, rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("N,w", [(1, 1), (9, 1), (9, 2), (23, 5), (40, 17), (40, 39)])
def test_self_window_equals_library_attention_with_an_explicit_band_mask(N, w):
    q, k, v = rnd((1, 3, N, 8), 510 + N), rnd((1, 3, N, 8), 511 + N), rnd((1, 3, N, 8), 512 + N)
    i = torch.arange(N)[:, None]
    j = torch.arange(N)[None, :]
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v), attn_mask=(i - j).abs() < w).numpy()
    np.testing.assert_allclose(oracle.window_attn_self(q, k, v, w), ref, rtol=1e-11, atol=1e-12)


def test_self_window_mirror_symmetry_and_relation_to_the_causal_window():
    q, k, v = rnd((1, 2, 50, 8), 520), rnd((1, 2, 50, 8), 521), rnd((1, 2, 50, 8), 522)
    w = 7
    fwd = oracle.window_attn_self(q, k, v, w)
    rev = oracle.window_attn_self(q[:, :, ::-1], k[:, :, ::-1], v[:, :, ::-1], w)
    np.testing.assert_allclose(rev[:, :, ::-1], fwd, rtol=1e-12, atol=1e-13)  # the rule has no direction
    # the last row has nothing to its right: it is the causal window's last row
    np.testing.assert_allclose(fwd[:, :, -1], oracle.window_attn(q, k, v, w)[:, :, -1], rtol=1e-12, atol=1e-13)
    # w = 1: every token sees only itself
    np.testing.assert_allclose(oracle.window_attn_self(q, k, v, 1), v, rtol=0, atol=1e-15)
    # a needle w - 1 to the right is seen, one at distance w is not
    qn = np.zeros((1, 1, 30, 4)); kn = np.zeros((1, 1, 30, 4)); vn = np.zeros((1, 1, 30, 4))
    qn[0, 0, 10, 0] = 30.0; kn[0, 0, 16, 0] = 30.0; vn[0, 0, 16, :] = 1.0
    assert oracle.window_attn_self(qn, kn, vn, 7, scale=1.0)[0, 0, 10, 0] > 0.99
    assert oracle.window_attn_self(qn, kn, vn, 6, scale=1.0)[0, 0, 10, 0] == 0.0


def test_self_linear_equals_the_quadratic_unmasked_form_and_the_causal_last_row():
    q, k, v = rnd((2, 2, 33, 8), 530), rnd((2, 2, 33, 8), 531), rnd((2, 2, 33, 8), 532)
    got = oracle.linear_attn_self(q, k, v)
    # (phi(Q) phi(K)^T) V with rows normalised: the N x N attention matrix written out
    A = np.einsum("bhia,bhja->bhij", np_phi(q), np_phi(k))
    ref = np.einsum("bhij,bhjc->bhic", A / A.sum(axis=-1, keepdims=True), v)
    np.testing.assert_allclose(got, ref, rtol=1e-11, atol=1e-12)
    # the last token of Algorithm 1 has seen every key: same row
    np.testing.assert_allclose(got[:, :, -1], oracle.causal_linear_attn(q, k, v)[:, :, -1], rtol=1e-11, atol=1e-12)
    # the keys form a set: permuting (k_j, v_j) pairs changes nothing; permuting queries permutes rows
    perm = np.random.default_rng(5).permutation(33)
    np.testing.assert_allclose(oracle.linear_attn_self(q, k[:, :, perm], v[:, :, perm]), got, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(oracle.linear_attn_self(q[:, :, perm], k, v), got[:, :, perm], rtol=1e-11, atol=1e-12)
    # rows are convex combinations of the values (phi > 0): constant values come back, outputs stay in range
    np.testing.assert_allclose(oracle.linear_attn_self(q, k, np.full_like(v, 2.5)), 2.5, rtol=1e-12)
    assert (got <= v.max(axis=2, keepdims=True) + 1e-12).all() and (got >= v.min(axis=2, keepdims=True) - 1e-12).all()


def test_self_hybrid_routes_heads_like_the_causal_layer():
    q, k, v = rnd((2, 5, 21, 8), 540), rnd((2, 5, 21, 8), 541), rnd((2, 5, 21, 8), 542)
    o = oracle.hybrid_attn_self(q, k, v, 4, h_sparse=2)
    np.testing.assert_array_equal(o[:, :2], oracle.window_attn_self(q[:, :2], k[:, :2], v[:, :2], 4))
    np.testing.assert_array_equal(o[:, 2:], oracle.linear_attn_self(q[:, 2:], k[:, 2:], v[:, 2:]))
    assert oracle.hybrid_attn_self(q, k, v, 4).shape == q.shape  # default split: max(1, round(3 H / 16)) = 1
    np.testing.assert_array_equal(oracle.hybrid_attn_self(q, k, v, 4)[:, 1:], oracle.linear_attn_self(q[:, 1:], k[:, 1:], v[:, 1:]))


# ----------------------------------------------------------------------------- head partition (Algorithm 2)
def test_partition_balance_hand_worked_and_invariants():
    from oracle import partition as op

    # equal cost and speed: half each.  Engine 0 needs twice the work per unit at the same speed:
    # 2 p = 1 - p, p' = 1/3.  Engine 1 three times faster on equal work: p = (1 - p) / 3, p' = 1/4.
    assert op.balance(100, 7.0, 7.0, 2.0, 2.0) == pytest.approx(0.5, abs=1e-14)
    assert op.balance(64, 2.0, 1.0, 1.0, 1.0) == pytest.approx(1.0 / 3.0, abs=1e-14)
    assert op.balance(64, 1.0, 1.0, 1.0, 3.0) == pytest.approx(0.25, abs=1e-14)
    rng = np.random.default_rng(11)
    for _ in range(50):
        f0, f1, p0, p1 = (float(x) for x in 10.0 ** rng.uniform(-1, 1, 4))  # shares stay away from 0 and 1
        size = float(rng.integers(1, 10**6))
        p = op.balance(size, f0, f1, p0, p1)
        l0, l1 = op.latencies(p, size, f0, f1, p0, p1)
        assert 0.0 < p < 1.0 and l0 == pytest.approx(l1, rel=1e-9)
        # the work is conserved: both shares together are the whole problem
        assert p * size + (1 - p) * size == pytest.approx(size, rel=1e-15)
        # naming the engines the other way round mirrors the split; the problem size and a common
        # speed-up of both engines do not move it
        assert op.balance(size, f1, f0, p1, p0) == pytest.approx(1.0 - p, abs=1e-12)
        assert op.balance(3 * size, f0, f1, 5 * p0, 5 * p1) == pytest.approx(p, abs=1e-12)
        # a faster engine 0 gets more
        assert op.balance(size, f0, f1, 2 * p0, p1) > p


def test_partition_latency_step_values():
    from oracle import partition as op

    # p = 0.25 of 8 units at 3 flops each on a 2 flop/s engine: 0.25 * 8 * 3 / 2 = 3 s;
    # the other 6 units at 5 flops each on a 10 flop/s engine: 6 * 5 / 10 = 3 s
    assert op.latencies(0.25, 8, 3.0, 5.0, 2.0, 10.0) == (3.0, 3.0)
    assert op.balance(8, 3.0, 5.0, 2.0, 10.0) == pytest.approx(0.25, abs=1e-14)


def test_partition_heads_hand_worked_and_brackets_the_crossing():
    from oracle import partition as op

    # B = N = E = W = 1, unit speeds, H = 4: linear 8 (4 - h)^2 = 128, 72, 32, 8, 0 against sparse
    # 5 h = 0, 5, 10, 15, 20: gaps 128, 67, 22, 7, 20 -> 3 sparse heads
    assert [op.model_latencies(1, 4, 1, 1, 1, h, 1.0, 1.0) for h in range(5)] == [
        (0.0, 128.0), (5.0, 72.0), (10.0, 32.0), (15.0, 8.0), (20.0, 0.0)]
    assert op.partition_heads(1, 4, 1, 1, 1, 1.0, 1.0) == 3
    # the three terms of the linear model (feature maps 4, K^T V 2, Q C 2) add up to the printed 8
    B, H, N, E, W = 2, 16, 1024, 64, 256
    h1e2 = float((H - 3) * E) ** 2
    assert op.model_latencies(B, H, N, E, W, 3, 1.0, 1.0)[1] == (4 + 2 + 2) * B * N * h1e2
    rng = np.random.default_rng(12)
    for _ in range(40):
        H = int(rng.integers(1, 65)); E = int(rng.choice([32, 64, 128])); W = int(rng.choice([64, 256, 1024]))
        ps, pl = (float(x) for x in 10.0 ** rng.uniform(9, 15, 2))
        h0 = op.partition_heads(B, H, N, E, W, ps, pl)
        gap = lambda h: op.model_latencies(B, H, N, E, W, h, ps, pl)[0] - op.model_latencies(B, H, N, E, W, h, ps, pl)[1]
        # sparse - linear grows with the sparse head count, from negative (no sparse head) to positive
        # (no linear head): the chosen count sits at the sign change
        assert gap(0) < 0 < gap(H)
        assert all(gap(h) < gap(h + 1) for h in range(H))
        if h0 > 0:
            assert gap(h0 - 1) < 0
        if h0 < H:
            assert gap(h0 + 1) > 0
        # B and N scale both estimates alike; a faster sparse engine never gets fewer heads
        assert op.partition_heads(7 * B, H, 3 * N, E, W, ps, pl) == h0
        assert op.partition_heads(B, H, N, E, W, 4 * ps, pl) >= h0


def test_partition_printed_example_is_not_what_the_printed_model_gives():
    """Sec. IV-C reports 3 sparse heads of 16 (4k tokens, 13.37 and 2.31 TFLOP/s).  The printed
    formulas with those rates balance far from it whatever the window, so the example is no pin;
    this records the fact rather than bending the model to it."""
    from oracle import partition as op

    counts = [op.partition_heads(1, 16, 4096, 64, W, 2.31e12, 13.37e12) for W in (16, 32, 64, 128, 256, 512, 1024)]
    assert counts == [16, 16, 15, 15, 14, 14, 13]


# ----------------------------------------------------------------------------- positive random features
# (Sec. III-A / III-C: the feature map the linear heads use; formula of the cited Performer paper)
def _num(x):
    if isinstance(x, str):
        return {"0.5+ln2": 0.5 + math.log(2.0), "0.5+ln3": 0.5 + math.log(3.0)}[x]
    return float(x)


def _favor_golden():
    with open(os.path.join(HERE, "golden", "hand_worked.json")) as f:
        g = json.load(f)["favor"]
    W = np.array([[[_num(x) for x in row] for row in m] for m in g["W"]])
    return g, W


def test_favor_features_hand_worked():
    g, W = _favor_golden()
    got = oracle.phi_favor(np.array(g["x"]), W[0]) * math.sqrt(2.0)
    np.testing.assert_allclose(got, np.array(g["phi_times_sqrt2"]), rtol=1e-14)


def test_favor_linear_attention_hand_worked():
    g, W = _favor_golden()
    k, v = np.array(g["k"])[None, None], np.array(g["v"])[None, None]
    for q, want in ((g["q_a"], g["expected_a"]), (g["q_b"], g["expected_b"])):
        S, z = np.zeros((1, 1, 2, 2)), np.zeros((1, 1, 2))
        o = oracle.causal_linear_attn(np.array(q)[None, None], k, v, S, z, W=W)
        np.testing.assert_allclose(o[0, 0], np.array(want), rtol=1e-13)
        np.testing.assert_allclose(S[0, 0] * math.sqrt(2.0), np.array(g["expected_S_times_sqrt2"]), rtol=1e-13)
        np.testing.assert_allclose(z[0, 0] * math.sqrt(2.0), np.array(g["expected_z_times_sqrt2"]), rtol=1e-13)


def test_favor_features_are_positive_and_fall_with_the_norm():
    W = rnd((8, 8), 601)
    x = rnd((50, 8), 602, 2.0)
    f = oracle.phi_favor(x, W)
    assert (f > 0).all()
    # a vector orthogonal to every projection direction only sees the -|x|^2/2 term: with W = 0 the
    # features are the Gaussian exp(-|x|^2/2)/sqrt(d), the same in every coordinate
    f0 = oracle.phi_favor(x, np.zeros((8, 8)))
    np.testing.assert_allclose(f0, np.repeat(np.exp(-0.5 * (x ** 2).sum(1, keepdims=True)) / math.sqrt(8.0), 8, 1), rtol=1e-13)


@pytest.mark.parametrize("orthogonal", [False, True])
def test_favor_features_estimate_the_softmax_kernel(orthogonal):
    # E_W[ phi_W(q) . phi_W(k) ] = exp(q . k) for Gaussian projection rows (each row on its own is N(0, I)
    # also in the orthogonal draw): the mean over many independent draws converges to the kernel.
    from paper_2412_19829_b200 import synth  # input generators only: no attention arithmetic in there

    d, draws = 4, 6000
    q, k = rnd((3, d), 611, 0.5), rnd((3, d), 612, 0.5)
    Ws = synth.favor_projection(draws, d, seed=613, orthogonal=orthogonal).double().numpy()
    est = np.zeros((3, 3))
    for W in Ws:
        est += oracle.phi_favor(q, W) @ oracle.phi_favor(k, W).T
    est /= draws
    want = np.exp(q @ k.T)
    # Monte-Carlo: relative standard error of the mean is a few per cent per draw^(1/2) ~ 1.3 %; five sigma
    np.testing.assert_allclose(est, want, rtol=0.08)
    if orthogonal:  # the draw really is orthogonal, with Gaussian-like row norms
        G = Ws[0] @ Ws[0].T
        assert np.abs(G - np.diag(np.diag(G))).max() < 1e-5 * np.diag(G).max()


def test_favor_with_zero_projection_weights_keys_by_their_gaussian():
    # W = 0: phi(k_j) = exp(-|k_j|^2/2)/sqrt(d) in every coordinate, so row i is the mean of v_0..v_i
    # weighted by exp(-|k_j|^2/2); keys of equal norm give the plain cumulative mean
    B, H, N, d = 1, 2, 9, 4
    q, k, v = rnd((B, H, N, d), 621), rnd((B, H, N, d), 622), rnd((B, H, N, d), 623)
    W0 = np.zeros((H, d, d))
    o = oracle.causal_linear_attn(q, k, v, W=W0)
    wts = np.exp(-0.5 * (k ** 2).sum(-1))  # [B, H, N]
    want = np.cumsum(wts[..., None] * v, axis=2) / np.cumsum(wts, axis=2)[..., None]
    np.testing.assert_allclose(o, want, rtol=1e-12)
    k1 = k / np.linalg.norm(k, axis=-1, keepdims=True)
    o1 = oracle.causal_linear_attn(q, k1, v, W=W0)
    np.testing.assert_allclose(o1, np.cumsum(v, axis=2) / np.arange(1, N + 1)[None, None, :, None], rtol=1e-12)


def test_favor_linear_attention_equals_the_masked_quadratic_form_and_its_variants_agree():
    B, H, N, d, w, h0 = 2, 3, 12, 4, 5, 1
    q, k, v = rnd((B, H, N, d), 631, 0.7), rnd((B, H, N, d), 632, 0.7), rnd((B, H, N, d), 633)
    W = rnd((H, d, d), 634)
    o = oracle.causal_linear_attn(q, k, v, W=W)
    for b in range(B):
        for h in range(H):
            fq, fk = oracle.phi_favor(q[b, h], W[h]), oracle.phi_favor(k[b, h], W[h])
            A = np.tril(fq @ fk.T)  # weights of key j for query i, j <= i
            np.testing.assert_allclose(o[b, h], (A @ v[b, h]) / A.sum(1, keepdims=True), rtol=1e-11)
            # the bidirectional layer's global form: no mask
            A2 = fq @ fk.T
            og = oracle.linear_attn_self(q[b:b + 1, h:h + 1], k[b:b + 1, h:h + 1], v[b:b + 1, h:h + 1], W=W[h:h + 1])
            np.testing.assert_allclose(og[0, 0], (A2 @ v[b, h]) / A2.sum(1, keepdims=True), rtol=1e-11)
    # a per-row factor of phi(q) cancels: the -|q|^2/2 term and the 1/sqrt(m) do not matter for q, so
    # moving q along a direction orthogonal to every projection row (here: W has rank < d) changes nothing
    Wr = W.copy()
    Wr[:, :, -1] = 0.0  # no projection row sees the last coordinate
    q2 = q.copy()
    q2[..., -1] += 3.0
    np.testing.assert_allclose(oracle.causal_linear_attn(q2, k, v, W=Wr), oracle.causal_linear_attn(q, k, v, W=Wr), rtol=1e-11)
    # hybrid routing and decoding carry the projection of the linear heads only
    ref, st = oracle.hybrid_attn(q[:, :, :8], k[:, :, :8], v[:, :, :8], w, h_sparse=h0, export_state=True, W=W[h0:])
    full = oracle.hybrid_attn(q, k, v, w, h_sparse=h0, W=W[h0:])
    np.testing.assert_allclose(ref, full[:, :, :8], rtol=1e-12)
    np.testing.assert_allclose(full[:, h0:], o[:, h0:], rtol=1e-12)
    for t in range(8, N):
        ot = oracle.decode_step(q[:, :, t], k[:, :, t], v[:, :, t], st)
        np.testing.assert_allclose(ot, full[:, :, t], rtol=1e-10, atol=1e-12)
