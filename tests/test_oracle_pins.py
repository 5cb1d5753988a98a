"""Pins for the CPU oracle: what the paper and the mathematics fix, not the oracle itself.

Each test ties one part of ``oracle/lisa_oracle.c`` to something outside it: a
library routine on a special case (torch's fp64 scaled_dot_product_attention),
a closed form, an invariant, or a brute-force scalar script written
independently in this file.  A dropped term, wrong sign, wrong scale, swapped
index or transposed weight in the oracle fails at least one of them.
"""
import math

import numpy as np
import pytest
import torch

import oracle
from oracle import ACT_NONE, ACT_RELU, ACT_SILU, INTEGRATE_ADD, INTEGRATE_CONCAT, INTEGRATE_PLUS, Link


def rnd(seed, *shape, std=1.0):
    return np.random.default_rng(seed).standard_normal(shape) * std


def sdpa(q, k, v, scale):
    """Textbook causal attention via torch (fp64, CPU). q [B,N,Hq,x], k [B,N,Hkv,x], v [B,N,Hkv,d]."""
    Hq, Hkv = q.shape[2], k.shape[2]
    tq = torch.from_numpy(q).permute(0, 2, 1, 3)
    tk = torch.from_numpy(k).permute(0, 2, 1, 3).repeat_interleave(Hq // Hkv, dim=1)
    tv = torch.from_numpy(v).permute(0, 2, 1, 3).repeat_interleave(Hq // Hkv, dim=1)
    o = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True, scale=scale)
    return o.permute(0, 2, 1, 3).contiguous().numpy()


def make_case(seed, B=2, N=9, Hq=4, Hkv=2, d=6, r=3, m=8, c=2, integrate=INTEGRATE_ADD, act=ACT_RELU, bias=True,
              ffn_layers=2):
    q0, k0, v = rnd(seed, B, N, Hq, d), rnd(seed + 1, B, N, Hkv, d), rnd(seed + 2, B, N, Hkv, d)
    links = []
    for k in range(c):
        s = seed + 10 * (k + 1)
        hin = 2 * Hq if integrate == INTEGRATE_CONCAT else Hq
        mm = Hq if ffn_layers == 1 else m
        links.append(Link(qp=rnd(s, B, N, Hq, r), kp=rnd(s + 1, B, N, Hkv, r), w1=rnd(s + 2, hin, mm, std=hin ** -0.5),
                          w2=rnd(s + 3, mm, Hq, std=mm ** -0.5) if ffn_layers == 2 else None,
                          b1=rnd(s + 4, mm) if bias else None, b2=rnd(s + 5, Hq) if (bias and ffn_layers == 2) else None,
                          r=r, act=act, integrate=integrate, ffn_layers=ffn_layers))
    return q0, k0, v, links


# ---------------------------------------------------------------------------
# Brute force, written independently with scalar Python (Eq. 1-4, Sec. 5.1).
# ---------------------------------------------------------------------------
def brute_force(q0, k0, v, links):
    B, N, Hq, d = q0.shape
    Hkv = k0.shape[2]
    grp = Hq // Hkv
    out = np.zeros((B, N, Hq, d))
    logits = np.zeros((B, Hq, N, N))
    for b in range(B):
        for i in range(N):
            per_key = []
            for j in range(i + 1):
                vec = [sum(q0[b, i, h, x] * k0[b, j, h // grp, x] for x in range(d)) / math.sqrt(d) for h in range(Hq)]
                for lk in links:
                    r = lk.r
                    dl = [sum(lk.qp[b, i, h, x] * lk.kp[b, j, h // grp, x] for x in range(r)) / math.sqrt(r)
                          for h in range(Hq)]
                    if lk.integrate == INTEGRATE_PLUS:
                        vec = [vec[h] + dl[h] for h in range(Hq)]
                        continue
                    inp = vec + dl if lk.integrate == INTEGRATE_CONCAT else vec
                    mm = lk.w1.shape[1]
                    hid = [sum(inp[x] * lk.w1[x, u] for x in range(len(inp))) + (lk.b1[u] if lk.b1 is not None else 0.0)
                           for u in range(mm)]
                    if lk.ffn_layers == 2:
                        if lk.act == ACT_RELU:
                            hid = [max(t, 0.0) for t in hid]
                        elif lk.act == ACT_SILU:
                            hid = [t / (1.0 + math.exp(-t)) for t in hid]
                        y = [sum(hid[u] * lk.w2[u, g] for u in range(mm)) + (lk.b2[g] if lk.b2 is not None else 0.0)
                             for g in range(Hq)]
                    else:
                        y = hid
                    vec = [y[h] + dl[h] for h in range(Hq)] if lk.integrate == INTEGRATE_ADD else y
                per_key.append(vec)
            for h in range(Hq):
                col = [per_key[j][h] for j in range(i + 1)]
                for j in range(i + 1):
                    logits[b, h, i, j] = col[j]
                mx = max(col)
                e = [math.exp(t - mx) for t in col]
                z = sum(e)
                for x in range(d):
                    out[b, i, h, x] = sum(e[j] / z * v[b, j, h // grp, x] for j in range(i + 1))
    return out, logits


@pytest.mark.parametrize("integrate,act,layers,bias", [
    (INTEGRATE_ADD, ACT_RELU, 2, True), (INTEGRATE_ADD, ACT_SILU, 2, False), (INTEGRATE_CONCAT, ACT_RELU, 2, True),
    (INTEGRATE_CONCAT, ACT_NONE, 1, True), (INTEGRATE_PLUS, ACT_NONE, 2, False), (INTEGRATE_ADD, ACT_NONE, 1, False)])
def test_brute_force_tiny(integrate, act, layers, bias):
    q0, k0, v, links = make_case(3, B=1, N=5, Hq=4, Hkv=2, d=3, r=2, m=6, c=2, integrate=integrate, act=act, bias=bias,
                                 ffn_layers=layers)
    O, A = oracle.prefill_full(q0, k0, v, links, want_scores=True)
    Ob, Ab = brute_force(q0, k0, v, links)
    np.testing.assert_allclose(O, Ob, rtol=0, atol=1e-12)
    tril = np.tril(np.ones((5, 5), dtype=bool))
    np.testing.assert_allclose(A[:, :, tril], Ab[:, :, tril], rtol=0, atol=1e-12)


# ---------------------------------------------------------------------------
# Invariants the paper fixes.
# ---------------------------------------------------------------------------
def test_softmax_rows_sum_to_one_and_causal_zeros():
    q0, k0, v, links = make_case(5, N=17)
    _, A, P = oracle.prefill_full(q0, k0, v, links, want_scores=True, want_probs=True)
    assert np.all(np.abs(P.sum(-1) - 1.0) < 1e-12)
    iu = np.triu_indices(17, k=1)
    assert np.all(P[:, :, iu[0], iu[1]] == 0.0)
    assert np.all(P >= 0.0)
    assert np.all(np.isfinite(A))  # shared scores stay finite above the diagonal: the mask comes after the chain


def test_chain_len_zero_is_textbook_attention_with_gqa():
    q0, k0, v, _ = make_case(7, B=2, N=11, Hq=6, Hkv=2, d=8)
    O = oracle.prefill_full(q0, k0, v, [])
    np.testing.assert_allclose(O, sdpa(q0, k0, v, 1.0 / math.sqrt(8)), rtol=0, atol=1e-12)


@pytest.mark.parametrize("act", [ACT_RELU, ACT_SILU])
def test_identity_aligner_zero_lowrank_is_direct_sharing(act):
    """W1=[I,-I], W2=[I;-I]: relu(x)-relu(-x)=x and silu(x)-silu(-x)=x, so with Q'=K'=0 the layer
    is attention with the anchor's scores and the current layer's V (the paper's direct sharing)."""
    B, N, Hq, Hkv, d, r = 2, 10, 4, 4, 5, 3
    q0, k0, v_anchor, _ = make_case(11, B=B, N=N, Hq=Hq, Hkv=Hkv, d=d)
    v_cur = rnd(99, B, N, Hkv, d)
    eye = np.eye(Hq)
    lk = Link(qp=np.zeros((B, N, Hq, r)), kp=np.zeros((B, N, Hkv, r)), w1=np.concatenate([eye, -eye], 1),
              w2=np.concatenate([eye, -eye], 0), r=r, act=act)
    O = oracle.prefill_full(q0, k0, v_cur, [lk, lk])
    np.testing.assert_allclose(O, sdpa(q0, k0, v_cur, 1.0 / math.sqrt(d)), rtol=0, atol=1e-12)


def test_zero_aligner_is_attention_on_lowrank_qk_with_sqrt_r():
    B, N, Hq, Hkv, d, r = 1, 12, 4, 2, 6, 5
    q0, k0, v, links = make_case(13, B=B, N=N, Hq=Hq, Hkv=Hkv, d=d, r=r, c=1, bias=False)
    links[0].w2 = np.zeros_like(links[0].w2)
    O = oracle.prefill_full(q0, k0, v, links)
    np.testing.assert_allclose(O, sdpa(links[0].qp, links[0].kp, v, 1.0 / math.sqrt(r)), rtol=0, atol=1e-12)


@pytest.mark.parametrize("perm", [[2, 1, 0], [1, 2, 0]])
def test_permutation_aligner(perm):
    """Sec. 5.1's example (h=3; 1->3, 2->2, 3->1) and a 3-cycle (which a transposed weight would fail):
    a one-layer FFN whose weight is a permutation matrix makes output head g use anchor head perm[g]'s scores."""
    B, N, Hq, d, r = 1, 8, 3, 4, 2
    q0, k0, v = rnd(1, B, N, Hq, d), rnd(2, B, N, Hq, d), rnd(3, B, N, Hq, d)
    w = np.zeros((Hq, Hq))
    for g in range(Hq):
        w[perm[g], g] = 1.0  # row = input head, column = output head
    lk = Link(qp=np.zeros((B, N, Hq, r)), kp=np.zeros((B, N, Hq, r)), w1=w, r=r, act=ACT_NONE, ffn_layers=1)
    O = oracle.prefill_full(q0, k0, v, [lk])
    ref = sdpa(q0[:, :, perm, :], k0[:, :, perm, :], v, 1.0 / math.sqrt(d))
    np.testing.assert_allclose(O, ref, rtol=0, atol=1e-12)


def test_softmax_shift_invariance():
    q0, k0, v, links = make_case(17, c=1)
    O1 = oracle.prefill_full(q0, k0, v, links)
    links[0].b2 = links[0].b2 + np.array([3.0, -2.0, 0.5, 7.0])  # per-head constant over j
    O2 = oracle.prefill_full(q0, k0, v, links)
    np.testing.assert_allclose(O1, O2, rtol=0, atol=1e-11)


def test_causality_future_positions_do_not_matter():
    q0, k0, v, links = make_case(19, N=12)
    O1 = oracle.prefill_full(q0, k0, v, links)
    cut = 7
    q0b, k0b, vb = q0.copy(), k0.copy(), v.copy()
    q0b[:, cut:] += 5.0
    k0b[:, cut:] -= 3.0
    vb[:, cut:] *= -2.0
    for lk in links:
        lk.qp = lk.qp.copy(); lk.kp = lk.kp.copy()
        lk.qp[:, cut:] += 1.0
        lk.kp[:, cut:] += 1.0
    O2 = oracle.prefill_full(q0b, k0b, vb, links)
    assert np.array_equal(O1[:, :cut], O2[:, :cut])


def test_linear_chain_closed_form():
    """With no activation the chain is linear: A_c = M2^T (M1^T A_0 + c1 + D1) + c2 + D2 with M_k = W1_k W2_k.
    Distinct links catch a mix-up of which link's weights apply where."""
    B, N, Hq, Hkv, d, r = 1, 7, 4, 2, 5, 3
    q0, k0, v, links = make_case(23, B=B, N=N, Hq=Hq, Hkv=Hkv, d=d, r=r, c=2, act=ACT_NONE)
    _, A = oracle.prefill_full(q0, k0, v, links, want_scores=True)
    grp = Hq // Hkv
    A0 = np.einsum("bihx,bjhx->bhij", q0, np.repeat(k0, grp, axis=2)) / math.sqrt(d)
    cur = A0
    for lk in links:
        D = np.einsum("bihx,bjhx->bhij", lk.qp, np.repeat(lk.kp, grp, axis=2)) / math.sqrt(r)
        M = lk.w1 @ lk.w2                      # [h_in, h_out]
        const = lk.b1 @ lk.w2 + lk.b2          # [h_out]
        cur = np.einsum("bhij,hg->bgij", cur, M) + const[None, :, None, None] + D
    np.testing.assert_allclose(A, cur, rtol=0, atol=1e-11)


def test_concat_reduces_to_add_free_form():
    """CONCAT with the A_Delta half of W1 zeroed ignores Q'/K'; with the A_{n-1} half zeroed it ignores the anchor.
    Fixes the order [A_{n-1}; A_Delta] of the concatenation."""
    B, N, Hq, Hkv, d, r, m = 1, 6, 4, 4, 3, 2, 8
    q0, k0, v, links = make_case(29, B=B, N=N, Hq=Hq, Hkv=Hkv, d=d, r=r, m=m, c=1, integrate=INTEGRATE_CONCAT)
    lk = links[0]
    w_full = lk.w1.copy()
    lk.w1 = w_full.copy(); lk.w1[Hq:] = 0.0
    _, A_top = oracle.prefill_full(q0, k0, v, [lk], want_scores=True)
    add_like = Link(qp=np.zeros_like(lk.qp), kp=np.zeros_like(lk.kp), w1=w_full[:Hq], w2=lk.w2, b1=lk.b1, b2=lk.b2, r=r,
                    act=lk.act, integrate=INTEGRATE_ADD)
    _, A_ref = oracle.prefill_full(q0, k0, v, [add_like], want_scores=True)
    np.testing.assert_allclose(A_top, A_ref, rtol=0, atol=1e-12)
    lk.w1 = w_full.copy(); lk.w1[:Hq] = 0.0
    _, A_bot = oracle.prefill_full(q0, k0, v, [lk], want_scores=True)
    _, A_bot2 = oracle.prefill_full(q0 * 0 + 1.0, k0 * 3.0, v, [lk], want_scores=True)
    np.testing.assert_allclose(A_bot, A_bot2, rtol=0, atol=1e-12)


@pytest.mark.parametrize("act,fn", [(ACT_SILU, torch.nn.functional.silu), (ACT_RELU, torch.nn.functional.relu)])
def test_activation_against_torch(act, fn):
    """The oracle's activation through link_apply against torch's fp64 silu / relu (a library routine, not the formula
    retyped): with W1 = I (m = h), W2 = I and zero Q'/K', Eq. 4 (ADD) reduces to A_out = act(A_in + b1) element by element.
    Values span both signs and the range where SiLU is far from linear."""
    B, N, Hq = 1, 5, 6
    A_in = rnd(61, B, Hq, N, N, std=3.0)
    b1 = rnd(62, Hq)
    eye = np.eye(Hq)
    lk = Link(qp=np.zeros((B, N, Hq, 2)), kp=np.zeros((B, N, Hq, 2)), w1=eye, w2=eye, b1=b1, b2=None, r=2, act=act)
    got = oracle.link_apply(A_in, lk, Hkv=Hq)
    want = fn(torch.from_numpy(A_in + b1[None, :, None, None])).numpy()
    np.testing.assert_allclose(got, want, rtol=0, atol=1e-13)
    assert np.abs(want - (A_in + b1[None, :, None, None])).max() > 1.0     # the activation is not the identity on this data


def test_rows_mode_equals_full_mode():
    q0, k0, v, links = make_case(31, B=2, N=13, c=3)
    O, A = oracle.prefill_full(q0, k0, v, links, want_scores=True)
    rb = np.array([0, 1, 1, 0, 1]); ri = np.array([0, 12, 5, 7, 0])
    Or, Ar = oracle.prefill_rows(q0, k0, v, links, rb, ri, want_scores=True)
    for t in range(len(rb)):
        np.testing.assert_allclose(Or[t], O[rb[t], ri[t]], rtol=0, atol=1e-13)
        n = ri[t] + 1
        np.testing.assert_allclose(Ar[t][:, :n], A[rb[t], :, ri[t], :n], rtol=0, atol=1e-13)
        assert np.all(Ar[t][:, n:] == 0.0)


def test_rows_mode_against_sdpa_at_larger_size():
    """A size that spans many keys: chain of identity links keeps the textbook result."""
    B, N, Hq, Hkv, d, r = 1, 200, 4, 2, 16, 4
    q0, k0, v = rnd(1, B, N, Hq, d), rnd(2, B, N, Hkv, d), rnd(3, B, N, Hkv, d)
    eye = np.eye(Hq)
    lk = Link(qp=np.zeros((B, N, Hq, r)), kp=np.zeros((B, N, Hkv, r)), w1=np.concatenate([eye, -eye], 1),
              w2=np.concatenate([eye, -eye], 0), r=r, act=ACT_SILU)
    rows = np.arange(0, N, 7)
    Or = oracle.prefill_rows(q0, k0, v, [lk], np.zeros_like(rows), rows)
    ref = sdpa(q0, k0, v, 1.0 / math.sqrt(d))
    np.testing.assert_allclose(Or, ref[0, rows], rtol=0, atol=1e-12)


def test_prefill_decode_equivalence():
    """Decode at context t+1, fed row t of the previous layer's scores, reproduces prefill row t
    (both the output and the emitted score row): Sec. 5.2's two stages compute the same layer."""
    B, N, Hq, Hkv, d, r = 2, 10, 4, 2, 6, 3
    q0, k0, v, links = make_case(37, B=B, N=N, Hq=Hq, Hkv=Hkv, d=d, r=r, c=2)
    _, A1 = oracle.prefill_full(q0, k0, v, links[:1], want_scores=True)
    O2, A2 = oracle.prefill_full(q0, k0, v, links, want_scores=True)
    lens = np.array([N, 6], dtype=np.int32)
    prev = np.zeros((B, Hq, N))
    qp = np.zeros((B, Hq, r))
    for b in range(B):
        t = lens[b] - 1
        prev[b, :, :lens[b]] = A1[b, :, t, :lens[b]]
        qp[b] = links[1].qp[b, t]
    O, row = oracle.decode_shared(prev, qp, links[1].kp, v, links[1], lens)
    for b in range(B):
        t = lens[b] - 1
        np.testing.assert_allclose(O[b], O2[b, t], rtol=0, atol=1e-12)
        np.testing.assert_allclose(row[b, :, :lens[b]], A2[b, :, t, :lens[b]], rtol=0, atol=1e-12)
        assert np.all(row[b, :, lens[b]:] == 0.0)


def test_decode_anchor_is_last_row_of_textbook_attention():
    B, N, Hq, Hkv, d = 2, 14, 6, 3, 8
    q0, k0, v = rnd(41, B, N, Hq, d), rnd(42, B, N, Hkv, d), rnd(43, B, N, Hkv, d)
    lens = np.array([N, 9], dtype=np.int32)
    q = np.stack([q0[b, lens[b] - 1] for b in range(B)])
    O, row = oracle.decode_anchor(q, k0, v, lens)
    ref = sdpa(q0, k0, v, 1.0 / math.sqrt(d))
    A = oracle.scores(q0, k0)
    for b in range(B):
        t = lens[b] - 1
        np.testing.assert_allclose(O[b], ref[b, t], rtol=0, atol=1e-12)
        np.testing.assert_allclose(row[b, :, :lens[b]], A[b, :, t, :lens[b]], rtol=0, atol=1e-13)


def test_scores_match_einsum_and_head_grouping():
    q, k = rnd(51, 2, 5, 8, 4), rnd(52, 2, 5, 2, 4)
    A = oracle.scores(q, k)
    ref = np.einsum("bihx,bjhx->bhij", q, np.repeat(k, 4, axis=2)) / 2.0
    np.testing.assert_allclose(A, ref, rtol=0, atol=1e-13)


def test_memory_model_closed_forms():
    """Sec. 5.2: LLaMA2-7B-like numbers. 21 shared layers, h=32, d_k=128, r=20: prefill saving turns negative
    once l > |S|(d_k - r) = 2268; decode saving is always positive."""
    S, h, dk, r = 21, 32, 128, 20
    pre, dec = oracle.memory_saving(S, h, 2048, dk, r)
    assert pre == h * 2048 * (S * (dk - r) - 2048) * 2 and pre > 0
    assert dec == h * 2048 * (S * (dk - r) - 1) * 2
    pre_long, dec_long = oracle.memory_saving(S, h, 4096, dk, r)
    assert pre_long < 0 < dec_long
    assert oracle.memory_saving(S, h, S * (dk - r), dk, r)[0] == 0


def test_projection_is_a_plain_matrix_product():
    """oracle.project against numpy's matmul (a library routine) and a scalar loop, on shapes where every dimension differs
    (a transposed operand or swapped index fails), and the column blocks of [W_Q | W_K | W_V] against separate products
    (Eq. 1: the per-head H W^V_i are column blocks; Eq. 3: H W_LR)."""
    x = rnd(71, 2, 5, 7)
    w = rnd(72, 7, 11)
    got = oracle.project(x, w)
    np.testing.assert_allclose(got, x @ w, rtol=0, atol=1e-13)
    slow = np.zeros((2, 5, 11))
    for b in range(2):
        for n in range(5):
            for j in range(11):
                slow[b, n, j] = sum(x[b, n, k] * w[k, j] for k in range(7))
    np.testing.assert_allclose(got, slow, rtol=0, atol=1e-13)
    wq, wk, wv = w[:, :3], w[:, 3:5], w[:, 5:]
    np.testing.assert_allclose(got[..., 3:5], oracle.project(x, np.ascontiguousarray(wk)), rtol=0, atol=1e-13)
    np.testing.assert_allclose(got[..., 5:], x @ wv, rtol=0, atol=1e-13)
    # the low-rank difference built from projected operands equals Eq. 3 written out: (H W_Q)(H W_K)^T / sqrt(r)
    h = rnd(73, 1, 4, 7)
    q, k = oracle.project(h, np.ascontiguousarray(wq)), oracle.project(h, np.ascontiguousarray(wq))
    A = oracle.scores(q.reshape(1, 4, 1, 3), k.reshape(1, 4, 1, 3))
    np.testing.assert_allclose(A[0, 0], (h[0] @ wq) @ (h[0] @ wq).T / math.sqrt(3), rtol=0, atol=1e-12)
