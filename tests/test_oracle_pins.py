"""Pins of the float64 oracle against what the paper and the mathematics fix.

Every check here compares the oracle with something that is NOT the oracle:
published known-answer vectors, closed forms, exhaustive enumeration, textbook
dense attention in numpy, the three-stage form of Alg. 1 carried out with numpy
gathers, and central finite differences.  CPU only.
"""
import itertools
import math
import os

import numpy as np
import pytest

import oracle
from oracle import CAUSAL, LINEAR_WINDOW, SWA_ONE_SIDED

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
TOL = 1e-12


def band_of(n, w):
    h = (w + 1) // 2 - 1
    return min(n, 2 * h + 1)


def rand_perm(rng, B, n):
    perm = np.stack([rng.permutation(n) for _ in range(B)]).astype(np.int32)
    inv = np.empty_like(perm)
    for b in range(B):
        inv[b, perm[b]] = np.arange(n, dtype=np.int32)
    return perm, inv


def qkv(rng, B, Hq, Hkv, n, d):
    return (rng.standard_normal((B, Hq, n, d)), rng.standard_normal((B, Hkv, n, d)),
            rng.standard_normal((B, Hkv, n, d)))


# ------------------------------------------------------------- numpy textbook

def np_dense_attention(q, k, v, mask, scale):
    """Textbook softmax attention of one head with a boolean mask [n,n]."""
    s = (q @ k.T) * scale
    s = np.where(mask, s, -np.inf)
    m = s.max(axis=1, keepdims=True)
    e = np.exp(s - m)
    l = e.sum(axis=1, keepdims=True)
    return (e / l) @ v, (m + np.log(l))[:, 0]


def np_mask_eq3(inv, n, w, causal, circular=True):
    """Eq. 3 / Eq. 4 mask written with numpy broadcasting (tokens x tokens)."""
    s = np.asarray(inv, dtype=np.int64)
    dist = np.abs(s[:, None] - s[None, :])
    if circular:
        dist = np.minimum(dist, n - dist)
    m = dist < w / 2.0          # the printed strict inequality, in real numbers
    if causal:
        tok = np.arange(n)
        m &= tok[None, :] <= tok[:, None]
    return m


def np_all_heads(q, k, v, masks, scale):
    B, Hq, n, d = q.shape
    G = Hq // k.shape[1]
    y = np.empty_like(q)
    lse = np.empty((B, Hq, n))
    for b in range(B):
        for h in range(Hq):
            y[b, h], lse[b, h] = np_dense_attention(q[b, h], k[b, h // G], v[b, h // G],
                                                    masks[b], scale)
    return y, lse


# --------------------------------------------------------------------- Philox

def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        t = [int(x, 16) for x in r]
        assert oracle.philox4x32_10(t[:4], t[4:6]) == t[6:]


def test_sort_key_is_first_two_philox_words():
    seed = 0x0123456789ABCDEF
    out = oracle.philox4x32_10([77, 3, 9, 0], [seed & 0xFFFFFFFF, seed >> 32])
    assert oracle.sort_key(seed, 9, 3, 77) == (out[0] << 32) | out[1]


# ---------------------------------------------------------------- permutation

@pytest.mark.parametrize("B,n", [(1, 1), (3, 2), (2, 27), (4, 1000), (1, 131072)])
def test_perm_is_bijection_sorted_by_key(B, n):
    perm, inv = oracle.make_perm(11, 5, B, n)
    ar = np.arange(n)
    for b in range(B):
        assert np.array_equal(np.sort(perm[b]), ar)
        assert np.array_equal(inv[b][perm[b]], ar)      # inverse after permute = identity
        assert np.array_equal(perm[b][inv[b]], ar)
    if n <= 1000:
        for b in range(B):
            keys = [oracle.sort_key(11, 5, b, int(t)) for t in perm[b]]
            assert all((keys[p], perm[b][p]) < (keys[p + 1], perm[b][p + 1])
                       for p in range(n - 1))


def test_perm_depends_on_seed_layer_and_sequence():
    a, _ = oracle.make_perm(1, 0, 2, 64)
    b, _ = oracle.make_perm(2, 0, 2, 64)
    c, _ = oracle.make_perm(1, 1, 2, 64)
    assert not np.array_equal(a, b) and not np.array_equal(a, c)
    assert not np.array_equal(a[0], a[1])
    a2, _ = oracle.make_perm(1, 0, 2, 64)
    assert np.array_equal(a, a2)                          # pure function of its arguments


def test_perm_uniform_over_s4_and_mean_slot():
    # 120000 independent sequences of n=4: all 24 orders within 5 sigma of equal share
    B = 120000
    perm, inv = oracle.make_perm(2024, 0, B, 4)
    code = perm[:, 0] * 64 + perm[:, 1] * 16 + perm[:, 2] * 4 + perm[:, 3]
    _, counts = np.unique(code, return_counts=True)
    assert len(counts) == 24
    p = 1 / 24
    sd = math.sqrt(B * p * (1 - p))
    assert np.all(np.abs(counts - B * p) < 5 * sd)
    # E[sigma(i)] = (n-1)/2 for every token
    n = 64
    _, inv = oracle.make_perm(7, 3, 20000, n)
    mean = inv.mean(axis=0)
    sd_mean = math.sqrt((n * n - 1) / 12 / 20000)
    assert np.all(np.abs(mean - (n - 1) / 2) < 5 * sd_mean)


# ----------------------------------------------------------------------- mask

@pytest.mark.parametrize("n,w", [(27, 8), (64, 1), (64, 2), (64, 7), (50, 50), (50, 51), (9, 40)])
def test_mask_counts_closed_form(n, w):
    rng = np.random.default_rng(n * 100 + w)
    perm, inv = rand_perm(rng, 3, n)
    band = band_of(n, w)
    nnz, rc, _ = oracle.coverage(perm, inv, w, 0, 0)
    assert np.all(rc == band) and np.all(nnz == n * band)
    # causal: the mask is symmetric with a unit diagonal, so exactly half of the
    # off-diagonal entries survive, for EVERY permutation
    nnz_c, rc_c, _ = oracle.coverage(perm, inv, w, CAUSAL, 0)
    assert np.all(nnz_c == n + n * (band - 1) // 2)
    assert np.all(rc_c >= 1) and np.all(rc_c <= band)


@pytest.mark.parametrize("n,w", [(5, 3), (6, 3), (6, 4), (7, 5)])
def test_connection_probability_prop1_exhaustive(n, w):
    # Prop. 1: over all n! permutations Pr[j in N(i)] = (band-1)/(n-1) exactly
    band = band_of(n, w)
    hits = np.zeros((n, n), np.int64)
    total = 0
    for sigma in itertools.permutations(range(n)):
        inv = np.array(sigma, np.int32)
        total += 1
        for i in range(n):
            for j in range(n):
                hits[i, j] += oracle.visible(n, w, 0, inv, i, j)
    for i in range(n):
        for j in range(n):
            if i == j:
                assert hits[i, j] == total
            else:
                assert hits[i, j] * (n - 1) == total * (band - 1)


def test_mask_matches_eq3_broadcast_form():
    rng = np.random.default_rng(5)
    for n, w in [(27, 8), (32, 9), (16, 64)]:
        _, inv = rand_perm(rng, 1, n)
        for flags, causal, circ in [(0, False, True), (CAUSAL, True, True),
                                    (LINEAR_WINDOW, False, False),
                                    (CAUSAL | LINEAR_WINDOW, True, False)]:
            m = np_mask_eq3(inv[0], n, w, causal, circ)
            got = np.array([[oracle.visible(n, w, flags, inv[0], i, j) for j in range(n)]
                            for i in range(n)])
            assert np.array_equal(got, m)


def test_one_sided_swa_predicate():
    n, w = 20, 6
    for i in range(n):
        for j in range(n):
            assert oracle.swa_visible(n, w, CAUSAL | SWA_ONE_SIDED, i, j) == (0 <= i - j <= w - 1)


# -------------------------------------------------------------------- forward

def test_identity_permutation_is_swa():
    # stage 1 and 3 of Sec. 3.3 are no-ops for the identity: compare with a
    # contiguous-window loop written directly from Eq. 1
    rng = np.random.default_rng(0)
    B, Hq, Hkv, n, d, w = 2, 4, 2, 40, 8, 9
    q, k, v = qkv(rng, B, Hq, Hkv, n, d)
    ident = np.tile(np.arange(n, dtype=np.int32), (B, 1))
    h = (w + 1) // 2 - 1
    for flags in (0, CAUSAL):
        y, lse = oracle.sa_forward(q, k, v, ident, ident, w, flags)
        ys, lses = oracle.swa_forward(q, k, v, w, flags)
        ref = np.empty_like(q)
        for b in range(B):
            for hq in range(Hq):
                hk = hq // (Hq // Hkv)
                for i in range(n):
                    js = sorted({(i + o) % n for o in range(-h, h + 1)})
                    if flags & CAUSAL:
                        js = [j for j in js if j <= i]
                    s = np.array([q[b, hq, i] @ k[b, hk, j] for j in js]) / math.sqrt(d)
                    a = np.exp(s - s.max())
                    a /= a.sum()
                    ref[b, hq, i] = sum(a[t] * v[b, hk, j] for t, j in enumerate(js))
        assert np.abs(y - ref).max() < TOL
        assert np.abs(ys - ref).max() < TOL and np.abs(lse - lses).max() < TOL


@pytest.mark.parametrize("causal", [False, True])
def test_wide_window_is_full_attention(causal):
    rng = np.random.default_rng(1)
    B, Hq, Hkv, n, d = 1, 2, 1, 33, 16
    q, k, v = qkv(rng, B, Hq, Hkv, n, d)
    perm, inv = rand_perm(rng, B, n)
    mask = np.tril(np.ones((n, n), bool)) if causal else np.ones((n, n), bool)
    ref, ref_lse = np_all_heads(q, k, v, [mask], 1 / math.sqrt(d))
    y, lse = oracle.sa_forward(q, k, v, perm, inv, 2 * n, CAUSAL if causal else 0)
    assert np.abs(y - ref).max() < TOL and np.abs(lse - ref_lse).max() < TOL
    if causal:   # one-sided SWA with w >= n is dense causal attention too
        y1, _ = oracle.swa_forward(q, k, v, n, CAUSAL | SWA_ONE_SIDED)
        assert np.abs(y1 - ref).max() < TOL


def test_even_w_equal_n_excludes_antipode():
    # printed inequality |.|_n < w/2 with w = n even leaves out the slot at distance n/2
    n = 8
    _, rc, _ = oracle.coverage(np.arange(n, dtype=np.int32)[None], None, n, 0, 0)
    assert np.all(rc == n - 1)


@pytest.mark.parametrize("flags", [0, CAUSAL, LINEAR_WINDOW, CAUSAL | LINEAR_WINDOW])
@pytest.mark.parametrize("n,w", [(27, 8), (64, 9), (96, 33), (31, 31), (12, 100)])
def test_slot_walk_equals_dense_eq4(flags, n, w):
    rng = np.random.default_rng(n + w + flags)
    B, Hq, Hkv, d = 2, 4, 2, 8
    q, k, v = qkv(rng, B, Hq, Hkv, n, d)
    perm, inv = rand_perm(rng, B, n)
    y, lse = oracle.sa_forward(q, k, v, perm, inv, w, flags)
    yd, lsed = oracle.sa_forward_dense(q, k, v, perm, inv, w, flags)
    assert np.abs(y - yd).max() < TOL and np.abs(lse - lsed).max() < TOL
    masks = [np_mask_eq3(inv[b], n, w, bool(flags & CAUSAL), not flags & LINEAR_WINDOW)
             for b in range(B)]
    ref, ref_lse = np_all_heads(q, k, v, masks, 1 / math.sqrt(d))
    assert np.abs(y - ref).max() < TOL and np.abs(lse - ref_lse).max() < TOL


def test_three_stage_form_of_alg1():
    # Alg. 1: gather rows by sigma, symmetric SWA in the permuted order, gather by sigma^-1
    rng = np.random.default_rng(3)
    B, Hq, Hkv, n, d, w = 2, 2, 2, 48, 8, 11
    q, k, v = qkv(rng, B, Hq, Hkv, n, d)
    perm, inv = rand_perm(rng, B, n)
    y, _ = oracle.sa_forward(q, k, v, perm, inv, w, 0)
    band_mask = np_mask_eq3(np.arange(n), n, w, False)      # plain circulant band
    for b in range(B):
        qp, kp, vp = q[b][:, perm[b]], k[b][:, perm[b]], v[b][:, perm[b]]
        yt, _ = np_all_heads(qp[None], kp[None], vp[None], [band_mask], 1 / math.sqrt(d))
        assert np.abs(yt[0][:, inv[b]] - y[b]).max() < TOL


def test_gqa_uses_contiguous_head_groups():
    rng = np.random.default_rng(4)
    B, Hq, Hkv, n, d, w = 1, 6, 2, 24, 4, 7
    q, k, v = qkv(rng, B, Hq, Hkv, n, d)
    perm, inv = rand_perm(rng, B, n)
    y, _ = oracle.sa_forward(q, k, v, perm, inv, w, CAUSAL)
    kk, vv = np.repeat(k, Hq // Hkv, axis=1), np.repeat(v, Hq // Hkv, axis=1)
    y2, _ = oracle.sa_forward(q, kk, vv, perm, inv, w, CAUSAL)
    assert np.abs(y - y2).max() < TOL


def test_uniform_attention_limit_norm_bound_and_w1():
    rng = np.random.default_rng(6)
    B, Hq, Hkv, n, d, w = 1, 1, 1, 30, 5, 9
    q, k, v = qkv(rng, B, Hq, Hkv, n, d)
    perm, inv = rand_perm(rng, B, n)
    # Q = 0: every visible key gets the same weight -> mean of the visible V rows
    y, lse = oracle.sa_forward(np.zeros_like(q), k, v, perm, inv, w, CAUSAL)
    m = np_mask_eq3(inv[0], n, w, True)
    for i in range(n):
        assert np.abs(y[0, 0, i] - v[0, 0][m[i]].mean(axis=0)).max() < TOL
        assert abs(lse[0, 0, i] - math.log(m[i].sum())) < TOL
    # convex combination: ||Y_i|| <= max ||V_j||
    y, _ = oracle.sa_forward(q, k, v, perm, inv, w, 0)
    assert np.linalg.norm(y, axis=-1).max() <= np.linalg.norm(v, axis=-1).max() + TOL
    # w = 1: only the token itself is visible
    y, lse = oracle.sa_forward(q, k, v, perm, inv, 1, CAUSAL)
    assert np.abs(y - v).max() < TOL
    assert np.abs(lse[0, 0] - (q[0, 0] * k[0, 0]).sum(-1) / math.sqrt(d)).max() < TOL


def test_softmax_scale_argument():
    rng = np.random.default_rng(8)
    q, k, v = qkv(rng, 1, 1, 1, 16, 4)
    perm, inv = rand_perm(rng, 1, 16)
    y1, _ = oracle.sa_forward(q, k, v, perm, inv, 5, 0, scale=0.37)
    y2, _ = oracle.sa_forward(q * 0.37 * 2.0, k, v, perm, inv, 5, 0)   # default 1/sqrt(4)
    assert np.abs(y1 - y2).max() < TOL


def test_one_sided_swa_textbook():
    rng = np.random.default_rng(9)
    B, Hq, Hkv, n, d, w = 1, 2, 1, 37, 8, 6
    q, k, v = qkv(rng, B, Hq, Hkv, n, d)
    tok = np.arange(n)
    back = tok[:, None] - tok[None, :]
    mask = (back >= 0) & (back <= w - 1)
    ref, ref_lse = np_all_heads(q, k, v, [mask], 1 / math.sqrt(d))
    y, lse = oracle.swa_forward(q, k, v, w, CAUSAL | SWA_ONE_SIDED)
    yd, _ = oracle.swa_forward_dense(q, k, v, w, CAUSAL | SWA_ONE_SIDED)
    assert np.abs(y - ref).max() < TOL and np.abs(lse - ref_lse).max() < TOL
    assert np.abs(yd - ref).max() < TOL


# ----------------------------------------------------------------------- gate

def test_gate_limits_and_midpoint():
    rng = np.random.default_rng(10)
    B, Hq, Hkv, n, d, w = 1, 2, 1, 20, 4, 5
    q, k, v = qkv(rng, B, Hq, Hkv, n, d)
    perm, inv = rand_perm(rng, B, n)
    fl = CAUSAL | SWA_ONE_SIDED
    ysa, _ = oracle.sa_forward(q, k, v, perm, inv, w, fl)
    yswa, _ = oracle.swa_forward(q, k, v, w, fl)
    big = 50.0
    y = oracle.gated_forward(q, k, v, perm, inv, np.array([[big, big], [-big, -big]]), w, fl)[0]
    assert np.abs(y - ysa).max() < 1e-12
    y = oracle.gated_forward(q, k, v, perm, inv, np.array([[-big, -big], [big, big]]), w, fl)[0]
    assert np.abs(y - yswa).max() < 1e-12
    out = oracle.gated_forward(q, k, v, perm, inv, np.zeros((2, Hq)), w, fl)
    assert np.abs(out[0] - 0.5 * (ysa + yswa)).max() < TOL
    assert np.abs(out[1] - ysa).max() < TOL and np.abs(out[2] - yswa).max() < TOL
    # independent sigmoids: head 0 and head 1 get their own pair of gates
    lg = np.array([[0.3, -1.2], [2.0, 0.4]])
    y = oracle.gated_forward(q, k, v, perm, inv, lg, w, fl)[0]
    sig = 1 / (1 + np.exp(-lg))
    for h in range(Hq):
        assert np.abs(y[:, h] - (sig[0, h] * ysa[:, h] + sig[1, h] * yswa[:, h])).max() < TOL


# ------------------------------------------------------------------- backward

@pytest.mark.parametrize("gated", [False, True])
@pytest.mark.parametrize("flags", [0, CAUSAL | SWA_ONE_SIDED])
def test_backward_matches_finite_differences(gated, flags):
    rng = np.random.default_rng(12 + gated + flags)
    B, Hq, Hkv, n, d, w = 2, 4, 2, 12, 4, 5
    q, k, v = qkv(rng, B, Hq, Hkv, n, d)
    dy = rng.standard_normal(q.shape)
    perm, inv = rand_perm(rng, B, n)
    lg = rng.standard_normal((2, Hq)) if gated else None

    def f(q_, k_, v_, lg_):
        if gated:
            return oracle.gated_forward(q_, k_, v_, perm, inv, lg_, w, flags)[0]
        return oracle.sa_forward(q_, k_, v_, perm, inv, w, flags)[0]

    dq, dk, dv, dg = oracle.backward(q, k, v, perm, inv, lg, dy, w, flags)
    eps = 1e-6
    args = [q, k, v] + ([lg] if gated else [])
    grads = [dq, dk, dv] + ([dg] if gated else [])
    full = args if gated else args + [None]
    for a_idx, (a, g) in enumerate(zip(args, grads)):
        flat = a.reshape(-1)
        picks = rng.choice(flat.size, size=min(flat.size, 40), replace=False)
        for e in picks:
            old = flat[e]
            flat[e] = old + eps
            lp = float((f(*full) * dy).sum())
            flat[e] = old - eps
            lm = float((f(*full) * dy).sum())
            flat[e] = old
            fd = (lp - lm) / (2 * eps)
            assert abs(fd - g.reshape(-1)[e]) <= 1e-7 * max(1.0, abs(fd)), (a_idx, e)


def test_backward_gqa_sums_group_and_equivariance():
    rng = np.random.default_rng(14)
    B, Hq, Hkv, n, d, w = 1, 4, 2, 16, 4, 7
    q, k, v = qkv(rng, B, Hq, Hkv, n, d)
    dy = rng.standard_normal(q.shape)
    perm, inv = rand_perm(rng, B, n)
    dq, dk, dv, _ = oracle.backward(q, k, v, perm, inv, None, dy, w, 0)
    # MHA with repeated K/V: group-summing its dk/dv must give the GQA gradients
    G = Hq // Hkv
    dq2, dk2, dv2, _ = oracle.backward(q, np.repeat(k, G, 1), np.repeat(v, G, 1), perm, inv,
                                       None, dy, w, 0)
    assert np.abs(dq - dq2).max() < TOL
    assert np.abs(dk - dk2.reshape(B, Hkv, G, n, d).sum(2)).max() < TOL
    assert np.abs(dv - dv2.reshape(B, Hkv, G, n, d).sum(2)).max() < TOL
    # equivariance (non-causal): gradients of SA = un-permuted gradients of SWA on permuted data
    ident = np.arange(n, dtype=np.int32)[None]
    p = perm[0]
    dq3, dk3, dv3, _ = oracle.backward(q[:, :, p], k[:, :, p], v[:, :, p], ident, ident, None,
                                       dy[:, :, p], w, 0)
    assert np.abs(dq3[:, :, inv[0]] - dq).max() < TOL
    assert np.abs(dk3[:, :, inv[0]] - dk).max() < TOL
    assert np.abs(dv3[:, :, inv[0]] - dv).max() < TOL


# ------------------------------------------------------- selected-row variants

ROW_CASES = [
    # B, Hq, Hkv, n, d, w, flags
    (2, 4, 2, 37, 8, 9, CAUSAL | SWA_ONE_SIDED),
    (1, 6, 3, 50, 4, 16, 0),
    (3, 2, 2, 24, 8, 64, CAUSAL),                 # window wider than the sequence
    (2, 4, 1, 41, 4, 7, CAUSAL | LINEAR_WINDOW | SWA_ONE_SIDED),
]


def np_branch_mask(swa, inv, n, w, flags):
    """Mask [query token, key token] of one branch, from the printed inequalities."""
    if swa and flags & SWA_ONE_SIDED:
        i = np.arange(n)
        back = i[:, None] - i[None, :]
        return (back >= 0) & (back <= w - 1)
    slots = np.arange(n) if swa else inv
    return np_mask_eq3(slots, n, w, bool(flags & CAUSAL), circular=not flags & LINEAR_WINDOW)


@pytest.mark.parametrize("case", ROW_CASES)
def test_forward_rows_equals_full_forward_on_every_row(case):
    """Every flat row index, in shuffled order, against the whole-tensor functions (bitwise)
    and against textbook dense attention written in numpy (independent of the oracle)."""
    B, Hq, Hkv, n, d, w, flags = case
    rng = np.random.default_rng(B * 100 + n)
    q, k, v = qkv(rng, B, Hq, Hkv, n, d)
    perm, inv = rand_perm(rng, B, n)
    rows = rng.permutation(B * Hq * n).astype(np.int64)
    G = Hq // Hkv
    scale = 1.0 / math.sqrt(d)
    for swa in (0, 1):
        full_y, full_lse = (oracle.swa_forward(q, k, v, w, flags) if swa
                            else oracle.sa_forward(q, k, v, perm, inv, w, flags))
        y, lse = oracle.forward_rows(swa, q, k, v, perm, inv, w, flags, rows)
        assert np.array_equal(y, full_y.reshape(-1, d)[rows])
        assert np.array_equal(lse, full_lse.reshape(-1)[rows])
        # the row decoding r -> (b, hq, i) and hq -> hk, against numpy dense attention
        for t in rng.choice(rows.size, size=25, replace=False):
            r = int(rows[t])
            i, hq, b = r % n, (r // n) % Hq, r // (n * Hq)
            mask = np_branch_mask(swa, inv[b], n, w, flags)
            ry, rl = np_dense_attention(q[b, hq], k[b, hq // G], v[b, hq // G], mask, scale)
            assert np.abs(y[t] - ry[i]).max() < TOL and abs(lse[t] - rl[i]) < TOL
    # duplicates and an empty request
    y, lse = oracle.forward_rows(0, q, k, v, perm, inv, w, flags, [5, 5, 0])
    assert np.array_equal(y[0], y[1]) and y.shape == (3, d)
    y, lse = oracle.forward_rows(0, q, k, v, perm, inv, w, flags, [])
    assert y.shape == (0, d) and lse.shape == (0,)


def np_dense_backward(q, k, v, inv, lg, dy, w, flags):
    """Textbook gradients of sum(dy*y) with dense n x n matrices, numpy only.
    P = softmax(mask(S)), dV = P^T dY, dS = P o (dY V^T - rowsum(dY o Y)), dQ = scale dS K,
    dK = scale dS^T Q; both branches through Eq. 5 when lg is given."""
    B, Hq, n, d = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    scale = 1.0 / math.sqrt(d)
    dq, dk, dv = np.zeros_like(q), np.zeros_like(k), np.zeros_like(v)
    for b in range(B):
        for hq in range(Hq):
            hk = hq // G
            for x in range(2 if lg is not None else 1):
                g = 1.0 if lg is None else 1.0 / (1.0 + math.exp(-lg[x, hq]))
                mask = np_branch_mask(x, inv[b], n, w, flags)
                s = np.where(mask, (q[b, hq] @ k[b, hk].T) * scale, -np.inf)
                p = np.exp(s - s.max(axis=1, keepdims=True))
                p /= p.sum(axis=1, keepdims=True)
                dyx = g * dy[b, hq]
                yx = p @ v[b, hk]
                ds = p * (dyx @ v[b, hk].T - (dyx * yx).sum(axis=1, keepdims=True))
                dv[b, hk] += p.T @ dyx
                dq[b, hq] += scale * ds @ k[b, hk]
                dk[b, hk] += scale * ds.T @ q[b, hq]
    return dq, dk, dv


@pytest.mark.parametrize("gated", [False, True])
@pytest.mark.parametrize("case", ROW_CASES)
def test_backward_rows_equals_full_backward_on_every_row(case, gated):
    B, Hq, Hkv, n, d, w, flags = case
    rng = np.random.default_rng(B * 100 + n + gated)
    q, k, v = qkv(rng, B, Hq, Hkv, n, d)
    dy = rng.standard_normal(q.shape)
    perm, inv = rand_perm(rng, B, n)
    lg = rng.standard_normal((2, Hq)) if gated else None
    dq, dk, dv, _ = oracle.backward(q, k, v, perm, inv, lg, dy, w, flags)
    # the whole-tensor backward itself against dense numpy matrices (not the oracle)
    ndq, ndk, ndv = np_dense_backward(q, k, v, inv, lg, dy, w, flags)
    for a, b_ in ((dq, ndq), (dk, ndk), (dv, ndv)):
        assert np.abs(a - b_).max() < 1e-11 * max(1.0, np.abs(b_).max())
    q_rows = rng.permutation(B * Hq * n).astype(np.int64)
    kv_rows = rng.permutation(B * Hkv * n).astype(np.int64)
    rdq, rdk, rdv = oracle.backward_rows(q, k, v, perm, inv, lg, dy, w, flags, q_rows, kv_rows)
    for got, want in ((rdq, ndq.reshape(-1, d)[q_rows]), (rdk, ndk.reshape(-1, d)[kv_rows]),
                      (rdv, ndv.reshape(-1, d)[kv_rows])):
        assert np.abs(got - want).max() < 1e-11 * max(1.0, np.abs(want).max())
    for got, want in ((rdq, dq.reshape(-1, d)[q_rows]), (rdk, dk.reshape(-1, d)[kv_rows]),
                      (rdv, dv.reshape(-1, d)[kv_rows])):
        assert np.abs(got - want).max() < 1e-12 * max(1.0, np.abs(want).max())
    # one list may be empty
    a, b_, c = oracle.backward_rows(q, k, v, perm, inv, lg, dy, w, flags, [3], [])
    assert a.shape == (1, d) and b_.shape == (0, d) and c.shape == (0, d)
    assert np.array_equal(a[0], rdq[list(q_rows).index(3)])


# ------------------------------------------------------------------- coverage

def test_swa_reach_closed_form():
    n, w, L = 200, 9, 30
    h = (w + 1) // 2 - 1
    ident = np.tile(np.arange(n, dtype=np.int32), (L, 1))
    _, _, reach = oracle.coverage(ident, ident, w, 0, 17)
    assert list(reach) == [min(n, 2 * (l + 1) * h + 1) for l in range(L)]
    _, _, reach2 = oracle.coverage(ident, None, w, 0, 17)
    assert np.array_equal(reach, reach2)


def test_sa_reach_growth_and_prop2_bound():
    n, w, L = 2048, 32, 6       # Fig. 2 (left) setting
    band = band_of(n, w)
    p = (band - 1) / (n - 1)
    seeds = 12
    sizes = np.zeros((seeds, L))
    for s in range(seeds):
        pl = [oracle.make_perm(1000 + s, l, 1, n) for l in range(L)]
        perm = np.concatenate([a for a, _ in pl])
        inv = np.concatenate([b for _, b in pl])
        nnz, rc, reach = oracle.coverage(perm, inv, w, 0, 5)
        assert reach[0] == band and np.all(np.diff(reach) >= 0) and reach[-1] == n
        assert np.all(rc == band)
        sizes[s] = reach
    mean = sizes.mean(axis=0)
    # Prop. 2: E|R_{l+1}| >= r + (n-r)(1-(1-p)^r), checked on the seed average with slack
    for l in range(L - 1):
        r = sizes[:, l]
        bound = (r + (n - r) * (1 - (1 - p) ** r)).mean()
        assert mean[l + 1] >= 0.97 * bound
    # full coverage in O(log_w n) layers: 4 = ceil(log(2048)/log(31)) + slack
    assert mean[3] > 0.99 * n


def test_fixed_sigma_reach_is_linear_like_swa():
    """Deterministic mode (Sec. 3.3: one fixed permutation reused at every layer): in slot
    space every layer is the same window, so the reachable set is an interval of slots that
    grows by 2h per layer, min(n, 2lh+1) tokens, exactly as for plain SWA; it is the fresh
    permutation per layer that gives the fast growth of Prop. 2."""
    n, w, L = 600, 17, 8
    h = (w + 1) // 2 - 1
    perm1, inv1 = oracle.make_perm(77, 0, 1, n)
    perm = np.repeat(perm1, L, axis=0)
    inv = np.repeat(inv1, L, axis=0)
    for src in (0, 250, n - 1):
        _, _, reach = oracle.coverage(perm, inv, w, 0, src)
        assert list(reach) == [min(n, 2 * (l + 1) * h + 1) for l in range(L)]
    # independent permutations from the same source spread much faster
    pl = [oracle.make_perm(77, l, 1, n) for l in range(L)]
    _, _, fresh = oracle.coverage(np.concatenate([a for a, _ in pl]),
                                  np.concatenate([b for _, b in pl]), w, 0, 250)
    assert fresh[2] > 4 * reach[2] and fresh[3] == n


def test_causal_reach_only_moves_backwards():
    n, w, L = 64, 9, 4
    pl = [oracle.make_perm(3, l, 1, n) for l in range(L)]
    perm = np.concatenate([a for a, _ in pl])
    inv = np.concatenate([b for _, b in pl])
    _, _, reach = oracle.coverage(perm, inv, w, CAUSAL, 0)
    assert list(reach) == [1] * L                      # token 0 sees only itself
    _, _, reach = oracle.coverage(perm, inv, w, CAUSAL, n - 1)
    assert np.all(np.diff(reach) >= 0) and reach[0] >= 1
