"""Pins for the CPU oracle: each oracle function is checked against something
other than itself -- closed forms, brute force on tiny inputs, invariants the
paper states, special cases that reduce to textbook or library routines, and a
hand-derived exact example.  CPU only."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(1234)


# ----------------------------------------------------------------------------
# independent brute force: dense causal softmax attention, Eq. 2, written as a
# masked matrix computation (not the oracle's row loops)
# ----------------------------------------------------------------------------
def dense_causal_probs(Q, K, scale=None, key_mask=None):
    L, Hq, d = Q.shape
    Hkv = K.shape[1]
    G = Hq // Hkv
    scale = 1.0 / math.sqrt(d) if scale is None else scale
    Kx = np.repeat(K.astype(np.float64), G, axis=1)               # [L,Hq,d]
    S = np.einsum("ihd,jhd->hij", Q.astype(np.float64), Kx) * scale
    mask = np.tril(np.ones((L, L), bool))
    if key_mask is not None:
        mask = mask & key_mask[None, :]
    S = np.where(mask[None], S, -np.inf)
    with np.errstate(invalid="ignore"):     # a row that sees no key at all comes out as NaN
        S = S - S.max(axis=-1, keepdims=True)
        E = np.exp(S)
        return E / E.sum(axis=-1, keepdims=True)                  # [Hq, L, L]


def dense_causal_attention(Q, K, V, scale=None, key_mask=None):
    A = dense_causal_probs(Q, K, scale, key_mask)
    G = Q.shape[1] // K.shape[1]
    Vx = np.repeat(V.astype(np.float64), G, axis=1)
    return np.einsum("hij,jhd->ihd", A, Vx)                       # [L,Hq,d]


def rand_qkv(L, Hq, Hkv, d):
    f = lambda h: rng.standard_normal((L, h, d)).astype(np.float32)
    return f(Hq), f(Hkv), f(Hkv)


# ----------------------------------------------------------------------------
# scores (Eq. A, Eq. 6)
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("L,Hq,Hkv,d", [(1, 1, 1, 4), (7, 2, 2, 8), (33, 4, 2, 16), (64, 6, 2, 8)])
def test_scores_all_probes_equal_dense_column_sums(L, Hq, Hkv, d):
    Q, K, _ = rand_qkv(L, Hq, Hkv, d)
    acc, S = oracle.probe_scores(Q, K, np.arange(L))
    ref = dense_causal_probs(Q, K).sum(axis=(0, 1))
    np.testing.assert_allclose(acc, ref, rtol=1e-12, atol=1e-14)
    assert abs(S - L * Hq) < 1e-9 * L * Hq


def test_scores_probe_subset_equals_selected_rows_of_dense():
    L, Hq, Hkv, d = 50, 4, 1, 8
    Q, K, _ = rand_qkv(L, Hq, Hkv, d)
    probe = np.array([3, 10, 11, 40, 49])
    acc, S = oracle.probe_scores(Q, K, probe)
    ref = dense_causal_probs(Q, K)[:, probe, :].sum(axis=(0, 1))
    np.testing.assert_allclose(acc, ref, rtol=1e-12, atol=1e-14)
    # row-softmax identity quoted under Eq. 7: total mass = rows x heads
    assert abs(S - len(probe) * Hq) < 1e-10
    # columns behind the causal mask of every probe are exactly zero
    L2 = 30
    Q, K, _ = rand_qkv(L2, 2, 2, 4)
    acc, _ = oracle.probe_scores(Q, K, np.array([5, 9]))
    assert np.all(acc[10:] == 0.0) and np.all(acc[:10] > 0.0)


def test_scores_custom_scale_is_applied():
    L, H, d = 12, 2, 8
    Q, K, _ = rand_qkv(L, H, H, d)
    acc, _ = oracle.probe_scores(Q, K, np.arange(L), scale=0.37)
    ref = dense_causal_probs(Q, K, scale=0.37).sum(axis=(0, 1))
    np.testing.assert_allclose(acc, ref, rtol=1e-12)


@pytest.mark.parametrize("L,Hq", [(1, 1), (5, 3), (40, 2)])
def test_scores_zero_keys_harmonic_closed_form(L, Hq):
    # K == 0 makes every causal row uniform: row c gives 1/(c+1) to columns 0..c,
    # so a_j = Hq * (H_L - H_j) with H_n the n-th harmonic number.
    Q = rng.standard_normal((L, Hq, 4)).astype(np.float32)
    K = np.zeros((L, Hq, 4), np.float32)
    acc, S = oracle.probe_scores(Q, K, np.arange(L))
    Hn = [Fraction(0)]
    for t in range(1, L + 1):
        Hn.append(Hn[-1] + Fraction(1, t))
    exact = [float(Hq * (Hn[L] - Hn[j])) for j in range(L)]
    np.testing.assert_allclose(acc, exact, rtol=1e-13)
    assert abs(S - L * Hq) < 1e-11 * max(1, L * Hq)


def test_scores_single_probe_is_one_attention_row():
    L, d = 21, 8
    Q, K, _ = rand_qkv(L, 1, 1, d)
    c = 13
    acc, _ = oracle.probe_scores(Q, K, np.array([c]))
    s = (K[: c + 1, 0].astype(np.float64) @ Q[c, 0].astype(np.float64)) / math.sqrt(d)
    w = np.exp(s - s.max())
    w /= w.sum()
    np.testing.assert_allclose(acc[: c + 1], w, rtol=1e-13)
    assert np.all(acc[c + 1:] == 0)


def test_scores_two_token_closed_form():
    # L = 2, d = 1: a_0 = 1 + sigmoid(scale*q1*(k0-k1)), a_1 = 1 - that sigmoid
    q0, q1, k0, k1 = 0.5, -1.25, 2.0, 0.75
    Q = np.array([[[q0]], [[q1]]], np.float32)
    K = np.array([[[k0]], [[k1]]], np.float32)
    acc, _ = oracle.probe_scores(Q, K, np.arange(2))
    sg = 1.0 / (1.0 + math.exp(-(q1 * (k0 - k1))))
    np.testing.assert_allclose(acc, [1 + sg, 1 - sg], rtol=1e-14)


def test_scores_gqa_head_mapping():
    # query head h must read kv head h // G: make kv heads wildly different
    L, Hq, Hkv, d = 16, 6, 3, 4
    Q, K, _ = rand_qkv(L, Hq, Hkv, d)
    K[:, 1] *= 5.0
    K[:, 2] *= 0.0
    acc, _ = oracle.probe_scores(Q, K, np.arange(L))
    ref = dense_causal_probs(Q, K).sum(axis=(0, 1))
    np.testing.assert_allclose(acc, ref, rtol=1e-12)


# ----------------------------------------------------------------------------
# normalisation (Eq. 8)
# ----------------------------------------------------------------------------
def test_normalise_nnz_closed_forms():
    L, Hq = 100, 4
    acc = rng.random(L) + 0.1
    norm, nnz = oracle.normalise(acc, np.arange(L), Hq)
    assert np.array_equal(nnz, L - np.arange(L))               # all rows probe: L - j
    np.testing.assert_allclose(norm * nnz * Hq, acc, rtol=1e-14)
    probe = np.arange(L - 64, L)
    norm, nnz = oracle.normalise(acc, probe, Hq)
    assert np.array_equal(nnz, np.minimum(64, L - np.arange(L)))
    np.testing.assert_allclose(norm, acc / (Hq * nnz), rtol=1e-15)
    # mixed probe list: count by definition
    probe = np.array([2, 50, 51, 99])
    _, nnz = oracle.normalise(acc, probe, Hq)
    assert nnz[0] == 4 and nnz[2] == 4 and nnz[3] == 3 and nnz[51] == 2 and nnz[52] == 1
    # a column no probe can see gets 0 (its accumulated score is 0 too)
    acc2 = acc.copy()
    acc2[60:] = 0
    norm, nnz = oracle.normalise(acc2, np.array([10, 59]), Hq)
    assert np.all(nnz[60:] == 0) and np.all(norm[60:] == 0)


# ----------------------------------------------------------------------------
# budget (Eq. 7)
# ----------------------------------------------------------------------------
def brute_budget(a, tau):
    L = len(a)
    if tau >= 1.0:
        return L
    s = sorted((Fraction(float(x)) for x in a), reverse=True)
    S = sum(s)
    target = Fraction(float(tau)) * S
    C = Fraction(0)
    for i, x in enumerate(s, 1):
        C += x
        if C >= target:
            return i
    return L


@pytest.mark.parametrize("L", [1, 2, 5, 16])
def test_budget_brute_force_tiny(L):
    for trial in range(40):
        a = rng.random(L) ** 3
        for tau in (0.05, 0.5, 0.9, 0.97, 0.999, 1.0):
            p, diag = oracle.budget(a, tau)
            bp = brute_budget(a, tau)
            # exact-rational brute force; allow a difference only when a prefix sum
            # sits within rounding of the target
            if p != bp:
                assert min(abs(diag["C_p"] - diag["target"]), abs(diag["C_prev"] - diag["target"])) \
                    < 1e-12 * diag["S"]
            assert 1 <= p <= L


def test_budget_minimality_invariant_and_monotone():
    a = rng.random(500) ** 4
    last = 0
    for tau in np.linspace(0.01, 0.999, 60):
        p, diag = oracle.budget(a, tau)
        srt = np.sort(a)[::-1]
        C = np.cumsum(srt)
        assert C[p - 1] >= tau * a.sum() * (1 - 1e-14)
        if p > 1:
            assert C[p - 2] < tau * a.sum() * (1 + 1e-14)
        assert p >= last
        last = p
        assert abs(diag["S"] - a.sum()) < 1e-10


def test_budget_one_hot_and_tau_one():
    a = np.full(64, 1e-4)
    a[17] = 10.0
    assert oracle.budget(a, 0.95)[0] == 1
    assert oracle.budget(a, 1.0)[0] == 64
    assert oracle.budget(np.ones(9), 1.0)[0] == 9
    # uniform scores: p = ceil(tau * L)
    assert oracle.budget(np.ones(10), 0.5)[0] == 5
    assert oracle.budget(np.ones(10), 0.51)[0] == 6
    # equal values do not change any prefix sum
    a = np.array([3.0, 1.0, 3.0, 1.0, 2.0])
    assert oracle.budget(a, 0.6)[0] == 2           # 3+3 = 6 >= 6.0
    assert oracle.budget(a, 0.61)[0] == 3


def test_budget_single_probe_is_nucleus_truncation():
    # with one probe row the accumulated score is one probability distribution and
    # Eq. 7 is textbook nucleus (top-p) truncation of it
    L, d = 64, 8
    Q, K, _ = rand_qkv(L, 1, 1, d)
    K *= 3
    acc, S = oracle.probe_scores(Q, K, np.array([L - 1]))
    for top_p in (0.3, 0.8, 0.95):
        p, _ = oracle.budget(acc, top_p)
        order = np.argsort(-acc, kind="stable")
        cum = np.cumsum(acc[order])
        nucleus = int(np.searchsorted(cum, top_p * cum[-1], side="left")) + 1
        assert p == nucleus


def test_budget_zero_keys_closed_form():
    # K == 0, all probes, one head: a_j = H_L - H_j is already descending, so
    # C_i = sum_{j<i} (H_L - H_j) and p follows from exact rationals.
    L = 30
    Q = rng.standard_normal((L, 1, 4)).astype(np.float32)
    acc, S = oracle.probe_scores(Q, np.zeros((L, 1, 4), np.float32), np.arange(L))
    Hn = [Fraction(0)]
    for t in range(1, L + 1):
        Hn.append(Hn[-1] + Fraction(1, t))
    for tau in (Fraction(1, 2), Fraction(9, 10), Fraction(97, 100)):
        C, want = Fraction(0), None
        for i in range(1, L + 1):
            C += Hn[L] - Hn[i - 1]
            if C >= tau * L:
                want = i
                break
        assert oracle.budget(acc, float(tau))[0] == want


# ----------------------------------------------------------------------------
# top-k (Eq. 9)
# ----------------------------------------------------------------------------
def test_topk_matches_full_argsort_and_tie_rule():
    for L in (1, 2, 9, 257):
        m = rng.random(L)
        m[rng.integers(0, L, L // 3)] = 0.5          # plant ties
        for p in sorted({1, max(1, L // 2), L}):
            T = oracle.topk_index(m, p)
            order = np.lexsort((np.arange(L), -m))   # value desc, index asc
            want = np.sort(order[:p])
            assert np.array_equal(T, want)
            assert np.all(np.diff(T) > 0) and len(T) == p
            U = np.setdiff1d(np.arange(L), T)
            if len(U):
                assert m[T].min() >= m[U].max()
    # explicit tie: smaller index wins
    assert np.array_equal(oracle.topk_index(np.array([1.0, 2.0, 2.0, 2.0, 0.0]), 2), [1, 2])


def test_select_modes_and_fixed_k():
    acc = rng.random(200) ** 3
    norm = acc / (1 + np.arange(200)[::-1])
    p, T, _ = oracle.select(acc, norm, 0.9)
    assert p == oracle.budget(acc, 0.9)[0] and np.array_equal(T, oracle.topk_index(norm, p))
    # acc/acc pairing: the kept set itself holds at least tau of the mass
    p, T, _ = oracle.select(acc, norm, 0.9, topk_metric=oracle.METRIC_ACC)
    assert acc[T].sum() >= 0.9 * acc.sum() * (1 - 1e-14)
    p, T, _ = oracle.select(acc, norm, 0.9, budget_metric=oracle.METRIC_NORM)
    assert p == oracle.budget(norm, 0.9)[0]
    p, T, _ = oracle.select(acc, norm, 0.9, fixed_k=17)
    assert p == 17 and len(T) == 17


def test_keep_last_is_the_union_with_the_final_positions():
    """keep_last (outside the paper): brute force with Python sets on small rows."""
    for L in (1, 5, 64, 301):
        acc = rng.random(L) ** 4
        norm = acc / (1 + np.arange(L)[::-1])
        for r in (0, 1, 7, L, L + 3):
            for tau in (0.3, 0.9):
                p0, T0, _ = oracle.select(acc, norm, tau)
                k, T, _ = oracle.select(acc, norm, tau, keep_last=r)
                want = sorted(set(T0.tolist()) | set(range(max(0, L - r), L)))
                assert T.tolist() == want and k == len(want)
                assert p0 <= k <= min(L, p0 + r)
                # nothing but final positions was added, and every final position is in
                assert all(j >= L - r for j in set(T.tolist()) - set(T0.tolist()))
    k, T, _ = oracle.select(np.array([5.0, 1.0, 1.0, 1.0]), np.array([5.0, 1.0, 1.0, 1.0]), 0.5, keep_last=1)
    assert k == 2 and T.tolist() == [0, 3]
    k, T, _ = oracle.select(np.arange(6.0), np.arange(6.0), 0.5, fixed_k=2, keep_last=2)
    assert k == 2 and T.tolist() == [4, 5]          # already the top two: nothing to add


# ----------------------------------------------------------------------------
# sparse prefill (Algorithm 1; Eq. 2 on gathered tokens)
# ----------------------------------------------------------------------------
@pytest.mark.parametrize("L,Hq,Hkv,d", [(1, 1, 1, 4), (19, 4, 2, 8), (40, 3, 1, 16)])
def test_prefill_all_tokens_is_dense_causal_attention(L, Hq, Hkv, d):
    Q, K, V = rand_qkv(L, Hq, Hkv, d)
    out = oracle.sparse_prefill(Q, K, V, np.arange(L))
    np.testing.assert_allclose(out, dense_causal_attention(Q, K, V), rtol=1e-11, atol=1e-13)
    # library routine: torch's scaled_dot_product_attention, causal, fp64
    tq = torch.from_numpy(Q).double().permute(1, 0, 2)[None]
    G = Hq // Hkv
    tk = torch.from_numpy(K).double().repeat_interleave(G, 1).permute(1, 0, 2)[None]
    tv = torch.from_numpy(V).double().repeat_interleave(G, 1).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)
    np.testing.assert_allclose(out, ref[0].permute(1, 0, 2).numpy(), rtol=1e-9, atol=1e-11)


def test_prefill_arbitrary_T_equals_masked_dense():
    L, Hq, Hkv, d = 45, 4, 2, 8
    Q, K, V = rand_qkv(L, Hq, Hkv, d)
    T = np.sort(rng.choice(L, 17, replace=False)).astype(np.int32)
    km = np.zeros(L, bool)
    km[T] = True
    out = oracle.sparse_prefill(Q, K, V, T)
    ref = dense_causal_attention(Q, K, V, key_mask=km)[T]
    np.testing.assert_allclose(out, ref, rtol=1e-11, atol=1e-13)
    # a subset of rows gives the same rows
    rows = np.array([0, 5, 16])
    np.testing.assert_array_equal(oracle.sparse_prefill(Q, K, V, T, rows=rows), out[rows])
    # padded form: rows outside T are exactly zero
    full = oracle.pad_rows(out, T, L)
    U = np.setdiff1d(np.arange(L), T)
    assert np.all(full[U] == 0) and np.array_equal(full[T], out)


def test_tau_one_reproduces_dense_attention_end_to_end():
    L, Hq, Hkv, d = 37, 4, 4, 8
    Q, K, V = rand_qkv(L, Hq, Hkv, d)
    probe = np.arange(L - 8, L)
    acc, _ = oracle.probe_scores(Q, K, probe)
    norm, _ = oracle.normalise(acc, probe, Hq)
    p, T, _ = oracle.select(acc, norm, 1.0)
    assert p == L and np.array_equal(T, np.arange(L))
    out = oracle.sparse_prefill(Q, K, V, T)
    np.testing.assert_allclose(out, dense_causal_attention(Q, K, V), rtol=1e-11, atol=1e-13)


# ----------------------------------------------------------------------------
# compaction and decode (Algorithm 1 cache step, Algorithm 2)
# ----------------------------------------------------------------------------
def test_compaction_is_bitwise_gather():
    x = torch.randn(50, 3, 8, generator=torch.Generator().manual_seed(5)).to(torch.bfloat16)
    raw = x.view(torch.int16).numpy()
    T = np.array([0, 7, 8, 49], np.int32)
    np.testing.assert_array_equal(oracle.compact_rows(raw, T), raw[T])
    xf = rng.standard_normal((20, 2, 4)).astype(np.float32)
    xf[3, 0, 0] = -0.0
    xf[3, 0, 1] = np.nan
    got = oracle.compact_rows(xf, np.array([3, 19], np.int32))
    assert got.tobytes() == xf[[3, 19]].tobytes()
    assert oracle.compact_rows(xf, np.zeros(0, np.int32)).shape == (0, 2, 4)


def test_decode_equals_last_row_of_dense_attention_and_appends():
    B, Hq, Hkv, d = 3, 4, 2, 8
    lens = np.array([5, 1, 12], np.int32)
    cap = lens + 2
    off = np.concatenate([[0], np.cumsum(cap[:-1] * Hkv * d)]).astype(np.int64)
    kc = np.zeros(int((cap * Hkv * d).sum()), np.float32)
    vc = np.zeros_like(kc)
    Ks, Vs = [], []
    for b in range(B):
        k = rng.standard_normal((lens[b], Hkv, d)).astype(np.float32)
        v = rng.standard_normal((lens[b], Hkv, d)).astype(np.float32)
        kc[off[b]: off[b] + k.size] = k.ravel()
        vc[off[b]: off[b] + v.size] = v.ravel()
        Ks.append(k)
        Vs.append(v)
    seq = lens.copy()
    for step in range(2):
        q = rng.standard_normal((B, Hq, d)).astype(np.float32)
        kn = rng.standard_normal((B, Hkv, d)).astype(np.float32)
        vn = rng.standard_normal((B, Hkv, d)).astype(np.float32)
        out = oracle.decode_step(q, kn, vn, kc, vc, off, seq, Hkv)
        assert np.array_equal(seq, lens + step + 1)
        for b in range(B):
            Ks[b] = np.concatenate([Ks[b], kn[b:b + 1]])
            Vs[b] = np.concatenate([Vs[b], vn[b:b + 1]])
            n = len(Ks[b])
            # cache contents after the append
            got = kc[off[b]: off[b] + n * Hkv * d].reshape(n, Hkv, d)
            assert np.array_equal(got, Ks[b])
            # Eq. 5 = last row of dense causal attention whose last query is q
            Qfull = np.zeros((n, Hq, d), np.float32)
            Qfull[-1] = q[b]
            ref = dense_causal_attention(Qfull, Ks[b], Vs[b])[-1]
            np.testing.assert_allclose(out[b], ref, rtol=1e-11, atol=1e-13)
    # without new tokens nothing is appended
    out2 = oracle.decode_step(q, None, None, kc, vc, off, seq, Hkv)
    np.testing.assert_array_equal(out2, out)
    assert np.array_equal(seq, lens + 2)


def test_prefill_decode_consistency():
    # decoding token n over the uncompacted cache of tokens 0..n-1 reproduces the
    # dense prefill row of token n
    L, Hq, Hkv, d = 20, 4, 2, 8
    Q, K, V = rand_qkv(L, Hq, Hkv, d)
    dense = oracle.sparse_prefill(Q, K, V, np.arange(L))
    kc = np.zeros(L * Hkv * d, np.float32)
    vc = np.zeros_like(kc)
    kc[: (L - 1) * Hkv * d] = K[:-1].ravel()
    vc[: (L - 1) * Hkv * d] = V[:-1].ravel()
    seq = np.array([L - 1], np.int32)
    out = oracle.decode_step(Q[-1:], K[-1:], V[-1:], kc, vc, np.zeros(1, np.int64), seq, Hkv)
    np.testing.assert_allclose(out[0], dense[-1], rtol=1e-11, atol=1e-13)


# ----------------------------------------------------------------------------
# hand-derived exact example (tests/golden/worked_example_ln2.txt)
# ----------------------------------------------------------------------------
def _golden():
    vals = {}
    with open(os.path.join(GOLDEN, "worked_example_ln2.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            key, *rest = line.split()
            vals[key] = [Fraction(x) for x in rest]
    return vals


def test_worked_example_end_to_end():
    g = _golden()
    as3 = lambda key: np.array([float(x) for x in g[key]], np.float32).reshape(-1, 1, 1)
    Q, K, V = as3("q"), as3("k"), as3("v")
    scale = math.log(2.0)
    tau = float(g["tau"][0])
    probe = np.arange(3)
    acc, S = oracle.probe_scores(Q, K, probe, scale=scale)
    np.testing.assert_allclose(acc, [float(x) for x in g["acc"]], rtol=1e-14)
    assert abs(S - float(g["total"][0])) < 1e-14
    norm, nnz = oracle.normalise(acc, probe, 1)
    assert list(nnz) == [int(x) for x in g["nnz"]]
    np.testing.assert_allclose(norm, [float(x) for x in g["norm"]], rtol=1e-14)
    p, T, _ = oracle.select(acc, norm, tau)
    assert p == int(g["p"][0]) and list(T) == [int(x) for x in g["T"]]
    out = oracle.sparse_prefill(Q, K, V, T, scale=scale)
    np.testing.assert_allclose(out.ravel(), [float(x) for x in g["out_compact"]], rtol=1e-14)
    kc = np.zeros(3, np.float32)
    vc = np.zeros(3, np.float32)
    kc[:2] = oracle.compact_rows(K, T).ravel()
    vc[:2] = oracle.compact_rows(V, T).ravel()
    seq = np.array([2], np.int32)
    o = oracle.decode_step(as3("decode_q"), as3("decode_k"), as3("decode_v"), kc, vc,
                           np.zeros(1, np.int64), seq, 1, scale=scale)
    np.testing.assert_allclose(o.ravel(), [float(g["decode_out"][0])], rtol=1e-14)
    assert seq[0] == 3


def test_paged_decode_is_decode_on_the_gathered_rows():
    """The paged layout is storage only: with any permutation of the pool's pages the outputs
    equal those of decode_step on contiguous caches holding the same rows, the appended row
    lands in the page and slot its position names, and no other pool entry changes."""
    rng = np.random.default_rng(12)
    B, Hq, Hkv, d, page_rows = 3, 4, 2, 8, 4
    lens = np.array([7, 4, 0], np.int32)            # mid-page, page boundary (append opens a new page), empty
    max_pages = 3
    n_pages = 11
    perm = rng.permutation(n_pages)[: B * max_pages].reshape(B, max_pages).astype(np.int32)
    k_pages = rng.standard_normal((n_pages, page_rows, Hkv, d)).astype(np.float32)
    v_pages = rng.standard_normal((n_pages, page_rows, Hkv, d)).astype(np.float32)
    q = rng.standard_normal((B, Hq, d)).astype(np.float32)
    kn = rng.standard_normal((B, Hkv, d)).astype(np.float32)
    vn = rng.standard_normal((B, Hkv, d)).astype(np.float32)
    # contiguous reference built by hand from the table
    cap = max_pages * page_rows
    kc = np.stack([np.concatenate([k_pages[p_] for p_ in perm[b]]) for b in range(B)])
    vc = np.stack([np.concatenate([v_pages[p_] for p_ in perm[b]]) for b in range(B)])
    off = np.arange(B, dtype=np.int64) * cap * Hkv * d
    seq_ref = lens.copy()
    kc_flat, vc_flat = kc.reshape(-1).copy(), vc.reshape(-1).copy()
    want = oracle.decode_step(q, kn, vn, kc_flat, vc_flat, off, seq_ref, Hkv)
    kp, vp, seq = k_pages.copy(), v_pages.copy(), lens.copy()
    got = oracle.decode_step_paged(q, kn, vn, kp, vp, perm, seq)
    assert np.array_equal(got, want) and np.array_equal(seq, lens + 1)
    changed = np.argwhere((kp != k_pages).any(axis=(2, 3)))
    expect = sorted((int(perm[b, lens[b] // page_rows]), int(lens[b] % page_rows)) for b in range(B))
    assert sorted(map(tuple, changed.tolist())) == expect
    for b in range(B):
        assert np.array_equal(kp[perm[b, lens[b] // page_rows], lens[b] % page_rows], kn[b])
        assert np.array_equal(vp[perm[b, lens[b] // page_rows], lens[b] % page_rows], vn[b])


# ---- mixed-precision KV cache (Sec. 4.3, Table 3): the quantiser reading and its packing ----
def _grid_rows(rng, n, H, d, bits, zero=-1.5, scale=0.25):
    """Rows that lie exactly on a quantisation grid whose zero point and scale are exact in
    bfloat16, with the smallest and the largest code present in every (row, head)."""
    codes = rng.integers(0, 1 << bits, (n, H, d)).astype(np.uint8)
    codes[..., 0] = 0
    codes[..., 1] = (1 << bits) - 1
    return codes, (zero + scale * codes.astype(np.float32)).astype(np.float32)


def test_quantiser_recovers_rows_that_lie_on_its_grid():
    rng = np.random.default_rng(5)
    for bits in (4, 2):
        codes, x = _grid_rows(rng, 7, 3, 32, bits)
        c, s, z = oracle.quantize_rows(x, bits, "bf16")
        assert np.array_equal(c, codes) and np.all(s == 0.25) and np.all(z == -1.5)
        assert np.array_equal(oracle.dequantize_rows(c, s, z), x.astype(np.float64))


def test_quantiser_round_trip_error_is_half_a_step_plus_the_parameter_rounding():
    rng = np.random.default_rng(6)
    x = (rng.standard_normal((50, 4, 64)) * rng.uniform(0.1, 5.0, (50, 4, 1))).astype(np.float32)
    for bits in (4, 2):
        levels = (1 << bits) - 1
        c, s, z = oracle.quantize_rows(x, bits, "bf16")
        assert c.max() <= levels
        err = np.abs(oracle.dequantize_rows(c, s, z) - x)
        lo, hi = x.min(-1), x.max(-1)
        slack = np.maximum(0, (hi - z) - levels * s) + np.maximum(0, z - lo)      # what the bf16 parameters miss
        assert np.all(err <= (0.5 * s + slack)[..., None] * (1 + 1e-5) + 1e-7)
        # the parameters are the storage type's roundings of min and (max - min) / levels
        assert np.all(np.abs(z - lo) <= np.abs(lo) * 2.0 ** -8)
        assert np.all(np.abs(s - (hi - lo) / levels) <= (hi - lo) / levels * 2.0 ** -8)
        # codes are monotone in the value within a row
        order = np.argsort(x, axis=-1)
        assert np.all(np.diff(np.take_along_axis(c.astype(int), order, -1), axis=-1) >= 0)


def test_quantiser_constant_row_and_packing():
    x = np.full((2, 1, 8), 0.75, np.float32)
    c, s, z = oracle.quantize_rows(x, 4, "bf16")
    assert not c.any() and np.all(s == 0) and np.all(oracle.dequantize_rows(c, s, z) == 0.75)
    # bytes written out by hand: 4-bit pairs low nibble first, 2-bit quads lowest bits first
    assert oracle.pack_codes(np.array([[1, 2, 3, 4, 15, 0, 9, 10]], np.uint8), 4).tolist() == [[0x21, 0x43, 0x0F, 0xA9]]
    assert oracle.pack_codes(np.array([[1, 2, 3, 0, 3, 3, 3, 3]], np.uint8), 2).tolist() == [[0b00111001, 0xFF]]


def test_mixed_precision_cache_split_and_lossless_decode():
    """Tokens of T at 4 bits in T's order, the rest at 2 bits ascending; on data that both grids
    hold exactly, a decode step over the quantised cache is the dense decode step over all L
    rows (softmax attention does not depend on the order of the cached rows), and the appended
    token joins the 4-bit block."""
    rng = np.random.default_rng(7)
    L, Hq, Hkv, d = 40, 4, 2, 16
    T = np.sort(rng.choice(L, 13, replace=False))
    U = np.setdiff1d(np.arange(L), T)
    K = np.zeros((L, Hkv, d), np.float32)
    V = np.zeros((L, Hkv, d), np.float32)
    for toks, bits in ((T, 4), (U, 2)):
        K[toks] = _grid_rows(rng, len(toks), Hkv, d, bits)[1]
        V[toks] = _grid_rows(rng, len(toks), Hkv, d, bits, zero=0.5, scale=0.125)[1]
    cache = oracle.quantize_kv(K, V, T, "bf16")
    assert np.array_equal(cache["hi"]["tokens"], T) and np.array_equal(cache["lo"]["tokens"], U)
    assert cache["hi"]["k_codes"].max() <= 15 and cache["lo"]["k_codes"].max() <= 3
    q = rng.standard_normal((1, Hq, d)).astype(np.float32)
    kn = _grid_rows(rng, 1, Hkv, d, 4)[1]
    vn = _grid_rows(rng, 1, Hkv, d, 4, zero=0.5, scale=0.125)[1]
    got = oracle.decode_step_quant(q, kn, vn, cache, Hkv)
    kc = np.concatenate([K, np.zeros((1, Hkv, d), np.float32)]).reshape(-1)
    vc = np.concatenate([V, np.zeros((1, Hkv, d), np.float32)]).reshape(-1)
    seq = np.array([L], np.int32)
    want = oracle.decode_step(q, kn, vn, kc, vc, np.zeros(1, np.int64), seq, Hkv)
    assert np.abs(got - want).max() < 1e-12
    assert len(cache["hi"]["tokens"]) == len(T) + 1 and len(cache["lo"]["tokens"]) == len(U)
    assert np.array_equal(oracle.dequantize_rows(cache["hi"]["k_codes"][-1:], cache["hi"]["k_scale"][-1:],
                                                 cache["hi"]["k_zero"][-1:]), kn.astype(np.float64))
