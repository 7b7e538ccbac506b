"""Pins for the fp64 CPU oracle: everything here checks the oracle against something other than
itself -- values the paper prints, closed forms, invariants, brute force and textbook routines
written out again in this file with numpy.  None of these tests needs a GPU."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import sla_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = [int(v) for v in vals]
    return out


def rand(shape, seed, dtype=np.float64):
    return np.random.default_rng(seed).standard_normal(shape).astype(dtype)


# --------------------------------------------------------------------------- printed values
def test_worked_example_i30():
    """Caption of the structural non-exclusion figure: i=30, b=2, f=0."""
    g = read_golden("worked_example_i30.txt")
    i, b, f = g["i"][0], g["b"][0], g["f"][0]
    t, s = O.anchors(i)
    assert list(t) == g["anchors"]
    assert list(s) == [0, 1, 2, 3, 4]
    ell = O.base_len(i)
    assert ell == g["base_len"][0]
    assert (b + f) * ell == g["span_len"][0]
    covered = set()
    for a in t:
        lo, hi = O.span(i, int(a), ell, b, f)
        assert (lo, hi) == (max(0, int(a) - 12), int(a))   # span length 12 behind the anchor
        covered.update(range(lo, hi + 1))
    assert covered == set(range(g["covered_lo"][0], g["covered_hi"][0] + 1))


def test_anchor_sequence_and_gaps():
    g = read_golden("anchor_sequence.txt")
    for i in (15, 16, 100, 4095, 65535):
        t, _ = O.anchors(i)
        assert [i - int(x) for x in t[:4]] == g["offsets"]
        assert [int(t[j] - t[j + 1]) for j in range(3)] == g["gaps"]
        # all gaps are the odd numbers 3, 5, 7, ... (difference of consecutive squares)
        assert [int(t[j] - t[j + 1]) for j in range(len(t) - 1)] == [2 * j + 3 for j in range(len(t) - 1)]
        assert t[-1] >= 0 and i + 1 - (len(t) + 1) ** 2 < 0


def test_window_adjacency_w1088():
    """With w = 1088 the first surviving anchor sits exactly one position left of the window."""
    w = read_golden("anchor_sequence.txt")["window"][0]
    for i in (5000, 65535, 1_000_000):
        t, s = O.anchors(i, window=w)
        w_lo = i - w + 1
        assert int(t[0]) == w_lo - 1
        assert int(s[0]) == 32          # 33^2 - 1 = 1088
        t_all, _ = O.anchors(i)
        assert len(t) == len(t_all) - 32
    # candidate count: max(0, floor(sqrt(i+1)) - floor(sqrt(w)))
    for w_ in (0, 1, 3, 4, 10, 100):
        for i in range(0, 300, 7):
            t, _ = O.anchors(i, window=w_)
            assert len(t) == max(0, math.isqrt(i + 1) - math.isqrt(w_))
            assert all(x < i - w_ + 1 for x in t) or w_ == 0


def test_integer_roots():
    for x in list(range(0, 2000)) + [10**6 - 1, 10**6, 10**6 + 1, 2**40 - 1, 2**40, 2**40 + 1]:
        r = math.isqrt(x)
        c = r if r * r == x else r + 1
        assert O.ceil_isqrt(x) == c
        if x < 5000:
            assert O.isqrt(x) == r
    assert O.base_len(30) == 6 and O.base_len(0) == 0 and O.base_len(30, 64) == 64


# --------------------------------------------------------------------------- work counts
def closed_form_dots(L):
    """sum_{i<L} floor(sqrt(i+1)): j appears for the 2j+1 values m=i+1 in [j^2,(j+1)^2)."""
    r = math.isqrt(L)
    return sum(j * (2 * j + 1) for j in range(1, r)) + r * (L - r * r + 1)


def test_work_count_closed_form_and_scaling():
    known = {16: 38, 64: 316, 256: 2616, 1024: 21360, 4096: 172768}
    for L, want in known.items():
        assert closed_form_dots(L) == want
    D = 4
    counts = {}
    pairs = {}
    for L in (16, 64, 256, 1024, 4096):
        q = rand((1, 1, L, D), 1)
        k = rand((1, 1, L, D), 2)
        res = O.span_search(q, k, O.F64, top_k=4)
        assert res["n_dots"] == closed_form_dots(L)
        assert res["n_dots"] <= (2.0 / 3.0) * L ** 1.5 + L
        counts[L] = res["n_dots"]
        att = O.span_attention(q, k, k, O.F64, res["anchor"], span_len=0)
        pairs[L] = att["n_pairs"]
    # both stages grow like L^{3/2} (Section "Two-step mechanism and scaling analysis")
    for d in (counts, pairs):
        slope = math.log(d[4096] / d[1024]) / math.log(4.0)
        assert abs(slope - 1.5) < 0.06, slope


# --------------------------------------------------------------------------- coverage invariant
def test_coverage_invariant():
    """b >= 1/p = 2 makes the candidate spans of every query cover [0, i]; b = 1 does not."""
    def covered(i, b, span_len=0):
        t, _ = O.anchors(i)
        ell = O.base_len(i, span_len)
        m = np.zeros(i + 1, dtype=bool)
        for a in t:
            lo, hi = O.span(i, int(a), ell, b, 0)
            m[lo:hi + 1] = True
        return bool(m.all())

    assert all(covered(i, 2) for i in range(0, 1500))
    first_fail = next(i for i in range(0, 200) if not covered(i, 1))
    assert first_fail == 7
    # fixed base length 64 with b = 2 covers every query below 4096 (the tiny prefill case)
    assert all(covered(i, 2, 64) for i in range(0, 4096, 13)) and covered(4095, 2, 64)


# --------------------------------------------------------------------------- dense equivalence
def dense_causal(q, k, v, scale):
    """Textbook causal softmax attention with grouped heads, numpy, fp64."""
    B, Hq, L, D = q.shape
    G = Hq // k.shape[1]
    out = np.zeros((B, Hq, L, D))
    lse = np.zeros((B, Hq, L))
    mask = np.tril(np.ones((L, L), dtype=bool))
    for b in range(B):
        for h in range(Hq):
            x = scale * (q[b, h] @ k[b, h // G].T)
            x = np.where(mask, x, -np.inf)
            m = x.max(axis=1, keepdims=True)
            e = np.exp(x - m)
            z = e.sum(axis=1, keepdims=True)
            out[b, h] = (e / z) @ v[b, h // G]
            lse[b, h] = (m + np.log(z))[:, 0]
    return out, lse


@pytest.mark.parametrize("span_len,window", [(0, 0), (24, 0), (0, 8), (0, 48)])
def test_union_with_all_anchors_is_dense_causal(span_len, window):
    # windows are m^2 - 1 (8, 48): only then does the first surviving anchor touch the window, which
    # is the adjacency rule of Section "Span attention"; any other w leaves uncovered keys.
    B, Hq, Hkv, L, D = 2, 4, 2, 333, 16
    q_s, q = rand((B, Hq, L, D), 3), rand((B, Hq, L, D), 4)
    k, v = rand((B, Hkv, L, D), 5), rand((B, Hkv, L, D), 6)
    top_k = math.isqrt(L) + 1
    sr = O.span_search(q_s, k, O.F64, top_k=top_k, window=window)
    at = O.span_attention(q, k, v, O.F64, sr["anchor"], span_len=span_len, window=window, softmax_scale=0.3)
    ref_out, ref_lse = dense_causal(q, k, v, 0.3)
    np.testing.assert_allclose(at["out"], ref_out, rtol=0, atol=1e-12)
    np.testing.assert_allclose(at["lse"], ref_lse, rtol=0, atol=1e-12)
    assert at["n_pairs"] == B * Hq * L * (L + 1) // 2


def test_dense_equivalence_against_torch_sdpa():
    B, H, L, D = 1, 2, 200, 8
    q_s, q, k, v = (rand((B, H, L, D), s) for s in (7, 8, 9, 10))
    sr = O.span_search(q_s, k, O.F64, top_k=32)
    at = O.span_attention(q, k, v, O.F64, sr["anchor"], span_len=0)  # default scale 1/sqrt(D)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q), torch.from_numpy(k), torch.from_numpy(v), is_causal=True).numpy()
    np.testing.assert_allclose(at["out"], ref, rtol=0, atol=1e-12)


# --------------------------------------------------------------------------- exhaustive scoring
@pytest.mark.parametrize("top_k", [1, 3, 8])
def test_search_against_exhaustive_scoring(top_k):
    B, Hq, Hkv, L, D = 1, 4, 2, 256, 8
    q_s, k = rand((B, Hq, L, D), 11), rand((B, Hkv, L, D), 12)
    res = O.span_search(q_s, k, O.F64, top_k=top_k, search_scale=0.5)
    G = Hq // Hkv
    squares = {m * m for m in range(1, 40)}
    for h in range(Hq):
        full = 0.5 * (q_s[0, h] @ k[0, h // G].T)          # every (i, j) score
        for i in range(L):
            cand = [j for j in range(i + 1) if (i - j + 1) in squares]
            order = sorted(cand, key=lambda j: (-full[i, j], -j))  # ties: nearer anchor first
            want = order[:top_k]
            got = [int(a) for a in res["anchor"][0, h, i] if a >= 0]
            assert got == want, (h, i)
            np.testing.assert_allclose(res["score"][0, h, i, :len(want)], full[i, want], atol=1e-12)
            assert np.all(np.isneginf(res["score"][0, h, i, len(want):]))
            assert np.all(res["anchor"][0, h, i, len(want):] == -1)
            if len(order) > top_k:
                assert abs(res["gap"][0, h, i] - (full[i, order[top_k - 1]] - full[i, order[top_k]])) < 1e-12
            else:
                assert np.isposinf(res["gap"][0, h, i])


def test_tie_break_prefers_nearer_anchor():
    L, D = 64, 4
    q_s = np.ones((1, 1, L, D))
    k = np.ones((1, 1, L, D))       # every score equal
    res = O.span_search(q_s, k, O.F64, top_k=3)
    for i in (8, 30, 63):
        assert list(res["anchor"][0, 0, i]) == [i, i - 3, i - 8]


def test_search_scale_does_not_change_selection():
    q_s, k = rand((1, 2, 300, 8), 13), rand((1, 1, 300, 8), 14)
    a = O.span_search(q_s, k, O.F64, top_k=4, search_scale=1.0)
    b = O.span_search(q_s, k, O.F64, top_k=4, search_scale=0.5)
    assert np.array_equal(a["anchor"], b["anchor"])
    np.testing.assert_allclose(a["score"], 2.0 * b["score"])


# --------------------------------------------------------------------------- brute-force attention
def brute_union(q, k, v, i, anchors, ell, b, f, scale, window=0):
    keys = set()
    for t in anchors:
        if t < 0:
            continue
        keys.update(range(max(0, t - b * ell), min(i, t + f * ell) + 1))
    if window > 0:
        keys.update(range(max(0, i - window + 1), i + 1))
    keys = sorted(keys)
    if not keys:
        return np.zeros(q.shape[-1]), -np.inf
    x = scale * (k[keys] @ q)
    m = x.max()
    e = np.exp(x - m)
    return (e / e.sum()) @ v[keys], m + math.log(e.sum())


@pytest.mark.parametrize("b,f,window,span_len", [(2, 0, 0, 0), (4, 2, 0, 0), (2, 0, 12, 0), (1, 1, 0, 7), (0, 0, 0, 5)])
def test_union_attention_against_set_brute_force(b, f, window, span_len):
    B, Hq, Hkv, L, D = 1, 2, 1, 150, 8
    q_s, q = rand((B, Hq, L, D), 15), rand((B, Hq, L, D), 16)
    k, v = rand((B, Hkv, L, D), 17), rand((B, Hkv, L, D), 18)
    sr = O.span_search(q_s, k, O.F64, top_k=3, window=window)
    at = O.span_attention(q, k, v, O.F64, sr["anchor"], span_len=span_len, back_factor=b, fwd_factor=f,
                          window=window, softmax_scale=0.25)
    pairs = 0
    for h in range(Hq):
        for i in range(L):
            ell = span_len if span_len > 0 else (math.isqrt(i - 1) + 1 if i > 0 else 0)  # ceil(sqrt(i))
            o, l = brute_union(q[0, h, i], k[0, 0], v[0, 0], i, sr["anchor"][0, h, i], ell, b, f, 0.25, window)
            np.testing.assert_allclose(at["out"][0, h, i], o, atol=1e-12)
            assert abs(at["lse"][0, h, i] - l) < 1e-12 or (np.isneginf(l) and np.isneginf(at["lse"][0, h, i]))
    assert at["n_pairs"] > 0


def test_per_span_gate_against_brute_force():
    """Algorithm 1 literally: per-span softmax (the line for A_{i,t}), then the softmax gate of the
    Combination section.  Besides `out` this pins the two log-sum-exp outputs of the per-span mode:
    `lse_span[j]` is the log-sum-exp of the logits over J_t = S_t united with W of the j-th selected
    anchor, recomputed here from the key set itself (-inf on padding), and `lse` is the value of the
    best-scoring selected anchor (slot 0 of a selection that comes from the search).  Both checks
    fail on an oracle that swaps two `lse_span` slots or takes the wrong "first" span (verified by
    running the assertions on a copy with slots 0 and 1 exchanged, at the end)."""
    B, Hq, Hkv, L, D = 1, 2, 2, 120, 8
    q_s, q = rand((B, Hq, L, D), 19), rand((B, Hq, L, D), 20)
    k, v = rand((B, Hkv, L, D), 21), rand((B, Hkv, L, D), 22)
    for window in (0, 9):
        sr = O.span_search(q_s, k, O.F64, top_k=3, window=window)
        at = O.span_attention(q, k, v, O.F64, sr["anchor"], span_len=0, back_factor=2, fwd_factor=1,
                              window=window, mode=O.PER_SPAN, score=sr["score"], softmax_scale=0.25)
        want_span = np.full(at["lse_span"].shape, -np.inf)
        want_lse = np.full(at["lse"].shape, -np.inf)
        for h in range(Hq):
            for i in range(L):
                an = [int(a) for a in sr["anchor"][0, h, i] if a >= 0]
                ell = math.isqrt(i - 1) + 1 if i > 0 else 0
                if not an:
                    want, want_lse[0, h, i] = brute_union(q[0, h, i], k[0, h], v[0, h], i, [], ell, 2, 1, 0.25, window)
                else:
                    s = sr["score"][0, h, i, :len(an)]
                    alpha = np.exp(s - s.max())
                    alpha /= alpha.sum()
                    assert abs(alpha.sum() - 1.0) < 1e-12
                    per = [brute_union(q[0, h, i], k[0, h], v[0, h], i, [t], ell, 2, 1, 0.25, window) for t in an]
                    want = sum(al * o for al, (o, _) in zip(alpha, per))
                    want_span[0, h, i, :len(an)] = [l for _, l in per]
                    want_lse[0, h, i] = per[int(np.argmax(s))][1]    # the best-scoring selected anchor
                np.testing.assert_allclose(at["out"][0, h, i], want, atol=1e-12)

        def check(lse_span, lse):
            fin = np.isfinite(want_span)
            assert np.array_equal(np.isneginf(lse_span), ~fin)
            np.testing.assert_allclose(lse_span[fin], want_span[fin], atol=1e-12)
            finl = np.isfinite(want_lse)
            assert np.array_equal(np.isneginf(lse), ~finl)
            np.testing.assert_allclose(lse[finl], want_lse[finl], atol=1e-12)

        check(at["lse_span"], at["lse"])
        # the pin has teeth: two exchanged slots, or the second span's value as `lse`, are caught
        swapped = at["lse_span"].copy()
        swapped[..., [0, 1]] = swapped[..., [1, 0]]
        with pytest.raises(AssertionError):
            check(swapped, at["lse"])
        with pytest.raises(AssertionError):
            check(at["lse_span"], at["lse_span"][..., 1])


# --------------------------------------------------------------------------- special cases
def _small_problem(seed=30, B=1, Hq=4, Hkv=2, L=180, D=8):
    return (rand((B, Hq, L, D), seed), rand((B, Hq, L, D), seed + 1),
            rand((B, Hkv, L, D), seed + 2), rand((B, Hkv, L, D), seed + 3))


def test_k1_union_equals_per_span():
    q_s, q, k, v = _small_problem()
    sr = O.span_search(q_s, k, O.F64, top_k=1)
    a = O.span_attention(q, k, v, O.F64, sr["anchor"], span_len=0)
    b = O.span_attention(q, k, v, O.F64, sr["anchor"], span_len=0, mode=O.PER_SPAN, score=sr["score"])
    np.testing.assert_allclose(a["out"], b["out"], atol=1e-13)
    np.testing.assert_allclose(a["lse"], b["lse"], atol=1e-13)


def test_gqa_reduces_to_mha():
    q_s, q, k, v = _small_problem()
    sr = O.span_search(q_s, k, O.F64, top_k=3)
    at = O.span_attention(q, k, v, O.F64, sr["anchor"], span_len=0)
    k_rep, v_rep = np.repeat(k, 2, axis=1).copy(), np.repeat(v, 2, axis=1).copy()
    sr2 = O.span_search(q_s, k_rep, O.F64, top_k=3)
    at2 = O.span_attention(q, k_rep, v_rep, O.F64, sr2["anchor"], span_len=0)
    assert np.array_equal(sr["anchor"], sr2["anchor"])
    np.testing.assert_allclose(at["out"], at2["out"], atol=1e-14)


def test_constant_value_rows_and_convex_hull():
    q_s, q, k, v = _small_problem()
    sr = O.span_search(q_s, k, O.F64, top_k=3)
    vc = np.broadcast_to(np.arange(8.0), v.shape).copy()
    at = O.span_attention(q, k, vc, O.F64, sr["anchor"], span_len=0)
    np.testing.assert_allclose(at["out"], np.broadcast_to(np.arange(8.0), at["out"].shape), atol=1e-12)
    at = O.span_attention(q, k, v, O.F64, sr["anchor"], span_len=0)
    assert at["out"].max() <= v.max() + 1e-12 and at["out"].min() >= v.min() - 1e-12


def test_logit_shift_moves_lse_only():
    """Adding c*q/|q|^2... : a key shift along q adds a constant to every logit of that row."""
    _, q, k, v = _small_problem(B=1, Hq=1, Hkv=1)
    i = 150
    anchors = np.full((1, 1, 1, 2), -1, dtype=np.int32)
    anchors[0, 0, 0] = [i - 8, i - 48]
    qi = q[:, :, i:i + 1]
    base = O.span_attention(qi, k, v, O.F64, anchors, span_len=0, q_pos0=i, softmax_scale=1.0)
    shift = 0.7 * qi[0, 0, 0] / np.dot(qi[0, 0, 0], qi[0, 0, 0])
    moved = O.span_attention(qi, k + shift, v, O.F64, anchors, span_len=0, q_pos0=i, softmax_scale=1.0)
    np.testing.assert_allclose(moved["out"], base["out"], atol=1e-12)
    np.testing.assert_allclose(moved["lse"], base["lse"] + 0.7, atol=1e-12)


def test_anchor_permutation_and_duplicates_do_not_change_union():
    q_s, q, k, v = _small_problem()
    sr = O.span_search(q_s, k, O.F64, top_k=4)
    a = O.span_attention(q, k, v, O.F64, sr["anchor"], span_len=0)
    perm = sr["anchor"][..., ::-1].copy()
    b = O.span_attention(q, k, v, O.F64, perm, span_len=0)
    np.testing.assert_allclose(a["out"], b["out"], atol=1e-14)
    dup = np.concatenate([sr["anchor"], sr["anchor"][..., :2]], axis=-1)
    c = O.span_attention(q, k, v, O.F64, dup, span_len=0)
    np.testing.assert_allclose(a["out"], c["out"], atol=1e-14)
    assert c["n_pairs"] == a["n_pairs"]


def test_decode_equals_prefill_row_and_chunked_prefill():
    q_s, q, k, v = _small_problem(L=200)
    L = 200
    sr = O.span_search(q_s, k, O.F64, top_k=3)
    at = O.span_attention(q, k, v, O.F64, sr["anchor"], span_len=5)
    cap = 230
    kc = np.zeros((1, 2, cap, 8)); vc = np.zeros((1, 2, cap, 8))
    kc[:, :, :L] = k; vc[:, :, :L] = v
    for n_ctx in (1, 2, 17, 200):
        i = n_ctx - 1
        d = O.decode_step(q_s[:, :, i].copy(), q[:, :, i].copy(), kc, vc, O.F64, n_ctx=n_ctx, top_k=3, span_len=5)
        assert np.array_equal(d["anchor"], sr["anchor"][:, :, i])
        np.testing.assert_allclose(d["out"], at["out"][:, :, i], atol=1e-14)
        np.testing.assert_allclose(d["lse"], at["lse"][:, :, i], atol=1e-14)
    # chunked prefill (q_pos0 > 0) and row sampling give the same rows
    sr_c = O.span_search(q_s[:, :, 120:].copy(), k, O.F64, top_k=3, q_pos0=120)
    assert np.array_equal(sr_c["anchor"], sr["anchor"][:, :, 120:])
    rows = [0, 5, 150, 199]
    sr_r = O.span_search(q_s, k, O.F64, top_k=3, rows=rows)
    assert np.array_equal(sr_r["anchor"], sr["anchor"][:, :, rows])
    at_r = O.span_attention(q, k, v, O.F64, sr_r["anchor"], span_len=5, rows=rows)
    np.testing.assert_allclose(at_r["out"], at["out"][:, :, rows], atol=1e-14)


def test_padding_and_empty_selection():
    q_s, q, k, v = _small_problem(L=40)
    sr = O.span_search(q_s, k, O.F64, top_k=5)
    for i in range(40):
        n = math.isqrt(i + 1)
        assert np.all(sr["anchor"][0, :, i, :min(n, 5)] >= 0)
        assert np.all(sr["anchor"][0, :, i, min(n, 5):] == -1)
    none = np.full_like(sr["anchor"], -1)
    at = O.span_attention(q, k, v, O.F64, none, span_len=0)
    assert np.all(at["out"] == 0) and np.all(np.isneginf(at["lse"])) and at["n_pairs"] == 0
    # query 0 attends to itself only
    at = O.span_attention(q, k, v, O.F64, sr["anchor"], span_len=0)
    np.testing.assert_allclose(at["out"][0, :, 0], np.repeat(v[0, :, 0], 2, axis=0), atol=1e-14)


def test_input_dtypes_are_widened_exactly():
    """fp32 and bf16 inputs give the same result as their exact fp64 copies."""
    g = torch.Generator().manual_seed(5)
    shape_q, shape_k = (1, 2, 90, 16), (1, 1, 90, 16)
    t = [torch.randn(s, generator=g) for s in (shape_q, shape_q, shape_k, shape_k)]
    for dt, code in ((torch.float32, O.F32), (torch.bfloat16, O.BF16)):
        tl = [x.to(dt) for x in t]
        as_np = [x.view(torch.int16).numpy().view(np.uint16) if dt == torch.bfloat16 else x.numpy() for x in tl]
        as_64 = [x.to(torch.float64).numpy() for x in tl]
        a = O.span_search(as_np[0], as_np[2], code, top_k=3)
        b = O.span_search(as_64[0], as_64[2], O.F64, top_k=3)
        assert np.array_equal(a["anchor"], b["anchor"]) and np.array_equal(a["score"], b["score"])
        oa = O.span_attention(as_np[1], as_np[2], as_np[3], code, a["anchor"], span_len=4)
        ob = O.span_attention(as_64[1], as_64[2], as_64[3], O.F64, b["anchor"], span_len=4)
        assert np.array_equal(oa["out"], ob["out"])


# ---- general exponents (Section "Span attention": anchors at i - (s+1)^(1/p) + 1; Section "Training":
# search_exponent / span_exponent, e.g. 1/3 and 2/3) ------------------------------------------------

def icbrt(x: int) -> int:
    r = round(x ** (1.0 / 3.0))
    while r ** 3 > x:
        r -= 1
    while (r + 1) ** 3 <= x:
        r += 1
    return r


def test_stride_offsets_for_rational_exponents_are_exact_powers():
    """p = 1/2, 1/3, 1/4: (s+1)^(1/p) is an integer in exact arithmetic and must come out as that
    integer (the rounding of 1/p and of pow must not push it to the next one)."""
    for s in list(range(0, 300)) + [999, 1289]:          # offsets up to 2^31, the largest position
        assert O.stride_offset(s, 0.5) == (s + 1) ** 2
        assert O.stride_offset(s, 1.0 / 3.0) == (s + 1) ** 3
        if (s + 1) ** 4 < 2 ** 31:
            assert O.stride_offset(s, 0.25) == (s + 1) ** 4
    for p in (0.5, 1.0 / 3.0, 0.54, 0.4, 0.7):
        offs = [O.stride_offset(s, p) for s in range(400)]
        assert offs[0] == 1                                    # stride 0 is the query's own position
        assert all(b > a for a, b in zip(offs, offs[1:]))      # strictly increasing: distinct anchors
        # rounded up: the anchor never lies right of the real-valued position i - x + 1
        assert all(o >= (s + 1) ** (1.0 / p) * (1 - 2e-12) for s, o in enumerate(offs))
        assert all(o < (s + 1) ** (1.0 / p) + 1 for s, o in enumerate(offs))


def test_number_of_strides_matches_integer_roots_and_scales_as_i_to_p():
    for i in list(range(0, 2000)) + [10 ** 6, 10 ** 9 + 7]:
        assert O.n_strides(i, 0.5) == math.isqrt(i + 1)
        assert O.n_strides(i, 1.0 / 3.0) == icbrt(i + 1)
    for p in (0.4, 0.54, 0.6):
        n1, n2 = O.n_strides(10 ** 5, p), O.n_strides(10 ** 7, p)
        assert abs(n1 / (10 ** 5) ** p - 1) < 0.02 and abs(n2 / (10 ** 7) ** p - 1) < 0.01
        assert abs(math.log(n2 / n1) / math.log(100) - p) < 0.005   # O(i^p) candidates


def test_anchors_with_exponent_one_third():
    t, s = O.anchors(1000, 0, 1.0 / 3.0)
    assert list(t) == [1001 - m ** 3 for m in range(1, 11)] and list(s) == list(range(10))
    t, s = O.anchors(1000, 30, 1.0 / 3.0)          # W = [971, 1000]: offsets 1, 8, 27 fall inside
    assert list(t) == [1001 - m ** 3 for m in range(4, 11)] and list(s) == list(range(3, 10))


def test_base_len_with_span_exponent():
    for k in range(1, 60):
        assert O.base_len(k ** 3, 0, 2.0 / 3.0) == k * k          # exact at perfect cubes
        assert O.base_len(k ** 3 + 1, 0, 2.0 / 3.0) == k * k + 1  # rounded up right after
    assert O.base_len(0, 0, 2.0 / 3.0) == 0 and O.base_len(5, 7, 2.0 / 3.0) == 7
    for i in (1, 2, 30, 31, 1000, 65535):
        assert O.base_len(i, 0, 0.5) == math.isqrt(i - 1) + 1     # integer ceil-sqrt, as before


def test_coverage_and_dense_equivalence_with_exponents_one_third_two_thirds():
    """Span-length derivation of Section "Span attention" for general p: the gap between adjacent
    anchors is (s+1)^(1/p) - s^(1/p) <= (1/p) (s+1)^(1/p - 1) <= (1/p) i^(1-p); with p = 1/3 and
    l(i) = ceil(i^(2/3)) a backward factor of 3 covers every key, so attention over all anchors is
    dense causal attention; a backward factor of 1 is not enough."""
    B, Hq, Hkv, L, D = 1, 2, 1, 400, 8
    q_s, q = rand((B, Hq, L, D), 13), rand((B, Hq, L, D), 14)
    k, v = rand((B, Hkv, L, D), 15), rand((B, Hkv, L, D), 16)
    sr = O.span_search(q_s, k, O.F64, top_k=10, search_exponent=1.0 / 3.0)
    assert (sr["anchor"][0, 0, 399] >= 0).sum() == 7          # 1, 8, ..., 343 <= 400
    at = O.span_attention(q, k, v, O.F64, sr["anchor"], span_len=0, back_factor=3, softmax_scale=0.3,
                          span_exponent=2.0 / 3.0)
    ref_out, ref_lse = dense_causal(q, k, v, 0.3)
    np.testing.assert_allclose(at["out"], ref_out, rtol=0, atol=1e-12)
    np.testing.assert_allclose(at["lse"], ref_lse, rtol=0, atol=1e-12)
    at1 = O.span_attention(q, k, v, O.F64, sr["anchor"], span_len=0, back_factor=1, softmax_scale=0.3,
                           span_exponent=2.0 / 3.0)
    assert at1["n_pairs"] < at["n_pairs"]


def test_search_with_exponent_against_exhaustive_scoring():
    B, Hq, Hkv, L, D, top_k = 1, 2, 2, 130, 8, 3
    q_s, k = rand((B, Hq, L, D), 21), rand((B, Hkv, L, D), 22)
    for p, root in ((1.0 / 3.0, 3), (0.25, 4)):
        sr = O.span_search(q_s, k, O.F64, top_k=top_k, search_exponent=p)
        for h in range(Hq):
            for i in range(L):
                cand = [i + 1 - m ** root for m in range(1, 12) if i + 1 - m ** root >= 0]
                sc = np.array([q_s[0, h, i] @ k[0, h, t] for t in cand])
                order = np.argsort(-sc, kind="stable")[:top_k]
                want = [cand[j] for j in order] + [-1] * (top_k - len(order))
                assert list(sr["anchor"][0, h, i]) == want
