"""The parity checkers themselves, on CPU: fed with the oracle's own results they must pass, and every
kind of invalid selection they exist to catch must make them fail."""
import numpy as np
import pytest
import torch

import parity_util as P
from oracle import sla_oracle as O


def _problem(window=0, p=0.5, L=400, top_k=4, seed=5):
    rng = np.random.default_rng(seed)
    q_s = rng.standard_normal((1, 4, L, 8)).astype(np.float32)
    k = rng.standard_normal((1, 2, L, 8)).astype(np.float32)
    ref = O.span_search(q_s, k, O.F32, top_k=top_k, window=window, search_exponent=p)
    a = torch.from_numpy(ref["anchor"].copy())
    s = torch.from_numpy(ref["score"].astype(np.float32))
    return q_s, k, ref, a, s


@pytest.mark.parametrize("window,p", [(0, 0.5), (24, 0.5), (0, 1.0 / 3.0), (10, 0.54)])
def test_checker_accepts_the_oracles_own_selection(window, p):
    q_s, k, ref, a, s = _problem(window, p)
    P.compare_search(a, s, ref, q_s=q_s, k=k, window=window, search_exponent=p)
    rows = np.array([0, 1, 7, 100, 399])
    sub = O.span_search(q_s, k, O.F32, top_k=4, window=window, search_exponent=p, rows=rows)
    P.compare_search(a, s, sub, rows=rows, q_s=q_s, k=k, window=window, search_exponent=p)


def test_checker_rejects_invalid_selections():
    q_s, k, ref, a, s = _problem()
    i = 300
    # a near-tie row is exempt from set equality, but not from validity
    ref["gap"][0, 0, i] = 0.0

    def broken(fn):
        a2, s2 = a.clone(), s.clone()
        fn(a2, s2)
        with pytest.raises(AssertionError):
            P.compare_search(a2, s2, ref, q_s=q_s, k=k)

    def dup(a2, s2):
        a2[0, 0, i, 3], s2[0, 0, i, 3] = a2[0, 0, i, 2], s2[0, 0, i, 2]

    def off_pattern(a2, s2):
        a2[0, 0, i, 3] = i - 1            # distance 2 is not a square

    def wrong_score(a2, s2):
        s2[0, 0, i, 3] -= 0.01            # not the dot product of its anchor

    def far_below(a2, s2):                 # a valid candidate, but far from the k best
        worst = min(range(1, 17), key=lambda m: float(q_s[0, 0, i] @ k[0, 0, i + 1 - m * m]))
        a2[0, 0, i, 3] = i + 1 - worst * worst
        s2[0, 0, i, 3] = float(q_s[0, 0, i] @ k[0, 0, i + 1 - worst * worst])

    def missing(a2, s2):
        a2[0, 0, i, 3], s2[0, 0, i, 3] = -1, -np.inf

    for fn in (dup, off_pattern, wrong_score, far_below, missing):
        broken(fn)
    # and a clear-cut row with another (valid) set fails on the set comparison
    ref["gap"][0, 0, i] = 1.0
    with pytest.raises(AssertionError):
        a2 = a.clone()
        a2[0, 0, i, 3] = i + 1 - 17 * 17
        P.compare_search(a2, s, ref)


def test_checker_rejects_an_anchor_inside_the_window():
    q_s, k, ref, a, s = _problem(window=24)
    a2 = a.clone()
    a2[0, 1, 200, 3] = 200 + 1 - 4     # offset 4 <= w
    ref["gap"][0, 1, 200] = 0.0
    with pytest.raises(AssertionError):
        P.compare_search(a2, s, ref, window=24)


def test_empty_mask_is_an_error():
    out = torch.zeros(1, 1, 2, 4)
    ref = {"out": np.zeros((1, 1, 2, 4)), "lse": np.zeros((1, 1, 2))}
    with pytest.raises(AssertionError):
        P.compare_attention(out, torch.zeros(1, 1, 2), ref, "f32", where=np.zeros((1, 1, 2), dtype=bool))


@pytest.mark.parametrize("mode", [O.UNION, O.PER_SPAN])
def test_decode_checker_on_the_oracles_step_and_on_the_alternative(mode):
    rng = np.random.default_rng(9)
    B, Hq, Hkv, D, n_ctx, top_k = 1, 4, 2, 8, 500, 3
    q_s = rng.standard_normal((B, Hq, D)).astype(np.float32)
    q = rng.standard_normal((B, Hq, D)).astype(np.float32)
    hk = rng.standard_normal((B, Hkv, n_ctx, D)).astype(np.float32)
    hv = rng.standard_normal((B, Hkv, n_ctx, D)).astype(np.float32)
    ref = O.decode_step(q_s, q, hk, hv, O.F32, n_ctx=n_ctx, top_k=top_k, span_len=12, window=8, mode=mode)
    got = tuple(torch.from_numpy(np.asarray(ref[n], dtype=dt)) for n, dt in
                (("out", np.float32), ("lse", np.float32), ("anchor", np.int32), ("score", np.float32)))
    assert P.check_decode_step(got, q_s, q, hk, hv, O.F32, "f32", n_ctx=n_ctx, top_k=top_k, span_len=12, window=8,
                               mode=mode) == (Hq, 0, 0)
    # head 0 made a near-tie by hand: key of the best rejected anchor := key of the k-th selected one;
    # a step that holds the rejected anchor instead must be compared on that alternative selection
    wide = O.span_search(q_s[:, :, None], hk, O.F32, top_k=top_k + 1, q_pos0=n_ctx - 1, window=8)
    t_k, t_rej = int(wide["anchor"][0, 0, 0, top_k - 1]), int(wide["anchor"][0, 0, 0, top_k])
    hk[0, 0, t_rej] = hk[0, 0, t_k]
    hk[0, 1, t_rej] = hk[0, 1, t_k]       # heads 2, 3 (other group) see the same edit; their selections are their own
    wide = O.span_search(q_s[:, :, None], hk, O.F32, top_k=top_k + 1, q_pos0=n_ctx - 1, window=8)
    assert wide["score"][0, 0, 0, top_k - 1] == wide["score"][0, 0, 0, top_k]       # an exact tie at rank k
    alt_sel = wide["anchor"][0, 0, 0, :top_k].copy()
    alt_sel[top_k - 1] = wide["anchor"][0, 0, 0, top_k]                              # the one the oracle leaves out
    sc = np.array([q_s[0, 0] @ hk[0, 0, t] for t in alt_sel])
    one = O.span_attention(q[:, :1, None], hk[:, :1], hv[:, :1], O.F32, alt_sel[None, None, None].astype(np.int32),
                           span_len=12, window=8, mode=mode, q_pos0=n_ctx - 1, score=sc[None, None, None])
    ref2 = O.decode_step(q_s, q, hk, hv, O.F32, n_ctx=n_ctx, top_k=top_k, span_len=12, window=8, mode=mode)
    out, lse, an, s = (np.asarray(ref2[n]).copy() for n in ("out", "lse", "anchor", "score"))
    out[0, 0], lse[0, 0], an[0, 0], s[0, 0] = one["out"][0, 0, 0], one["lse"][0, 0, 0], alt_sel, sc
    got = (torch.from_numpy(out.astype(np.float32)), torch.from_numpy(lse.astype(np.float32)),
           torch.from_numpy(an.astype(np.int32)), torch.from_numpy(s.astype(np.float32)))
    n_same, n_alt, n_out = P.check_decode_step(got, q_s, q, hk, hv, O.F32, "f32", n_ctx=n_ctx, top_k=top_k,
                                               span_len=12, window=8, mode=mode)
    assert (n_same, n_alt, n_out) == (Hq - 1, 1, 0)
