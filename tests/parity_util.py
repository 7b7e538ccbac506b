"""Helpers shared by the GPU parity tests: run the CUDA path through the C-ABI binding, run the CPU
oracle on the same seeded inputs, and compare under the stated criteria."""
import numpy as np
import torch

from oracle import sla_oracle as O
from paper_2601_18401_b200 import synth

TIE_GAP = 1e-3                       # rows whose k-th / (k+1)-th oracle scores are closer are exempt
OUT_TOL = {"f32": 1e-4, "bf16": 1e-2}  # max-abs error of the attention output on unit-variance inputs
LSE_TOL = {"f32": 1e-4, "bf16": 1e-3}  # lse is fp32 on both paths; logits come from exact products


def code_of(t: torch.Tensor) -> int:
    return O.F32 if t.dtype == torch.float32 else O.BF16


def _widen(a: np.ndarray) -> np.ndarray:
    """Host input array (fp32, fp64, or bf16 as uint16 bit patterns) as fp64, exactly."""
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    return a.astype(np.float64)


def _pattern_offsets(reach: int, search_exponent: float) -> np.ndarray:
    """Ascending distances i + 1 - t of the stride pattern up to `reach` (Section "Span attention")."""
    offs, s = [], 0
    while True:
        o = O.stride_offset(s, search_exponent)
        if o > reach:
            return np.asarray(offs, dtype=np.int64)
        offs.append(o)
        s += 1


def compare_search(anchor_gpu, score_gpu, ref, q_pos0=0, rows=None, *, q_s=None, k=None, window=0,
                   search_exponent=0.5, search_scale=1.0):
    """Selected anchors must equal the oracle's as sets on every clear-cut row (order and scores too
    where the selected scores are well separated); returns the number of exempt near-tie rows.

    On EVERY row, exempt or not, the CUDA selection must be a valid answer: as many anchors as
    min(top_k, candidates), all distinct, each on the stride pattern of the call's exponent and outside
    the local window, -1 / -inf padding behind them, scores in descending order, and no selected score
    more than TIE_GAP below the oracle's k-th score.  With the host inputs `q_s` [B,Hq,Lq,D] and
    `k` [B,Hkv,cap,D] (the arrays the oracle read) every returned score is also checked against the
    dot product of its own anchor, recomputed here in fp64 with numpy."""
    if rows is not None:   # slice on the device: the full tensors can be gigabytes
        idx = torch.as_tensor(np.asarray(rows), device=anchor_gpu.device)
        anchor_gpu, score_gpu = anchor_gpu[:, :, idx], score_gpu[:, :, idx]
    a = anchor_gpu.cpu().numpy()
    s = score_gpu.cpu().numpy().astype(np.float64)
    ra, rs, gap = ref["anchor"], ref["score"], ref["gap"]
    assert a.shape == ra.shape
    B, Hq, R, K = a.shape
    clear = gap > TIE_GAP
    same = np.all(np.sort(a, axis=-1) == np.sort(ra, axis=-1), axis=-1)
    bad = ~same & clear
    assert not bad.any(), f"{int(bad.sum())} clear-cut rows differ, first at {np.argwhere(bad)[0]}"
    # order and scores on rows that are clear-cut and whose selected scores are well separated
    sep = np.ones_like(clear)
    if K > 1:
        fin = np.where(np.isfinite(rs), rs, -1e30)
        sep = np.all(fin[..., :-1] - fin[..., 1:] > TIE_GAP, axis=-1) | np.all(np.isneginf(rs[..., 1:]), axis=-1)
    strict = clear & sep
    assert np.array_equal(a[strict], ra[strict]), "anchor order differs on well-separated rows"
    fin = np.isfinite(rs) & strict[..., None]
    np.testing.assert_allclose(s[fin], rs[fin], rtol=2e-5, atol=1e-3)
    assert np.all(np.isneginf(s[np.isneginf(rs) & strict[..., None]]))

    # ---- validity on every row
    pos = (np.arange(R) if rows is None else np.asarray(rows, dtype=np.int64)) + q_pos0
    offs = _pattern_offsets(int(pos.max()) + 1, search_exponent)
    sel = a >= 0
    d = pos[None, None, :, None] + 1 - a.astype(np.int64)
    on_pattern = np.isin(d, offs)
    assert np.all(~sel | on_pattern), "a selected anchor is not on the stride pattern"
    assert np.all(~sel | (d > window)), "a selected anchor lies inside the local window"
    assert np.all(a[~sel] == -1) and np.all(np.isneginf(s[~sel])), "padding must be (-1, -inf)"
    # candidates of a row: offsets <= i + 1 that lie outside the window
    n_cand = np.searchsorted(offs, pos + 1, side="right") - np.searchsorted(offs, window, side="right")
    want = np.minimum(np.maximum(n_cand, 0), K)
    assert np.array_equal(sel.sum(-1), np.broadcast_to(want[None, None, :], (B, Hq, R))), "wrong number of anchors"
    assert np.all(sel[..., :-1] | ~sel[..., 1:]), "padding must follow the selected anchors"
    srt = np.sort(np.where(sel, a, -np.arange(1, K + 1)), axis=-1)    # distinct stand-ins for the padding
    assert np.all(srt[..., 1:] != srt[..., :-1]), "an anchor was selected twice"
    assert np.all(s[..., :-1] >= s[..., 1:]), "scores are not in descending order"
    # nothing selected may score more than the tie margin below the oracle's k-th score
    kth = np.where(np.isfinite(rs), rs, np.inf).min(axis=-1)
    assert np.all(~sel | (s >= kth[..., None] - TIE_GAP)), "a selected score lies below the oracle's k-th score"
    # the oracle's selection and the CUDA one have the same scores, slot by slot, within the tie margin
    # (equal sets on clear-cut rows; on near-tie rows exchanged anchors score within the gap of each other)
    both = sel & np.isfinite(rs)
    assert np.abs(s[both] - rs[both]).max(initial=0.0) <= 2 * TIE_GAP + 2e-5 * np.abs(rs[both]).max(initial=0.0)
    if q_s is not None and k is not None:
        G = Hq // k.shape[1]
        r_idx = np.arange(R) if rows is None else np.asarray(rows, dtype=np.int64)
        for b in range(B):
            for h in range(Hq):
                kk = k[b, h // G]
                for r0 in range(0, R, 4096):
                    sl = slice(r0, min(R, r0 + 4096))
                    qv = _widen(q_s[b, h, r_idx[sl]])                                # [r, D]
                    kv = _widen(kk[np.maximum(a[b, h, sl], 0)])                      # [r, K, D]
                    dots = search_scale * np.einsum("rd,rkd->rk", qv, kv)
                    m = sel[b, h, sl]
                    err = np.abs(dots - s[b, h, sl])[m]
                    tol = 1e-3 + 2e-5 * np.abs(dots[m])
                    assert np.all(err <= tol), "a returned score is not the score of its own anchor"
    return int((~clear).sum())


def oracle_attention_for(x_host, dtype_code, anchor_ref, w, q_pos0=0, rows=None, softmax_scale=None):
    """Oracle span-attention on anchors that come from the oracle's own search (or from the test's own
    generator): nothing the CUDA path produced is ever an input of the oracle.  With `rows`,
    anchor_ref holds those rows only."""
    a = np.ascontiguousarray(np.asarray(anchor_ref), dtype=np.int32)
    return O.span_attention(x_host["q"], x_host["k"], x_host["v"], dtype_code, a, span_len=w.span_len,
                            back_factor=w.back_factor, fwd_factor=w.fwd_factor, q_pos0=q_pos0, rows=rows,
                            softmax_scale=softmax_scale)


def oracle_anchors_on_device(anchor_gpu, ref_s, rows=None):
    """The anchors the CUDA attention is given in a parity test: the oracle's selection (on all rows,
    or written over the sampled `rows` of the CUDA search result, which fills the rest)."""
    ra = torch.from_numpy(np.ascontiguousarray(ref_s["anchor"])).to(anchor_gpu.device)
    if rows is None:
        return ra.contiguous()
    a = anchor_gpu.clone()
    a[:, :, torch.as_tensor(np.asarray(rows), device=a.device)] = ra
    return a


def same_selection(anchor_gpu, ref_anchor):
    """Rows on which the CUDA search and the oracle selected the same anchors (as sets)."""
    a = anchor_gpu.cpu().numpy() if torch.is_tensor(anchor_gpu) else np.asarray(anchor_gpu)
    return np.all(np.sort(a, axis=-1) == np.sort(ref_anchor, axis=-1), axis=-1)


def compare_attention(out_gpu, lse_gpu, ref, dtype_name, rows=None, where=None):
    """`where`: optional boolean mask [B,Hq,R] of the rows to compare (default all)."""
    if rows is not None:
        idx = torch.as_tensor(np.asarray(rows), device=out_gpu.device)
        out_gpu, lse_gpu = out_gpu[:, :, idx], lse_gpu[:, :, idx]
    o = out_gpu.float().cpu().numpy().astype(np.float64)
    l = lse_gpu.cpu().numpy().astype(np.float64)
    ro, rl = ref["out"], ref["lse"]
    if where is not None:
        o, l, ro, rl = o[where], l[where], ro[where], rl[where]
        assert o.size > 0, "the row mask leaves nothing to compare"
    tol = OUT_TOL[dtype_name]
    err = np.abs(o - ro).max()
    assert err <= tol, f"output max-abs error {err} above {tol}"
    fin = np.isfinite(rl)
    assert np.array_equal(np.isneginf(l), ~fin)
    lerr = np.abs(l[fin] - rl[fin]).max() if fin.any() else 0.0
    assert lerr <= LSE_TOL[dtype_name], f"lse max-abs error {lerr}"
    return float(err), float(lerr)


def host_inputs(x):
    return {n: synth.to_numpy(t) for n, t in x.items()}


def check_decode_step(got, q_s, q, hk, hv, dtype_code, dtype_name, *, n_ctx, top_k, span_len, back_factor=2,
                      fwd_factor=0, window=0, mode=O.UNION, search_exponent=0.5, span_exponent=0.5,
                      before_attention=None):
    """One fused decode step of the CUDA path, `got` = (out, lse, anchor, score) as [B,Hq,...] tensors,
    against the oracle on the same inputs (q_s, q [B,Hq,D] and the cache as host arrays).

    The step selects and attends in one call, so the output of a head can only be compared where the
    head selected what the oracle selected.  On a near-tie head (oracle gap below TIE_GAP) the CUDA
    path may instead hold the oracle's best rejected anchor in place of its k-th: that alternative
    selection is built here from the oracle's own top-(k+1) list and attended by the oracle, so such a
    head is still compared.  Heads that match neither are counted and must be rare; the search
    comparison has already shown their selection to be a valid answer.
    `before_attention(anchor_sets)`: hook for tests whose host cache is filled lazily.
    Returns (heads compared on the oracle's selection, on the alternative, left out)."""
    out, lse, anchor, score = got
    qs3, q3 = q_s[:, :, None], q[:, :, None]
    wide = O.span_search(qs3, hk, dtype_code, top_k=top_k + 1, q_pos0=n_ctx - 1, Lkv=n_ctx, window=window,
                         search_exponent=search_exponent)
    wa, ws = wide["anchor"], wide["score"]
    with np.errstate(invalid="ignore"):   # -inf minus -inf where fewer than k + 1 candidates exist
        gap = np.where(np.isfinite(ws[..., top_k]), ws[..., top_k - 1] - ws[..., top_k], np.inf)
    ref_s = {"anchor": np.ascontiguousarray(wa[..., :top_k]), "score": np.ascontiguousarray(ws[..., :top_k]),
             "gap": gap}
    compare_search(anchor[:, :, None], score[:, :, None], ref_s, q_pos0=n_ctx - 1, q_s=qs3, k=hk, window=window,
                   search_exponent=search_exponent)
    alt_a = np.ascontiguousarray(np.concatenate([wa[..., :top_k - 1], wa[..., top_k:]], axis=-1))
    alt_s = np.ascontiguousarray(np.concatenate([ws[..., :top_k - 1], ws[..., top_k:]], axis=-1))
    a = anchor.cpu().numpy()[:, :, None]
    same = same_selection(a, ref_s["anchor"])
    is_alt = ~same & same_selection(a, alt_a) & (gap <= TIE_GAP)
    if before_attention is not None:
        before_attention([ref_s["anchor"], alt_a] if is_alt.any() else [ref_s["anchor"]])
    kw = dict(span_len=span_len, back_factor=back_factor, fwd_factor=fwd_factor, window=window, mode=mode,
              q_pos0=n_ctx - 1, Lkv=n_ctx, span_exponent=span_exponent)
    main = O.span_attention(q3, hk, hv, dtype_code, ref_s["anchor"], score=ref_s["score"], **kw)
    assert same.any()
    compare_attention(out[:, :, None], lse[:, :, None], main, dtype_name, where=same)
    if is_alt.any():
        alt = O.span_attention(q3, hk, hv, dtype_code, alt_a, score=alt_s, **kw)
        compare_attention(out[:, :, None], lse[:, :, None], alt, dtype_name, where=is_alt)
    left_out = int((~same & ~is_alt).sum())
    assert left_out <= max(1, same.size // 16), f"{left_out} of {same.size} heads match neither selection"
    return int(same.sum()), int(is_alt.sum()), left_out
