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


def compare_search(anchor_gpu, score_gpu, ref, q_pos0=0, rows=None):
    """Selected anchors must equal the oracle's as sets on every clear-cut row; returns the number of
    exempt near-tie rows.  On every row the GPU's anchors must be valid candidates."""
    if rows is not None:   # slice on the device: the full tensors can be gigabytes
        idx = torch.as_tensor(np.asarray(rows), device=anchor_gpu.device)
        anchor_gpu, score_gpu = anchor_gpu[:, :, idx], score_gpu[:, :, idx]
    a = anchor_gpu.cpu().numpy()
    s = score_gpu.cpu().numpy().astype(np.float64)
    ra, rs, gap = ref["anchor"], ref["score"], ref["gap"]
    assert a.shape == ra.shape
    clear = gap > TIE_GAP
    same = np.all(np.sort(a, axis=-1) == np.sort(ra, axis=-1), axis=-1)
    bad = ~same & clear
    assert not bad.any(), f"{int(bad.sum())} clear-cut rows differ, first at {np.argwhere(bad)[0]}"
    # order and scores on rows that are clear-cut and whose selected scores are well separated
    sep = np.ones_like(clear)
    if ra.shape[-1] > 1:
        fin = np.where(np.isfinite(rs), rs, -1e30)
        sep = np.all(fin[..., :-1] - fin[..., 1:] > TIE_GAP, axis=-1) | np.all(np.isneginf(rs[..., 1:]), axis=-1)
    strict = clear & sep
    assert np.array_equal(a[strict], ra[strict]), "anchor order differs on well-separated rows"
    fin = np.isfinite(rs) & strict[..., None]
    np.testing.assert_allclose(s[fin], rs[fin], rtol=2e-5, atol=1e-3)
    assert np.all(np.isneginf(s[np.isneginf(rs) & strict[..., None]]))
    # validity everywhere: every anchor is -1 or i + 1 - m^2 for an integer m >= 1
    R = a.shape[2]
    pos = (np.arange(R) if rows is None else np.asarray(rows)) + q_pos0
    d = pos[None, None, :, None] + 1 - a.astype(np.int64)
    m = np.round(np.sqrt(np.maximum(d, 0))).astype(np.int64)
    assert np.all((a == -1) | ((m * m == d) & (m >= 1) & (a >= 0)))
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
        if o.size == 0:
            return 0.0, 0.0
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
