"""GPU parity of the two output modes and the local window (Algorithm 1: W = [max(0, i-w+1), i],
anchors inside W are no candidates, J_t = S_t united with W; Section "Combination": the softmax gate
over the selected anchors' search scores) against the oracle, element by element."""
import numpy as np
import pytest
import torch

import parity_util as P
from oracle import sla_oracle as O

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sla():
    import paper_2601_18401_b200 as sla_pkg
    return sla_pkg


@pytest.fixture(scope="module")
def handle(sla):
    h = sla.Handle(0, 256 << 20)
    sla.sla_set_debug_canaries(h, True)   # every attention and decode call of this module is checked for overruns
    yield h
    h.close()


def workload(**kw):
    from paper_2601_18401_b200 import synth
    base = synth.Workload("modes", "prefill", 1, 4, 2, 128, 1111, "bf16", 16, 4, seed=77)
    return base.scaled(**kw)


def run_modes(sla, handle, w, window, q_pos0=0):
    from paper_2601_18401_b200 import synth
    x = synth.make_prefill(w, device="cuda:0")
    L = w.seq_len
    q_s, q = x["q_s"][:, :, q_pos0:], x["q"][:, :, q_pos0:]
    host = P.host_inputs({"q_s": q_s, "q": q, "k": x["k"], "v": x["v"]})
    code = synth.dtype_code(w.dtype)
    # search: anchors inside the window are excluded
    pu = sla.make_params(w.top_k, w.span_len, w.back_factor, w.fwd_factor, window=window, head_dim=w.head_dim)
    anchor, score = sla.sla_span_search(handle, q_s, x["k"], pu, q_pos0=q_pos0)
    torch.cuda.synchronize()
    ref_s = O.span_search(host["q_s"], host["k"], code, top_k=w.top_k, q_pos0=q_pos0, window=window)
    P.compare_search(anchor, score, ref_s, q_pos0=q_pos0, q_s=host["q_s"], k=host["k"], window=window)
    a_gpu = anchor.cpu().numpy()
    inside = (a_gpu >= 0) & (a_gpu > (np.arange(q_pos0, L)[None, None, :, None] - window))
    assert not inside.any(), "an anchor inside the window was selected"
    kw = dict(span_len=w.span_len, back_factor=w.back_factor, fwd_factor=w.fwd_factor, window=window,
              q_pos0=q_pos0)
    # both attention modes run on the oracle's selection and scores, on both sides
    anchor = P.oracle_anchors_on_device(anchor, ref_s)
    score = torch.from_numpy(ref_s["score"].astype(np.float32)).to(anchor.device)
    # union mode: one softmax over spans and window
    out, lse = sla.sla_span_attention(handle, q, x["k"], x["v"], anchor, pu, q_pos0=q_pos0)
    torch.cuda.synchronize()
    ref_u = O.span_attention(host["q"], host["k"], host["v"], code, ref_s["anchor"], mode=O.UNION, **kw)
    P.compare_attention(out, lse, ref_u, w.dtype)
    # per-span mode with the gate
    pg = sla.make_params(w.top_k, w.span_len, w.back_factor, w.fwd_factor, window=window,
                         mode=sla.SLA_PER_SPAN, head_dim=w.head_dim)
    out_g, lse_g, lse_span = sla.sla_span_attention_gated(handle, q, x["k"], x["v"], anchor, score, pg,
                                                         q_pos0=q_pos0)
    torch.cuda.synchronize()
    assert sla.sla_poll_status(handle) == sla.SLA_OK
    ref_g = O.span_attention(host["q"], host["k"], host["v"], code, ref_s["anchor"], mode=O.PER_SPAN,
                             score=ref_s["score"], **kw)
    P.compare_attention(out_g, lse_g, ref_g, w.dtype)
    ls = lse_span.cpu().numpy().astype(np.float64)
    fin = np.isfinite(ref_g["lse_span"])
    assert np.array_equal(np.isneginf(ls), ~fin)
    assert not fin.any() or np.abs(ls[fin] - ref_g["lse_span"][fin]).max() <= P.LSE_TOL[w.dtype]
    return dict(out=out, out_g=out_g, anchor=anchor)


@pytest.mark.parametrize("window", [0, 8, 48, 300])
@pytest.mark.parametrize("kw", [
    dict(),                                                        # bf16 D128 GQA (tensor-core shapes)
    dict(dtype="f32", head_dim=64, n_q_heads=2, n_kv_heads=1, seq_len=700),
    dict(span_len=0, back_factor=4, fwd_factor=2, top_k=2),        # the paper's kernel settings
    dict(top_k=40, seq_len=300, span_len=5),                       # padding; rows with nothing selected
    dict(top_k=8, span_len=10, seq_len=777),                       # the largest k of the row-parallel gated merge
    dict(top_k=9, span_len=10, seq_len=777),                       # the smallest k of the general one
    dict(n_q_heads=8, n_kv_heads=2, top_k=6, span_len=14, seq_len=1400),   # groups of four query heads
])
def test_modes_and_window(sla, handle, kw, window):
    run_modes(sla, handle, workload(**kw), window)


def test_chunked_prefill_with_window(sla, handle):
    run_modes(sla, handle, workload(seq_len=1500), 100, q_pos0=900)


def test_single_anchor_modes_agree(sla, handle):
    """With top_k = 1 the gate is 1 and both modes compute the same attention (up to the rounding
    order of the two merge routines: one bf16 step)."""
    r = run_modes(sla, handle, workload(top_k=1, span_len=40), 24)
    assert (r["out"].float() - r["out_g"].float()).abs().max().item() <= 2.0 ** -5


@pytest.mark.parametrize("mode", ["union", "per_span"])
@pytest.mark.parametrize("window,n_ctx0,span_len,top_k,dtype,D,Hq,Hkv", [
    (0, 3000, 40, 4, "bf16", 128, 8, 2),
    (64, 3000, 40, 4, "bf16", 128, 8, 2),
    (1088, 5000, 0, 2, "bf16", 128, 4, 4),       # the paper's window; l(i) = ceil(sqrt(i))
    (100, 700, 16, 5, "f32", 64, 3, 1),
    (900, 800, 16, 3, "bf16", 128, 4, 2),        # window covers the whole context: nothing to select
])
def test_decode_modes_and_window(sla, handle, mode, window, n_ctx0, span_len, top_k, dtype, D, Hq, Hkv):
    """Decode step with the local window and in both modes against the oracle's decode step."""
    from paper_2601_18401_b200 import synth
    w = synth.Workload("dm", "decode", 2, Hq, Hkv, D, n_ctx0, dtype, span_len, top_k, seed=91)
    steps = 3
    kc, vc = synth.make_decode_cache(w, "cuda:0", capacity=n_ctx0 + steps)
    hk, hv = synth.to_numpy(kc), synth.to_numpy(vc)
    code = synth.dtype_code(dtype)
    m_gpu = sla.SLA_PER_SPAN if mode == "per_span" else sla.SLA_UNION
    m_ref = O.PER_SPAN if mode == "per_span" else O.UNION
    params = sla.make_params(top_k, span_len, window=window, mode=m_gpu, head_dim=D)
    for s in range(steps):
        x = synth.make_decode_step_inputs(w, s, "cuda:0")
        n_ctx = n_ctx0 + s + 1
        kc[:, :, n_ctx - 1] = x["k_new"]
        vc[:, :, n_ctx - 1] = x["v_new"]
        hk[:, :, n_ctx - 1] = synth.to_numpy(x["k_new"])
        hv[:, :, n_ctx - 1] = synth.to_numpy(x["v_new"])
        got = sla.sla_decode_step(handle, x["q_s"], x["q"], kc, vc, n_ctx, params)
        torch.cuda.synchronize()
        assert sla.sla_poll_status(handle) == sla.SLA_OK
        P.check_decode_step(got, synth.to_numpy(x["q_s"]), synth.to_numpy(x["q"]), hk, hv, code, dtype, n_ctx=n_ctx,
                            top_k=top_k, span_len=span_len, window=window, mode=m_ref)


def run_exponents(sla, handle, w, p_search, p_span, window=0, mode="union", top_k=None, back=2):
    """Search + attention with general exponents (anchors at i + 1 - ceil((s+1)^(1/p)), base length
    ceil(i^p_span)) against the oracle with the same exponents."""
    from paper_2601_18401_b200 import synth
    x = synth.make_prefill(w, device="cuda:0")
    host = P.host_inputs(x)
    code = synth.dtype_code(w.dtype)
    k_sel = top_k or w.top_k
    m_gpu = sla.SLA_PER_SPAN if mode == "per_span" else sla.SLA_UNION
    m_ref = O.PER_SPAN if mode == "per_span" else O.UNION
    params = sla.make_params(k_sel, w.span_len, back, w.fwd_factor, window=window, mode=m_gpu,
                             head_dim=w.head_dim, search_exponent=p_search, span_exponent=p_span)
    anchor, score = sla.sla_span_search(handle, x["q_s"], x["k"], params)
    torch.cuda.synchronize()
    ref_s = O.span_search(host["q_s"], host["k"], code, top_k=k_sel, window=window, search_exponent=p_search)
    # equal sets on clear-cut rows; on every row anchors on the stride pattern of p_search, outside the window
    P.compare_search(anchor, score, ref_s, q_s=host["q_s"], k=host["k"], window=window, search_exponent=p_search)
    kw = dict(span_len=w.span_len, back_factor=back, fwd_factor=w.fwd_factor, window=window, mode=m_ref,
              span_exponent=p_span, score=ref_s["score"])
    ref_a = O.span_attention(host["q"], host["k"], host["v"], code, ref_s["anchor"], **kw)
    # the attention runs on the oracle's selection and scores, on both sides
    anchor = P.oracle_anchors_on_device(anchor, ref_s)
    score = torch.from_numpy(ref_s["score"].astype(np.float32)).to(anchor.device)
    if mode == "per_span":
        out, lse, _ = sla.sla_span_attention_gated(handle, x["q"], x["k"], x["v"], anchor, score, params)
    else:
        out, lse = sla.sla_span_attention(handle, x["q"], x["k"], x["v"], anchor, params)
    torch.cuda.synchronize()
    assert sla.sla_poll_status(handle) == sla.SLA_OK
    P.compare_attention(out, lse, ref_a, w.dtype)
    return anchor, out, lse


@pytest.mark.parametrize("p_search,p_span", [(1.0 / 3.0, 2.0 / 3.0), (0.54, 0.54), (0.4, 0.5), (0.5, 0.6)])
@pytest.mark.parametrize("kw", [
    dict(span_len=0, top_k=3),                                          # bf16 D128 GQA, l(i) from the exponent
    dict(span_len=0, dtype="f32", head_dim=64, n_q_heads=2, n_kv_heads=1, seq_len=600, top_k=2),
    dict(span_len=12, top_k=4),                                         # fixed base length
    dict(span_len=0, top_k=5, n_q_heads=8, n_kv_heads=2, seq_len=1300),  # groups of four query heads
])
def test_general_exponents(sla, handle, kw, p_search, p_span):
    run_exponents(sla, handle, workload(**kw), p_search, p_span)


def test_general_exponents_with_window_and_gate(sla, handle):
    run_exponents(sla, handle, workload(span_len=0, top_k=2, seq_len=1500), 1.0 / 3.0, 2.0 / 3.0, window=100,
                  mode="per_span", back=3)
    run_exponents(sla, handle, workload(span_len=0, top_k=2, seq_len=900), 0.54, 0.54, window=64, mode="union")


def test_exponents_one_third_two_thirds_cover_everything(sla, handle):
    """All anchors selected, p = (1/3, 2/3), backward factor 3: the union attends to every key, so the
    result is dense causal attention (the coverage argument of Section "Span attention" for general p)."""
    from paper_2601_18401_b200 import synth
    w = workload(span_len=0, top_k=12, seq_len=900, n_q_heads=2, n_kv_heads=1)
    anchor, out, lse = run_exponents(sla, handle, w, 1.0 / 3.0, 2.0 / 3.0, back=3)
    x = synth.make_prefill(w, device="cuda:0")
    q, k, v = x["q"].float(), x["k"].float(), x["v"].float()
    k, v = k.repeat_interleave(2, dim=1), v.repeat_interleave(2, dim=1)
    ref = torch.nn.functional.scaled_dot_product_attention(q, k, v, is_causal=True)
    assert (out.float() - ref).abs().max().item() <= P.OUT_TOL["bf16"]


def test_decode_with_general_exponents(sla, handle):
    from paper_2601_18401_b200 import synth
    w = synth.Workload("de", "decode", 1, 8, 2, 128, 4000, "bf16", 0, 3, seed=93)
    kc, vc = synth.make_decode_cache(w, "cuda:0", capacity=4002)
    hk, hv = synth.to_numpy(kc), synth.to_numpy(vc)
    code = synth.dtype_code("bf16")
    for p_search, p_span, back in ((1.0 / 3.0, 2.0 / 3.0, 3), (0.54, 0.54, 2)):
        params = sla.make_params(3, 0, back, head_dim=128, search_exponent=p_search, span_exponent=p_span)
        x = synth.make_decode_step_inputs(w, 0, "cuda:0")
        n_ctx = 4001
        kc[:, :, n_ctx - 1] = x["k_new"]; vc[:, :, n_ctx - 1] = x["v_new"]
        hk[:, :, n_ctx - 1] = synth.to_numpy(x["k_new"]); hv[:, :, n_ctx - 1] = synth.to_numpy(x["v_new"])
        got = sla.sla_decode_step(handle, x["q_s"], x["q"], kc, vc, n_ctx, params)
        torch.cuda.synchronize()
        P.check_decode_step(got, synth.to_numpy(x["q_s"]), synth.to_numpy(x["q"]), hk, hv, code, "bf16", n_ctx=n_ctx,
                            top_k=3, span_len=0, back_factor=back, search_exponent=p_search, span_exponent=p_span)


def test_pattern_tables_follow_a_change_of_stream(sla):
    """The handle copies its stride table to the device on the stream of the call that builds it; a call with
    the same exponent that follows on another stream (no dependency between the streams) must still see
    the complete table: the library orders the two itself."""
    from paper_2601_18401_b200 import synth
    w = workload(span_len=0, top_k=3, seq_len=60000, n_q_heads=4, n_kv_heads=1)
    x = synth.make_prefill(w, device="cuda:0")
    params = sla.make_params(3, 0, 3, head_dim=128, search_exponent=1.0 / 3.0, span_exponent=2.0 / 3.0)
    torch.cuda.synchronize()
    results = []
    for rep in range(3):
        h = sla.Handle(0, 64 << 20)          # a fresh handle: the table is built by the first call
        s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
        with torch.cuda.stream(s1):
            a1, v1 = sla.sla_span_search(h, x["q_s"], x["k"], params)
        with torch.cuda.stream(s2):
            a2, v2 = sla.sla_span_search(h, x["q_s"], x["k"], params)
        torch.cuda.synchronize()
        assert torch.equal(a1, a2) and torch.equal(v1, v2)
        results.append(a1)
        h.close()
    assert torch.equal(results[0], results[1]) and torch.equal(results[0], results[2])
    host = P.host_inputs(x)
    rows = np.unique(np.random.default_rng(3).integers(0, w.seq_len, 300))
    ref = O.span_search(host["q_s"], host["k"], O.BF16, top_k=3, search_exponent=1.0 / 3.0, rows=rows)
    P.compare_search(results[0], v1, ref, rows=rows, q_s=host["q_s"], k=host["k"], search_exponent=1.0 / 3.0)
