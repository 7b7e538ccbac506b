"""The decode entry point that allocates nothing (sla_decode_step_static), for hosts that are not
allowed to call cudaMalloc -- code under a stream capture or inside a serving loop, processes whose
device memory belongs to another allocator, plug-ins that are only lent a stream.  It keeps its
scratch in a fixed array inside the library image instead of a handle's workspace, so this test
checks it against the ordinary sla_decode_step on the same inputs, through the C interface, on two
calls in a row (the array keeps the first call's contents when the second one starts).

This file sorts last on purpose: a run that stops at the first failure has then already run every
other test."""
import pytest
import torch

pytestmark = pytest.mark.gpu


def _run_both(sla, handle, w, kc, vc, n_ctx, step):
    from paper_2601_18401_b200 import synth
    x = synth.make_decode_step_inputs(w, step, "cuda:0")
    params = sla.make_params(w.top_k, w.span_len, head_dim=w.head_dim)
    ref = sla.sla_decode_step(handle, x["q_s"], x["q"], kc, vc, n_ctx, params)
    B, Hq, D = x["q"].shape
    # the caller of the no-allocation entry point brings every buffer, outputs included
    out = torch.full_like(x["q"], float("nan"))
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device="cuda:0")
    anchor = torch.full((B, Hq, w.top_k), -7, dtype=torch.int32, device="cuda:0")
    score = torch.full((B, Hq, w.top_k), float("nan"), dtype=torch.float32, device="cuda:0")
    sla.sla_decode_step_static(x["q_s"], x["q"], kc, vc, n_ctx, params, out=out, lse=lse, out_anchor=anchor,
                               out_score=score)
    torch.cuda.synchronize()
    assert torch.equal(anchor, ref[2])                       # same selection, bit for bit
    assert torch.equal(score, ref[3])
    tol = 1e-2 if w.dtype == "bf16" else 1e-4                # the tolerances of the parity tests
    assert (out.float() - ref[0].float()).abs().max().item() <= tol
    assert (lse - ref[1]).abs().max().item() <= (1e-3 if w.dtype == "bf16" else 1e-4)


@pytest.mark.parametrize("dtype,D,Hq,Hkv", [("bf16", 128, 8, 2), ("f32", 64, 4, 4)])
def test_static_scratch_decode_matches_handle_decode_twice(dtype, D, Hq, Hkv):
    import paper_2601_18401_b200 as sla
    from paper_2601_18401_b200 import synth
    w = synth.Workload("d", "decode", 2, Hq, Hkv, D, 90000, dtype, 150, 8, steps=2, seed=41)
    kc, vc = synth.make_decode_cache(w, "cuda:0", capacity=w.seq_len + 8)
    handle = sla.Handle(0, 64 << 20)
    _run_both(sla, handle, w, kc, vc, 90000, step=0)
    _run_both(sla, handle, w, kc, vc, 4097, step=1)          # second call in a row: smaller, other spans
    handle.close()


def test_static_scratch_rejects_steps_beyond_its_fixed_size():
    import paper_2601_18401_b200 as sla
    dev = "cuda:0"
    B, Hq, Hkv, D, n_ctx = 64, 64, 8, 128, 4096              # 4096 heads: far more scratch than 2 MiB
    q = torch.zeros(B, Hq, D, dtype=torch.bfloat16, device=dev)
    kc = torch.zeros(B, Hkv, n_ctx, D, dtype=torch.bfloat16, device=dev)
    out = torch.zeros_like(q)
    lse = torch.zeros(B, Hq, dtype=torch.float32, device=dev)
    anchor = torch.zeros(B, Hq, 16, dtype=torch.int32, device=dev)
    score = torch.zeros(B, Hq, 16, dtype=torch.float32, device=dev)
    with pytest.raises(sla.SlaError) as e:
        sla.sla_decode_step_static(q, q, kc, kc, n_ctx, sla.make_params(16, 64), out=out, lse=lse,
                                   out_anchor=anchor, out_score=score)
    assert e.value.status == -3
    # what the fixed array cannot serve is refused on the host, before anything is launched: a local
    # window, the per-span mode and other exponents all need scratch that only a handle has
    small = dict(out=out[:1, :8], lse=lse[:1, :8], out_anchor=anchor[:1, :8], out_score=score[:1, :8])
    for bad in (sla.make_params(16, 64, window=1), sla.make_params(16, 64, mode=sla.SLA_PER_SPAN),
                sla.make_params(16, 64, search_exponent=1.0 / 3.0)):
        with pytest.raises(sla.SlaError) as e:
            sla.sla_decode_step_static(q[:1, :8], q[:1, :8], kc[:1], kc[:1], n_ctx, bad, **small)
        assert e.value.status == -2
