"""Sequence-sharded decode step on one GPU: the ranks' calls are run one after the other on slices of
the cache and the two exchanges are done by stacking, then the result is compared with the unsharded
step of the library and with the oracle's step."""
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


def run_sharded(sla, handle, x, kc, vc, n_ctx, params, world):
    from paper_2601_18401_b200 import sharded
    cap = kc.shape[2]
    parts = []
    for r in range(world):
        lo, ln = sharded.shard_range(cap, r, world)
        parts.append((lo, ln, kc[:, :, lo:lo + ln].contiguous() if ln else kc[:, :, :1].contiguous(),
                      vc[:, :, lo:lo + ln].contiguous() if ln else vc[:, :, :1].contiguous()))
    cands = [sla.sla_decode_shard_search(handle, x["q_s"], kl, lo, n_ctx, params, shard_len=ln)
             for lo, ln, kl, vl in parts]
    all_a = torch.stack([c[0] for c in cands]).contiguous()
    all_s = torch.stack([c[1] for c in cands]).contiguous()
    res = [sla.sla_decode_shard_attend(handle, x["q"], kl, vl, lo, n_ctx, params, all_a, all_s, shard_len=ln)
           for lo, ln, kl, vl in parts]
    for a, s, _ in res[1:]:                       # every rank arrives at the same selection
        assert torch.equal(a, res[0][0]) and torch.equal(s, res[0][1])
    all_p = torch.stack([r[2] for r in res]).contiguous()
    out, lse = sla.sla_decode_shard_merge(handle, all_p, x["q"])
    return out, lse, res[0][0], res[0][1]


@pytest.mark.parametrize("world", [1, 2, 3, 8])
@pytest.mark.parametrize("n_ctx0,span_len,top_k,dtype,D,Hq,Hkv,pexp", [
    (5000, 40, 4, "bf16", 128, 8, 2, 0.5),
    (3000, 0, 3, "bf16", 128, 4, 4, 0.5),
    (900, 16, 5, "f32", 64, 3, 1, 0.5),
    (4000, 0, 3, "bf16", 128, 8, 2, 1.0 / 3.0),
])
def test_sharded_step_equals_unsharded(sla, world, n_ctx0, span_len, top_k, dtype, D, Hq, Hkv, pexp):
    from paper_2601_18401_b200 import synth
    w = synth.Workload("sd", "decode", 2, Hq, Hkv, D, n_ctx0, dtype, span_len, top_k, seed=97)
    handle = sla.Handle(0, 64 << 20)
    kc, vc = synth.make_decode_cache(w, "cuda:0", capacity=n_ctx0 + 7)
    hk, hv = synth.to_numpy(kc), synth.to_numpy(vc)
    code = synth.dtype_code(dtype)
    back = 3 if pexp != 0.5 else 2
    params = sla.make_params(top_k, span_len, back, head_dim=D, search_exponent=pexp,
                             span_exponent=(1 - pexp) if pexp != 0.5 else 0.5)
    for s in range(2):
        x = synth.make_decode_step_inputs(w, s, "cuda:0")
        n_ctx = n_ctx0 + s + 1
        kc[:, :, n_ctx - 1] = x["k_new"]; vc[:, :, n_ctx - 1] = x["v_new"]
        hk[:, :, n_ctx - 1] = synth.to_numpy(x["k_new"]); hv[:, :, n_ctx - 1] = synth.to_numpy(x["v_new"])
        out, lse, anchor, score = run_sharded(sla, handle, x, kc, vc, n_ctx, params, world)
        ref_out, ref_lse, ref_anchor, ref_score = sla.sla_decode_step(handle, x["q_s"], x["q"], kc, vc, n_ctx, params)
        torch.cuda.synchronize()
        assert sla.sla_poll_status(handle) == sla.SLA_OK
        # same selection as the unsharded step, bit for bit; outputs up to the order of the merges
        assert torch.equal(anchor, ref_anchor) and torch.equal(score, ref_score)
        assert (out.float() - ref_out.float()).abs().max().item() <= (2.0 ** -6 if dtype == "bf16" else 1e-5)
        assert (lse - ref_lse).abs().max().item() <= 1e-4
        # and the oracle's own step
        P.check_decode_step((out, lse, anchor, score), synth.to_numpy(x["q_s"]), synth.to_numpy(x["q"]), hk, hv, code,
                            dtype, n_ctx=n_ctx, top_k=top_k, span_len=span_len, back_factor=back,
                            search_exponent=pexp, span_exponent=(1 - pexp) if pexp != 0.5 else 0.5)
    handle.close()
