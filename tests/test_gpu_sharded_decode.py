"""Sequence-sharded decode step.  On one GPU in one process: the ranks' calls are run one after the other
on slices of the cache and the two exchanges are done by stacking.  As two processes (both on the one
GPU, a gloo group between them): every rank holds half of the cache and calls the package's
decode_step_sharded, which does the two all-gathers.  Either way the result is compared with the
unsharded step of the library and with the oracle's step."""
import os
import sys

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
    if world == 1:   # the function a user calls, as a single rank
        return sharded.decode_step_sharded(handle, x["q_s"], x["q"], kc, vc, 0, n_ctx, params, shard_len=cap)
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


def _rank_main(rank, world, port, n_ctx0, out_q):
    """One rank of the two-process run: its own process, CUDA context and handle on device 0."""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    for p in (root, os.path.join(root, "tests")):
        if p not in sys.path:
            sys.path.insert(0, p)
    import torch.distributed as dist
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import paper_2601_18401_b200 as sla
    from paper_2601_18401_b200 import sharded, synth
    torch.cuda.set_device(0)
    w = synth.Workload("sd2", "decode", 1, 8, 2, 128, n_ctx0, "bf16", 150, 8, seed=131)
    steps = 2
    kc, vc = synth.make_decode_cache(w, "cuda:0", capacity=n_ctx0 + steps)    # same seed: the same cache on every rank
    lo, ln = sharded.shard_range(n_ctx0 + steps, rank, world)
    handle = sla.Handle(0, 64 << 20)
    params = sla.make_params(w.top_k, w.span_len, head_dim=128)
    res = []
    for s in range(steps):
        x = synth.make_decode_step_inputs(w, s, "cuda:0")
        n_ctx = n_ctx0 + s + 1
        kc[:, :, n_ctx - 1] = x["k_new"]
        vc[:, :, n_ctx - 1] = x["v_new"]
        # the rank keeps only its slice of the cache
        k_loc, v_loc = kc[:, :, lo:lo + ln].contiguous(), vc[:, :, lo:lo + ln].contiguous()
        out, lse, anchor, score = sharded.decode_step_sharded(handle, x["q_s"], x["q"], k_loc, v_loc, lo, n_ctx, params,
                                                              shard_len=ln)
        torch.cuda.synchronize()
        assert sla.sla_poll_status(handle) == sla.SLA_OK
        res.append(tuple(t.cpu() for t in (out.float(), lse, anchor, score)))
    dist.barrier()
    out_q.put((rank, res))
    dist.barrier()
    dist.destroy_process_group()
    handle.close()


def test_two_processes_each_with_half_of_the_cache(sla):
    """decode_step_sharded as a user runs it: two ranks, two processes, a process group between them; each
    holds half of a 100,000-token cache.  Both ranks must return the unsharded step's selection bit for bit
    and its output to rounding, and the oracle's step within the parity bounds."""
    import torch.multiprocessing as mp
    from paper_2601_18401_b200 import synth
    n_ctx0, world = 100000, 2
    ctx = mp.get_context("spawn")
    out_q = ctx.Queue()
    port = 31500 + os.getpid() % 1000
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, n_ctx0, out_q)) for r in range(world)]
    for p in procs:
        p.start()
    got = dict(out_q.get(timeout=300) for _ in procs)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    # the same steps, unsharded, in this process
    w = synth.Workload("sd2", "decode", 1, 8, 2, 128, n_ctx0, "bf16", 150, 8, seed=131)
    kc, vc = synth.make_decode_cache(w, "cuda:0", capacity=n_ctx0 + 2)
    hk, hv = synth.to_numpy(kc), synth.to_numpy(vc)
    handle = sla.Handle(0, 64 << 20)
    params = sla.make_params(w.top_k, w.span_len, head_dim=128)
    for s in range(2):
        x = synth.make_decode_step_inputs(w, s, "cuda:0")
        n_ctx = n_ctx0 + s + 1
        kc[:, :, n_ctx - 1] = x["k_new"]; vc[:, :, n_ctx - 1] = x["v_new"]
        hk[:, :, n_ctx - 1] = synth.to_numpy(x["k_new"]); hv[:, :, n_ctx - 1] = synth.to_numpy(x["v_new"])
        ref_out, ref_lse, ref_anchor, ref_score = sla.sla_decode_step(handle, x["q_s"], x["q"], kc, vc, n_ctx, params)
        torch.cuda.synchronize()
        for rank in range(world):
            out, lse, anchor, score = got[rank][s]
            assert torch.equal(anchor, ref_anchor.cpu()) and torch.equal(score, ref_score.cpu())
            assert (out - ref_out.float().cpu()).abs().max().item() <= 2.0 ** -6
            assert (lse - ref_lse.cpu()).abs().max().item() <= 1e-4
        out, lse, anchor, score = (t.cuda() for t in got[0][s])
        P.check_decode_step((out, lse, anchor, score), synth.to_numpy(x["q_s"]), synth.to_numpy(x["q"]), hk, hv,
                            synth.dtype_code("bf16"), "bf16", n_ctx=n_ctx, top_k=w.top_k, span_len=w.span_len)
    handle.close()
