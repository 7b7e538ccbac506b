#!/usr/bin/env python
"""Benchmark of the span-search + span-attention hot path on B200.

One "step" is one pass of the prefill hot path -- sla_span_search followed by sla_span_attention --
over one batch of seeded synthetic input of the second benchmark configuration (batch 1, 32 query /
8 KV heads, head_dim 128, L = 65536, bf16, 16 planted key spans per head, span length 256, top_k 8).
The headline value is prefill tokens/s per attention layer with the inputs resident in HBM; the
same run also measures the end-to-end figure through the host-buffer C call, the decode step at
1M and 10M context (microseconds per token per layer), the roofline fractions, and the CPU oracle
on a bounded sample as a baseline.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (launched under torchrun, one rank per GPU) every rank runs the same workload on its own
sequence -- the path shards over independent sequences with no exchange step -- and the value is
the total over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2601_18401_b200 import synth

METRIC = "prefill_tokens_per_s_per_layer"
UNIT = "tokens/s"
# dram__bytes_read.sum + dram__bytes_write.sum of one tc_attend launch of the default workload
# (L = 65536): a CONSTANT taken from the one-pass ncu capture of the full-size launch summarised in
# the profiles folder, not something this run measures
TC_ATTEND_DRAM_BYTES_PER_LAUNCH = {65536: 4.74e9, 16384: 0.887e9}
TRAFFIC_SOURCE = "constant from the one-pass ncu capture summarised under profiles/, not measured by this run"
NOMINAL_BF16_TFLOPS = 2250.0   # dense bf16, per GPU
# the same for one decode_attn launch (the dominant kernel of a decode step), by workload
DECODE_ATTN_DRAM_BYTES_PER_LAUNCH = {"decode_1M": 485.2e6, "decode_10M": 1571.4e6}
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def tensor_roofline(flops, kern_ms, region_s, clocks, peaks):
    """Roofline entry of a tensor-core kernel.  The denominator is the measured burst rate of a bf16
    matmul when the timed region is short (under a second) or the sampled SM clock stayed at 95 % of
    its maximum or more -- the conditions under which the burst figure was measured -- and the
    sustained rate (measured over seconds under the power cap) otherwise; both fractions and the one
    of the nominal dense peak are given beside it."""
    tflops = flops / (kern_ms * 1e-3) / 1e12
    burst, sustained = peaks["bf16_tflops"], peaks["bf16_tflops_sustained"]
    mhz, mx = clocks.get("sm_mhz"), clocks.get("sm_max_mhz")
    at_full_clock = bool(mhz and mx and mhz >= 0.95 * mx)
    use_burst = region_s < 1.0 or at_full_clock
    peak = burst if use_burst else sustained
    return {"bound": "tensor", "achieved": tflops, "peak": peak, "unit": "TFLOP/s", "frac": tflops / peak,
            "frac_of_burst": tflops / burst, "frac_of_sustained": tflops / sustained,
            "frac_of_nominal": tflops / NOMINAL_BF16_TFLOPS, "nominal_peak": NOMINAL_BF16_TFLOPS,
            "peak_rule": ("burst" if use_burst else "sustained") + f": timed region {region_s:.2f} s, median SM clock "
                         f"{mhz} of {mx} MHz",
            "ms_times_sm_mhz": (kern_ms * mhz) if mhz else None,
            "flops_per_launch": flops, "ms_per_launch": kern_ms, "peak_source": peaks["_source"]}


def search_key_bytes(B, Hkv, L, D, elem, window=0):
    """Algorithmic bytes of the span-search kernel's dominant stream: one key row per (position, stride,
    KV head) -- sum over i of the number of candidate strides floor(sqrt(i+1)) - floor(sqrt(w))."""
    i = np.arange(1, L + 1, dtype=np.float64)
    n = np.floor(np.sqrt(i)).astype(np.int64)
    n = np.where((n * n > i), n - 1, n)
    n = np.where(((n + 1) * (n + 1) <= i), n + 1, n)
    n = np.maximum(n - int(np.floor(np.sqrt(window))), 0)
    return int(n.sum()) * B * Hkv * D * elem


def measure_l2_probe(sla, handle, dev, mib=32, iters=2, reps=5):
    """GB/s of the library's read-only L2 probe over an L2-resident buffer."""
    buf = torch.empty(mib << 20, dtype=torch.uint8, device=dev).zero_()
    for _ in range(3):
        nbytes = sla.sla_probe_l2_read(handle, buf, iters)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(reps):
        sla.sla_probe_l2_read(handle, buf, iters)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / reps
    return {"gbs": nbytes / (ms * 1e-3) / 1e9, "buffer_mib": mib, "bytes_per_launch": nbytes, "ms_per_launch": ms,
            "how": "every CTA of a 4 x SM-count grid reads the whole buffer with 32-byte loads"}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        p["_source"] = "measured"
        return p
    p = dict(FALLBACK_PEAKS)
    p["_source"] = "fallback"
    return p


# ------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) in a background thread during
    the timed region; falls back to one nvidia-smi query when NVML is not importable."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, index: int):
        self.index, self.samples, self.masks, self.max_mhz = index, [], [], None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                self.masks.append(int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)))
            except Exception:
                pass
            time.sleep(0.004)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        if self.nv is None:
            try:
                out = subprocess.run(["nvidia-smi", f"--id={self.index}", "--query-gpu=clocks.sm,clocks.max.sm",
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True).stdout
                a, b = [float(x) for x in out.strip().split(",")]
                return {"sm_mhz": a, "sm_max_mhz": b, "reasons": ["nvml unavailable: one nvidia-smi sample after the run"]}
            except Exception:
                return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no clock source"]}
        self._stop.set()
        self._thread.join(timeout=1.0)
        reasons = sorted({name for m in self.masks for bit, name in self.REASONS.items() if m & bit})
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": reasons, "samples": len(self.samples)}


# ------------------------------------------------------------------------------------ bookkeeping
def attended_pairs(anchor: torch.Tensor, span_len: int, back: int, fwd: int) -> int:
    """(query, key) pairs the union of the selected spans holds -- bookkeeping for the FLOP count
    (4 * head_dim per pair), computed with torch ops from the anchors the search produced."""
    B, H, L, K = anchor.shape
    i = torch.arange(L, device=anchor.device, dtype=torch.int64)[None, None, :, None]
    t = anchor.to(torch.int64)
    lo = torch.clamp(t - back * span_len, min=0)
    hi = torch.minimum(t + fwd * span_len, i.expand_as(t))
    valid = t >= 0
    lo = torch.where(valid, lo, torch.full_like(lo, 1 << 40))
    hi = torch.where(valid, hi, torch.full_like(hi, -1))
    lo, order = torch.sort(lo, dim=-1)
    hi = torch.gather(hi, -1, order)
    run_hi = torch.cummax(hi, dim=-1).values
    prev = torch.cat([torch.full_like(run_hi[..., :1], -1), run_hi[..., :-1]], dim=-1)
    start = torch.maximum(lo, prev + 1)
    return int(torch.clamp(hi - start + 1, min=0).sum().item())


def config_of(w, world: int):
    """The `config` object of the JSON line: the same for both arms, so that they can be matched."""
    return {"workload": w.name, "batch_per_gpu": w.batch, "q_heads": w.n_q_heads, "kv_heads": w.n_kv_heads,
            "head_dim": w.head_dim, "seq_len": w.seq_len, "span_len": w.span_len, "top_k": w.top_k,
            "back_factor": w.back_factor, "fwd_factor": w.fwd_factor, "planted_spans": w.planted_spans,
            "l2": "inputs (1.3 GB) exceed the 126 MB L2; no flush between steps",
            "parallelism": f"independent sequences x{world}"}


def oracle_sample_rows(L: int, n: int):
    return np.unique(np.linspace(0, L - 1, n).astype(np.int64))


def time_oracle_prefill(w, host, rows):
    """Runs the CPU oracle (search + attention) on `rows` of every head; returns seconds."""
    from oracle import sla_oracle as O
    code = synth.dtype_code(w.dtype)
    t0 = time.perf_counter()
    s = O.span_search(host["q_s"], host["k"], code, top_k=w.top_k, rows=rows)
    O.span_attention(host["q"], host["k"], host["v"], code, s["anchor"], span_len=w.span_len,
                     back_factor=w.back_factor, fwd_factor=w.fwd_factor, rows=rows)
    return time.perf_counter() - t0


# ------------------------------------------------------------------------------------ arms
def run_reference(args, w):
    """The CPU oracle as it stands, on host cores, on a bounded row sample per step."""
    from oracle import sla_oracle as O
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    x = synth.make_prefill(w, device="cpu")
    host = {n: synth.to_numpy(t) for n, t in x.items()}
    # the sample of one step is bounded so that the whole run stays near 150 s of oracle time: a
    # calibration pass on 256 positions gives the rate, the per-step sample follows from it
    calib = oracle_sample_rows(w.seq_len, 256)
    rate = len(calib) / time_oracle_prefill(w, host, calib)
    n_rows = int(min(args.ref_rows, max(64, 150.0 * rate / max(1, args.steps))))
    rows = oracle_sample_rows(w.seq_len, n_rows)
    for _ in range(args.warmup):
        time_oracle_prefill(w, host, rows[: max(4, len(rows) // 16)])
    secs = [time_oracle_prefill(w, host, rows) for _ in range(args.steps)]
    per_step = float(np.mean(secs))
    value = len(rows) * w.batch / per_step
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(w, args.gpus),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": O.threads(), "kind": "oracle",
                         "sample": f"{len(rows)} evenly spaced query positions x all {w.n_q_heads} heads per step"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def oracle_decode_us(w, kc, vc, x, n_ctx):
    """The CPU oracle's decode step on the same cache and inputs, timed on the host cores.  The host
    copy of the cache is sparse -- only the rows the step reads (its anchor rows, then the spans of the
    anchors the oracle itself selects) are fetched; the rest of the (virtual) array is never touched."""
    from oracle import sla_oracle as O
    shape = tuple(kc.shape)
    hk, hv = np.empty(shape, dtype=np.uint16), np.empty(shape, dtype=np.uint16)
    i = n_ctx - 1
    m = np.arange(1, int(np.floor(np.sqrt(i + 1))) + 2, dtype=np.int64)
    t = i + 1 - m * m
    t = torch.from_numpy(t[t >= 0]).to(kc.device)
    hk[:, :, t.cpu().numpy()] = synth.to_numpy(kc[:, :, t])
    q_s, q = synth.to_numpy(x["q_s"]), synth.to_numpy(x["q"])
    code = synth.dtype_code(w.dtype)
    sel = O.span_search(q_s[:, :, None], hk, code, top_k=w.top_k, q_pos0=i, Lkv=n_ctx)["anchor"]
    span = w.back_factor * w.span_len
    for tpos in np.unique(sel[sel >= 0]):
        lo, hi = max(0, int(tpos) - span), min(i, int(tpos) + w.fwd_factor * w.span_len)
        hk[:, :, lo:hi + 1] = synth.to_numpy(kc[:, :, lo:hi + 1])
        hv[:, :, lo:hi + 1] = synth.to_numpy(vc[:, :, lo:hi + 1])
    t0 = time.perf_counter()
    O.decode_step(q_s, q, hk, hv, code, n_ctx=n_ctx, top_k=w.top_k, span_len=w.span_len,
                  back_factor=w.back_factor, fwd_factor=w.fwd_factor)
    return {"value": (time.perf_counter() - t0) * 1e6, "unit": "us per decode step", "cores": O.threads(), "kind": "oracle",
            "sample": "one whole decode step (search over all anchors + attention over the selected spans)"}


def bench_decode(sla, handle, w, steps, peaks, dev, with_oracle=False):
    """Decode loop: append the new token's K/V, then one sla_decode_step, `steps` times."""
    kc, vc = synth.make_decode_cache(w, dev, capacity=w.seq_len + steps + 8)
    params = sla.make_params(w.top_k, w.span_len, w.back_factor, w.fwd_factor, head_dim=w.head_dim)
    ins = [synth.make_decode_step_inputs(w, s, dev) for s in range(8)]
    out = sla.sla_decode_step(handle, ins[0]["q_s"], ins[0]["q"], kc, vc, w.seq_len, params)

    def one(step):
        x = ins[step % len(ins)]
        n_ctx = w.seq_len + step + 1
        kc[:, :, n_ctx - 1] = x["k_new"]
        vc[:, :, n_ctx - 1] = x["v_new"]
        sla.sla_decode_step(handle, x["q_s"], x["q"], kc, vc, n_ctx, params, out=out[0], lse=out[1],
                            out_anchor=out[2], out_score=out[3])
    for s in range(5):
        one(s)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for s in range(steps):
        one(s)
    e1.record()
    torch.cuda.synchronize()
    us = e0.elapsed_time(e1) * 1e3 / steps
    # kernel-only: the decode call alone, same cache, back to back
    e0.record()
    for s in range(steps):
        x = ins[s % len(ins)]
        sla.sla_decode_step(handle, x["q_s"], x["q"], kc, vc, w.seq_len + steps, params, out=out[0], lse=out[1],
                            out_anchor=out[2], out_score=out[3])
    e1.record()
    torch.cuda.synchronize()
    us_call = e0.elapsed_time(e1) * 1e3 / steps
    # tokens of the de-duplicated union of the selected spans (bookkeeping for the byte count)
    anchor = out[2].to(torch.int64)
    i = w.seq_len + steps - 1
    lo = torch.clamp(anchor - w.back_factor * w.span_len, min=0)
    hi = torch.clamp(anchor + w.fwd_factor * w.span_len, max=i)
    lo, order = torch.sort(lo, dim=-1)
    hi = torch.gather(hi, -1, order)
    run_hi = torch.cummax(hi, dim=-1).values
    prev = torch.cat([torch.full_like(run_hi[..., :1], -1), run_hi[..., :-1]], dim=-1)
    pairs = int(torch.clamp(hi - torch.maximum(lo, prev + 1) + 1, min=0).sum().item())
    elem = 2 if w.dtype == "bf16" else 4
    n_anchor = int(np.floor(np.sqrt(w.seq_len + steps)))
    bytes_step = pairs * 2 * w.head_dim * elem + n_anchor * w.batch * w.n_kv_heads * w.head_dim * elem
    gbs = bytes_step / (us_call * 1e-6) / 1e9
    cpu = oracle_decode_us(w, kc, vc, ins[(steps - 1) % len(ins)], w.seq_len + steps) if with_oracle else None
    del kc, vc
    torch.cuda.empty_cache()
    return {"workload": w.name, "us_per_token_per_layer": us, "us_per_decode_call": us_call, "steps": steps,
            "algorithmic_bytes_per_step": bytes_step, "cpu_baseline": cpu,
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                         "frac": gbs / peaks["hbm_gbs"], "frac_of_nominal_8000": gbs / 8000.0,
                         "traffic": DECODE_ATTN_DRAM_BYTES_PER_LAUNCH.get(w.name), "traffic_source": TRAFFIC_SOURCE,
                         "peak_source": peaks["_source"]}}


def max_over_ranks(value: float, dist, device) -> float:
    """The slowest rank's figure (every multi-rank number is a max over ranks); identity without dist."""
    if dist is None:
        return float(value)
    t = torch.tensor([float(value)], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def bench_paper_config(sla, handle, dev, steps):
    """Chunked prefill in the kernel configuration the paper reports (w = 1088, topK = 2, factors 4/2,
    l(i) = ceil(sqrt(i)), 32K-token chunks), per-span softmax + gate: search and gated attention of
    every chunk, tokens/s over the whole sequence."""
    w = synth.CONFIGS[5]
    x = synth.make_prefill(w, device=dev)
    B, Hq, L, D = x["q"].shape
    p = sla.make_params(w.top_k, w.span_len, w.back_factor, w.fwd_factor, window=w.window,
                        mode=sla.SLA_PER_SPAN, head_dim=D)
    ch = synth.PAPER_CHUNK
    anchor = torch.empty(B, Hq, ch, w.top_k, dtype=torch.int32, device=dev)
    score = torch.empty(B, Hq, ch, w.top_k, dtype=torch.float32, device=dev)
    lse = torch.empty(B, Hq, ch, dtype=torch.float32, device=dev)
    lse_span = torch.empty(B, Hq, ch, w.top_k, dtype=torch.float32, device=dev)
    out = torch.empty_like(x["q"])

    def step():
        for q0 in range(0, L, ch):
            qs, q = x["q_s"][:, :, q0:q0 + ch], x["q"][:, :, q0:q0 + ch]
            sla.sla_span_search(handle, qs, x["k"], p, q_pos0=q0, Lkv=q0 + ch, out_anchor=anchor, out_score=score)
            sla.sla_span_attention_gated(handle, q, x["k"], x["v"], anchor, score, p, q_pos0=q0, Lkv=q0 + ch,
                                         out=out[:, :, q0:q0 + ch], lse=lse, lse_span=lse_span)

    for _ in range(3):
        step()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    assert sla.sla_poll_status(handle) == sla.SLA_OK
    return {"workload": w.name, "mode": "per-span softmax + gate", "window": w.window, "top_k": w.top_k,
            "back_factor": w.back_factor, "fwd_factor": w.fwd_factor, "span_len": "ceil(sqrt(i))",
            "chunk": ch, "ms_per_step": ms, "tokens_per_s": B * L / (ms * 1e-3), "steps": steps}


def rank_workload(w, rank: int):
    """Every rank works on its own sequence: same shapes, its own seed (weak scaling, no exchange)."""
    return w.scaled(seed=w.seed + 7919 * rank)


def measure_e2e(sla, handle, host, params, args, dist, dev, world, B, L):
    """The same step through sla_prefill_host: pinned host inputs in, host outputs out, all copies
    inside the timed region."""
    ho = sla.sla_prefill_host(handle, host["q_s"], host["q"], host["k"], host["v"], params)
    n_e2e = max(2, min(args.steps, 5))
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    tt = time.perf_counter()
    for _ in range(n_e2e):
        sla.sla_prefill_host(handle, host["q_s"], host["q"], host["k"], host["v"], params,
                             out=ho[0], lse=ho[1], anchor=ho[2], score=ho[3])
    e2e_s = max_over_ranks((time.perf_counter() - tt) / n_e2e, dist, dev)
    h2d = sum(host[n].numel() * host[n].element_size() for n in ("q_s", "q", "k", "v"))
    d2h = sum(t.numel() * t.element_size() for t in ho)
    return {"value": world * B * L / e2e_s, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "ms_per_step": e2e_s * 1e3}


def measure_prefill(sla, handle, w, x, steps, warmup, local, dist, dev, peaks):
    """Times `steps` prefill steps (sla_span_search + sla_span_attention over the whole batch) with CUDA
    events on the launching stream; returns the timings, the clocks sampled meanwhile, the launches
    counted, the roofline of the attention kernel and that of the search kernel."""
    B, Hq, L, D = x["q"].shape
    params = sla.make_params(w.top_k, w.span_len, w.back_factor, w.fwd_factor, head_dim=w.head_dim)
    anchor = torch.empty(B, Hq, L, w.top_k, dtype=torch.int32, device=dev)
    score = torch.empty(B, Hq, L, w.top_k, dtype=torch.float32, device=dev)
    out = torch.empty_like(x["q"])
    lse = torch.empty(B, Hq, L, dtype=torch.float32, device=dev)

    def step(ev=None):
        sla.sla_span_search(handle, x["q_s"], x["k"], params, out_anchor=anchor, out_score=score)
        if ev is not None:
            ev[0].record()
        sla.sla_span_attention(handle, x["q"], x["k"], x["v"], anchor, params, out=out, lse=lse)
        if ev is not None:
            ev[1].record()

    for _ in range(max(3, warmup)):
        step()
    torch.cuda.synchronize()
    sla.sla_set_kernel_timing(handle, True)   # events around the main attention kernel, on its stream
    launches0 = sla.sla_kernel_launches(handle)
    sampler = ClockSampler(local)
    sampler.start()
    if dist:
        dist.barrier()
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    for s in range(steps):
        step(evs[s])
    t1.record()
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    clocks = sampler.stop()
    launches = sla.sla_kernel_launches(handle) - launches0
    total_ms = t0.elapsed_time(t1)
    attn_ms = float(np.mean([a.elapsed_time(b) for a, b in evs]))
    kern_ms_sum, kern_n = sla.sla_kernel_time_ms(handle)
    sla.sla_set_kernel_timing(handle, False)
    kern_ms = kern_ms_sum / steps if kern_n else attn_ms   # generic path: whole call
    total_ms = max_over_ranks(total_ms, dist, dev)
    ms_per_step = total_ms / steps
    search_ms = ms_per_step - attn_ms

    # roofline of the dominant kernel (span-attention): 4*D flops per attended (query, key) pair
    pairs = attended_pairs(anchor, w.span_len, w.back_factor, w.fwd_factor)
    flops = 4.0 * D * pairs
    roofline = tensor_roofline(flops, kern_ms, total_ms * 1e-3, clocks, peaks)
    roofline["kernel"] = "tc_attend (tcgen05 span-attention)" if kern_n else "attn_rows_simt"
    roofline["launches_timed"] = kern_n
    roofline["traffic"] = TC_ATTEND_DRAM_BYTES_PER_LAUNCH.get(L) if (kern_n and w.name.startswith("prefill_L65536")) else None
    roofline["traffic_source"] = TRAFFIC_SOURCE if roofline["traffic"] else None
    roofline["whole_call"] = {"sla_span_attention_ms": attn_ms, "sla_span_search_ms": search_ms,
                              "attention_tflops": flops / (attn_ms * 1e-3) / 1e12,
                              "attention_frac_of_burst": flops / (attn_ms * 1e-3) / 1e12 / peaks["bf16_tflops"],
                              "attention_frac_of_sustained": flops / (attn_ms * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"]}
    del anchor, score, out, lse
    return {"ms_per_step": ms_per_step, "attn_ms": attn_ms, "search_ms": search_ms, "kern_ms": kern_ms,
            "clocks": clocks, "launches": int(launches), "roofline": roofline, "params": params}


def search_roofline(w, search_ms, probe):
    """The span-search kernel streams one key row per (position, stride, KV head) out of L2 (K is
    L2-resident per KV head); its roofline is the L2 read bandwidth the probe measured in this run."""
    elem = 2 if w.dtype == "bf16" else 4
    nbytes = search_key_bytes(w.batch, w.n_kv_heads, w.seq_len, w.head_dim, elem, w.window)
    gbs = nbytes / (search_ms * 1e-3) / 1e9
    return {"bound": "l2", "kernel": "search_diag (span-search, selection folded into the scoring loop)",
            "achieved": gbs, "peak": probe["gbs"], "unit": "GB/s", "frac": gbs / probe["gbs"],
            "algorithmic_bytes_per_launch": nbytes, "ms_per_launch": search_ms, "traffic": None,
            "peak_source": f"read-only L2 probe of this run ({probe['buffer_mib']} MiB buffer, {probe['how']})"}


def run_ours(args, w):
    import paper_2601_18401_b200 as sla
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)
    sla.load_library()
    peaks = load_peaks()

    wr = rank_workload(w, rank)
    x = synth.make_prefill(wr, device=dev)
    params = sla.make_params(w.top_k, w.span_len, w.back_factor, w.fwd_factor, head_dim=w.head_dim)
    layout = sla.make_layout(x["q"], x["k"])
    work = sla.sla_workspace_bytes(layout, params, w.seq_len, w.seq_len)
    stage = sla.sla_host_staging_bytes(layout, params, w.seq_len)
    handle = sla.Handle(local, work + stage + (64 << 20))
    B, Hq, L, D = x["q"].shape
    m = measure_prefill(sla, handle, w, x, args.steps, args.warmup, local, dist, dev, peaks)
    value = world * B * L / (m["ms_per_step"] * 1e-3)
    probe = measure_l2_probe(sla, handle, dev)

    # end to end through the host-buffer C call: pinned host inputs, host outputs, copies inside
    host = None
    if not (args.no_e2e and args.no_cpu_baseline):
        host = {n: t.cpu().pin_memory() for n, t in x.items()}
    e2e = None if args.no_e2e else measure_e2e(sla, handle, host, params, args, dist, dev, world, B, L)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": m["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": config_of(w, world),
        "clocks": m["clocks"], "e2e": e2e, "gpu_launches": m["launches"], "roofline": m["roofline"],
        "roofline_search": search_roofline(w, m["search_ms"], probe), "l2_probe": probe,
    }

    if rank == 0 and not args.no_decode and not args.seq_len:
        line["paper_kernel_config"] = bench_paper_config(sla, handle, dev, max(3, min(args.steps, 10)))
    cpu_rows = None
    if rank == 0 and not args.no_cpu_baseline:
        cpu_rows = oracle_sample_rows(L, args.ref_rows)
        cpu_rows = cpu_rows[cpu_rows < L]
        cpu_host = {n: synth.to_numpy(t) for n, t in host.items()}
    del x
    handle.close()
    torch.cuda.empty_cache()
    if rank == 0 and not args.no_decode and not args.seq_len and not args.no_stress:
        line["prefill_stress_L262144"] = bench_stress(sla, local, dev, peaks, probe, max(3, min(args.steps, 5)))
    if rank == 0 and not args.no_decode:
        dh = sla.Handle(local, 64 << 20)
        dec = []
        for ci, steps in ((3, 256), (4, 128)):
            if args.decode_only and args.decode_only != synth.CONFIGS[ci].name:
                continue
            try:
                dec.append(bench_decode(sla, dh, synth.CONFIGS[ci], steps if not args.quick else 16, peaks, dev,
                                        with_oracle=not args.no_cpu_baseline))
            except torch.cuda.OutOfMemoryError as e:  # pragma: no cover
                dec.append({"workload": synth.CONFIGS[ci].name, "skipped": f"out of memory: {e}"})
        line["decode"] = dec
        dh.close()
    if cpu_rows is not None:
        from oracle import sla_oracle as O
        secs = time_oracle_prefill(w, cpu_host, cpu_rows)
        line["cpu_baseline"] = {"value": len(cpu_rows) * B / secs, "unit": UNIT, "cores": O.threads(), "kind": "oracle",
                                "sample": f"{len(cpu_rows)} evenly spaced query positions x all {Hq} heads, "
                                          f"search + attention, {secs:.1f} s"}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist:
        dist.barrier()
        dist.destroy_process_group()


def bench_stress(sla, local, dev, peaks, probe, steps):
    """The largest prefill configuration (batch 2, 16/4 heads, L = 262144, l = 512, k = 16): the same step,
    timed the same way, reported beside the headline."""
    w = synth.CONFIGS[2]
    x = synth.make_prefill(w, device=dev)
    params = sla.make_params(w.top_k, w.span_len, w.back_factor, w.fwd_factor, head_dim=w.head_dim)
    layout = sla.make_layout(x["q"], x["k"])
    handle = sla.Handle(local, sla.sla_workspace_bytes(layout, params, w.seq_len, w.seq_len) + (64 << 20))
    m = measure_prefill(sla, handle, w, x, steps, 3, local, None, dev, peaks)
    B, Hq, L, D = x["q"].shape
    del x
    handle.close()
    torch.cuda.empty_cache()
    return {"workload": w.name, "batch": B, "q_heads": Hq, "kv_heads": w.n_kv_heads, "seq_len": L, "span_len": w.span_len,
            "top_k": w.top_k, "steps": steps, "ms_per_step": m["ms_per_step"], "tokens_per_s": B * L / (m["ms_per_step"] * 1e-3),
            "clocks": m["clocks"], "gpu_launches": m["launches"], "roofline": m["roofline"],
            "roofline_search": search_roofline(w, m["search_ms"], probe)}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=1, help="index into the benchmark configurations (prefill ones)")
    ap.add_argument("--ref-rows", type=int, default=4096, help="query positions the CPU oracle is timed on")
    ap.add_argument("--no-decode", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--seq-len", type=int, default=0, help="shorter prefill sequence (for profiler captures)")
    ap.add_argument("--decode-only", default="", help="decode_1M or decode_10M: only that decode loop besides the prefill part")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-stress", action="store_true", help="skip the L = 262144 configuration reported beside the headline")
    ap.add_argument("--quick", action="store_true", help="short decode loops (for smoke runs)")
    args = ap.parse_args()
    w = synth.CONFIGS[args.workload]
    if args.seq_len:
        w = w.scaled(seq_len=args.seq_len, name=f"{w.name}_cut_to_{args.seq_len}")
    if w.kind != "prefill":
        raise SystemExit("--workload must name a prefill configuration; decode is reported alongside")
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
