"""Seeded synthetic inputs for span-search / span-attention.

This module only draws random tensors of the right shapes; it contains none of the method's
arithmetic (no anchors, scores, top-k, spans or softmax).  Both the CUDA path and the test oracle
read the buffers produced here, so that they see bit-identical inputs.

The tensors stand in for the paper's workload (routing queries, queries, keys and values of a
fine-tuned hybrid model on long-context retrieval prompts), which needs weights and data that are
not available.  Shapes follow the five benchmark configurations; values are i.i.d. N(0,1) drawn in
fp32 and then rounded to the run's dtype, with optional "planted" key spans that mimic a needle:
inside each planted span the keys of a KV head are shifted along a fixed unit direction, and every
routing query of that head's group is shifted along the same direction, so anchors that land in a
planted span score far above the background and many queries route to the same regions.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Optional

import numpy as np
import torch


@dataclass(frozen=True)
class Workload:
    name: str
    kind: str            # "prefill" or "decode"
    batch: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    seq_len: int         # L for prefill, starting n_ctx for decode
    dtype: str           # "f32" or "bf16"
    span_len: int        # fixed base span length l
    top_k: int
    back_factor: int = 2
    fwd_factor: int = 0
    window: int = 0
    planted_spans: int = 0   # planted key spans per KV head
    steps: int = 1           # decode steps
    seed: int = 0

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)


# The five benchmark configurations (index 0..4) and, last, the kernel configuration the paper reports
# its throughput with (Section "Experimental setup", "Kernel configuration": w = 1088, topK = 2,
# backward/forward factors 4 and 2, l(i) = ceil(sqrt(i)), 32K-token prefill chunks) on the shapes of
# the second configuration.
CONFIGS = [
    Workload("tiny_prefill_L4096", "prefill", 1, 1, 1, 64, 4096, "f32", 64, 4, seed=1001),
    Workload("prefill_L65536", "prefill", 1, 32, 8, 128, 65536, "bf16", 256, 8, planted_spans=16, seed=1002),
    Workload("prefill_stress_L262144", "prefill", 2, 16, 4, 128, 262144, "bf16", 512, 16, seed=1003),
    Workload("decode_1M", "decode", 1, 32, 4, 128, 1048576, "bf16", 1024, 16, steps=256, seed=1004),
    Workload("decode_10M", "decode", 1, 32, 4, 128, 10485760, "bf16", 3072, 16, steps=128, seed=1005),
    Workload("prefill_paper_kernel_config_L65536", "prefill", 1, 32, 8, 128, 65536, "bf16", 0, 2, back_factor=4,
             fwd_factor=2, window=1088, seed=1006),
]
PAPER_CHUNK = 32768   # query positions per call in the paper's chunked prefill


def torch_dtype(name: str) -> torch.dtype:
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _randn_into(dst: torch.Tensor, gen: torch.Generator, chunk_elems: int = 1 << 25) -> None:
    """Fill ``dst`` (any float dtype) with N(0,1) drawn in fp32, chunk by chunk along the flat view."""
    flat = dst.view(-1)
    n = flat.numel()
    for s in range(0, n, chunk_elems):
        e = min(n, s + chunk_elems)
        flat[s:e] = torch.randn(e - s, generator=gen, device=dst.device, dtype=torch.float32).to(dst.dtype)


def planted_starts(w: Workload, kv_head_index: int) -> np.ndarray:
    """Seeded, non-overlapping start positions of the planted spans (each 2*l tokens long)."""
    n, span = w.planted_spans, 2 * w.span_len
    rng = np.random.default_rng(w.seed * 7919 + kv_head_index)
    slots = w.seq_len // (2 * span)            # slots of 2*span tokens; one planted span per slot
    pick = np.sort(rng.choice(slots, size=n, replace=False))
    jitter = rng.integers(0, span, size=n)
    return pick.astype(np.int64) * (2 * span) + jitter  # disjoint: each stays inside its own slot


def make_prefill(w: Workload, device="cpu", amplitude: float = 10.0):
    """Returns dict(q_s, q, k, v) with q* [B,Hq,L,D] and k,v [B,Hkv,L,D] in the workload's dtype.

    Draw order Q_s, Q, K, V from one generator seeded with ``w.seed``.
    """
    assert w.kind == "prefill"
    dt = torch_dtype(w.dtype)
    gen = _gen(device, w.seed)
    B, Hq, Hkv, D, L = w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim, w.seq_len
    G = Hq // Hkv
    out = {}
    for name, H in (("q_s", Hq), ("q", Hq), ("k", Hkv), ("v", Hkv)):
        t = torch.empty(B, H, L, D, dtype=dt, device=device)
        if w.planted_spans and name in ("q_s", "k"):
            # shift in fp32 before rounding to the run's dtype
            t32 = torch.empty(B, H, L, D, dtype=torch.float32, device=device)
            _randn_into(t32, gen)
            dir_gen = _gen("cpu", w.seed + 17)
            u = torch.randn(Hkv, D, generator=dir_gen, dtype=torch.float32)
            u = (u / u.norm(dim=-1, keepdim=True)).to(device)
            if name == "q_s":
                for h in range(Hq):
                    t32[:, h] += amplitude * u[h // G]
            else:
                for g in range(Hkv):
                    for s in planted_starts(w, g):
                        t32[:, g, int(s): int(s) + 2 * w.span_len] += amplitude * u[g]
            t.copy_(t32)
            del t32
        else:
            _randn_into(t, gen)
        out[name] = t
    return out


def make_decode_cache(w: Workload, device, capacity: Optional[int] = None):
    """K and V caches [B,Hkv,capacity,D]; positions 0..seq_len-1 are filled, the rest is zero."""
    assert w.kind == "decode"
    dt = torch_dtype(w.dtype)
    cap = int(capacity if capacity is not None else w.seq_len + w.steps)
    gen = _gen(device, w.seed)
    B, Hkv, D = w.batch, w.n_kv_heads, w.head_dim
    caches = []
    for _ in range(2):
        c = torch.zeros(B, Hkv, cap, D, dtype=dt, device=device)
        for b in range(B):
            for g in range(Hkv):
                _randn_into(c[b, g, : w.seq_len], gen)
        caches.append(c)
    return caches[0], caches[1]


def make_decode_step_inputs(w: Workload, step: int, device):
    """Fresh q_s, q [B,Hq,D] and the new token's k_new, v_new [B,Hkv,D] for decode step ``step``."""
    dt = torch_dtype(w.dtype)
    gen = _gen(device, w.seed * 100003 + 1 + step)
    B, Hq, Hkv, D = w.batch, w.n_q_heads, w.n_kv_heads, w.head_dim
    mk = lambda H: torch.randn(B, H, D, generator=gen, device=device, dtype=torch.float32).to(dt)
    return dict(q_s=mk(Hq), q=mk(Hq), k_new=mk(Hkv), v_new=mk(Hkv))


def to_numpy(t: torch.Tensor) -> np.ndarray:
    """Host numpy view for the oracle: fp32 as float32, bf16 as its uint16 bit patterns."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def dtype_code(name: str) -> int:
    """Element-type code shared by the C interfaces: 0 = fp32, 1 = bf16."""
    return {"f32": 0, "bf16": 1}[name]
