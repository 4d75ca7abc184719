"""Seeded synthetic inputs for the FLy verification step.

This module only DRAWS inputs (logits, draft tokens, hidden states, LM-head
weights) with the shapes and value distributions of the five benchmark
workloads.  It holds none of the verification arithmetic: no entropy, no
gate, no window.  Where an input recipe depends on a quantity the method
computes (rows are redrawn when their entropy lies too close to the gate
threshold), the caller passes that quantity in as a function.

The paper evaluates on Llama-3 targets (|V| = 128256, K = 15 or 25) over
public datasets; these draws stand in for those logits.

Both the CPU oracle's tests and the CUDA path's tests/benchmark consume the
tensors produced here, so both sides always see identical bits.
"""
from __future__ import annotations

import hashlib
import math
from dataclasses import dataclass, replace
from typing import Callable, Optional

import torch


@dataclass(frozen=True)
class Workload:
    name: str
    B: int
    K: int
    V: int
    dtype: str                   # "f32" | "bf16": storage type of the logits
    scale: Optional[tuple]       # per-row std ~ U(lo, hi); None = 1
    spike_frac: float            # fraction of rows that get one spiked index
    spike: tuple                 # spike height ~ U(lo, hi) (lo == hi: constant)
    draft_mix: tuple             # P(argmax), P(rank 2..5), P(uniform over V)
    theta: float = 1.0           # gate threshold, nats
    W: int = 3
    boundary: str = "reject"     # "reject" (paper) | "carry"
    steps: int = 1
    hidden: int = 0              # > 0: fused LM-head workload (hidden size)
    weight_std: float = 0.02

    @property
    def rows(self) -> int:
        return self.B * (self.K + 1)

    @property
    def elem_bytes(self) -> int:
        return 4 if self.dtype == "f32" else 2

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16


TINY = Workload("tiny_verify", B=1, K=8, V=32000, dtype="f32", scale=None,
                spike_frac=0.5, spike=(12.0, 12.0), draft_mix=(0.7, 0.0, 0.3), steps=200)
LLAMA3 = Workload("llama3_vocab_batch", B=16, K=8, V=128256, dtype="bf16", scale=(0.5, 4.0),
                  spike_frac=0.4, spike=(8.0, 16.0), draft_mix=(0.6, 0.3, 0.1), steps=1000)
LONG_DRAFT = Workload("long_draft_batch", B=64, K=16, V=128256, dtype="bf16", scale=(0.5, 4.0),
                      spike_frac=0.4, spike=(8.0, 16.0), draft_mix=(0.6, 0.3, 0.1), steps=500)
SERVING = Workload("high_batch_serving", B=256, K=8, V=152064, dtype="bf16", scale=(0.3, 5.0),
                   spike_frac=0.5, spike=(8.0, 16.0), draft_mix=(0.65, 0.35, 0.0),
                   boundary="carry", steps=512)
FUSED = Workload("fused_lm_head", B=32, K=8, V=128256, dtype="bf16", scale=None,
                 spike_frac=0.0, spike=(0.0, 0.0), draft_mix=(0.7, 0.0, 0.3), steps=200,
                 hidden=8192)

# The paper's own operating point (Section 3, implementation details): threshold 0.3 on the NORMALISED
# entropy h = H / log|V| (= 3.53 nats at |V| = 128256), window W = 6, K = 15 drafts for the 70B target
# and K = 25 for the 405B target, one sequence at a time.  Rows are drawn as for the Llama-3 batch.
PAPER_70B = Workload("paper_default_70b", B=1, K=15, V=128256, dtype="bf16", scale=(0.5, 4.0),
                     spike_frac=0.4, spike=(8.0, 16.0), draft_mix=(0.6, 0.3, 0.1), theta=0.3 * math.log(128256),
                     W=6, steps=1000)
PAPER_405B = Workload("paper_default_405b", B=1, K=25, V=128256, dtype="bf16", scale=(0.5, 4.0),
                      spike_frac=0.4, spike=(8.0, 16.0), draft_mix=(0.6, 0.3, 0.1), theta=0.3 * math.log(128256),
                      W=6, steps=1000)

WORKLOADS = {w.name: w for w in (TINY, LLAMA3, LONG_DRAFT, SERVING, FUSED, PAPER_70B, PAPER_405B)}
LONG_DRAFT_SETTINGS = [(th, W) for th in (0.5, 1.0, 2.0) for W in (1, 3, 5)]


def shrink(w: Workload, **kw) -> Workload:
    """Same recipe at other sizes (parity tests run reduced copies)."""
    return replace(w, **kw)


def seed_for(*key) -> int:
    """63-bit seed from (workload, setting, step, tensor, attempt ...)."""
    h = hashlib.blake2b(repr(key).encode(), digest_size=8).digest()
    return int.from_bytes(h, "little") & ((1 << 63) - 1)


def _gen(device, *key) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed_for(*key))
    return g


def _draw_rows(w: Workload, device, *key) -> torch.Tensor:
    """[rows, V] in the storage dtype.  Values are drawn and the spike added
    in fp32, then rounded to nearest-even into the storage type."""
    R, V = w.rows, w.V
    g = _gen(device, w.name, "logits", *key)
    x = torch.randn(R, V, generator=g, device=device, dtype=torch.float32)
    if w.scale is not None:
        lo, hi = w.scale
        s = lo + (hi - lo) * torch.rand(R, 1, generator=g, device=device)
        x *= s
    if w.spike_frac > 0:
        spiked = torch.rand(R, generator=g, device=device) < w.spike_frac
        lo, hi = w.spike
        height = lo + (hi - lo) * torch.rand(R, generator=g, device=device)
        where = torch.randint(0, V, (R,), generator=g, device=device)
        rows = torch.nonzero(spiked).flatten()
        x[rows, where[rows]] += height[rows]
    return x.to(w.torch_dtype)


def make_logits(w: Workload, step: int, device="cpu", setting=0,
                entropy_fn: Optional[Callable[[torch.Tensor], torch.Tensor]] = None,
                theta_nats: Optional[float] = None, guard: float = 1e-3) -> torch.Tensor:
    """Logits [B, K+1, V] for one step.

    entropy_fn(rows[n, V]) -> entropy in nats [n] (supplied by the caller; the
    tests pass the fp64 oracle).  With it, a row whose entropy lies within
    `guard` of the gate threshold (or of any threshold in a list) is redrawn so that the gate decision is the
    same in any reasonable precision.
    """
    x = _draw_rows(w, device, setting, step, 0)
    if entropy_fn is not None:
        ths = w.theta if theta_nats is None else theta_nats
        ths = list(ths) if isinstance(ths, (list, tuple)) else [ths]
        for attempt in range(1, 8):
            H = torch.as_tensor(entropy_fn(x)).to("cpu", torch.float64)
            near = torch.zeros_like(H, dtype=torch.bool)
            for th in ths:
                near |= (H - th).abs() < guard
            bad = torch.nonzero(near).flatten()
            if bad.numel() == 0:
                break
            fresh = _draw_rows(w, device, setting, step, attempt)
            x[bad.to(x.device)] = fresh[bad.to(x.device)]
        else:
            raise RuntimeError("could not move every entropy away from the threshold")
    return x.view(w.B, w.K + 1, w.V)


def rank5(rows: torch.Tensor, block: int = 128) -> torch.Tensor:
    """Indices of the five largest entries of each row, ordered by value
    (descending) then index (ascending).  Only used to pick what the synthetic
    drafter proposes."""
    out = []
    for r0 in range(0, rows.shape[0], block):
        blk = rows[r0:r0 + block].float()
        _, idx = torch.sort(blk, dim=-1, descending=True, stable=True)
        out.append(idx[:, :5].clone())
    return torch.cat(out, 0)


def make_draft(w: Workload, step: int, top5: torch.Tensor, setting=0) -> torch.Tensor:
    """Draft tokens [B, K] int32.  top5 is [B*(K+1), 5] (see rank5) or
    [B*(K+1), 1] holding only the rank-1 index when the mix has no
    near-miss component."""
    device = top5.device
    g = _gen(device, w.name, "draft", setting, step)
    B, K, V = w.B, w.K, w.V
    top = top5.view(B, K + 1, -1)[:, :K]
    u = torch.rand(B, K, generator=g, device=device)
    near = torch.randint(1, 5, (B, K), generator=g, device=device).clamp_(max=top.shape[-1] - 1)
    anyv = torch.randint(0, V, (B, K), generator=g, device=device)
    p_arg, p_near, _ = w.draft_mix
    d = top[..., 0].clone()
    if p_near > 0:
        pick = torch.gather(top, 2, near.unsqueeze(-1)).squeeze(-1)
        sel = (u >= p_arg) & (u < p_arg + p_near)
        d[sel] = pick[sel]
    sel = u >= p_arg + p_near
    d[sel] = anyv[sel]
    return d.to(torch.int32)


def make_hidden(w: Workload, step: int, device="cpu", attempt: int = 0) -> torch.Tensor:
    """Hidden states [B*(K+1), hidden] bf16 ~ N(0, 1)."""
    g = _gen(device, w.name, "hidden", step, attempt)
    return torch.randn(w.rows, w.hidden, generator=g, device=device).to(torch.bfloat16)


def make_weight(w: Workload, device="cpu") -> torch.Tensor:
    """LM-head weight [hidden, V] bf16 ~ N(0, weight_std), fixed across steps."""
    g = _gen(device, w.name, "weight")
    x = torch.randn(w.hidden, w.V, generator=g, device=device)
    return (x * w.weight_std).to(torch.bfloat16)
