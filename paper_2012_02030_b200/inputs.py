"""Seeded synthetic workloads shaped like the paper's experiments.

This module only draws inputs.  It holds none of the method's arithmetic (no
softmax, no selection, no attention) and is the one module that both the CUDA
tests/benchmarks and the CPU oracle's tests use, so that both sides see the
same numbers.  Everything is generated on the host with a seeded
``torch.Generator``, in fp32, and rounded once to the workload's dtype.

The five workloads stand in for: a tiny fp32 case; encoder self-attention of a
BERT-base-shaped classifier (GLUE setting: sequences of 128, batch 32); causal
language-model self-attention (Transformer-XL setting); the decoder-self and
encoder-decoder attention of a seq2seq translation model; and a long-context
causal case (context 4096, head width 128 as in the Llama-2 experiment).  The
real datasets and trained weights are not available, so the calibration logits
get an additive per-head bias that produces the patterns the paper describes
for trained models: a band around the diagonal, a few always-attended "sink"
columns, and strided columns.
"""
from __future__ import annotations

import dataclasses

import torch

TILE = 128


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    Lq: int
    Lk: int
    d: int
    dtype: str  # "f32" or "bf16"
    causal: bool
    keep_frac: float
    keep_diag: bool
    calib_batches: int
    bias: str  # name of the calibration-bias recipe
    seed0: int

    @property
    def torch_dtype(self):
        return {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[self.dtype]

    @property
    def n_valid(self) -> int:
        """Entries of one head's domain."""
        if self.causal:  # row i sees keys j <= i + (Lk - Lq): memory keys, then its own segment
            return self.Lq * (self.Lq + 1) // 2 + self.Lq * (self.Lk - self.Lq)
        return self.Lq * self.Lk

    @property
    def n_forced(self) -> int:
        return self.Lq if (self.keep_diag and (self.Lq == self.Lk or self.causal)) else 0

    def scaled(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def _seed(c: int) -> int:
    return 20120 + 1000 * c


WORKLOADS = {
    "tiny": Workload("tiny", 2, 2, 128, 128, 64, "f32", False, 0.10, True, 16, "band8_sink4", _seed(0)),
    "bert": Workload("bert", 32, 12, 128, 128, 64, "bf16", False, 0.50, True, 64, "band_h_colnoise", _seed(1)),
    "lm": Workload("lm", 16, 16, 512, 512, 64, "bf16", True, 0.10, True, 64, "causal16_sink8", _seed(2)),
    "s2s_self": Workload("s2s_self", 64, 8, 256, 256, 64, "bf16", True, 0.50, True, 64, "causal12", _seed(3)),
    "s2s_cross": Workload("s2s_cross", 64, 8, 256, 256, 64, "bf16", False, 0.50, False, 64, "cross12", _seed(3) + 500),
    "long": Workload("long", 4, 16, 4096, 4096, 128, "bf16", True, 0.05, True, 16, "causal64_sink16_stride256", _seed(4)),
    # beyond the five prescribed configurations: a segment of 384 tokens attending to 384 cached
    # positions of earlier segments plus itself (Transformer-XL's recurrence), and the long causal
    # shape with the head count of the paper's Llama-2 experiment
    "txl": Workload("txl", 16, 16, 384, 768, 64, "bf16", True, 0.10, True, 16, "mem32_sink8", _seed(5)),
    "llama": Workload("llama", 1, 32, 4096, 4096, 128, "bf16", True, 0.05, True, 16, "causal64_sink16_stride256",
                      _seed(6)),
}


def _randn(shape, seed: int, dtype) -> torch.Tensor:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return torch.randn(shape, generator=g, dtype=torch.float32).to(dtype).contiguous()


def eval_qkv(w: Workload):
    """Q[B,H,Lq,d], K,V[B,H,Lk,d] ~ N(0,1) in the workload's dtype (host tensors)."""
    q = _randn((w.B, w.H, w.Lq, w.d), w.seed0, w.torch_dtype)
    k = _randn((w.B, w.H, w.Lk, w.d), w.seed0 + 100_003, w.torch_dtype)
    v = _randn((w.B, w.H, w.Lk, w.d), w.seed0 + 200_003, w.torch_dtype)
    return q, k, v


def calib_qk(w: Workload, t: int):
    """Q,K of calibration batch t (B sequences), same distribution as the evaluation tensors."""
    q = _randn((w.B, w.H, w.Lq, w.d), w.seed0 + 1 + t, w.torch_dtype)
    k = _randn((w.B, w.H, w.Lk, w.d), w.seed0 + 300_007 + t, w.torch_dtype)
    return q, k


def calib_bias(w: Workload) -> torch.Tensor:
    """Additive bias on the scaled calibration logits, fp32 [H,Lq,Lk].

    Evaluated in fp64 and rounded once.  Under the causal constraint the
    formulas are evaluated inside the domain only; the rest is 0 and never read.
    """
    i = torch.arange(w.Lq, dtype=torch.float64).view(1, -1, 1)
    j = torch.arange(w.Lk, dtype=torch.float64).view(1, 1, -1)
    h = torch.arange(w.H, dtype=torch.float64).view(-1, 1, 1)
    kind = w.bias
    if kind == "none":
        b = torch.zeros((1, w.Lq, w.Lk), dtype=torch.float64)
    elif kind == "band8_sink4":
        b = (3.0 * torch.exp(-(i - j).abs() / 8.0) + 2.0 * (j < 4))
    elif kind == "band_h_colnoise":
        g = torch.Generator(device="cpu")
        g.manual_seed(w.seed0 + 999)
        col = torch.randn((w.H, 1, w.Lk), generator=g, dtype=torch.float32).to(torch.float64)
        b = 2.0 * torch.exp(-(i - j).abs() / (4.0 + h)) + col
    elif kind == "causal16_sink8":
        dist = (i - j).clamp(min=0.0)
        b = (3.0 * torch.exp(-dist / 16.0) + 2.0 * (j < 8))
    elif kind == "causal12":
        dist = (i - j).clamp(min=0.0)
        b = (2.0 * torch.exp(-dist / 12.0))
    elif kind == "cross12":
        b = (2.0 * torch.exp(-(i * (w.Lk / w.Lq) - j).abs() / 12.0))
    elif kind == "causal64_sink16_stride256":
        dist = (i - j).clamp(min=0.0)
        b = (3.0 * torch.exp(-dist / 64.0) + 2.0 * (j < 16) + 1.5 * (torch.remainder(j, 256) == 0))
    elif kind == "mem32_sink8":
        dist = (i + (w.Lk - w.Lq) - j).clamp(min=0.0)  # distance from the query's own position
        b = (3.0 * torch.exp(-dist / 32.0) + 2.0 * (j < 8))
    else:
        raise ValueError(kind)
    if w.causal:
        b = b * (j <= i + (w.Lk - w.Lq))
    return b.to(torch.float32).expand(w.H, w.Lq, w.Lk).contiguous()


def random_mask(H: int, Lq: int, Lk: int, density: float, seed: int, causal: bool = False,
                empty_rows=()) -> torch.Tensor:
    """Random element mask (uint8 [H,Lq,Lk]) for tests of the forward pass: the
    random-mask control of the paper's Section 8, here only as a test input."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    m = (torch.rand((H, Lq, Lk), generator=g) < density)
    if causal:
        m &= torch.tril(torch.ones((Lq, Lk), dtype=torch.bool), diagonal=Lk - Lq)
    for r in empty_rows:
        m[:, r, :] = False
    return m.to(torch.uint8).contiguous()


def group_sparse_mask(H: int, Lq: int, Lk: int, group_frac: float, fill: float, seed: int,
                      full_tile_frac: float = 0.0, causal: bool = False) -> torch.Tensor:
    """Structured random mask (uint8 [H,Lq,Lk]) for tests of the forward pass: per (head, block of
    128 query rows) each group of 16 key columns is active with probability group_frac, and only
    inside active groups entries are kept (each with probability fill), so that most 16-column
    groups of a tile stay empty, as in masks made of bands and a few heavy columns.  A fraction
    full_tile_frac of the 128 x 128 tiles is kept entirely."""
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    n_qt, n_g, n_kt = -(-Lq // 128), -(-Lk // 16), -(-Lk // 128)
    active = torch.rand((H, n_qt, n_g), generator=g) < group_frac
    m = torch.rand((H, Lq, Lk), generator=g) < fill
    act = active.repeat_interleave(128, dim=1)[:, :Lq].repeat_interleave(16, dim=2)[:, :, :Lk]
    m &= act
    if full_tile_frac > 0.0:
        full = torch.rand((H, n_qt, n_kt), generator=g) < full_tile_frac
        m |= full.repeat_interleave(128, dim=1)[:, :Lq].repeat_interleave(128, dim=2)[:, :, :Lk]
    if causal:
        m &= torch.tril(torch.ones((Lq, Lk), dtype=torch.bool))
    return m.to(torch.uint8).contiguous()


def widen(t: torch.Tensor):
    """Host tensor -> float32 numpy array with exactly the same values."""
    return t.to(torch.float32).numpy()
