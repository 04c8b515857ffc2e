"""Seeded synthetic workloads: tensor shape lists and input generators.

This module holds NO arithmetic of the sharded weight update.  It only says
which tensors a model-shaped workload has (shapes in the order a framework
would list them), which optimizer hyper-parameters the workload uses, and how
to draw seeded random weights / optimizer slots / per-replica gradients with
the stated distributions.  Both the CUDA path's tests and the CPU oracle's
tests draw their inputs here, so the two sides see the same bytes.

The paper evaluates on the MLPerf-0.6 ResNet-50 and Transformer (Section 6,
Table 1); the weight update never looks at training data, only at tensors with
the models' shapes, so shape-faithful random tensors stand in for them.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Dict, List, Sequence, Tuple

import torch

Shape = Tuple[int, ...]

# optimizer codes shared by name only (values mirror the public C enum and the
# oracle's enum; each side defines its own copy)
SGDM, ADAM, LAMB, LARS, ADAFACTOR = "sgdm", "adam", "lamb", "lars", "adafactor"


@dataclass
class Workload:
    name: str
    shapes: List[Shape]
    R: int                      # logical replicas = shard count
    opt: str                    # "sgdm" | "adam" | "lamb"
    hyper: Dict[str, float]     # lr, beta1, beta2, eps, weight_decay, momentum, grad_scale, step
    grad_dtype: torch.dtype = torch.float32
    out_dtype: torch.dtype = torch.float32   # dtype of the gathered weight copy
    grad_std: float = 1e-3
    w_std: float = 0.02
    m_std: float = 1e-3
    v_std: float = 1e-5
    outlier_frac: float = 0.0   # fraction of gradient entries scaled by outlier_scale
    outlier_scale: float = 1.0
    seed: int = 0
    R_sweep: Sequence[int] = field(default_factory=tuple)

    @property
    def numels(self) -> List[int]:
        return [int(math.prod(s)) for s in self.shapes]

    @property
    def N(self) -> int:
        return sum(self.numels)

    @property
    def T(self) -> int:
        return len(self.shapes)


def _hyper(**kw) -> Dict[str, float]:
    h = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0,
             momentum=0.0, grad_scale=1.0, step=10, trust_coeff=0.001)
    h.update(kw)
    return h


# --------------------------------------------------------------------------
# shape lists
# --------------------------------------------------------------------------
def tiny_shapes() -> List[Shape]:
    return [(64, 128), (128,), (3, 3, 16, 32), (32,), (512, 64), (64,)]


def resnet50_shapes() -> List[Shape]:
    """ResNet-50 v1 bottleneck network, HWIO conv filters, BN gamma/beta after
    every conv, 1000-way classifier."""
    s: List[Shape] = [(7, 7, 3, 64), (64,), (64,)]
    cin = 64
    for width, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        for b in range(blocks):
            s += [(1, 1, cin, width), (width,), (width,)]
            s += [(3, 3, width, width), (width,), (width,)]
            s += [(1, 1, width, 4 * width), (4 * width,), (4 * width,)]
            if b == 0:
                s += [(1, 1, cin, 4 * width), (4 * width,), (4 * width,)]
            cin = 4 * width
    s += [(2048, 1000), (1000,)]
    return s


def _attn(d: int, bias: bool) -> List[Shape]:
    out: List[Shape] = []
    for _ in range(4):
        out.append((d, d))
        if bias:
            out.append((d,))
    return out


def transformer_shapes(d: int = 1024, ffn: int = 4096, vocab: int = 33708,
                       layers: int = 6) -> List[Shape]:
    """Encoder-decoder Transformer ("big"), shared embedding, post-LN blocks."""
    ln = [(d,), (d,)]
    ff = [(d, ffn), (ffn,), (ffn, d), (d,)]
    s: List[Shape] = [(vocab, d)]
    for _ in range(layers):
        s += _attn(d, False) + ln + ff + ln
    s += ln
    for _ in range(layers):
        s += _attn(d, False) + ln + _attn(d, False) + ln + ff + ln
    s += ln
    return s


def bert_large_shapes(d: int = 1024, ffn: int = 4096, vocab: int = 30522,
                      max_pos: int = 512, layers: int = 24) -> List[Shape]:
    ln = [(d,), (d,)]
    s: List[Shape] = [(vocab, d), (max_pos, d), (2, d)] + ln
    for _ in range(layers):
        s += _attn(d, True) + ln + [(d, ffn), (ffn,), (ffn, d), (d,)] + ln
    s += [(d, d), (d,)]
    return s


def decoder_1p5b_shapes(d: int = 1600, ffn: int = 6400, vocab: int = 50257,
                        n_pos: int = 1024, layers: int = 48) -> List[Shape]:
    ln = [(d,), (d,)]
    s: List[Shape] = [(vocab, d), (n_pos, d)]
    for _ in range(layers):
        s += ln + [(d, 3 * d), (3 * d,), (d, d), (d,)] + ln
        s += [(d, ffn), (ffn,), (ffn, d), (d,)]
    s += ln
    return s


# --------------------------------------------------------------------------
# the five named workloads
# --------------------------------------------------------------------------
def tiny() -> Workload:
    return Workload("tiny", tiny_shapes(), R=4, opt=ADAM, hyper=_hyper(),
                    grad_std=1e-2, seed=0)


def resnet50() -> Workload:
    return Workload("resnet50", resnet50_shapes(), R=8, opt=SGDM,
                    hyper=_hyper(lr=0.1, momentum=0.9, weight_decay=5e-5),
                    seed=2)


def resnet50_lars() -> Workload:
    """The ResNet-50 tensor set under LARS, the optimizer of the paper's ResNet-50 runs (Table 1)."""
    return Workload("resnet50_lars", resnet50_shapes(), R=8, opt=LARS,
                    hyper=_hyper(lr=10.0, momentum=0.9, weight_decay=5e-5, trust_coeff=0.001), seed=6)


def transformer(R: int = 8) -> Workload:
    return Workload("transformer", transformer_shapes(), R=R, opt=ADAM,
                    hyper=_hyper(), seed=3, R_sweep=(1, 2, 8, 32, 128, 1024))


def transformer_adafactor(R: int = 8) -> Workload:
    """The Transformer tensor set under Adafactor, the optimizer the paper names (with LARS) for its
    reduce operators (Section 4.1): factored second moments, clipping at 1, relative step size."""
    return Workload("transformer_adafactor", transformer_shapes(), R=R, opt=ADAFACTOR,
                    hyper=_hyper(lr=1e-2, eps=1e-30, eps2=1e-3, clip_threshold=1.0, decay_exponent=0.8), seed=7)


def bert_large() -> Workload:
    return Workload("bert_large", bert_large_shapes(), R=16, opt=LAMB,
                    hyper=_hyper(eps=1e-6, weight_decay=0.01), seed=4)


def decoder_1p5b() -> Workload:
    return Workload("decoder_1p5b", decoder_1p5b_shapes(), R=4, opt=ADAM,
                    hyper=_hyper(), grad_dtype=torch.bfloat16,
                    out_dtype=torch.bfloat16, outlier_frac=0.01,
                    outlier_scale=100.0, seed=5)


WORKLOADS = {
    "tiny": tiny, "resnet50": resnet50, "transformer": transformer,
    "bert_large": bert_large, "decoder_1p5b": decoder_1p5b, "resnet50_lars": resnet50_lars,
    "transformer_adafactor": transformer_adafactor,
}


def scaled_down(wl: Workload, max_dim: int) -> Workload:
    """Same tensor list with every dimension clipped to ``max_dim`` - keeps the
    count, order and rank mix of the tensors (many small 1-D ones between big
    matrices) at a size a CPU oracle finishes in seconds."""
    shapes = [tuple(min(x, max_dim) for x in s) for s in wl.shapes]
    out = Workload(**{**wl.__dict__})
    out.shapes = shapes
    out.name = f"{wl.name}_clip{max_dim}"
    return out


# --------------------------------------------------------------------------
# seeded generators (no method arithmetic)
# --------------------------------------------------------------------------
_ROLE = {"w": 1, "m": 2, "v": 3, "g": 4, "f": 5}


def _gen(device, seed: int, role: str, k: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1_000_003 + _ROLE[role] * 10_007 + k) & 0x7FFFFFFF)
    return g


def _normal(n: int, std: float, gen: torch.Generator, device) -> torch.Tensor:
    t = torch.empty(n, dtype=torch.float32, device=device)
    t.normal_(0.0, std, generator=gen)
    return t


def make_state(wl: Workload, device="cpu"):
    """Weights, first and second optimizer slots as flat fp32 tensors, one per
    model tensor: w ~ N(0, w_std), m ~ N(0, m_std), v = |N(0, v_std)|."""
    gw, gm, gv = (_gen(device, wl.seed, r, 0) for r in "wmv")
    w = [_normal(n, wl.w_std, gw, device) for n in wl.numels]
    m = [_normal(n, wl.m_std, gm, device) for n in wl.numels]
    v = [_normal(n, wl.v_std, gv, device).abs_() for n in wl.numels]
    return w, m, v


def make_factored_state(wl: Workload, n: int, device="cpu") -> torch.Tensor:
    """Adafactor's row / column accumulators (n floats for the whole model): uniform in
    [1e-6, 1e-3], the size of sums of squared gradients a few steps into training."""
    gen = _gen(device, wl.seed, "f", 0)
    return torch.empty(n, dtype=torch.float32, device=device).uniform_(1e-6, 1e-3, generator=gen)


def make_grads_one(wl: Workload, k: int, device="cpu", numels=None) -> List[torch.Tensor]:
    """Replica k's local gradients: N(0, grad_std) drawn in fp32, a Bernoulli
    fraction of entries multiplied by ``outlier_scale``, then narrowed to the
    workload's gradient dtype."""
    gen = _gen(device, wl.seed, "g", k)
    out = []
    for n in (numels if numels is not None else wl.numels):
        g = _normal(n, wl.grad_std, gen, device)
        if wl.outlier_frac > 0.0:
            mask = torch.empty(n, dtype=torch.float32, device=device).uniform_(generator=gen) < wl.outlier_frac
            g = torch.where(mask, g * wl.outlier_scale, g)
        out.append(g.to(wl.grad_dtype))
    return out


def make_grads(wl: Workload, device="cpu") -> List[List[torch.Tensor]]:
    return [make_grads_one(wl, k, device) for k in range(wl.R)]
