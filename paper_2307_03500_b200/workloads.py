"""Seeded synthetic gradient vectors shaped like the models the DEFT paper trains.

This module only draws random numbers.  It holds none of the method's
arithmetic (no norms, no k allocation, no packing, no selection) and imports
neither the CUDA binding nor the CPU oracle, so both sides of a parity test can
take their inputs from it.

The paper (Section 5.1, Table 2) measures on gradients of ResNet-18/CIFAR-10,
an LSTM language model/WikiText-2 and NCF/MovieLens-20M.  Those datasets and
models are not available offline, so each workload below is a flat fp32 vector
whose tensor sizes are those of a standard architecture and whose values follow
a stated distribution; every draw comes from ``numpy.random.default_rng`` with
one child stream per tensor (``SeedSequence(seed).spawn``).
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Callable, List

import numpy as np


# --------------------------------------------------------------------------
# Tensor size lists (parameter tensors in registration order)
# --------------------------------------------------------------------------
def tiny_sizes() -> List[int]:
    return [4096, 64, 16384, 256, 32768, 128, 40960, 10]


def resnet18_sizes() -> List[int]:
    """ResNet-18 with a 7x7 stem and a 1000-way classifier: 62 tensors, 11,689,512 elements."""
    s: List[int] = [64 * 3 * 7 * 7, 64, 64]
    cin = 64
    for stage, cout in enumerate((64, 128, 256, 512)):
        for block in range(2):
            first_in = cin if block == 0 else cout
            s += [cout * first_in * 9, cout, cout, cout * cout * 9, cout, cout]
            if block == 0 and stage > 0:
                s += [cout * cin, cout, cout]  # 1x1 downsample conv + its BN
        cin = cout
    s += [512 * 1000, 1000]
    return s


def lstm_lm_sizes() -> List[int]:
    """2-layer LSTM LM, vocabulary 33278, width 1500: 11 tensors, 135,891,278 elements."""
    v, h = 33278, 1500
    s = [v * h]
    for _ in range(2):
        s += [4 * h * h, 4 * h * h, 4 * h, 4 * h]
    s += [h * v, v]
    return s


def bert_large_sizes() -> List[int]:
    """BERT-large encoder + word embedding: 385 tensors, 333,563,904 elements."""
    d, f, v = 1024, 4096, 30522
    s = [v * d]
    for _ in range(24):
        for _ in range(4):  # Q, K, V, O
            s += [d * d, d]
        s += [d * f, f, f * d, d]
        s += [d, d, d, d]  # two LayerNorms (gamma, beta)
    return s


def gpt2_medium_sizes() -> List[int]:
    """GPT-2 medium: 292 tensors, 354,823,168 elements."""
    d, v, ctx = 1024, 50257, 1024
    s = [v * d, ctx * d]
    for _ in range(24):
        s += [d, d, d * 3 * d, 3 * d, d * d, d, d, d, d * 4 * d, 4 * d, 4 * d * d, d]
    s += [d, d]
    return s


# --------------------------------------------------------------------------
# Workload descriptions
# --------------------------------------------------------------------------
@dataclass
class Workload:
    name: str
    sizes: List[int]
    n_workers: int
    density: float
    seed: int
    dist: str                      # "gauss" | "laplace" | "lstm_rows"
    scale_lo: float
    scale_hi: float
    scale_is_norm: bool = False    # True: the drawn number is the tensor's target L2 norm
    steps: int = 1
    sparse_tensors: List[int] = field(default_factory=list)
    row_len: int = 0
    row_keep: float = 1.0

    @property
    def n_g(self) -> int:
        return int(sum(self.sizes))

    @property
    def k(self) -> int:
        return max(1, int(math.floor(float(self.n_g) * self.density)))

    # ----- scales ---------------------------------------------------------
    def scales(self) -> np.ndarray:
        """One positive number per tensor, log-uniform in [scale_lo, scale_hi]."""
        rng = np.random.default_rng(np.random.SeedSequence([self.seed, 0xDEF7]))
        u = rng.uniform(math.log(self.scale_lo), math.log(self.scale_hi), size=len(self.sizes))
        s = np.exp(u)
        if self.scale_is_norm:
            s = s / np.sqrt(np.asarray(self.sizes, dtype=np.float64))
        return s

    # ----- one step's gradient ---------------------------------------------
    def gradient(self, step: int = 0, out: np.ndarray | None = None) -> np.ndarray:
        """The flat fp32 gradient of training step ``step`` (already scaled by the learning rate)."""
        n = self.n_g
        g = out if out is not None else np.empty(n, dtype=np.float32)
        assert g.dtype == np.float32 and g.size == n
        scales = self.scales()
        children = np.random.SeedSequence([self.seed, step]).spawn(len(self.sizes))
        pos = 0
        for t, size in enumerate(self.sizes):
            rng = np.random.default_rng(children[t])
            view = g[pos:pos + size]
            if self.dist == "laplace":
                view[:] = rng.laplace(0.0, scales[t], size=size).astype(np.float32)
            else:
                rng.standard_normal(size=size, dtype=np.float32, out=view)
                view *= np.float32(scales[t])
                if self.dist == "lstm_rows" and t in self.sparse_tensors:
                    rows = size // self.row_len
                    keep = rng.random(rows) < self.row_keep
                    view.reshape(rows, self.row_len)[~keep, :] = 0.0
            pos += size
        return g


def device_gradient(w: "Workload", step: int, device, out=None):
    """The same distribution as ``Workload.gradient`` drawn on the GPU with torch's generator
    (seeded by (seed, step); NOT the same numbers as the host draw): a benchmark needs a fresh
    vector every step and the host generator takes seconds per draw at full size.  Input
    generation only — nothing of the method is computed here."""
    import torch
    gen = torch.Generator(device=device)
    gen.manual_seed(((w.seed & 0xFFFF) << 32) + 0xD00D0000 + int(step))
    g = out if out is not None else torch.empty(w.n_g, dtype=torch.float32, device=device)
    scales = w.scales()
    pos = 0
    for t, size in enumerate(w.sizes):
        view = g[pos:pos + size]
        if w.dist == "laplace":
            u = torch.rand(size, generator=gen, device=device, dtype=torch.float32) - 0.5
            view.copy_(-float(scales[t]) * torch.sign(u) * torch.log1p(-2.0 * u.abs()).clamp_(min=-80.0))
        else:
            view.normal_(0.0, float(scales[t]), generator=gen)
            if w.dist == "lstm_rows" and t in w.sparse_tensors:
                rows = size // w.row_len
                keep = torch.rand(rows, generator=gen, device=device) < w.row_keep
                view.view(rows, w.row_len).mul_(keep.to(torch.float32).unsqueeze(1))
        pos += size
    return g


def tiny() -> Workload:
    return Workload("tiny", tiny_sizes(), 4, 0.01, 0, "gauss", 1e-4, 1e-1)


def resnet18() -> Workload:
    return Workload("resnet18", resnet18_sizes(), 16, 0.01, 1, "laplace", 1e-5, 1e-2)


def lstm_lm() -> Workload:
    return Workload("lstm_lm", lstm_lm_sizes(), 16, 0.001, 2, "lstm_rows", 1e-3, 1e-2, steps=10,
                    sparse_tensors=[0, 9], row_len=1500, row_keep=0.05)


def bert_large() -> Workload:
    return Workload("bert_large", bert_large_sizes(), 32, 0.001, 3, "gauss", 1e-2, 1e2, scale_is_norm=True)


def gpt2_medium(n_workers: int = 16, density: float = 0.01) -> Workload:
    return Workload("gpt2_medium", gpt2_medium_sizes(), n_workers, density, 4, "gauss", 1e-4, 1e-1)


def scaled_down(w: Workload, factor: int, name: str | None = None) -> Workload:
    """The same tensor list with every size divided by ``factor`` (at least 1 element):
    keeps the mix of huge and tiny tensors at a size the CPU oracle sorts in seconds."""
    sizes = [max(1, s // factor) for s in w.sizes]
    row_len = w.row_len
    if w.dist == "lstm_rows":
        # keep whole rows in the row-sparse tensors
        for t in w.sparse_tensors:
            sizes[t] = max(row_len, (sizes[t] // row_len) * row_len)
    return Workload(name or (w.name + "_div%d" % factor), sizes, w.n_workers, w.density, w.seed, w.dist,
                    w.scale_lo, w.scale_hi, w.scale_is_norm, w.steps, list(w.sparse_tensors), row_len, w.row_keep)


WORKLOADS: dict[str, Callable[[], Workload]] = {
    "tiny": tiny,
    "resnet18": resnet18,
    "lstm_lm": lstm_lm,
    "bert_large": bert_large,
    "gpt2_medium": gpt2_medium,
}


# --------------------------------------------------------------------------
# Adversarial vectors for edge-case tests (pure data, no method arithmetic)
# --------------------------------------------------------------------------
def adversarial_vector(kind: str, n: int, seed: int = 0) -> np.ndarray:
    rng = np.random.default_rng(np.random.SeedSequence([seed, 0xAD]))
    if kind == "all_equal":
        return np.full(n, 0.25, dtype=np.float32)
    if kind == "all_zero":
        return np.zeros(n, dtype=np.float32)
    if kind == "signed_zero":
        x = np.zeros(n, dtype=np.float32)
        x[::2] = -0.0
        return x
    if kind == "mostly_zero":
        x = np.zeros(n, dtype=np.float32)
        m = rng.random(n) < 0.05
        x[m] = rng.standard_normal(int(m.sum()), dtype=np.float32)
        return x
    if kind == "outlier":
        x = (rng.standard_normal(n, dtype=np.float32) * np.float32(1e-3))
        x[n // 3] = np.float32(-1e6)
        return x
    if kind == "few_values":
        vals = np.array([0.5, -0.5, 0.25, 1.0, -1.0, 0.125, 3.0, -3.0], dtype=np.float32)
        return vals[rng.integers(0, vals.size, size=n)]
    if kind == "bf16_like":
        x = rng.standard_normal(n, dtype=np.float32)
        b = x.view(np.uint32) & np.uint32(0xFFFF0000)
        return b.view(np.float32).copy()
    if kind == "denormal":
        b = rng.integers(0, 1 << 23, size=n, dtype=np.uint32)
        b[::3] |= np.uint32(0x80000000)
        return b.view(np.float32).copy()
    if kind == "wide_exponent":
        e = rng.integers(-60, 60, size=n)
        return (rng.standard_normal(n) * np.exp2(e)).astype(np.float32)
    if kind == "gauss":
        return rng.standard_normal(n, dtype=np.float32)
    raise ValueError(kind)
