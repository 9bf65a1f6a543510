"""Seeded synthetic gradient streams shaped like the paper's workloads.

This module only draws inputs; it holds none of the method's arithmetic, so both the CUDA
path and the CPU oracle can be fed from it (the oracle receives the same bytes, copied to
the host).  ``N(a, b)`` below means mean a and VARIANCE b.

The five workloads take the shapes of the settings the paper runs (Section 5 and
Appendix C: logistic regression, an LSTM language model, a GPT-2-sized model, with m
workers of n local examples each); the datasets themselves are not used.
"""
from __future__ import annotations

import dataclasses
import math

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    m: int          # logical workers
    n: int          # examples per worker (even)
    d: int          # gradient dimension
    dtype: str      # "f32" or "bf16" storage of the gradients
    epochs: int
    kind: str       # recipe selector
    seed: int = 0

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def elem_bytes(self):
        return 4 if self.dtype == "f32" else 2

    @property
    def steps_per_epoch(self):
        return self.n // 2

    def scaled(self, **kw) -> "Workload":
        """Same recipe at other sizes (tests use reduced d / n)."""
        return dataclasses.replace(self, **kw)


WORKLOADS = {
    "tiny": Workload("tiny", 4, 64, 1024, "f32", 1, "mean_offset"),
    "logreg": Workload("logreg", 8, 1024, 4096, "f32", 3, "logreg"),
    "mid": Workload("mid", 16, 4096, 1 << 20, "f32", 1, "heavy_tail"),
    "lstm": Workload("lstm", 32, 512, 13_500_000, "bf16", 1, "layer_scale"),
    "gpt2": Workload("gpt2", 64, 128, 124_000_000, "bf16", 1, "low_rank"),
}

# 2-layer LSTM, hidden 650, vocabulary 10k: embedding, 2 x (W_ih, W_hh, biases), decoder
# bias, remainder up to the stated d.  Used as proportions when d is scaled down.
_LSTM_BLOCKS = (6_500_000, 1_690_000, 1_690_000, 5_200, 1_690_000, 1_690_000, 5_200, 10_000,
                219_600)


def _gen(device, *key: int) -> torch.Generator:
    g = torch.Generator(device=device)
    h = 0x9E3779B97F4A7C15
    for k in key:
        h = (h ^ (int(k) + 0x7F4A7C15 + ((h << 6) & 0xFFFFFFFFFFFFFFFF) + (h >> 2))) & 0x7FFFFFFFFFFFFFFF
    g.manual_seed(h)
    return g


class GradientStream:
    """Per-step stale-gradient buffers ``[2][m][d]`` for one workload.

    ``step(k, epoch)`` returns the two consecutive gather buffers of pair index k: slab 0
    holds, for every worker, the gradient at position 2k of its current order, slab 1 the
    one at position 2k+1.  Every (epoch, k) has its own generator seed, so any step can be
    drawn again on its own.
    """

    def __init__(self, wl: Workload, device="cpu"):
        if wl.kind == "logreg":
            raise ValueError("the logistic-regression workload is drawn by LogregProblem")
        self.wl = wl
        self.device = torch.device(device)
        m, d = wl.m, wl.d
        g0 = _gen(self.device, wl.seed, 0xA11)
        if wl.kind == "mean_offset":
            # shared mean offset N(0, 0.1) per coordinate
            self.mu = torch.randn(d, generator=g0, device=self.device) * math.sqrt(0.1)
        elif wl.kind == "heavy_tail":
            # shared mean N(0,1); a fixed 1 % of the coordinates is scaled x10
            self.mu = torch.randn(d, generator=g0, device=self.device)
            self.scale = torch.ones(d, device=self.device)
            nh = max(1, d // 100)
            idx = torch.randperm(d, generator=g0, device=self.device)[:nh]
            self.scale[idx] = 10.0
            self.mu = self.mu * self.scale
        elif wl.kind == "layer_scale":
            # per-layer scale 10^U(-2,0), one draw per block of the LSTM layout
            u = torch.rand(len(_LSTM_BLOCKS), generator=g0, device=self.device) * -2.0
            scales = torch.pow(torch.tensor(10.0, device=self.device), u)
            total = sum(_LSTM_BLOCKS)
            bounds, acc = [], 0
            for b in _LSTM_BLOCKS:
                acc += b
                bounds.append(min(d, (acc * d + total - 1) // total))
            bounds[-1] = d
            self.scale = torch.empty(d, device=self.device)
            lo = 0
            for hi, s in zip(bounds, scales):
                self.scale[lo:hi] = s
                lo = hi
        elif wl.kind == "low_rank":
            # shared rank-16 factor, kept in bf16 as [16][d]
            self.rank = 16
            self.U = torch.empty(self.rank, d, dtype=torch.bfloat16, device=self.device)
            for q in range(self.rank):
                self.U[q] = torch.randn(d, generator=g0, device=self.device).to(torch.bfloat16)
        else:
            raise ValueError(wl.kind)

    def _rows(self, gen, count: int) -> torch.Tensor:
        """`count` gradient rows [count][d] in fp32 from one pass over the generator."""
        wl, d, dev = self.wl, self.wl.d, self.device
        if wl.kind == "mean_offset":
            return self.mu + torch.randn(count, d, generator=gen, device=dev)
        if wl.kind == "heavy_tail":
            return self.mu + torch.randn(count, d, generator=gen, device=dev) * (math.sqrt(0.5) * self.scale)
        if wl.kind == "layer_scale":
            return torch.randn(count, d, generator=gen, device=dev) * (math.sqrt(1e-3) * self.scale)
        # low_rank: per-coordinate variance 1e-4, half in the shared rank-16 subspace
        a = torch.randn(count, self.rank, generator=gen, device=dev)
        low = (a.to(torch.bfloat16) @ self.U).float() / math.sqrt(2.0 * self.rank)
        eps = torch.randn(count, d, generator=gen, device=dev) / math.sqrt(2.0)
        return (low + eps) * 1e-2

    def step(self, k: int, epoch: int = 0, out: torch.Tensor | None = None) -> torch.Tensor:
        wl = self.wl
        if out is None:
            out = torch.empty(2, wl.m, wl.d, dtype=wl.torch_dtype, device=self.device)
        gen = _gen(self.device, wl.seed, 0xB22, epoch, k)
        # as many rows per draw as keep the fp32 temporaries near 1 GiB: small shapes come out of a
        # single call, the largest ones two rows at a time
        flat = out.view(2 * wl.m, wl.d)
        per = max(1, min(2 * wl.m, (1 << 28) // wl.d))
        for lo in range(0, 2 * wl.m, per):
            hi = min(2 * wl.m, lo + per)
            flat[lo:hi] = self._rows(gen, hi - lo).to(wl.torch_dtype)
        return out


class LogregProblem:
    """Logistic-regression inputs: X[m][n][d] ~ N(0,1), w* ~ N(0,1/d),
    y ~ Bernoulli(sigmoid(X w*)), evaluation point w ~ N(0,0.01) held fixed."""

    def __init__(self, wl: Workload, device="cpu"):
        assert wl.kind == "logreg"
        self.wl = wl
        dev = torch.device(device)
        g0 = _gen(dev, wl.seed, 0xC33)
        self.X = torch.randn(wl.m, wl.n, wl.d, generator=g0, device=dev)
        w_star = torch.randn(wl.d, generator=g0, device=dev) / math.sqrt(wl.d)
        p = torch.sigmoid(self.X @ w_star)
        self.y = (torch.rand(wl.m, wl.n, generator=g0, device=dev) < p).float()
        self.w = torch.randn(wl.d, generator=g0, device=dev) * 0.1


def herding_vectors(total: int, d: int = 16, seed: int = 0, device="cpu") -> torch.Tensor:
    """The vectors of the paper's synthetic herding study (experiment-details appendix, simulated
    ablation): `total` points uniform in [0,1)^d, zero-centred, then scaled to unit Euclidean norm."""
    g = _gen(torch.device(device), seed, 0xD44, total, d)
    z = torch.rand(total, d, generator=g, device=device)
    z = z - z.mean(dim=0)
    return (z / z.norm(dim=1, keepdim=True)).contiguous()


def random_orders(m: int, n: int, seed: int, device="cpu") -> torch.Tensor:
    """m independent uniformly random permutations of [0, n) as int32 [m][n] (random reshuffling)."""
    g = _gen(torch.device(device), seed, 0xE55, m, n)
    return torch.argsort(torch.rand(m, n, generator=g, device=device), dim=1).to(torch.int32).contiguous()


def bf16_bits(t: torch.Tensor):
    """Host numpy view of a bf16 tensor as uint16 bit patterns (what the oracle reads)."""
    import numpy as np
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def to_host(t: torch.Tensor):
    """Host numpy array of the exact bytes of a gradient tensor (f32, or bf16 bit patterns)."""
    if t.dtype == torch.bfloat16:
        return bf16_bits(t)
    return t.detach().contiguous().cpu().numpy()
