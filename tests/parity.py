"""Shared harness of the GPU parity tests: runs the CUDA library (through its C ABI binding)
and the CPU oracle on the same bytes and applies the acceptance rule.

Acceptance rule: permutations bit-exact; signs equal at every position where
|<r,c>| > tau * ||r|| * ||c|| (tau = 1e-6 for fp32 inputs, 1e-3 for bf16 inputs); inside that
band the oracle adopts the GPU's sign, continues, and the position is counted as a near-tie;
final r within relative L2 error 1e-5 (fp32 inputs) or 2e-3 (bf16 storage, fp32 accumulate).
"""
from __future__ import annotations

import dataclasses

import numpy as np
import torch

from oracle import PairBalanceOracle
from paper_2302_00845_b200 import binding, synth

TAU = {"f32": 1e-6, "bf16": 1e-3}
R_TOL = {"f32": 1e-5, "bf16": 2e-3}


@dataclasses.dataclass
class ParityReport:
    positions: int
    near_ties: int
    mismatches: int
    raw_agreement: float
    r_rel_err: float
    path: str

    def __str__(self):
        return (f"path={self.path} positions={self.positions} near_ties={self.near_ties} "
                f"mismatches={self.mismatches} raw_agree={self.raw_agreement:.6f} "
                f"r_rel_err={self.r_rel_err:.3e}")


def rel_l2(a: np.ndarray, b: np.ndarray) -> float:
    den = float(np.linalg.norm(b))
    return float(np.linalg.norm(a - b)) / den if den > 0 else float(np.linalg.norm(a))


class Pair:
    """One CUDA handle and one oracle fed with identical bytes."""

    def __init__(self, m, n, d, dtype, perms0=None):
        self.m, self.n, self.d, self.dtype = m, n, d, dtype
        self.gpu = binding.CdGrab(m, n, d, dtype)
        self.cpu = PairBalanceOracle(m, n, d)
        if perms0 is not None:
            p = np.ascontiguousarray(perms0, dtype=np.int32)
            self.gpu.set_perms(p)
            self.cpu.set_perms(p)
        self.raw_equal = 0
        self.positions = 0
        self.k = 0

    def begin(self):
        self.gpu.begin_epoch()
        self.cpu.begin_epoch()
        self.k = 0

    def step(self, grads: torch.Tensor):
        """grads: CUDA tensor [2][m][d]."""
        self.gpu.step(grads)
        s = self.gpu.signs()[:, self.k].cpu().numpy()
        assert set(np.unique(s).tolist()) <= {-1, 1}, s
        self.cpu.step(synth.to_host(grads), replay=s, tau=TAU[self.dtype])
        own = self.cpu.own_signs()[:, self.k]
        self.raw_equal += int((own == s).sum())
        self.positions += self.m
        self.k += 1

    def check_partial(self) -> ParityReport:
        """Signs, filled permutation slots and r after the steps taken so far."""
        k = self.k
        gs = self.gpu.signs().cpu().numpy()
        cs = self.cpu.signs()
        assert self.cpu.mismatches == 0, f"{self.cpu.mismatches} sign mismatches outside the tie band"
        assert np.array_equal(gs[:, :k], cs[:, :k])
        gp = self.gpu.next_perms().cpu().numpy()
        cp = self.cpu.perm_next()
        n = self.n
        assert np.array_equal(gp[:, :k], cp[:, :k])
        assert np.array_equal(gp[:, n - k:], cp[:, n - k:])
        err = rel_l2(self.gpu.r().cpu().numpy().astype(np.float64), self.cpu.r())
        assert err <= R_TOL[self.dtype], f"r relative L2 error {err:.3e}"
        self.gpu.check_status()
        return ParityReport(self.positions, self.cpu.near_ties, self.cpu.mismatches,
                            self.raw_equal / max(1, self.positions), err, self.gpu.path)

    def end(self) -> ParityReport:
        rep = self.check_partial()
        out = torch.empty(self.m, self.n, dtype=torch.int32, device="cuda")
        self.gpu.end_epoch(out)
        torch.cuda.synchronize()
        want = self.cpu.end_epoch()
        got = out.cpu().numpy()
        assert np.array_equal(got, want), "next-epoch permutations differ"
        for i in range(self.m):
            assert np.array_equal(np.sort(got[i]), np.arange(self.n))
        assert np.array_equal(self.gpu.perms().cpu().numpy(), want)
        return rep

    def close(self):
        self.gpu.destroy()
        self.cpu.close()


def run_stream_epoch(wl: synth.Workload, steps=None, perms0=None) -> ParityReport:
    """One epoch (or its first `steps` steps) of a synthetic gradient stream on both sides."""
    gs = synth.GradientStream(wl, device="cuda")
    pr = Pair(wl.m, wl.n, wl.d, wl.dtype, perms0)
    try:
        pr.begin()
        total = wl.steps_per_epoch if steps is None else steps
        buf = None
        for k in range(total):
            buf = gs.step(k, out=buf)
            pr.step(buf)
        return pr.end() if total == wl.steps_per_epoch else pr.check_partial()
    finally:
        pr.close()
