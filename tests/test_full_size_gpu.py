"""Parity at the full sizes of the large workloads, in the launch configuration bench.py times.

The oracle cannot replay a whole epoch at d = 124 M in test time, so these run the first steps of
the epoch at full (m, d) on both sides: every sign of those steps, the filled permutation slots
and the running sum are compared.  Gradient rows are streamed to the host one worker pair at a
time (two rows of d elements), never a whole step."""
import numpy as np
import pytest
import torch

from oracle import PairBalanceOracle
from paper_2302_00845_b200 import binding, synth
from parity import TAU, R_TOL, rel_l2

pytestmark = pytest.mark.gpu


def run_full(name, steps):
    wl = synth.WORKLOADS[name]
    m, n, d = wl.m, wl.n, wl.d
    gs = synth.GradientStream(wl, device="cuda")
    gpu = binding.CdGrab(m, n, d, wl.dtype)
    cpu = PairBalanceOracle(m, n, d)
    raw = 0
    try:
        gpu.begin_epoch(); cpu.begin_epoch()
        buf = None
        for k in range(steps):
            buf = gs.step(k, out=buf)
            gpu.step(buf)
            s = gpu.signs()[:, k].cpu().numpy()
            for i in range(m):
                got = cpu.balance_one(i, synth.to_host(buf[0, i]), synth.to_host(buf[1, i]),
                                      replay=int(s[i]), tau=TAU[wl.dtype])
                assert got == int(s[i])
            raw += int((cpu.own_signs()[:, k] == s).sum())
        assert cpu.mismatches == 0
        gp = gpu.next_perms().cpu().numpy(); cp = cpu.perm_next()
        assert np.array_equal(gp[:, :steps], cp[:, :steps])
        assert np.array_equal(gp[:, n - steps:], cp[:, n - steps:])
        err = rel_l2(gpu.r().cpu().numpy().astype(np.float64), cpu.r())
        assert err <= R_TOL[wl.dtype], err
        assert gpu.status() == binding.OK
        # accuracy of the GPU's <r,c>: its relative margins against the oracle's fp64 trace
        t, rn, cn = cpu.trace()
        want = np.where(rn * cn > 0, np.abs(t) / np.maximum(rn * cn, 1e-300), 0.0)[:, :steps]
        got = gpu.margins().cpu().numpy()[:, :steps].astype(np.float64)
        margin_err = float(np.abs(got - want).max())
        assert margin_err <= 0.05 * TAU[wl.dtype], margin_err   # far inside the tie band
        print(f"{name} full size, {steps} steps: path={gpu.path} near_ties={cpu.near_ties} "
              f"raw_agree={raw / (m * steps):.4f} r_rel_err={err:.2e} max_margin_err={margin_err:.2e}")
        return gpu.path
    finally:
        gpu.destroy(); cpu.close()


def test_mid_full_size_sampled_steps():
    assert run_full("mid", 6) == "fma"


def test_lstm_full_size_sampled_steps():
    assert run_full("lstm", 3) == "umma"


@pytest.mark.slow
def test_gpt2_full_size_sampled_steps():
    assert run_full("gpt2", 2) == "umma"


def test_logreg_full_size_first_epoch_steps():
    """Workload 2 at full (m, n, d): the first steps of the first epoch, gradients from the
    device kernel, single-launch path."""
    wl = synth.WORKLOADS["logreg"]
    prob = synth.LogregProblem(wl, device="cuda")
    m, n, d = wl.m, wl.n, wl.d
    gpu = binding.CdGrab(m, n, d, "f32")
    cpu = PairBalanceOracle(m, n, d)
    grads = torch.empty(2, m, d, device="cuda")
    steps = 64
    try:
        assert gpu.path == "fused"
        gpu.begin_epoch(); cpu.begin_epoch()
        for k in range(steps):
            gpu.logreg_grads(prob.X, prob.y, prob.w, grads)
            gpu.step(grads)
            s = gpu.signs()[:, k].cpu().numpy()
            cpu.step(synth.to_host(grads), replay=s, tau=TAU["f32"])
        assert cpu.mismatches == 0
        err = rel_l2(gpu.r().cpu().numpy().astype(np.float64), cpu.r())
        assert err <= R_TOL["f32"], err
        gp = gpu.next_perms().cpu().numpy(); cp = cpu.perm_next()
        assert np.array_equal(gp[:, :steps], cp[:, :steps])
        assert np.array_equal(gp[:, n - steps:], cp[:, n - steps:])
    finally:
        gpu.destroy(); cpu.close()
