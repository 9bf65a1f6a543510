"""The single-launch Gram form for many workers with short rows (17 <= m <= 128, the step's
differences in shared memory) against the CPU oracle, against single steps, and against the
literal form."""
import numpy as np
import pytest
import torch

from oracle import PairBalanceOracle
from paper_2302_00845_b200 import binding, synth
from parity import Pair, TAU

pytestmark = pytest.mark.gpu


def grads(m, d, dtype, seed, mean=0.1):
    g = torch.Generator(device="cuda").manual_seed(seed)
    return (torch.randn(2, m, d, generator=g, device="cuda") + mean).to(
        torch.float32 if dtype == "f32" else torch.bfloat16)


@pytest.mark.parametrize("m,n,d,dtype", [
    (100, 8, 16, "f32"),      # the synthetic herding study's largest worker count
    (50, 6, 16, "f32"),
    (20, 10, 16, "bf16"),
    (128, 4, 96, "f32"),      # the most workers this form holds
    (32, 6, 1024, "f32"),
    (17, 4, 2000, "bf16"),
    (33, 6, 1000, "f32"),     # rows longer than one 64-column chunk of the fp32 sums, ragged end
    (64, 4, 516, "f32"),
])
def test_small_form_matches_oracle(m, n, d, dtype, monkeypatch):
    if d > 64:
        monkeypatch.setenv("CDGRAB_FORCE_PATH", "fused")     # by default this form serves rows of <= 64 columns
    pr = Pair(m, n, d, dtype)
    try:
        assert pr.gpu.path == "fused"
        pr.begin()
        for k in range(n // 2):
            pr.step(grads(m, d, dtype, 13 * m + k))
        rep = pr.end()
        print(f"small m={m} n={n} d={d} {dtype}:", rep)
        assert rep.raw_agreement == 1.0
        assert pr.gpu.launch_count == n // 2
    finally:
        pr.close()


@pytest.mark.parametrize("m,n,d,dtype", [(40, 10, 64, "f32"), (100, 12, 16, "f32"), (24, 8, 512, "bf16")])
def test_staged_steps_in_one_launch_equal_single_steps(m, n, d, dtype, monkeypatch):
    if d > 64:
        monkeypatch.setenv("CDGRAB_FORCE_PATH", "fused")
    g = torch.stack([grads(m, d, dtype, 700 + k) for k in range(n // 2)]).contiguous()
    with binding.CdGrab(m, n, d, dtype) as a, binding.CdGrab(m, n, d, dtype) as b:
        assert a.path == "fused"
        a.begin_epoch(); b.begin_epoch()
        before = a.launch_count
        a.step_many(g)
        assert a.launch_count - before == 1
        for k in range(n // 2):
            b.step(g[k])
        assert torch.equal(a.signs(), b.signs())
        assert torch.equal(a.r(), b.r())
        assert torch.equal(a.margins(), b.margins())
        assert torch.equal(a.next_perms(), b.next_perms())
        assert a.status() == binding.OK and b.status() == binding.OK


def test_small_and_literal_forms_agree(monkeypatch):
    m, n, d = 48, 8, 256
    out = {}
    for path in ("fused", "literal"):
        monkeypatch.setenv("CDGRAB_FORCE_PATH", path)
        with binding.CdGrab(m, n, d, "f32") as h:
            assert h.path == path
            h.begin_epoch()
            for k in range(n // 2):
                h.step(grads(m, d, "f32", 70 + k, mean=0.3))
            out[path] = (h.signs().cpu(), h.r().cpu(), h.margins().cpu())
    assert torch.equal(out["literal"][0], out["fused"][0])
    np.testing.assert_allclose(out["literal"][1].numpy(), out["fused"][1].numpy(), rtol=0, atol=2e-5)
    np.testing.assert_allclose(out["literal"][2].numpy(), out["fused"][2].numpy(), rtol=1e-3, atol=1e-6)


def test_randomized_rule_and_mean_on_the_small_form():
    m, n, d, dtype = 40, 8, 64, "f32"
    w = 0.2 * d
    gpu = binding.CdGrab(m, n, d, dtype)
    cpu = PairBalanceOracle(m, n, d)
    gen = torch.Generator(device="cuda").manual_seed(5)
    mean = torch.empty(2, d, dtype=torch.float32, device="cuda")
    try:
        assert gpu.path == "fused"
        gpu.begin_epoch(); cpu.begin_epoch()
        for k in range(n // 2):
            g = grads(m, d, dtype, 300 + k)
            u = torch.rand(m, generator=gen, device="cuda")
            if k % 2 == 0:
                gpu.step_randomized(g, u, w)
                s = gpu.signs()[:, k].cpu().numpy()
                cpu.step_randomized(synth.to_host(g), u.cpu().numpy().astype(np.float64), w, replay=s, tau=TAU[dtype])
            else:
                gpu.step_mean(g, mean)
                s = gpu.signs()[:, k].cpu().numpy()
                cpu.step(synth.to_host(g), replay=s, tau=TAU[dtype])
                want = g.double().mean(dim=1)
                assert (mean.double() - want).abs().max().item() <= 2e-6 * max(1.0, want.abs().max().item())
        assert cpu.mismatches == 0
        assert gpu.status() == binding.OK
    finally:
        gpu.destroy(); cpu.close()
