"""Parity of the tensor-core (tcgen05) Gram path against the CPU oracle, bf16 inputs."""
import os

import numpy as np
import pytest
import torch

from paper_2302_00845_b200 import binding
from parity import Pair

pytestmark = pytest.mark.gpu


def grads(m, d, seed, mean=0.0, scale=1.0):
    g = torch.Generator(device="cuda").manual_seed(seed)
    return (torch.randn(2, m, d, generator=g, device="cuda") * scale + mean).to(torch.bfloat16)


def run(m, n, d, seed, mean=0.0, scale=1.0):
    pr = Pair(m, n, d, "bf16")
    try:
        assert pr.gpu.path == "umma"
        pr.begin()
        for k in range(n // 2):
            pr.step(grads(m, d, seed * 100 + k, mean, scale))
        return pr.end()
    finally:
        pr.close()


@pytest.mark.parametrize("m,n,d", [
    (17, 4, 5000),           # 51 rows of bf16 terms, ragged last block, fewer blocks than SMs
    (24, 4, 200_000),        # 72 rows
    (42, 4, 70_000),         # 126 rows: the term rows just fit one 128-row tile
    (32, 6, 1_000_000 + 8),  # many accumulator chunks per CTA
    (8, 4, 100_000),         # forced onto this path (the FMA kernels are the default for m <= 16)
    (43, 4, 70_004),         # 129 term rows: past one 128-row tile; d a multiple of 4 only
    (50, 4, 100_000),
    (64, 4, 8192),           # the largest m: 192 term rows; fewer blocks than SMs
    (61, 4, 150_000),        # eight converter warps (six would take six rows per thread), 3 idle row slots
    (60, 4, 150_000),        # the last m on six converter warps
    (32, 4, 150_000),        # the last m with MMA M = 64 (2m = 64 rows of A)
    (33, 4, 150_000),        # the first m with M = 128
    (64, 6, 1_000_000 + 4),  # many accumulator chunks per CTA, ragged last block
    (64, 4, 64 * 148 * 2 + 12),  # two blocks per CTA, odd tail
    (33, 4, 300_000),
])
def test_fp32_gradients_on_the_tensor_cores(m, n, d, monkeypatch):
    """fp32 inputs: the differences go through the MMA as three bf16 terms each, formed inside the
    kernel; the fp32 sign tolerance (1e-6) applies."""
    monkeypatch.setenv("CDGRAB_FORCE_PATH", "umma")
    pr = Pair(m, n, d, "f32")
    try:
        assert pr.gpu.path == "umma"
        pr.begin()
        g = torch.Generator(device="cuda").manual_seed(m + d % 11)
        for k in range(n // 2):
            pr.step(torch.randn(2, m, d, generator=g, device="cuda") + 0.1)
        rep = pr.end()
        print(f"umma fp32 m={m} n={n} d={d}:", rep)
        assert rep.raw_agreement == 1.0
    finally:
        pr.close()


@pytest.mark.parametrize("m,n,d", [
    (4, 4, 4096),          # one 16-row box, few K blocks: fewer CTAs than SMs
    (64, 4, 8192),         # full 128-row tile
    (32, 4, 64 * 148 * 3 + 8),   # every SM busy, ragged last K block
    (17, 6, 100_000),      # 2m not a multiple of 16
    (64, 4, 1_000_000),    # many pipeline turns per CTA
    (32, 6, 1_000_000 + 24),   # two blocks per MMA, whole stages per CTA, ragged last block
    (20, 4, 300_000),      # two blocks per MMA with unused row groups in both halves
    (18, 4, 64 * 8 * 40),  # fewer stages than SMs; 2m = 36: a ragged row group beside the 4-D copy
    (33, 4, 200_000),      # first m past the two-block mode
])
def test_umma_shapes(m, n, d, monkeypatch):
    monkeypatch.setenv("CDGRAB_FORCE_PATH", "umma")
    rep = run(m, n, d, seed=m + d % 7)
    print(f"umma m={m} n={n} d={d}:", rep)
    assert rep.raw_agreement > 0.9


def test_umma_with_common_mean(monkeypatch):
    """A shared mean ten times the noise: the raw-gradient Gram cancels in four terms."""
    monkeypatch.setenv("CDGRAB_FORCE_PATH", "umma")
    rep = run(16, 6, 262_144, seed=3, mean=1.0, scale=0.1)
    print("umma common mean:", rep)


def test_umma_matches_fma_path_signs(monkeypatch):
    m, n, d = 8, 6, 65536
    out = {}
    for path in ("umma", "fma"):
        monkeypatch.setenv("CDGRAB_FORCE_PATH", path)
        with binding.CdGrab(m, n, d, "bf16") as h:
            assert h.path == path
            h.begin_epoch()
            for k in range(n // 2):
                h.step(grads(m, d, 500 + k, mean=0.2))
            out[path] = (h.signs().cpu(), h.r().cpu(), h.margins().cpu())
            assert h.status() == binding.OK
    assert torch.equal(out["umma"][0], out["fma"][0])
    assert torch.equal(out["umma"][1], out["fma"][1])   # same signs -> same fp32 update order
    np.testing.assert_allclose(out["umma"][2].numpy(), out["fma"][2].numpy(), rtol=1e-3, atol=1e-6)


@pytest.mark.parametrize("mean,scale", [(0.3, 0.1), (1.0, 0.1)])
def test_umma_long_rows_with_common_mean(mean, scale, monkeypatch):
    """Rows of 16 M columns (about 108 K columns per CTA, many accumulator chunks) whose shared
    mean is 3x / 10x the per-example noise: the four-term cancellation G = H - H - H + H has to
    survive the tensor core's accumulation error."""
    monkeypatch.setenv("CDGRAB_FORCE_PATH", "umma")
    m, n, d = 8, 4, 16_000_000
    pr = Pair(m, n, d, "bf16")
    try:
        assert pr.gpu.path == "umma"
        pr.begin()
        for k in range(n // 2):
            pr.step(grads(m, d, 40 + k, mean, scale))
        rep = pr.end()
        print(f"umma long rows mean={mean} scale={scale}:", rep)
        assert rep.raw_agreement == 1.0
    finally:
        pr.close()


@pytest.mark.parametrize("m,n,d", [
    (65, 4, 8192),            # first m past one 128-row tile of raw rows; fewer blocks than SMs
    (72, 4, 100_000),         # passes of 40 rows
    (73, 4, 70_008),          # ragged last block (d a multiple of 8 only)
    (100, 4, 300_000),
    (128, 4, 64 * 148 * 2 + 8),   # the largest m: N = 256, both TMEM buffers full width
    (128, 6, 1_000_000),      # several accumulator chunks per CTA
    (113, 4, 120_000),        # eight converter warps, passes of 64 rows of which 57 / 56 are real
    (112, 4, 120_000),        # the last m on six converter warps (passes of 56 rows)
])
def test_bf16_more_than_64_workers_on_the_tensor_cores(m, n, d):
    """bf16 gradients with 65..128 workers: the differences go through the MMA as two bf16 terms
    each, formed inside the kernel; the bf16 sign tolerance (1e-3) applies."""
    if os.environ.get("CDGRAB_UMMA_BF16_WIDE") == "0":
        pytest.skip("the knob under test keeps these shapes off the tensor cores")
    rep = run(m, n, d, seed=m + d % 5)
    print(f"umma bf16 wide m={m} n={n} d={d}:", rep)
    assert rep.raw_agreement > 0.9


def test_bf16_wide_matches_the_fma_route(monkeypatch):
    """Same steps with the term-splitting kernel and with the blocked FMA Gram: same signs, same r."""
    m, n, d = 96, 6, 131_072
    out = {}
    for wide in ("1", "0"):
        monkeypatch.setenv("CDGRAB_UMMA_BF16_WIDE", wide)
        with binding.CdGrab(m, n, d, "bf16") as h:
            assert h.path == ("umma" if wide == "1" else "fma")
            h.begin_epoch()
            for k in range(n // 2):
                h.step(grads(m, d, 900 + k, mean=0.2))
            out[wide] = (h.signs().cpu(), h.r().cpu(), h.margins().cpu())
            assert h.status() == binding.OK
    assert torch.equal(out["1"][0], out["0"][0])
    assert torch.equal(out["1"][1], out["0"][1])
    np.testing.assert_allclose(out["1"][2].numpy(), out["0"][2].numpy(), rtol=2e-3, atol=1e-5)
