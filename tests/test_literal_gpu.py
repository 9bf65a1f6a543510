"""The literal form of the step (Algorithm 6 applied worker by worker in one CTA, short rows)
against the CPU oracle, and against the Gram-form paths."""
import numpy as np
import pytest
import torch

from paper_2302_00845_b200 import binding
from parity import Pair

pytestmark = pytest.mark.gpu


def grads(m, d, dtype, seed, mean=0.1):
    g = torch.Generator(device="cuda").manual_seed(seed)
    return (torch.randn(2, m, d, generator=g, device="cuda") + mean).to(
        torch.float32 if dtype == "f32" else torch.bfloat16)


@pytest.mark.parametrize("m,n,d,dtype", [
    (100, 8, 16, "f32"),      # the synthetic herding study's largest worker count
    (50, 6, 16, "f32"),
    (20, 10, 16, "bf16"),
    (4, 64, 1024, "f32"),     # the tiny workload's shape
    (8, 8, 4096, "f32"),      # the logistic-regression workload's shape: every thread of the CTA busy
    (33, 6, 1000, "f32"),     # a ragged last warp
    (1, 12, 4, "f32"),        # one worker, one 4-column group
    (1024, 2, 8, "f32"),      # the most workers a step may have
    (7, 6, 2052, "bf16"),
])
def test_literal_path_matches_oracle(m, n, d, dtype, monkeypatch):
    monkeypatch.setenv("CDGRAB_FORCE_PATH", "literal")
    pr = Pair(m, n, d, dtype)
    try:
        assert pr.gpu.path == "literal"
        pr.begin()
        for k in range(n // 2):
            pr.step(grads(m, d, dtype, 31 * m + k))
        rep = pr.end()
        print(f"literal m={m} n={n} d={d} {dtype}:", rep)
        assert rep.raw_agreement == 1.0
    finally:
        pr.close()


def test_default_paths_for_short_rows():
    with binding.CdGrab(100, 4, 16, "f32") as h:
        assert h.path == "fused"         # many workers, differences fit shared memory: Gram form in one CTA
    with binding.CdGrab(1024, 4, 64, "f32") as h:
        assert h.path == "literal"       # more workers than that form holds
    with binding.CdGrab(8, 4, 1024, "f32") as h:
        assert h.path == "literal"
    with binding.CdGrab(8, 4, 2048, "f32") as h:
        assert h.path == "fused"
    with binding.CdGrab(64, 4, 2048, "f32") as h:
        assert h.path == "fma"


@pytest.mark.parametrize("m,n,d,dtype", [(8, 16, 4096, "f32"), (40, 10, 64, "f32"), (4, 64, 1024, "bf16")])
def test_staged_epoch_in_one_launch_equals_single_steps(m, n, d, dtype, monkeypatch):
    """cdgrab_step_many on this path runs the steps of the call in one launch with r in registers,
    rounded to fp32 once per step as single launches store it: same bits."""
    monkeypatch.setenv("CDGRAB_FORCE_PATH", "literal")
    g = torch.stack([grads(m, d, dtype, 900 + k) for k in range(n // 2)]).contiguous()
    with binding.CdGrab(m, n, d, dtype) as a, binding.CdGrab(m, n, d, dtype) as b:
        a.begin_epoch(); b.begin_epoch()
        before = a.launch_count
        a.step_many(g)
        assert a.launch_count - before == 1
        for k in range(n // 2):
            b.step(g[k])
        assert torch.equal(a.signs(), b.signs())
        assert torch.equal(a.next_perms(), b.next_perms())
        assert torch.equal(a.r(), b.r())
        assert torch.equal(a.margins(), b.margins())
        assert a.status() == binding.OK and b.status() == binding.OK


def test_literal_and_gram_forms_agree(monkeypatch):
    m, n, d = 8, 8, 2048
    out = {}
    for path in ("literal", "fused"):
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
