"""The entry point for callers that must not allocate device memory.

cdgrab_step_noalloc serves code that cannot call cudaMalloc (plug-ins handed only buffers and a
stream, code living inside a framework's caching allocator, loops that cannot afford the
device-wide synchronisation of an allocation).  It keeps its scratch in a fixed array inside the
library, so this test checks what such a caller relies on: two calls in a row, fed the same
gradients as two cdgrab_step calls on a regular handle, leave the same signs and the same
running sum, although the second call finds the first call's leftovers in the shared scratch.

The file name sorts last on purpose: a run that stops at the first failure has then already
run every other test.
"""
import numpy as np
import pytest
import torch

from oracle import PairBalanceOracle
from paper_2302_00845_b200 import binding, synth

pytestmark = pytest.mark.gpu


def _grads(m, d, dtype, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    return (torch.randn(2, m, d, generator=g, device="cuda") + 0.25).to(dtype)


@pytest.mark.parametrize("m,d,dtype", [(8, 65536 + 12, torch.float32), (16, 300_000, torch.float32),
                                       (3, 4096, torch.bfloat16)])
def test_two_calls_match_the_handle_based_step(m, d, dtype, monkeypatch):
    monkeypatch.setenv("CDGRAB_FORCE_PATH", "fma")   # the handle runs the same two-pass kernels,
    monkeypatch.setenv("CDGRAB_FMA_TMA", "0")        # with the same summation order in pass 1
    steps = [_grads(m, d, dtype, 7 * m + k) for k in range(2)]
    name = "f32" if dtype == torch.float32 else "bf16"
    with binding.CdGrab(m, 4, d, name) as h:
        h.begin_epoch()
        for g in steps:
            h.step(g)
        want_signs = h.signs()          # [m][2]
        want_r = h.r()
        assert h.status() == binding.OK

    r = torch.zeros(d, dtype=torch.float32, device="cuda")
    signs = torch.zeros(2, m, dtype=torch.int8, device="cuda")
    binding.step_noalloc(steps[0], r.clone(), signs[0].clone())   # the first call on a device sets up
    torch.cuda.synchronize()
    before = torch.cuda.memory_allocated()
    free_before = torch.cuda.mem_get_info()[0]                   # the driver's own count
    for k, g in enumerate(steps):
        binding.step_noalloc(g, r, signs[k])
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before
    assert torch.cuda.mem_get_info()[0] == free_before
    assert binding.noalloc_status() == binding.OK
    assert torch.equal(signs.t().contiguous(), want_signs)
    # same kernels in the same order: the tests' tolerance for r is 1e-5 relative L2 (fp32 inputs)
    err = (r.double() - want_r.double()).norm() / want_r.double().norm()
    assert float(err) <= 1e-5
    assert torch.equal(r, want_r)


@pytest.mark.parametrize("m,d,dtype", [(16, 70_000, torch.float32), (5, 40_960, torch.bfloat16)])
def test_two_calls_match_the_oracle(m, d, dtype):
    """The same two steps replayed through the CPU oracle: signs outside the tie band, final r."""
    name = "f32" if dtype == torch.float32 else "bf16"
    tau, rtol = (1e-6, 1e-5) if name == "f32" else (1e-3, 2e-3)
    steps = [_grads(m, d, dtype, 11 * m + k) for k in range(2)]
    r = torch.zeros(d, dtype=torch.float32, device="cuda")
    signs = torch.zeros(2, m, dtype=torch.int8, device="cuda")
    cpu = PairBalanceOracle(m, 4, d)
    cpu.begin_epoch()
    raw_equal = 0
    for k, g in enumerate(steps):
        binding.step_noalloc(g, r, signs[k])
        s = signs[k].cpu().numpy()
        assert set(np.unique(s).tolist()) <= {-1, 1}
        cpu.step(synth.to_host(g), replay=s, tau=tau)
        raw_equal += int((cpu.own_signs()[:, k] == s).sum())
    assert cpu.mismatches == 0
    assert raw_equal == 2 * m          # nothing here sits inside the tie band
    want = cpu.r()
    err = np.linalg.norm(r.cpu().numpy().astype(np.float64) - want) / np.linalg.norm(want)
    assert err <= rtol, err
    assert binding.noalloc_status() == binding.OK
    cpu.close()


def test_non_finite_input_is_reported_and_cleared():
    m, d = 4, 8192
    g = _grads(m, d, torch.float32, 3)
    r = torch.zeros(d, dtype=torch.float32, device="cuda")
    s = torch.zeros(m, dtype=torch.int8, device="cuda")
    binding.step_noalloc(g, r, s)                        # r != 0 from here on
    assert binding.noalloc_status() == binding.OK
    g[0, 2, 100] = float("nan")
    binding.step_noalloc(g, r, s)
    assert binding.noalloc_status() == binding.ERR_NONFINITE
    assert binding.noalloc_status() == binding.OK        # reading it clears it


def test_sizes_beyond_the_fixed_scratch_are_rejected():
    m, d = 17, 4096
    g = torch.zeros(2, m, d, device="cuda")
    r = torch.zeros(d, device="cuda")
    s = torch.zeros(m, dtype=torch.int8, device="cuda")
    with pytest.raises(binding.CdgrabError) as e:
        binding.step_noalloc(g, r, s)
    assert e.value.code == binding.ERR_TOO_LARGE
    assert "fixed scratch" in str(e.value)
    with pytest.raises(binding.CdgrabError) as e:
        binding.step_noalloc(torch.zeros(2, 4, 1002, device="cuda"), torch.zeros(1002, device="cuda"), s)
    assert e.value.code == binding.ERR_INVALID   # d must be a multiple of 4
