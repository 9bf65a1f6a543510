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
import pytest
import torch

from paper_2302_00845_b200 import binding

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
    before = torch.cuda.memory_allocated()
    for k, g in enumerate(steps):
        binding.step_noalloc(g, r, signs[k])
    torch.cuda.synchronize()
    assert torch.cuda.memory_allocated() == before
    assert torch.equal(signs.t().contiguous(), want_signs)
    # same kernels in the same order: the tests' tolerance for r is 1e-5 relative L2 (fp32 inputs)
    err = (r.double() - want_r.double()).norm() / want_r.double().norm()
    assert float(err) <= 1e-5
    assert torch.equal(r, want_r)


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
