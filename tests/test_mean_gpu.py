"""cdgrab_step_mean: the balancing step that also returns the parameter-server average of the two
gather buffers (Algorithm 4).  The average is checked against its definition in fp64, and the
step itself must be unchanged by asking for it."""
import numpy as np
import pytest
import torch

from paper_2302_00845_b200 import binding

pytestmark = pytest.mark.gpu


def grads(m, d, dtype, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    t = torch.randn(2, m, d, generator=g, device="cuda") + 0.5
    return t.to(torch.float32 if dtype == "f32" else torch.bfloat16)


@pytest.mark.parametrize("m,d,dtype,path", [
    (4, 1024, "f32", "literal"),      # single-launch steps: separate averaging kernel
    (8, 4096, "f32", "fused"),
    (16, 100_000, "f32", "fma"),      # TMA-fed Gram, pass 2 with 256-bit loads
    (5, 1023, "f32", "fma"),          # scalar pass 2
    (12, 70_004, "bf16", "fma"),      # 8-column pass 2 (rows not 32-byte aligned)
    (32, 9_008, "bf16", "umma"),      # 16-column pass 2 that also writes the split copy of r
])
def test_mean_matches_definition_and_step_is_unchanged(m, d, dtype, path):
    n = 6
    steps = [grads(m, d, dtype, 31 * m + k) for k in range(n // 2)]
    mean = torch.empty(2, d, dtype=torch.float32, device="cuda")
    with binding.CdGrab(m, n, d, dtype) as a, binding.CdGrab(m, n, d, dtype) as b:
        assert a.path == path
        a.begin_epoch(); b.begin_epoch()
        for g in steps:
            mean.fill_(float("nan"))
            a.step_mean(g, mean)
            b.step(g)
            torch.cuda.synchronize()
            want = g.double().mean(dim=1)                      # [2][d], the definition in fp64
            err = (mean.double() - want).abs().max().item()
            assert err <= 2e-6 * max(1.0, want.abs().max().item()), err
        assert torch.equal(a.signs(), b.signs())
        assert torch.equal(a.r(), b.r())
        assert a.status() == binding.OK


def test_mean_argument_errors():
    with binding.CdGrab(2, 4, 64, "f32") as h:
        h.begin_epoch()
        rc = binding.lib().cdgrab_step_mean(h._h, grads(2, 64, "f32", 1).data_ptr(), None, None)
        assert rc == binding.ERR_INVALID


def test_misaligned_destination_is_refused_on_the_host():
    """The averages are written with 16-byte vector stores; a destination off that boundary is an
    argument error, not a device fault."""
    m, n, d = 4, 4, 4096
    with binding.CdGrab(m, n, d, "f32") as h:
        h.begin_epoch()
        g = torch.zeros(2, m, d, device="cuda")
        out = torch.zeros(2 * d + 4, device="cuda")[1:1 + 2 * d]
        with pytest.raises(binding.CdgrabError) as e:
            h.step_mean(g, out)
        assert e.value.code == binding.ERR_INVALID
        assert h.launch_count == 0
        h.step_mean(g, torch.zeros(2, d, device="cuda"))
