"""Checkpoint / resume: an epoch interrupted after some steps and continued in a fresh handle from
the saved state gives bit-identical signs, running sum and permutations."""
import pytest
import torch

from paper_2302_00845_b200 import binding

pytestmark = pytest.mark.gpu


def grads(m, d, dtype, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    t = torch.randn(2, m, d, generator=g, device="cuda") + 0.1
    return t.to(torch.float32 if dtype == "f32" else torch.bfloat16)


@pytest.mark.parametrize("m,d,dtype,independent", [(4, 2048, "f32", False), (16, 150_000, "f32", False),
                                                    (32, 40_000, "bf16", False), (6, 30_000, "bf16", True),
                                                    (24, 40_000, "f32", False), (48, 6_000, "f32", False)])
def test_resume_is_bit_identical(m, d, dtype, independent):
    n = 8
    steps = [grads(m, d, dtype, 50 + k) for k in range(n)]          # two epochs of n/2 steps
    def finish(h, first, count):
        for k in range(first, first + count):
            h.step(steps[k])
    with binding.CdGrab(m, n, d, dtype, independent=independent) as ref:
        ref.begin_epoch(); finish(ref, 0, n // 2); ref.end_epoch()
        ref.begin_epoch(); finish(ref, n // 2, n // 2)
        want = (ref.signs().cpu(), ref.r().cpu(), ref.next_perms().cpu(), ref.perms().cpu(), ref.margins().cpu())
    with binding.CdGrab(m, n, d, dtype, independent=independent) as a:
        a.begin_epoch(); finish(a, 0, n // 2); a.end_epoch()
        a.begin_epoch(); finish(a, n // 2, 1)                       # stop inside the second epoch
        saved = a.save_state()
    with binding.CdGrab(m, n, d, dtype, independent=independent) as b:
        b.load_state(saved)
        finish(b, n // 2 + 1, n // 2 - 1)
        got = (b.signs().cpu(), b.r().cpu(), b.next_perms().cpu(), b.perms().cpu(), b.margins().cpu())
        assert b.status() == binding.OK
        b.end_epoch()
    for x, y in zip(want, got):
        assert torch.equal(x, y)


def test_state_of_another_shape_is_refused():
    with binding.CdGrab(4, 4, 1024, "f32") as a, binding.CdGrab(4, 4, 2048, "f32") as b:
        saved = a.save_state()
        with pytest.raises(binding.CdgrabError) as e:
            b.load_state(saved)
        assert e.value.code == binding.ERR_INVALID
