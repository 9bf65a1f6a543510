"""cdgrab_step_randomized against the CPU oracle: the randomized balance rule (Algorithm 2's
subroutine with the bound w of Algorithm 5), the uniform draws handed in by the caller.  Signs
must match wherever the draw is not within the tolerance band of the probability; the oracle
adopts the GPU's sign inside the band."""
import numpy as np
import pytest
import torch

from oracle import PairBalanceOracle
from paper_2302_00845_b200 import binding, synth
from parity import TAU, R_TOL, rel_l2

pytestmark = pytest.mark.gpu


def grads(m, d, dtype, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    t = torch.randn(2, m, d, generator=g, device="cuda")
    return t.to(torch.float32 if dtype == "f32" else torch.bfloat16)


@pytest.mark.parametrize("m,d,dtype,path", [
    (4, 4096, "f32", "fused"),
    (4, 1024, "f32", "literal"),      # Algorithm 6 worker by worker in one CTA
    (40, 128, "bf16", "literal"),
    (40, 64, "bf16", "fused"),        # many workers, short rows: the Gram form in one CTA
    (8, 16_384, "bf16", "fused"),
    (16, 100_000, "f32", "fma"),      # decisions taken in the tail of the TMA-fed Gram kernel
    (5, 3_001, "f32", "fma"),         # generic tiles + stand-alone scan
    (32, 20_000, "bf16", "umma"),
])
def test_randomized_rule_matches_oracle(m, d, dtype, path):
    n = 8
    w = 0.05 * d            # |<r,c>| straddles the bound: both regimes are exercised
    gpu = binding.CdGrab(m, n, d, dtype)
    cpu = PairBalanceOracle(m, n, d)
    gen = torch.Generator(device="cuda").manual_seed(99 + m)
    try:
        assert gpu.path == path
        gpu.begin_epoch(); cpu.begin_epoch()
        plus = 0
        for k in range(n // 2):
            g = grads(m, d, dtype, 17 * m + k)
            u = torch.rand(m, generator=gen, device="cuda")
            gpu.step_randomized(g, u, w)
            s = gpu.signs()[:, k].cpu().numpy()
            cpu.step_randomized(synth.to_host(g), u.cpu().numpy().astype(np.float64), w, replay=s,
                                tau=TAU[dtype])
            plus += int((s == 1).sum())
        assert cpu.mismatches == 0
        assert np.array_equal(gpu.signs().cpu().numpy(), cpu.signs())
        assert 0 < plus < m * n // 2                     # not degenerate
        assert gpu.out_of_bound == cpu.out_of_bound
        err = rel_l2(gpu.r().cpu().numpy().astype(np.float64), cpu.r())
        assert err <= R_TOL[dtype], err
        out = torch.empty(m, n, dtype=torch.int32, device="cuda")
        gpu.end_epoch(out)
        torch.cuda.synchronize()
        assert np.array_equal(out.cpu().numpy(), cpu.end_epoch())
        assert gpu.status() == binding.OK
        print(f"randomized m={m} d={d} {dtype} {path}: plus={plus}/{m * n // 2} out_of_bound={cpu.out_of_bound} "
              f"near_ties={cpu.near_ties} r_err={err:.2e}")
    finally:
        gpu.destroy(); cpu.close()


def test_randomized_then_greedy_steps_mix_and_arguments():
    m, n, d = 4, 4, 4096
    with binding.CdGrab(m, n, d, "f32") as a, binding.CdGrab(m, n, d, "f32") as b:
        a.begin_epoch(); b.begin_epoch()
        g0, g1 = grads(m, d, "f32", 1), grads(m, d, "f32", 2)
        u = torch.full((m,), 0.25, device="cuda")
        with pytest.raises(binding.CdgrabError) as e:
            a.step_randomized(g0, u, 0.0)
        assert e.value.code == binding.ERR_INVALID
        # with an enormous bound every p is 1/2: u = 0.25 gives +1 everywhere
        a.step_randomized(g0, u, 1e30)
        assert torch.all(a.signs()[:, 0] == 1)
        # the rule is per call: the next plain step is greedy again
        a.step(g1)
        b.step_randomized(g0, u, 1e30); b.step(g1)
        assert torch.equal(a.signs(), b.signs()) and torch.equal(a.r(), b.r())
        assert a.out_of_bound == 0


def test_seeded_draws_equal_the_oracles_generator_bit_for_bit():
    """Both sides implement Philox4x32-10 from its published definition: the device's draws for a
    grid of (seed, epoch, k) equal the oracle's, as floats, exactly."""
    import oracle
    for seed, epoch, k, m in [(0, 0, 0, 7), (987654321012345678, 5, 31, 200), (2**64 - 1, 2**32 - 1, 2**31, 33)]:
        got = binding.randomized_uniforms(seed, epoch, k, m).cpu().numpy()
        want = np.array([oracle.uniform(seed, epoch, k, i) for i in range(m)], dtype=np.float32)
        assert np.array_equal(got, want)


@pytest.mark.parametrize("m,d,dtype", [(4, 1024, "f32"), (8, 4096, "f32"), (16, 100_000, "f32"), (32, 20_000, "bf16"),
                                       (24, 8_192, "f32")])
def test_seeded_randomized_epoch_matches_oracle_and_repeats(m, d, dtype):
    """A randomized epoch from (seed, epoch) alone: the oracle draws the same uniforms with its own
    generator; the same seed gives the same signs again, another seed does not."""
    import oracle
    n, w, seed, epoch = 8, 0.05 * d, 20260101, 3
    runs = []
    for sd in (seed, seed, seed + 1):
        gpu = binding.CdGrab(m, n, d, dtype)
        cpu = PairBalanceOracle(m, n, d)
        try:
            gpu.begin_epoch(); cpu.begin_epoch()
            for k in range(n // 2):
                g = grads(m, d, dtype, 23 * m + k)
                gpu.step_randomized_seeded(g, sd, epoch, w)
                s = gpu.signs()[:, k].cpu().numpy()
                u = np.array([oracle.uniform(sd, epoch, k, i) for i in range(m)])
                cpu.step_randomized(synth.to_host(g), u, w, replay=s, tau=TAU[dtype])
            assert cpu.mismatches == 0
            assert gpu.status() == binding.OK
            runs.append(gpu.signs().cpu().numpy().copy())
        finally:
            gpu.destroy(); cpu.close()
    assert np.array_equal(runs[0], runs[1])
    assert not np.array_equal(runs[0], runs[2])
