"""ID-GraB (PairBal) mode: every worker balances against its own running sum.  The oracle for it
is m separate single-worker oracles (m = 1 is centralized PairBalance, pinned on the CPU)."""
import numpy as np
import pytest
import torch

from oracle import PairBalanceOracle
from paper_2302_00845_b200 import binding, synth
from parity import TAU, R_TOL, rel_l2

pytestmark = pytest.mark.gpu


def grads(m, d, dtype, seed, mean=0.2):
    g = torch.Generator(device="cuda").manual_seed(seed)
    t = torch.randn(2, m, d, generator=g, device="cuda") + mean
    return t.to(torch.float32 if dtype == "f32" else torch.bfloat16)


@pytest.mark.parametrize("m,n,d,dtype", [(1, 6, 4096, "f32"), (5, 8, 10_003, "f32"), (16, 6, 262_144, "f32"),
                                         (7, 6, 50_000, "bf16"), (64, 4, 9_001, "bf16")])
def test_independent_mode_matches_single_worker_oracles(m, n, d, dtype):
    rng = np.random.default_rng(m)
    perms0 = np.stack([rng.permutation(n) for _ in range(m)]).astype(np.int32)
    gpu = binding.CdGrab(m, n, d, dtype, independent=True)
    cpus = [PairBalanceOracle(1, n, d) for _ in range(m)]
    try:
        assert gpu.path == "independent"
        gpu.set_perms(perms0)
        for i, o in enumerate(cpus):
            o.set_perms(perms0[i:i + 1]); o.begin_epoch()
        gpu.begin_epoch()
        raw = 0
        for k in range(n // 2):
            g = grads(m, d, dtype, 100 * m + k)
            gpu.step(g)
            s = gpu.signs()[:, k].cpu().numpy()
            host = synth.to_host(g)
            for i, o in enumerate(cpus):
                o.balance_one(0, host[0, i], host[1, i], replay=int(s[i]), tau=TAU[dtype])
                raw += int(o.own_signs()[0, k] == s[i])
        assert all(o.mismatches == 0 for o in cpus)
        out = torch.empty(m, n, dtype=torch.int32, device="cuda")
        gpu.end_epoch(out)
        torch.cuda.synchronize()
        got = out.cpu().numpy()
        for i, o in enumerate(cpus):
            assert np.array_equal(gpu.signs()[i].cpu().numpy(), o.signs()[0])
            err = rel_l2(gpu.r_worker(i).cpu().numpy().astype(np.float64), o.r())
            assert err <= R_TOL[dtype], (i, err)
            assert np.array_equal(got[i], o.end_epoch()[0])
        assert torch.equal(gpu.r(), gpu.r_worker(0))
        assert gpu.status() == binding.OK
        print(f"independent m={m} d={d} {dtype}: raw_agree={raw / (m * n // 2):.4f}")
    finally:
        gpu.destroy()
        for o in cpus:
            o.close()


def test_workers_do_not_interact_and_differ_from_coordinated():
    m, n, d = 4, 8, 20_000
    steps = [grads(m, d, "f32", 300 + k) for k in range(n // 2)]
    def run(independent, alter=False):
        with binding.CdGrab(m, n, d, "f32", independent=independent) as h:
            h.begin_epoch()
            for g in steps:
                if alter:
                    g = g.clone(); g[:, 0] = -3.0 * g[:, 0]       # another worker 0
                h.step(g)
            return h.signs().cpu()
    ind, ind_alt, coord = run(True), run(True, alter=True), run(False)
    assert torch.equal(ind[1:], ind_alt[1:])          # workers 1.. never see worker 0
    assert not torch.equal(ind, coord)                # the coordinated order shares one running sum
    assert torch.all(ind[:, 0] == -1)                 # every worker's first decision sees r_i = 0


def test_unsupported_calls_in_independent_mode():
    with binding.CdGrab(2, 4, 64, "f32", independent=True) as h:
        h.begin_epoch()
        g = grads(2, 64, "f32", 1)
        with pytest.raises(binding.CdgrabError) as e:
            h.step_randomized(g, torch.rand(2, device="cuda"), 1.0)
        assert e.value.code == binding.ERR_INVALID
    with binding.CdGrab(2, 4, 64, "f32") as h:
        with pytest.raises(binding.CdgrabError):
            h.r_worker(0)                             # only for independent-mode handles
