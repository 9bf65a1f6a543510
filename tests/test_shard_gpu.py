"""Column-sharded order server on one GPU: the shards are handles over column slices, the
all-reduce of the m*m + m partial sums is a plain tensor sum.  Every shard must take the oracle's
decisions, the concatenated slices of r must be the oracle's r, and all shards must produce the
same permutations."""
import numpy as np
import pytest
import torch

from oracle import PairBalanceOracle
from paper_2302_00845_b200 import binding, synth
from parity import TAU, R_TOL, rel_l2

pytestmark = pytest.mark.gpu


def grads(m, d, dtype, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    t = torch.randn(2, m, d, generator=g, device="cuda") + 0.1
    return t.to(torch.float32 if dtype == "f32" else torch.bfloat16)


@pytest.mark.parametrize("m,d,dtype,cuts", [
    (8, 200_000, "f32", [0, 100_000, 200_000]),          # TMA-fed FMA Gram, decisions deferred
    (32, 80_000, "bf16", [0, 40_000, 80_000]),           # tensor-core Gram
    (4, 4_096, "f32", [0, 2_048, 4_096]),                # small: register Gram, never the one-launch path
    (16, 300_000, "f32", [0, 70_000, 200_000, 300_000]), # three uneven shards
    (5, 3_003, "f32", [0, 1_001, 3_003]),                # generic tiles
    (24, 80_000, "f32", [0, 40_000, 80_000]),            # fp32 on the tensor cores (three bf16 terms)
    (48, 10_000, "f32", [0, 6_000, 10_000]),             # blocked FMA Gram
    (80, 6_000, "bf16", [0, 2_000, 6_000]),              # scan with G staged above the default 48 KB of shared memory
])
def test_sharded_steps_match_oracle(m, d, dtype, cuts):
    n = 6
    shards = [binding.CdGrab(m, n, hi - lo, dtype, shard=True) for lo, hi in zip(cuts[:-1], cuts[1:])]
    cpu = PairBalanceOracle(m, n, d)
    parts = [torch.empty(m * m + m, dtype=torch.float64, device="cuda") for _ in shards]
    try:
        for h in shards:
            h.begin_epoch()
        cpu.begin_epoch()
        for k in range(n // 2):
            g = grads(m, d, dtype, 60 + k)
            slices = [g[:, :, lo:hi].contiguous() for lo, hi in zip(cuts[:-1], cuts[1:])]
            for h, gs, p in zip(shards, slices, parts):
                h.step_begin(gs, p)
            total = parts[0].clone()
            for p in parts[1:]:
                total += p                                   # what the all-reduce would deliver
            for h, gs in zip(shards, slices):
                h.step_finish(gs, total)
            s = shards[0].signs()[:, k].cpu().numpy()
            cpu.step(synth.to_host(g), replay=s, tau=TAU[dtype])
        assert cpu.mismatches == 0
        want_signs = cpu.signs()
        for h in shards:
            assert np.array_equal(h.signs().cpu().numpy(), want_signs)     # identical on every shard
            assert h.status() == binding.OK
        r = torch.cat([h.r() for h in shards]).cpu().numpy().astype(np.float64)
        err = rel_l2(r, cpu.r())
        assert err <= R_TOL[dtype], err
        want_perm = cpu.end_epoch()
        for h in shards:
            out = torch.empty(m, n, dtype=torch.int32, device="cuda")
            h.end_epoch(out)
            torch.cuda.synchronize()
            assert np.array_equal(out.cpu().numpy(), want_perm)
    finally:
        for h in shards:
            h.destroy()
        cpu.close()


def test_shard_state_machine():
    m, n, d = 4, 4, 2048
    with binding.CdGrab(m, n, d, "f32", shard=True) as h:
        g = grads(m, d, "f32", 1)
        p = torch.zeros(m * m + m, dtype=torch.float64, device="cuda")
        h.begin_epoch()
        with pytest.raises(binding.CdgrabError) as e:
            h.step(g)                              # a shard does not step on its own
        assert e.value.code == binding.ERR_INVALID
        with pytest.raises(binding.CdgrabError) as e:
            h.step_finish(g, p)                    # nothing begun
        assert e.value.code == binding.ERR_STATE
        h.step_begin(g, p)
        with pytest.raises(binding.CdgrabError) as e:
            h.step_begin(g, p)                     # finish first
        assert e.value.code == binding.ERR_STATE
        h.step_finish(g, p)
        # pointers the kernels would touch with vector accesses are refused on the host
        h.step_begin(g, p)
        odd = torch.zeros(2 * m * d + 4, device="cuda")[1:1 + 2 * m * d].view(2, m, d)
        pp = torch.zeros(2 * (m * m + m) + 2, dtype=torch.float32, device="cuda")[1:1 + 2 * (m * m + m)]
        L = binding.lib()
        st = torch.cuda.current_stream().cuda_stream
        assert L.cdgrab_step_finish(h._h, odd.data_ptr(), p.data_ptr(), st) == binding.ERR_INVALID
        assert L.cdgrab_step_finish(h._h, g.data_ptr(), pp.data_ptr(), st) == binding.ERR_INVALID
        h.step_finish(g, p)                        # still pending after the refusals
    with binding.CdGrab(m, n, d, "f32") as h:
        h.begin_epoch()
        with pytest.raises(binding.CdgrabError):
            h.step_begin(grads(m, d, "f32", 1), torch.zeros(m * m + m, dtype=torch.float64, device="cuda"))


def test_single_rank_wrapper_equals_plain_handle():
    m, n, d = 8, 4, 100_000
    sh = binding.ShardedCdGrab(m, n, d, "f32")
    with binding.CdGrab(m, n, d, "f32") as ref:
        sh.begin_epoch(); ref.begin_epoch()
        for k in range(n // 2):
            g = grads(m, d, "f32", 9 + k)
            sh.step(g); ref.step(g)
        assert torch.equal(sh.h.signs(), ref.signs())
        assert torch.equal(sh.h.r(), ref.r())
    sh.destroy()
