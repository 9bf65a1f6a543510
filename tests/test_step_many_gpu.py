"""cdgrab_step_many: several steps per call.  Bit-identical to the same steps taken one by one,
and the oracle's decisions, on the single-launch path (where the steps share one kernel launch)
and on a two-pass path (where the call loops)."""
import time

import numpy as np
import pytest
import torch

from oracle import PairBalanceOracle
from paper_2302_00845_b200 import binding, synth
from parity import TAU, R_TOL, rel_l2

pytestmark = pytest.mark.gpu


def epoch(m, n, d, dtype, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    t = torch.randn(n // 2, 2, m, d, generator=g, device="cuda") + 0.1
    return t.to(torch.float32 if dtype == "f32" else torch.bfloat16).contiguous()


@pytest.mark.parametrize("m,n,d,dtype,path", [
    (4, 64, 1024, "f32", "literal"),     # the tiny workload: a whole epoch in one launch
    (8, 16, 4096, "f32", "fused"),
    (16, 8, 2048, "bf16", "fused"),
    (3, 10, 516, "f32", "literal"),
    (6, 10, 1028, "f32", "fused"),
    (40, 6, 128, "bf16", "literal"),
    (40, 6, 64, "bf16", "fused"),        # many workers, short rows: the Gram form in one CTA
    (8, 6, 200_000, "f32", "fma"),       # two-pass path, TMA-fed pass 1: the call loops over single steps, or
    (16, 8, 1 << 18, "f32", "fma"),      # (CDGRAB_DEFER=1) the update of a step rides in the next step's pass 1
    (16, 8, 300_008, "bf16", "fma"),
    (4, 6, 70_000, "f32", "fma"),
    (3, 12, 65_540, "bf16", "fma"),
    (8, 6, 40_000, "f32", "fma"),        # short rows: register-load pass 1, the call loops over single steps
])
@pytest.mark.parametrize("defer", ["0", "1"])
def test_many_equals_single_steps_and_oracle(m, n, d, dtype, path, defer, monkeypatch):
    if defer == "1" and (path != "fma" or d < 65536):
        pytest.skip("the deferred update exists on the TMA-fed two-pass path only")
    monkeypatch.setenv("CDGRAB_DEFER", defer)
    g = epoch(m, n, d, dtype, 5 + m)
    with binding.CdGrab(m, n, d, dtype) as a, binding.CdGrab(m, n, d, dtype) as b:
        assert a.path == path
        a.begin_epoch(); b.begin_epoch()
        split = n // 2 // 3                       # two calls with different counts
        if split:
            a.step_many(g[:split])
        a.step_many(g[split:])
        for k in range(n // 2):
            b.step(g[k])
        assert torch.equal(a.signs(), b.signs())
        assert torch.equal(a.r(), b.r())
        assert torch.equal(a.margins(), b.margins())
        assert torch.equal(a.next_perms(), b.next_perms())
        cpu = PairBalanceOracle(m, n, d)
        try:
            cpu.begin_epoch()
            s = a.signs().cpu().numpy()
            for k in range(n // 2):
                cpu.step(synth.to_host(g[k]), replay=s[:, k], tau=TAU[dtype])
            assert cpu.mismatches == 0
            assert rel_l2(a.r().cpu().numpy().astype(np.float64), cpu.r()) <= R_TOL[dtype]
            out = torch.empty(m, n, dtype=torch.int32, device="cuda")
            a.end_epoch(out)
            torch.cuda.synchronize()
            assert np.array_equal(out.cpu().numpy(), cpu.end_epoch())
        finally:
            cpu.close()
        assert a.status() == binding.OK


def test_deferred_update_launch_count_and_switch(monkeypatch):
    """With CDGRAB_DEFER=1, count steps in one call take count + 1 streaming launches on the TMA-fed
    path; by default the call loops over single steps (2 launches each).  Same bits either way."""
    m, n, d = 8, 12, 131_072
    g = epoch(m, n, d, "f32", 77)
    out = {}
    for defer in ("1", "0"):
        monkeypatch.setenv("CDGRAB_DEFER", defer)
        with binding.CdGrab(m, n, d, "f32") as h:
            h.begin_epoch()
            before = h.launch_count
            h.step_many(g)
            out[defer] = (h.launch_count - before, h.signs().clone(), h.r().clone(), h.next_perms().clone())
            assert h.status() == binding.OK
    assert out["1"][0] == n // 2 + 1 and out["0"][0] == 2 * (n // 2)
    for a, b in zip(out["1"][1:], out["0"][1:]):
        assert torch.equal(a, b)


def test_many_rejects_more_steps_than_the_epoch_has():
    m, n, d = 4, 8, 1024
    g = epoch(m, n, d, "f32", 1)
    with binding.CdGrab(m, n, d, "f32") as h:
        h.begin_epoch()
        h.step(g[0])
        with pytest.raises(binding.CdgrabError) as e:
            h.step_many(g)                       # 4 steps asked, 3 left: nothing is done
        assert e.value.code == binding.ERR_STATE
        h.step_many(g[1:])
        out = torch.empty(m, n, dtype=torch.int32, device="cuda")
        h.end_epoch(out)


def test_many_timing_tiny_epoch():
    """Prints the time of a tiny epoch taken as 32 calls and as one call (run with -s)."""
    m, n, d = 4, 64, 1024
    g = epoch(m, n, d, "f32", 2)
    with binding.CdGrab(m, n, d, "f32") as h:
        res = {}
        for mode in ("single", "many", "single", "many"):
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
            torch.cuda.synchronize()
            ev[0].record()
            for _ in range(20):
                h.begin_epoch()
                if mode == "many":
                    h.step_many(g)
                else:
                    for k in range(n // 2):
                        h.step(g[k])
                h.end_epoch()
            ev[1].record()
            torch.cuda.synchronize()
            res[mode] = ev[0].elapsed_time(ev[1]) / 20 * 1e3
        print(f"tiny epoch (32 steps, 256 examples): one step per call {res['single']:.0f} us, "
              f"one call {res['many']:.0f} us")
        assert res["many"] < res["single"]
