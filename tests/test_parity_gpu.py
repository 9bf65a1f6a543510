"""GPU parity tests: the CUDA library, called through its C ABI, against the CPU oracle on the
same seeded inputs, element by element.  Sizes are chosen so the oracle finishes in seconds
while the kernels still span several tiles/blocks and a ragged tail."""
import os

import numpy as np
import pytest
import torch

from paper_2302_00845_b200 import binding, synth
from parity import Pair, run_stream_epoch, rel_l2, TAU, R_TOL
import oracle

pytestmark = pytest.mark.gpu

# Inside the tie band the acceptance rule takes either sign, and with bf16 inputs most positions
# of a near-isotropic stream sit inside it; so the workload tests also require that the signs
# agree with the oracle's own (un-replayed) decisions nearly everywhere, band or not.
RAW_MIN = 0.999


@pytest.fixture(autouse=True)
def _no_forced_path(monkeypatch):
    monkeypatch.delenv("CDGRAB_FORCE_PATH", raising=False)


def random_grads(m, d, dtype, seed, scale=1.0, mean=0.0):
    g = torch.Generator(device="cuda").manual_seed(seed)
    t = torch.randn(2, m, d, generator=g, device="cuda") * scale + mean
    return t.to(torch.float32 if dtype == "f32" else torch.bfloat16)


def run_random_epoch(m, n, d, dtype, seed=0, perms0=None, mean=0.3):
    pr = Pair(m, n, d, dtype, perms0)
    try:
        pr.begin()
        for k in range(n // 2):
            pr.step(random_grads(m, d, dtype, seed * 1000 + k, mean=mean))
        return pr.end()
    finally:
        pr.close()


# ---- the five workloads, at full or reduced size ------------------------------------------
def test_tiny_workload_full_size():
    rep = run_stream_epoch(synth.WORKLOADS["tiny"])
    print("tiny:", rep)
    assert rep.path == "literal"
    assert rep.raw_agreement >= RAW_MIN, rep


def test_mid_workload_reduced():
    # same recipe and m, d cut to 64Ki + a ragged tail of column groups, 16 steps
    wl = synth.WORKLOADS["mid"].scaled(n=32, d=65536 + 4 * 37)
    rep = run_stream_epoch(wl)
    print("mid(reduced):", rep)
    assert rep.path == "fma"
    assert rep.raw_agreement >= RAW_MIN, rep


def test_lstm_workload_reduced():
    wl = synth.WORKLOADS["lstm"].scaled(n=8, d=135_000 + 8)
    rep = run_stream_epoch(wl)
    print("lstm(reduced):", rep)
    assert rep.path == "umma"
    assert rep.raw_agreement >= RAW_MIN, rep


def test_gpt2_workload_reduced():
    wl = synth.WORKLOADS["gpt2"].scaled(n=6, d=124_000 + 64)
    rep = run_stream_epoch(wl)
    print("gpt2(reduced):", rep)
    assert rep.path == "umma"
    assert rep.raw_agreement >= RAW_MIN, rep


def test_logreg_workload_three_epochs_reduced():
    """Logistic regression: gradients computed on the device from X, y, w in visiting order,
    checked against the fp64 formula, then balanced; the order produced by epoch t is the
    visiting order of epoch t+1."""
    wl = synth.WORKLOADS["logreg"].scaled(n=64, d=1024)
    prob = synth.LogregProblem(wl, device="cuda")
    m, n, d = wl.m, wl.n, wl.d
    pr = Pair(m, n, d, "f32")
    Xh, yh, wh = prob.X.cpu().numpy(), prob.y.cpu().numpy(), prob.w.cpu().numpy()
    grads = torch.empty(2, m, d, device="cuda")
    try:
        for epoch in range(wl.epochs):
            cur = pr.cpu.perm_cur()
            assert np.array_equal(pr.gpu.perms().cpu().numpy(), cur)
            pr.begin()
            for k in range(n // 2):
                pr.gpu.logreg_grads(prob.X, prob.y, prob.w, grads)
                torch.cuda.synchronize()
                gh = grads.cpu().numpy()
                for i in range(m):      # every worker: a wrong row offset anywhere shows here
                    for q in (0, 1):
                        item = cur[i, 2 * k + q]
                        want = oracle.logistic_grad(Xh[i, item], yh[i, item], wh)
                        assert rel_l2(gh[q, i].astype(np.float64), want) < 1e-5
                pr.step(grads)  # balancing parity on the bytes the device produced
            rep = pr.end()
            print(f"logreg epoch {epoch}:", rep)
            assert rep.raw_agreement >= RAW_MIN, rep
    finally:
        pr.close()


# ---- shapes that exercise every kernel variant ---------------------------------------------
@pytest.mark.parametrize("m,n,d,dtype", [
    (1, 8, 4096, "f32"),       # m = 1: centralized PairBalance
    (2, 2, 8, "f32"),          # a single pair per worker
    (3, 6, 1, "f32"),          # d = 1, scalar tail path
    (5, 6, 1023, "f32"),       # d not a multiple of 4 -> generic tiles + scalar update
    (7, 4, 40004, "f32"),      # fused/fma with M = 8
    (16, 4, 30000, "f32"),     # M = 16
    (17, 4, 5000, "f32"),      # three row tiles, last one ragged
    (33, 4, 2048, "f32"),      # five row tiles
    (64, 2, 4096, "f32"),      # fp32 with many workers
    (4, 6, 2052, "bf16"),
    (12, 4, 70000, "bf16"),
    (5, 4, 1001, "bf16"),      # odd d: scalar paths
    (32, 4, 9000, "bf16"),
    (64, 2, 20008, "bf16"),
    (70, 2, 3000, "bf16"),     # more workers than one 128-row tile holds
    (300, 2, 1000, "bf16"),    # scan with G left in global memory
    (1024, 2, 64, "f32"),      # the largest m the library accepts
])
def test_shapes(m, n, d, dtype):
    rep = run_random_epoch(m, n, d, dtype, seed=m * 7 + d % 13)
    print(f"m={m} n={n} d={d} {dtype}:", rep)


@pytest.mark.parametrize("path", ["fused", "fma"])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_forced_paths_agree(path, dtype, monkeypatch):
    monkeypatch.setenv("CDGRAB_FORCE_PATH", path)
    rep = run_random_epoch(8, 6, 16384 + 8, dtype, seed=3)
    assert rep.path == path
    print(path, dtype, rep)


def test_fma_path_many_blocks():
    # 2 MiB rows: the multi-block Gram kernel runs its full grid and loops
    rep = run_random_epoch(16, 4, 600_000, "f32", seed=5)
    assert rep.path == "fma"
    print(rep)


def test_initial_permutations_and_two_epochs():
    rng = np.random.default_rng(0)
    m, n, d = 4, 16, 2048
    perms0 = np.stack([rng.permutation(n) for _ in range(m)]).astype(np.int32)
    z = torch.randn(m, n, d, generator=torch.Generator(device="cuda").manual_seed(1), device="cuda")
    pr = Pair(m, n, d, "f32", perms0)
    try:
        for _ in range(2):
            cur = torch.from_numpy(pr.cpu.perm_cur()).cuda().long()
            pr.begin()
            for k in range(n // 2):
                g = torch.stack([z[torch.arange(m), cur[:, 2 * k]], z[torch.arange(m), cur[:, 2 * k + 1]]])
                pr.step(g.contiguous())
            pr.end()
    finally:
        pr.close()


# ---- degenerate inputs ----------------------------------------------------------------------
def test_all_zero_gradients_are_ties():
    m, n, d = 4, 8, 4096
    with binding.CdGrab(m, n, d, "f32") as h:
        h.begin_epoch()
        g = torch.zeros(2, m, d, device="cuda")
        for _ in range(n // 2):
            h.step(g)
        assert torch.all(h.signs() == -1)
        assert torch.all(h.r() == 0)
        out = torch.empty(m, n, dtype=torch.int32, device="cuda")
        h.end_epoch(out)
        torch.cuda.synchronize()
        # all -1: second member of each pair to the front, first members reversed at the back
        want = list(range(1, n, 2)) + list(range(n - 2, -1, -2))
        assert out[0].tolist() == want
        assert h.status() == binding.OK


def test_first_decision_is_minus_one_and_margin_zero():
    m, n, d = 3, 4, 8192
    with binding.CdGrab(m, n, d, "f32") as h:
        h.begin_epoch()
        h.step(random_grads(m, d, "f32", 11))
        assert int(h.signs()[0, 0]) == -1
        assert float(h.margins()[0, 0]) == 0.0
        assert float(h.margins()[1, 0]) > 0.0


def test_margins_match_oracle_trace():
    m, n, d = 6, 8, 50000
    pr = Pair(m, n, d, "f32")
    try:
        pr.begin()
        for k in range(n // 2):
            pr.step(random_grads(m, d, "f32", 40 + k, mean=0.1))
        t, rn, cn = pr.cpu.trace()
        want = np.where(rn * cn > 0, np.abs(t) / np.maximum(rn * cn, 1e-300), 0.0)
        got = pr.gpu.margins().cpu().numpy()
        np.testing.assert_allclose(got, want, rtol=2e-3, atol=1e-7)
    finally:
        pr.close()


def test_nonfinite_input_raises_status_flag_without_fault():
    m, n, d = 2, 4, 4096
    with binding.CdGrab(m, n, d, "f32") as h:
        h.begin_epoch()
        g = random_grads(m, d, "f32", 2)
        g[0, 1, 17] = float("nan")
        h.step(g)
        assert h.status() == binding.ERR_NONFINITE


def test_deterministic_bitwise():
    outs = []
    for _ in range(2):
        m, n, d = 16, 4, 300_000
        with binding.CdGrab(m, n, d, "f32") as h:
            h.begin_epoch()
            for k in range(n // 2):
                h.step(random_grads(m, d, "f32", 70 + k))
            outs.append((h.signs().cpu(), h.r().cpu(), h.margins().cpu()))
    for a, b in zip(*outs):
        assert torch.equal(a, b)


# ---- state machine and arguments ---------------------------------------------------------------
@pytest.mark.parametrize("m,n,d,dtype", [(4, 6, 1024, "f32"), (8, 4, 4096, "f32"), (16, 4, 300_000, "f32"),
                                       (32, 4, 100_032, "bf16"), (64, 4, 70_000, "bf16"), (5, 4, 1001, "f32")])
def test_chained_launches_change_nothing(m, n, d, dtype, monkeypatch):
    """Launches queued behind their predecessor (the default) and plain stream order give the same bits."""
    outs = []
    for pdl in ("1", "0"):
        monkeypatch.setenv("CDGRAB_PDL", pdl)
        with binding.CdGrab(m, n, d, dtype) as h:
            h.begin_epoch()
            for k in range(n // 2):
                h.step(random_grads(m, d, dtype, 90 + k))
            out = torch.empty(m, n, dtype=torch.int32, device="cuda")
            h.end_epoch(out)
            outs.append((h.signs().cpu(), h.r().cpu(), h.margins().cpu(), out.cpu()))
    for a, b in zip(*outs):
        assert torch.equal(a, b)


def test_state_machine_and_argument_errors():
    m, n, d = 2, 4, 64
    L = binding.lib()
    with binding.CdGrab(m, n, d, "f32") as h:
        g = torch.zeros(2, m, d, device="cuda")
        with pytest.raises(binding.CdgrabError) as e:
            h.step(g)
        assert e.value.code == binding.ERR_STATE  # no epoch open
        h.begin_epoch()
        with pytest.raises(binding.CdgrabError) as e:
            h.begin_epoch()
        assert e.value.code == binding.ERR_STATE
        with pytest.raises(binding.CdgrabError) as e:
            h.end_epoch()
        assert e.value.code == binding.ERR_STATE  # early end
        with pytest.raises(binding.CdgrabError) as e:
            h.step(g.view(-1)[1:1 + 2 * m * d - 4])  # misaligned pointer
        assert e.value.code == binding.ERR_INVALID
        with pytest.raises(binding.CdgrabError) as e:
            h.set_perms(np.zeros((m, n), dtype=np.int32))
        assert e.value.code == binding.ERR_STATE  # epoch open
        h.step(g); h.step(g)
        with pytest.raises(binding.CdgrabError) as e:
            h.step(g)
        assert e.value.code == binding.ERR_STATE  # more than n/2 steps
        h.end_epoch()
        with pytest.raises(binding.CdgrabError) as e:
            h.set_perms(np.zeros((m, n), dtype=np.int32))
        assert e.value.code == binding.ERR_INVALID  # not a permutation
        assert h.launch_count == 2
    import ctypes as C
    hh = C.c_void_p()
    assert L.cdgrab_create(2, 5, 8, 0, C.byref(hh)) == binding.ERR_INVALID


def test_step_host_matches_step():
    m, n, d = 8, 4, 10000
    g = [random_grads(m, d, "f32", 90 + k) for k in range(n // 2)]
    with binding.CdGrab(m, n, d, "f32") as a, binding.CdGrab(m, n, d, "f32") as b:
        a.begin_epoch(); b.begin_epoch()
        staging = torch.empty(2, m, d, device="cuda")
        for k in range(n // 2):
            a.step(g[k])
            host = g[k].cpu().pin_memory()
            b.step_host(host, staging)
            torch.cuda.synchronize()
        assert torch.equal(a.signs(), b.signs())
        assert torch.equal(a.r(), b.r())


@pytest.mark.parametrize("m,d,dtype", [(16, 65536 * 5 + 4 * 33, "f32"), (7, 148 * 256 * 3, "f32"),
                                       (12, 70_000 + 8 * 11, "bf16"), (3, 65536 * 3, "bf16")])
def test_tma_pipelined_fma_gram(m, d, dtype):
    """Long rows with m <= 16: pass 1 runs the TMA-fed FMA kernel (several ring turns per CTA,
    ragged last tile); the same shapes with that kernel switched off must agree."""
    rep = run_random_epoch(m, 6, d, dtype, seed=m + 3)
    assert rep.path == "fma"
    print(f"tma-fma m={m} d={d} {dtype}:", rep)


def test_tma_fma_gram_matches_register_kernel(monkeypatch):
    m, n, d = 16, 4, 1_000_000
    out = []
    for knob in ("1", "0"):
        monkeypatch.setenv("CDGRAB_FMA_TMA", knob)
        with binding.CdGrab(m, n, d, "f32") as h:
            h.begin_epoch()
            for k in range(n // 2):
                h.step(random_grads(m, d, "f32", 900 + k, mean=0.1))
            out.append((h.signs().cpu(), h.r().cpu(), h.margins().cpu()))
            assert h.status() == binding.OK
    assert torch.equal(out[0][0], out[1][0])
    assert torch.equal(out[0][1], out[1][1])
    np.testing.assert_allclose(out[0][2].numpy(), out[1][2].numpy(), rtol=1e-4, atol=1e-7)


@pytest.mark.parametrize("m,d,dtype", [
    (16, 1 << 20, "f32"),            # 27-28 tiles per CTA: six stay in the ring, the rest come back in reverse
    (16, 65_536 + 4 * 33, "f32"),    # fewer tiles than CTAs, ragged last tile
    (9, 148 * 256 * 5, "f32"),       # exactly five tiles per CTA: fewer than the ring holds
    (5, 148 * 256 * 9 + 8, "bf16"),  # bf16 rows, fp32 adds in pass 2
    (16, 3_000_000, "f32"),          # long rows: pass 2 mostly from memory
])
def test_whole_step_launch_matches_two_launches(m, d, dtype, monkeypatch):
    """The TMA-fed FMA path runs pass 2 inside the pass-1 launch (its CTAs meet at a bounded wait
    between the passes); with that switched off pass 2 is the separate update kernel.  Same sums in
    the same order: signs, r, margins and permutations must agree bit for bit, over several steps
    (the arrival counters of the reduction tree carry over from launch to launch)."""
    n = 8
    outs = []
    for whole in ("1", "0"):
        monkeypatch.setenv("CDGRAB_FT_WHOLE", whole)
        with binding.CdGrab(m, n, d, dtype) as h:
            assert h.path == "fma"
            h.begin_epoch()
            l0 = h.launch_count
            for k in range(n // 2):
                h.step(random_grads(m, d, dtype, 5100 + k, mean=0.05))
            assert h.launch_count - l0 == (n // 2) * (1 if whole == "1" else 2)
            out = torch.empty(m, n, dtype=torch.int32, device="cuda")
            h.end_epoch(out)
            assert h.status() == binding.OK
            outs.append((h.signs().cpu(), h.r().cpu(), h.margins().cpu(), out.cpu()))
    for a, b in zip(*outs):
        assert torch.equal(a, b)
    assert float(outs[0][1].abs().max()) > 0


@pytest.mark.parametrize("m,d,dtype", [(16, 100_000, "f32"), (8, 65_536, "bf16"), (32, 50_048, "bf16")])
def test_handles_side_by_side_do_not_disturb_each_other(m, d, dtype):
    """Three handles of the same shape alive at once, stepped in turn on the same inputs: each
    owns its scratch, so all must agree bit for bit (a scratch buffer sized for the wrong grid
    once let one handle write into its neighbour's memory)."""
    n = 6
    hs = [binding.CdGrab(m, n, d, dtype) for _ in range(3)]
    try:
        for h in hs:
            h.begin_epoch()
        for k in range(n // 2):
            g = random_grads(m, d, dtype, 7000 + k, mean=0.2)
            for h in hs:
                h.step(g)
        ref = (hs[0].signs(), hs[0].r(), hs[0].margins())
        assert float(ref[2].max()) > 0
        for h in hs[1:]:
            assert torch.equal(h.signs(), ref[0]) and torch.equal(h.r(), ref[1]) and torch.equal(h.margins(), ref[2])
            assert h.status() == binding.OK
    finally:
        for h in hs:
            h.destroy()


@pytest.mark.parametrize("m,d,dtype", [(4, 2048, "f32"), (16, 200_000, "f32"), (32, 30_016, "bf16")])
def test_work_follows_the_callers_stream(m, d, dtype):
    """An epoch issued on a side stream (inputs produced on that stream too) gives the same result
    as on the default stream: nothing in the library falls back to another stream."""
    n = 6
    def run(stream):
        with torch.cuda.stream(stream):
            with binding.CdGrab(m, n, d, dtype) as h:
                h.begin_epoch(stream)
                for k in range(n // 2):
                    g = random_grads(m, d, dtype, 4200 + k, mean=0.1)
                    g = g * 1.0            # produced by a kernel on this stream just before the step
                    h.step(g, stream)
                out = torch.empty(m, n, dtype=torch.int32, device="cuda")
                h.end_epoch(out, stream)
                stream.synchronize()
                res = (h.signs().cpu(), h.r().cpu(), out.cpu())
                assert h.status() == binding.OK
                return res
    a = run(torch.cuda.default_stream())
    b = run(torch.cuda.Stream())
    for x, y in zip(a, b):
        assert torch.equal(x, y)
