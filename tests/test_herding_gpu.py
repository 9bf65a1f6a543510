"""Device evaluator of the parallel herding objective (Eq. 7) against the CPU oracle, and the
quality check it exists for: PairBalance orders from the CUDA library shrink the bound on the
paper's synthetic recipe (uniform vectors, centred, normalised)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2302_00845_b200 import binding, synth
from parity import Pair
from test_oracle_pins import load_herding_cases

pytestmark = pytest.mark.gpu


def device_objective(z, perms):
    zt = torch.as_tensor(np.ascontiguousarray(z, dtype=np.float32)).cuda()
    pt = torch.as_tensor(np.ascontiguousarray(perms, dtype=np.int32)).cuda()
    return binding.herding_objective(zt, pt)


def test_hand_computed_cases_on_device():
    for name, z, perms, want in load_herding_cases():
        assert device_objective(z, perms) == want, name


@pytest.mark.parametrize("m,n,d", [(1, 1, 1), (3, 17, 5), (5, 1000, 16), (2, 64, 3000), (7, 333, 33),
                                   (4, 40, 70_000)])
def test_random_shapes_match_oracle(m, n, d):
    rng = np.random.default_rng(m * 1000 + n + d)
    z = (rng.random((m, n, d)) + 0.25).astype(np.float32)      # a mean far from zero
    perms = np.stack([rng.permutation(n) for _ in range(m)]).astype(np.int32)
    want = oracle.herding_objective(z, perms)
    got = device_objective(z, perms)
    assert abs(got - want) <= 1e-9 * max(1.0, want), (got, want)


def test_argument_errors():
    L = binding.lib()
    assert L.cdgrab_herding_workspace_bytes(0, 4, 4) == -1
    z = torch.zeros(2, 4, 4, device="cuda"); p = torch.zeros(2, 4, dtype=torch.int32, device="cuda")
    out = torch.zeros(1, dtype=torch.float64, device="cuda")
    ws = torch.zeros(4, dtype=torch.float64, device="cuda")
    rc = L.cdgrab_herding_objective(z.data_ptr(), p.data_ptr(), 2, 4, 4, ws.data_ptr(), 32, out.data_ptr(), None)
    assert rc == binding.ERR_INVALID      # workspace too small


def test_pairbalance_orders_shrink_the_bound():
    """Lemma 1 in practice: a few epochs of coordinated PairBalance bring the bound far below
    that of the random initial orders; device and oracle agree on the value."""
    m, n, d = 5, 2000, 16
    g = torch.Generator(device="cuda").manual_seed(4)
    z = torch.rand(m * n, d, generator=g, device="cuda")
    z = z - z.mean(dim=0)
    z = (z / z.norm(dim=1, keepdim=True)).reshape(m, n, d).contiguous()
    rng = np.random.default_rng(4)
    perms = np.stack([rng.permutation(n) for _ in range(m)]).astype(np.int32)
    start = binding.herding_objective(z, torch.as_tensor(perms).cuda())
    rows = torch.arange(m, device="cuda")
    with binding.CdGrab(m, n, d, "f32") as h:
        h.set_perms(perms)
        cur = torch.as_tensor(perms).cuda()
        out = torch.empty(m, n, dtype=torch.int32, device="cuda")
        history = [start]
        for _ in range(4):
            h.begin_epoch()
            curl = cur.long()
            for k in range(n // 2):
                grads = torch.stack([z[rows, curl[:, 2 * k]], z[rows, curl[:, 2 * k + 1]]]).contiguous()
                h.step(grads)
            h.end_epoch(out)
            torch.cuda.synchronize()
            cur = out.clone()
            history.append(binding.herding_objective(z, cur))
        assert h.status() == binding.OK
    print("herding bound per epoch:", [round(v, 3) for v in history])
    assert history[-1] < 0.25 * start
    want = oracle.herding_objective(z.cpu().numpy(), cur.cpu().numpy())
    assert abs(history[-1] - want) <= 1e-9 * max(1.0, want)


def _staged_epoch(z, cur):
    m, n, d = z.shape
    rows = torch.arange(m, device="cuda")[:, None]
    return z[rows, cur.long()].reshape(m, n // 2, 2, d).permute(1, 2, 0, 3).contiguous()


@pytest.mark.parametrize("m", [5, 10, 20, 50, 100])
def test_herding_study_reduced_beats_random_reshuffling(m):
    """The synthetic study at reduced size (20 000 vectors in R^16): after four epochs the bound of
    the library's coordinated orders is below that of every random-reshuffling order drawn."""
    n, d = (20_000 // m) & ~1, 16
    z = synth.herding_vectors(m * n, d, 7, "cuda").reshape(m, n, d)
    cur = synth.random_orders(m, n, 70, "cuda")
    rr = [binding.herding_objective(z, synth.random_orders(m, n, 71 + e, "cuda")) for e in range(4)]
    out = torch.empty(m, n, dtype=torch.int32, device="cuda")
    hist = [binding.herding_objective(z, cur)]
    with binding.CdGrab(m, n, d, "f32") as h:
        h.set_perms(cur.cpu().numpy())
        for _ in range(4):
            h.begin_epoch()
            h.step_many(_staged_epoch(z, cur))
            h.end_epoch(out)
            torch.cuda.synchronize()
            cur = out.clone()
            hist.append(binding.herding_objective(z, cur))
        assert h.status() == binding.OK
    print(f"m={m}: PairBalance {[round(v, 2) for v in hist]}  random reshuffling {[round(v, 2) for v in rr]}")
    assert hist[-1] < min(rr)
    assert hist[-1] < 0.5 * hist[0]


def test_herding_study_largest_worker_count_against_the_oracle():
    """m = 100 workers, short rows: signs, permutations and Eq. (7) of one epoch against the oracle."""
    m, n, d = 100, 60, 16
    z = synth.herding_vectors(m * n, d, 3, "cuda").reshape(m, n, d)
    cur = synth.random_orders(m, n, 30, "cuda")
    g = _staged_epoch(z, cur)
    pr = Pair(m, n, d, "f32", perms0=cur.cpu().numpy())
    try:
        pr.begin()
        for k in range(n // 2):
            pr.step(g[k])
        rep = pr.end()
        assert rep.raw_agreement == 1.0
        got = pr.gpu.perms()
        want = oracle.herding_objective(z.cpu().numpy(), got.cpu().numpy())
        dev = binding.herding_objective(z, got)
        assert abs(dev - want) <= 1e-9 * max(1.0, want)
    finally:
        pr.close()
