"""cdgrab_step_logreg: the logistic-regression step formed straight from the feature rows.  The
oracle gets the gradients from the fp64 formula (rounded to the fp32 the library would store);
the two-launch route (gradient kernel, then step) must give the same signs."""
import numpy as np
import pytest
import torch

import oracle
from oracle import PairBalanceOracle
from paper_2302_00845_b200 import binding, synth
from parity import TAU, R_TOL, rel_l2

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("m,n,d,epochs", [(8, 64, 1024, 2), (4, 16, 2048, 1), (16, 8, 512, 1), (8, 32, 4096, 1)])
def test_fused_logreg_step_matches_oracle_and_two_launch_route(m, n, d, epochs):
    wl = synth.WORKLOADS["logreg"].scaled(m=m, n=n, d=d)
    prob = synth.LogregProblem(wl, device="cuda")
    Xh, yh, wh = prob.X.cpu().numpy(), prob.y.cpu().numpy(), prob.w.cpu().numpy()
    fused = binding.CdGrab(m, n, d, "f32")
    two = binding.CdGrab(m, n, d, "f32")
    cpu = PairBalanceOracle(m, n, d)
    grads = torch.empty(2, m, d, device="cuda")
    try:
        assert fused.path in ("fused", "literal")   # short rows take the literal form for cdgrab_step
        for _ in range(epochs):
            cur = cpu.perm_cur()
            fused.begin_epoch(); two.begin_epoch(); cpu.begin_epoch()
            for k in range(n // 2):
                fused.step_logreg(prob.X, prob.y, prob.w)
                two.logreg_grads(prob.X, prob.y, prob.w, grads)
                two.step(grads)
                s = fused.signs()[:, k].cpu().numpy()
                g = np.empty((2, m, d), dtype=np.float32)
                for i in range(m):
                    for q in (0, 1):
                        item = cur[i, 2 * k + q]
                        g[q, i] = oracle.logistic_grad(Xh[i, item], yh[i, item], wh).astype(np.float32)
                cpu.step(g, replay=s, tau=TAU["f32"])
            assert cpu.mismatches == 0
            assert torch.equal(fused.signs(), two.signs())
            err = rel_l2(fused.r().cpu().numpy().astype(np.float64), cpu.r())
            assert err <= R_TOL["f32"], err
            assert rel_l2(fused.r().cpu().numpy().astype(np.float64), two.r().cpu().numpy().astype(np.float64)) < 1e-5
            out = torch.empty(m, n, dtype=torch.int32, device="cuda")
            fused.end_epoch(out); two.end_epoch()
            torch.cuda.synchronize()
            assert np.array_equal(out.cpu().numpy(), cpu.end_epoch())
        assert fused.status() == binding.OK
        assert fused.launch_count == epochs * (n // 2)      # one launch per step
    finally:
        fused.destroy(); two.destroy(); cpu.close()


def test_fused_logreg_needs_the_single_launch_path():
    with binding.CdGrab(8, 4, 200_000, "f32") as h:        # too large for one CTA
        h.begin_epoch()
        X = torch.zeros(8, 4, 200_000, device="cuda"); y = torch.zeros(8, 4, device="cuda")
        w = torch.zeros(200_000, device="cuda")
        with pytest.raises(binding.CdgrabError) as e:
            h.step_logreg(X, y, w)
        assert e.value.code == binding.ERR_INVALID
