"""Pins for the CPU oracle: it is checked against what the paper and the mathematics fix,
never against itself or the CUDA path.  All tests here run without a GPU."""
import itertools
import os
import subprocess
import sys

import numpy as np
import pytest

import oracle
from oracle import PairBalanceOracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def run_epoch(z, perms=None, replay=None, tau=0.0):
    """z: [m][n][d] float32 indexed by ITEM id; visits follow the current permutation."""
    m, n, d = z.shape
    o = PairBalanceOracle(m, n, d)
    if perms is not None:
        o.set_perms(perms)
    cur = o.perm_cur()
    o.begin_epoch()
    for k in range(n // 2):
        g = np.empty((2, m, d), dtype=np.float32)
        for i in range(m):
            g[0, i] = z[i, cur[i, 2 * k]]
            g[1, i] = z[i, cur[i, 2 * k + 1]]
        o.step(g, None if replay is None else replay[:, k], tau)
    return o


# --------------------------------------------------------------------------------------
# Worked example derived by hand from Algorithms 6, 2, 7 and 1 (see the fixture's header).
# --------------------------------------------------------------------------------------
def load_golden(path):
    z1, z2, signs, perm, meta, r_final = {}, {}, {}, {}, {}, None
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        tok = line.split()
        if tok[0] in ("m", "n", "d"):
            meta[tok[0]] = int(tok[1])
        elif tok[0] in ("z1", "z2"):
            (z1 if tok[0] == "z1" else z2)[(int(tok[1]), int(tok[2]))] = [float(v) for v in tok[3:]]
        elif tok[0] == "signs":
            signs[int(tok[1])] = [int(v) for v in tok[2:]]
        elif tok[0] == "perm":
            perm[int(tok[1])] = [int(v) for v in tok[2:]]
        elif tok[0] == "r_final":
            r_final = [float(v) for v in tok[1:]]
    return meta, z1, z2, signs, perm, r_final


def test_hand_derived_onehot_example():
    meta, z1, z2, signs, perm, r_final = load_golden(os.path.join(GOLDEN, "onehot_m2_n8_d3.txt"))
    m, n, d = meta["m"], meta["n"], meta["d"]
    o = PairBalanceOracle(m, n, d)
    o.begin_epoch()
    for k in range(n // 2):
        g = np.zeros((2, m, d), dtype=np.float32)
        for i in range(m):
            g[0, i] = z1[(k, i)]
            g[1, i] = z2[(k, i)]
        o.step(g)
    got = o.signs()
    for i in range(m):
        assert got[i].tolist() == signs[i]
    assert o.r().tolist() == r_final
    p = o.end_epoch()
    for i in range(m):
        assert p[i].tolist() == perm[i]


def test_onehot_visit_rule_random_sequences():
    """Axis-aligned differences c = sigma*e_a: a coordinate's running value is 0 at odd
    visits (tie, so -1 and r[a] <- -sigma) and returns to 0 after even visits, where the
    sign is +1 exactly if sigma repeats the previous visit's sigma (Algorithm 6 by hand)."""
    rng = np.random.default_rng(5)
    m, n, d = 3, 40, 4
    o = PairBalanceOracle(m, n, d)
    o.begin_epoch()
    visits = {a: [] for a in range(d)}
    expect = np.zeros((m, n // 2), dtype=np.int8)
    for k in range(n // 2):
        g = np.zeros((2, m, d), dtype=np.float32)
        for i in range(m):
            a = int(rng.integers(d)); sigma = float(rng.choice([-1.0, 1.0]))
            # put the vector in the first or the second slot of the pair at random
            if rng.random() < 0.5:
                g[0, i, a] = sigma
            else:
                g[1, i, a] = -sigma
            hist = visits[a]
            if len(hist) % 2 == 0:
                expect[i, k] = -1
            else:
                expect[i, k] = +1 if hist[-1] == sigma else -1
            hist.append(sigma)
        o.step(g)
    assert np.array_equal(o.signs(), expect)
    r = o.r()
    for a in range(d):
        hist = visits[a]
        assert r[a] == (0.0 if len(hist) % 2 == 0 else -hist[-1])


# --------------------------------------------------------------------------------------
# Brute force on tiny inputs: each greedy choice is the argmin of the two candidate norms.
# --------------------------------------------------------------------------------------
@pytest.mark.parametrize("m,d", list(itertools.product([1, 2, 3, 4], [1, 2])))
def test_bruteforce_argmin_small_integers(m, d):
    rng = np.random.default_rng(100 * m + d)
    n = 12
    z = rng.integers(-3, 4, size=(m, n, d)).astype(np.float32)
    o = PairBalanceOracle(m, n, d)
    o.begin_epoch()
    r = np.zeros(d)
    n_ties = 0
    for k in range(n // 2):
        for i in range(m):
            c = z[i, 2 * k].astype(np.float64) - z[i, 2 * k + 1]
            plus = float(np.sum((r + c) ** 2))     # integers: exact in fp64
            minus = float(np.sum((r - c) ** 2))
            want = +1 if plus < minus else -1      # strict '<': ties give -1
            n_ties += plus == minus
            got = o.balance_one(i, z[i, 2 * k], z[i, 2 * k + 1])
            assert got == want, (k, i, r, c)
            r = r + want * c
            assert np.array_equal(o.r(), r)
    assert n_ties > 0  # the tie branch was exercised


def test_first_decision_of_every_epoch_is_minus_one():
    rng = np.random.default_rng(1)
    z = rng.standard_normal((3, 6, 17)).astype(np.float32)
    o = run_epoch(z)
    assert o.signs()[0, 0] == -1
    p = o.end_epoch()
    o.begin_epoch()
    assert np.all(o.r() == 0.0)  # Algorithm 4: the running sum restarts at zero
    g = np.stack([z[np.arange(3), p[:, 0]], z[np.arange(3), p[:, 1]]])
    o.step(g)
    assert o.signs()[0, 0] == -1


def test_zero_difference_is_a_tie():
    z = np.ones((1, 4, 5), dtype=np.float32)
    o = run_epoch(z)
    assert o.signs().tolist() == [[-1, -1]]
    assert np.all(o.r() == 0.0)


# --------------------------------------------------------------------------------------
# Invariants of the greedy rule.
# --------------------------------------------------------------------------------------
def test_norm_invariant_and_dot_vs_norm_form():
    rng = np.random.default_rng(2)
    m, n, d = 4, 32, 257
    z = (rng.standard_normal((m, n, d)) + 0.3).astype(np.float32)
    o = PairBalanceOracle(m, n, d)
    o.begin_epoch()
    r = np.zeros(d)
    for k in range(n // 2):
        for i in range(m):
            c = z[i, 2 * k].astype(np.float64) - z[i, 2 * k + 1].astype(np.float64)
            before = float(r @ r)
            s = o.balance_one(i, z[i, 2 * k], z[i, 2 * k + 1])
            # the printed norm form
            np_, nm = np.linalg.norm(r + c), np.linalg.norm(r - c)
            if abs(np_ - nm) > 1e-9 * (np_ + nm):
                assert s == (+1 if np_ < nm else -1)
            r = r + s * c
            # greedy never does worse than an orthogonal step
            assert float(r @ r) <= before + float(c @ c) + 1e-9 * (before + 1)
            np.testing.assert_allclose(o.r(), r, rtol=0, atol=1e-12)


def test_r_final_is_signed_sum_of_differences():
    rng = np.random.default_rng(3)
    m, n, d = 5, 20, 4100  # spans two summation chunks with a ragged tail
    z = rng.standard_normal((m, n, d)).astype(np.float32)
    o = run_epoch(z)
    S = o.signs()
    diff = z[:, 0::2].astype(np.float64) - z[:, 1::2].astype(np.float64)  # [m][n/2][d]
    want = np.einsum("ik,ikx->x", S.astype(np.float64), diff)
    np.testing.assert_allclose(o.r(), want, rtol=0, atol=1e-10)


def test_gram_form_identity():
    """t_i = b_i + sum_{k<i} s_k G_ki and ||r_m||^2 = ||r_0||^2 + 2 s.b + s.G.s inside a step
    (what the two-pass formulation relies on), checked on the oracle's recorded trace."""
    rng = np.random.default_rng(4)
    m, n, d = 6, 8, 300
    z = rng.standard_normal((m, n, d)).astype(np.float32)
    o = PairBalanceOracle(m, n, d)
    o.begin_epoch()
    for k in range(n // 2):
        r0 = o.r()
        g = np.stack([z[:, 2 * k], z[:, 2 * k + 1]])
        o.step(g)
        Cm = g[0].astype(np.float64) - g[1].astype(np.float64)   # [m][d]
        G, b = Cm @ Cm.T, Cm @ r0
        s = o.signs()[:, k].astype(np.float64)
        t = o.trace()[0][:, k]
        for i in range(m):
            ti = b[i] + np.dot(s[:i], G[:i, i])
            assert abs(ti - t[i]) <= 1e-11 * (np.linalg.norm(Cm[i]) * (np.linalg.norm(r0) + np.linalg.norm(Cm) ) + 1)
        r1 = o.r()
        np.testing.assert_allclose(r1 @ r1, r0 @ r0 + 2 * s @ b + s @ G @ s, rtol=1e-11)


# --------------------------------------------------------------------------------------
# m = 1 is centralized PairBalance; coordination couples workers.
# --------------------------------------------------------------------------------------
def centralized_pairbalance(z):
    """Centralized online PairBalance written separately (Appendix A.4): one worker,
    consecutive pairs, greedy sign on the difference, then the reorder of Algorithm 1."""
    n, d = z.shape
    r = np.zeros(d)
    pos, neg = [], []
    for j in range(0, n, 2):
        c = z[j].astype(np.float64) - z[j + 1].astype(np.float64)
        s = 1 if np.linalg.norm(r + c) ** 2 < np.linalg.norm(r - c) ** 2 else -1
        r += s * c
        (pos if s == 1 else neg).append(j)
        (neg if s == 1 else pos).append(j + 1)
    return pos + neg[::-1], r


def test_m1_equals_centralized():
    rng = np.random.default_rng(6)
    z = rng.standard_normal((1, 50, 33)).astype(np.float32)
    o = run_epoch(z)
    want_perm, want_r = centralized_pairbalance(z[0])
    np.testing.assert_allclose(o.r(), want_r, atol=1e-12)
    assert o.end_epoch()[0].tolist() == want_perm


def test_coordination_couples_workers():
    rng = np.random.default_rng(7)
    m, n, d = 3, 16, 40
    z = rng.standard_normal((m, n, d)).astype(np.float32)
    coord = run_epoch(z).signs()
    indep = np.stack([run_epoch(z[i:i + 1]).signs()[0] for i in range(m)])
    # worker 0's first decision sees r = 0 in both; later ones see the shared running sum
    assert not np.array_equal(coord, indep)
    # independent instances do not react to another worker's data, the coordinated one does
    z2 = z.copy(); z2[0] = rng.standard_normal((n, d)).astype(np.float32)
    assert np.array_equal(run_epoch(z2[1:2]).signs()[0], indep[1])
    assert not np.array_equal(run_epoch(z2).signs()[1:], coord[1:])
    # order of the workers inside a pair index matters (worker-minor interleaving)
    swapped = run_epoch(z[[1, 0, 2]]).signs()
    assert not np.array_equal(swapped[[1, 0, 2]], coord)


# --------------------------------------------------------------------------------------
# Reorder: Algorithm 1 written with lists, driven through arbitrary sign patterns.
# --------------------------------------------------------------------------------------
def reorder_lists(perm, pair_signs):
    pos, neg = [], []
    for k, s in enumerate(pair_signs):
        item_signs = (s, -s)  # Algorithm 2: s for z1, -s for z2
        for off in (0, 1):
            (pos if item_signs[off] == 1 else neg).append(int(perm[2 * k + off]))
    return pos + neg[::-1]


@pytest.mark.parametrize("pattern", ["plus", "minus", "random"])
def test_reorder_matches_list_formulation(pattern):
    rng = np.random.default_rng(8)
    m, n, d = 3, 14, 6
    z = rng.standard_normal((m, n, d)).astype(np.float32)
    perms = np.stack([rng.permutation(n) for _ in range(m)]).astype(np.int32)
    if pattern == "plus":
        S = np.ones((m, n // 2), dtype=np.int8)
    elif pattern == "minus":
        S = -np.ones((m, n // 2), dtype=np.int8)
    else:
        S = rng.choice([-1, 1], size=(m, n // 2)).astype(np.int8)
    # a tie band that covers everything makes the oracle adopt the handed-in signs
    o = run_epoch(z, perms=perms, replay=S, tau=1e30)
    assert np.array_equal(o.signs(), S)
    assert o.near_ties == m * (n // 2)
    out = o.end_epoch()
    for i in range(m):
        assert out[i].tolist() == reorder_lists(perms[i], S[i])
    if pattern == "plus":
        assert out[0].tolist() == perms[0][0::2].tolist() + perms[0][1::2][::-1].tolist()
    if pattern == "minus":
        assert out[0].tolist() == perms[0][1::2].tolist() + perms[0][0::2][::-1].tolist()


def test_permutation_structure():
    rng = np.random.default_rng(9)
    m, n, d = 4, 30, 19
    z = rng.standard_normal((m, n, d)).astype(np.float32)
    perms = np.stack([rng.permutation(n) for _ in range(m)]).astype(np.int32)
    o = run_epoch(z, perms=perms)
    out = o.end_epoch()
    for i in range(m):
        assert sorted(out[i].tolist()) == list(range(n))
        for k in range(n // 2):
            assert {int(out[i, k]), int(out[i, n - 1 - k])} == {int(perms[i, 2 * k]), int(perms[i, 2 * k + 1])}
    assert np.array_equal(o.perm_cur(), out)  # the new order is the next epoch's current order


def test_replay_band_counts_and_mismatch():
    rng = np.random.default_rng(10)
    m, n, d = 2, 10, 64
    z = rng.standard_normal((m, n, d)).astype(np.float32)
    own = run_epoch(z).signs()
    o = run_epoch(z, replay=own, tau=1e-6)
    assert o.mismatches == 0 and np.array_equal(o.signs(), own)
    assert o.near_ties >= 1  # the very first decision has r = 0
    flipped = own.copy(); flipped[1, 3] *= -1
    o2 = run_epoch(z, replay=flipped, tau=1e-6)
    assert o2.mismatches >= 1
    assert o2.signs()[1, 3] == own[1, 3]  # outside the band the oracle keeps its own sign


# --------------------------------------------------------------------------------------
# bf16 inputs are widened exactly; state machine; thread-count independence.
# --------------------------------------------------------------------------------------
def test_bf16_widening_is_exact():
    rng = np.random.default_rng(11)
    m, n, d = 2, 6, 100
    bits = (rng.standard_normal((m, n, d)).astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
    as_f32 = (bits.astype(np.uint32) << 16).view(np.float32)
    a = PairBalanceOracle(m, n, d); a.begin_epoch()
    b = PairBalanceOracle(m, n, d); b.begin_epoch()
    for k in range(n // 2):
        a.step(np.stack([bits[:, 2 * k], bits[:, 2 * k + 1]]))
        b.step(np.stack([as_f32[:, 2 * k], as_f32[:, 2 * k + 1]]))
    assert np.array_equal(a.signs(), b.signs())
    assert np.array_equal(a.r(), b.r())


def test_state_machine_errors():
    with pytest.raises(ValueError):
        PairBalanceOracle(2, 5, 3)  # odd n is rejected
    o = PairBalanceOracle(1, 2, 3)
    g = np.zeros((2, 1, 3), dtype=np.float32)
    with pytest.raises(RuntimeError):
        o.step(g)  # no epoch open
    o.begin_epoch()
    with pytest.raises(RuntimeError):
        o.end_epoch()  # early
    o.step(g)
    with pytest.raises(RuntimeError):
        o.step(g)  # past n/2
    o.end_epoch()


def test_result_independent_of_thread_count():
    code = (
        "import numpy as np, sys; sys.path.insert(0, %r); import oracle;"
        "rng=np.random.default_rng(0); z=rng.standard_normal((2,8,20000)).astype(np.float32);"
        "o=oracle.PairBalanceOracle(2,8,20000); o.begin_epoch();\n"
        "for k in range(4): o.step(np.stack([z[:,2*k],z[:,2*k+1]]))\n"
        "sys.stdout.write(o.r().tobytes().hex()[:4000]+str(o.trace()[0].tobytes().hex()))"
    ) % os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    outs = []
    for nt in ("1", "3"):
        env = dict(os.environ, OMP_NUM_THREADS=nt)
        outs.append(subprocess.check_output([sys.executable, "-c", code], env=env))
    assert outs[0] == outs[1]


# --------------------------------------------------------------------------------------
# Soft quality check: Lemma 1 says each application roughly halves the herding bound.
# --------------------------------------------------------------------------------------
def test_herding_objective_drops_over_epochs():
    # the paper's synthetic recipe in small: Unif(0,1)^16, centred, L2-normalised
    rng = np.random.default_rng(12)
    m, n, d = 5, 200, 16
    z = rng.random((m * n, d))
    z -= z.mean(axis=0)
    z /= np.linalg.norm(z, axis=1, keepdims=True)
    z = z.reshape(m, n, d).astype(np.float32)
    perms = np.stack([rng.permutation(n) for _ in range(m)]).astype(np.int32)
    start = oracle.herding_objective(z, perms)
    o = PairBalanceOracle(m, n, d)
    o.set_perms(perms)
    cur = perms
    for _ in range(5):
        o.begin_epoch()
        for k in range(n // 2):
            g = np.stack([z[np.arange(m), cur[:, 2 * k]], z[np.arange(m), cur[:, 2 * k + 1]]])
            o.step(g)
        cur = o.end_epoch()
    assert oracle.herding_objective(z, cur) < 0.5 * start


# --------------------------------------------------------------------------------------
# Logistic-regression gradient: pinned by finite differences of the loss.
# --------------------------------------------------------------------------------------
def test_logistic_gradient_matches_finite_differences():
    rng = np.random.default_rng(13)
    d = 7
    x = rng.standard_normal(d); w = rng.standard_normal(d) * 0.3
    for y in (0.0, 1.0):
        loss = lambda w_: np.log1p(np.exp(w_ @ x)) - y * (w_ @ x)
        g = oracle.logistic_grad(x, y, w)
        for a in range(d):
            e = np.zeros(d); e[a] = 1e-6
            fd = (loss(w + e) - loss(w - e)) / 2e-6
            assert abs(fd - g[a]) < 1e-8


# --------------------------------------------------------------------------------------
# Parallel herding objective, Eq. (7): hand-computed examples and invariants.
# --------------------------------------------------------------------------------------
def load_herding_cases():
    out = []
    for line in open(os.path.join(GOLDEN, "herding_objective_examples.txt")):
        if not line.startswith("case"):
            continue
        head, zs, ps, want = [t.strip() for t in line.split("|")]
        _, name, m, n, d = head.split()
        m, n, d = int(m), int(n), int(d)
        z = np.array([float(v) for v in zs.split()]).reshape(m, n, d)
        perms = np.array([int(v) for v in ps.split()]).reshape(m, n)
        out.append((name, z, perms, float(want)))
    return out


def test_herding_objective_hand_examples():
    cases = load_herding_cases()
    assert len(cases) == 7
    for name, z, perms, want in cases:
        assert oracle.herding_objective(z, perms) == want, name


def test_herding_objective_invariants():
    rng = np.random.default_rng(21)
    m, n, d = 3, 17, 5
    z = rng.standard_normal((m, n, d))
    perms = np.stack([rng.permutation(n) for _ in range(m)])
    base = oracle.herding_objective(z, perms)
    # cumulative-sum formulation with a library routine
    zbar = z.reshape(-1, d).mean(axis=0)
    steps = sum(z[i, perms[i]] for i in range(m)) - m * zbar            # [n][d]
    assert abs(np.abs(np.cumsum(steps, axis=0)).max() - base) < 1e-12
    # the centred vectors sum to zero, so walking every order backwards gives the same bound
    assert abs(oracle.herding_objective(z, perms[:, ::-1]) - base) < 1e-12
    # relabelling the workers changes nothing; a constant shift of all vectors changes nothing
    assert abs(oracle.herding_objective(z[::-1], perms[::-1]) - base) < 1e-12
    assert abs(oracle.herding_objective(z + 3.5, perms) - base) < 1e-10
    # scaling scales the bound
    assert abs(oracle.herding_objective(2 * z, perms) - 2 * base) < 1e-12
    # identical vectors: nothing to balance
    assert oracle.herding_objective(np.ones((2, 4, 3)), np.tile(np.arange(4), (2, 1))) == 0.0


# --------------------------------------------------------------------------------------
# RandomizedBalance (Algorithm 2's subroutine with the bound w of Algorithm 5).
# --------------------------------------------------------------------------------------
def _rand_state(seed, d=40):
    """An oracle whose running sum is r = z0 - z1 of a first (greedy) pair, plus a second pair."""
    rng = np.random.default_rng(seed)
    z = rng.standard_normal((1, 4, d)).astype(np.float32)
    o = PairBalanceOracle(1, 4, d)
    o.begin_epoch()
    s0 = o.balance_one(0, z[0, 0], z[0, 1])
    r = s0 * (z[0, 0].astype(np.float64) - z[0, 1])
    c = z[0, 2].astype(np.float64) - z[0, 3]
    return o, z, r, c


def test_randomized_probability_formula_and_update():
    for seed in range(6):
        o, z, r, c = _rand_state(seed)
        t = float(r @ c)
        w = 3.0 * abs(t) + 1.0
        p = 0.5 - t / (2 * w)                       # Algorithm 5 / Algorithm 2 with w made explicit
        assert 0 < p < 1 and (p > 0.5) == (t < 0)   # leaning towards the greedy sign
        for u, want in ((max(p - 1e-3, 0.0), +1), (min(p + 1e-3, 1 - 1e-12), -1)):
            o2, z2, _, _ = _rand_state(seed)
            s = o2.balance_one_randomized(0, z2[0, 2], z2[0, 3], u, w)
            assert s == want
            np.testing.assert_allclose(o2.r(), r + want * c, atol=1e-12)
            assert o2.out_of_bound == 0


def test_randomized_limits():
    o, z, r, c = _rand_state(11)
    t = float(r @ c)
    # a huge bound makes it a fair coin
    for u, want in ((0.49999, +1), (0.50001, -1)):
        o2, z2, _, _ = _rand_state(11)
        assert o2.balance_one_randomized(0, z2[0, 2], z2[0, 3], u, 1e18) == want
    # |<r,c>| beyond the bound: the draw no longer matters, the greedy sign comes out, counted
    for u in (0.0, 0.3, 0.999999):
        o2, z2, _, _ = _rand_state(11)
        s = o2.balance_one_randomized(0, z2[0, 2], z2[0, 3], u, abs(t) * 0.5)
        assert s == (+1 if t < 0 else -1) and o2.out_of_bound == 1
    with pytest.raises(RuntimeError):
        o.balance_one_randomized(0, z[0, 2], z[0, 3], 0.5, 0.0)


def test_randomized_expected_sign_is_minus_t_over_w():
    o, z, r, c = _rand_state(3)
    t = float(r @ c)
    w = 2.0 * abs(t)
    us = (np.arange(4000) + 0.5) / 4000            # an even grid of draws
    total = 0
    for u in us:
        o2, z2, _, _ = _rand_state(3)
        total += o2.balance_one_randomized(0, z2[0, 2], z2[0, 3], float(u), w)
    assert abs(total / len(us) - (-t / w)) < 2e-3  # E[s] = 2p - 1 = -<r,c>/w


def test_randomized_replay_band():
    o, z, r, c = _rand_state(5)
    t = float(r @ c); w = 4 * abs(t) + 1; p = 0.5 - t / (2 * w)
    rn, cn = np.linalg.norm(r), np.linalg.norm(c)
    tau = 1e-3
    band = tau * rn * cn / (2 * w)
    o2, z2, _, _ = _rand_state(5)
    s = o2.balance_one_randomized(0, z2[0, 2], z2[0, 3], p + 0.5 * band, w, replay=+1, tau=tau)
    assert s == +1 and o2.near_ties == 1 and o2.mismatches == 0      # inside the band: adopted
    o3, z3, _, _ = _rand_state(5)
    s = o3.balance_one_randomized(0, z3[0, 2], z3[0, 3], p + 2.0 * band, w, replay=+1, tau=tau)
    assert s == -1 and o3.mismatches == 1                              # outside: own sign kept


# ---- the seeded draws of RandomizedBalance: Philox4x32-10 -----------------------------------------
def test_philox_known_answer_vectors():
    """The generator's published known-answer vectors (tests/golden/philox4x32_10_kat.txt)."""
    rows = [l for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for line in rows:
        ctr, key, want = [[int(w, 16) for w in part.split()] for part in line.split("|")]
        assert oracle.philox4x32_10(ctr, key).tolist() == want


def test_philox_reduced_rounds_would_not_pass_and_words_are_not_swapped():
    """A dropped round, swapped multipliers or a swapped key word all change the first vector."""
    M0, M1, W0, W1 = 0xD2511F53, 0xCD9E8D57, 0x9E3779B9, 0xBB67AE85

    def ref(ctr, key, rounds=10, m0=M0, m1=M1):
        c, k = list(ctr), list(key)
        for _ in range(rounds):
            p0, p1 = m0 * c[0], m1 * c[2]
            c = [(p1 >> 32) ^ c[1] ^ k[0], p1 & 0xFFFFFFFF, (p0 >> 32) ^ c[3] ^ k[1], p0 & 0xFFFFFFFF]
            k = [(k[0] + W0) & 0xFFFFFFFF, (k[1] + W1) & 0xFFFFFFFF]
        return c
    ctr, key = [1, 2, 3, 4], [5, 6]
    good = oracle.philox4x32_10(ctr, key).tolist()
    assert good == ref(ctr, key)
    assert good != ref(ctr, key, rounds=9) and good != ref(ctr, key, m0=M1, m1=M0) and good != ref(ctr, [6, 5])


def test_seeded_uniform_is_a_24_bit_fraction_of_the_first_word():
    for seed, epoch, k, i in [(0, 0, 0, 0), (12345678901234567, 3, 17, 99), (2**64 - 1, 2**32 - 1, 7, 1023)]:
        x0 = int(oracle.philox4x32_10([i, k, epoch, 0], [seed & 0xFFFFFFFF, seed >> 32])[0])
        u = oracle.uniform(seed, epoch, k, i)
        assert u == (x0 >> 8) / 2.0**24 and 0.0 <= u < 1.0


def test_seeded_uniforms_look_uniform():
    u = np.array([oracle.uniform(42, 1, k, i) for k in range(200) for i in range(100)])
    assert abs(u.mean() - 0.5) < 0.01 and abs(u.var() - 1 / 12) < 0.005
    hist, _ = np.histogram(u, bins=10, range=(0, 1))
    assert hist.min() > 1800 and hist.max() < 2200
    assert len(np.unique(u)) > 19_900                       # distinct counters give distinct draws
