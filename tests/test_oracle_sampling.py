"""Pins for the oracle's noise, post-processing and Modified Rejection Sampling.

Each test checks the oracle against something other than itself: published known-answer
vectors, closed forms of the paper's propositions, library softmax / top-k, or exact counting
over the whole 2^24 noise range (the decision functions are monotone in the noise value, so
interval lengths are found by bisection)."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
N24 = 1 << 24


# --------------------------------------------------------------------------------- noise
def test_philox_known_answers():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt"))
            if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        h = [int(x, 16) for x in r]
        out = oracle.philox4x32_10(h[4:6], h[0:4])
        assert [int(x) for x in out] == h[6:]


def test_noise_key_layout_and_uniformity():
    # word 0 >> 8 of Philox(key=seed, ctr=(sub, position, iteration, stream | batch<<8))
    seed = 0x1234567890ABCDEF
    u = oracle.noise_u24(seed, 2, 5, 77, 9, 3)
    ref = oracle.philox4x32_10([seed & 0xFFFFFFFF, seed >> 32], [3, 77, 9, 2 | (5 << 8)])
    assert u == int(ref[0]) >> 8
    # every key component changes the draw
    base = oracle.noise_u24(1, 1, 0, 10, 0)
    assert len({base, oracle.noise_u24(2, 1, 0, 10, 0), oracle.noise_u24(1, 2, 0, 10, 0),
                oracle.noise_u24(1, 1, 1, 10, 0), oracle.noise_u24(1, 1, 0, 11, 0),
                oracle.noise_u24(1, 1, 0, 10, 1)}) == 6
    # chi-square uniformity over 64 bins, 64k draws
    draws = np.array([oracle.noise_u24(7, 1, 0, p, 0) for p in range(65536)])
    hist = np.bincount(draws >> 18, minlength=64)
    chi2 = ((hist - 1024.0) ** 2 / 1024.0).sum()
    assert chi2 < 63 + 5 * math.sqrt(2 * 63)


# --------------------------------------------------------------------------------- scd_exp
def test_scd_exp_against_libm():
    xs = np.concatenate([np.linspace(-21.9, 0, 20001), -np.logspace(-8, 1.3, 2000)])
    worst = 0.0
    for x in xs.astype(np.float32):
        got, want = oracle.scd_exp(float(x)), math.exp(float(x))
        worst = max(worst, abs(got - want) / want)
    assert worst < 4e-7
    assert oracle.scd_exp(0.0) == 1.0
    assert oracle.scd_exp(-22.5) == 0.0 and oracle.scd_exp(-1e30) == 0.0
    # monotone on a fine grid (weights must not reorder logits)
    grid = np.linspace(-21.9, 0, 50001).astype(np.float32)
    vals = [oracle.scd_exp(float(x)) for x in grid]
    assert all(b >= a for a, b in zip(vals, vals[1:]))


# --------------------------------------------------------------------------------- post-processing
def test_postprocess_matches_library_softmax_topk():
    rng = np.random.default_rng(0)
    for V, k, T in [(1024, 64, 1.0), (1000, 37, 0.7), (513, 0, 1.3), (64, 64, 1.0), (50, 1, 1.0)]:
        logits = (rng.standard_normal(V) * 3).astype(np.float32)
        W, Z, x = oracle.postprocess(logits, temperature=T, top_k=k, want_x=True)
        t = torch.from_numpy(logits).double() / T
        if 0 < k < V:
            kth = torch.topk(t, k).values[-1]
            t = torch.where(t >= kth, t, torch.full_like(t, -float("inf")))
        ref = torch.softmax(t, dim=0).numpy()
        got = W.astype(np.float64) / Z
        assert np.abs(got - ref).max() < 2e-6
        assert ((W > 0) == (ref > 1e-9)).all() or k == 0
        if 0 < k < V:
            assert (W > 0).sum() == k            # no ties in continuous data
        assert int(W.astype(np.uint64).sum()) == Z
        assert W.max() == 1 << 30               # the max logit gets weight exactly 2^30


def test_postprocess_topk_keeps_ties_and_allowed_range():
    logits = np.array([1.0, 3.0, 3.0, 2.0, 3.0, 0.5, 9.0, 9.0], dtype=np.float32)
    # allowed ids 0..5 only; top-2 threshold is 3.0 and all three 3.0's stay
    W, Z = oracle.postprocess(logits, lo=0, hi=6, top_k=2)
    assert list(W > 0) == [False, True, True, False, True, False, False, False]
    assert W[1] == W[2] == W[4] == 1 << 30 and Z == 3 << 30
    # fewer allowed ids than k: keep all allowed
    W, Z = oracle.postprocess(logits, lo=2, hi=4, top_k=5)
    assert list(W > 0) == [False, False, True, True, False, False, False, False]
    # one-hot allowed range (forced token)
    W, Z = oracle.postprocess(logits, lo=5, hi=6, top_k=2)
    assert W[5] == 1 << 30 and Z == 1 << 30 and W.sum() == 1 << 30


def test_postprocess_cfg_mix_and_order():
    # Sec. 5.1: mixed logit (1+lambda) c - lambda u on raw logits, then temperature, then top-k
    rng = np.random.default_rng(1)
    V, lam, T, k = 300, 3.0, 0.8, 40
    c = rng.standard_normal(V).astype(np.float32) * 2
    u = rng.standard_normal(V).astype(np.float32) * 2
    W, Z, x = oracle.postprocess(c, u, temperature=T, top_k=k, cfg_lambda=lam, want_x=True)
    mix = ((1 + lam) * c.astype(np.float64) - lam * u.astype(np.float64)) / T
    assert np.abs(x - mix).max() < 1e-5
    kth = np.sort(mix)[-k]
    ref = np.where(mix >= kth, np.exp(mix - mix.max()), 0.0)
    ref /= ref.sum()
    assert np.abs(W / Z - ref).max() < 2e-6
    # lambda = 0 ignores u
    W0, Z0 = oracle.postprocess(c, None, temperature=T, top_k=k)
    W1, Z1 = oracle.postprocess(c, u, temperature=T, top_k=k, cfg_lambda=0.0)
    assert (W0 == W1).all() and Z0 == Z1


# --------------------------------------------------------------------------------- MRS, Algorithm 1
def _weights(p):
    """Hand-built distribution -> integer weights with an arbitrary (non power-of-two) total."""
    W = np.array(p, dtype=np.uint32)
    return W, int(W.sum())


def _count_accept(Wp, Zp, Wq, Zq, X):
    """#{U in [0,2^24) : MRS accepts}. Acceptance is monotone decreasing in U."""
    if oracle.mrs(Wp, Zp, Wq, Zq, X, 0, 0)[0] == 0:
        return 0
    lo, hi = 0, N24          # accept at lo, reject at hi (virtual)
    while hi - lo > 1:
        mid = (lo + hi) // 2
        if oracle.mrs(Wp, Zp, Wq, Zq, X, mid, 0)[0]:
            lo = mid
        else:
            hi = mid
    return lo + 1


def _residual_counts(Wp, Zp, Wq, Zq, X):
    """For a rejected draw, #{U_res : Y = y} for each y (Y is monotone in U_res)."""
    V = len(Wp)
    counts = np.zeros(V, dtype=np.int64)
    U_rej = N24 - 1
    assert oracle.mrs(Wp, Zp, Wq, Zq, X, U_rej, 0)[0] == 0
    start = 0
    while start < N24:
        y = oracle.mrs(Wp, Zp, Wq, Zq, X, U_rej, start)[1]
        lo, hi = start, N24
        while hi - lo > 1:
            mid = (lo + hi) // 2
            if oracle.mrs(Wp, Zp, Wq, Zq, X, U_rej, mid)[1] == y:
                lo = mid
            else:
                hi = mid
        counts[y] += hi - start
        start = hi
    return counts


CASES = [
    ([5, 1, 3, 7, 0, 2, 9, 4], [1, 6, 3, 2, 8, 0, 5, 6]),
    ([10, 20, 30, 40], [40, 30, 20, 10]),
    ([1, 1, 1, 1, 1], [3, 0, 2, 0, 5]),
    ([700, 1, 1, 1], [1, 1, 1, 700]),
]


@pytest.mark.parametrize("p,q", CASES)
def test_mrs_accept_rule_residual_and_marginal(p, q):
    Wp, Zp = _weights(p)
    Wq, Zq = _weights(q)
    V = len(p)
    P = [Fraction(int(a), Zp) for a in p]
    Q = [Fraction(int(a), Zq) for a in q]
    tvd = sum(abs(a - b) for a, b in zip(P, Q)) / 2
    res_den = sum(max(Fraction(0), a - b) for a, b in zip(P, Q))
    assert res_den == tvd                                     # normaliser of the residual = D_TV
    assert abs(oracle.tv(Wp, Zp, Wq, Zq) - float(tvd)) < 1e-12

    acc_total = Fraction(0)
    marg = [Fraction(0)] * V
    joint_same = Fraction(0)
    for X in range(V):
        if q[X] == 0:
            continue
        n_acc = _count_accept(Wp, Zp, Wq, Zq, X)
        alpha = min(Fraction(1), P[X] / Q[X])                 # the accept probability of Algorithm 1
        assert abs(Fraction(n_acc, N24) - alpha) <= Fraction(1, N24)
        acc_total += Q[X] * Fraction(n_acc, N24)
        marg[X] += Q[X] * Fraction(n_acc, N24)
        joint_same += Q[X] * Fraction(n_acc, N24)
        if n_acc < N24:
            counts = _residual_counts(Wp, Zp, Wq, Zq, X)
            for y in range(V):
                r = max(Fraction(0), P[y] - Q[y]) / res_den   # the residual distribution of Algorithm 1
                assert abs(Fraction(int(counts[y]), N24) - r) <= Fraction(2, N24)
                if r == 0:
                    assert counts[y] == 0
                marg[y] += Q[X] * (1 - Fraction(n_acc, N24)) * Fraction(int(counts[y]), N24)
    # Prop. 2.1: acceptance rate = 1 - D_TV and the output follows p
    assert abs(acc_total - (1 - tvd)) <= Fraction(V, N24)
    for y in range(V):
        assert abs(marg[y] - P[y]) <= Fraction(3 * V, N24)
    # maximal coupling theorem: Pr[X = Y] = 1 - D_TV (a rejected draw never returns X itself
    # because the residual vanishes wherever q >= p, and rejection needs q(X) > p(X))
    assert abs(joint_same - (1 - tvd)) <= Fraction(V, N24)


def test_mrs_special_cases():
    Wp, Zp = _weights([3, 5, 7, 11])
    # p == q (even with different integer scale): always accept
    Wq, Zq = _weights([6, 10, 14, 22])
    for X in range(4):
        for U in (0, 1, N24 // 2, N24 - 1):
            assert oracle.mrs(Wp, Zp, Wq, Zq, X, U, 0) == (1, X)
    # disjoint supports: always reject and Y ~ p
    Wp, Zp = _weights([1, 3, 0, 0])
    Wq, Zq = _weights([0, 0, 5, 5])
    for U in (0, N24 - 1):
        assert oracle.mrs(Wp, Zp, Wq, Zq, 2, U, 0)[0] == 0
    ys = [oracle.mrs(Wp, Zp, Wq, Zq, 2, N24 - 1, U)[1] for U in range(0, N24, N24 // 64)]
    assert set(ys) == {0, 1} and ys.count(0) == 16
    # p(X) = 0 is never accepted, even with the smallest noise value
    Wp, Zp = _weights([0, 4])
    Wq, Zq = _weights([4, 4])
    assert oracle.mrs(Wp, Zp, Wq, Zq, 0, 0, 0) == (0, 1)


def test_inverse_cdf_sample_intervals():
    W, Z = _weights([5, 0, 3, 7, 1])
    counts = np.zeros(5, dtype=np.int64)
    start = 0
    while start < N24:
        y = oracle.sample(W, Z, start)
        lo, hi = start, N24
        while hi - lo > 1:
            mid = (lo + hi) // 2
            if oracle.sample(W, Z, mid) == y:
                lo = mid
            else:
                hi = mid
        counts[y] += hi - start
        start = hi
    for v in range(5):
        assert abs(counts[v] / N24 - W[v] / Z) <= 2 / N24
    assert counts[1] == 0


def test_independent_coupling_collision_and_renyi_bound():
    # Prop. (SJD collision): Pr[X = Y] = sum p q <= exp(-(H2(p) + H2(q)) / 2)
    rng = np.random.default_rng(3)
    for _ in range(5):
        p = rng.integers(1, 50, size=8)
        q = rng.integers(1, 50, size=8)
        Wp, Zp = _weights(p)
        Wq, Zq = _weights(q)
        # draw X ~ q and Y ~ p with independent noise through the oracle's sampler
        n = 1 << 12
        xs = np.array([oracle.sample(Wq, Zq, (i * N24) // n) for i in range(n)])
        ys = np.array([oracle.sample(Wp, Zp, (i * N24) // n) for i in range(n)])
        fq = np.bincount(xs, minlength=8) / n
        fp = np.bincount(ys, minlength=8) / n
        coll = float((fq * fp).sum())
        exact = float((p / p.sum() * q / q.sum()).sum())
        assert abs(coll - exact) < 5e-3
        h2p = -math.log(((p / p.sum()) ** 2).sum())
        h2q = -math.log(((q / q.sum()) ** 2).sum())
        assert exact <= math.exp(-0.5 * (h2p + h2q)) + 1e-12


def test_top_p_is_the_smallest_most_probable_set_reaching_the_mass():
    """Nucleus truncation against its definition worked out with exact fractions and a plain sort,
    against the textbook sort / cumulative-sum recipe (torch) where there are no ties, and on the
    degenerate settings."""
    from fractions import Fraction
    import torch
    rng = np.random.default_rng(11)
    for trial in range(200):
        V = int(rng.integers(1, 40))
        W = rng.integers(0, 50 if trial % 2 else 2**30, size=V).astype(np.uint32)   # small range: many ties
        if W.sum() == 0:
            W[0] = 3
        Z = int(W.sum())
        top_p = float(np.float32(rng.uniform(0.01, 0.99)))
        P24 = int(top_p * 2**24 + 0.5)
        got, Zg = oracle.top_p_filter(W, Z, top_p)
        # definition: walk the distinct weight values downwards until the kept mass reaches P24/2^24 of Z
        theta = None
        for cand in sorted(set(int(w) for w in W if w > 0), reverse=True):
            mass = sum(int(w) for w in W if w >= cand)
            if Fraction(mass, Z) >= Fraction(P24, 2**24):
                theta = cand
                break
        want = np.where(W >= theta, W, 0).astype(np.uint32)
        assert np.array_equal(got, want) and Zg == int(want.sum())
        # minimality: dropping the least probable kept ids falls short of the mass
        above = sum(int(w) for w in W if w > theta)
        assert Fraction(above, Z) < Fraction(P24, 2**24) <= Fraction(Zg, Z)
    # no ties: the usual recipe (sort descending, cumulative sum, keep while the mass before < p)
    for trial in range(50):
        V = 64
        W = rng.permutation(np.arange(1, V + 1) * 1000 + rng.integers(0, 999, V)).astype(np.uint32)
        top_p = float(np.float32(rng.uniform(0.05, 0.95)))
        probs = torch.tensor(W.astype(np.float64) / W.sum())
        sp, si = torch.sort(probs, descending=True)
        before = torch.cumsum(sp, 0) - sp
        keep = torch.zeros(V, dtype=torch.bool)
        keep[si[before < top_p - 1e-9]] = True
        keep2 = torch.zeros(V, dtype=torch.bool)
        keep2[si[before < top_p + 1e-9]] = True
        got, _ = oracle.top_p_filter(W, int(W.sum()), top_p)
        kept = torch.tensor(got > 0)
        assert torch.equal(kept, keep) or torch.equal(kept, keep2)
    # degenerate settings
    W = np.array([5, 9, 9, 1, 0], dtype=np.uint32)
    for off in (0.0, -1.0, 1.0, 2.0):
        got, Zg = oracle.top_p_filter(W, 24, off)
        assert np.array_equal(got, W) and Zg == 24
    got, Zg = oracle.top_p_filter(W, 24, 1e-6)                # the most probable ids only, ties kept
    assert np.array_equal(got, [0, 9, 9, 0, 0]) and Zg == 18
    got, Zg = oracle.top_p_filter(W, 24, 0.75)                # 18/24 = 0.75 exactly: reached
    assert np.array_equal(got, [0, 9, 9, 0, 0]) and Zg == 18
    got, Zg = oracle.top_p_filter(W, 24, 0.76)
    assert np.array_equal(got, [5, 9, 9, 0, 0]) and Zg == 23


def test_race_time_is_the_logarithm_of_the_uniform():
    """The fixed-point -log2 u behind the Gumbel race (Algorithm 4: g = -log(-log u)) against the
    library logarithm, over the whole 24-bit range: a dropped digit, a wrong exponent or an
    off-by-one in u = (U + 1/2) / 2^24 shows here."""
    import math
    rng = np.random.default_rng(3)
    Us = np.concatenate([np.arange(0, 4096), np.arange(2**24 - 4096, 2**24),
                         2 ** np.arange(1, 24), 2 ** np.arange(1, 24) - 1,
                         rng.integers(0, 2**24, 20000)])
    prev = None
    for U in Us.tolist():
        T = oracle.neglog2_q40(U)
        want = -math.log2((U + 0.5) / 2.0**24)
        assert T > 0
        assert abs(T / 2.0**40 - want) < 2.0**-36, (U, T / 2.0**40, want)
    # exact values where the logarithm is an integer or a known constant
    assert oracle.neglog2_q40(0) == 25 << 40                       # u = 2^-25
    assert abs(oracle.neglog2_q40(2**23) / 2.0**40 - (1.0 - math.log2(1.0 + 2.0**-24))) < 2.0**-38
    # monotone: a larger uniform never races later
    seq = [oracle.neglog2_q40(U) for U in range(0, 2**24, 997)]
    assert all(a > b for a, b in zip(seq, seq[1:]))


def test_gumbel_coupling_eq6_marginals_and_bound():
    # Theorem (Gumbel coupling): Pr[X=Y=k] = 1 / sum_j max(P_j/P_k, Q_j/Q_k); marginals P, Q;
    # cost >= (1 - TV) / (1 + TV).
    p = np.array([5, 1, 3, 7, 2, 6], dtype=np.float64)
    q = np.array([2, 6, 3, 1, 8, 4], dtype=np.float64)
    Wp, Zp = _weights(p.astype(int))
    Wq, Zq = _weights(q.astype(int))
    P, Q = p / p.sum(), q / q.sum()
    n = 120000
    xs = np.array([oracle.gumbel_argmax(Wp, 11, 0, pos) for pos in range(n)])
    ys = np.array([oracle.gumbel_argmax(Wq, 11, 0, pos) for pos in range(n)])
    for k in range(6):
        want = 1.0 / np.maximum(P / P[k], Q / Q[k]).sum()
        got = float(((xs == k) & (ys == k)).mean())
        assert abs(got - want) < 5 * math.sqrt(want * (1 - want) / n) + 1e-4
        assert abs((xs == k).mean() - P[k]) < 5 * math.sqrt(P[k] * (1 - P[k]) / n)
        assert abs((ys == k).mean() - Q[k]) < 5 * math.sqrt(Q[k] * (1 - Q[k]) / n)
    tvd = 0.5 * np.abs(P - Q).sum()
    cost = float((xs == ys).mean())
    assert cost >= (1 - tvd) / (1 + tvd) - 0.01
    assert cost <= (1 - tvd) + 0.01


def test_verify_window_first_rejection_and_alpha_mixture():
    # Algorithm 6: all rows evaluated, Accept = first k = 0, a = Accept + 1 (or L if none).
    rng = np.random.default_rng(5)
    L, V = 6, 8
    n_same = {0.0: 0, 0.5: 0, 1.0: 0}
    n_rows = 0
    for trial in range(400):
        p = rng.integers(1, 30, size=(L, V)).astype(np.uint32)
        q = rng.integers(1, 30, size=(L, V)).astype(np.uint32)
        Zp, Zq = p.sum(1).astype(np.uint64), q.sum(1).astype(np.uint64)
        X = np.array([oracle.sample(q[k], int(Zq[k]), int(rng.integers(0, N24))) for k in range(L)])
        a, acc, Y = oracle.verify_window(p, Zp, q, Zq, X, pos0=100 + trial, iteration=trial, seed=9)
        # per-row results equal stand-alone MRS with the row's own noise
        for k in range(L):
            Ua = oracle.noise_u24(9, oracle.NOISE_ACCEPT, 0, 100 + trial + k, trial)
            Ur = oracle.noise_u24(9, oracle.NOISE_RESIDUAL, 0, 100 + trial + k, trial)
            assert (int(acc[k]), int(Y[k])) == oracle.mrs(p[k], int(Zp[k]), q[k], int(Zq[k]), int(X[k]), Ua, Ur)
        rej = [k for k in range(L) if not acc[k]]
        assert a == (rej[0] + 1 if rej else L)
        # SJD / alpha modes leave the committed prefix alone and only redraw rows >= a
        for alpha in (0.0, 0.5, 1.0):
            a2, acc2, Y2 = oracle.verify_window(p, Zp, q, Zq, X, 100 + trial, trial, 9, mode=2, alpha=alpha)
            assert a2 == a and (Y2[:a] == Y[:a]).all()
            n_same[alpha] += int((Y2[a:] == X[a:]).sum())
        n_rows += L - a
    # alpha = 1 is the coupling itself; more coupling -> more identical redraws (Sec. 5.1)
    assert n_same[1.0] > n_same[0.5] > n_same[0.0]


@pytest.mark.parametrize("alpha", [0.0, 0.3, 0.75, 1.0])
def test_alpha_coin_rate_and_coupling_cost(alpha):
    """Algorithm 5 (alpha-coupling): every row beyond the committed prefix keeps its coupled
    redraft with probability alpha and takes an independent draw from p otherwise, so that
    Pr[X = Y] = alpha (1 - TV(p, q)) + (1 - alpha) sum_x p(x) q(x)   (Sec. 5.1, coupling strength).
    The rate of the coin itself is counted on rows where the two candidate outputs differ (what the
    row received then says which branch ran); the cost is counted on all rows. Both within five
    standard deviations over more than 10^5 (position, iteration) keys: a coin firing with alpha/2,
    alpha^2 or 1 - alpha fails for every alpha strictly inside (0, 1), and at the ends."""
    L, V, seed = 33, 8, 77
    p = np.array([9, 1, 14, 3, 0, 6, 11, 4], dtype=np.uint32)
    q = np.array([2, 12, 5, 3, 7, 0, 9, 10], dtype=np.uint32)
    Zp, Zq = int(p.sum()), int(q.sum())
    P, Q = p / Zp, q / Zq
    # row 0 always rejects (its draft has no mass under p0): a = 1, so rows 1..L-1 all meet the coin
    p0 = np.array([1, 1, 1, 1, 0, 0, 0, 0], dtype=np.uint32)
    q0 = np.array([0, 0, 0, 0, 1, 1, 1, 1], dtype=np.uint32)
    Wp = np.vstack([p0] + [p] * (L - 1))
    Wq = np.vstack([q0] + [q] * (L - 1))
    Zps = np.array([4] + [Zp] * (L - 1), dtype=np.uint64)
    Zqs = np.array([4] + [Zq] * (L - 1), dtype=np.uint64)
    rng = np.random.default_rng(int(alpha * 100) + 1)
    n_dist = n_kept = n_rows = n_same = 0
    for trial in range(3200):
        pos0, it = 1000 + 40 * trial, trial % 97
        X = np.array([5] + [oracle.sample(q, Zq, int(u)) for u in rng.integers(0, N24, L - 1)], dtype=np.int32)
        a_mc, _, Y_mc = oracle.verify_window(Wp, Zps, Wq, Zqs, X, pos0, it, seed, mode=0)
        a, _, Y = oracle.verify_window(Wp, Zps, Wq, Zqs, X, pos0, it, seed, mode=2, alpha=alpha)
        assert a_mc == 1 and a == 1 and Y[0] == Y_mc[0]
        for k in range(1, L):
            Ui = oracle.noise_u24(seed, oracle.NOISE_INDEP, 0, pos0 + k, it)
            y_ind = oracle.sample(p, Zp, Ui)
            assert Y[k] in (Y_mc[k], y_ind)
            if Y_mc[k] != y_ind:
                n_dist += 1
                n_kept += int(Y[k] == Y_mc[k])
        n_rows += L - 1
        n_same += int((Y[1:] == X[1:]).sum())
    assert n_rows >= 100_000 and n_dist >= 50_000
    assert abs(n_kept - alpha * n_dist) <= 5 * math.sqrt(alpha * (1 - alpha) * n_dist)
    if alpha in (0.0, 1.0):
        assert n_kept == int(alpha) * n_dist
    tvd = 0.5 * np.abs(P - Q).sum()
    cost = alpha * (1.0 - tvd) + (1.0 - alpha) * float((P * Q).sum())
    assert abs(n_same / n_rows - cost) <= 5 * math.sqrt(cost * (1 - cost) / n_rows)


def test_mrs_never_emits_an_id_without_mass():
    # Algorithm 1 returns a sample of p (Prop. 2.1): a draft outside the support of p is rejected even
    # when it is outside the support of q as well (a caller's mistake, since X ~ q), and the output
    # then comes from norm(max(0, p - q)), whose support lies inside that of p.
    Wp = np.array([0, 5, 0, 3, 9, 0], dtype=np.uint32)
    Wq = np.array([0, 2, 7, 0, 4, 1], dtype=np.uint32)
    Zp, Zq = int(Wp.sum()), int(Wq.sum())
    for X in (0, 2, 5):                                   # p(X) = 0; q(X) = 0 for X = 0
        for Ua in (0, 1, N24 // 2, N24 - 1):
            for Ur in (0, N24 // 3, N24 - 1):
                k, Y = oracle.mrs(Wp, Zp, Wq, Zq, X, Ua, Ur)
                assert k == 0 and Wp[Y] > 0
