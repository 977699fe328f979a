"""Pins of the CPU oracle's verification round against what the paper and the mathematics fix.

Nothing here compares the oracle with itself: the expected values are the paper's printed
numbers (tests/golden), closed forms, invariants, library routines or brute-force enumeration.
"""
import math
import os

import numpy as np
import pytest

from oracle import oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
NEG = -1.0e4          # a logit whose probability is exactly 0 in float64


def read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, val = line.split()
            out[key] = float(val)
    return out


# ------------------------------------------------------------------ Philox
def test_philox_known_answers():
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        rows = [l.split() for l in f if l.strip() and not l.startswith("#")]
    assert len(rows) == 3
    for r in rows:
        vals = [int(x, 16) for x in r]
        got = O.philox4x32_10(vals[0:4], vals[4:6])
        assert [int(x) for x in got] == vals[6:10]


def test_uniform_is_top_24_bits_in_unit_interval():
    assert O.uniform24(0) == 0.0
    assert O.uniform24(0xFFFFFFFF) == 1.0 - 2.0 ** -24
    assert O.uniform24(0x80000000) == 0.5
    assert O.uniform24(0x000000FF) == 0.0           # low 8 bits are dropped
    # each (seed, sequence, round, position) has its own uniforms; they look uniform
    us = np.array([O.round_uniforms(7, s, r, p) for s in range(20) for r in range(20) for p in range(5)])
    assert len({tuple(u) for u in us}) == len(us)
    assert abs(us[:, 0].mean() - 0.5) < 0.02 and abs(us[:, 1].mean() - 0.5) < 0.02
    assert abs(np.corrcoef(us[:, 0], us[:, 1])[0, 1]) < 0.06
    # the seed's high word is part of the key
    assert O.round_uniforms(1, 0, 0, 0) != O.round_uniforms(1 + (1 << 32), 0, 0, 0)


# ------------------------------------------------------------------ softmax
def test_softmax_closed_forms():
    p, bad = O.softmax(np.full(1000, 3.25))
    assert not bad and np.allclose(p, 1e-3, rtol=0, atol=1e-18)
    # two-point row: p0 = 1 / (1 + exp(-(a-b)/T))
    for a, b, T in [(1.0, 0.0, 1.0), (2.5, -1.0, 0.7), (0.0, 3.0, 2.0)]:
        p, _ = O.softmax([a, b], T)
        assert abs(p[0] - 1.0 / (1.0 + math.exp(-(a - b) / T))) < 1e-15
    # shift invariance and temperature scaling: softmax(x/T) == softmax of (x/T) at T=1
    x = np.array([0.3, -1.2, 4.0, 2.2, -7.0])
    p1, _ = O.softmax(x, 0.7)
    p2, _ = O.softmax(x + 123.0, 0.7)
    p3, _ = O.softmax(x / 0.7, 1.0)
    assert np.allclose(p1, p2, atol=1e-13) and np.allclose(p1, p3, atol=1e-15)
    assert abs(p1.sum() - 1.0) < 1e-15
    # hand values: logits ln(1), ln(2), ln(5) -> 1/8, 2/8, 5/8
    p, _ = O.softmax(np.log([1.0, 2.0, 5.0]))
    assert np.allclose(p, [0.125, 0.25, 0.625], atol=1e-15)
    # T = 0.5 squares the odds: 1 : 4 : 25
    p, _ = O.softmax(np.log([1.0, 2.0, 5.0]), 0.5)
    assert np.allclose(p, np.array([1.0, 4.0, 25.0]) / 30.0, atol=1e-15)
    # agrees with scipy on a long random row
    from scipy.special import softmax as sp_softmax
    rng = np.random.RandomState(0)
    x = rng.normal(0, 3, 5000)
    p, _ = O.softmax(x, 0.9)
    assert np.allclose(p, sp_softmax(x / 0.9), atol=1e-15)
    # -inf entries are legal (masked tokens); NaN / +inf / all -inf rows are flagged
    p, bad = O.softmax([0.0, -np.inf, 0.0])
    assert not bad and np.allclose(p, [0.5, 0.0, 0.5])
    for row in ([0.0, np.nan], [0.0, np.inf], [-np.inf, -np.inf]):
        assert O.softmax(row)[1]


def test_argmax_lowest_index_on_ties():
    assert O.argmax([1.0, 3.0, 3.0, 2.0]) == 1
    assert O.argmax([5.0, 5.0, 5.0]) == 0
    rng = np.random.RandomState(1)
    x = np.round(rng.normal(0, 2, 4000) * 4) / 4       # many exact ties
    assert O.argmax(x) == int(np.argmax(x))


# ------------------------------------------------------------------ d_TV
def test_tv_distance_three_way_identity():
    rng = np.random.RandomState(2)
    for V in (2, 7, 1000):
        p = rng.dirichlet(np.ones(V) * 0.3)
        q = rng.dirichlet(np.ones(V) * 0.3)
        d = O.tv_distance(p, q)
        assert abs(d - np.maximum(p - q, 0).sum()) < 1e-14
        assert abs(d - (1.0 - np.minimum(p, q).sum())) < 1e-14
        assert 0.0 <= d <= 1.0
    assert O.tv_distance([0.5, 0.5, 0], [0.5, 0.5, 0]) == 0.0
    assert O.tv_distance([1.0, 0, 0], [0, 0, 1.0]) == 1.0
    assert abs(O.tv_distance([0.5, 0.5], [0.75, 0.25]) - 0.25) < 1e-16


# ------------------------------------------------------------------ inverse CDF
def test_inverse_cdf_rule():
    w = np.array([0.0, 0.2, 0.0, 0.3, 0.5])
    # CDF edges: 0.2 (token 1), 0.5 (token 3), 1.0 (token 4); strict '>' at the edges
    assert O.inverse_cdf(w, 0.0)[0] == 1
    assert O.inverse_cdf(w, 0.19)[0] == 1
    assert O.inverse_cdf(w, 0.2)[0] == 3
    assert O.inverse_cdf(w, 0.49)[0] == 3
    assert O.inverse_cdf(w, 0.5)[0] == 4
    assert O.inverse_cdf(w, 0.999999)[0] == 4
    # unnormalised weights: u scales with the total
    assert O.inverse_cdf(w * 7.0, 0.3)[0] == 3
    # matches numpy's searchsorted on the cumulative sum
    rng = np.random.RandomState(3)
    w = rng.gamma(0.3, size=500) * (rng.rand(500) < 0.5)
    c = np.cumsum(w)
    for u in rng.rand(200):
        tok, margin = O.inverse_cdf(w, u)
        assert tok == int(np.searchsorted(c, u * c[-1], side="right"))
        assert margin >= 0
    assert O.inverse_cdf(np.zeros(4), 0.3)[0] == -1


# ------------------------------------------------------------------ exact law of a round
def _threshold(decide, iters=50):
    """sup{u in [0,1): decide(u)} for a decision that holds on [0, theta)."""
    if not decide(0.0):
        return 0.0
    if decide(1.0 - 2.0 ** -53):
        return 1.0
    lo, hi = 0.0, 1.0
    for _ in range(iters):
        mid = 0.5 * (lo + hi)
        if decide(mid):
            lo = mid
        else:
            hi = mid
    return 0.5 * (lo + hi)


def _step_measure(f, lo=0.0, hi=1.0 - 2.0 ** -53, iters=50):
    """Lebesgue measure of {u: f(u) = y} for a non-decreasing step function f on [0,1)."""
    out = {}

    def rec(a, fa, b, fb):
        if fa == fb:
            return [(a, fa)]
        lo_, hi_ = a, b
        for _ in range(iters):
            mid = 0.5 * (lo_ + hi_)
            if f(mid) == fa:
                lo_ = mid
            else:
                hi_ = mid
        edge = 0.5 * (lo_ + hi_)
        fh = f(hi_)
        return [(a, fa)] + [(edge if i == 0 else s, v) for i, (s, v) in enumerate(rec(hi_, fh, b, fb))]

    segs = rec(lo, f(lo), hi, f(hi))
    starts = [s for s, _ in segs] + [1.0]
    starts[0] = 0.0
    for i, (_, v) in enumerate(segs):
        out[v] = out.get(v, 0.0) + starts[i + 1] - starts[i]
    return out


def exact_round_law(target, draft, T):
    """Brute-force law of one round of the oracle's verification.

    Enumerates every drafted block x in V^k with its probability prod_j q_j(x_j) and measures, by
    bisection on the uniforms the oracle is given, the probability of every outcome.  Returns
    (law of N_acc, dict position m -> P(reach position m and emit token y there))."""
    target, draft = np.asarray(target, float), np.asarray(draft, float)
    k, V = draft.shape
    q = [O.softmax(draft[j], T)[0] for j in range(k)]
    n_acc_law = np.zeros(k + 1)
    emit = [np.zeros(V) for _ in range(k + 1)]     # emit[m][y]: token y is the m-th emitted token
    support = [np.nonzero(q[j] > 0)[0] for j in range(k)]

    def blocks(j):
        if j == k:
            yield (), 1.0
            return
        for rest, pr in blocks(j + 1):
            for x in support[j]:
                yield (int(x),) + rest, pr * q[j][x]

    for x, prob_x in blocks(0):
        theta = []
        for j in range(k):
            def decide(u, j=j):
                ua = np.zeros(k)
                ua[j] = u
                return bool(O.verify_sequence(target, draft, x, T, ua, np.zeros(k + 1))["accept"][j])
            theta.append(_threshold(decide))
        reach = 1.0
        for n in range(k + 1):
            p_here = reach * ((1.0 - theta[n]) if n < k else 1.0)   # N_acc = n given x
            n_acc_law[n] += prob_x * p_here
            # emitted tokens: positions 0..n-1 are the accepted drafts, position n the correction/bonus
            if n < k:
                emit[n][x[n]] += prob_x * reach * theta[n]
            if p_here > 0:
                ua = np.array([0.0 if j < n else (1.0 - 2.0 ** -53) for j in range(k)])
                if n < k:
                    ua[n] = 0.5 * (theta[n] + 1.0)

                def sample(u, n=n, ua=ua):
                    us = np.zeros(k + 1)
                    us[n] = u
                    r = O.verify_sequence(target, draft, x, T, ua, us)
                    assert r["accepted_len"] == n
                    return r["next_token"]
                for y, m in _step_measure(sample).items():
                    emit[n][y] += prob_x * p_here * m
            if n < k:
                reach *= theta[n]
    return n_acc_law, emit


@pytest.mark.parametrize("V,k,T", [(2, 1, 1.0), (3, 2, 1.0), (3, 2, 0.7), (5, 1, 1.3), (4, 3, 1.0)])
def test_losslessness_by_exact_enumeration(V, k, T):
    """The m-th emitted token, given that the round reaches position m, follows the target's
    distribution at that position (speculative sampling is lossless)."""
    rng = np.random.RandomState(100 * V + k)
    target = rng.normal(0, 1.5, (k + 1, V))
    draft = target[:k] + rng.normal(0, 1.0, (k, V))
    n_acc_law, emit = exact_round_law(target, draft, T)
    assert abs(n_acc_law.sum() - 1.0) < 1e-12
    from scipy.special import softmax as sp_softmax
    reach = 1.0
    for m in range(k + 1):
        p_m = sp_softmax(target[m] / T)
        assert abs(emit[m].sum() - reach) < 1e-11
        assert np.allclose(emit[m] / reach, p_m, atol=1e-10), (m, emit[m] / reach, p_m)
        if m < k:
            reach -= n_acc_law[m]          # P(N_acc > m) = P(reach position m+1)


def _constant_alpha_rows(alpha, k):
    """Rows with sum_v min(p, q) = alpha at every position: p = (a, 1-a, 0), q = (a, 0, 1-a)."""
    with np.errstate(divide="ignore"):
        lp = np.log(np.array([alpha, 1 - alpha, 0.0]))
        lq = np.log(np.array([alpha, 0.0, 1 - alpha]))
    lp[np.isneginf(lp)] = NEG
    lq[np.isneginf(lq)] = NEG
    return np.tile(lp, (k + 1, 1)), np.tile(lq, (k, 1))


@pytest.mark.parametrize("alpha,k", [(0.1, 5), (0.5, 5), (0.8, 5), (0.6, 3)])
def test_accepted_length_statistics_closed_forms(alpha, k):
    """E[N_acc] and Var[N_acc] of the lemma "BE reward statistics", and the BE/BD ratio lemma."""
    target, draft = _constant_alpha_rows(alpha, k)
    law, _ = exact_round_law(target, draft, 1.0)
    n = np.arange(k + 1)
    mean = (law * n).sum()
    var = (law * n * n).sum() - mean ** 2
    a = alpha
    assert abs(mean - (a - a ** (k + 1)) / (1 - a)) < 1e-10
    closed_var = a * (1 - (2 * k + 1) * a ** k + (2 * k + 1) * a ** (k + 1) - a ** (2 * k + 1)) / (1 - a) ** 2
    assert abs(var - closed_var) < 1e-10
    # BD reward of these rows is alpha (1 - d_TV = alpha at every position) ...
    r = O.verify_sequence(target, draft, [0] * k, 1.0, np.zeros(k), np.zeros(k + 1))
    assert abs(r["reward"] - a) < 1e-14 and np.allclose(r["D"], 1 - a, atol=1e-14)
    # ... and E[r_BE] = (1 - a^k) / (k (1 - a)) * E[r_BD]
    assert abs(mean / k - (1 - a ** k) / (k * (1 - a)) * r["reward"]) < 1e-10


def test_worked_example_of_the_stopping_time_lemma():
    g = read_golden("worked_example_stopping_time.txt")
    k = int(g["n_max"])
    means, rewards = {}, {}
    for name in ("alpha_1", "alpha_2", "alpha_3"):
        target, draft = _constant_alpha_rows(g[name], k)
        law, _ = exact_round_law(target, draft, 1.0)
        means[name] = (law * np.arange(k + 1)).sum()
        rewards[name] = O.verify_sequence(target, draft, [0] * k, 1.0, np.zeros(k), np.zeros(k + 1))["reward"]
    assert abs(means["alpha_1"] + means["alpha_3"] - g["expected_accepted_first_two_rounds_pi1"]) < 1e-9
    assert abs(2 * means["alpha_2"] - g["expected_accepted_first_two_rounds_pi2"]) < 1e-9
    best = rewards["alpha_3"]
    assert abs((best - rewards["alpha_1"]) + (best - rewards["alpha_3"]) - g["bd_regret_pi1"]) < 1e-12
    assert abs(2 * (best - rewards["alpha_2"]) - g["bd_regret_pi2"]) < 1e-12


def test_be_reward_variance_peaks_where_the_paper_says():
    g = read_golden("be_variance_n5.txt")
    k = int(g["n_max"])
    alphas = np.round(np.arange(0.775, 0.856, 0.005), 3)
    var = []
    for a in alphas:
        target, draft = _constant_alpha_rows(a, k)
        law, _ = exact_round_law(target, draft, 1.0)
        n = np.arange(k + 1) / k                      # r_BE = N_acc / N_max
        var.append((law * n * n).sum() - (law * n).sum() ** 2)
    var = np.array(var)
    peak = alphas[int(np.argmax(var))]
    assert abs(peak - g["argmax_alpha_of_var_be"]) <= 0.0051
    assert np.all(np.diff(var[alphas <= peak]) > 0)   # increasing up to the peak


# ------------------------------------------------------------------ the real Philox stream
def test_chi_square_with_the_philox_stream():
    """With the oracle's own uniforms the emitted tokens still follow the target (V = 8, k = 2)."""
    from scipy.stats import chi2
    from scipy.special import softmax as sp_softmax
    V, k, B, rounds = 8, 2, 2000, 100
    rng = np.random.RandomState(5)
    base = np.array([1.2, 0.3, -0.5, 0.9, 0.0, -1.0, 0.6, -0.2])
    target = np.stack([base, base[::-1], np.roll(base, 3)]).astype(np.float32)
    draft = (target[:k] + rng.normal(0, 0.8, (k, V))).astype(np.float32)
    p = [sp_softmax(target[j].astype(float)) for j in range(k + 1)]
    q = [sp_softmax(draft[j].astype(float)) for j in range(k)]
    assert min(pp.min() for pp in p) > 1e-3
    cfg = O.OracleConfig(max_batch=B, n_drafters=1, vocab=V)
    orc = O.OracleMetaSD(cfg)
    tgt = np.ascontiguousarray(np.broadcast_to(target, (B, k + 1, V)))
    drf = np.ascontiguousarray(np.broadcast_to(draft, (B, k, V)))
    counts = [np.zeros(V) for _ in range(k + 1)]
    acc_hist = np.zeros(k + 1)
    for _ in range(rounds):
        tokens = np.stack([rng.choice(V, size=B, p=q[j]) for j in range(k)], axis=1).astype(np.int32)
        out = orc.verify(tgt, drf, tokens, 1.0, seed=2024)
        n_acc = out["accepted_len"]
        assert n_acc.min() >= 0 and n_acc.max() <= k
        acc_hist += np.bincount(n_acc, minlength=k + 1)
        for m in range(k + 1):
            took_draft = n_acc > m
            counts[m] += np.bincount(tokens[took_draft, m], minlength=V) if m < k else 0
            counts[m] += np.bincount(out["next_token"][n_acc == m], minlength=V)
    assert orc.t[0] == rounds                       # the round counter keys fresh uniforms each round
    for m in range(k + 1):
        n = counts[m].sum()
        stat = ((counts[m] - n * p[m]) ** 2 / (n * p[m])).sum()
        assert stat < chi2.ppf(1 - 1e-4, V - 1), (m, stat)
    # acceptance frequency at position 0 is 1 - d_TV(p_0, q_0)
    alpha0 = np.minimum(p[0], q[0]).sum()
    assert abs(1 - acc_hist[0] / (B * rounds) - alpha0) < 4 * math.sqrt(alpha0 * (1 - alpha0) / (B * rounds))
    assert abs(out["D"][0, 0] - (1 - alpha0)) < 1e-12


# ------------------------------------------------------------------ special cases
def test_identical_and_disjoint_distributions():
    rng = np.random.RandomState(6)
    k, V = 4, 50
    target = rng.normal(0, 2, (k + 1, V))
    # q == p: every token accepted whatever the uniforms, N_acc = k, reward 1
    for trial in range(20):
        r = O.verify_sequence(target, target[:k], rng.randint(0, V, k), 1.0, rng.rand(k), rng.rand(k + 1))
        assert r["accepted_len"] == k and r["accept"].all() and abs(r["reward"] - 1) < 1e-15
    # disjoint supports: nothing accepted, correction token follows p_0
    tgt = np.full((k + 1, V), NEG)
    drf = np.full((k, V), NEG)
    tgt[:, : V // 2] = rng.normal(0, 1, (k + 1, V // 2))
    drf[:, V // 2:] = rng.normal(0, 1, (k, V // 2))
    p0 = O.softmax(tgt[0])[0]
    cdf = np.cumsum(p0)
    for u in rng.rand(50):
        r = O.verify_sequence(tgt, drf, rng.randint(V // 2, V, k), 1.0, rng.rand(k), np.full(k + 1, u))
        assert r["accepted_len"] == 0 and abs(r["reward"]) < 1e-15
        assert r["next_token"] == int(np.searchsorted(cdf, u * cdf[-1], side="right"))


def test_accept_rule_is_strict_and_division_free():
    # p(x) = 1/4, q(x) = 1/2  ->  accept iff u < 1/2 (strict)
    target = np.log(np.array([[0.25, 0.75], [0.5, 0.5]]))
    draft = np.log(np.array([[0.5, 0.5]]))
    for u, want in [(0.0, 1), (0.4999999, 1), (0.5, 0), (0.75, 0)]:
        r = O.verify_sequence(target, draft, [0], 1.0, [u], [0.3, 0.3])
        assert r["accept"][0] == want
    # p(x) >= q(x): accepted for every u in [0, 1)
    r = O.verify_sequence(target, draft, [1], 1.0, [1 - 2.0 ** -24], [0.3, 0.3])
    assert r["accept"][0] == 1 and r["accepted_len"] == 1
    # rejected at token 0: residual (p - q)+ = (0, 0.25) -> always token 1
    r = O.verify_sequence(target, draft, [0], 1.0, [0.9], [0.01, 0.3])
    assert r["accepted_len"] == 0 and r["next_token"] == 1
    # q(x) = 0 < p(x): accepted and flagged; p(x) = q(x) = 0: rejected
    t2 = np.array([[0.0, 0.0, NEG], [0.0, 0.0, 0.0]])
    d2 = np.array([[0.0, NEG, NEG]])
    r = O.verify_sequence(t2, d2, [1], 1.0, [0.99], [0.5, 0.5])
    assert r["accept"][0] == 1 and r["status"] & O.STATUS_Q_ZERO
    r = O.verify_sequence(t2, d2, [2], 1.0, [0.0], [0.5, 0.5])
    assert r["accept"][0] == 0
    # token id out of range: rejected and flagged
    r = O.verify_sequence(t2, d2, [3], 1.0, [0.0], [0.5, 0.5])
    assert r["accept"][0] == 0 and r["status"] & O.STATUS_TOKEN_OOR
    r = O.verify_sequence(t2, d2, [-1], 1.0, [0.0], [0.5, 0.5])
    assert r["accept"][0] == 0 and r["status"] & O.STATUS_TOKEN_OOR


def test_nonfinite_rows_have_defined_outcomes():
    target = np.zeros((3, 4))
    draft = np.zeros((2, 4))
    draft[1, 2] = np.nan
    r = O.verify_sequence(target, draft, [0, 0], 1.0, [0.0, 0.0], [0.5] * 3)
    assert r["status"] & O.STATUS_NONFINITE
    assert r["accept"].tolist() == [1, 0] and r["accepted_len"] == 1
    assert r["D"][1] == 1.0 and r["next_token"] == -1
    assert abs(r["reward"] - 0.5) < 1e-15


# ------------------------------------------------------------------ greedy
def test_greedy_mode_follows_the_target_argmax_chain():
    rng = np.random.RandomState(7)
    k, V = 6, 300
    for trial in range(30):
        target = np.round(rng.normal(0, 3, (k + 1, V)) * 8) / 8     # ties happen
        draft = target[:k] + rng.normal(0, 0.6, (k, V))
        tokens = draft.argmax(axis=1)
        chain = target.argmax(axis=1)                                 # numpy: first index on ties
        match = tokens == chain[:k]
        want_len = k if match.all() else int(np.argmin(match))
        r = O.verify_sequence(target, draft, tokens, 0.0, rng.rand(k), rng.rand(k + 1))
        assert r["accepted_len"] == want_len
        assert r["next_token"] == chain[want_len]
        assert r["accept"].tolist() == match.astype(int).tolist()
        # the reward still comes from the soft distributions (reward temperature 1): in (0, 1]
        assert 0.0 < r["reward"] <= 1.0
        from scipy.special import softmax as sp_softmax
        d = [0.5 * np.abs(sp_softmax(target[j]) - sp_softmax(draft[j])).sum() for j in range(k)]
        assert abs(r["reward"] - (1 - np.mean(d))) < 1e-13


# ------------------------------------------------------------------ rewards
def test_bd_reward_statistics_on_toy_rows():
    """E[r_BD] = alpha and Var[r_BD] <= 1/(4 N_max) when 1 - d_TV is i.i.d. with mean alpha."""
    rng = np.random.RandomState(8)
    k, n_rounds = 5, 3000
    rewards = []
    for _ in range(n_rounds):
        alphas = rng.beta(2.0, 2.0, size=k)             # mean 0.5
        target = np.zeros((k + 1, 3))
        draft = np.zeros((k, 3))
        for j, a in enumerate(alphas):
            t_, d_ = _constant_alpha_rows(a, 1)
            target[j], draft[j] = t_[0], d_[0]
        r = O.verify_sequence(target, draft, [0] * k, 1.0, rng.rand(k), rng.rand(k + 1))
        assert 0.0 < r["reward"] <= 1.0
        assert abs(r["reward"] - alphas.mean()) < 1e-12
        rewards.append(r["reward"])
    rewards = np.array(rewards)
    assert abs(rewards.mean() - 0.5) < 4 * rewards.std() / math.sqrt(n_rounds)
    assert rewards.var() <= 1.0 / (4 * k)


def test_be_reward_is_accepted_fraction():
    rng = np.random.RandomState(9)
    k, V = 5, 20
    target = rng.normal(0, 1, (k + 1, V))
    draft = target[:k] + rng.normal(0, 1, (k, V))
    for _ in range(50):
        r = O.verify_sequence(target, draft, rng.randint(0, V, k), 1.0, rng.rand(k), rng.rand(k + 1),
                              reward_kind=O.REWARD_BE)
        assert r["reward"] == r["accepted_len"] / k


# ------------------------------------------------------------------ serving loop
def test_single_drafter_stopping_time_bounds():
    """Lemma "single process stopping time": playing one drafter until B_tok tokens are out,
    B(1-a)/(1-a^(N+1)) - 1 < E[tau] <= (B+1)(1-a)/(1-a^(N+1))."""
    alpha, k, B_tok, n_seq = 0.6, 5, 200, 4000
    target, draft = _constant_alpha_rows(alpha, k)
    cfg = O.OracleConfig(max_batch=n_seq, n_drafters=1, vocab=3)
    orc = O.OracleMetaSD(cfg)
    tgt = np.ascontiguousarray(np.broadcast_to(target.astype(np.float32), (n_seq, k + 1, 3)))
    drf = np.ascontiguousarray(np.broadcast_to(draft.astype(np.float32), (n_seq, k, 3)))
    rng = np.random.RandomState(10)
    length = np.zeros(n_seq, dtype=np.int64)
    tau = np.zeros(n_seq, dtype=np.int64)
    while (length < B_tok).any():
        tokens = np.where(rng.rand(n_seq, k) < alpha, 0, 2).astype(np.int32)    # x ~ q
        out = orc.verify(tgt, drf, tokens, 1.0, seed=99)
        live = length < B_tok
        tau += live
        length += np.where(live, out["accepted_len"] + 1, 0)      # l <- l + N_acc + 1 (Algorithm 1)
    scale = (1 - alpha) / (1 - alpha ** (k + 1))
    se = tau.std() / math.sqrt(n_seq)
    assert B_tok * scale - 1 - 4 * se < tau.mean() <= (B_tok + 1) * scale + 4 * se
    # tokens out = rounds + accepted tokens (proof of the stopping-time lemma), per sequence
    assert (length >= B_tok).all() and (length < B_tok + k + 1).all()


def test_ragged_round_equals_the_fixed_length_round_on_the_truncated_rows():
    """A sequence that drafted kb < k tokens is a round of draft length kb on its first kb + 1 target rows and
    kb draft rows: same uniforms (keyed by position), reward normalised by kb, nothing behind those rows is read."""
    rng = np.random.RandomState(5)
    B, k, V = 6, 5, 97
    target = rng.randn(B, k + 1, V).astype(np.float32) * 2
    draft = (target[:, :k] + rng.randn(B, k, V).astype(np.float32)).astype(np.float32)
    tokens = rng.randint(0, V, size=(B, k)).astype(np.int32)
    lens = np.array([1, 2, 3, 4, 5, 3], dtype=np.int32)
    poisoned_t, poisoned_d = target.copy(), draft.copy()
    for b in range(B):                                   # rows behind the drafted ones must not matter
        poisoned_t[b, lens[b] + 1:] = np.nan
        poisoned_d[b, lens[b]:] = np.nan
    for reward in (O.REWARD_BD, O.REWARD_BE):
        cfg = O.OracleConfig(max_batch=B, n_drafters=2, vocab=V, reward=reward)
        ragged = O.OracleMetaSD(cfg).verify(poisoned_t, poisoned_d, tokens, 1.0, 77, update=False, draft_len=lens)
        assert (ragged["status"] == 0).all()
        for b in range(B):
            kb = int(lens[b])
            one = O.OracleMetaSD(O.OracleConfig(max_batch=1, n_drafters=2, vocab=V, reward=reward, sequence_base=b))
            fixed = one.verify(target[b:b + 1, :kb + 1], draft[b:b + 1, :kb], tokens[b:b + 1, :kb], 1.0, 77,
                               update=False)
            assert ragged["accepted_len"][b] == fixed["accepted_len"][0] <= kb
            assert ragged["next_token"][b] == fixed["next_token"][0]
            assert ragged["reward"][b] == fixed["reward"][0]
            assert np.array_equal(ragged["D"][b, :kb], fixed["D"][0])
            assert np.array_equal(ragged["accept"][b, :kb], fixed["accept"][0])
    full = O.OracleMetaSD(cfg).verify(target, draft, tokens, 1.0, 77, update=False, draft_len=np.full(B, k))
    plain = O.OracleMetaSD(cfg).verify(target, draft, tokens, 1.0, 77, update=False)
    for key in ("accepted_len", "next_token", "reward", "D", "accept"):
        assert np.array_equal(full[key], plain[key])


# ------------------------------------------------------------------ random-number keying, pointer-table mode
def _documented_uniforms(seed, sequence, round_, position):
    """The convention fixed for both sides: Philox4x32-10 with key (seed low, seed high) at counter
    (sequence, round, position, 0); word 0 is the accept test's uniform, word 1 the draw's; top 24 bits."""
    w = O.philox4x32_10([sequence, round_, position, 0], [seed & 0xFFFFFFFF, seed >> 32])
    return (int(w[0]) >> 8) / 2.0 ** 24, (int(w[1]) >> 8) / 2.0 ** 24


def test_round_uniforms_follow_the_documented_counter_and_words():
    for seed, seq, rnd, pos in [(0, 0, 0, 0), (7, 1, 2, 3), (0xDEADBEEF12345678, 4000000000, 17, 5),
                                (1 << 40, 9, 300, 16), (555, 3, 1, 2), (555, 1, 3, 2), (555, 2, 1, 3)]:
        assert O.round_uniforms(seed, seq, rnd, pos) == _documented_uniforms(seed, seq, rnd, pos)
    # swapping any two counter fields gives other numbers (the three cases above with 1, 2, 3 permuted)
    assert len({O.round_uniforms(555, *c) for c in [(3, 1, 2), (1, 3, 2), (2, 1, 3)]}) == 3


def test_batch_round_draws_its_uniforms_by_sequence_round_and_position():
    """The batch call, replayed sequence by sequence with uniforms rebuilt from the Philox block of
    (sequence_base + b, round of b, position): accept uniforms from word 0, the draw at position j from word 1
    of position j's block.  A swapped counter field or word would move tokens and accepted lengths."""
    rng = np.random.RandomState(12)
    B, k, V, base, seed = 24, 4, 61, 1000, 0x1234ABCD5678
    target = (rng.randn(B, k + 1, V) * 2).astype(np.float32)
    draft = (target[:, :k] + rng.randn(B, k, V)).astype(np.float32)
    tokens = rng.randint(0, V, size=(B, k)).astype(np.int32)
    orc = O.OracleMetaSD(O.OracleConfig(max_batch=B, n_drafters=3, vocab=V, sequence_base=base))
    orc.t[:] = rng.randint(0, 50, size=B)
    rounds = orc.t.copy()
    out = orc.verify(target, draft, tokens, 0.9, seed, update=False)
    lens = set()
    for b in range(B):
        ua = [_documented_uniforms(seed, base + b, int(rounds[b]), j)[0] for j in range(k)]
        us = [_documented_uniforms(seed, base + b, int(rounds[b]), j)[1] for j in range(k + 1)]
        assert np.array_equal(out["u_accept"][b], ua)
        one = O.verify_sequence(target[b], draft[b], tokens[b], 0.9, ua, us)
        assert one["accepted_len"] == out["accepted_len"][b] and one["next_token"] == out["next_token"][b]
        assert np.array_equal(one["accept"], out["accept"][b])
        lens.add(one["accepted_len"])
    assert len(lens) >= 3          # rejections at several positions and full acceptance are all covered


def test_pointer_table_mode_equals_gathered_mode():
    """Reading drafter arm[b]'s rows through the table of K tensors is the same round as reading rows that
    were gathered by arm beforehand: every output, bit for bit, and the same bandit state afterwards."""
    rng = np.random.RandomState(3)
    B, K, k, V = 7, 3, 3, 53
    for bandit in (O.UCB, O.SWUCB):
        tab = O.OracleMetaSD(O.OracleConfig(max_batch=B, n_drafters=K, vocab=V, bandit=bandit, tau=4))
        gat = O.OracleMetaSD(O.OracleConfig(max_batch=B, n_drafters=K, vocab=V, bandit=bandit, tau=4))
        for t in range(9):
            target = (rng.randn(B, k + 1, V) * 2).astype(np.float32)
            drafts = [(target[:, :k] + (0.3 + i) * rng.randn(B, k, V)).astype(np.float32) for i in range(K)]
            tokens = rng.randint(0, V, size=(K, B, k)).astype(np.int32)
            arm = gat.select()
            assert np.array_equal(arm, tab.select())
            rows = np.stack(drafts)[arm, np.arange(B)]
            toks = tokens[arm, np.arange(B)]
            # a table rotated by one drafter gives another round: the table really is indexed by the arm
            wrong = tab.verify(target, None, toks, 1.0, 99, drafter_tables=[drafts[(i + 1) % K] for i in range(K)],
                               update=False)
            a = tab.verify(target, None, toks, 1.0, 99, drafter_tables=drafts)
            b = gat.verify(target, rows, toks, 1.0, 99)
            for key in ("accepted_len", "next_token", "reward", "p_x", "q_x", "D", "accept", "u_accept", "sample_margin"):
                assert np.array_equal(a[key], b[key]), key
            assert not (wrong["D"] == a["D"]).any()
        assert np.array_equal(tab.stat_a, gat.stat_a) and np.array_equal(tab.t, gat.t)
