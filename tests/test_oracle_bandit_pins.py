"""Pins of the CPU oracle's bandit policies (MetaSD-UCB, Discounted UCB, Sliding-window UCB, EXP3, Rand, PETC).

Expected values are invariants, textbook consequences of the index rule, the explicit-constant
pull bound the paper quotes, and reductions between the variants -- never the oracle's own output.
"""
import math

import numpy as np
import pytest

from oracle import oracle as O


def run_bandit(variant, K, reward_fn, rounds, beta=1.0, gamma=1.0, tau=10 ** 6, seed=0):
    """Drive one oracle bandit instance with rewards reward_fn(arm, t, rng); returns the logs."""
    cfg = O.OracleConfig(max_batch=1, n_drafters=K, vocab=1, bandit=variant, beta=beta, gamma=gamma,
                         tau=min(tau, rounds + 1))
    orc = O.OracleMetaSD(cfg)
    rng = np.random.RandomState(seed)
    arms, rewards = [], []
    for t in range(rounds):
        a = int(orc.select()[0])
        r = float(reward_fn(a, t, rng))
        orc.update([a], [r])
        arms.append(a)
        rewards.append(r)
    return np.array(arms), np.array(rewards), orc


def test_init_sweep_plays_every_arm_once_in_order():
    for variant in (O.UCB, O.DUCB, O.SWUCB):
        arms, _, orc = run_bandit(variant, 5, lambda a, t, g: g.rand(), 5, gamma=0.9, tau=50)
        assert arms.tolist() == [0, 1, 2, 3, 4]
        assert orc.t[0] == 5
    arms, _, _ = run_bandit(O.UCB, 1, lambda a, t, g: g.rand(), 20)      # K = 1: ln 1 = 0, always arm 0
    assert (arms == 0).all()


def test_ucb_mean_is_the_batch_mean_and_counts_are_pull_counts():
    arms, rewards, orc = run_bandit(O.UCB, 4, lambda a, t, g: g.beta(1 + a, 2), 400, beta=0.5, seed=3)
    mu, n = orc.mean_estimates()
    for i in range(4):
        assert n[0, i] == (arms == i).sum()
        assert abs(mu[0, i] - rewards[arms == i].mean()) < 1e-12
    assert n.sum() == 400


def test_equal_means_make_ucb_round_robin():
    """With identical constant rewards the index differs only by sqrt(2 ln t / n_i): the least
    pulled arm wins, lowest index first, so the arms are played in strict rotation."""
    arms, _, _ = run_bandit(O.UCB, 4, lambda a, t, g: 0.5, 80, beta=0.3)
    assert arms.tolist() == [t % 4 for t in range(80)]


def test_zero_exploration_is_greedy_on_the_means():
    means = [0.2, 0.7, 0.4]
    arms, _, _ = run_bandit(O.UCB, 3, lambda a, t, g: means[a], 50, beta=0.0)
    assert arms[:3].tolist() == [0, 1, 2] and (arms[3:] == 1).all()


@pytest.mark.parametrize("beta,delta,T", [(1.0, 0.5, 20000), (0.5, 0.3, 20000), (1.0, 0.25, 50000)])
def test_deterministic_two_arm_pull_count_matches_index_equalisation(beta, delta, T):
    """Two arms with constant rewards c0 > c1.  UCB keeps the two indices level, so after T rounds
    the worse arm's count n1 solves c1 + beta sqrt(2 ln T / n1) = c0 + beta sqrt(2 ln T / (T - n1)).
    This fixes the constant 2, the natural logarithm and beta in the exploration term."""
    c0, c1 = 0.8, 0.8 - delta
    arms, _, _ = run_bandit(O.UCB, 2, lambda a, t, g: (c0, c1)[a], T, beta=beta)
    n1 = int((arms == 1).sum())
    L = 2.0 * math.log(T)
    x = 1.0
    for _ in range(200):                              # fixed point of the level-index equation
        x = beta ** 2 * L / (delta + beta * math.sqrt(L / (T - x))) ** 2
    assert abs(n1 - x) <= 0.05 * x + 2, (n1, x)
    # a missing factor 2, log10 or log2 instead of ln would be far outside this band
    assert abs(x / 2 - n1) > 0.2 * x and abs(x / math.log(10) - n1) > 0.2 * x


def test_suboptimal_pull_bound_with_explicit_constants():
    """E[n_i(tau)] <= 8 ln tau / Delta_i^2 + 1 + pi^2/3 for beta = 1 (the lemma quoted from Auer et al.)."""
    means = np.array([0.75, 0.55, 0.35])
    rounds, seeds = 3000, 60
    pulls = np.zeros((seeds, 3))
    for s in range(seeds):
        arms, _, _ = run_bandit(O.UCB, 3, lambda a, t, g: g.beta(4 * means[a], 4 * (1 - means[a])), rounds,
                                beta=1.0, seed=s)
        pulls[s] = np.bincount(arms, minlength=3)
    for i in (1, 2):
        delta = means[0] - means[i]
        bound = 8 * math.log(rounds) / delta ** 2 + 1 + math.pi ** 2 / 3
        assert pulls[:, i].mean() <= bound
    assert pulls[:, 0].mean() > 0.6 * rounds            # the best arm dominates
    # the number of suboptimal pulls grows like ln(rounds), not linearly: x10 rounds -> far less than x10 pulls
    short = np.mean([np.bincount(run_bandit(O.UCB, 3, lambda a, t, g: g.beta(4 * means[a], 4 * (1 - means[a])),
                                            300, beta=1.0, seed=s)[0], minlength=3)[1:].sum() for s in range(30)])
    assert pulls[:, 1:].sum(axis=1).mean() < 4.0 * short


def test_bd_form_of_the_pull_bound():
    """With the BD reward (mean of N_max i.i.d. alignment samples) and beta = 1/sqrt(N_max) the
    bound tightens to 8 ln tau / (N_max Delta^2) + 1 + pi^2/3."""
    k = 5
    alphas = np.array([0.8, 0.6])
    rounds, seeds = 3000, 60
    pulls = []
    for s in range(seeds):
        arms, _, _ = run_bandit(
            O.UCB, 2, lambda a, t, g: g.beta(4 * alphas[a], 4 * (1 - alphas[a]), size=k).mean(), rounds,
            beta=1 / math.sqrt(k), seed=1000 + s)
        pulls.append((arms == 1).sum())
    bound = 8 * math.log(rounds) / (k * 0.2 ** 2) + 1 + math.pi ** 2 / 3
    assert np.mean(pulls) <= bound


def test_ducb_and_swucb_reduce_to_ucb():
    """gamma = 1 and a window longer than the run reproduce Algorithm 2 arm for arm."""
    fn = lambda a, t, g: g.beta(2 + a, 3)
    for beta in (0.01, 0.4, 1.0):
        base, rew, _ = run_bandit(O.UCB, 5, fn, 600, beta=beta, seed=11)
        d_arms, d_rew, _ = run_bandit(O.DUCB, 5, fn, 600, beta=beta, gamma=1.0, seed=11)
        s_arms, s_rew, _ = run_bandit(O.SWUCB, 5, fn, 600, beta=beta, tau=10 ** 6, seed=11)
        assert d_arms.tolist() == base.tolist() and np.array_equal(d_rew, rew)
        assert s_arms.tolist() == base.tolist() and np.array_equal(s_rew, rew)


def test_ducb_recursion_equals_the_direct_discounted_sums():
    gamma = 0.93
    arms, rewards, orc = run_bandit(O.DUCB, 4, lambda a, t, g: g.rand(), 300, beta=0.2, gamma=gamma, seed=5)
    t_end = len(arms)
    w = gamma ** (t_end - 1 - np.arange(t_end))        # weight of round s once round t_end-1 is in
    mu, n = orc.mean_estimates()
    for i in range(4):
        S = (w * rewards * (arms == i)).sum()
        N = (w * (arms == i)).sum()
        assert abs(n[0, i] - N) < 1e-10 and abs(mu[0, i] - S / N) < 1e-10


def test_swucb_window_holds_exactly_the_last_tau_rounds():
    tau = 17
    arms, rewards, orc = run_bandit(O.SWUCB, 3, lambda a, t, g: g.rand(), 200, beta=0.3, tau=tau, seed=6)
    mu, n = orc.mean_estimates()
    last_a, last_r = arms[-tau:], rewards[-tau:]
    for i in range(3):
        assert n[0, i] == (last_a == i).sum()
        if n[0, i] > 0:
            assert abs(mu[0, i] - last_r[last_a == i].mean()) < 1e-12


def test_swucb_arm_that_left_the_window_is_played_again():
    """An arm with no pull inside the window has an infinite index (lowest index first)."""
    means = [0.9, 0.1, 0.1]
    arms, _, _ = run_bandit(O.SWUCB, 3, lambda a, t, g: means[a], 60, beta=0.01, tau=8)
    # arm 0 is best, but every arm reappears at least once in any stretch of tau + 3 rounds
    for start in range(3, 60 - 11):
        assert set(arms[start:start + 11].tolist()) == {0, 1, 2}


def test_nonstationary_variants_recover_after_a_swap():
    """After the arm means swap, D-UCB and SW-UCB return to the new best arm; plain UCB lags."""
    def fn(a, t, g):
        means = (0.8, 0.5) if t < 1500 else (0.4, 0.5)
        return g.beta(8 * means[a], 8 * (1 - means[a]))
    ratio = {}
    for name, variant, kw in (("ucb", O.UCB, {}), ("ducb", O.DUCB, dict(gamma=0.97)),
                              ("sw", O.SWUCB, dict(tau=100))):
        hits = []
        for s in range(10):
            arms, _, _ = run_bandit(variant, 2, fn, 2000, beta=0.1, seed=s, **kw)
            hits.append((arms[1600:] == 1).mean())
        ratio[name] = np.mean(hits)
    assert ratio["ducb"] > 0.7 and ratio["sw"] > 0.8 and ratio["ucb"] < 0.2
    

def test_select_reports_the_index_gap():
    stat_a = np.array([0.5, 0.4, 0.1])
    stat_b = np.array([10.0, 10.0, 10.0])
    a, gap = O.bandit_select(O.UCB, 3, 0.2, 1, 30, stat_a, stat_b)
    assert a == 0 and abs(gap - 0.1) < 1e-12           # equal counts: the gap is the mean gap
    a, gap = O.bandit_select(O.UCB, 3, 0.2, 1, 30, np.array([0.4, 0.4, 0.1]), stat_b)
    assert a == 0 and gap == 0.0                         # exact tie: lowest index


def test_first_selection_after_the_sweep_uses_ln_of_completed_rounds():
    """Algorithm 2 increments t in the init loop, so the selection after t completed rounds uses ln t.
    Hand case, K = 2, t = 3, mu_hat = (0.5, 0), n = (2, 1):
      index_0 = 0.5 + beta sqrt(2 ln 3 / 2) = 0.5 + 1.04815 beta,  index_1 = beta sqrt(2 ln 3) = 1.48230 beta,
    so arm 1 wins iff beta > 0.5 / 0.43415 = 1.1517.  (With ln(t+1) the boundary would be 1.0252,
    with ln(t-1) it would be 1.4498.)"""
    mu, n = np.array([0.5, 0.0]), np.array([2.0, 1.0])
    assert O.bandit_select(O.UCB, 2, 1.10, 1, 3, mu, n)[0] == 0
    assert O.bandit_select(O.UCB, 2, 1.14, 1, 3, mu, n)[0] == 0
    assert O.bandit_select(O.UCB, 2, 1.16, 1, 3, mu, n)[0] == 1
    assert O.bandit_select(O.UCB, 2, 1.40, 1, 3, mu, n)[0] == 1


# ---------------------------------------------------------------------------------------------
# MetaSD-EXP3 and the uniformly random baseline (the algorithm box "MetaSD-EXP3"; "Rand" in the tables)
# ---------------------------------------------------------------------------------------------
SELECT_POSITION = 0xFFFFFFFF


def select_uniform(seed, sequence, t):
    """The 24-bit uniform that draws a randomised policy's arm: word 2 of the block (sequence, t, 0xFFFFFFFF, 0)."""
    w = O.philox4x32_10((sequence, t, SELECT_POSITION, 0), (seed & 0xFFFFFFFF, seed >> 32))
    return (w[2] >> 8) / float(1 << 24), w[2]


def exp3_probabilities(w, gamma):
    w = np.asarray(w, dtype=np.float64)
    return (1.0 - gamma) * w / w.sum() + gamma / len(w)


def test_exp3_one_round_by_hand():
    """K = 2, gamma = 1/2, first round: p = (1/2, 1/2); reward r on arm a gives w_a = exp(gamma r / (K p_a)) = exp(r / 2)."""
    o = O.OracleMetaSD(O.OracleConfig(max_batch=1, n_drafters=2, vocab=4, bandit=O.EXP3, gamma=0.5))
    a = int(o.select()[0])
    o.update(np.array([a]), np.array([0.8]))
    w = o.stat_a[0]
    assert w.max() == 1.0                                        # kept divided by the largest weight
    ratio = w[a] / w[1 - a]
    assert abs(ratio - np.exp(0.4)) < 1e-14
    p = exp3_probabilities([np.exp(0.4), 1.0] if a == 0 else [1.0, np.exp(0.4)], 0.5)
    assert abs(p[a] - (0.5 * np.exp(0.4) / (np.exp(0.4) + 1.0) + 0.25)) < 1e-15
    assert o.t[0] == 1


def test_exp3_weights_follow_the_closed_form_of_the_importance_weighted_sums():
    """log(w_j / w_i) = (gamma / K) (sum_t r_hat_j - sum_t r_hat_i), with r_hat = r / p_t(a_t) on the played arm."""
    K, gamma, T = 4, 0.2, 300
    o = O.OracleMetaSD(O.OracleConfig(max_batch=1, n_drafters=K, vocab=4, bandit=O.EXP3, gamma=gamma))
    rng = np.random.RandomState(5)
    sums = np.zeros(K)
    w_ref = np.ones(K)
    for t in range(T):
        a = int(o.select()[0])
        p = exp3_probabilities(w_ref, gamma)
        r = float(rng.uniform(0.0, 1.0)) * (0.9 if a == 1 else 0.4)
        sums[a] += r / p[a]
        w_ref = np.exp(gamma / K * (sums - sums.max()))
        o.update(np.array([a]), np.array([r]))
        assert np.allclose(o.stat_a[0], w_ref, rtol=1e-11, atol=0)
    assert sums.argmax() == 1                                     # the arm with the larger rewards collects the weight


def test_exp3_draw_is_the_inverse_cdf_of_its_probabilities_on_the_documented_uniform():
    K, gamma = 5, 0.3
    B = 400
    o = O.OracleMetaSD(O.OracleConfig(max_batch=B, n_drafters=K, vocab=4, bandit=O.EXP3, gamma=gamma, sequence_base=11))
    rng = np.random.RandomState(2)
    o.stat_a[:] = rng.uniform(0.05, 1.0, size=(B, K))
    o.t[:] = rng.randint(0, 50, size=B)
    o.select_seed = 0x1234567890
    arm = o.select()
    for b in range(B):
        u, _ = select_uniform(0x1234567890, 11 + b, int(o.t[b]))
        cdf = np.cumsum(exp3_probabilities(o.stat_a[b], gamma))
        assert arm[b] == min(int(np.searchsorted(cdf, u, side="right")), K - 1)      # smallest i with cdf_i > u
        edges = np.abs(u - cdf[:-1])
        assert abs(o.last_gap[b] - edges.min()) < 1e-15


def test_exp3_with_gamma_one_is_uniform_whatever_the_rewards():
    K, B, T = 4, 64, 200
    o = O.OracleMetaSD(O.OracleConfig(max_batch=B, n_drafters=K, vocab=4, bandit=O.EXP3, gamma=1.0))
    counts = np.zeros(K)
    for t in range(T):
        a = o.select()
        counts += np.bincount(a, minlength=K)
        o.update(a, np.where(a == 0, 1.0, 0.0))                  # arm 0 always wins: irrelevant at gamma = 1
        o.select_seed = t + 1
    chi2 = ((counts - B * T / K) ** 2 / (B * T / K)).sum()
    assert chi2 < 16.27                                          # chi-square, 3 degrees of freedom, p = 0.001


def test_exp3_selection_frequencies_match_its_probabilities():
    K, gamma, B = 3, 0.2, 30000
    o = O.OracleMetaSD(O.OracleConfig(max_batch=B, n_drafters=K, vocab=4, bandit=O.EXP3, gamma=gamma))
    o.stat_a[:] = np.array([1.0, 0.25, 0.5])
    o.select_seed = 99
    counts = np.bincount(o.select(), minlength=K)
    expect = B * exp3_probabilities([1.0, 0.25, 0.5], gamma)
    assert (((counts - expect) ** 2) / expect).sum() < 13.82     # chi-square, 2 degrees of freedom, p = 0.001


def test_exp3_gain_respects_the_bound_of_its_source():
    """Auer et al. (2002), Theorem 3.1: G_max - E[G_EXP3] <= (e - 1) gamma G_max + K ln K / gamma."""
    K, gamma, T, B = 3, 0.15, 600, 64
    means = np.array([0.2, 0.8, 0.5])
    o = O.OracleMetaSD(O.OracleConfig(max_batch=B, n_drafters=K, vocab=4, bandit=O.EXP3, gamma=gamma))
    rng = np.random.RandomState(3)
    gain = np.zeros(B)
    for t in range(T):
        a = o.select()
        r = np.clip(means[a] + rng.uniform(-0.1, 0.1, size=B), 0.0, 1.0)
        gain += r
        o.update(a, r)
        o.select_seed = 1000 + t
    g_max = means.max() * T
    assert gain.mean() >= g_max - ((np.e - 1.0) * gamma * g_max + K * np.log(K) / gamma)
    assert gain.mean() > means.mean() * T + 0.15 * T * (means.max() - means.mean())   # and it does learn


def test_rand_is_floor_of_u_times_k_in_integers_and_uniform():
    K, B = 7, 21000
    o = O.OracleMetaSD(O.OracleConfig(max_batch=B, n_drafters=K, vocab=4, bandit=O.RAND, sequence_base=3))
    o.t[:] = np.arange(B) % 17
    o.select_seed = 42
    arm = o.select()
    for b in range(0, B, 97):
        _, word = select_uniform(42, 3 + b, int(o.t[b]))
        assert arm[b] == ((word >> 8) * K) >> 24
    counts = np.bincount(arm, minlength=K)
    assert (((counts - B / K) ** 2) / (B / K)).sum() < 22.46     # chi-square, 6 degrees of freedom, p = 0.001
    before = o.stat_a.copy()
    o.update(arm, np.ones(B))
    assert np.array_equal(o.stat_a, before) and (o.t == np.arange(B) % 17 + 1).all()   # no statistics, t advances


# ---------------------------------------------------------------------------------------------
# Pure exploration-then-commit with Sequential Halving (the two algorithm boxes of the switching-cost appendix)
# ---------------------------------------------------------------------------------------------
def test_petc_schedule_worked_by_hand_for_four_drafters():
    # K = 4, budget 16: L = 2 phases; phase 0: floor(16 / (4 * 2)) = 2 pulls each of 0,1,2,3;
    # phase 1: floor(16 / (2 * 2)) = 4 pulls each of the two with the larger phase-0 sums; then the winner.
    means = [0.2, 0.9, 0.4, 0.7]
    arms, _, _ = run_bandit(O.PETC, 4, lambda a, t, g: means[a], 30, tau=16)
    assert arms[:8].tolist() == [0, 0, 1, 1, 2, 2, 3, 3]
    assert arms[8:16].tolist() == [1, 1, 1, 1, 3, 3, 3, 3]          # survivors in index order
    assert (arms[16:] == 1).all()                                     # committed to the best


def test_petc_phase_sums_restart_and_only_the_current_phase_counts():
    # drafter 3 wins phase 0 by far (2 x 1.0 against 2 x 0.55) and is slightly worse afterwards (4 x 0.5 against
    # 4 x 0.55): with sums restarted it loses phase 1 to drafter 1; carried over (4.0 against 3.3) it would win
    def reward(a, t, g):
        if a == 3:
            return 1.0 if t < 8 else 0.5
        return [0.1, 0.55, 0.2][a]
    arms, _, orc = run_bandit(O.PETC, 4, reward, 20, tau=16)
    assert sorted(set(arms[8:16].tolist())) == [1, 3]
    assert (arms[16:] == 1).all()
    assert orc.stat_b[0].tolist() == [0.0, 1.0, 0.0, 0.0]             # S after the last halving


@pytest.mark.parametrize("K", [1, 2, 3, 5, 6, 7, 8, 9, 16])
def test_petc_halves_ceil_log2_times_and_spends_at_most_its_budget(K):
    budget = 12 * K
    L = math.ceil(math.log2(K)) if K > 1 else 0
    rng_means = np.random.RandomState(K).permutation(np.linspace(0.1, 0.9, K)) if K > 1 else np.array([0.5])
    arms, _, orc = run_bandit(O.PETC, K, lambda a, t, g: rng_means[a] + 0.01 * g.rand(), budget + 25, tau=budget)
    # exploration length: sum over phases of n_r |S_r| with |S_{r+1}| = ceil(|S_r| / 2)
    size, spent, sizes = K, 0, []
    for _ in range(L):
        sizes.append(size)
        spent += (budget // (size * L)) * size
        size = (size + 1) // 2
    assert size == 1 and spent <= budget
    tail = arms[spent:]
    assert (tail == tail[0]).all()                                    # one drafter for every later round
    assert int(orc.stat_b[0].sum()) == 1 and orc.stat_b[0][tail[0]] == 1.0
    # inside phase r exactly |S_r| distinct drafters are played, each the same number of times
    pos = 0
    for s in sizes:
        n = budget // (s * L)
        block = arms[pos:pos + n * s]
        values, counts = np.unique(block, return_counts=True)
        assert len(values) == s and (counts == n).all()
        # the means are far apart next to the noise: S_r is exactly the |S_r| best drafters
        assert set(values.tolist()) == set(np.argsort(-rng_means)[:s].tolist())
        pos += n * s
    # with well separated means the best drafter survives
    assert tail[0] == int(np.argmax(rng_means))


def test_petc_keeps_the_lower_index_on_equal_sums_and_pulls_at_least_once():
    arms, _, orc = run_bandit(O.PETC, 4, lambda a, t, g: 0.5, 12, tau=1)     # budget too small: n_r = 1
    assert arms[:4].tolist() == [0, 1, 2, 3] and arms[4:6].tolist() == [0, 1]
    assert (arms[6:] == 0).all()


def test_sequential_halving_error_rate_respects_the_bound_the_paper_quotes():
    # P(wrong survivor) <= 3 log2(K) exp(-T / (8 H2 log2 K)), H2 = max_i i / Delta_i^2 (gaps sorted increasingly)
    means = np.array([0.9, 0.5, 0.45, 0.4])
    K, T = 4, 1600
    gaps = np.sort(means.max() - means)[1:]                                  # Delta_(2) <= ... <= Delta_(K)
    H2 = max((i + 2) / gaps[i] ** 2 for i in range(K - 1))
    bound = 3 * math.log2(K) * math.exp(-T / (8 * H2 * math.log2(K)))
    assert bound < 0.02                                                      # not a vacuous statement
    wrong, runs = 0, 150
    for s in range(runs):
        arms, _, _ = run_bandit(O.PETC, K, lambda a, t, g: float(g.rand() < means[a]), T + 1, tau=T, seed=s)
        wrong += int(arms[-1] != 0)
    assert wrong / runs <= bound + 3 * math.sqrt(max(bound * (1 - bound), 1e-4) / runs)
    assert wrong / runs < 0.05                                               # and it does find the best drafter
