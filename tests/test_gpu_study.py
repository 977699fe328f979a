"""The paper's statements about its two rewards, checked THROUGH the CUDA path on rows of prescribed alignment.

Sec. 2.3 of the paper: with i.i.d. per-position alignments alpha_j = 1 - d_TV(p_j, q_j) of mean alpha,
  * E[r^BD] = alpha and Var[r^BD] <= 1 / (4 N_max)                      (lemma "BD reward statistics"),
  * E[r^BE] = (alpha - alpha^(N+1)) / ((1 - alpha) N)                   (lemma "BE reward statistics"),
  * E[r^BE] / E[r^BD] = (1 - alpha^N) / (N (1 - alpha))                 (the lemma relating the two rewards).
The expected values on the right are closed forms typed in here; nothing on the CPU recomputes the round.
"""
import numpy as np
import pytest
import torch

from paper_2604_05417_b200 import binding as M
from paper_2604_05417_b200 import study

pytestmark = pytest.mark.gpu


def run_rounds(alphas_of_round, B, k, V, dtype, rounds, reward):
    msd = M.MetaSD(B, 1, k, V, dtype=dtype, reward=reward)
    bd, be, lib = [], [], []
    for t in range(rounds):
        target, draft, tokens = study.constant_alignment_rows(B, k, V, alphas_of_round(t), dtype=M_TORCH[dtype], seed=100 + t)
        res = msd.verify(target, draft, tokens, 1.0, 2024, want_diag=True)
        r_bd, r_be = study.both_rewards(res, k)
        bd.append(r_bd)
        be.append(r_be)
        lib.append(res.reward.cpu().numpy().astype(np.float64))
    assert msd.last_status() == 0
    msd.close()
    return np.concatenate(bd), np.concatenate(be), np.concatenate(lib)


M_TORCH = {"bf16": torch.bfloat16, "fp32": torch.float32}


@pytest.mark.parametrize("alpha", [0.3, 0.6, 0.85])
def test_be_to_bd_ratio_on_rows_of_constant_alignment(alpha):
    B, k, V, rounds = 2048, 5, 256, 10
    const = lambda t: np.full((B, k), alpha)
    bd, be, lib_bd = run_rounds(const, B, k, V, "fp32", rounds, M.REWARD_BD)
    _, be2, lib_be = run_rounds(const, B, k, V, "fp32", rounds, M.REWARD_BE)
    np.testing.assert_allclose(bd, alpha, atol=1e-5)                       # E[r^BD] = alpha (here: every round)
    np.testing.assert_allclose(lib_bd, bd, atol=2e-6)                      # the library's reward is that BD value
    assert np.array_equal(be, be2) and np.allclose(lib_be, be, atol=1e-7)  # ... and N_acc / k under the BE setting
    n = be.size
    mean_nacc = (alpha - alpha ** (k + 1)) / (1 - alpha)
    var_nacc = alpha * (1 - (2 * k + 1) * alpha ** k + (2 * k + 1) * alpha ** (k + 1) - alpha ** (2 * k + 1)) / (1 - alpha) ** 2
    se = np.sqrt(var_nacc / n) / k
    assert abs(be.mean() - mean_nacc / k) < 4.5 * se
    ratio = be.mean() / bd.mean()
    assert abs(ratio - (1 - alpha ** k) / (k * (1 - alpha))) < 4.5 * se / alpha
    assert abs(be.var() - var_nacc / k ** 2) < 0.1 * var_nacc / k ** 2     # the BE variance follows its closed form


@pytest.mark.parametrize("law", ["two_point", "beta"])
def test_bd_variance_stays_under_its_bound(law):
    B, k, V, rounds = 2048, 4, 200, 8
    rng = np.random.RandomState(7)
    if law == "two_point":      # alpha_j in {0, 1} with equal odds: the largest variance a [0, 1] variable can have
        draw = lambda t: rng.randint(0, 2, size=(B, k)).astype(np.float64)
        var_one = 0.25
    else:
        draw = lambda t: rng.beta(2.0, 2.0, size=(B, k))
        var_one = 0.05
    bd, be, lib = run_rounds(draw, B, k, V, "fp32", rounds, M.REWARD_BD)
    assert abs(bd.mean() - 0.5) < 0.01
    bound = 1.0 / (4 * k)
    assert bd.var() <= bound * 1.03
    assert abs(bd.var() - var_one / k) < 0.05 * var_one / k               # the mean of k i.i.d. alignments
    assert be.var() > bd.var()                                             # the paper's point: BE is the noisier reward


def test_best_arm_ratio_and_histogram_of_a_short_bandit_run():
    wl = study.WORKLOADS["cfg2_nonstationary"].scaled(B=16, V=8192, period=40)
    out = study.bandit_run(wl, rounds=60, reward=M.REWARD_BD, bandit="ducb", window=20)
    assert out["status"] == 0 and sum(out["arm_histogram"]) == 60 * 16
    assert len(out["best_arm_ratio_by_window"]) == 3 and 0.0 <= out["best_arm_ratio"] <= 1.0
    assert out["best_arm_ratio_by_window"][1] > 1.0 / wl.N                 # better than guessing once the sweep is over
    assert 0 < out["mean_bd"] <= 1 and 1.0 <= out["block_efficiency"] <= wl.k + 1
    rows = study.drafter_reward_statistics(wl, rounds=2)
    assert len(rows) == wl.N and all(r["var_be"] >= 0 for r in rows)
    # Theorem 1's feedback signal of every drafter against the best (the smallest noise level): BD's is the stronger
    assert np.isnan(rows[0]["signal_bd"]) and all(r["signal_bd"] > r["signal_be"] > 0 for r in rows[1:])
