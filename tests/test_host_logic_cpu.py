"""CPU checks of the host-side pieces around the library: the input generator's vocabulary orders, the reward-study
bookkeeping and the benchmark's lookup of committed DRAM-traffic captures."""
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

from paper_2604_05417_b200.workloads import RoundGenerator, Workload


def small(order):
    return Workload(name="t", B=4, N=2, k=2, V=4096, rounds=1, temperature=1.0, dtype="fp32", bandit="ucb",
                    sigmas=(0.5, 2.0), order=order)


def test_vocabulary_orders_move_the_likely_tokens():
    """rank: the prior falls with the token id; reversed: it rises; shuffled: a seeded permutation of the same prior.
    The Gaussian part of the logits is the same draw in all three (same seeds), so only the prior moves."""
    t = {o: RoundGenerator(small(o), seed=3).target_logits(0).double() for o in ("rank", "reversed", "shuffled")}
    mean = {o: x.mean(dim=(0, 1)) for o, x in t.items()}
    V = 4096
    head, tail = slice(0, V // 8), slice(V - V // 8, V)
    assert mean["rank"][head].mean() > mean["rank"][tail].mean() + 3.0
    assert mean["reversed"][tail].mean() > mean["reversed"][head].mean() + 3.0
    assert abs(mean["shuffled"][head].mean() - mean["shuffled"][tail].mean()) < 1.0
    # the prior of "reversed" is the prior of "rank" read backwards; "shuffled" holds the same values in another order
    prior = lambda o: RoundGenerator(small(o), seed=3)._log_rank
    assert torch.equal(prior("reversed"), prior("rank").flip(0))
    assert torch.equal(prior("shuffled").sort().values, prior("rank").sort().values)
    assert not torch.equal(prior("shuffled"), prior("rank"))
    assert torch.equal(prior("shuffled"), RoundGenerator(small("shuffled"), seed=3)._log_rank)   # seeded


def test_running_moments_and_table_format():
    from paper_2604_05417_b200 import study
    rng = np.random.RandomState(0)
    x = rng.rand(1000)
    m = study.RunningMoments()
    for part in np.array_split(x, 7):
        m.add(part)
    assert m.n == 1000 and abs(m.mean - x.mean()) < 1e-12 and abs(m.var - x.var()) < 1e-12
    text = study.format_table([dict(a=1, b=0.5)], ["a", "b"])
    assert text.splitlines()[0] == "| a | b |" and text.splitlines()[-1] == "| 1 | 0.5000 |"


def test_feedback_signal_on_the_papers_reward_statistics_table():
    """Theorem 1's feedback signal R = Delta^2 / max(Var[r_i], Var[r_best]) evaluated on the statistics the paper prints
    for its five drafters: BD gives every suboptimal drafter the stronger signal, which is the paper's reading of that
    table.  The two figures for the Russian drafter are worked out by hand from the printed numbers:
    BD (0.488 - 0.294)^2 / 0.044 = 0.855, BE (0.232 - 0.099)^2 / 0.093 = 0.190."""
    import os
    from paper_2604_05417_b200 import study
    rows = []
    with open(os.path.join(os.path.dirname(__file__), "golden", "reward_statistics_table.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, mean_be, mean_bd, var_be, var_bd, zero = line.split()
            # the study's rows are keyed by noise level, smallest = best: give the best drafter (first line) level 0
            rows.append(dict(name=name, sigma=float(len(rows)), mean_be=float(mean_be), mean_bd=float(mean_bd),
                             var_be=float(var_be), var_bd=float(var_bd)))
    rows = study.add_feedback_signal(rows)
    assert rows[0]["name"] == "Ja" and np.isnan(rows[0]["signal_bd"]) and np.isnan(rows[0]["signal_be"])
    assert all(r["signal_bd"] > r["signal_be"] > 0 for r in rows[1:])
    ru = rows[1]
    assert abs(ru["signal_bd"] - 0.855) < 1e-3 and abs(ru["signal_be"] - 0.190) < 1e-3
    assert study.feedback_signal(0.5, 0.0, 0.25, 0.0) == float("inf")          # rewards that do not vary
    # the larger of the two variances counts, whichever drafter it belongs to
    assert study.feedback_signal(0.5, 0.01, 0.3, 0.04) == study.feedback_signal(0.5, 0.04, 0.3, 0.01) == 0.2 ** 2 / 0.04


def test_constant_alignment_rows_have_the_prescribed_alignment():
    """The rows of the reward pins: 1 - d_TV(p_j, q_j) is the requested alpha, and the drafted token is the drafter's
    only token (float64 softmax of the generated logits, typed out here)."""
    from paper_2604_05417_b200 import study
    alphas = np.array([[0.3, 0.9, 0.0], [1.0, 0.5, 0.25]])
    target, draft, tokens = study.constant_alignment_rows(2, 3, 64, alphas, dtype=torch.float32, device="cpu", seed=1)
    p = torch.softmax(target[:, :3].double(), dim=-1)
    q = torch.softmax(draft.double(), dim=-1)
    tv = 0.5 * (p - q).abs().sum(-1)
    assert np.allclose(1.0 - tv.numpy(), alphas, atol=1e-6)
    picked = torch.gather(q, 2, tokens.long().unsqueeze(-1)).squeeze(-1)
    assert torch.allclose(picked, torch.ones_like(picked))


def test_traffic_lookup_matches_only_the_captured_kernel_variant():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.known_traffic("staged/bf16/t0/s0/keep0", "cfg4_greedy") > 2.6e9      # above the algorithmic bytes
    assert bench.known_traffic("staged/bf16/t0/s0/keep0", "cfg1_tiny") is None
    assert bench.known_traffic("bulk/bf16/t0/s0/keep0", "cfg4_greedy") is None        # another variant: no stale figure
    assert bench.known_traffic("staged/bf16/t1024/s6/keep0", "cfg4_greedy") is None
