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
