"""Synthetic counterpart of the paper's reward study: block divergence (BD) against block efficiency (BE).

The paper compares its two alignment rewards on real drafters: their means and variances, how often BE is exactly
zero, and how quickly a bandit fed with either reward settles on the best drafter (Sec. 2.3: the BE definition and
the lemma that relates E[r^BE] to E[r^BD]; Theorem 1's feedback signal; the reward-statistics table; the best-arm-ratio
figure).  This module
produces the same quantities for the synthetic workloads, whose generator knows which drafter is best for every
sequence in every round.  Every round runs through the library (C ABI, CUDA kernels); what is computed here is
bookkeeping on its outputs: means, variances, counts.

    python -m paper_2604_05417_b200.study --workload cfg2_nonstationary --rounds 300 [--bandits ucb,ducb]

prints one JSON object and a table.
"""
from __future__ import annotations

import argparse
import json
from typing import Dict, List, Sequence

import numpy as np
import torch

from . import binding as M
from .workloads import WORKLOADS, RoundGenerator, Workload


class RunningMoments:
    """Mean and (population) variance of a stream of arrays."""

    def __init__(self):
        self.n, self.s1, self.s2 = 0, 0.0, 0.0

    def add(self, x):
        x = np.asarray(x, dtype=np.float64)
        self.n += x.size
        self.s1 += float(x.sum())
        self.s2 += float((x * x).sum())

    @property
    def mean(self):
        return self.s1 / self.n if self.n else float("nan")

    @property
    def var(self):
        return max(self.s2 / self.n - self.mean ** 2, 0.0) if self.n else float("nan")


def both_rewards(res: M.VerifyResult, k: int):
    """(r_BD, r_BE) per sequence from one round's outputs: BD = 1 - mean_j d_TV (from the per-position diagnostics),
    BE = N_acc / k."""
    D = res.diag_fields()[2].cpu().numpy().astype(np.float64)
    return 1.0 - D.mean(axis=1), res.accepted_len.cpu().numpy().astype(np.float64) / k


def drafter_reward_statistics(wl: Workload, rounds: int, device=0, seed: int = 0, lib_seed: int = 99) -> List[dict]:
    """Plays every drafter in turn for `rounds` rounds on all sequences (no bandit: the rows are gathered for a
    fixed drafter index) and returns, per NOISE LEVEL of the drafter (the generator's alignment knob; which drafter
    has which level differs between sequences and over time): mean and variance of BD and BE, the share of rounds
    with BE = 0, the mean accepted length and the block efficiency 1 + E[N_acc]."""
    dev = torch.device("cuda", device)
    gen = RoundGenerator(wl, device=dev, seed=seed)
    acc: Dict[float, dict] = {}
    for i in range(wl.N):
        msd = M.MetaSD(wl.B, 1, wl.k, wl.V, dtype=wl.dtype, bandit="ucb", device=device)
        for t in range(rounds):
            rd = gen.gathered_round(t, np.full(wl.B, i))
            res = msd.verify(rd["target"], rd["draft"], rd["tokens"], wl.temperature, lib_seed, want_diag=True)
            r_bd, r_be = both_rewards(res, wl.k)
            level = np.round(np.asarray(rd["sigma"], dtype=np.float64), 3)
            for value in np.unique(level):
                pick = level == value
                a = acc.setdefault(float(value), dict(bd=RunningMoments(), be=RunningMoments(), zero=0))
                a["bd"].add(r_bd[pick])
                a["be"].add(r_be[pick])
                a["zero"] += int((r_be[pick] == 0).sum())
        msd.close()
    rows = []
    for value in sorted(acc):
        bd, be = acc[value]["bd"], acc[value]["be"]
        rows.append(dict(sigma=value, samples=be.n, mean_bd=bd.mean, var_bd=bd.var, mean_be=be.mean, var_be=be.var,
                         be_zero_ratio=acc[value]["zero"] / be.n, mean_accepted=be.mean * wl.k,
                         block_efficiency=1.0 + be.mean * wl.k))
    return add_feedback_signal(rows)


def feedback_signal(mean_best: float, var_best: float, mean_i: float, var_i: float) -> float:
    """The bandit feedback signal of a suboptimal drafter i under one reward design (the equation of Theorem 1):
    R = Delta_i^2 / max(Var[r_i], Var[r_best]) with Delta_i = mu_best - mu_i.  Infinite when neither reward varies."""
    gap, spread = mean_best - mean_i, max(var_i, var_best)
    if spread > 0.0:
        return gap * gap / spread
    return float("inf") if gap != 0.0 else float("nan")


def add_feedback_signal(rows: List[dict]) -> List[dict]:
    """Adds `signal_bd` and `signal_be` to the rows of drafter_reward_statistics: the feedback signal of every
    drafter against the best one, which is the row with the smallest noise level (the generator's best drafter;
    its own signal is NaN)."""
    best = min(rows, key=lambda r: r["sigma"])
    for r in rows:
        if r is best:
            r["signal_bd"] = r["signal_be"] = float("nan")
        else:
            r["signal_bd"] = feedback_signal(best["mean_bd"], best["var_bd"], r["mean_bd"], r["var_bd"])
            r["signal_be"] = feedback_signal(best["mean_be"], best["var_be"], r["mean_be"], r["var_be"])
    return rows


def bandit_run(wl: Workload, rounds: int, reward: int, bandit: str, device=0, seed: int = 0, lib_seed: int = 99,
               window: int = 25) -> dict:
    """`rounds` rounds of the workload with the bandit choosing the drafter (pointer-table mode) and `reward`
    (M.REWARD_BD or M.REWARD_BE) fed back.  Returns the best-arm ratio per round (share of sequences that played the
    drafter with the smallest noise level that round) and per window of rounds, the arm histogram, means and
    variances of both rewards, the BE zero ratio and the block efficiency 1 + E[N_acc]."""
    dev = torch.device("cuda", device)
    gen = RoundGenerator(wl, device=dev, seed=seed)
    msd = M.MetaSD(wl.B, wl.N, wl.k, wl.V, dtype=wl.dtype, bandit=bandit, beta=wl.beta, gamma=wl.gamma, window=wl.tau,
                   reward=reward, device=device)
    ratio = np.zeros(rounds)
    hist = np.zeros(wl.N, dtype=np.int64)
    bd, be, zero, acc = RunningMoments(), RunningMoments(), 0, RunningMoments()
    for t in range(rounds):
        arm = msd.select().cpu().numpy()
        rd = gen.table_round(t)
        table = M.pointer_table(rd["drafts"])
        res = msd.verify(rd["target"], None, rd["tokens"], wl.temperature, lib_seed, drafter_table=table,
                         token_arm_stride=wl.B * wl.k, want_diag=True)
        r_bd, r_be = both_rewards(res, wl.k)
        bd.add(r_bd)
        be.add(r_be)
        zero += int((r_be == 0).sum())
        acc.add(res.accepted_len.cpu().numpy())
        ratio[t] = float((arm == gen.best_arm(t)).mean())
        hist += np.bincount(arm, minlength=wl.N)
    status = msd.last_status()
    msd.close()
    n_win = (rounds + window - 1) // window
    return dict(workload=wl.name, bandit=bandit, reward="BD" if reward == M.REWARD_BD else "BE", rounds=rounds,
                best_arm_ratio=float(ratio.mean()),
                best_arm_ratio_by_window=[float(ratio[w * window:(w + 1) * window].mean()) for w in range(n_win)],
                window=window, arm_histogram=hist.tolist(), mean_bd=bd.mean, var_bd=bd.var, mean_be=be.mean,
                var_be=be.var, be_zero_ratio=zero / be.n, block_efficiency=1.0 + acc.mean, status=status)


def constant_alignment_rows(B: int, k: int, V: int, alphas, dtype=torch.float32, device="cuda", seed: int = 0):
    """Rows with a prescribed alignment 1 - d_TV(p_j, q_j) = alphas[b, j]: the drafter puts all its mass on one
    token x (which is therefore the drafted token), the target gives x the probability alpha and a second token the
    rest, so the accept test passes with probability alpha, independently per position (the paper's Assumption 1).
    Returns target [B, k+1, V], draft [B, k, V], tokens [B, k]."""
    g = torch.Generator(device="cpu").manual_seed(seed)
    alphas = torch.as_tensor(np.asarray(alphas, dtype=np.float64)).reshape(B, k)
    x = torch.randint(0, V, (B, k), generator=g)
    y = (x + 1 + torch.randint(0, V - 1, (B, k), generator=g)) % V           # a second token, different from x
    neg = -1.0e4                                                              # probability exactly 0 after the softmax
    target = torch.full((B, k + 1, V), neg, dtype=torch.float64)
    draft = torch.full((B, k, V), neg, dtype=torch.float64)
    bi, ji = torch.meshgrid(torch.arange(B), torch.arange(k), indexing="ij")
    tiny = 1e-300
    target[bi, ji, x] = torch.log(alphas.clamp_min(tiny))
    target[bi, ji, y] = torch.log((1.0 - alphas).clamp_min(tiny))
    target[:, k, 0] = 0.0                                                     # the bonus row: any distribution
    draft[bi, ji, x] = 0.0
    return (target.to(dtype).to(device), draft.to(dtype).to(device), x.to(torch.int32).to(device))


def format_table(rows: Sequence[Dict], columns: Sequence[str]) -> str:
    out = ["| " + " | ".join(columns) + " |", "|" + "---|" * len(columns)]
    for r in rows:
        out.append("| " + " | ".join(("%.4f" % r[c]) if isinstance(r[c], float) else str(r[c]) for c in columns) + " |")
    return "\n".join(out)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="cfg2_nonstationary", choices=sorted(WORKLOADS))
    ap.add_argument("--rounds", type=int, default=300)
    ap.add_argument("--batch", type=int, default=0)
    ap.add_argument("--bandits", default="ucb,ducb")
    ap.add_argument("--window", type=int, default=25)
    ap.add_argument("--drafter-rounds", type=int, default=10, help="rounds per drafter of the reward-statistics table")
    args = ap.parse_args()
    wl = WORKLOADS[args.workload]
    if args.batch:
        wl = wl.scaled(B=args.batch)
    report = {"workload": wl.name, "B": wl.B, "rounds": args.rounds}
    report["drafters"] = drafter_reward_statistics(wl, args.drafter_rounds)
    report["runs"] = [bandit_run(wl, args.rounds, reward, bandit, window=args.window)
                      for bandit in args.bandits.split(",") for reward in (M.REWARD_BD, M.REWARD_BE)]
    print(json.dumps(report))
    print(format_table(report["drafters"], ["sigma", "samples", "mean_bd", "var_bd", "mean_be", "var_be", "be_zero_ratio",
                                            "block_efficiency", "signal_bd", "signal_be"]))
    print(format_table(report["runs"], ["bandit", "reward", "best_arm_ratio", "mean_bd", "var_bd", "mean_be", "var_be",
                                        "be_zero_ratio", "block_efficiency"]))
    for r in report["runs"]:
        print("%s/%s best-arm ratio per %d rounds: %s" % (r["bandit"], r["reward"], r["window"],
                                                         " ".join("%.2f" % v for v in r["best_arm_ratio_by_window"])))


if __name__ == "__main__":
    main()
