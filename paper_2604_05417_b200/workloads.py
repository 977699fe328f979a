"""Seeded synthetic inputs for the draft-verify round: logits and drafted tokens.

This module only *makes inputs*.  It holds none of the method's arithmetic (no
softmax, no accept test, no reward, no bandit): the CUDA path and the CPU oracle
both receive the exact bytes produced here.

Recipe (stand-in for the paper's Vicuna-7B target + task-specialised drafters,
whose weights and datasets are not available):

* target[b, j, v] = round(dtype, 3 * z - s_b * ln(rank(v))),  z ~ N(0, 1) i.i.d.
  (a Zipf(s_b) log-prior over token ids plus Gaussian noise of std 3).  rank(v) = v + 1 by default (the likely
  tokens have the small ids, as in a frequency-sorted vocabulary); ``order="reversed"`` puts them at the END of the
  vocabulary and ``order="shuffled"`` spreads them by a seeded permutation, so that an implementation that walks the
  vocabulary in id order cannot profit from where the mass sits.
* draft[b, j, v]  = round(dtype, float(target[b, j, v]) + sigma * z'),  z' ~ N(0, 1)
  where sigma is the noise level of the drafter that produced the block; a
  better-aligned drafter has a smaller sigma.
* drafted tokens: x_j = argmax_v(draft[b, j, v] / T + Gumbel noise), i.e. a
  sample from the drafter's own distribution; greedy decoding (T = 0) drafts
  argmax_v draft[b, j, v].

The five named workloads are the configurations the benchmark specification
lists; ``Workload.scaled`` shrinks one for parity tests.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Optional, Tuple

import numpy as np
import torch

_TORCH_DTYPE = {"bf16": torch.bfloat16, "fp32": torch.float32}


@dataclass(frozen=True)
class Workload:
    name: str
    B: int                      # independent sequences
    N: int                      # drafters (the paper's K)
    k: int                      # drafted tokens per round (the paper's N_max)
    V: int                      # vocabulary
    rounds: int
    temperature: float          # 0 => greedy
    dtype: str                  # "bf16" | "fp32"
    bandit: str                 # "ucb" | "ducb" | "swucb"
    sigmas: Tuple[float, ...]
    schedule: str = "fixed"     # "fixed" | "permute" | "task" | "sine"
    period: int = 100           # permute: re-draw period; sine: see sigma_table
    zipf: Tuple[float, ...] = (1.1,)   # exponent of task (b mod len(zipf))
    beta: float = 0.01
    gamma: float = 0.975
    tau: int = 50
    order: str = "rank"         # which token ids are the likely ones: "rank" | "reversed" | "shuffled"

    def scaled(self, **kw) -> "Workload":
        return replace(self, **kw)

    @property
    def torch_dtype(self):
        return _TORCH_DTYPE[self.dtype]

    @property
    def bytes_per_round(self) -> int:
        """Logit bytes one round reads: B * (2k + 1) * V * sizeof(logit)."""
        return self.B * (2 * self.k + 1) * self.V * (2 if self.dtype == "bf16" else 4)


WORKLOADS = {
    "cfg1_tiny": Workload("cfg1_tiny", B=1, N=3, k=4, V=32000, rounds=200, temperature=1.0,
                          dtype="bf16", bandit="ucb", sigmas=(0.5, 1.5, 3.0)),
    "cfg2_nonstationary": Workload("cfg2_nonstationary", B=64, N=5, k=5, V=32000, rounds=1000,
                                   temperature=1.0, dtype="bf16", bandit="ducb",
                                   sigmas=(0.3, 0.8, 1.5, 2.5, 4.0), schedule="permute", period=100),
    "cfg3_tasks": Workload("cfg3_tasks", B=256, N=8, k=7, V=128256, rounds=500, temperature=0.7,
                           dtype="bf16", bandit="ucb",
                           sigmas=tuple(0.2 + i * 3.8 / 7 for i in range(8)), schedule="task",
                           zipf=(0.9, 0.9 + 0.5 / 3, 0.9 + 1.0 / 3, 1.4)),
    "cfg4_greedy": Workload("cfg4_greedy", B=512, N=4, k=8, V=152064, rounds=300, temperature=0.0,
                            dtype="bf16", bandit="ucb", sigmas=(0.1, 0.5, 1.0, 2.0)),
    "cfg5_fp32_stress": Workload("cfg5_fp32_stress", B=1024, N=8, k=5, V=128256, rounds=200,
                                 temperature=1.0, dtype="fp32", bandit="ucb",
                                 sigmas=(1.5,) * 8, schedule="sine", period=50),
}


def _seed(*parts: int) -> int:
    """Mix integers into one 63-bit generator seed (splitmix64 steps)."""
    x = 0x9E3779B97F4A7C15
    for p in parts:
        x = (x ^ (int(p) & 0xFFFFFFFFFFFFFFFF)) & 0xFFFFFFFFFFFFFFFF
        x = (x + 0x9E3779B97F4A7C15) & 0xFFFFFFFFFFFFFFFF
        x = ((x ^ (x >> 30)) * 0xBF58476D1CE4E5B9) & 0xFFFFFFFFFFFFFFFF
        x = ((x ^ (x >> 27)) * 0x94D049BB133111EB) & 0xFFFFFFFFFFFFFFFF
        x = x ^ (x >> 31)
    return x & 0x7FFFFFFFFFFFFFFF


class RoundGenerator:
    """Makes the inputs of round t for a workload, on any torch device."""

    TARGET, DRAFT, TOKENS, SIGMA = 1, 2, 3, 4

    def __init__(self, wl: Workload, device="cpu", seed: int = 0, chunk_sequences: Optional[int] = None):
        self.wl = wl
        self.device = torch.device(device)
        self.seed = seed
        if chunk_sequences is None:
            # bound the fp32 temporaries to about 1 GiB
            per_seq = (wl.k + 1) * wl.V * 4 * 3
            chunk_sequences = max(1, min(wl.B, (1 << 30) // per_seq))
        self.chunk = chunk_sequences
        v = torch.arange(1, wl.V + 1, dtype=torch.float32, device=self.device)
        if wl.order == "reversed":
            v = v.flip(0)
        elif wl.order == "shuffled":
            perm = np.random.RandomState(_seed(seed, 77) % (2 ** 32)).permutation(wl.V)
            v = v[torch.from_numpy(perm).to(self.device)]
        elif wl.order != "rank":
            raise ValueError(wl.order)
        self._log_rank = torch.log(v)
        zipf = np.asarray([wl.zipf[b % len(wl.zipf)] for b in range(wl.B)], dtype=np.float32)
        self._zipf = torch.from_numpy(zipf).to(self.device)

    def _gen(self, *parts):
        g = torch.Generator(device=self.device)
        g.manual_seed(_seed(self.seed, *parts))
        return g

    # -- drafter noise levels ------------------------------------------------
    def sigma_table(self, t: int) -> np.ndarray:
        """sigma[b, i]: noise level of drafter i on sequence b in round t."""
        wl = self.wl
        base = np.asarray(wl.sigmas, dtype=np.float64)
        if wl.schedule == "fixed":
            return np.tile(base, (wl.B, 1))
        if wl.schedule == "permute":
            rng = np.random.RandomState(_seed(self.seed, self.SIGMA, t // wl.period) % (2 ** 32))
            return np.stack([base[rng.permutation(wl.N)] for _ in range(wl.B)])
        if wl.schedule == "task":
            n_task = len(wl.zipf)
            out = np.empty((wl.B, wl.N))
            for b in range(wl.B):
                task = b % n_task
                out[b] = [base[(i + 2 * task) % wl.N] for i in range(wl.N)]
            return out
        if wl.schedule == "sine":
            i = np.arange(wl.N)
            row = 1.5 + 1.2 * np.sin(2.0 * math.pi * t / wl.period + i)
            return np.tile(row, (wl.B, 1))
        raise ValueError(wl.schedule)

    def best_arm(self, t: int) -> np.ndarray:
        return self.sigma_table(t).argmin(axis=1)

    # -- logits ---------------------------------------------------------------
    def target_logits(self, t: int) -> torch.Tensor:
        wl = self.wl
        out = torch.empty((wl.B, wl.k + 1, wl.V), dtype=wl.torch_dtype, device=self.device)
        for b0 in range(0, wl.B, self.chunk):
            b1 = min(wl.B, b0 + self.chunk)
            z = torch.randn((b1 - b0, wl.k + 1, wl.V), dtype=torch.float32, device=self.device,
                            generator=self._gen(self.TARGET, t, b0))
            z.mul_(3.0)
            z.sub_(self._zipf[b0:b1, None, None] * self._log_rank[None, None, :])
            out[b0:b1] = z.to(wl.torch_dtype)
        return out

    def draft_logits(self, t: int, target: torch.Tensor, sigma_per_sequence, drafter_tag: int = 0) -> torch.Tensor:
        """Draft rows of the drafter whose noise level on sequence b is sigma_per_sequence[b]."""
        wl = self.wl
        sig = torch.as_tensor(np.asarray(sigma_per_sequence, dtype=np.float32), device=self.device)
        out = torch.empty((wl.B, wl.k, wl.V), dtype=wl.torch_dtype, device=self.device)
        for b0 in range(0, wl.B, self.chunk):
            b1 = min(wl.B, b0 + self.chunk)
            z = torch.randn((b1 - b0, wl.k, wl.V), dtype=torch.float32, device=self.device,
                            generator=self._gen(self.DRAFT, t, b0, drafter_tag))
            z.mul_(sig[b0:b1, None, None])
            z.add_(target[b0:b1, : wl.k].to(torch.float32))
            out[b0:b1] = z.to(wl.torch_dtype)
        return out

    def draft_tokens(self, t: int, draft: torch.Tensor, drafter_tag: int = 0) -> torch.Tensor:
        """Tokens the drafter proposes: a Gumbel-max draw at temperature T, or argmax when greedy."""
        wl = self.wl
        out = torch.empty((wl.B, wl.k), dtype=torch.int32, device=self.device)
        for b0 in range(0, wl.B, self.chunk):
            b1 = min(wl.B, b0 + self.chunk)
            x = draft[b0:b1].to(torch.float32)
            if wl.temperature > 0:
                u = torch.rand(x.shape, dtype=torch.float32, device=self.device,
                               generator=self._gen(self.TOKENS, t, b0, drafter_tag))
                u.clamp_(min=1e-20, max=1.0 - 1e-7)
                x = x / wl.temperature - torch.log(-torch.log(u))
            out[b0:b1] = torch.argmax(x, dim=-1).to(torch.int32)
        return out

    # -- whole rounds -----------------------------------------------------------
    def gathered_round(self, t: int, arm) -> dict:
        """Inputs of round t when sequence b plays arm[b]: draft rows gathered by arm."""
        arm = np.asarray(arm, dtype=np.int64)
        sig = self.sigma_table(t)[np.arange(self.wl.B), arm]
        target = self.target_logits(t)
        draft = self.draft_logits(t, target, sig)
        tokens = self.draft_tokens(t, draft)
        return dict(target=target, draft=draft, tokens=tokens, sigma=sig)

    def table_round(self, t: int) -> dict:
        """Inputs of round t for every drafter: N draft tensors and an [N, B, k] token table."""
        sig = self.sigma_table(t)
        target = self.target_logits(t)
        drafts, tokens = [], []
        for i in range(self.wl.N):
            d = self.draft_logits(t, target, sig[:, i], drafter_tag=i + 1)
            drafts.append(d)
            tokens.append(self.draft_tokens(t, d, drafter_tag=i + 1))
        return dict(target=target, drafts=drafts, tokens=torch.stack(tokens), sigma=sig)
