"""ctypes binding of the float64 CPU oracle (``metasd_oracle.c``).

TEST INFRASTRUCTURE, NOT THE PRODUCT.  Only tests, the smoke check and the
benchmark's CPU-baseline leg import this module; the CUDA path never does and
shares no code with it.  The C file is compiled with gcc on first use.

Notation follows the paper: K drafters (arms), k = N_max drafted tokens per
round, p / q = target / drafter distributions over a vocabulary of V tokens.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "metasd_oracle.c")
_LIB = os.path.join(_HERE, "libmetasd_oracle.so")

DTYPE_BF16, DTYPE_FP32 = 0, 1
UCB, DUCB, SWUCB, EXP3, RAND, PETC = 0, 1, 2, 3, 4, 5
REWARD_BD, REWARD_BE = 0, 1
STATUS_NONFINITE, STATUS_TOKEN_OOR, STATUS_Q_ZERO = 1, 2, 4

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (plain -O2, no fast-math, no FMA contraction)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
             _SRC, "-o", tmp, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.msdo_uniform24.restype = C.c_double
        _lib.msdo_uniform24.argtypes = [C.c_uint32]
        _lib.msdo_tv_distance.restype = C.c_double
        _lib.msdo_argmax.restype = C.c_int
        _lib.msdo_softmax.restype = C.c_int
        _lib.msdo_inverse_cdf.restype = C.c_int
        _lib.msdo_bandit_select.restype = C.c_int
        _lib.msdo_max_threads.restype = C.c_int
    return _lib


def _p(a, ctype=None):
    if a is None:
        return None
    return a.ctypes.data_as(C.c_void_p if ctype is None else C.POINTER(ctype))


def _f64(x):
    return np.ascontiguousarray(np.asarray(x, dtype=np.float64))


# ----------------------------------------------------------------------------
# Single functions (used by the pins)
# ----------------------------------------------------------------------------
def philox4x32_10(counter, key):
    ctr = np.asarray(counter, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().msdo_philox4x32_10(_p(ctr), _p(k), _p(out))
    return out


def uniform24(word: int) -> float:
    return lib().msdo_uniform24(C.c_uint32(int(word) & 0xFFFFFFFF))


def round_uniforms(seed: int, sequence: int, round_: int, position: int):
    ua, us = C.c_double(), C.c_double()
    lib().msdo_round_uniforms(C.c_uint64(seed), C.c_uint32(sequence), C.c_uint32(round_),
                              C.c_uint32(position), C.byref(ua), C.byref(us))
    return ua.value, us.value


def softmax(x, T: float = 1.0):
    x = _f64(x)
    p = np.empty_like(x)
    bad = lib().msdo_softmax(_p(x), C.c_int(x.size), C.c_double(T), _p(p))
    return p, bool(bad)


def argmax(x) -> int:
    x = _f64(x)
    return lib().msdo_argmax(_p(x), C.c_int(x.size))


def tv_distance(p, q) -> float:
    p, q = _f64(p), _f64(q)
    return lib().msdo_tv_distance(_p(p), _p(q), C.c_int(p.size))


def inverse_cdf(weight, u: float):
    w = _f64(weight)
    margin = C.c_double()
    tok = lib().msdo_inverse_cdf(_p(w), C.c_int(w.size), C.c_double(u), C.byref(margin))
    return tok, margin.value


def verify_sequence(target, draft, tokens, temperature, u_accept, u_sample,
                    reward_temperature: float = 1.0, reward_kind: int = REWARD_BD):
    """One round for one sequence with the uniforms given (Algorithm 4's verification).

    target: (k+1, V) logits, draft: (k, V) logits, tokens: k ids,
    u_accept: k uniforms, u_sample: k+1 uniforms."""
    target, draft = _f64(target), _f64(draft)
    k, V = draft.shape
    assert target.shape == (k + 1, V)
    tokens = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
    ua, us = _f64(u_accept), _f64(u_sample)
    assert ua.size == k and us.size == k + 1
    n_acc, tok, status = C.c_int32(), C.c_int32(), C.c_uint32()
    reward, margin = C.c_double(), C.c_double()
    p_x, q_x, D = np.zeros(k), np.zeros(k), np.zeros(k)
    accept = np.zeros(k, dtype=np.int32)
    scratch = np.zeros(3 * V)
    lib().msdo_verify_sequence(_p(target), _p(draft), _p(tokens), C.c_int(k), C.c_int(V),
                               C.c_double(temperature), C.c_double(reward_temperature),
                               C.c_int(reward_kind), _p(ua), _p(us), C.byref(n_acc), C.byref(tok),
                               C.byref(reward), _p(p_x), _p(q_x), _p(D), _p(accept),
                               C.byref(margin), C.byref(status), _p(scratch))
    return dict(accepted_len=n_acc.value, next_token=tok.value, reward=reward.value, p_x=p_x,
                q_x=q_x, D=D, accept=accept, sample_margin=margin.value, status=status.value)


def bandit_select(variant, K, beta, tau, t, stat_a, stat_b, win_arm=None, win_reward=None):
    gap = C.c_double()
    a = lib().msdo_bandit_select(C.c_int(variant), C.c_int(K), C.c_double(beta), C.c_int(tau),
                                 C.c_int(t), _p(stat_a), _p(stat_b), _p(win_arm), _p(win_reward),
                                 C.byref(gap))
    return a, gap.value


# ----------------------------------------------------------------------------
# Batch object mirroring the library's select / verify / state calls
# ----------------------------------------------------------------------------
def _logit_array(x):
    """numpy view + dtype code of a logits tensor (torch bf16/fp32, numpy uint16/float32)."""
    if isinstance(x, np.ndarray):
        if x.dtype == np.uint16:
            return np.ascontiguousarray(x), DTYPE_BF16
        if x.dtype == np.float32:
            return np.ascontiguousarray(x), DTYPE_FP32
        raise TypeError("logits must be uint16 (bf16 bits) or float32")
    import torch
    x = x.detach().cpu().contiguous()
    if x.dtype == torch.bfloat16:
        return x.view(torch.int16).numpy().view(np.uint16), DTYPE_BF16
    if x.dtype == torch.float32:
        return x.numpy(), DTYPE_FP32
    raise TypeError("logits must be bf16 or fp32")


@dataclass
class OracleConfig:
    max_batch: int
    n_drafters: int           # K
    vocab: int                # V
    bandit: int = UCB
    beta: float = 0.01
    gamma: float = 0.975      # D-UCB discount
    tau: int = 50             # SW-UCB window; PETC: the exploration budget in rounds
    reward: int = REWARD_BD
    reward_temperature: float = 1.0
    sequence_base: int = 0


class OracleMetaSD:
    """B independent bandit instances + the verification round, all float64."""

    def __init__(self, cfg: OracleConfig):
        self.cfg = cfg
        B, K = cfg.max_batch, cfg.n_drafters
        self.t = np.zeros(B, dtype=np.int32)
        self.stat_a = np.zeros((B, K))
        self.stat_b = np.zeros((B, K))
        tau = max(cfg.tau, 1)
        self.win_arm = np.zeros((B, tau), dtype=np.int32)
        self.win_reward = np.zeros((B, tau))
        self.last_gap = np.full(B, np.inf)
        self.select_seed = 0            # key of a randomised policy's arm draw: 0 until the first verify call,
        if cfg.bandit == EXP3:          # then the seed of the latest one
            self.stat_a[:] = 1.0
        if cfg.bandit == PETC:          # S_0 = [K]
            self.stat_b[:] = 1.0
        self.halving_margin = np.full(B, np.inf)    # PETC: the closest call of any halving so far

    def reset(self, seq_ids=None):
        ids = slice(None) if seq_ids is None else np.asarray(seq_ids)
        self.t[ids] = 0
        self.stat_a[ids] = 1.0 if self.cfg.bandit == EXP3 else 0.0      # EXP3: w_0(i) = 1
        self.stat_b[ids] = 1.0 if self.cfg.bandit == PETC else 0.0     # PETC: every drafter is in S_0
        self.halving_margin[ids] = np.inf
        self.win_arm[ids] = 0
        self.win_reward[ids] = 0

    def select(self, batch=None):
        c = self.cfg
        B = c.max_batch if batch is None else batch
        arm = np.zeros(B, dtype=np.int32)
        gap = np.zeros(B)
        lib().msdo_select_batch(C.c_int(B), C.c_int(c.bandit), C.c_int(c.n_drafters),
                                C.c_double(c.beta), C.c_double(c.gamma), C.c_int(max(c.tau, 1)),
                                C.c_uint64(self.select_seed), C.c_uint32(c.sequence_base), _p(self.t),
                                _p(self.stat_a), _p(self.stat_b), _p(self.win_arm),
                                _p(self.win_reward), _p(arm), _p(gap))
        self.last_gap[:B] = np.minimum(gap, self.halving_margin[:B]) if c.bandit == PETC else gap
        return arm

    def verify(self, target_logits, draft_logits, draft_tokens, temperature, seed,
               drafter_tables=None, update=True, draft_len=None):
        """One round.  draft_logits: [B,k,V] gathered by arm, or None with
        drafter_tables = list of K [B,k,V] tensors (indexed by this oracle's own arm)."""
        c = self.cfg
        tgt, dtype = _logit_array(target_logits)
        B, kp1, V = tgt.shape
        k = kp1 - 1
        assert V == c.vocab and B <= c.max_batch
        arm = self.select(B)
        keep = [tgt]
        if draft_logits is not None:
            d, dt2 = _logit_array(draft_logits)
            assert dt2 == dtype and d.shape == (B, k, V)
            keep.append(d)
            d_ptr, tab_ptr = _p(d), None
        else:
            tabs = []
            for tnsr in drafter_tables:
                d, dt2 = _logit_array(tnsr)
                assert dt2 == dtype and d.shape == (B, k, V)
                tabs.append(d)
            keep.extend(tabs)
            arr = (C.c_void_p * len(tabs))(*[t_.ctypes.data for t_ in tabs])
            d_ptr, tab_ptr = None, arr
        tok = np.ascontiguousarray(np.asarray(draft_tokens, dtype=np.int32)).reshape(B, k)
        lens = None if draft_len is None else np.ascontiguousarray(np.asarray(draft_len, dtype=np.int32)).reshape(B)
        out = dict(
            arm=arm,
            accepted_len=np.zeros(B, dtype=np.int32), next_token=np.zeros(B, dtype=np.int32),
            reward=np.zeros(B), p_x=np.zeros((B, k)), q_x=np.zeros((B, k)), D=np.zeros((B, k)),
            accept=np.zeros((B, k), dtype=np.int32), u_accept=np.zeros((B, k)),
            sample_margin=np.zeros(B), status=np.zeros(B, dtype=np.uint32),
            round=self.t[:B].copy())
        lib().msdo_verify_batch(
            C.c_int(B), C.c_int(k), C.c_int(V), C.c_int(dtype), _p(tgt), d_ptr, tab_ptr, _p(arm),
            _p(tok), None if lens is None else _p(lens), C.c_double(temperature), C.c_double(c.reward_temperature), C.c_int(c.reward),
            C.c_uint64(seed), C.c_uint32(c.sequence_base), _p(self.t), _p(out["accepted_len"]),
            _p(out["next_token"]), _p(out["reward"]), _p(out["p_x"]), _p(out["q_x"]), _p(out["D"]),
            _p(out["accept"]), _p(out["u_accept"]), _p(out["sample_margin"]), _p(out["status"]))
        if update:
            self.update(arm, out["reward"])
            self.select_seed = seed
        out["next_arm"] = self.select(B) if update else None
        out["next_gap"] = self.last_gap[:B].copy()
        return out

    def update(self, arm, reward):
        c = self.cfg
        B = len(arm)
        arm = np.ascontiguousarray(arm, dtype=np.int32)
        reward = _f64(reward)
        margin = np.full(B, np.inf)
        lib().msdo_update_batch(C.c_int(B), C.c_int(c.bandit), C.c_int(c.n_drafters),
                                C.c_double(c.gamma), C.c_int(max(c.tau, 1)), _p(self.t),
                                _p(self.stat_a), _p(self.stat_b), _p(self.win_arm),
                                _p(self.win_reward), _p(arm), _p(reward), _p(margin))
        self.halving_margin[:B] = np.minimum(self.halving_margin[:B], margin)

    def mean_estimates(self):
        """mu_hat and n per arm, as the selection rule sees them (for tests)."""
        c = self.cfg
        B, K, tau = c.max_batch, c.n_drafters, max(c.tau, 1)
        mu, n = np.zeros((B, K)), np.zeros((B, K))
        for b in range(B):
            lib().msdo_arm_estimates(C.c_int(c.bandit), C.c_int(K), C.c_int(tau), C.c_int(int(self.t[b])),
                                     _p(self.stat_a[b]), _p(self.stat_b[b]), _p(self.win_arm[b]),
                                     _p(self.win_reward[b]), _p(mu[b]), _p(n[b]))
        return mu, n


def max_threads() -> int:
    return lib().msdo_max_threads()
