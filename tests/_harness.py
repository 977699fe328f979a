"""Lock-step driver for the parity tests: the CUDA library and the CPU oracle see the same bytes.

Comparison rules (what "results identical to the oracle" means here):
  * accepted_len, next_token and arm choices of greedy rounds: bit-exact;
  * p_x, q_x, d_TV per position and the reward: within 1e-5 absolute;
  * accept bits: identical, except where the uniform lies within 1e-6 of p(x)/q(x) (counted);
  * sampled next_token: identical, except where the oracle's CDF margin is below 1e-6 and the GPU
    token is its neighbour in the CDF: the tokens strictly between them carry at most 2e-6 of the mass (counted);
  * arm choices: identical; a difference is tolerated only when the oracle's index gap is below 1e-6
    (counted, then the GPU state is re-synchronised from the oracle's).
"""
from __future__ import annotations

import json
import os

import numpy as np
import torch

from oracle import oracle as O
from paper_2604_05417_b200 import binding as M
from paper_2604_05417_b200.workloads import RoundGenerator, Workload

TOL = 1e-5
NEAR = 1e-6


def new_context(*args, **kw):
    """M.MetaSD(...), skipping the test when the fused path was asked for a shape its geometry cannot take."""
    import pytest
    try:
        return M.MetaSD(*args, **kw)
    except M.MetasdError as e:
        if kw.get("path") == M.PATH_FUSED and e.code == M.ERR_UNSUPPORTED:
            pytest.skip("the fused cluster kernel does not take this shape")
        raise


def make_pair(wl: Workload, path=M.PATH_AUTO, reward=M.REWARD_BD, bandit=None, device=0, sequence_base=0,
              beta=None, host_staging=False, **tuning):
    bandit = bandit or wl.bandit
    beta = wl.beta if beta is None else beta
    gpu = new_context(wl.B, wl.N, wl.k, wl.V, dtype=wl.dtype, bandit=bandit, beta=beta, gamma=wl.gamma,
                      window=wl.tau, reward=reward, device=device, path=path, sequence_base=sequence_base,
                      host_staging=host_staging, **tuning)
    orc = O.OracleMetaSD(O.OracleConfig(max_batch=wl.B, n_drafters=wl.N, vocab=wl.V, bandit=M.BANDITS[bandit],
                                        beta=beta, gamma=wl.gamma, tau=wl.tau, reward=reward,
                                        sequence_base=sequence_base))
    return gpu, orc


def oracle_state_blob(orc: O.OracleMetaSD) -> bytes:
    c = orc.cfg
    parts = dict(header=np.array([0x4D534453, 1, c.max_batch, c.n_drafters, max(c.tau, 1), c.bandit], dtype=np.int64)
                 .astype(np.uint32).view(np.int32),
                 t=orc.t, arm=orc.select(), stat_a=orc.stat_a, stat_b=orc.stat_b, win_arm=orc.win_arm,
                 win_reward=orc.win_reward)
    return M.pack_state(parts)


def _row_weights(target_row, draft_row, T):
    """float64 weights of the draw for one row (test-side, only used to check neighbour tokens)."""
    p = O.softmax(target_row, T)[0]
    if draft_row is None:
        return p
    q = O.softmax(draft_row, T)[0]
    return np.maximum(p - q, 0.0)


def compare_round(res, out, target, draft, T, reward_T, counts):
    """Checks one round's GPU results `res` against the oracle's `out`; updates `counts`."""
    B, k = out["accept"].shape
    greedy = not (T > 0)
    p_x, q_x, D, u, acc = [x.cpu().numpy() for x in res.diag_fields()]
    g_len = res.accepted_len.cpu().numpy()
    g_tok = res.next_token.cpu().numpy()
    g_rew = res.reward.cpu().numpy()

    assert np.array_equal(u.astype(np.float64), out["u_accept"]), "Philox uniforms differ"
    np.testing.assert_allclose(p_x, out["p_x"], rtol=0, atol=TOL)
    np.testing.assert_allclose(q_x, out["q_x"], rtol=0, atol=TOL)
    np.testing.assert_allclose(D, out["D"], rtol=0, atol=TOL)
    counts["max_err_D"] = max(counts.get("max_err_D", 0.0), float(np.abs(D - out["D"]).max()))
    counts["max_err_px"] = max(counts.get("max_err_px", 0.0), float(np.abs(p_x - out["p_x"]).max()))

    diverged = np.zeros(B, dtype=bool)
    mism = acc != out["accept"]
    if mism.any():
        assert not greedy, "greedy accept bits must be bit-exact"
        with np.errstate(divide="ignore", invalid="ignore"):
            ratio = out["p_x"] / out["q_x"]
        near = np.abs(out["u_accept"] - ratio) < NEAR
        assert (near | ~mism).all(), "accept bit differs away from a near tie"
        counts["near_tie_accept"] = counts.get("near_tie_accept", 0) + int(mism.sum())
        diverged = mism.any(axis=1)

    ok = ~diverged
    assert np.array_equal(g_len[ok], out["accepted_len"][ok])
    assert (g_len >= 0).all() and (g_len <= k).all()
    if reward_kind_is_bd(out, k):
        np.testing.assert_allclose(g_rew, out["reward"], rtol=0, atol=TOL)
    else:
        np.testing.assert_allclose(g_rew[ok], out["reward"][ok], rtol=0, atol=TOL)
    counts["max_err_reward"] = max(counts.get("max_err_reward", 0.0), float(np.abs(g_rew - out["reward"])[ok].max(initial=0)))

    tok_mism = ok & (g_tok != out["next_token"])
    if tok_mism.any():
        assert not greedy, "greedy tokens must be bit-exact"
        for b in np.nonzero(tok_mism)[0]:
            assert out["sample_margin"][b] < NEAR, "sampled token differs away from a CDF edge"
            j = int(out["accepted_len"][b])
            row = lambda x: x.float().cpu().numpy().astype(np.float64)
            w = _row_weights(row(target[b, j]), row(draft[b, j]) if j < k else None, T)
            # the two tokens must be neighbours in the CDF: what lies strictly between them carries (next to) no mass.
            # In float64 that is "the neighbouring token with mass"; fp32 may flush weights of 1e-12 that float64
            # still sees, so the bound is on the mass in between, not on the count of tokens.
            lo, hi = sorted((int(g_tok[b]), int(out["next_token"][b])))
            between = float(w[lo + 1:hi].sum())
            assert 0 <= lo and hi < len(w) and between <= 2 * NEAR * float(w.sum()), \
                "GPU token is not the oracle's neighbour in the CDF"
        counts["near_tie_token"] = counts.get("near_tie_token", 0) + int(tok_mism.sum())
    counts["rounds"] = counts.get("rounds", 0) + 1
    counts["tokens"] = counts.get("tokens", 0) + int((g_len + 1).sum())
    return diverged


def reward_kind_is_bd(out, k):
    return out.get("_reward_kind", M.REWARD_BD) == M.REWARD_BD


def gather_by_arm(drafts, tokens, arm, dev):
    """Rows and tokens of the drafter each sequence plays, picked out of the K per-drafter tensors (input
    marshalling for the oracle, which then reads [B,k,V] instead of K such tensors)."""
    idx = torch.as_tensor(arm, device=dev, dtype=torch.long)
    draft = torch.empty_like(drafts[0])
    toks = torch.empty_like(tokens[0])
    for i in range(len(drafts)):
        rows = torch.nonzero(idx == i).flatten()
        if rows.numel():
            draft[rows] = drafts[i][rows]
            toks[rows] = tokens[i][rows]
    return draft, toks


def write_report(label: str, counts: dict):
    """Appends the counters of a lock-step run to the JSON-lines file named by METASD_PARITY_REPORT (if set)."""
    path = os.environ.get("METASD_PARITY_REPORT")
    if not path:
        return
    row = {"case": label}
    row.update({k: (v if isinstance(v, (int, float, str)) else float(v)) for k, v in counts.items()})
    with open(path, "a") as f:
        f.write(json.dumps(row) + "\n")


def run_lockstep(wl: Workload, rounds: int, seed: int = 0, lib_seed: int = 1234, path=M.PATH_AUTO,
                 reward=M.REWARD_BD, bandit=None, table_mode=False, device=0, sequence_base=0, beta=None,
                 check_state=True, oracle_reads_tables=True, label=None, **tuning):
    """Runs `rounds` rounds of the workload on both sides and compares every round.  table_mode: the library reads
    the K drafters' tensors through its pointer table; the oracle then reads the same tables, or (for the large
    configurations, oracle_reads_tables=False) the rows gathered by its own arm choice."""
    dev = torch.device("cuda", device)
    gen = RoundGenerator(wl, device=dev, seed=seed)
    gpu, orc = make_pair(wl, path=path, reward=reward, bandit=bandit, device=device,
                         sequence_base=sequence_base, beta=beta, **tuning)
    counts = {"sequences": wl.B, "near_tie_accept": 0, "near_tie_token": 0, "near_tie_arm": 0, "best_arm_plays": 0}
    T = wl.temperature
    try:
        for t in range(rounds):
            arm_g = gpu.select().cpu().numpy()
            arm_o = orc.select()
            if not np.array_equal(arm_g, arm_o):
                bad = np.nonzero(arm_g != arm_o)[0]
                assert (orc.last_gap[bad] < NEAR).all(), "arm choice differs away from a near tie (round %d)" % t
                counts["near_tie_arm"] = counts.get("near_tie_arm", 0) + len(bad)
                gpu.state_import(oracle_state_blob(orc))
                arm_g = gpu.select().cpu().numpy()
                assert np.array_equal(arm_g, arm_o)
            if table_mode:
                rd = gen.table_round(t)
                table = M.pointer_table(rd["drafts"])
                res = gpu.verify(rd["target"], None, rd["tokens"], T, lib_seed, drafter_table=table,
                                 token_arm_stride=wl.B * wl.k, want_diag=True)
                draft, tokens = gather_by_arm(rd["drafts"], rd["tokens"], arm_o, dev)
                if oracle_reads_tables:
                    out = orc.verify(rd["target"], None, tokens.cpu().numpy(), T, lib_seed,
                                     drafter_tables=rd["drafts"])
                else:
                    out = orc.verify(rd["target"], draft, tokens.cpu().numpy(), T, lib_seed)
            else:
                rd = gen.gathered_round(t, arm_o)
                draft = rd["draft"]
                res = gpu.verify(rd["target"], draft, rd["tokens"], T, lib_seed, want_diag=True)
                out = orc.verify(rd["target"], draft, rd["tokens"].cpu().numpy(), T, lib_seed)
            out["_reward_kind"] = reward
            counts["best_arm_plays"] += int((arm_o == gen.best_arm(t)).sum())
            diverged = compare_round(res, out, rd["target"], draft, T, 1.0, counts)
            if diverged.any() and reward == M.REWARD_BE:
                gpu.state_import(oracle_state_blob(orc))   # BE feeds accept bits into the bandit
        if check_state:
            st = M.parse_state(gpu.state_export(), wl.B, wl.N, wl.tau)
            assert np.array_equal(st["t"], orc.t)
            np.testing.assert_allclose(st["stat_a"], orc.stat_a, rtol=0, atol=1e-5)
            np.testing.assert_allclose(st["stat_b"], orc.stat_b, rtol=0, atol=1e-9)
            if M.BANDITS[bandit or wl.bandit] == M.SWUCB:
                assert np.array_equal(st["win_arm"], orc.win_arm)
                np.testing.assert_allclose(st["win_reward"], orc.win_reward, rtol=0, atol=1e-5)
        counts["status"] = gpu.last_status()
        counts["launches"] = gpu.kernel_launches()
        counts["path"] = gpu.resolved_path(wl.k)
        counts["row_kernel"] = gpu.resolved_row_kernel()
    finally:
        gpu.close()
    write_report(label or wl.name, counts)
    return counts
