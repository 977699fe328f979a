"""GPU parity: the CUDA library against the float64 CPU oracle on the same seeded bytes (C ABI calls)."""
import numpy as np
import pytest
import torch

from paper_2604_05417_b200 import binding as M
from paper_2604_05417_b200.workloads import WORKLOADS, RoundGenerator, Workload

pytestmark = pytest.mark.gpu


def small(name, **kw):
    return WORKLOADS[name].scaled(**kw)


def base(**kw):
    d = dict(name="t", B=3, N=3, k=4, V=1000, rounds=8, temperature=1.0, dtype="bf16", bandit="ucb",
             sigmas=(0.5, 1.5, 3.0))
    d.update(kw)
    return Workload(**d)


def report(counts):
    print({k: v for k, v in counts.items()})
    return counts


PATHS = [M.PATH_STREAMING, M.PATH_FUSED]   # a shape the fused geometry cannot take is skipped


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
@pytest.mark.parametrize("V,k,B", [(5, 1, 1), (17, 3, 2), (1000, 4, 3), (20008, 5, 4), (4100, 16, 2), (32000, 2, 7)])
def test_small_shapes_sampled(path, dtype, V, k, B):
    """Tiny to several-tile vocabularies, ragged tails, scalar (V % 8 != 0) and vector rows."""
    from _harness import run_lockstep
    wl = base(B=B, k=k, V=V, dtype=dtype, temperature=0.8)
    c = report(run_lockstep(wl, rounds=8, path=path))
    assert c["rounds"] == 8


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
@pytest.mark.parametrize("V,k,B", [(17, 3, 2), (1000, 4, 3), (20008, 5, 4)])
def test_small_shapes_greedy_bit_exact(path, dtype, V, k, B):
    from _harness import run_lockstep
    wl = base(B=B, k=k, V=V, dtype=dtype, temperature=0.0, sigmas=(0.1, 0.5, 2.0))
    c = report(run_lockstep(wl, rounds=8, path=path))
    assert c.get("near_tie_accept", 0) == 0 and c.get("near_tie_token", 0) == 0 and c.get("near_tie_arm", 0) == 0


@pytest.mark.parametrize("path", PATHS)
def test_cfg1_tiny_full_length(path):
    from _harness import run_lockstep
    wl = WORKLOADS["cfg1_tiny"]
    c = report(run_lockstep(wl, rounds=wl.rounds, path=path))
    assert c["rounds"] == 200 and c.get("near_tie_arm", 0) == 0


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("bandit", ["ducb", "swucb"])
def test_cfg2_nonstationary_scaled(path, bandit):
    """D-UCB and SW-UCB on the re-permuted drafter noise (period shortened so the best arm moves)."""
    from _harness import run_lockstep
    wl = small("cfg2_nonstationary", B=16, rounds=60, period=20, tau=15, gamma=0.9)
    c = report(run_lockstep(wl, rounds=60, path=path, bandit=bandit))
    assert c.get("near_tie_arm", 0) == 0


@pytest.mark.parametrize("path", PATHS)
def test_cfg3_tasks_scaled(path):
    from _harness import run_lockstep
    wl = small("cfg3_tasks", B=8, rounds=12)
    report(run_lockstep(wl, rounds=12, path=path))


@pytest.mark.parametrize("path", PATHS)
def test_cfg4_greedy_scaled_bit_exact(path):
    from _harness import run_lockstep
    wl = small("cfg4_greedy", B=16, rounds=8)
    c = report(run_lockstep(wl, rounds=8, path=path))
    assert c.get("near_tie_accept", 0) == 0 and c.get("near_tie_token", 0) == 0 and c.get("near_tie_arm", 0) == 0


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("bandit", ["ucb", "ducb"])
def test_cfg5_fp32_scaled(path, bandit):
    from _harness import run_lockstep
    wl = small("cfg5_fp32_stress", B=8, rounds=12)
    report(run_lockstep(wl, rounds=12, path=path, bandit=bandit))


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("bandit", ["exp3", "rand"])
def test_randomised_policies(path, bandit):
    """MetaSD-EXP3 and the uniformly random baseline: arm draws, weights and round counters follow the oracle."""
    from _harness import run_lockstep
    wl = base(B=9, N=4, k=3, V=2048, sigmas=(0.3, 1.0, 2.0, 3.5)).scaled(gamma=0.2)
    c = report(run_lockstep(wl, rounds=40, path=path, bandit=bandit, table_mode=True))
    assert c["rounds"] == 40


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("N,budget", [(5, 30), (4, 16), (3, 2)])
def test_pure_exploration_then_commit(path, N, budget):
    """PETC: the Sequential Halving schedule, every halving and the committed drafter follow the oracle."""
    from _harness import run_lockstep
    sig = (0.3, 1.0, 2.0, 3.5, 0.6)[:N]
    wl = base(B=7, N=N, k=3, V=2048, sigmas=sig).scaled(tau=budget)
    c = report(run_lockstep(wl, rounds=budget + 12, path=path, bandit="petc", table_mode=True))
    assert c["rounds"] == budget + 12 and c.get("near_tie_arm", 0) == 0


@pytest.mark.parametrize("dtype,V,T,k,bandit", [("bf16", 152064, 1.0, 8, "ucb"), ("fp32", 128256, 1.0, 5, "ducb"),
                                                ("bf16", 50264, 1.3, 6, "petc")])
def test_many_rounds_on_large_vocabularies(dtype, V, T, k, bandit):
    """Lock-step rounds at the benchmark's vocabulary sizes (several trips of every staging depth, ragged last trip),
    sampled mode, pointer-table inputs: every round's outputs and the bandit state follow the oracle."""
    from _harness import run_lockstep
    wl = base(B=12, N=4, k=k, V=V, sigmas=(0.3, 1.0, 2.0, 3.0)).scaled(dtype=dtype, temperature=T, tau=20)
    c = report(run_lockstep(wl, rounds=12, seed=V % 97, path=M.PATH_STREAMING, bandit=bandit, table_mode=True))
    assert c["rounds"] == 12 and c["status"] == 0 and c["max_err_D"] < 5e-6


@pytest.mark.parametrize("path", PATHS)
def test_pointer_table_mode(path):
    """The kernel indexes a table of K drafter tensors and a [K,B,k] token table by arm."""
    from _harness import run_lockstep
    wl = base(B=5, N=4, k=3, V=4096, sigmas=(0.3, 1.0, 2.0, 3.0))
    report(run_lockstep(wl, rounds=10, path=path, table_mode=True))


@pytest.mark.parametrize("path", PATHS)
def test_be_reward_mode(path):
    from _harness import run_lockstep
    wl = base(B=6, N=3, k=5, V=2048)
    report(run_lockstep(wl, rounds=12, path=path, reward=M.REWARD_BE))


@pytest.mark.parametrize("path", PATHS)
def test_batch_shard_uses_global_sequence_ids(path):
    """Two shards with sequence_base 0 and B/2 reproduce the unsharded results (no collective needed)."""
    wl = base(B=8, N=2, k=3, V=1024, sigmas=(0.5, 2.0))
    dev = torch.device("cuda", 0)
    gen = RoundGenerator(wl, device=dev, seed=3)
    full = M.MetaSD(8, 2, 3, 1024, path=path)
    lo = M.MetaSD(4, 2, 3, 1024, path=path, sequence_base=0)
    hi = M.MetaSD(4, 2, 3, 1024, path=path, sequence_base=4)
    for t in range(5):
        arm = full.select().cpu().numpy()
        rd = gen.gathered_round(t, arm)
        r = full.verify(rd["target"], rd["draft"], rd["tokens"], 1.0, 77)
        r0 = lo.verify(rd["target"][:4].contiguous(), rd["draft"][:4].contiguous(), rd["tokens"][:4].contiguous(), 1.0, 77)
        r1 = hi.verify(rd["target"][4:].contiguous(), rd["draft"][4:].contiguous(), rd["tokens"][4:].contiguous(), 1.0, 77)
        for name in ("accepted_len", "next_token", "reward"):
            assert torch.equal(getattr(r, name), torch.cat([getattr(r0, name), getattr(r1, name)]))
        assert torch.equal(full.select(), torch.cat([lo.select(), hi.select()]))
    for m in (full, lo, hi):
        m.close()


@pytest.mark.parametrize("T", [1.0, 0.0])
@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
def test_per_sequence_draft_lengths(T, dtype):
    """Sequences that drafted fewer than k tokens: only their own rows are read (the rest is poisoned with NaN),
    accepted lengths, tokens, rewards and the bandit follow the oracle's ragged round."""
    from _harness import make_pair, TOL, NEAR
    wl = base(B=11, N=3, k=5, V=4096 + 8, sigmas=(0.4, 1.2, 2.5)).scaled(dtype=dtype, temperature=T)
    dev = torch.device("cuda", 0)
    gen = RoundGenerator(wl, device=dev, seed=11)
    gpu, orc = make_pair(wl, path=M.PATH_STREAMING)
    rng = np.random.RandomState(2)
    lens_dev = torch.zeros(wl.B, dtype=torch.int32, device=dev)
    gpu.set_draft_lengths(lens_dev)
    try:
        for t in range(8):
            lens = rng.randint(1, wl.k + 1, size=wl.B).astype(np.int32)
            if t == 0:
                lens[:] = wl.k
            lens_dev.copy_(torch.from_numpy(lens))
            arm = orc.select()
            assert np.array_equal(gpu.select().cpu().numpy(), arm)
            rd = gen.gathered_round(t, arm)
            target, draft = rd["target"].clone(), rd["draft"].clone()
            for b in range(wl.B):
                target[b, lens[b] + 1:] = float("nan")
                draft[b, lens[b]:] = float("nan")
            res = gpu.verify(target, draft, rd["tokens"], T, 99, want_diag=True)
            out = orc.verify(target, draft, rd["tokens"].cpu().numpy(), T, 99, draft_len=lens)
            assert gpu.last_status() == 0 and (out["status"] == 0).all()
            g_len = res.accepted_len.cpu().numpy()
            assert np.array_equal(g_len, out["accepted_len"]) and (g_len <= lens).all()
            g_tok = res.next_token.cpu().numpy()
            firm = out["sample_margin"] > NEAR if T > 0 else np.ones(wl.B, dtype=bool)
            assert np.array_equal(g_tok[firm], out["next_token"][firm])
            np.testing.assert_allclose(res.reward.cpu().numpy(), out["reward"], rtol=0, atol=TOL)
            D = res.diag_fields()[2].cpu().numpy()
            for b in range(wl.B):
                np.testing.assert_allclose(D[b, :lens[b]], out["D"][b, :lens[b]], rtol=0, atol=TOL)
        st = M.parse_state(gpu.state_export(), wl.B, wl.N, wl.tau)
        assert np.array_equal(st["t"], orc.t)
        np.testing.assert_allclose(st["stat_a"], orc.stat_a, rtol=0, atol=1e-5)
        # lengths outside 1 .. k are clamped and flagged; clearing the registration restores the fixed length
        lens_dev.copy_(torch.tensor([0, wl.k + 7] + [2] * (wl.B - 2), dtype=torch.int32))
        arm = orc.select()
        rd = gen.gathered_round(8, arm)
        res = gpu.verify(rd["target"], rd["draft"], rd["tokens"], T, 99)
        out = orc.verify(rd["target"], rd["draft"], rd["tokens"].cpu().numpy(), T, 99,
                         draft_len=np.array([1, wl.k] + [2] * (wl.B - 2)))
        assert gpu.last_status() == M.STATUS_BAD_LENGTH
        assert np.array_equal(res.accepted_len.cpu().numpy(), out["accepted_len"])
        gpu.set_draft_lengths(None)
        arm = orc.select()
        rd = gen.gathered_round(9, arm)
        res = gpu.verify(rd["target"], rd["draft"], rd["tokens"], T, 99)
        out = orc.verify(rd["target"], rd["draft"], rd["tokens"].cpu().numpy(), T, 99)
        assert gpu.last_status() == 0
        assert np.array_equal(res.accepted_len.cpu().numpy(), out["accepted_len"])
    finally:
        gpu.close()


def test_fused_path_declines_per_sequence_draft_lengths():
    from _harness import new_context
    gpu = new_context(4, 2, 3, 4096, path=M.PATH_FUSED)
    dev = torch.device("cuda", 0)
    try:
        gpu.set_draft_lengths(torch.full((4,), 2, dtype=torch.int32, device=dev))
        wl = base(B=4, N=2, k=3, V=4096, sigmas=(0.5, 2.0))
        rd = RoundGenerator(wl, device=dev, seed=1).gathered_round(0, np.zeros(4, dtype=np.int64))
        with pytest.raises(M.MetasdError) as err:
            gpu.verify(rd["target"], rd["draft"], rd["tokens"], 1.0, 5)
        assert err.value.code == M.ERR_UNSUPPORTED
    finally:
        gpu.close()


@pytest.mark.parametrize("tuning", [dict(row_kernel=M.ROWS_STAGED, row_threads=640), dict(row_kernel=M.ROWS_STAGED, row_stages=5),
                                    dict(row_kernel=M.ROWS_STAGED, row_cluster=4), dict(row_kernel=M.ROWS_BULK, row_cluster=2),
                                    dict(row_kernel=M.ROWS_PLAIN, row_cluster=2), dict(row_kernel=M.ROWS_BULK, row_stages=9)],
                         ids=lambda d: "-".join("%s%s" % kv for kv in d.items()))
def test_a_row_kernel_shape_that_is_not_built_is_declined_at_init(tuning):
    """Only the built shapes of the row-statistics kernels are accepted; anything else is UNSUPPORTED, not a fallback."""
    with pytest.raises(M.MetasdError) as err:
        M.MetaSD(4, 2, 3, 4096, dtype="bf16", device=0, **tuning)
    assert err.value.code == M.ERR_UNSUPPORTED


@pytest.mark.parametrize("dtype", ["bf16", "fp32"])
@pytest.mark.parametrize("T", [1.0, 0.5])
def test_draft_rows_on_another_scale_than_the_target(dtype, T):
    """Softmax is shift invariant, so a drafter whose logits sit hundreds of units above or below the target's is
    legal input.  The row-statistics kernel sums the draft row relative to the target's maximum where that is
    safe and must notice where it is not (these offsets overflow or flush that sum) and redo the row.  The offsets
    stay where fp32 exponents still resolve 1e-5: an offset M c is rounded at its own size, so |M| c is kept
    below about 450."""
    from _harness import make_pair, compare_round
    wl = base(B=8, N=1, k=3, V=8192, sigmas=(0.8,)).scaled(dtype=dtype, temperature=T)
    dev = torch.device("cuda", 0)
    gen = RoundGenerator(wl, device=dev, seed=4)
    gpu, orc = make_pair(wl, path=M.PATH_STREAMING)
    offsets = torch.tensor([0.0, -150.0, 150.0, -70.0, 70.0, -110.0, 110.0, 20.0], device=dev)
    counts = {}
    try:
        for t in range(3):
            arm = orc.select()
            rd = gen.gathered_round(t, arm)
            draft = (rd["draft"].float() + offsets.view(-1, 1, 1)).to(rd["draft"].dtype)
            res = gpu.verify(rd["target"], draft, rd["tokens"], T, 31, want_diag=True)
            out = orc.verify(rd["target"], draft, rd["tokens"].cpu().numpy(), T, 31)
            compare_round(res, out, rd["target"], draft, T, 1.0, counts)
            assert gpu.last_status() == 0
    finally:
        gpu.close()


@pytest.mark.parametrize("path", PATHS)
def test_defined_outcomes_of_anomalous_inputs(path):
    """NaN rows, masked (-inf) logits, out-of-range tokens: same defined outputs and status bits."""
    from _harness import make_pair, compare_round
    wl = base(B=4, N=1, k=3, V=1024, sigmas=(1.0,))
    dev = torch.device("cuda", 0)
    gen = RoundGenerator(wl, device=dev, seed=5)
    gpu, orc = make_pair(wl, path=path)
    rd = gen.gathered_round(0, np.zeros(4, dtype=np.int64))
    target, draft, tokens = rd["target"], rd["draft"], rd["tokens"].clone()
    draft[0, 1, 100] = float("nan")            # sequence 0: NaN in draft row 1
    target[1, :, 200:700] = float("-inf")      # sequence 1: masked target tokens
    draft[1, :, 300:800] = float("-inf")
    tokens[2, 0] = 5000                         # sequence 2: token out of range
    tokens[3, 2] = -7
    res = gpu.verify(target, draft, tokens, 1.0, 9, want_diag=True)
    out = orc.verify(target, draft, tokens.cpu().numpy(), 1.0, 9)
    compare_round(res, out, target, draft, 1.0, 1.0, {})
    status = gpu.last_status()
    assert status & M.STATUS_NONFINITE and status & M.STATUS_TOKEN_OOR
    assert out["status"][0] & M.STATUS_NONFINITE and out["status"][2] & M.STATUS_TOKEN_OOR
    assert gpu.last_status() == 0              # reading clears the word
    gpu.close()


@pytest.mark.parametrize("path", PATHS)
def test_identical_drafter_accepts_everything(path):
    wl = base(B=3, N=1, k=4, V=2048, sigmas=(0.0,))
    dev = torch.device("cuda", 0)
    gen = RoundGenerator(wl, device=dev, seed=6)
    gpu = M.MetaSD(3, 1, 4, 2048, path=path)
    rd = gen.gathered_round(0, np.zeros(3, dtype=np.int64))
    res = gpu.verify(rd["target"], rd["target"][:, :4].contiguous(), rd["tokens"], 1.0, 1)
    assert (res.accepted_len == 4).all()
    assert torch.allclose(res.reward, torch.ones(3, device=dev), atol=1e-6)
    gpu.close()


@pytest.mark.parametrize("path", PATHS)
def test_reset_and_state_roundtrip(path):
    """Export -> destroy -> init -> import continues identically; reset re-initialises chosen sequences."""
    wl = base(B=6, N=3, k=2, V=1024)
    dev = torch.device("cuda", 0)
    gen = RoundGenerator(wl, device=dev, seed=8)
    a = M.MetaSD(6, 3, 2, 1024, path=path, bandit="swucb", window=4)
    rounds = [gen.gathered_round(t, np.zeros(6, dtype=np.int64)) for t in range(8)]
    for t in range(5):
        a.verify(rounds[t]["target"], rounds[t]["draft"], rounds[t]["tokens"], 1.0, 3)
    blob = a.state_export()
    b = M.MetaSD(6, 3, 2, 1024, path=path, bandit="swucb", window=4)
    b.state_import(blob)
    for t in range(5, 8):
        ra = a.verify(rounds[t]["target"], rounds[t]["draft"], rounds[t]["tokens"], 1.0, 3)
        rb = b.verify(rounds[t]["target"], rounds[t]["draft"], rounds[t]["tokens"], 1.0, 3)
        assert torch.equal(ra.next_token, rb.next_token) and torch.equal(ra.reward, rb.reward)
        assert torch.equal(a.select(), b.select())
    assert a.state_export() == b.state_export()
    # a blob from a differently shaped context is refused
    c = M.MetaSD(6, 3, 2, 1024, path=path, bandit="ucb", window=4)
    with pytest.raises(M.MetasdError) as e:
        c.state_import(blob)
    assert e.value.code == M.ERR_BAD_STATE_BLOB
    with pytest.raises(M.MetasdError) as e:
        c.state_import(blob[:-8])                      # too short for this context
    assert e.value.code == M.ERR_INVALID_ARGUMENT
    # reset two sequences
    a.reset(torch.tensor([1, 4], dtype=torch.int32, device=dev))
    st = M.parse_state(a.state_export(), 6, 3, 4)
    assert st["t"].tolist() == [8, 0, 8, 8, 0, 8] and (st["arm"][[1, 4]] == 0).all()
    assert (st["win_reward"][[1, 4]] == 0).all()
    a.reset()
    assert (M.parse_state(a.state_export(), 6, 3, 4)["t"] == 0).all()
    for m in (a, b, c):
        m.close()


@pytest.mark.parametrize("path", PATHS)
def test_misaligned_drafter_table_entry_is_flagged_not_dereferenced(path):
    """A table pointer that is not 16-byte aligned sets a status bit; the rows behind it are never read."""
    wl = base(B=4, N=2, k=3, V=1024, sigmas=(0.5, 2.0))
    dev = torch.device("cuda", 0)
    gen = RoundGenerator(wl, device=dev, seed=13)
    from _harness import new_context
    gpu = new_context(4, 2, 3, 1024, path=path)
    rd = gen.table_round(0)
    backing = torch.zeros(4 * 3 * 1024 + 8, dtype=torch.bfloat16, device=dev)
    crooked = backing[1:1 + 4 * 3 * 1024].view(4, 3, 1024)          # starts 2 bytes past a 16-byte boundary
    crooked.copy_(rd["drafts"][0])
    assert crooked.data_ptr() % 16 == 2
    table = M.pointer_table([crooked, rd["drafts"][1]])
    for t in range(2):                                               # round 0 plays drafter 0 (the crooked one), round 1 drafter 1
        res = gpu.verify(rd["target"], None, rd["tokens"], 1.0, 3, drafter_table=table, token_arm_stride=4 * 3)
        torch.cuda.synchronize()
        status = gpu.last_status()
        assert status & M.STATUS_BAD_POINTER                         # flagged on every call that is handed this table
        assert ((res.accepted_len >= 0) & (res.accepted_len <= 3)).all()
    gpu.close()


def test_argument_validation_on_device():
    gpu = M.MetaSD(2, 2, 3, 512)
    dev = torch.device("cuda", 0)
    tgt = torch.zeros((2, 4, 512), dtype=torch.bfloat16, device=dev)
    drf = torch.zeros((2, 3, 512), dtype=torch.bfloat16, device=dev)
    tok = torch.zeros((2, 3), dtype=torch.int32, device=dev)
    lib, ctx = gpu.lib, gpu._ctx
    out = [torch.zeros(2, dtype=torch.int32, device=dev), torch.zeros(2, dtype=torch.int32, device=dev),
           torch.zeros(2, dtype=torch.float32, device=dev)]
    import ctypes as C
    def call(batch=2, k=3, t=tgt, d=drf, tab=None, T=1.0):
        return lib.metasd_verify(ctx, batch, k, M._ptr(t), M._ptr(d), M._ptr(tab), M._ptr(tok), 0, C.c_float(T),
                                 C.c_uint64(0), M._ptr(out[0]), M._ptr(out[1]), M._ptr(out[2]), None, None)
    assert call() == M.OK
    assert call(batch=3) == M.ERR_INVALID_ARGUMENT
    assert call(k=4) == M.ERR_INVALID_ARGUMENT
    assert call(k=0) == M.ERR_INVALID_ARGUMENT
    assert call(t=None) == M.ERR_INVALID_ARGUMENT
    assert call(d=None) == M.ERR_INVALID_ARGUMENT                       # neither draft source
    assert call(tab=torch.zeros(2, dtype=torch.int64, device=dev)) == M.ERR_INVALID_ARGUMENT   # both
    assert call(T=-1.0) == M.ERR_INVALID_ARGUMENT
    assert call(T=float("nan")) == M.ERR_INVALID_ARGUMENT
    assert lib.metasd_select(ctx, 5, M._ptr(out[0]), None) == M.ERR_INVALID_ARGUMENT
    assert lib.metasd_verify_host(ctx, 2, 3, None, None, None, C.c_float(1.0), C.c_uint64(0), None, None, None, None,
                                  None) == M.ERR_INVALID_ARGUMENT       # no staging in this context
    torch.cuda.synchronize()
    gpu.close()


def test_verify_host_matches_device_call():
    wl = base(B=4, N=2, k=3, V=2048, sigmas=(0.5, 2.0))
    dev = torch.device("cuda", 0)
    gen = RoundGenerator(wl, device=dev, seed=11)
    a = M.MetaSD(4, 2, 3, 2048)
    b = M.MetaSD(4, 2, 3, 2048, host_staging=True)
    for t in range(4):
        arm = a.select().cpu().numpy()
        rd = gen.gathered_round(t, arm)
        ra = a.verify(rd["target"], rd["draft"], rd["tokens"], 0.9, 21)
        h = [x.cpu().pin_memory() for x in (rd["target"], rd["draft"], rd["tokens"])]
        acc = torch.zeros(4, dtype=torch.int32).pin_memory()
        tok = torch.zeros(4, dtype=torch.int32).pin_memory()
        rew = torch.zeros(4, dtype=torch.float32).pin_memory()
        nxt = torch.zeros(4, dtype=torch.int32).pin_memory()
        b.verify_host(h[0], h[1], h[2], 0.9, 21, acc, tok, rew, nxt)
        assert torch.equal(ra.accepted_len.cpu(), acc) and torch.equal(ra.next_token.cpu(), tok)
        assert torch.equal(ra.reward.cpu(), rew) and torch.equal(a.select().cpu(), nxt)
    a.close(); b.close()


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("name", ["cfg4_greedy", "cfg3_tasks", "cfg5_fp32_stress", "cfg2_nonstationary"])
def test_full_size_launch_sampled_against_oracle(name, path):
    """The benchmark's launch configuration at full batch and vocabulary; the oracle re-computes a
    sample of sequences one by one (each keyed by its global sequence id)."""
    from oracle import oracle as O
    wl = WORKLOADS[name]
    dev = torch.device("cuda", 0)
    gen = RoundGenerator(wl, device=dev, seed=1)
    gpu = M.MetaSD(wl.B, wl.N, wl.k, wl.V, dtype=wl.dtype, bandit=wl.bandit, path=path)
    sample = [0, 1, wl.B // 2 + 3, wl.B - 1]
    T = wl.temperature
    for t in range(2):
        arm = gpu.select().cpu().numpy()
        assert (arm == t).all()                       # initial sweep
        rd = gen.gathered_round(t, arm)
        res = gpu.verify(rd["target"], rd["draft"], rd["tokens"], T, 555, want_diag=True)
        p_x, q_x, D, u, acc = [x.cpu().numpy() for x in res.diag_fields()]
        n_acc = res.accepted_len.cpu().numpy()
        assert (n_acc >= 0).all() and (n_acc <= wl.k).all()
        rew = res.reward.cpu().numpy()
        assert ((rew > 0) & (rew <= 1 + 1e-6)).all()
        np.testing.assert_allclose(rew, 1 - D.mean(axis=1), atol=2e-6)
        lead = np.where(acc.all(axis=1), wl.k, np.argmin(acc, axis=1))
        assert np.array_equal(lead, n_acc)
        for b in sample:
            orc = O.OracleMetaSD(O.OracleConfig(max_batch=1, n_drafters=wl.N, vocab=wl.V, sequence_base=b))
            orc.t[0] = t
            out = orc.verify(rd["target"][b:b + 1], rd["draft"][b:b + 1], rd["tokens"][b:b + 1].cpu().numpy(), T, 555,
                             update=False)
            np.testing.assert_allclose(D[b], out["D"][0], atol=1e-5)
            np.testing.assert_allclose(p_x[b], out["p_x"][0], atol=1e-5)
            np.testing.assert_allclose(rew[b], out["reward"][0], atol=1e-5)
            if T == 0 or (np.abs(out["u_accept"][0] - out["p_x"][0] / np.maximum(out["q_x"][0], 1e-300)) > 1e-6).all():
                assert n_acc[b] == out["accepted_len"][0]
                if T == 0 or out["sample_margin"][0] > 1e-6:
                    assert res.next_token[b].item() == out["next_token"][0]
    gpu.close()


# ------------------------------------------------------------------------------------------------------------------
# The five benchmark configurations at their full batch, every sequence in lock-step with the oracle, well past the
# initial sweep, the bandit choosing the drafter through the pointer table.
# ------------------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("bandit", ["ducb", "swucb"])
def test_cfg2_full_batch_nonstationary(bandit):
    """All 64 sequences, 250 rounds at the real period of 100: the drafter noise is re-permuted twice, and the
    discounted / sliding-window statistics follow the oracle's through both changes."""
    from _harness import run_lockstep
    wl = WORKLOADS["cfg2_nonstationary"]
    c = report(run_lockstep(wl, rounds=250, bandit=bandit, table_mode=True, label="cfg2_full_%s" % bandit))
    assert c["rounds"] == 250 and c["sequences"] == 64 and c["near_tie_arm"] == 0 and c["status"] == 0
    assert c["best_arm_plays"] > 0.3 * 250 * 64     # the policies do track the moving best drafter


def test_cfg3_full_batch():
    from _harness import run_lockstep
    wl = WORKLOADS["cfg3_tasks"]
    c = report(run_lockstep(wl, rounds=30, table_mode=True, oracle_reads_tables=False, label="cfg3_full"))
    assert c["rounds"] == 30 and c["sequences"] == 256 and c["near_tie_arm"] == 0 and c["status"] == 0


def test_cfg4_full_batch_greedy_bit_exact():
    from _harness import run_lockstep
    wl = WORKLOADS["cfg4_greedy"]
    c = report(run_lockstep(wl, rounds=24, table_mode=True, oracle_reads_tables=False, label="cfg4_full"))
    assert c["rounds"] == 24 and c["sequences"] == 512 and c["status"] == 0
    assert c["near_tie_accept"] == 0 and c["near_tie_token"] == 0 and c["near_tie_arm"] == 0


@pytest.mark.parametrize("bandit", ["ucb", "ducb"])
def test_cfg5_full_batch(bandit):
    from _harness import run_lockstep
    wl = WORKLOADS["cfg5_fp32_stress"]
    c = report(run_lockstep(wl, rounds=20, bandit=bandit, table_mode=True, oracle_reads_tables=False,
                            label="cfg5_full_%s" % bandit))
    assert c["rounds"] == 20 and c["sequences"] == 1024 and c["near_tie_arm"] == 0 and c["status"] == 0


# ------------------------------------------------------------------------------------------------------------------
# Every row-statistics variant and the draw's early stop
# ------------------------------------------------------------------------------------------------------------------
ROW_KERNELS = [dict(row_kernel=M.ROWS_PLAIN), dict(row_kernel=M.ROWS_STAGED),
               dict(row_kernel=M.ROWS_STAGED, row_threads=1024, row_stages=6),
               dict(row_kernel=M.ROWS_STAGED, row_threads=768, row_stages=4),
               dict(row_kernel=M.ROWS_STAGED, row_threads=512, row_stages=4, row_cluster=3),
               dict(row_kernel=M.ROWS_STAGED, row_threads=768, row_stages=4, row_cluster=2),
               dict(row_kernel=M.ROWS_STAGED, row_threads=512, row_stages=4, row_cluster=2),
               dict(row_kernel=M.ROWS_BULK), dict(row_kernel=M.ROWS_BULK, row_threads=512, row_stages=3),
               dict(row_kernel=M.ROWS_BULK, row_threads=1024, row_stages=7),
               dict(row_kernel=M.ROWS_BULK, row_threads=768, row_stages=8)]


@pytest.mark.parametrize("tuning", ROW_KERNELS, ids=lambda d: "-".join(str(v) for v in d.values()))
@pytest.mark.parametrize("dtype,V,T", [("bf16", 152064, 0.0), ("bf16", 50264, 1.3), ("fp32", 128256, 1.0),
                                       ("bf16", 8200, 0.8), ("fp32", 1000, 1.0), ("bf16", 32000, 1.0)])
def test_row_kernel_variants(tuning, dtype, V, T):
    """Plain loads, per-thread staged copies and the bulk-copy ring give the oracle's round at vocabularies from
    less than one chunk to many trips of every ring depth, with a ragged last chunk."""
    from _harness import run_lockstep
    wl = base(B=10, N=3, k=4, V=V, sigmas=(0.3, 1.0, 2.5)).scaled(dtype=dtype, temperature=T)
    c = report(run_lockstep(wl, rounds=6, seed=V % 89, path=M.PATH_STREAMING, table_mode=True, **tuning))
    assert c["rounds"] == 6 and c["status"] == 0 and c["row_kernel"] == tuning["row_kernel"]
    if T == 0.0:
        assert c["near_tie_accept"] == 0 and c["near_tie_token"] == 0 and c["near_tie_arm"] == 0


@pytest.mark.parametrize("tuning", [dict(row_kernel=M.ROWS_STAGED), dict(row_kernel=M.ROWS_BULK),
                                    dict(row_kernel=M.ROWS_STAGED, row_threads=512, row_stages=4, row_cluster=3)],
                         ids=["staged", "bulk", "staged-cluster3"])
def test_row_kernels_with_per_sequence_draft_lengths_and_odd_logit_scales(tuning):
    """The bulk-copy kernel skips positions behind a sequence's draft length and redoes a draft row whose sum the
    shared reference flushed, like the staged kernel does."""
    from _harness import make_pair, compare_round
    wl = base(B=9, N=1, k=4, V=30000, sigmas=(0.8,)).scaled(temperature=0.9)
    dev = torch.device("cuda", 0)
    gen = RoundGenerator(wl, device=dev, seed=21)
    gpu, orc = make_pair(wl, path=M.PATH_STREAMING, **tuning)
    offsets = torch.tensor([0.0, -150.0, 150.0, -70.0, 70.0, -110.0, 110.0, 20.0, 0.0], device=dev)
    lens = np.array([4, 1, 2, 3, 4, 2, 1, 3, 4], dtype=np.int32)
    lens_dev = torch.from_numpy(lens).to(dev)
    gpu.set_draft_lengths(lens_dev)
    counts = {}
    try:
        for t in range(3):
            arm = orc.select()
            rd = gen.gathered_round(t, arm)
            draft = (rd["draft"].float() + offsets.view(-1, 1, 1)).to(rd["draft"].dtype)
            target = rd["target"].clone()
            for b in range(wl.B):
                target[b, lens[b] + 1:] = float("nan")
                draft[b, lens[b]:] = float("nan")
            res = gpu.verify(target, draft, rd["tokens"], 0.9, 31, want_diag=True)
            out = orc.verify(target, draft, rd["tokens"].cpu().numpy(), 0.9, 31, draft_len=lens)
            assert gpu.last_status() == 0 and (out["status"] == 0).all()
            assert np.array_equal(res.accepted_len.cpu().numpy(), out["accepted_len"])
            np.testing.assert_allclose(res.reward.cpu().numpy(), out["reward"], rtol=0, atol=1e-5)
            D = res.diag_fields()[2].cpu().numpy()
            for b in range(wl.B):
                np.testing.assert_allclose(D[b, :lens[b]], out["D"][b, :lens[b]], rtol=0, atol=1e-5)
            firm = out["sample_margin"] > 1e-6
            assert np.array_equal(res.next_token.cpu().numpy()[firm], out["next_token"][firm])
    finally:
        gpu.close()


@pytest.mark.parametrize("order", ["rank", "reversed", "shuffled"])
@pytest.mark.parametrize("dtype,V", [("bf16", 152064), ("fp32", 50264), ("bf16", 600)])
def test_draw_is_the_oracles_wherever_the_mass_sits(order, dtype, V):
    """The inverse-CDF draw searches the first eighth of the vocabulary (in id order) before it walks the whole row.
    With the likely tokens at the front most draws end in that probe, with the likely tokens at the END of the
    vocabulary (reversed) none does, with shuffled ids about one in eight: the drawn tokens are the oracle's in every
    case (V = 600 is too short for a probe at all)."""
    from _harness import run_lockstep
    wl = base(B=24, N=3, k=3, V=V, sigmas=(0.2, 1.0, 3.0)).scaled(dtype=dtype, temperature=1.0, order=order)
    c = report(run_lockstep(wl, rounds=8, seed=5, path=M.PATH_STREAMING, table_mode=True))
    assert c["rounds"] == 8 and c["status"] == 0


def test_a_device_wait_that_runs_out_sets_the_timeout_bit_and_the_call_still_ends():
    """wait_poll_limit = 1 makes the consumers of the bulk-copy ring give up on the first chunk that has not landed
    when they look: the call ends, the status word carries METASD_STATUS_TIMEOUT (its outputs are undefined), and
    the device keeps working -- a context with the default limit gives the oracle's round right after."""
    from _harness import run_lockstep
    wl = base(B=6, N=2, k=3, V=152064, sigmas=(0.5, 2.0))
    dev = torch.device("cuda", 0)
    gen = RoundGenerator(wl, device=dev, seed=2)
    gpu = M.MetaSD(wl.B, wl.N, wl.k, wl.V, row_kernel=M.ROWS_BULK, wait_poll_limit=1)
    rd = gen.gathered_round(0, np.zeros(wl.B, dtype=np.int64))
    res = gpu.verify(rd["target"], rd["draft"], rd["tokens"], 1.0, 4)
    torch.cuda.synchronize()
    assert gpu.last_status() & M.STATUS_TIMEOUT
    assert res.accepted_len.shape == (wl.B,)
    gpu.reset()
    gpu.close()
    c = run_lockstep(wl, rounds=3, path=M.PATH_STREAMING, row_kernel=M.ROWS_BULK)
    assert c["status"] == 0 and c["rounds"] == 3


def test_state_import_refuses_out_of_range_values_before_they_reach_the_device():
    gpu = M.MetaSD(4, 3, 2, 1024, bandit="swucb", window=6)
    parts = M.parse_state(gpu.state_export(), 4, 3, 6)
    for field, index, value in [("arm", 2, 3), ("arm", 0, -1), ("t", 1, -5), ("win_arm", (3, 5), 99),
                                ("stat_b", (0, 0), float("nan"))]:
        bad = {k: np.array(v, copy=True) for k, v in parts.items()}
        bad[field][index] = value
        with pytest.raises(M.MetasdError) as e:
            gpu.state_import(M.pack_state(bad))
        assert e.value.code == M.ERR_BAD_STATE_BLOB
    gpu.state_import(M.pack_state(parts))            # the untouched blob is accepted
    assert gpu.state_export() == M.pack_state(parts)
    gpu.close()


def test_context_calls_run_on_the_contexts_device_and_leave_the_callers_current_device_alone():
    dev = torch.device("cuda", 0)
    before = torch.cuda.current_device()
    gpu = M.MetaSD(2, 2, 2, 512, device=0)
    gpu.select()
    assert torch.cuda.current_device() == before
    gpu.close()


# ------------------------------------------------------------------------------------------------------------------
# Replay from a CUDA graph
# ------------------------------------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype,T", [("bf16", 0.0), ("fp32", 1.0)])
def test_select_and_verify_replayed_from_a_cuda_graph(dtype, T):
    """metasd_select + metasd_verify neither allocate nor synchronise, and the round counter that keys the random
    numbers lives in the device state: one captured round, replayed on buffers that are refilled in place, gives the
    oracle's rounds one after the other (pointer-table mode, so the bandit's own choice picks the rows)."""
    from _harness import make_pair, compare_round, gather_by_arm
    wl = base(B=12, N=3, k=4, V=16384, sigmas=(0.3, 1.0, 2.5)).scaled(dtype=dtype, temperature=T)
    dev = torch.device("cuda", 0)
    gen = RoundGenerator(wl, device=dev, seed=17)
    gpu, orc = make_pair(wl, path=M.PATH_STREAMING)
    first = gen.table_round(0)
    target, tokens = first["target"].clone(), first["tokens"].clone()
    drafts = [d.clone() for d in first["drafts"]]
    table = M.pointer_table(drafts)
    arm_out = torch.empty(wl.B, dtype=torch.int32, device=dev)
    res = M.VerifyResult(torch.empty(wl.B, dtype=torch.int32, device=dev), torch.empty(wl.B, dtype=torch.int32, device=dev),
                         torch.empty(wl.B, dtype=torch.float32, device=dev))
    res.diag = torch.zeros((wl.B, wl.k, 5), dtype=torch.float32, device=dev)
    counts = {"sequences": wl.B, "near_tie_accept": 0, "near_tie_token": 0, "near_tie_arm": 0}
    try:
        launches_before = gpu.kernel_launches()
        graph = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(torch.cuda.current_stream(dev))
        with torch.cuda.graph(graph, stream=side):
            gpu.select(out=arm_out)
            gpu.verify(target, None, tokens, T, 77, drafter_table=table, token_arm_stride=wl.B * wl.k, out=res)
        torch.cuda.synchronize()
        assert M.parse_state(gpu.state_export(), wl.B, wl.N, wl.tau)["t"].max() == 0, "capturing does not run the round"
        assert gpu.kernel_launches() - launches_before == 3      # select, row statistics, epilogue: the captured round
        for t in range(7):
            rd = gen.table_round(t)
            target.copy_(rd["target"]); tokens.copy_(rd["tokens"])
            for dst, src in zip(drafts, rd["drafts"]):
                dst.copy_(src)
            graph.replay()
            torch.cuda.synchronize()
            arm_o = orc.select()
            assert np.array_equal(arm_out.cpu().numpy(), arm_o)
            draft, tok = gather_by_arm(rd["drafts"], rd["tokens"], arm_o, dev)
            out = orc.verify(rd["target"], None, tok.cpu().numpy(), T, 77, drafter_tables=rd["drafts"])
            out["_reward_kind"] = M.REWARD_BD
            compare_round(res, out, rd["target"], draft, T, 1.0, counts)
        assert gpu.last_status() == 0
        assert np.array_equal(M.parse_state(gpu.state_export(), wl.B, wl.N, wl.tau)["t"], orc.t)
    finally:
        gpu.close()
