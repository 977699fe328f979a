"""The allocation-free entry point against the context-based one (runs last in the collection order).

`metasd_verify_noalloc` exists for callers that cannot call cudaMalloc -- a serving loop whose pool
owns the device, a plugin that may not allocate after start-up -- and therefore cannot create a
context.  Its scratch is a fixed array inside the library.  This test drives it through the C ABI on
two consecutive rounds and checks that it returns what `metasd_verify` returns for the same inputs,
seed, sequence ids and round counters, and what the float64 CPU oracle computes for them: integers
exactly (a sampled decision may differ only where the oracle itself marks it a near tie, as in the
parity tests), the reward within the 1e-5 the parity tests use.  It builds its own contexts and inputs,
so it passes alone in a fresh process as well as after the rest of the suite.
"""
import numpy as np
import pytest
import torch

from paper_2604_05417_b200 import binding as M
from paper_2604_05417_b200.workloads import RoundGenerator, Workload

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,temperature,V", [("bf16", 1.0, 20008), ("fp32", 0.0, 4100), ("bf16", 0.7, 1001)])
def test_noalloc_matches_context_call_on_two_rounds(dtype, temperature, V):
    wl = Workload(name="noalloc", B=6, N=1, k=4, V=V, rounds=2, temperature=temperature, dtype=dtype,
                  bandit="ucb", sigmas=(1.0,))
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    gen = RoundGenerator(wl, device=dev, seed=17)
    from oracle import oracle as O
    ctx = M.MetaSD(wl.B, 1, wl.k, V, dtype=dtype, path=M.PATH_STREAMING, sequence_base=40)
    orc = O.OracleMetaSD(O.OracleConfig(max_batch=wl.B, n_drafters=1, vocab=V, sequence_base=40))
    acc = torch.full((wl.B,), -9, dtype=torch.int32, device=dev)
    tok = torch.full((wl.B,), -9, dtype=torch.int32, device=dev)
    rew = torch.full((wl.B,), -9.0, dtype=torch.float32, device=dev)
    status = torch.full((1,), 99, dtype=torch.int32, device=dev)
    for t in range(2):                                   # two calls in a row share the library's scratch
        rd = gen.gathered_round(t, np.zeros(wl.B, dtype=np.int64))
        want = ctx.verify(rd["target"], rd["draft"], rd["tokens"], temperature, 31337)
        rc = M.verify_noalloc(rd["target"], rd["draft"], rd["tokens"], temperature, 31337, t, acc, tok, rew,
                              status=status, sequence_base=40)
        assert rc == M.OK
        torch.cuda.synchronize()
        out = orc.verify(rd["target"], rd["draft"], rd["tokens"].cpu().numpy(), temperature, 31337)
        assert (out["round"] == t).all()
        with np.errstate(divide="ignore", invalid="ignore"):
            firm = ~(np.abs(out["u_accept"] - out["p_x"] / out["q_x"]) < 1e-6).any(axis=1)
        if temperature == 0:
            firm[:] = True
        firm_t = torch.from_numpy(firm).to(dev)
        assert torch.equal(acc[firm_t], want.accepted_len[firm_t])
        assert np.array_equal(acc.cpu().numpy()[firm], out["accepted_len"][firm])
        if temperature > 0:
            firm &= out["sample_margin"] > 1e-6
            firm_t = torch.from_numpy(firm).to(dev)
        assert torch.equal(tok[firm_t], want.next_token[firm_t])
        assert np.array_equal(tok.cpu().numpy()[firm], out["next_token"][firm])
        assert firm.sum() >= wl.B - 1
        assert torch.allclose(rew, want.reward, rtol=0, atol=1e-5)
        np.testing.assert_allclose(rew.cpu().numpy(), out["reward"], rtol=0, atol=1e-5)
        assert status.item() == ctx.last_status()
    ctx.close()


def test_noalloc_rejects_sizes_beyond_its_fixed_scratch():
    dev = torch.device("cuda", 0)
    z = torch.zeros(8, dtype=torch.int32, device=dev)
    lib = M.load_library()
    import ctypes as C

    def call(batch, k, vocab=64):
        return lib.metasd_verify_noalloc(batch, k, vocab, M.BF16, M._ptr(z), M._ptr(z), M._ptr(z), C.c_float(1.0),
                                         C.c_float(1.0), M.REWARD_BD, C.c_uint64(0), 0, 0, M._ptr(z), M._ptr(z),
                                         M._ptr(z), None, None)
    assert call(4097, 1) == M.ERR_UNSUPPORTED            # more sequences than METASD_NOALLOC_MAX_BATCH
    assert call(2048, 8) == M.ERR_UNSUPPORTED            # 2048 * 9 rows > METASD_NOALLOC_MAX_ROWS
    assert call(0, 1) == M.ERR_INVALID_ARGUMENT
    assert call(4, 17) == M.ERR_INVALID_ARGUMENT
    torch.cuda.synchronize()
