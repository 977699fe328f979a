"""The N > 1 path on CPU: two gloo ranks shard a batch, each runs the round on its block with its
`sequence_base`, and the assembled results equal the unsharded run (the float64 oracle stands in for
the GPU here; the GPU twin of this test is test_batch_shard_uses_global_sequence_ids)."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2604_05417_b200.sharding import gather_outputs, reduce_report, shard_range  # noqa: E402
from paper_2604_05417_b200.workloads import RoundGenerator, Workload  # noqa: E402

WL = Workload(name="shard", B=7, N=3, k=3, V=512, rounds=4, temperature=1.0, dtype="bf16", bandit="ducb",
              sigmas=(0.4, 1.2, 2.5), gamma=0.9)


def run_rounds(first, last, rounds):
    """Oracle rounds for sequences [first, last) of the workload; returns per-round outputs."""
    from oracle import oracle as O
    n = last - first
    orc = O.OracleMetaSD(O.OracleConfig(max_batch=n, n_drafters=WL.N, vocab=WL.V, bandit=1, beta=WL.beta, gamma=WL.gamma,
                                        tau=WL.tau, sequence_base=first))
    gen = RoundGenerator(WL, device="cpu", seed=9)
    out = []
    for t in range(rounds):
        arm = orc.select()
        rd = gen.table_round(t)                       # every drafter's rows for all B sequences
        idx = torch.arange(first, last)
        draft = torch.stack(rd["drafts"])[torch.as_tensor(arm, dtype=torch.long), idx]
        tokens = rd["tokens"][torch.as_tensor(arm, dtype=torch.long), idx]
        res = orc.verify(rd["target"][first:last], draft, tokens.numpy(), WL.temperature, 77)
        out.append((arm.copy(), res["accepted_len"].copy(), res["next_token"].copy(), res["reward"].copy()))
    return out


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        lo, hi = shard_range(WL.B, rank, world)
        mine = run_rounds(lo, hi, WL.rounds)
        tokens = sum(int((acc + 1).sum()) for _, acc, _, _ in mine)
        total_tokens, slowest = reduce_report(tokens, 1.0 + rank)
        last = mine[-1]
        gathered = [gather_outputs(torch.as_tensor(x), WL.B).numpy() for x in last]
        if rank == 0:
            q.put((total_tokens, slowest, gathered))
    finally:
        dist.destroy_process_group()


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_shard_range_covers_the_batch_once():
    for batch in (0, 1, 7, 64, 513):
        for world in (1, 2, 3, 8):
            blocks = [shard_range(batch, r, world) for r in range(world)]
            assert blocks[0][0] == 0 and blocks[-1][1] == batch
            assert all(blocks[i][1] == blocks[i + 1][0] for i in range(world - 1))
            sizes = [hi - lo for lo, hi in blocks]
            assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    with pytest.raises(ValueError):
        shard_range(4, 2, 2)


@pytest.mark.timeout(300)
def test_two_gloo_ranks_reproduce_the_unsharded_round():
    world = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    total_tokens, slowest, gathered = q.get(timeout=240)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    full = run_rounds(0, WL.B, WL.rounds)
    assert total_tokens == sum(int((acc + 1).sum()) for _, acc, _, _ in full)
    assert slowest == 2.0                                  # the maximum over ranks, not the sum or rank 0's
    for got, want in zip(gathered, full[-1]):
        assert np.array_equal(got, want)
