#!/usr/bin/env python
"""Benchmark of the MetaSD draft-verify hot path: verified tokens/s and HBM roofline fraction.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

A step is one whole round (select + verify: softmax statistics, accept tests, first rejection,
correction/bonus draw, reward, bandit update, next selection) over one batch of synthetic logits.
Prints ONE JSON line.  With N > 1 (torchrun) every rank runs the same per-GPU batch on its own GPU
(weak scaling, no data-path collective; sequence ids are offset per rank).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2604_05417_b200.workloads import WORKLOADS, RoundGenerator  # noqa: E402

METRIC = "verified_tokens_per_sec"
UNIT = "tokens/s"
DEFAULT_WORKLOAD = "cfg4_greedy"   # the largest-vocabulary configuration: the one the metric is quoted on
LIB_SEED = 20260427


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1500)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--buffers", type=int, default=3, help="distinct pre-generated rounds that the steps cycle through")
    ap.add_argument("--path", default="auto", choices=["auto", "streaming", "fused"])
    ap.add_argument("--e2e-steps", type=int, default=4)
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="CPU work budget of the oracle baseline")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (testing only)")
    ap.add_argument("--k", type=int, default=0, help="override the workload's draft length (the N_max sweep)")
    ap.add_argument("--ragged", action="store_true",
                    help="per-sequence draft lengths, uniform in 1..k (seeded); bytes are counted per sequence")
    return ap.parse_args()


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# DRAM bytes (read + write) of ONE launch of the dominant kernel, from the one-pass ncu capture of the full-size
# launch that profiles/row_stats_staged_kernel.md summarises.  An entry is removed when its kernel changes.
KNOWN_TRAFFIC = {
    ("cfg4_greedy", "streaming"): 3.386e9 + 3.4e6,
    ("cfg5_fp32_stress", "streaming"): 6.735e9 + 3.7e6,
    ("cfg3_tasks", "streaming"): 1.238e9 + 5.9e6,
}


def known_traffic(workload: str, path_name: str):
    return KNOWN_TRAFFIC.get((workload, path_name))


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc, self.thread = index, [], None, None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        def pump():
            for line in self.proc.stdout:
                self.rows.append((time.time(), [x.strip() for x in line.split(",")]))
        self.thread = threading.Thread(target=pump, daemon=True)
        self.thread.start()

    def stop(self, t_begin=0.0, t_end=float("inf")):
        """Median SM clock and the throttle reasons of the samples taken in [t_begin, t_end]."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        if self.thread is not None:
            self.thread.join(timeout=2)
        clocks, reasons, mx = [], set(), None
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        inside = [r for ts, r in self.rows if t_begin <= ts <= t_end]
        for r in (inside or [r for _, r in self.rows[-3:]]):
            try:
                clocks.append(float(r[0]))
                mx = float(r[1])
                for name, val in zip(names, r[2:6]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            except Exception:
                continue
        return {"sm_mhz": statistics.median(clocks) if clocks else None, "sm_max_mhz": mx,
                "reasons": sorted(reasons), "samples": len(clocks)}


def oracle_sample_run(wl, host_rounds, seconds: float):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload's sequences.
    host_rounds: list of (target, draft, tokens) CPU tensors holding at least the sample."""
    from oracle import oracle as O
    cores = O.max_threads()
    avail = host_rounds[0][0].shape[0]

    def run(n_seq, rounds):
        orc = O.OracleMetaSD(O.OracleConfig(max_batch=n_seq, n_drafters=wl.N, vocab=wl.V,
                                            bandit={"ucb": 0, "ducb": 1, "swucb": 2}[wl.bandit], beta=wl.beta,
                                            gamma=wl.gamma, tau=wl.tau))
        tokens = 0
        t0 = time.perf_counter()
        for r in range(rounds):
            tg, dr, tk = host_rounds[r % len(host_rounds)]
            out = orc.verify(tg[:n_seq], dr[:n_seq], tk[:n_seq].numpy(), wl.temperature, LIB_SEED)
            tokens += int((out["accepted_len"] + 1).sum())
        return tokens, time.perf_counter() - t0

    n0 = min(avail, cores)
    _, dt = run(n0, 1)                                   # calibration (also warms the caches)
    wall_per_round = max(dt, 1e-6) * (avail / n0)        # one round of all `avail` sequences
    n_seq = avail
    rounds = int(max(2, min(200, seconds / wall_per_round)))
    tokens, dt = run(n_seq, rounds)
    return {"value": tokens / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "%d sequences x %d rounds of %s (float64, OpenMP over sequences), %.1f s" % (n_seq, rounds, wl.name, dt)}


def main():
    args = parse_args()
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    wl = WORKLOADS[args.workload]
    if args.batch:
        wl = wl.scaled(B=args.batch)
    if args.k:
        wl = wl.scaled(k=args.k)

    if args.impl == "reference":
        return reference_arm(args, wl, rank)

    from paper_2604_05417_b200 import binding as M

    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    path = {"auto": M.PATH_AUTO, "streaming": M.PATH_STREAMING, "fused": M.PATH_FUSED}[args.path]
    msd = M.MetaSD(wl.B, wl.N, wl.k, wl.V, dtype=wl.dtype, bandit=wl.bandit, beta=wl.beta, gamma=wl.gamma,
                   window=wl.tau, device=local_rank, path=path, sequence_base=rank * wl.B)
    path_name = {M.PATH_STREAMING: "streaming", M.PATH_FUSED: "fused"}[msd.resolved_path(wl.k)]

    # ---- inputs: R distinct rounds, every drafter's logits and tokens resident in HBM
    gen = RoundGenerator(wl, device=dev, seed=1000 + rank)
    rounds = []
    for r in range(max(1, args.buffers)):
        rd = gen.table_round(r)
        rd["table"] = M.pointer_table(rd["drafts"])
        rounds.append(rd)
    stride = wl.B * wl.k
    lens = None
    if args.ragged:
        g = torch.Generator().manual_seed(4242 + rank)
        lens = torch.randint(1, wl.k + 1, (wl.B,), generator=g, dtype=torch.int32)
        lens_dev = lens.to(dev)
        msd.set_draft_lengths(lens_dev)
    arm_buf = torch.empty(wl.B, dtype=torch.int32, device=dev)
    n_all = args.warmup + args.steps
    acc_all = torch.zeros((n_all, wl.B), dtype=torch.int32, device=dev)     # every step writes its own slice:
    tok_all = torch.zeros((n_all, wl.B), dtype=torch.int32, device=dev)     # no torch kernel runs inside the
    rew_all = torch.zeros((n_all, wl.B), dtype=torch.float32, device=dev)   # timed region
    outs = [M.VerifyResult(acc_all[i], tok_all[i], rew_all[i]) for i in range(n_all)]

    def step(i):
        rd = rounds[i % len(rounds)]
        msd.select(out=arm_buf)
        msd.verify(rd["target"], None, rd["tokens"], wl.temperature, LIB_SEED, drafter_table=rd["table"],
                   token_arm_stride=stride, out=outs[i])

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    sampler.start()
    for i in range(args.warmup):
        step(i)
    barrier()
    launches0 = msd.kernel_launches()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    host_begin = time.time()
    t_start.record()
    for i in range(args.steps):
        ev[i][0].record()
        step(args.warmup + i)
        ev[i][1].record()
    t_end.record()
    barrier()
    clocks = sampler.stop(host_begin, time.time())
    launches = msd.kernel_launches() - launches0
    total_ms = t_start.elapsed_time(t_end)
    step_ms = [a.elapsed_time(b) for a, b in ev]
    tokens = int(acc_all[args.warmup:].sum().item()) + args.steps * wl.B   # verified tokens: sum(N_acc + 1)

    if world > 1:
        import torch.distributed as dist
        tmax = torch.tensor([total_ms], dtype=torch.float64, device=dev)
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        tok = torch.tensor([tokens], dtype=torch.int64, device=dev)
        dist.all_reduce(tok, op=dist.ReduceOp.SUM)
        total_ms, tokens = float(tmax.item()), int(tok.item())

    # ---- roofline of the dominant kernel: algorithmic logit bytes of one round / its device time
    bytes_round = wl.bytes_per_round
    if lens is not None:   # a sequence reads 2 k_b + 1 rows
        bytes_round = int((2 * lens.to(torch.int64) + 1).sum().item()) * wl.V * (2 if wl.dtype == "bf16" else 4)
    kernel_ms = statistics.mean(step_ms)
    peak, peak_kind = measured_peak_gbs()
    achieved = bytes_round / (kernel_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": known_traffic(wl.name, path_name) if not (args.batch or args.k or args.ragged) else None, "peak_kind": "of " + peak_kind,
                "algorithmic_bytes_per_launch": bytes_round, "kernel_ms": kernel_ms,
                "frac_of_8TBs_nominal": achieved / 8000.0,
                # the same over the first timed steps only: before the power cap pulls the SM clock down
                "first_40_steps": {"kernel_ms": statistics.mean(step_ms[:40]),
                                   "frac": bytes_round / (statistics.mean(step_ms[:40]) * 1e-3) / 1e9 / peak},
                "note": "duration = CUDA events around select+verify of one step (%s path)" % path_name}

    result = {
        "metric": METRIC, "value": tokens / (total_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": wl.name, "B_per_gpu": wl.B, "N": wl.N, "k": wl.k, "V": wl.V, "logits": wl.dtype,
                   "temperature": wl.temperature, "bandit": wl.bandit, "path": path_name,
                   "draft_len": "uniform 1..k per sequence" if args.ragged else "k for every sequence",
                   "l2": "inputs larger than L2: %.2f GB read per step, %d rotating input sets" % (bytes_round / 1e9, len(rounds))},
        "rounds_per_s": world * args.steps / (total_ms * 1e-3),
        "mean_accepted_len": tokens / (world * args.steps * wl.B) - 1.0,
        "roofline": roofline, "gpu_launches": int(launches), "clocks": clocks,
    }

    # ---- end to end through the C ABI with host buffers (copies inside the timed region)
    if not args.no_e2e:
        result["e2e"] = e2e_run(args, wl, M, msd, rounds, dev, world, rank)
    # ---- the CPU oracle on this machine's host cores (rank 0, N = 1 only)
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        n = min(wl.B, 256)
        arm0 = rounds[0]["sigma"].argmin(axis=1)
        host = []
        for rd in rounds[:2]:
            idx = torch.as_tensor(arm0[:n], device=dev, dtype=torch.long)
            draft = torch.stack([d[:n] for d in rd["drafts"]])[idx, torch.arange(n, device=dev)]
            toks = rd["tokens"][:, :n][idx, torch.arange(n, device=dev)]
            host.append((rd["target"][:n].cpu(), draft.cpu(), toks.cpu()))
        result["cpu_baseline"] = oracle_sample_run(wl, host, args.cpu_seconds)
    msd.close()
    if rank == 0:
        print(json.dumps(result))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def e2e_run(args, wl, M, msd_dev, rounds, dev, world, rank):
    """The same metric through metasd_verify_host: pinned host logits in, results out, every step."""
    n_steps = max(1, args.e2e_steps)
    msd = M.MetaSD(wl.B, wl.N, wl.k, wl.V, dtype=wl.dtype, bandit=wl.bandit, beta=wl.beta, gamma=wl.gamma,
                   window=wl.tau, device=dev.index, sequence_base=rank * wl.B, host_staging=True)
    # host copies of one round per buffer, draft rows gathered for the best drafter of each sequence
    host = []
    for rd in rounds[:2]:
        arm = torch.as_tensor(rd["sigma"].argmin(axis=1), device=dev, dtype=torch.long)
        ar = torch.arange(wl.B, device=dev)
        draft = torch.stack(rd["drafts"])[arm, ar]
        toks = rd["tokens"][arm, ar]
        host.append(tuple(x.cpu().pin_memory() for x in (rd["target"], draft, toks)))
        del draft
    acc = torch.zeros(wl.B, dtype=torch.int32).pin_memory()
    tok = torch.zeros(wl.B, dtype=torch.int32).pin_memory()
    rew = torch.zeros(wl.B, dtype=torch.float32).pin_memory()
    nxt = torch.zeros(wl.B, dtype=torch.int32).pin_memory()
    msd.verify_host(*host[0], wl.temperature, LIB_SEED, acc, tok, rew, nxt)     # warm-up
    torch.cuda.synchronize()
    tokens = 0
    t0 = time.perf_counter()
    for i in range(n_steps):
        msd.verify_host(*host[i % len(host)], wl.temperature, LIB_SEED, acc, tok, rew, nxt)
        tokens += int(acc.sum()) + wl.B
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    if world > 1:
        import torch.distributed as dist
        tmax = torch.tensor([dt], dtype=torch.float64, device=dev)
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        tk = torch.tensor([tokens], dtype=torch.int64, device=dev)
        dist.all_reduce(tk, op=dist.ReduceOp.SUM)
        dt, tokens = float(tmax.item()), int(tk.item())
    h2d = sum(x.numel() * x.element_size() for x in host[0])
    d2h = sum(x.numel() * x.element_size() for x in (acc, tok, rew, nxt))
    msd.close()
    return {"value": tokens / dt, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
            "steps": n_steps, "ms_per_step": dt / n_steps * 1e3,
            "note": "metasd_verify_host: pinned host logits -> device staging -> kernels -> host results"}


def reference_arm(args, wl, rank):
    """--impl reference: the CPU oracle as it stands on this machine's host cores (rank 0 only)."""
    if rank != 0:
        return
    from oracle import oracle as O
    n = min(wl.B, 4 * O.max_threads())
    small = wl.scaled(B=n)
    gen = RoundGenerator(small, device="cpu", seed=1000)
    host = []
    for r in range(2):
        rd = gen.gathered_round(r, gen.best_arm(r))
        host.append((rd["target"], rd["draft"], rd["tokens"]))
    orc = O.OracleMetaSD(O.OracleConfig(max_batch=n, n_drafters=wl.N, vocab=wl.V,
                                        bandit={"ucb": 0, "ducb": 1, "swucb": 2}[wl.bandit], beta=wl.beta,
                                        gamma=wl.gamma, tau=wl.tau))
    def step(i):
        tg, dr, tk = host[i % 2]
        out = orc.verify(tg, dr, tk.numpy(), wl.temperature, LIB_SEED)
        return int((out["accepted_len"] + 1).sum())
    for i in range(min(args.warmup, 1)):
        step(i)
    steps = max(1, min(args.steps, 8))
    tokens = 0
    t0 = time.perf_counter()
    for i in range(steps):
        tokens += step(i)
    dt = time.perf_counter() - t0
    value = tokens / dt
    sample = "%d of %d sequences per step, %d steps, float64 oracle with OpenMP over sequences" % (n, wl.B, steps)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": min(args.warmup, 1), "ms_per_step": dt / steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": wl.name, "B_per_gpu": wl.B, "N": wl.N, "k": wl.k, "V": wl.V, "logits": wl.dtype,
                   "temperature": wl.temperature, "bandit": wl.bandit, "path": "cpu-oracle", "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": O.max_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


if __name__ == "__main__":
    main()
