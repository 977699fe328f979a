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
    ap.add_argument("--row-kernel", default="auto", choices=["auto", "plain", "staged", "bulk"])
    ap.add_argument("--row-threads", type=int, default=0)
    ap.add_argument("--row-stages", type=int, default=0)
    ap.add_argument("--row-cluster", type=int, default=0, help="CTAs that share one row pair (staged row kernel)")
    ap.add_argument("--keep-permille", type=int, default=0)
    ap.add_argument("--graph", action="store_true",
                    help="capture every step (select + verify) into a CUDA graph before the timed region and replay it there")
    ap.add_argument("--order", default="rank", choices=["rank", "reversed", "shuffled"],
                    help="where the likely tokens sit in the vocabulary (the draw walks it in id order)")
    ap.add_argument("--sustained-seconds", type=float, default=1.0,
                    help="length of the extra back-to-back leg that is run when the timed region is under half a second")
    ap.add_argument("--no-parity", action="store_true")
    return ap.parse_args()


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def known_traffic(kernel_key: str, workload: str):
    """DRAM bytes (read + write) of one launch of the dominant kernel from the committed ncu capture of exactly this
    kernel variant on this workload, or None when there is no such capture (a changed variant has another key)."""
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.txt")) as f:
            for line in f:
                parts = line.split()
                if len(parts) == 3 and not line.startswith("#") and parts[0] == kernel_key and parts[1] == workload:
                    return float(parts[2])
    except Exception:
        pass
    return None


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
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        def pump():
            for line in self.proc.stdout:
                self.rows.append((time.time(), [x.strip() for x in line.split(",")]))
        self.thread = threading.Thread(target=pump, daemon=True)
        self.thread.start()

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        if self.thread is not None:
            self.thread.join(timeout=2)
        self.proc = None

    def window(self, t_begin, t_end):
        """Median SM clock and the throttle reasons of the samples taken in [t_begin, t_end]; a region shorter than
        the sampling period takes the samples on either side of it."""
        if not self.rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        clocks, reasons, mx = [], set(), None
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        inside = [r for ts, r in self.rows if t_begin <= ts <= t_end]
        if not inside:
            before = [r for ts, r in self.rows if ts < t_begin][-1:]
            after = [r for ts, r in self.rows if ts > t_end][:1]
            inside = before + after
        for r in inside:
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
        tokens, outs = 0, []
        t0 = time.perf_counter()
        for r in range(rounds):
            tg, dr, tk = host_rounds[r % len(host_rounds)]
            out = orc.verify(tg[:n_seq], dr[:n_seq], tk[:n_seq].numpy(), wl.temperature, LIB_SEED)
            tokens += int((out["accepted_len"] + 1).sum())
            outs.append(out)
        return tokens, time.perf_counter() - t0, outs

    n0 = min(avail, cores)
    _, dt, _ = run(n0, 1)                                # calibration (also warms the caches)
    wall_per_round = max(dt, 1e-6) * (avail / n0)        # one round of all `avail` sequences
    n_seq = avail
    rounds = int(max(2, min(200, seconds / wall_per_round)))
    tokens, dt, outs = run(n_seq, rounds)
    return {"value": tokens / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "%d sequences x %d rounds of %s (float64, OpenMP over sequences), %.1f s" % (n_seq, rounds, wl.name, dt)}, outs


def parity_against_oracle(wl, M, host_rounds, outs, dev, tuning):
    """The library on the very rounds the CPU-baseline leg gave the oracle (outside every timed region): what differs,
    counted by the comparison rules of the parity tests.  Integers must agree except at the oracle's own near ties
    (uniform within 1e-6 of p/q; CDF margin below 1e-6; index gap below 1e-6), floats within 1e-5.
    This leg feeds every sequence the rows of one fixed drafter whatever arm its bandit picks (the oracle cannot hold
    all K drafters' rows of 256 sequences on the host), so the arms earn identical rewards and their indices tie far
    more often than in real use.  A sequence whose arm differs at such a tie is counted once (near_tie_arm) and its
    later arm choices are left out, since the two bandits then hold different statistics; every other output is
    independent of the arm here and stays in the comparison."""
    import numpy as np
    n = outs[0]["accepted_len"].shape[0]
    gpu = M.MetaSD(n, wl.N, wl.k, wl.V, dtype=wl.dtype, bandit=wl.bandit, beta=wl.beta, gamma=wl.gamma, window=wl.tau,
                   device=dev.index, **tuning)
    dev_rounds = [tuple(x[:n].to(dev) for x in hr) for hr in host_rounds]
    rep = {"sequences": n, "rounds": len(outs), "near_tie_accept": 0, "near_tie_token": 0, "near_tie_arm": 0,
           "mismatch_accept": 0, "mismatch_token": 0, "mismatch_arm": 0, "max_err_D": 0.0, "max_err_p": 0.0,
           "max_err_reward": 0.0, "uniforms_identical": True}
    greedy = not (wl.temperature > 0)
    in_step = np.ones(n, dtype=bool)       # sequences whose two bandits still hold the same statistics
    for r, out in enumerate(outs):
        tg, dr, tk = dev_rounds[r % len(dev_rounds)]
        arm_g = gpu.select().cpu().numpy()
        differs = (arm_g != out["arm"]) & in_step
        # a stored gap belongs to the selection that FOLLOWED the previous round
        near = differs & (outs[r - 1]["next_gap"] < 1e-6) if r else np.zeros(n, dtype=bool)
        rep["near_tie_arm"] += int(near.sum())
        rep["mismatch_arm"] += int((differs & ~near).sum())
        in_step &= ~differs
        res = gpu.verify(tg, dr, tk, wl.temperature, LIB_SEED, want_diag=True)
        p_x, q_x, D, u, acc = [x.cpu().numpy() for x in res.diag_fields()]
        rep["uniforms_identical"] &= bool(np.array_equal(u.astype(np.float64), out["u_accept"]))
        rep["max_err_D"] = max(rep["max_err_D"], float(np.abs(D - out["D"]).max()))
        rep["max_err_p"] = max(rep["max_err_p"], float(np.abs(p_x - out["p_x"]).max()), float(np.abs(q_x - out["q_x"]).max()))
        rep["max_err_reward"] = max(rep["max_err_reward"], float(np.abs(res.reward.cpu().numpy() - out["reward"]).max()))
        bits = acc != out["accept"]
        with np.errstate(divide="ignore", invalid="ignore"):
            tie = np.abs(out["u_accept"] - out["p_x"] / out["q_x"]) < 1e-6
        rep["near_tie_accept"] += int((bits & tie).sum())
        rep["mismatch_accept"] += int((bits & ~tie).sum())
        same_len = res.accepted_len.cpu().numpy() == out["accepted_len"]
        rep["mismatch_accept"] += int((~same_len & ~bits.any(axis=1)).sum())
        tok = (res.next_token.cpu().numpy() != out["next_token"]) & same_len
        edge = tok & (out["sample_margin"] < 1e-6) & (not greedy)
        rep["near_tie_token"] += int(edge.sum())
        rep["mismatch_token"] += int((tok & ~edge).sum())
    rep["status"] = gpu.last_status()
    rep["arm_sequences_compared_to_the_end"] = int(in_step.sum())
    gpu.close()
    rep["ok"] = bool(rep["mismatch_accept"] == 0 and rep["mismatch_token"] == 0 and rep["mismatch_arm"] == 0 and
                     rep["uniforms_identical"] and max(rep["max_err_D"], rep["max_err_p"], rep["max_err_reward"]) < 1e-5)
    return rep


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
    if args.order != "rank":
        wl = wl.scaled(order=args.order)

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
    tuning = dict(row_kernel={"auto": M.ROWS_AUTO, "plain": M.ROWS_PLAIN, "staged": M.ROWS_STAGED, "bulk": M.ROWS_BULK}[args.row_kernel],
                  row_threads=args.row_threads, row_stages=args.row_stages, keep_permille=args.keep_permille,
                  row_cluster=args.row_cluster)
    msd = M.MetaSD(wl.B, wl.N, wl.k, wl.V, dtype=wl.dtype, bandit=wl.bandit, beta=wl.beta, gamma=wl.gamma,
                   window=wl.tau, device=local_rank, path=path, sequence_base=rank * wl.B, **tuning)
    path_name = {M.PATH_STREAMING: "streaming", M.PATH_FUSED: "fused"}[msd.resolved_path(wl.k)]
    row_kernel = {M.ROWS_PLAIN: "plain", M.ROWS_STAGED: "staged", M.ROWS_BULK: "bulk"}[msd.resolved_row_kernel()]
    # names the dominant kernel's variant: a capture of DRAM traffic counts only for the variant it was taken on
    kernel_key = path_name if path_name == "fused" else "%s/%s/t%d/s%d/keep%d" % (
        row_kernel, wl.dtype, args.row_threads, args.row_stages, args.keep_permille)
    if args.row_cluster > 1:
        kernel_key += "/c%d" % args.row_cluster

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

    def launch_step(i):
        rd = rounds[i % len(rounds)]
        msd.select(out=arm_buf)
        msd.verify(rd["target"], None, rd["tokens"], wl.temperature, LIB_SEED, drafter_table=rd["table"],
                   token_arm_stride=stride, out=outs[i])

    step, graphs = launch_step, []
    if args.graph:
        # neither call allocates or synchronises and the round counter lives in the device state, so a captured step
        # replays as the next round; one graph per step because every step writes its own output slice
        side = torch.cuda.Stream(device=dev)
        side.wait_stream(torch.cuda.current_stream(dev))
        before = msd.kernel_launches()
        for i in range(n_all):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                launch_step(i)
            graphs.append(g)
        torch.cuda.synchronize()
        launches_per_step = (msd.kernel_launches() - before) // n_all
        step = lambda i: graphs[i].replay()

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
    host_end = time.time()
    launches = launches_per_step * args.steps if args.graph else msd.kernel_launches() - launches0
    # ---- a timed region under half a second says little about sustained rounds (the power cap acts after a few
    # hundred milliseconds): run an extra leg of back-to-back rounds and report it beside the timed one
    sustained = None
    if t_start.elapsed_time(t_end) < 500.0 and args.sustained_seconds > 0:
        per_step = max(t_start.elapsed_time(t_end) / args.steps, 1e-3)
        n_sus = int(min(20000, max(args.steps, args.sustained_seconds * 1e3 / per_step)))
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        sus_begin = time.time()
        s0.record()
        for i in range(n_sus):
            step(i % n_all)
        s1.record()
        barrier()
        sus_end = time.time()
        sustained = {"steps": n_sus, "kernel_ms": s0.elapsed_time(s1) / n_sus, "window": (sus_begin, sus_end)}
    time.sleep(0.05)
    sampler.stop()
    clocks = sampler.window(host_begin, host_end)
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
                "traffic": known_traffic(kernel_key, wl.name) if not (args.batch or args.k or args.ragged) else None,
                "traffic_key": kernel_key, "peak_kind": "of " + peak_kind,
                "algorithmic_bytes_per_launch": bytes_round, "kernel_ms": kernel_ms,
                "frac_of_8TBs_nominal": achieved / 8000.0,
                # the same over the first timed steps only: before the power cap pulls the SM clock down
                "first_40_steps": {"kernel_ms": statistics.mean(step_ms[:40]),
                                   "frac": bytes_round / (statistics.mean(step_ms[:40]) * 1e-3) / 1e9 / peak},
                "note": "duration = CUDA events around select+verify of one step (%s path, %s row kernel)" % (path_name, row_kernel)}
    if sustained is not None:
        ms = sustained["kernel_ms"]
        roofline["sustained"] = {"steps": sustained["steps"], "kernel_ms": ms, "frac": bytes_round / (ms * 1e-3) / 1e9 / peak,
                                 "clocks": sampler.window(*sustained["window"])}

    result = {
        "metric": METRIC, "value": tokens / (total_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": wl.name, "B_per_gpu": wl.B, "N": wl.N, "k": wl.k, "V": wl.V, "logits": wl.dtype,
                   "temperature": wl.temperature, "bandit": wl.bandit, "path": path_name, "row_kernel": row_kernel,
                   "vocab_order": wl.order, "launch": "cuda graph replay, one graph per step" if args.graph else "stream launches",
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
        result["cpu_baseline"], outs = oracle_sample_run(wl, host, args.cpu_seconds)
        if not args.no_parity:
            result["parity"] = parity_against_oracle(wl, M, host, outs, dev, tuning)
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
