#!/usr/bin/env python
"""Benchmark of the batched speculative-verification round (one JSON line on stdout).

A step is one pass of the whole hot path over one batch of synthetic input:
  bs_bandit_select -> bs_softmax_verify -> bs_residual_sample -> bs_bandit_update
captured as one CUDA graph per input set.  Inputs rotate through a ring of distinct sets
whose total size exceeds twice the L2, so every step reads its logits from HBM.

  value      rounds/s with the inputs resident in HBM (whole job, all ranks)
  e2e        the same round driven from pinned HOST buffers: the step's logits, tokens and
             uniforms are copied to the device and the emitted tokens read back inside the
             timed region
  roofline   bs_softmax_verify's kernel: algorithmic bytes (every valid logit once) divided by
             its mean duration between CUDA events on the launching stream
  cpu_baseline  the CPU oracle, as it stands, on a bounded sample of the same workload

`--impl reference` times the CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "batched spec-verify rounds/sec"
UNIT = "rounds/s"
L2_BYTES = 126 * 1024 * 1024
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) of one launch of the dominant kernel,
# from profiler captures of smaller cases of the same kernels: (read traffic per algorithmic byte,
# bytes written per launch).  Read traffic grows with the bytes, the writes (workspace partials,
# write-backs) do not.  An entry is only valid for the kernel it was captured on: when that kernel
# changes, the entry goes to None until the capture is repeated.
NCU_TRAFFIC = {
    "qwen_exp3": (1.0003, 4.1e6),          # fp32 statistics kernel, captured at B=32
    "llama3_ucb": (1.0005, 3.9e6),         # bf16 statistics kernel
    "llama3_tree": (1.0004, 4.5e6),        # the same kernel in greedy mode
    "lmhead_llama3": (1.0000, 30.6e6),     # B=16 (logits still dirty in L2 are not counted)
    "lmhead_llama3_b128": (1.0180, 568.1e6),
}


HOLD_CYCLES = 400_000          # about 0.2 ms of a spinning kernel


def hold_gpu():
    """Keeps the stream busy while the host enqueues the events and launches that follow, so that an event
    pair brackets the kernel's own duration and not the host's time between two enqueue calls (which
    shows once a launch is shorter than the host needs to issue it)."""
    import torch
    torch.cuda._sleep(HOLD_CYCLES)


def ncu_traffic(name: str, algorithmic_read_bytes: float):
    t = NCU_TRAFFIC.get(name)
    return None if t is None else t[0] * algorithmic_read_bytes + t[1]


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--workload", default="qwen_exp3",
                    choices=["tiny_ucb", "llama2_fixed", "llama3_ucb", "qwen_exp3", "llama3_tput", "lmhead_llama3",
                             "lmhead_llama3_b128", "llama3_tree", "tiny_tree"])
    ap.add_argument("--batch", type=int, default=0,
                    help="override the workload's batch size (smaller cases for profiler captures)")
    ap.add_argument("--fixed-gamma", type=int, default=0,
                    help="replace the workload's arms by one arm of this speculation length, so that the bytes "
                         "of every launch are known exactly (profiler captures)")
    ap.add_argument("--drafted", action="store_true",
                    help="the round with drafting on the device: select -> bs_draft_sample per position -> "
                         "bs_softmax_verify_drafted -> bs_residual_sample -> update")
    ap.add_argument("--walk", action="store_true",
                    help="the round with early exit: select -> bs_verify_walk (verification up to the first "
                         "rejection + resampling in one launch) -> update")
    ap.add_argument("--auto-path", action="store_true",
                    help="time a few rounds of the two-call path and of the early-exit path first and run the timed "
                         "region on the faster one (config.path says which); early exit emits the same tokens but forms "
                         "the token probabilities only up to the first rejection")
    ap.add_argument("--no-others", action="store_true",
                    help="skip the short runs of the other workloads that the default invocation adds to its line")
    ap.add_argument("--bandit-step", action="store_true",
                    help="one bs_bandit_step per round (update + next round's select) instead of bs_bandit_select "
                         "and bs_bandit_update; measured: no faster, the two small launches already overlap")
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=4)
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="budget of the CPU-oracle sample")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-all-cores", action="store_true",
                    help="also time the oracle sample in one single-threaded process per host core")
    ap.add_argument("--oracle-worker", action="store_true", help=argparse.SUPPRESS)
    ap.add_argument("--no-graph", action="store_true", help="launch the four calls directly each step")
    return ap.parse_args()


def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:
        return os.cpu_count() or 1


# ---------------------------------------------------------------------------------------------
# CPU oracle timing (cpu_baseline leg and --impl reference)
# ---------------------------------------------------------------------------------------------

ORACLE_SAMPLE_SEQS = 16        # sequences of round 1 that both CPU legs time, over and over


def oracle_inputs(w):
    """The bounded sample both CPU legs time: the first sequences of round 1 with the arms that shape
    the benchmark's first input set, generated on the host and converted to the oracle's input arrays
    before any clock starts."""
    from paper_2505_15141_b200 import workloads as wl
    nb = min(w.B, ORACLE_SAMPLE_SEQS)
    rnd = wl.make_round(w, 1, default_arms(w, 0), device="cpu", B=nb)
    toks = rnd.tokens.cpu().numpy()
    seqs = []
    for b in range(nb):
        g = int(rnd.gamma[b])
        seqs.append((rnd.target[b, :g + 1].float().numpy(), rnd.draft[b, :g].float().numpy(), toks[b], g,
                     rnd.uniforms.u_accept[b], float(rnd.uniforms.u_resample[b])))
    return seqs


def oracle_sample(w, seqs, seconds: float):
    """Runs the oracle's verification over the sample, again and again, until `seconds` are used.
    Returns (sequences done, elapsed seconds)."""
    from oracle import verify as ov
    done, t0 = 0, time.perf_counter()
    while True:
        t_rows, d_rows, toks, g, u_acc, u_res = seqs[done % len(seqs)]
        ov.verify_sequence(t_rows, d_rows, toks, g, u_acc, u_res, w.temperature)
        done += 1
        if time.perf_counter() - t0 > seconds:
            break
    return done, time.perf_counter() - t0


def oracle_worker(args, w):
    """One process of the all-core figure: times its own copy of the sample, prints wall-clock marks."""
    import torch
    torch.set_num_threads(1)
    seqs = oracle_inputs(w)
    t0 = time.time()
    n, _ = oracle_sample(w, seqs, args.cpu_seconds)
    print(json.dumps({"seqs": n, "t0": t0, "t1": time.time()}))


def oracle_all_cores(args, w, cores: int):
    """The same sample in `cores` single-threaded processes at once (sequences are independent, so the
    oracle parallelises over them and over nothing else).  Rounds/s = all sequences done, over the span
    from the first start to the last end.  Every child has a hard limit; stragglers are killed by PID."""
    cmd = [sys.executable, os.path.abspath(__file__), "--impl", "reference", "--oracle-worker", "--workload", w.name,
           "--cpu-seconds", str(args.cpu_seconds)]
    if args.batch:
        cmd += ["--batch", str(args.batch)]
    if args.fixed_gamma:
        cmd += ["--fixed-gamma", str(args.fixed_gamma)]
    env = dict(os.environ, OMP_NUM_THREADS="1", MKL_NUM_THREADS="1", CUDA_VISIBLE_DEVICES="")
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        env.pop(k, None)
    procs = [subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True, env=env)
             for _ in range(cores)]
    deadline = time.time() + args.cpu_seconds + 240.0
    marks = []
    for pr in procs:
        try:
            out, _ = pr.communicate(timeout=max(1.0, deadline - time.time()))
            marks.append(json.loads(out.strip().splitlines()[-1]))
        except Exception:
            pr.kill()
    if not marks:
        return None
    span = max(m["t1"] for m in marks) - min(m["t0"] for m in marks)
    n = sum(m["seqs"] for m in marks)
    return {"value": (n / w.B) / span, "unit": UNIT, "cores": len(marks),
            "sample": f"{n} sequences in {len(marks)} single-threaded processes over {span:.1f} s"}


def rank_round_index(rank: int, i: int) -> int:
    """Round number that seeds input set i of a rank: every rank verifies its own batches."""
    return 1 + i + 1000 * rank


def reduce_over_ranks(ms: float, nbytes: float, device):
    """Whole-job timing: the slowest rank's time (MAX) and the bytes of all ranks (SUM).
    Sequences are independent, so this is the only exchange between ranks."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms), float(nbytes)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    b = torch.tensor([nbytes], dtype=torch.float64, device=device)
    dist.all_reduce(b, op=dist.ReduceOp.SUM)
    return float(t.item()), float(b.item())


def job_rounds_per_s(world: int, steps: int, ms: float) -> float:
    """Each rank completes `steps` rounds of its own batch in the common time `ms`."""
    return world * steps / (ms * 1e-3)


def default_arms(w, step: int) -> np.ndarray:
    """Arms used to shape the pre-generated inputs (the device bandit picks its own gamma)."""
    return ((np.arange(w.B) + step) % w.K).astype(np.int32)


def run_reference(args, w):
    """The oracle, as it stands, on the host cores: each step is a bounded sample of one round (the
    same sample the CUDA arm's cpu_baseline leg times)."""
    import torch
    torch.set_num_threads(1)
    per_step = max(0.2, min(10.0, 90.0 / max(1, args.steps + args.warmup), args.cpu_seconds))
    seqs_in = oracle_inputs(w)
    times, seqs = [], []
    for i in range(args.warmup + args.steps):
        n, dt = oracle_sample(w, seqs_in, per_step)
        if i >= args.warmup:
            times.append(dt); seqs.append(n)
    rounds = sum(seqs) / w.B
    total = sum(times)
    val = rounds / total
    world = int(os.environ.get("WORLD_SIZE", "1"))
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / max(1, args.steps),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": cpu_config(w),
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": f"{sum(seqs)} verifications of the first {len(seqs_in)} sequences of a "
                                   f"{w.B}-sequence round in {total:.1f} s, verification only (numpy fp64, one "
                                   f"thread; rank 0 of {world} runs it, the others idle)"},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def cpu_config(w) -> dict:
    """The workload keys both arms print."""
    return {"workload": w.name, "B": w.B, "V": w.V, "arm_gamma": list(w.arm_gamma), "bandit": w.alg or "fixed",
            "logits_dtype": w.dtype, "temperature": w.temperature}


# ---------------------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------------------

class ClockSampler:
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def stop(self) -> dict:
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()                    # the exact child started above
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for name, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ---------------------------------------------------------------------------------------------
# CUDA arm
# ---------------------------------------------------------------------------------------------

def run_cuda(args, w):
    import torch
    import torch.distributed as dist
    import __graft_entry__ as entry

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group(backend="nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if rank == 0:
        entry.build()
    if world > 1:
        dist.barrier()
    from paper_2505_15141_b200 import binding as bs, workloads as wl

    B, K, G, V = w.B, w.K, w.Gmax, w.V
    alg = {"exp3": bs.BS_EXP3, "ucb_reward": bs.BS_UCB_REWARD}.get(w.alg, bs.BS_UCB)   # a fixed arm is a 1-armed UCBSpec
    reward = w.alg == "ucb_reward"
    es = w.elem_size
    arm_gamma = np.asarray(w.arm_gamma)

    # ---- ring of input sets, > 2 x L2 in total ----
    set_bytes = es * V * B * (2 * G + 1)
    ring = max(2, -(-2 * L2_BYTES // set_bytes) + 1)
    sets = []
    for i in range(ring):
        rnd = wl.make_round(w, rank_round_index(rank, i), default_arms(w, i), device=dev)
        sets.append(dict(
            target=rnd.target, draft=rnd.draft, tokens=rnd.tokens.contiguous(),
            u_accept=torch.as_tensor(rnd.uniforms.u_accept, device=dev),
            u_resample=torch.as_tensor(rnd.uniforms.u_resample, device=dev),
            u_arm=torch.as_tensor(rnd.uniforms.u_arm, device=dev),
            u_draft=torch.as_tensor(rnd.uniforms.u_draft, device=dev), rnd=rnd))
    state = bs.new_bandit(alg, B, w.arm_gamma, w.delta, dev, reward_width=w.reward_width if reward else None)
    ws = bs.new_workspace(B, G, V, dev)
    reward_d = torch.zeros(B, dtype=torch.float64, device=dev)
    # Throughput reward: a serving loop passes the duration it measured for the step; the arms are chosen on
    # the device here and never read back inside the timed region, so the duration is one constant, the
    # workload's stand-in for a step at the longest speculation length.
    step_s = wl.step_seconds(w, arm_gamma) if reward else None

    def update_call():
        if reward:
            bs.bs_throughput_reward(out_len, None, B, step_s, w.whole_batch, reward_d)
            bs.bs_bandit_update_reward(state, B, K, arm_d, reward_d)
        else:
            bs.bs_bandit_update(state, alg, B, K, arm_d, out_len)

    fused_bandit = args.bandit_step

    def step_bandit_call(s_next):
        """History step of this round and select step of the next (whose uniforms are s_next's) in one launch."""
        if reward:
            bs.bs_throughput_reward(out_len, None, B, step_s, w.whole_batch, reward_d)
            bs.bs_bandit_step(state, alg, B, K, reward_d, None, None, arm_d, gamma_d)
        else:
            bs.bs_bandit_step(state, alg, B, K, out_len, s_next["u_arm"], None, arm_d, gamma_d)

    def init_call():
        if reward:
            bs.bs_bandit_init_reward(state, B, K, w.arm_gamma, w.delta, w.reward_width)
        else:
            bs.bs_bandit_init(state, alg, B, K, w.arm_gamma, w.delta)
    arm_d = torch.zeros(B, dtype=torch.int32, device=dev)
    gamma_d = torch.zeros(B, dtype=torch.int32, device=dev)
    accept_len = torch.zeros(B, dtype=torch.int32, device=dev)
    p_tok = torch.zeros(B, G, dtype=torch.float32, device=dev)
    q_tok = torch.zeros(B, G, dtype=torch.float32, device=dev)
    out_tokens = torch.zeros(B, G + 1, dtype=torch.int32, device=dev)
    out_len = torch.zeros(B, dtype=torch.int32, device=dev)

    drafted = args.drafted
    rows_per_gamma = (arm_gamma + 1) if drafted else (2 * arm_gamma + 1)     # rows the verify call streams
    tok_d = torch.zeros(B, G, dtype=torch.int32, device=dev)                 # tokens drafted on the device

    def verify_call(s):
        if drafted:
            bs.bs_softmax_verify_drafted(s["target"], s["draft"], tok_d, gamma_d, s["u_accept"], w.temperature,
                                         accept_len, p_tok, q_tok, ws)
        else:
            bs.bs_softmax_verify(s["target"], s["draft"], s["tokens"], gamma_d, s["u_accept"], w.temperature,
                                 accept_len, p_tok, q_tok, ws)

    def draft_calls(s):
        for j in range(G):
            bs.bs_draft_sample(s["draft"], j, gamma_d, s["u_draft"], w.temperature, tok_d, ws)

    walk = args.walk

    def walk_call(s):
        fn = bs.bs_verify_walk_drafted if drafted else bs.bs_verify_walk
        fn(s["target"], s["draft"], tok_d if drafted else s["tokens"], gamma_d, s["u_accept"], s["u_resample"],
           w.temperature, accept_len, p_tok, q_tok, out_tokens, out_len, ws)

    def step_calls(s, s_next):
        # the arms of this round: chosen here, or by the step call that ended the round before
        if not fused_bandit:
            bs.bs_bandit_select(state, alg, B, K, s["u_arm"], None, arm_d, gamma_d)
        if walk:
            if drafted:
                draft_calls(s)
            walk_call(s)
        else:
            if drafted:
                draft_calls(s)
                s = dict(s, tokens=tok_d)
            verify_call(s)
            bs.bs_residual_sample(s["target"], s["draft"], s["tokens"], gamma_d, accept_len, s["u_resample"],
                                  w.temperature, out_tokens, out_len, ws)
        if fused_bandit:
            step_bandit_call(s_next)
        else:
            update_call()

    def first_select():
        if fused_bandit:
            bs.bs_bandit_select(state, alg, B, K, sets[0]["u_arm"], None, arm_d, gamma_d)

    side = torch.cuda.Stream(device=dev)
    path_choice = None
    if args.auto_path and not drafted and w.temperature > 0.0:
        # one graph per path on the first input set, replayed: the same inputs and the same cache state for both
        trial = {}
        with torch.cuda.stream(side):
            for cand in (False, True):
                walk = cand
                first_select()
                step_calls(sets[0], sets[1 % ring])
                side.synchronize()
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    step_calls(sets[0], sets[1 % ring])
                for _ in range(5):
                    g.replay()
                a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(side)
                for _ in range(40):
                    g.replay()
                b_.record(side)
                side.synchronize()
                trial[cand] = a.elapsed_time(b_) / 40
                del g
        walk = trial[True] < trial[False]
        path_choice = {"two_call_ms": trial[False], "early_exit_ms": trial[True], "chosen": "early_exit" if walk else "two_call"}
        torch.cuda.synchronize()
        init_call()
    graphs = []
    if not args.no_graph:
        with torch.cuda.stream(side):
            first_select()
            step_calls(sets[0], sets[1 % ring])                # first launch outside capture
            side.synchronize()
            for i, s in enumerate(sets):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    step_calls(s, sets[(i + 1) % ring])
                graphs.append(g)
        torch.cuda.synchronize()
        # start from a clean bandit: the capture warm-up above played one round
        init_call()
    first_select()

    def run_step(i):
        if graphs:
            graphs[i % ring].replay()
        else:
            step_calls(sets[i % ring], sets[(i + 1) % ring])

    def pulls():
        return bs.bs_bandit_read(state, alg, B, K)["n"].copy()

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- warm-up, then the timed region ----
    for i in range(args.warmup):
        run_step(i)
    sync_all()
    n0 = pulls()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    sync_all()
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    y_sum = torch.zeros((), dtype=torch.int64, device=dev)
    e0.record(stream)
    for i in range(args.steps):
        run_step(args.warmup + i)
    e1.record(stream)
    sync_all()
    ms = e0.elapsed_time(e1)
    if rank == 0:
        time.sleep(0.15)
        clocks = sampler.stop()
    n1 = pulls()
    dn = (n1 - n0)                                             # [B, K] pulls inside the timed region
    assert dn.sum() == B * args.steps, "every sequence must have played every timed round"
    rows_timed = int((dn * (2 * arm_gamma + 1)[None, :]).sum())     # drafted or not: every valid row once
    bytes_timed = rows_timed * V * es
    ms, bytes_all = reduce_over_ranks(ms, bytes_timed, dev)
    value = job_rounds_per_s(world, args.steps, ms)

    # ---- kernel pass: CUDA events around bs_softmax_verify on its launching stream ----
    ksteps = min(args.steps, 50)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(ksteps)]
    rsd = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(ksteps)]
    dft = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(ksteps)]
    walk_rows = torch.zeros((), dtype=torch.int64, device=dev)
    resid_rows = torch.zeros((), dtype=torch.int64, device=dev)   # rows bs_residual_sample must read
    nk0 = pulls()
    for i in range(ksteps):
        s = sets[(args.warmup + args.steps + i) % ring]
        bs.bs_bandit_select(state, alg, B, K, s["u_arm"], None, arm_d, gamma_d)
        hold_gpu()
        if drafted:
            dft[i][0].record(stream)
            draft_calls(s)
            dft[i][1].record(stream)
            s = dict(s, tokens=tok_d)
        evs[i][0].record(stream)
        if walk:
            walk_call(s)
        else:
            verify_call(s)
        evs[i][1].record(stream)
        rsd[i][0].record(stream)
        if not walk:
            bs.bs_residual_sample(s["target"], s["draft"], s["tokens"], gamma_d, accept_len, s["u_resample"],
                                  w.temperature, out_tokens, out_len, ws)
        rsd[i][1].record(stream)
        if not walk and w.temperature > 0.0:                   # the row pair of a rejected position, or the bonus row alone
            resid_rows += torch.where(accept_len < gamma_d, 2, 1).sum()
        if walk:                                               # rows the walk had to read: up to the stop position
            tau = accept_len.to(torch.int64); gm = gamma_d.to(torch.int64)
            walk_rows += (tau + 1).sum() if drafted else torch.where(tau < gm, 2 * (tau + 1), 2 * gm + 1).sum()
        update_call()
        y_sum += out_len.sum()
    torch.cuda.synchronize()
    verify_ms = sum(a.elapsed_time(b) for a, b in evs) / ksteps
    resid_ms = sum(a.elapsed_time(b) for a, b in rsd) / ksteps
    dk = pulls() - nk0
    verify_bytes = float((dk * rows_per_gamma[None, :]).sum()) * V * es / ksteps   # per launch
    full_bytes = verify_bytes
    if walk:
        verify_bytes = float(walk_rows.item()) * V * es / ksteps
    resid_bytes = float(resid_rows.item()) * V * es / ksteps
    draft_ms = sum(a.elapsed_time(b) for a, b in dft) / ksteps if drafted else None
    draft_bytes = float((dk * arm_gamma[None, :]).sum()) * V * es / ksteps if drafted else None
    mean_y = float(y_sum.item()) / (B * ksteps)
    status = bs.bs_get_device_status(ws, B, G, V)
    assert (status & ~bs.BS_DEV_RESIDUAL_FALLBACK == 0).all(), f"device status {status}"

    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
    else:
        peak, peak_src = FALLBACK_HBM_GBS, "fallback"
    achieved = verify_bytes / (verify_ms * 1e-3) / 1e9

    # ---- the same call launched back to back on the rotating input sets, one event pair around the lot: what a
    # launch takes in a busy stream.  An event pair around ONE short launch (the figure above) also times the
    # gap before the kernel starts and the event itself, 4-5 us that no kernel change can touch. ----
    back_to_back = None
    if not walk and not drafted:
        nb = min(args.steps, 50)
        for i in range(3):
            verify_call(sets[i % ring])
        a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record(stream)
        for i in range(nb):
            verify_call(sets[(3 + i) % ring])
        b_.record(stream)
        torch.cuda.synchronize()
        gm = gamma_d.to(torch.int64)
        b2b_bytes = float((gm + 1).sum().item() if w.temperature == 0.0 else (2 * gm + 1).sum().item()) * V * es
        b2b_ms = a.elapsed_time(b_) / nb
        back_to_back = {"launches": nb, "ms_per_launch": b2b_ms, "bytes_per_launch": b2b_bytes,
                        "achieved": b2b_bytes / (b2b_ms * 1e-3) / 1e9, "frac": b2b_bytes / (b2b_ms * 1e-3) / 1e9 / peak}

    # ---- the same rounds through the early-exit entry point, for comparison (plain runs only) ----
    variants = None
    if not walk and not drafted and w.temperature > 0.0:
        def walk_step(s):
            bs.bs_bandit_select(state, alg, B, K, s["u_arm"], None, arm_d, gamma_d)
            walk_call(s)
            update_call()
        for i in range(min(args.warmup, 5)):
            walk_step(sets[i % ring])
        sync_all()
        a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        nw = min(args.steps, 100)
        a.record(stream)
        for i in range(nw):
            walk_step(sets[i % ring])
        b_.record(stream)
        sync_all()
        wms, _ = reduce_over_ranks(a.elapsed_time(b_), 0.0, dev)
        variants = {"early_exit": {"value": job_rounds_per_s(world, nw, wms), "unit": UNIT, "ms_per_step": wms / nw,
                                   "steps": nw, "launch": "direct launches",
                                   "path": "select, bs_verify_walk, update (see --walk)"}}

    # ---- end to end from pinned host buffers ----
    e2e = None
    if args.e2e_steps > 0:
        s0 = sets[0]
        host = {k: torch.empty(s0[k].shape, dtype=s0[k].dtype, pin_memory=True).copy_(s0[k])
                for k in ("target", "draft", "tokens", "u_accept", "u_resample", "u_arm", "u_draft")}
        devb = {k: torch.empty_like(s0[k]) for k in host}
        h_tokens = torch.empty(out_tokens.shape, dtype=out_tokens.dtype, pin_memory=True)
        h_len = torch.empty(out_len.shape, dtype=out_len.dtype, pin_memory=True)
        h2d = sum(t.numel() * t.element_size() for t in host.values())
        d2h = h_tokens.numel() * 4 + h_len.numel() * 4

        def e2e_step():
            for k in host:
                devb[k].copy_(host[k], non_blocking=True)
            step_calls(devb, devb)                             # the uniforms of the next round arrive with it
            h_tokens.copy_(out_tokens, non_blocking=True)
            h_len.copy_(out_len, non_blocking=True)
            torch.cuda.current_stream().synchronize()          # the caller reads the tokens every round

        for _ in range(2):
            e2e_step()
        sync_all()
        a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(args.e2e_steps):
            e2e_step()
        b_.record(stream)
        sync_all()
        e2e_ms = a.elapsed_time(b_)
        if world > 1:
            t = torch.tensor([e2e_ms], dtype=torch.float64, device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e2e_ms = float(t.item())
        e2e = {"value": world * args.e2e_steps / (e2e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "steps": args.e2e_steps}
        del host, devb

    # ---- CPU oracle on a bounded sample (rank 0, N = 1 only) ----
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        torch.set_num_threads(1)
        seqs_in = oracle_inputs(w)
        n, dt = oracle_sample(w, seqs_in, args.cpu_seconds)
        cpu = {"value": (n / B) / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"{n} verifications of the first {len(seqs_in)} sequences of a {B}-sequence round in "
                         f"{dt:.1f} s, verification only (numpy fp64, one thread; host has {host_cores()} cores)"}
        if args.cpu_all_cores:
            cpu["all_cores"] = oracle_all_cores(args, w, host_cores())

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {**cpu_config(w),
                       "l2": f"ring of {ring} input sets, {ring * set_bytes / 1e6:.0f} MB > 2 x L2",
                       "launch": "one CUDA graph per step" if graphs else "direct launches",
                       "path": ("select, draft x Gmax, verify with early exit on drafted statistics + resample "
                                "in one launch, update" if walk and drafted else
                                "select, verify with early exit + resample in one launch, update" if walk else
                                "select, draft x Gmax, verify on drafted statistics, resample, update"
                                if drafted else "select, verify, resample, update"),
                       "bandit_calls": ("bs_bandit_step: the update and the next round's select in one launch"
                                        if fused_bandit else "bs_bandit_select and bs_bandit_update, two launches"),
                       "multi_gpu": "one independent batch per rank, no collective on the data path"},
            "tokens_per_s": mean_y * B * value,
            "mean_accepted_len": mean_y,
            "algorithmic_gbs": bytes_all / (ms * 1e-3) / 1e9,
            "roofline": {"bound": "hbm", "kernel": "verify_stream_kernel (bs_softmax_verify)", "achieved": achieved,
                         "peak": peak, "peak_source": peak_src, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": ncu_traffic(w.name, verify_bytes), "bytes_per_launch": verify_bytes,
                         "nominal_peak": 8000.0, "frac_of_nominal": achieved / 8000.0,
                         "ms_per_launch": verify_ms, "residual_ms_per_launch": resid_ms,
                         "back_to_back": back_to_back,
                         # The second call of the round; `stop_row_bytes` are the rows it streams again (the row
                         # pair of a rejected position, or the bonus row alone).
                         "residual": (None if walk or resid_bytes <= 0 else
                                      {"kernel": "residual_stream_kernel (bs_residual_sample)",
                                       "ms_per_launch": resid_ms, "stop_row_bytes": resid_bytes}),
                         # both calls together against the same single-touch bytes
                         "verify_plus_residual": (None if walk else
                                                  {"ms": verify_ms + resid_ms,
                                                   "achieved": verify_bytes / ((verify_ms + resid_ms) * 1e-3) / 1e9,
                                                   "frac": verify_bytes / ((verify_ms + resid_ms) * 1e-3) / 1e9 / peak})},
            "e2e": e2e, "cpu_baseline": cpu, "clocks": clocks, "variants": variants, "path_choice": path_choice,
            "other_workloads": getattr(args, "others", None),
            "gpu_launches": ((3 if walk else 4) - (1 if fused_bandit else 0) + (2 * G if drafted else 0)
                             + (1 if reward else 0)) * args.steps,
        }
        if walk:
            line["roofline"]["kernel"] = "verify_walk_kernel (bs_verify_walk)"
            line["roofline"]["traffic"] = None
            line["early_exit"] = {"bytes_per_launch": verify_bytes, "bytes_without_early_exit": full_bytes,
                                  "note": "rows up to the stop position only; the second pass over the stop "
                                          "position's rows (mostly L2) is not credited"}
        if drafted:
            line["drafting"] = {"ms_per_round": draft_ms, "calls": G, "row_bytes_per_round": draft_bytes,
                                "note": "each call reads its draft rows once for the statistics and once more "
                                        "(mostly from L2) for the inverse CDF"}
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


# ---------------------------------------------------------------------------------------------
# fused LM-head path: bs_lmhead_verify -> bs_residual_sample
# ---------------------------------------------------------------------------------------------

def lmhead_counts(w):
    """Algorithmic flops and bytes of one round: both products, W and H read once, fp32 logits
    written once."""
    Mt, Md = w.B * (w.gamma + 1), w.B * w.gamma
    flops = 2.0 * w.V * (Mt * w.d_t + Md * w.d_d)
    nbytes = 2.0 * w.V * (w.d_t + w.d_d) + 2.0 * (Mt * w.d_t + Md * w.d_d) + 4.0 * w.V * (Mt + Md)
    return flops, nbytes


def lmhead_oracle_sample(w, inp, seconds: float, cols: int = 4096):
    """The oracle's fp64 product on a slice of vocabulary columns, repeated until `seconds` are
    used.  Returns (fraction of one round's multiply-adds done, elapsed seconds)."""
    from oracle import lmhead as ol
    Ht, Hd = inp.H_t.float().cpu().numpy(), inp.H_d.float().cpu().numpy()
    Wt, Wd = inp.W_t[:, :cols].float().cpu().numpy(), inp.W_d[:, :cols].float().cpu().numpy()
    done, t0 = 0.0, time.perf_counter()
    while True:
        ol.lmhead_logits(Ht, Wt)
        ol.lmhead_logits(Hd, Wd)
        done += cols / w.V
        if time.perf_counter() - t0 > seconds:
            break
    return done, time.perf_counter() - t0


def run_lmhead_reference(args, w):
    from paper_2505_15141_b200 import workloads as wl
    import torch
    torch.set_num_threads(1)
    inp = wl.make_lmhead_inputs(w, 1, "cpu")
    per_step = max(0.5, min(10.0, 90.0 / max(1, args.steps + args.warmup)))
    fr, tt = 0.0, 0.0
    for i in range(args.warmup + args.steps):
        f, dt = lmhead_oracle_sample(w, inp, per_step)
        if i >= args.warmup:
            fr += f; tt += dt
    val = fr / tt
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * tt / max(1, args.steps), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "gamma": w.gamma, "V": w.V, "d_t": w.d_t, "d_d": w.d_d},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": f"fp64 products on 4096-column slices of the vocabulary, {fr:.3f} rounds' worth "
                                   f"of multiply-adds in {tt:.1f} s (numpy, one thread); verification not included"},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def run_lmhead(args, w):
    import torch
    import torch.distributed as dist
    import __graft_entry__ as entry

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group(backend="nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if rank == 0:
        entry.build()
    if world > 1:
        dist.barrier()
    from paper_2505_15141_b200 import binding as bs, workloads as wl

    B, G, V = w.B, w.gamma, w.V
    # two sets of hidden states / tokens / uniforms per rank; the embeddings (1.58 GB, far larger
    # than L2) are the model's and stay put: every round streams them from HBM again
    first = wl.make_lmhead_inputs(w, rank_round_index(rank, 0), dev)
    sets = [first, wl.make_lmhead_inputs(w, rank_round_index(rank, 1), dev, weights=(first.W_t, first.W_d))]
    dsets = [dict(H_t=s.H_t, H_d=s.H_d, tokens=s.tokens, gamma=torch.as_tensor(s.gamma, device=dev),
                  u_accept=torch.as_tensor(s.uniforms.u_accept, device=dev),
                  u_resample=torch.as_tensor(s.uniforms.u_resample, device=dev)) for s in sets]
    W_t, W_d = first.W_t, first.W_d
    ws = bs.new_lmhead_workspace(B, G, V, dev)
    lt = torch.empty(B, G + 1, V, dtype=torch.float32, device=dev)
    ld = torch.empty(B, G, V, dtype=torch.float32, device=dev)
    accept_len = torch.zeros(B, dtype=torch.int32, device=dev)
    p_tok = torch.zeros(B, G, dtype=torch.float32, device=dev)
    q_tok = torch.zeros(B, G, dtype=torch.float32, device=dev)
    out_tokens = torch.zeros(B, G + 1, dtype=torch.int32, device=dev)
    out_len = torch.zeros(B, dtype=torch.int32, device=dev)

    def lm_call(s):
        bs.bs_lmhead_verify(s["H_t"], W_t, s["H_d"], W_d, s["tokens"], s["gamma"], s["u_accept"], w.temperature,
                            B, G, lt, ld, accept_len, p_tok, q_tok, ws)

    def res_call(s):
        bs.bs_residual_sample(lt, ld, s["tokens"], s["gamma"], accept_len, s["u_resample"], w.temperature,
                              out_tokens, out_len, ws)

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        lm_call(dsets[i % 2]); res_call(dsets[i % 2])
    sync_all()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    sync_all()
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(args.steps):
        s = dsets[(args.warmup + i) % 2]
        lm_call(s); res_call(s)
    e1.record(stream)
    sync_all()
    ms = e0.elapsed_time(e1)
    clocks = None
    if rank == 0:
        time.sleep(0.15)
        clocks = sampler.stop()
    flops, nbytes = lmhead_counts(w)
    ms, _ = reduce_over_ranks(ms, 0.0, dev)
    value = job_rounds_per_s(world, args.steps, ms)

    # kernel pass: events around bs_lmhead_verify (product kernel + merge kernel) and the resampler
    ksteps = min(args.steps, 50)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(ksteps)]
    y_sum = torch.zeros((), dtype=torch.int64, device=dev)
    for i in range(ksteps):
        s = dsets[i % 2]
        hold_gpu()
        evs[i][0].record(stream); lm_call(s)
        evs[i][1].record(stream); res_call(s)
        evs[i][2].record(stream)
        y_sum += out_len.sum()
    torch.cuda.synchronize()
    lm_ms = sum(e[0].elapsed_time(e[1]) for e in evs) / ksteps
    res_ms = sum(e[1].elapsed_time(e[2]) for e in evs) / ksteps
    mean_y = float(y_sum.item()) / (B * ksteps)
    status = bs.bs_get_device_status(ws, B, G, V)
    assert (status & ~bs.BS_DEV_RESIDUAL_FALLBACK == 0).all(), f"device status {status}"

    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peaks = json.load(open(peaks_path)) if os.path.exists(peaks_path) else None
    hbm_peak = float(peaks["hbm_gbs"]) if peaks else FALLBACK_HBM_GBS
    tc_peak = float(peaks["bf16_tflops"]) if peaks else 1590.0
    src = "measured" if peaks else "fallback"
    gbs = nbytes / (lm_ms * 1e-3) / 1e9
    tfs = flops / (lm_ms * 1e-3) / 1e12
    # which roof is lower for this shape decides the bound that is reported
    hbm_bound = nbytes / (hbm_peak * 1e9) >= flops / (tc_peak * 1e12)
    roof = ({"bound": "hbm", "achieved": gbs, "peak": hbm_peak, "unit": "GB/s", "frac": gbs / hbm_peak}
            if hbm_bound else
            {"bound": "tensor", "achieved": tfs, "peak": tc_peak, "unit": "TFLOP/s", "frac": tfs / tc_peak})
    roof.update({"nominal_hbm_gbs": 8000.0, "hbm_frac_of_nominal": gbs / 8000.0,
                 "nominal_bf16_tflops": 2250.0, "tensor_frac_of_nominal": tfs / 2250.0})
    roof.update({"kernel": "lmhead_gemm_kernel (bs_lmhead_verify)", "peak_source": src,
                 "traffic": ncu_traffic(w.name, 2.0 * w.V * (w.d_t + w.d_d) + 2.0 * w.B * ((w.gamma + 1) * w.d_t + w.gamma * w.d_d)),
                 "bytes_per_launch": nbytes, "flops_per_launch": flops,
                 "ms_per_launch": lm_ms, "residual_ms_per_launch": res_ms,
                 "hbm_gbs": gbs, "hbm_frac": gbs / hbm_peak, "tensor_tflops": tfs, "tensor_frac": tfs / tc_peak})
    if peaks and peaks.get("bf16_tflops_sustained"):
        # `peak` is the burst figure (the stricter one); the launches here run back to back under the
        # power cap, where the library product itself settles at the sustained figure
        sus = float(peaks["bf16_tflops_sustained"])
        roof.update({"bf16_tflops_sustained": sus, "tensor_frac_of_sustained": tfs / sus})

    e2e = None
    if args.e2e_steps > 0:
        keys = ("H_t", "H_d", "tokens", "gamma", "u_accept", "u_resample")
        host = {k: torch.empty(dsets[0][k].shape, dtype=dsets[0][k].dtype, pin_memory=True).copy_(dsets[0][k])
                for k in keys}
        devb = {k: torch.empty_like(dsets[0][k]) for k in keys}
        h_tokens = torch.empty(out_tokens.shape, dtype=out_tokens.dtype, pin_memory=True)
        h_len = torch.empty(out_len.shape, dtype=out_len.dtype, pin_memory=True)
        h2d = sum(t.numel() * t.element_size() for t in host.values())
        d2h = h_tokens.numel() * 4 + h_len.numel() * 4

        def e2e_step():
            for k in keys:
                devb[k].copy_(host[k], non_blocking=True)
            lm_call(devb); res_call(devb)
            h_tokens.copy_(out_tokens, non_blocking=True)
            h_len.copy_(out_len, non_blocking=True)
            torch.cuda.current_stream().synchronize()

        n_e2e = max(args.e2e_steps, 20)
        for _ in range(3):
            e2e_step()
        sync_all()
        a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(n_e2e):
            e2e_step()
        b_.record(stream)
        sync_all()
        e2e_ms, _ = reduce_over_ranks(a.elapsed_time(b_), 0.0, dev)
        e2e = {"value": world * n_e2e / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(d2h), "steps": n_e2e,
               "note": "hidden states, tokens and uniforms come from the host every step; the embeddings are resident"}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        torch.set_num_threads(1)
        fr, dt = lmhead_oracle_sample(w, sets[0], args.cpu_seconds)
        cpu = {"value": fr / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"fp64 products on 4096-column slices of the vocabulary, {fr:.3f} rounds' worth of "
                         f"multiply-adds in {dt:.1f} s (numpy, one thread; host has {host_cores()} cores); "
                         f"verification not included"}

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "B": B, "gamma": G, "V": V, "d_t": w.d_t, "d_d": w.d_d,
                       "temperature": w.temperature,
                       "l2": "the embeddings read every round are 1576 MB, larger than L2",
                       "launch": "direct launches", "multi_gpu": "one independent batch per rank"},
            "tokens_per_s": mean_y * B * value, "mean_accepted_len": mean_y,
            "roofline": roof, "e2e": e2e, "cpu_baseline": cpu, "clocks": clocks,
            "gpu_launches": 3 * args.steps}))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


# ---------------------------------------------------------------------------------------------
# greedy verification of a tree of drafts, tree shapes as the arms of UCBSpec
# ---------------------------------------------------------------------------------------------

def tree_oracle_inputs(w):
    from paper_2505_15141_b200 import workloads as wl
    import dataclasses as dc
    inp = wl.make_tree_inputs(dc.replace(w, B=min(w.B, ORACLE_SAMPLE_SEQS)), 1, "cpu")
    t = inp.target.float().numpy()
    return [(t[b], [int(x) for x in w.shapes[b % w.K]], inp.tokens[b % w.K, b].numpy(), len(w.shapes[b % w.K]))
            for b in range(t.shape[0])]


def tree_oracle_sample(seqs, seconds: float):
    from oracle import tree as otree
    done, t0 = 0, time.perf_counter()
    while True:
        rows, parent, tokens, n = seqs[done % len(seqs)]
        otree.verify_tree_greedy(rows, parent, tokens, n)
        done += 1
        if time.perf_counter() - t0 > seconds:
            break
    return done, time.perf_counter() - t0


def tree_config(w) -> dict:
    return {"workload": w.name, "B": w.B, "V": w.V, "logits_dtype": w.dtype, "temperature": 0.0,
            "shapes": {"nodes": [len(x) for x in w.shapes], "depth": list(w.depths)}, "bandit": "ucb over the shapes"}


def run_tree_reference(args, w):
    import torch
    torch.set_num_threads(1)
    per_step = max(0.2, min(10.0, 90.0 / max(1, args.steps + args.warmup), args.cpu_seconds))
    seqs = tree_oracle_inputs(w)
    n_tot, t_tot = 0, 0.0
    for i in range(args.warmup + args.steps):
        n, dt = tree_oracle_sample(seqs, per_step)
        if i >= args.warmup:
            n_tot += n; t_tot += dt
    val = (n_tot / w.B) / t_tot
    world = int(os.environ.get("WORLD_SIZE", "1"))
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * t_tot / max(1, args.steps), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic", "config": tree_config(w),
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": 1, "kind": "oracle",
                         "sample": f"{n_tot} tree verifications of the first {len(seqs)} sequences in {t_tot:.1f} s "
                                   f"(numpy, one thread)"},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}, "gpu_launches": 0}))


def run_tree(args, w):
    import torch
    import torch.distributed as dist
    import __graft_entry__ as entry

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group(backend="nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if rank == 0:
        entry.build()
    if world > 1:
        dist.barrier()
    from paper_2505_15141_b200 import binding as bs, workloads as wl

    B, K, N, V, es = w.B, w.K, w.Nmax, w.V, w.elem_size
    set_bytes = es * V * B * (N + 1)
    ring = max(2, -(-2 * L2_BYTES // set_bytes) + 1)
    sets = [wl.make_tree_inputs(w, rank_round_index(rank, i), dev) for i in range(ring)]
    sp_d, sn_d = sets[0].shape_parent, sets[0].shape_nodes
    state = bs.new_bandit(bs.BS_UCB, B, w.depths, w.delta, dev)
    ws = bs.new_workspace(B, N, V, dev)
    arm_d = torch.zeros(B, dtype=torch.int32, device=dev); gam_d = torch.zeros_like(arm_d)
    parent_d = torch.zeros(B, N, dtype=torch.int32, device=dev); n_d = torch.zeros(B, dtype=torch.int32, device=dev)
    tok_d = torch.zeros(B, N, dtype=torch.int32, device=dev)
    acc = torch.zeros(B, dtype=torch.int32, device=dev); on = torch.zeros(B, N, dtype=torch.int32, device=dev)
    otk = torch.zeros(B, N + 1, dtype=torch.int32, device=dev); ol = torch.zeros(B, dtype=torch.int32, device=dev)
    rows_b = torch.arange(B, device=dev)

    def step_calls(s):
        bs.bs_bandit_select(state, bs.BS_UCB, B, K, None, None, arm_d, gam_d)
        bs.bs_tree_expand_shapes(sp_d, sn_d, arm_d, parent_d, n_d)
        tok_d.copy_(s.tokens[arm_d.long(), rows_b])           # stands in for the draft model drafting along the chosen shape
        bs.bs_tree_verify_greedy(s.target, parent_d, tok_d, n_d, acc, on, otk, ol, ws)
        bs.bs_bandit_update(state, bs.BS_UCB, B, K, arm_d, ol)

    def sync_all():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    side = torch.cuda.Stream(device=dev)
    graphs = []
    if not args.no_graph:
        with torch.cuda.stream(side):
            step_calls(sets[0])
            side.synchronize()
            for s_ in sets:
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=side):
                    step_calls(s_)
                graphs.append(g)
        torch.cuda.synchronize()
        bs.bs_bandit_init(state, bs.BS_UCB, B, K, w.depths, w.delta)

    def run_step(i):
        if graphs:
            graphs[i % ring].replay()
        else:
            step_calls(sets[i % ring])

    for i in range(args.warmup):
        run_step(i)
    sync_all()
    n0 = bs.bs_bandit_read(state, bs.BS_UCB, B, K)["n"].copy()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)
    sync_all()
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(args.steps):
        run_step(args.warmup + i)
    e1.record(stream)
    sync_all()
    ms = e0.elapsed_time(e1)
    clocks = None
    if rank == 0:
        time.sleep(0.15)
        clocks = sampler.stop()
    nodes = np.asarray([len(x) for x in w.shapes])
    dn = bs.bs_bandit_read(state, bs.BS_UCB, B, K)["n"] - n0
    assert dn.sum() == B * args.steps
    bytes_timed = float((dn * (nodes + 1)[None, :]).sum()) * V * es
    ms, bytes_all = reduce_over_ranks(ms, bytes_timed, dev)
    value = job_rounds_per_s(world, args.steps, ms)

    # kernel pass: events around bs_tree_verify_greedy (statistics kernel in greedy mode + the walk over the nodes)
    ksteps = min(args.steps, 50)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(ksteps)]
    y_sum = torch.zeros((), dtype=torch.int64, device=dev)
    nk0 = bs.bs_bandit_read(state, bs.BS_UCB, B, K)["n"].copy()
    for i in range(ksteps):
        s_ = sets[(args.warmup + args.steps + i) % ring]
        bs.bs_bandit_select(state, bs.BS_UCB, B, K, None, None, arm_d, gam_d)
        bs.bs_tree_expand_shapes(sp_d, sn_d, arm_d, parent_d, n_d)
        tok_d.copy_(s_.tokens[arm_d.long(), rows_b])
        hold_gpu()
        evs[i][0].record(stream)
        bs.bs_tree_verify_greedy(s_.target, parent_d, tok_d, n_d, acc, on, otk, ol, ws)
        evs[i][1].record(stream)
        bs.bs_bandit_update(state, bs.BS_UCB, B, K, arm_d, ol)
        y_sum += ol.sum()
    torch.cuda.synchronize()
    k_ms = sum(a.elapsed_time(b) for a, b in evs) / ksteps
    dk = bs.bs_bandit_read(state, bs.BS_UCB, B, K)["n"] - nk0
    k_bytes = float((dk * (nodes + 1)[None, :]).sum()) * V * es / ksteps
    mean_y = float(y_sum.item()) / (B * ksteps)
    assert (bs.bs_get_device_status(ws, B, N, V) == 0).all()
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_src = float(json.load(open(peaks_path))["hbm_gbs"]), "measured"
    else:
        peak, peak_src = FALLBACK_HBM_GBS, "fallback"
    achieved = k_bytes / (k_ms * 1e-3) / 1e9

    e2e = None
    if args.e2e_steps > 0:
        s0 = sets[0]
        host = {"target": torch.empty(s0.target.shape, dtype=s0.target.dtype, pin_memory=True).copy_(s0.target),
                "tokens": torch.empty(s0.tokens.shape, dtype=s0.tokens.dtype, pin_memory=True).copy_(s0.tokens)}
        devb = wl.TreeInputs(target=torch.empty_like(s0.target), tokens=torch.empty_like(s0.tokens),
                             shape_parent=sp_d, shape_nodes=sn_d)
        h_tok = torch.empty(otk.shape, dtype=otk.dtype, pin_memory=True)
        h_len = torch.empty(ol.shape, dtype=ol.dtype, pin_memory=True)
        h2d = sum(t.numel() * t.element_size() for t in host.values())
        d2h = h_tok.numel() * 4 + h_len.numel() * 4

        def e2e_step():
            devb.target.copy_(host["target"], non_blocking=True)
            devb.tokens.copy_(host["tokens"], non_blocking=True)
            step_calls(devb)
            h_tok.copy_(otk, non_blocking=True)
            h_len.copy_(ol, non_blocking=True)
            torch.cuda.current_stream().synchronize()

        for _ in range(2):
            e2e_step()
        sync_all()
        a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(args.e2e_steps):
            e2e_step()
        b_.record(stream)
        sync_all()
        e2e_ms, _ = reduce_over_ranks(a.elapsed_time(b_), 0.0, dev)
        e2e = {"value": world * args.e2e_steps / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(d2h), "steps": args.e2e_steps}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        torch.set_num_threads(1)
        seqs = tree_oracle_inputs(w)
        n, dt = tree_oracle_sample(seqs, args.cpu_seconds)
        cpu = {"value": (n / B) / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"{n} tree verifications of the first {len(seqs)} sequences in {dt:.1f} s (numpy, one thread; "
                         f"host has {host_cores()} cores)"}
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {**tree_config(w), "l2": f"ring of {ring} input sets, {ring * set_bytes / 1e6:.0f} MB > 2 x L2",
                       "launch": "one CUDA graph per step" if graphs else "direct launches",
                       "path": "select, expand shapes, (token table lookup: torch), tree verify (2 launches), update",
                       "multi_gpu": "one independent batch per rank, no collective on the data path"},
            "tokens_per_s": mean_y * B * value, "mean_accepted_len": mean_y,
            "algorithmic_gbs": bytes_all / (ms * 1e-3) / 1e9,
            "roofline": {"bound": "hbm", "kernel": "verify_stream_kernel, greedy mode + tree_walk_kernel (bs_tree_verify_greedy)",
                         "achieved": achieved, "peak": peak, "peak_source": peak_src, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": ncu_traffic(w.name, k_bytes), "bytes_per_launch": k_bytes, "ms_per_launch": k_ms,
                         "residual_ms_per_launch": 0.0},
            "e2e": e2e, "cpu_baseline": cpu, "clocks": clocks, "gpu_launches": 5 * args.steps}))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


OTHER_WORKLOADS = ("llama3_ucb", "llama2_fixed", "llama3_tput", "llama3_tree", "lmhead_llama3", "lmhead_llama3_b128")


def other_workloads_summary():
    """Short runs of the other workloads, each in a process of its own before this one touches the
    GPU: rounds/s and the dominant kernel's roofline line, for the record next to the main line."""
    out = {}
    for name in OTHER_WORKLOADS:
        cmd = [sys.executable, os.path.abspath(__file__), "--workload", name, "--steps", "200", "--warmup", "20",
               "--no-cpu-baseline", "--e2e-steps", "0", "--no-others"]
        try:
            res = subprocess.run(cmd, capture_output=True, text=True, timeout=240)
            d = json.loads(res.stdout.strip().splitlines()[-1])
            r = d["roofline"]
            out[name] = {"value": d["value"], "unit": d["unit"], "ms_per_step": d["ms_per_step"],
                         "algorithmic_gbs": d.get("algorithmic_gbs"),
                         "roofline": {k: r.get(k) for k in ("bound", "kernel", "achieved", "peak", "unit", "frac",
                                                            "ms_per_launch", "residual_ms_per_launch", "back_to_back")},
                         "variants": d.get("variants")}
        except Exception as e:                                   # the main line must not depend on these
            out[name] = {"error": f"{type(e).__name__}: {e}"[:200]}
    return out


def spawn_ranks(n: int) -> int:
    """`--gpus N` without a launcher: start N ranks of this script on this node, as
    `python -m torch.distributed.run --nnodes=1 --nproc-per-node N` would be asked to, and pass their
    output through (rank 0 prints the line)."""
    import socket
    sk = socket.socket()
    sk.bind(("127.0.0.1", 0))
    port = sk.getsockname()[1]
    sk.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *sys.argv[1:]]
    return subprocess.run(cmd).returncode


def main():
    args = parse_args()
    from paper_2505_15141_b200 import workloads as wl
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args.gpus))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.gpus != world:
        sys.exit(f"bench.py: --gpus {args.gpus} but the launcher started {world} rank(s)")
    rank = int(os.environ.get("RANK", "0"))
    if args.impl == "reference" and world > 1:
        print(f"bench.py: rank {rank} of {world} ({'runs the oracle' if rank == 0 else 'idle'})", file=sys.stderr)
    plain_default = (args.workload == "qwen_exp3" and args.impl == "cuda" and not (args.batch or args.fixed_gamma
                     or args.walk or args.drafted or args.no_others) and world == 1)
    args.others = other_workloads_summary() if plain_default else None
    if plain_default:
        args.cpu_all_cores = True
    if args.workload in wl.LMHEAD_WORKLOADS:
        w = wl.LMHEAD_WORKLOADS[args.workload]
        if args.batch:
            w = dataclasses.replace(w, B=args.batch)
        if args.impl == "reference":
            if rank == 0:
                run_lmhead_reference(args, w)
            return
        run_lmhead(args, w)
        return
    if args.workload in wl.TREE_WORKLOADS:
        w = wl.TREE_WORKLOADS[args.workload]
        if args.batch:
            w = dataclasses.replace(w, B=args.batch)
        if args.impl == "reference":
            if rank == 0:
                run_tree_reference(args, w)
            return
        run_tree(args, w)
        return
    w = wl.WORKLOADS[args.workload]
    if args.batch:
        w = dataclasses.replace(w, B=args.batch)
    if args.fixed_gamma:
        w = dataclasses.replace(w, arm_gamma=(args.fixed_gamma,), alg=None)
    if args.impl == "reference":
        if args.oracle_worker:
            oracle_worker(args, w)
        elif rank == 0:
            run_reference(args, w)
        return
    run_cuda(args, w)


if __name__ == "__main__":
    main()
