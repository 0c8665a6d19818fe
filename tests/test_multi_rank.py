"""The N > 1 path on CPU: two `gloo` ranks.  Sequences are independent, so a batch is sharded
across ranks with no collective on the data path; the only exchange is the timing reduction
(max of times, sum of bytes) that the benchmark performs."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close(); return p


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from oracle import verify as ov
    from paper_2505_15141_b200 import workloads as wl
    # 1. the benchmark's reduction: slowest rank's time, all ranks' bytes
    ms, nbytes = bench.reduce_over_ranks(10.0 + 5.0 * rank, 1000.0 * (rank + 1), "cpu")
    assert ms == 15.0 and nbytes == 3000.0
    assert bench.job_rounds_per_s(world, 30, ms) == world * 30 / 0.015
    assert bench.rank_round_index(0, 3) != bench.rank_round_index(1, 3)
    # 2. shard a batch of sequences over the ranks, verify each shard on its own, gather
    w = wl.WORKLOADS["tiny_ucb"]
    rnd = wl.make_round(w, 2, np.array([0, 1, 2, 1]))
    t, d = rnd.target.numpy(), rnd.draft.numpy()
    mine = list(range(rank, w.B, world))
    res = [ov.verify_sequence(t[b], d[b], rnd.tokens[b].numpy(), int(rnd.gamma[b]), rnd.uniforms.u_accept[b],
                              float(rnd.uniforms.u_resample[b]), w.temperature) for b in mine]
    local = [(b, r.tau, r.token) for b, r in zip(mine, res)]
    gathered = [None] * world
    dist.all_gather_object(gathered, local)
    if rank == 0:
        whole = ov.verify_round(t, d, rnd.tokens.numpy(), rnd.gamma, rnd.uniforms.u_accept,
                                rnd.uniforms.u_resample, w.temperature)
        merged = sorted(x for part in gathered for x in part)
        assert merged == [(b, r.tau, r.token) for b, r in enumerate(whole)]
        out.put("ok")
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_sequences_without_data_collectives():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(timeout=180)
        assert p.exitcode == 0
    assert out.get(timeout=5) == "ok"


def test_bench_gpus_flag_starts_that_many_ranks():
    """`bench.py --gpus 2` with no launcher around it must itself start two ranks.  The reference arm
    needs no GPU: rank 0 times the oracle and prints the line with n_gpus = 2, rank 1 exits idle."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--impl", "reference",
                          "--workload", "tiny_ucb", "--steps", "2", "--warmup", "1", "--cpu-seconds", "0.3"],
                         capture_output=True, text=True, timeout=300, cwd=ROOT, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [ln for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                                        # rank 0 alone prints
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0
    assert "rank 0 of 2" in res.stderr and "rank 1 of 2" in res.stderr
    # a launcher that started a different number of ranks than --gpus says is an error, not a silent 1-GPU run
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "4", "--impl", "reference",
                          "--workload", "tiny_ucb"], capture_output=True, text=True, timeout=120, cwd=ROOT,
                         env=dict(env, WORLD_SIZE="1", RANK="0"))
    assert res.returncode != 0 and "--gpus 4" in res.stderr
