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
