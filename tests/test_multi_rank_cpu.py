"""The N > 1 path of bench.py on CPU: two gloo ranks, 127.0.0.1 rendezvous.  The hot path shards by
(sequence, layer, KV head) without any exchange, so the multi-rank logic is: barrier, slowest rank's
time, whole-job throughput; and independent ranks must give results identical to one rank doing all
units (checked here with the CPU oracle standing in for the per-rank work)."""
import os
import socket
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _unit_result(seed):
    """One independent unit's decode step on the oracle (small shapes)."""
    from oracle import tb_oracle as orc
    from paper_2503_07518_b200 import workloads as wl
    r = np.random.Generator(np.random.PCG64(seed))
    L, D, dp, g = 400, 128, 32, 4
    K = wl.to_storage(r.standard_normal((L, D)).astype(np.float32), wl.BF16)
    V = wl.to_storage(r.standard_normal((L, D)).astype(np.float32), wl.BF16)
    W = wl.to_storage((r.standard_normal((D, dp)) / np.sqrt(D)).astype(np.float32), wl.BF16)
    u = orc.Unit(K, V, orc.project_keys(K, W, wl.BF16), 40)
    qi = r.standard_normal((g, dp)).astype(np.float32)
    q = wl.to_storage(r.standard_normal((g, D)).astype(np.float32), wl.BF16)
    return orc.step_units([u], [L], [qi], [q], [1], g=g, D=D, dp=dp, dtype=wl.BF16, budget=40, sinks=2, recent=8)[0]


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms_local = 10.0 + 5.0 * rank                        # rank 1 is the slow one
    dist.barrier()
    ms = bench.max_over_ranks(ms_local)
    value = bench.whole_job_tokens_per_s(8, world, ms)
    # units are dealt round-robin; no rank needs anything from another to finish its units
    mine = {u: _unit_result(1000 + u) for u in range(6) if u % world == rank}
    gathered = [None] * world
    dist.all_gather_object(gathered, mine)               # only to compare results, not part of the path
    if rank == 0:
        q.put((ms, value, gathered))
    dist.destroy_process_group()


def test_two_gloo_ranks_max_time_and_independent_units():
    from oracle import tb_oracle
    tb_oracle.build()
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    ms, value, gathered = q.get(timeout=240)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert ms == 15.0                                    # the slowest rank decides
    assert abs(value - 8 * 2 / 15e-3) < 1e-6             # whole-job tokens/s over both ranks
    merged = {}
    for d in gathered:
        merged.update(d)
    assert sorted(merged) == list(range(6))
    for u in range(6):
        assert np.array_equal(merged[u], _unit_result(1000 + u))   # same as one rank doing every unit


def test_single_process_helpers_are_identity():
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.whole_job_tokens_per_s(16, 1, 2.0) == 8000.0
