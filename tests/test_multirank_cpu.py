"""The N > 1 plumbing of the benchmark on CPU: two gloo ranks.  The path shards by sequence with no data
exchange, so what is multi-rank is only the timing reduction (max over ranks), the whole-job aggregation and
the per-rank input streams."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import bench
    from paper_2408_05646_b200 import synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.rank_env() == (rank, world, rank)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, torch.device("cpu"))       # rank 1 is the slow one
    dist.barrier()
    # each rank draws its own sequences for its batch shard
    wl = synth.WORKLOADS["tiny_fp32"]
    W = synth.mixing_matrices(wl.n_heads, wl.rho, wl.d_head, wl.index, "W_K")
    rows = synth.lowrank_rows(W, 1, 4, wl.sigma, wl.index, "K", chunk=bench.rank_chunk_base(rank), dtype=torch.float32)
    q.put((rank, ms, bench.whole_job_gbs(1_000_000_000, world, ms), float(rows.sum())))
    dist.destroy_process_group()


def test_two_gloo_ranks_reduce_timing_and_aggregate():
    world, port = 2, 29533 + os.getpid() % 200
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[1] for r in res] == [15.0, 15.0]                     # both ranks see the slowest rank's time
    assert all(abs(r[2] - 2 * 1e9 / 15e-3 / 1e9) < 1e-9 for r in res)   # whole job = sum over ranks / max time
    assert res[0][3] != res[1][3]                                   # different sequences per shard


def test_reference_arm_other_ranks_do_nothing(monkeypatch, capsys):
    sys.path.insert(0, ROOT)
    import bench
    monkeypatch.setenv("RANK", "1")
    monkeypatch.setenv("WORLD_SIZE", "2")
    monkeypatch.setattr(sys, "argv", ["bench.py", "--impl", "reference", "--workload", "tiny_fp32"])
    bench.main()
    assert capsys.readouterr().out == ""
