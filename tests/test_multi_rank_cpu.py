"""The N > 1 plumbing of bench.py on CPU: two gloo ranks on 127.0.0.1.

The path shards by batch element with no data-path collective, so what the ranks share is only
the rendezvous, the barriers around the timed region, the max-over-ranks time and the whole-job
throughput computed from it.  Each rank must also draw its own batch element."""
import os
import socket
import sys

import pytest
import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    import bench
    from paper_2609_33135_b200 import workloads as wl
    r, w, _ = bench.dist_setup(world, backend="gloo")
    assert (r, w) == (rank, world)
    bench.barrier(w)
    local_ms = 10.0 + 5.0 * rank                       # rank 1 is the slow one
    total_ms = bench.max_over_ranks(local_ms, w)
    bench.barrier(w)
    wk = wl.prefill_workload("t", bench.rank_seed(7, rank), 1, 128, 2, 1, True)
    torch.save({"rank": r, "total_ms": total_ms, "value": bench.whole_job_value(w, 1e12, total_ms),
                "q_sum": float(wk.q.float().sum())}, os.path.join(out_dir, f"r{rank}.pt"))
    import torch.distributed as dist
    dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_two_gloo_ranks_share_time_and_report_whole_job(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    res = [torch.load(tmp_path / f"r{r}.pt") for r in range(world)]
    assert [x["rank"] for x in res] == [0, 1]
    # every rank sees the slowest rank's time, and the job value counts both ranks' work over it
    assert all(x["total_ms"] == 15.0 for x in res)
    assert all(abs(x["value"] - 2 * 1e12 / 15e-3 / 1e12) < 1e-9 for x in res)
    # different batch elements per rank
    assert res[0]["q_sum"] != res[1]["q_sum"]


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.dist_setup(1) == (0, 1, 0)
    assert bench.max_over_ranks(3.5, 1) == 3.5
    assert bench.whole_job_value(1, 2e12, 1000.0) == 2.0
    assert bench.rank_seed(1002, 0) == 1002 and bench.rank_seed(1002, 3) != bench.rank_seed(1002, 2)


def test_reference_arm_runs_on_rank_zero_only(capsys):
    sys.path.insert(0, ROOT)
    import bench

    class A:
        gpus, steps, warmup = 2, 1, 0
    bench.run_reference(A, rank=1)        # other ranks exit without work or output
    assert capsys.readouterr().out == ""


def _spawn_probe(rank, n, port, argv):
    """Stands in for bench._spawned_rank: same arguments; sets the same environment through it but stops before
    the CUDA part, then goes through the rendezvous on gloo."""
    sys.path.insert(0, ROOT)
    import bench
    orig_main = bench.main
    seen = {}
    bench.main = lambda: seen.update(rank=os.environ["RANK"], world=os.environ["WORLD_SIZE"],
                                     local=os.environ["LOCAL_RANK"], addr=os.environ["MASTER_ADDR"], argv=list(sys.argv))
    try:
        bench._spawned_rank(rank, n, port, argv)
    finally:
        bench.main = orig_main
    assert seen == {"rank": str(rank), "world": str(n), "local": str(rank), "addr": "127.0.0.1", "argv": argv}
    r, w, _ = bench.dist_setup(n, backend="gloo")
    assert (r, w) == (rank, n)
    assert bench.max_over_ranks(float(rank), w) == float(n - 1)
    import torch.distributed as dist
    dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_plain_invocation_with_gpus_spawns_its_own_ranks(monkeypatch):
    """`python bench.py --gpus 2` without a launcher (no RANK in the environment) must start the ranks itself."""
    sys.path.insert(0, ROOT)
    import bench
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT"):
        monkeypatch.delenv(k, raising=False)
    monkeypatch.setattr(sys, "argv", ["bench.py", "--gpus", "2", "--steps", "1"])
    bench.spawn_ranks(2, fn=_spawn_probe)
    # and main() takes that route when RANK is unset
    called = {}
    monkeypatch.setattr(bench, "spawn_ranks", lambda n: called.setdefault("n", n))
    bench.main()
    assert called == {"n": 2}
