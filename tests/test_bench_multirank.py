"""The N > 1 plumbing of bench.py on CPU: two gloo ranks, no GPU.  The path
shards into independent replicas, so the only cross-rank steps are the barrier
and the max-time / sum-of-units reduction."""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    import bench

    r, w = bench.dist_init("gloo")
    bench.barrier()
    ms, units = bench.reduce_step_time(10.0 + 5.0 * rank, 100.0 * (rank + 1))
    agree_all = bench.all_ranks_agree(True)
    agree_one = bench.all_ranks_agree(rank == 0)      # rank 1 objects: nobody proceeds
    bench.barrier()
    q.put((r, w, ms, units, agree_all, agree_one))
    import torch.distributed as dist

    dist.destroy_process_group()


def test_time_is_max_and_units_are_summed_over_ranks():
    import torch.multiprocessing as mp

    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[0] for g in got] == [0, 1]
    for _, world, ms, units, agree_all, agree_one in got:
        assert world == 2 and ms == 15.0 and units == 300.0
        assert agree_all is True and agree_one is False


def test_single_process_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench

    assert bench.reduce_step_time(3.0, 7.0) == (3.0, 7.0)
    assert bench.all_ranks_agree(True) and not bench.all_ranks_agree(False)
    bench.barrier()


def test_reference_arm_runs_on_rank0_only():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--gpus", "2", "--steps", "1", "--warmup", "0"], env=env,
                         capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""


def test_step_bytes_accounting_matches_the_library():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2408_08147_b200 import binding as B
    from paper_2408_08147_b200 import build as pdkv_build
    from paper_2408_08147_b200 import workloads as W

    pdkv_build.build_library()
    B.pdkv_tune("dry_run", 1)
    try:
        for w in (W.make_config(5, num_layers=2, n_req=50), W.make_config(3, num_layers=1, n_req=9)):
            ps = B.pdkv_pool_create(B.desc_of(w.src), 0x7F0000000000, w.src.num_bytes(), 0)
            pd = B.pdkv_pool_create(B.desc_of(w.dst), 0x7E0000000000, w.dst.num_bytes(), 0)
            b = w.batch
            plan = B.pdkv_plan_create(ps, pd, 0, b.seq_len, b.src_tbl_off, b.src_tbl, b.dst_tbl_off,
                                      b.dst_tbl, b.dst_skip)
            per_op = [sum(B.pdkv_plan_traffic(plan, op)) for op in range(3)]
            assert sum(per_op) == bench.step_bytes_of(w)
            assert per_op == [bench.op_bytes_of(w)[k] for k in ("pack", "unpack", "fused")]
            B.pdkv_plan_destroy(plan)
            B.pdkv_pool_destroy(ps)
            B.pdkv_pool_destroy(pd)
    finally:
        B.pdkv_tune("dry_run", 0)
