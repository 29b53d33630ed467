"""The N > 1 path of bench.py on CPU: two gloo ranks, max-over-ranks timing and whole-job throughput.
(The aggregation path has no exchange step, so ranks are independent replicas; only the reporting is shared.)"""
import os
import socket
import sys

import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist

    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank)          # rank 1 is the slower one
    dist.barrier()
    q.put((rank, ms, bench.whole_job_value(2_000_000_000, world, ms)))
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_summed_throughput():
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
    assert [g[1] for g in got] == [15.0, 15.0]
    assert abs(got[0][2] - 2 * 2e9 / 15e-3 / 1e9) < 1e-9


def test_single_process_is_passthrough():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert abs(bench.whole_job_value(10**9, 1, 1.0) - 1000.0) < 1e-9


def test_median_operation_count_of_small_networks():
    """Three inputs: comparators (0,1), (0,2), (1,2); the middle output needs min of the last, max of the second and
    both outputs of the first = 4 operations.  One input needs none; 129 to 256 rows are counted for the two-lane
    scheme (two full sorts of half the rows, the split and the reduction); larger sizes report 0."""
    import bench
    assert bench.median_minmax_ops(1) == 0
    assert bench.median_minmax_ops(3) == 4
    assert bench.median_minmax_ops(300) == 0
    H = 104                                   # 200 rows: two lanes of 104 keys
    assert bench.median_minmax_ops(200) == 2 * (2 * len(bench.merge_exchange_net(H)) + 2 * H - 1)
    assert bench.median_minmax_ops(45) < bench.median_minmax_ops(105)
