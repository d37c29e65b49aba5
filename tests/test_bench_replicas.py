"""The N > 1 path of the benchmark on CPU: world size 2 over gloo. The hot path has no exchange
step, so N GPUs run N independent replicas; what the ranks share is the barrier and the
max-over-ranks of the timing from which whole-job throughput is computed."""
import os
import socket
import sys
from pathlib import Path

import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, str(ROOT))
    import torch.distributed as dist
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    bench.barrier()
    mine = 10.0 + 5.0 * rank            # rank 1 is the slow replica
    worst = bench.max_over_ranks(mine)
    summ = bench.replica_summary(tokens_per_rank_step=4096, steps=4, max_ms=worst, world=world)
    out.put((rank, worst, summ["value"], summ["ms_per_step"]))
    bench.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_max_time_and_aggregate_throughput():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, worst, value, ms in res:
        assert worst == 15.0                                   # every rank sees the slowest replica's time
        assert abs(value - 2 * 4096 * 4 / 15e-3) < 1e-6        # both replicas' tokens over that time
        assert abs(ms - 15.0 / 4) < 1e-12


def test_single_process_is_identity():
    sys.path.insert(0, str(ROOT))
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    bench.barrier()
    assert bench.replica_summary(100, 2, 10.0, 1) == {"value": 100 * 2 / 10e-3, "ms_per_step": 5.0}
    sh = bench.workload_shape("cfg2")
    assert sh["n_layers"] == 28 and sh["b"] == 1024
    # algorithmic bytes: K and V of all 3584 units at 1088 keys dominate (~2.0 GB)
    assert abs(bench.algorithmic_bytes(sh, 1088, False) / 1e9 - 2.0) < 0.05
