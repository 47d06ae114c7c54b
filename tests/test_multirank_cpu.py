"""The N > 1 path of the benchmark on CPU: the path does not shard (independent replicas, no
data-path collective), so all that crosses ranks is the max-over-ranks timing.  Two gloo ranks."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, device="cpu")       # rank 1 is the slow one
    val = bench.aggregate_value(bench.step_bytes(1000), world, ms)
    out.put((rank, ms, val))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_report_the_slowest_time_and_the_aggregate_rate():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    import bench
    assert [r[1] for r in res] == [15.0, 15.0]                                # both ranks see the max
    want = bench.step_bytes(1000) * 2 / 15e-3 / 1e9
    assert all(abs(r[2] - want) < 1e-9 * want for r in res)


def test_single_rank_is_the_identity_and_step_bytes_match_the_bit_budget():
    import bench
    assert bench.max_over_ranks(3.5, 1) == 3.5
    n = 1 << 20
    # 3 formats x 2 directions x (4 + (2 + b/8) + (b/8 + 2)) bytes per element, b = 4, 6, 9 (Table II)
    assert bench.step_bytes(n) == 2 * sum(8 + 2 * b / 8 for b in (4, 6, 9)) * n
