"""The N > 1 path of bench.py on CPU: the score path has no exchange step, so N ranks are N independent replicas and
the only cross-rank logic is the timing aggregation (max over ranks) and the whole-job throughput.  Run here as two
gloo processes; on GPUs the same functions run over NCCL."""
import os
import socket
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    import torch.distributed as dist
    import bench
    from paper_2605_08840_b200.inputs import CONFIGS, make_inputs

    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        # every rank draws its own replica of the layer, as bench.py does (seed offset by rank)
        case = CONFIGS["cfg1b"]
        inp = make_inputs(case, seed=case.seed + 1000 * rank)
        my_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
        total = bench.max_over_ranks(my_ms, world, "cpu")
        value = bench.whole_job_value(case.batch * case.n, world, 4, total)
        out.put((rank, total, value, float(inp.K[0, 0, 0, 0])))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_take_the_slowest_rank_and_count_both():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, t0, v0, k0), (r1, t1, v1, k1) = got
    assert (r0, r1) == (0, 1)
    assert t0 == t1 == 15.0                            # max over ranks, the same on both
    assert v0 == v1 == pytest.approx(2 * 1024 * 4 / 15e-3)   # both replicas' tokens over the slowest rank's time
    assert k0 != k1                                    # the replicas are not the same data


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(3.5, 1, "cpu") == 3.5
    assert bench.whole_job_value(1000, 1, 2, 4.0) == pytest.approx(1000 * 2 / 4e-3)
