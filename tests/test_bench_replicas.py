"""N > 1 is "replicas only": ranks decode independent sequences and bench.py only aggregates
timings (MAX over ranks) and token counts (SUM).  Covered here with two gloo ranks on CPU."""
import os
import socket
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import bench
        # rank r: r+1 seconds of device time, 10(r+1) ms end to end, 100+r and 200+r tokens
        res = bench.aggregate_over_ranks(1000.0 * (rank + 1), 0.01 * (rank + 1), 100 + rank, 200 + rank, "cpu")
        out.put((rank, res))
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_two_replicas_max_time_sum_tokens():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = dict(out.get(timeout=90) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for r in range(world):
        ms, e2e, tok, tok_e2e = got[r]
        assert ms == 2000.0 and e2e == pytest.approx(0.02)
        assert tok == 201.0 and tok_e2e == 401.0
    # whole-job throughput = all ranks' tokens over the slowest rank's time
    assert got[0][2] / (got[0][0] * 1e-3) == pytest.approx(100.5)


def test_reference_arm_only_rank0_works():
    """Under torchrun the oracle arm runs on rank 0 alone; other ranks leave without work."""
    import subprocess
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1", "--warmup", "0"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_pipelined_steps_keeps_two_in_flight_and_collects_every_result():
    """bench.pipelined_steps against a fake context: never more than two steps enqueued and not yet waited
    for, results handed back oldest first, nothing left in flight, every step's tokens counted."""
    sys.path.insert(0, ROOT)
    import bench

    class Fake:
        def __init__(self):
            self.queue, self.max_in_flight, self.order = [], 0, []

        def step_async(self, seqs, forced):
            self.queue.append(list(forced))
            self.max_in_flight = max(self.max_in_flight, len(self.queue))
            assert len(self.queue) <= 2

        def step_wait(self):
            f = self.queue.pop(0)
            self.order.append(f)
            return [[0] * x for x in f], f

    for n in (0, 1, 2, 5):
        t = Fake()
        forced = [[1 + i % 3, 2] for i in range(n)]
        assert bench.pipelined_steps(t, [0, 1], forced) == sum(sum(f) for f in forced)
        assert t.queue == [] and t.order == forced and t.max_in_flight == min(n, 2)
