"""The N>1 path of the benchmark on CPU: two gloo ranks, each with its own replica of the workload (no
data-path collective), timings reduced with MAX over ranks, whole-job value = world * per-rank work /
slowest rank's time.  Also: the reference arm runs on rank 0 only."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    my_ms = [10.0 + 5.0 * rank, 30.0 - 7.0 * rank]            # rank 1 is slower on the first, faster on the second
    red = bench.max_over_ranks(torch, dist, my_ms, "cpu")
    dist.barrier()
    q.put((rank, red, bench.whole_job_value(world, 2.0e12, red[0])))
    dist.destroy_process_group()


def test_two_ranks_reduce_with_max_and_aggregate():
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
    for rank, red, value in got:
        assert red == [15.0, 30.0]                             # slowest rank decides
        assert abs(value - 2 * 2.0e12 / 15.0e-3 / 1e12) < 1e-9   # whole job = 2 replicas / slowest time


def test_single_process_has_no_collective():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(torch, None, [1.5, 2.5], "cpu") == [1.5, 2.5]
    assert bench.whole_job_value(1, 1.0e12, 1.0) == 1000.0      # 1e12 flop in 1 ms = 1000 TFLOP/s


def test_reference_arm_runs_on_rank0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env["RANK"] = "0"
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0", "--ref-rows", "4"], env=env, capture_output=True, text=True,
                         timeout=300)
    assert out.returncode == 0
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0


def test_flop_accounting_follows_eq1_and_timed_loop_marks():
    # the benchmark's flop numerator is Eq. (1) summed over the batch; the sparse event marks of very short steps
    # still bracket exactly `steps` steps
    sys.path.insert(0, ROOT)
    import bench
    from oracle import reference as orc
    from paper_2609_04774_b200 import workloads as wl
    for cfg in (1, 2, 4, 5):
        w = bench.get_workload(cfg)
        assert bench.pairs_of(w) == sum(orc.remaining_workload(r.new_len, r.prefix_len) for r in w.requests)
        assert bench.flops_of(w) == 4 * 128 * w.Hq * bench.pairs_of(w)
    assert bench.pairs_of(wl.config2()) == 58722304 and bench.flops_of(wl.config3()) == 4 * 128 * 32 * 8590000128

    class FakeEvent:
        clock = 0.0

        def __init__(self, enable_timing=True):
            self.t = None

        def record(self):
            self.t = FakeEvent.clock

        def elapsed_time(self, other):
            return other.t - self.t

    class FakeCuda:
        Event = FakeEvent

        @staticmethod
        def synchronize():
            pass

    class FakeTorch:
        cuda = FakeCuda

    calls = []

    def step():
        calls.append(1)
        FakeEvent.clock += 2.0

    total, per = bench.timed_loop(FakeTorch, step, 37, 3, stride=16)
    assert len(calls) == 40 and total == 74.0 and per == [2.0, 2.0, 2.0]
    total, per = bench.timed_loop(FakeTorch, step, 5, 0)
    assert total == 10.0 and per == [2.0] * 5
