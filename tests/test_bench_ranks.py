"""The benchmark's multi-rank bookkeeping on CPU: two gloo ranks on 127.0.0.1.  The path itself needs no
exchange between GPUs (every rank runs a replica), so what N > 1 adds is the max-over-ranks time, the
whole-job rate, and the rule that only rank 0 reports."""
import io
import os
import socket
import sys
from contextlib import redirect_stdout

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 * (rank + 1), dist, torch.device("cpu"))
    rate = bench.whole_job_rate(world, 1000, 4, ms)
    dist.barrier()
    dist.destroy_process_group()
    out.put((rank, ms, rate))


def _two_ranks():
    """Runs _rank as two gloo processes; None when the rendezvous itself failed (the port was taken between
    finding it and binding it, a rank did not come up), so that the caller can try again on another port."""
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = []
    try:
        got = sorted(out.get(timeout=120) for _ in procs)
    except Exception:
        pass
    for p in procs:
        p.join(timeout=60)
        if p.is_alive():
            p.kill()
            p.join()
    if len(got) != 2 or any(p.exitcode != 0 for p in procs):
        return None
    return got


def test_two_ranks_agree_on_the_slowest_time_and_the_whole_job_rate():
    got = None
    for _ in range(3):
        got = _two_ranks()
        if got is not None:
            break
    assert got is not None, "two gloo ranks did not come up on 127.0.0.1 in three tries"
    assert [g[1] for g in got] == [20.0, 20.0]                       # the slower rank's 20 ms on both
    assert [g[2] for g in got] == [2 * 1000 * 4 / 0.020] * 2          # both replicas' units over that time


def test_single_process_needs_no_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(7.5, None, torch.device("cpu")) == 7.5
    assert bench.whole_job_rate(1, 10, 2, 4.0) == 5000.0


def test_reference_arm_is_silent_on_other_ranks():
    sys.path.insert(0, ROOT)
    import bench
    import synth

    class Args:
        gpus, steps, warmup = 2, 1, 0

    buf = io.StringIO()
    with redirect_stdout(buf):
        bench.run_reference(Args, synth.WORKLOADS["cfg1"], rank=1)
    assert buf.getvalue() == ""
