"""The multi-GPU mode is independent replicas: no exchange on the data path, only the aggregation of the
per-rank figures (bytes are added, time is the slowest rank's).  Checked here with two gloo ranks on CPU."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2601_20309_b200 import metrics as M


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        nbytes = 7.0e9 + rank * 1.0e9            # rank 0 moved 7 GB, rank 1 moved 8 GB
        ms = 100.0 + 50.0 * rank                 # rank 1 is the slow one
        q.put((rank, M.reduce_over_ranks(nbytes, "sum", dist), M.reduce_over_ranks(ms, "max", dist),
               M.replicas_gbs(nbytes, ms, dist)))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_add_bytes_and_take_the_slowest_time():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for _, total, slowest, gbs in got:
        assert total == 15.0e9 and slowest == 150.0
        assert gbs == pytest.approx(15.0e9 / 0.150 / 1e9)


def test_single_process_is_the_identity():
    assert M.reduce_over_ranks(3.5, "max") == 3.5
    assert M.replicas_gbs(2e9, 1000.0) == pytest.approx(2.0)


def test_launcher_starts_one_replica_per_rank_and_passes_rank_zero_through():
    """What ``bench.py --gpus N`` does when no launcher started it: N processes with the rendezvous
    variables set, rank 0's single JSON line as the only output."""
    import json
    import sys
    from paper_2601_20309_b200 import replicas as R
    stub = os.path.join(os.path.dirname(os.path.abspath(__file__)), "stub_replica.py")
    codes, text = R.spawn(2, [sys.executable, stub], timeout_s=240, capture=True)
    assert codes == [0, 0]
    lines = [ln for ln in text.splitlines() if ln.strip()]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["n_gpus"] == 2
    assert rec["value"] == pytest.approx((4.0e9 + 6.0e9) / 0.075 / 1e9)     # bytes added, slowest rank's time
    codes, _ = R.spawn(2, [sys.executable, stub, "--fail-rank", "1"], timeout_s=240, capture=True)
    assert codes == [0, 3]                                                  # a failing rank is reported


def test_rank_environment():
    from paper_2601_20309_b200 import replicas as R
    env = R.rank_env(3, 8, 29511, base={"KEEP": "1"})
    assert env == {"KEEP": "1", "RANK": "3", "LOCAL_RANK": "3", "WORLD_SIZE": "8", "LOCAL_WORLD_SIZE": "8",
                   "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": "29511"}


def test_bench_gpus_flag_starts_that_many_replicas():
    """`python bench.py --gpus 2` without a launcher must start two ranks itself.  On a machine without a
    GPU each rank stops with the no-fallback message, which is enough to count them."""
    import subprocess
    import sys
    if torch.cuda.is_available():
        pytest.skip("counts ranks by their no-GPU message; covered by the stub test on a GPU box")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--steps", "1"],
                         capture_output=True, text=True, env=env, timeout=600)
    assert res.returncode != 0
    assert res.stderr.count("needs a CUDA device") == 2
    assert res.stdout.strip() == ""
