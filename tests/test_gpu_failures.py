"""Failure handling on the GPU, exercised without faulting or hanging anything: a bounded device-side
wait is made to run out (a limit of zero on healthy loads; a barrier that nothing completes, with a 1 ms
limit), the kernel returns normally, the host reads the status, and the device stays usable."""
import numpy as np
import pytest

from paper_2601_20309_b200 import binding as B
from paper_2601_20309_b200 import workload as W

pytestmark = pytest.mark.gpu


def _pair(*a, **k):
    from gpu_harness import Pair
    return Pair(*a, **k)


def _guards_intact(p):
    p.torch.cuda.synchronize()
    lo, hi = p.buf[:p.guard], p.buf[p.guard + p.oracle.G.size:]
    return bool((lo == 0xC3).all()) and bool((hi == 0xC3).all())


def test_bounded_wait_gives_up_on_a_barrier_that_nothing_completes():
    """The wait the copy kernels use, on a barrier that expects bytes no copy delivers: it must return
    "ran out" after about the limit, and the kernel must end by itself."""
    import torch
    from paper_2601_20309_b200 import poolfill as F
    gave_up, waited_ns = F.wait_runs_out(1_000_000)
    assert gave_up
    assert 900_000 <= waited_ns <= 50_000_000, waited_ns
    gave_up, waited_ns = F.wait_runs_out(0)                   # no time allowed after the immediate polls
    assert gave_up and waited_ns < 1_000_000
    x = torch.arange(1000, device="cuda:0")
    assert int(x.sum().item()) == 499500                      # the context is alive


@pytest.mark.parametrize("path", ["zerocopy", "staged"])
def test_a_wait_that_runs_out_is_reported_and_the_device_stays_usable(path):
    """Every address is valid and every load is healthy; the pool is only told to allow its kernels'
    waits no time at all.  The kernels must record the timeout, wait for what they have in flight and
    return; kv_sync must say KV_ERR_TIMEOUT; nothing outside the pools may be written; a fresh pool on the
    same device must then rotate bit-exactly."""
    w = W.config1_tiny()
    r = w.steps[0]
    p = _pair(w.shape, w.nb_gpu, w.nb_host, seed=w.seed, path={"zerocopy": 1, "staged": 2}[path])
    try:
        assert p.pool.kv_pool_set_wait_limit(0, 0) == 0
        assert p.pool.kv_rotate(r.out_gpu, r.out_host, r.in_host, r.in_gpu, check=False) == 0   # issued fine
        assert p.pool.kv_sync(check=False) == B.KV_ERR_TIMEOUT
        assert "status 0x1" in p.pool.kv_last_error()
        assert p.pool.kv_get_stats()["device_status"] & 1
        assert _guards_intact(p)
        # the error is sticky: the pool keeps reporting it, and refuses nothing else silently
        assert p.pool.kv_sync(check=False) == B.KV_ERR_TIMEOUT
    finally:
        p.close()
    q = _pair(w.shape, w.nb_gpu, w.nb_host, seed=w.seed, path={"zerocopy": 1, "staged": 2}[path])
    try:
        assert q.rotate_both(r) == 0
        q.assert_equal("rotation on a fresh pool after the timed-out one")
        assert q.pool.kv_get_stats()["device_status"] == 0
    finally:
        q.close()


@pytest.mark.parametrize("path", ["zerocopy", "staged"])
def test_a_wait_that_runs_out_with_several_issuing_warps_per_cta(path):
    """The same with 2 KiB segments, where every CTA runs several rings (one per warp): each ring's thread
    records the timeout, waits for its own loads in flight and returns."""
    shape = W.KVShape(2, 8, 1, 128)
    nbg, nbh, n = 256, 512, 40
    rng = np.random.default_rng(11)
    pg, ph = rng.permutation(nbg).astype(np.int32), rng.permutation(nbh).astype(np.int32)
    r = W.Rotation(pg[:n], ph[:n], ph[n:2 * n], pg[n:2 * n], np.zeros(1), np.zeros(1))
    pid = {"zerocopy": 1, "staged": 2}[path]
    p = _pair(shape, nbg, nbh, seed=5, path=pid)
    try:
        assert p.pool.kv_pool_set_wait_limit(0, 0) == 0
        assert p.pool.kv_rotate(r.out_gpu, r.out_host, r.in_host, r.in_gpu, check=False) == 0
        assert p.pool.kv_sync(check=False) == B.KV_ERR_TIMEOUT
        assert p.pool.kv_get_stats()["device_status"] & 1
        assert _guards_intact(p)
    finally:
        p.close()
    q = _pair(shape, nbg, nbh, seed=5, path=pid)
    try:
        assert q.rotate_both(r) == 0
        q.assert_equal("rotation on a fresh pool after the timed-out one")
        assert q.pool.kv_get_stats()["device_status"] == 0
    finally:
        q.close()


def test_wait_limit_arguments():
    w = W.config1_tiny()
    p = _pair(w.shape, w.nb_gpu, w.nb_host, seed=w.seed, path=1)
    try:
        assert p.pool.kv_pool_set_wait_limit(16, 61 * 10 ** 9, check=False) == B.KV_ERR_INVALID_ARG
        assert p.pool.kv_pool_set_wait_limit(4, 10 ** 9) == 0          # a shorter but ample bound changes nothing
        assert p.rotate_both(w.steps[0]) == 0
        p.assert_equal("rotation with a 1 s wait bound")
    finally:
        p.close()
