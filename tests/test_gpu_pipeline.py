"""Rotation beside other work on the GPU (the paper's cross-iteration pipeline, section 4.3.2, overlaps the
transfers of the next iteration with the computation of the current one), the completion events a compute
stream waits on, and the entry points and switches around them.  All against the CPU oracle, bit for bit."""
import ctypes as C
import os

import numpy as np
import pytest

from paper_2601_20309_b200 import binding as B
from paper_2601_20309_b200 import workload as W

pytestmark = pytest.mark.gpu

PATHS = {"auto": 0, "zerocopy": 1, "staged": 2, "ce2d": 3}


def _pair(*a, **k):
    from gpu_harness import Pair
    return Pair(*a, **k)


def _driver():
    """The CUDA driver API, used here only to make a torch stream wait for an event the library owns."""
    d = C.CDLL("libcuda.so.1")
    d.cuStreamWaitEvent.restype = C.c_int
    d.cuStreamWaitEvent.argtypes = [C.c_void_p, C.c_void_p, C.c_uint]
    d.cuEventQuery.restype = C.c_int
    d.cuEventQuery.argtypes = [C.c_void_p]
    d.cuEventSynchronize.restype = C.c_int
    d.cuEventSynchronize.argtypes = [C.c_void_p]
    return d


@pytest.mark.parametrize("path", ["zerocopy", "staged"])
def test_rotation_beside_a_busy_compute_stream_matches_the_oracle(path):
    """Config 2 scaled down (8B shape, 2 MiB blocks): the paired rotation and the pairwise ones are issued
    while an unrelated element-wise kernel keeps every SM busy on a third stream, before and after and all
    the while; both pools must still equal the oracle, and the bystander's own result must be right."""
    import torch
    w = W.config2_8b(nb_gpu=320, nb_host=448, n_req=16, median=96, max_tokens=512, n_rot=4)
    p = _pair(w.shape, w.nb_gpu, w.nb_host, seed=w.seed, path=PATHS[path])
    try:
        side = torch.cuda.Stream()
        x = torch.ones(64 << 20, dtype=torch.float32, device="cuda:0")          # 256 MiB: HBM-bound passes
        passes = 0
        with torch.cuda.stream(side):
            for _ in range(40):
                x.add_(1.0)
                passes += 1
        assert p.rotate_both(w.steps[0]) == 0
        for r in w.extra["pairs"]:
            with torch.cuda.stream(side):
                for _ in range(6):
                    x.add_(1.0)
                    passes += 1
            assert p.rotate_both(r) == 0
        p.assert_equal(f"rotation beside compute ({path})")
        side.synchronize()
        assert float(x[0].item()) == 1.0 + passes and float(x[-1].item()) == 1.0 + passes
        assert p.pool.kv_get_stats()["device_status"] == 0
    finally:
        p.close()


@pytest.mark.parametrize("path", ["auto", "zerocopy", "staged"])
def test_completion_event_lets_a_compute_stream_pick_up_swapped_in_blocks(path):
    import torch
    drv = _driver()
    shape = W.SHAPE_8B
    p = _pair(shape, 96, 96, seed=13, path=PATHS[path])
    try:
        assert p.pool.kv_completion_event(0) is None and p.pool.kv_completion_event(1) is None
        rng = np.random.default_rng(2)
        ih = rng.choice(96, 64, replace=False).astype(np.int32)
        ig = rng.choice(96, 64, replace=False).astype(np.int32)
        assert p.oracle.swap_in(ih, ig) == 0
        snap = torch.empty_like(p.dev)
        consumer = torch.cuda.Stream()
        assert p.pool.kv_swap_in(ih, ig) == 0                                   # 128 MiB: still in flight below
        ev = p.pool.kv_completion_event(1)
        assert ev is not None and p.pool.kv_completion_event(0) is None
        assert drv.cuStreamWaitEvent(consumer.cuda_stream, ev, 0) == 0
        with torch.cuda.stream(consumer):
            snap.copy_(p.dev, non_blocking=True)                                # would see half-written blocks without the wait
        consumer.synchronize()
        assert np.array_equal(snap.cpu().numpy(), p.oracle.G)
        assert drv.cuEventQuery(ev) == 0                                        # complete
        # a swap-out has an event of its own; the swap-in's stays what it was
        og = rng.choice(96, 8, replace=False).astype(np.int32)
        oh = np.setdiff1d(np.arange(96), ih)[:8].astype(np.int32)
        assert p.oracle.swap_out(og, oh) == 0 and p.pool.kv_swap_out(og, oh) == 0
        ev_out = p.pool.kv_completion_event(0)
        assert ev_out is not None and ev_out != ev and p.pool.kv_completion_event(1) == ev
        assert drv.cuEventSynchronize(ev_out) == 0
        p.assert_equal("after waiting on the exported events")
    finally:
        p.close()


@pytest.mark.parametrize("kernel", [0, B.KV_FLAG_LDST_KERNEL], ids=["bulk", "ldst"])
@pytest.mark.parametrize("path", ["zerocopy", "staged"])
def test_bounds_checking_kernels_move_the_same_bytes_and_report_nothing_on_valid_lists(path, kernel):
    """KV_FLAG_DEBUG_BOUNDS: every list handed to the kernels here is valid (the host refuses the others
    before any launch), so the check must change nothing and the status word must stay clean."""
    w = W.config2_8b(nb_gpu=160, nb_host=224, n_req=16, median=48, max_tokens=256, n_rot=4)
    p = _pair(w.shape, w.nb_gpu, w.nb_host, seed=w.seed, path=PATHS[path], flags=B.KV_FLAG_DEBUG_BOUNDS | kernel,
              staging_bytes=24 * w.shape.block_bytes)
    try:
        assert p.rotate_both(w.steps[0]) == 0
        for r in w.extra["pairs"][:6]:
            assert p.rotate_both(r) == 0
        p.assert_equal("bounds-checked rotation")
        assert p.pool.kv_get_stats()["device_status"] == 0
        assert p.pool.kv_swap_out([w.nb_gpu], [0], check=False) == B.KV_ERR_RANGE       # refused on the host, as ever
        assert p.pool.kv_sync(check=False) == B.KV_OK
    finally:
        p.close()


def test_rotate_with_request_boundaries_moves_the_same_bytes_and_counts_requests():
    w = W.config2_8b(nb_gpu=160, nb_host=224, n_req=16, median=48, max_tokens=256, n_rot=4)
    r = w.steps[0]
    p = _pair(w.shape, w.nb_gpu, w.nb_host, seed=w.seed)
    try:
        P = p.pool
        assert p.oracle.rotate(r.out_gpu, r.out_host, r.in_host, r.in_gpu) == 0
        assert P.kv_rotate_req(r.out_gpu, r.out_host, r.out_req_offsets, r.in_host, r.in_gpu, r.in_req_offsets) == 0
        p.assert_equal("kv_rotate_req")
        st = P.kv_get_stats()
        assert (st["requests_out"], st["requests_in"]) == (4, 4)
        assert st["bytes_out"] == r.n_out * w.shape.block_bytes and st["bytes_in"] == r.n_in * w.shape.block_bytes
        # offsets that do not describe the lists: refused, nothing moves, nothing counted
        r2 = w.extra["pairs"][0]
        bad = [np.array([0, r2.n_out - 1]), np.array([1, r2.n_out]), np.array([0, r2.n_out + 1, r2.n_out])]
        for off in bad:
            assert P.kv_rotate_req(r2.out_gpu, r2.out_host, off, r2.in_host, r2.in_gpu, r2.in_req_offsets,
                                   check=False) == B.KV_ERR_INVALID_ARG
        assert P.kv_rotate_req(r2.out_gpu, r2.out_host, [], r2.in_host, r2.in_gpu, r2.in_req_offsets,
                               check=False) == B.KV_ERR_INVALID_ARG
        p.assert_equal("after refused kv_rotate_req calls")
        assert P.kv_get_stats()["requests_out"] == 4
        # one direction empty
        assert p.oracle.swap_in(r2.in_host, r2.in_gpu) == 0
        assert P.kv_rotate_req([], [], [], r2.in_host, r2.in_gpu, r2.in_req_offsets) == 0
        p.assert_equal("kv_rotate_req, swap-in only")
        st = P.kv_get_stats()
        assert (st["requests_out"], st["requests_in"]) == (4, 5)
    finally:
        p.close()


def test_environment_overrides_of_path_and_cta_counts():
    import torch
    w = W.config1_tiny()
    r = w.steps[0]
    keys = ("DUPLEXKV_PATH", "DUPLEXKV_SMS_OUT", "DUPLEXKV_SMS_IN")
    saved = {k: os.environ.pop(k, None) for k in keys}
    try:
        for name, want in (("staged", 2), ("naive", 4), ("zerocopy", 1)):
            os.environ["DUPLEXKV_PATH"] = name
            os.environ["DUPLEXKV_SMS_OUT"], os.environ["DUPLEXKV_SMS_IN"] = "3", "5"
            p = _pair(w.shape, w.nb_gpu, w.nb_host, seed=w.seed, path=3)                # the config says ce2d
            try:
                assert p.rotate_both(r) == 0
                p.assert_equal(f"DUPLEXKV_PATH={name}")
                st = p.pool.kv_get_stats()
                assert (st["last_path_out"], st["last_path_in"]) == (want, want)
            finally:
                p.close()
        dev = torch.zeros(w.nb_gpu * w.shape.block_bytes, dtype=torch.uint8, device="cuda:0")
        for k, v in (("DUPLEXKV_PATH", "fastest"), ("DUPLEXKV_SMS_OUT", "many"), ("DUPLEXKV_SMS_IN", "-2")):
            for kk in keys:
                os.environ.pop(kk, None)
            os.environ[k] = v
            with pytest.raises(B.KVError) as e:
                B.KVPool(w.shape.num_layers, w.shape.block_size, w.shape.kv_heads, w.shape.head_dim, w.nb_gpu,
                         w.nb_host, dev.data_ptr())
            assert e.value.code == B.KV_ERR_INVALID_ARG
    finally:
        for k in keys:
            os.environ.pop(k, None)
            if saved[k] is not None:
                os.environ[k] = saved[k]


def test_cta_count_setter_changes_nothing_but_the_launch_shape():
    w = W.config2_8b(nb_gpu=160, nb_host=224, n_req=16, median=48, max_tokens=256, n_rot=4)
    p = _pair(w.shape, w.nb_gpu, w.nb_host, seed=w.seed, path=1)
    try:
        for k, (co, ci) in enumerate(((8, 8), (1, 148), (0, 0))):
            assert p.pool.kv_pool_set_ctas(co, ci) == 0
            assert p.rotate_both(w.extra["pairs"][k]) == 0
        assert p.pool.kv_pool_set_ctas(-1, 4, check=False) == B.KV_ERR_INVALID_ARG
        p.assert_equal("rotations with 8, 1/148 and default CTAs")
    finally:
        p.close()


def test_second_pool_over_page_locked_memory_of_the_first():
    """Host memory that is page-locked already (here: another pool's) is taken as it is, so pools of
    different shapes can use one host buffer in turn without pinning it again."""
    import torch
    a = _pair(W.KVShape(4, 16, 8, 128), 40, 60, seed=21, path=2)                # 256 KiB blocks
    try:
        base, nbytes = a.pool.kv_host_ptr()
        shape_b = W.KVShape(2, 16, 8, 128)                                      # 128 KiB blocks: twice as many fit
        from oracle.kv_oracle import ByteOracle
        nbg, nbh = 80, nbytes // shape_b.block_bytes
        ob = ByteOracle(shape_b.num_layers, shape_b.block_size, shape_b.kv_heads, shape_b.head_dim, nbg, nbh)
        ob.G[:] = a.gpu_bytes()                                                 # the same bytes, seen with another shape
        ob.Hs[:] = a.pool.host_array()
        pb = B.KVPool(shape_b.num_layers, shape_b.block_size, shape_b.kv_heads, shape_b.head_dim, nbg, nbh,
                      a.dev.data_ptr(), host_base=base, path=2)
        rng = np.random.default_rng(5)
        og, oh = rng.choice(nbg, 30, replace=False).astype(np.int32), rng.choice(nbh, 30, replace=False).astype(np.int32)
        ig = np.setdiff1d(np.arange(nbg), og)[:20].astype(np.int32)
        ih = np.setdiff1d(np.arange(nbh), oh)[:20].astype(np.int32)
        assert ob.rotate(og, oh, ih, ig) == 0
        assert pb.kv_rotate(og, oh, ih, ig) == 0
        pb.kv_sync()
        torch.cuda.synchronize()
        assert np.array_equal(a.dev.cpu().numpy(), ob.G)
        assert np.array_equal(pb.host_array(), ob.Hs)
        pb.destroy()                                                            # must leave the first pool's memory page-locked
        a.oracle.G[:] = ob.G
        a.oracle.Hs[:] = ob.Hs
        r = np.arange(10, dtype=np.int32)
        assert a.oracle.swap_out(r, r + 5) == 0 and a.pool.kv_swap_out(r, r + 5) == 0
        a.assert_equal("first pool after the second one is gone")
    finally:
        a.close()


@pytest.mark.parametrize("how", ["cuda", None], ids=["cudaHostAlloc", "huge-page-mapping"])
@pytest.mark.parametrize("path", [1, 2], ids=["zerocopy", "staged"])
def test_both_ways_of_allocating_the_host_pool(how, path):
    """The library's own host pool is a registered huge-page mapping by default and cudaHostAlloc memory on
    DUPLEXKV_HOST_ALLOC=cuda (and whenever the mapping cannot be had): same results, and the pool's memory can
    be written and read through kv_host_ptr either way.  300 MiB, so that several threads touch it."""
    shape = W.KVShape(4, 16, 8, 128)                                              # 256 KiB blocks
    nbg, nbh = 300, 1200
    saved = os.environ.pop("DUPLEXKV_HOST_ALLOC", None)
    try:
        if how:
            os.environ["DUPLEXKV_HOST_ALLOC"] = how
        p = _pair(shape, nbg, nbh, seed=31, path=path)
        try:
            base, nbytes = p.pool.kv_host_ptr()
            assert nbytes == nbh * shape.block_bytes and base % 4096 == 0
            rng = np.random.default_rng(8)
            pg, ph = rng.permutation(nbg).astype(np.int32), rng.permutation(nbh).astype(np.int32)
            r = W.Rotation(pg[:140], ph[:140], ph[140:280], pg[140:280], np.zeros(1), np.zeros(1))
            assert p.rotate_both(r) == 0
            p.assert_equal(f"host pool allocated by {how or 'the default'}")
        finally:
            p.close()
    finally:
        os.environ.pop("DUPLEXKV_HOST_ALLOC", None)
        if saved is not None:
            os.environ["DUPLEXKV_HOST_ALLOC"] = saved
