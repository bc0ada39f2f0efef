"""Parity at full size, in the launch configuration bench.py times (default path, default staging).

The pools are too large for a second copy, so the expected state comes from the oracle's tag model
(which original block each slot must hold after the calls) and the seeded content generator:
  * every block of both pools is digested on the GPU before and after by a test-only reduction; after
    the calls each digest must equal the digest its tag's origin had before (untouched blocks: their own);
  * a sample of the "before" digests is recomputed on the CPU from regenerated content, which pins the
    digests themselves;
  * a sample of touched and untouched blocks is read back in full (plain copies, not the library) and
    compared bit for bit with the regenerated content of the origin the tag model names.
"""
import numpy as np
import pytest

from paper_2601_20309_b200 import workload as W

pytestmark = pytest.mark.gpu


def _mem_available():
    with open("/proc/meminfo") as f:
        for line in f:
            if line.startswith("MemAvailable:"):
                return int(line.split()[1]) * 1024
    return 0


def _fit_host_pool(shape, nb_host):
    """bench.py's rule: shrink the host pool only if the box cannot pin it."""
    budget = int(0.70 * _mem_available())
    if nb_host * shape.block_bytes > budget:
        nb_host = max(8192, budget // shape.block_bytes)
    return nb_host


# Pinning 120 GB takes the better part of a minute, so the tests of this file share one page-locked area:
# a keeper pool of small blocks owns it, and every test's pool is created over that memory (the library
# takes memory that is page-locked already as it is).
_KEEPER = {"pool": None, "dev": None, "bytes": 0}


def _shared_host(nbytes):
    import torch
    from paper_2601_20309_b200 import binding as B
    k = _KEEPER
    if k["pool"] is not None and k["bytes"] < nbytes:
        k["pool"].destroy()
        k["pool"] = None
    if k["pool"] is None:
        shape = W.KVShape(1, 16, 8, 128)                      # 64 KiB blocks
        nb = -(-nbytes // shape.block_bytes)
        k["dev"] = torch.empty(8 * shape.block_bytes, dtype=torch.uint8, device="cuda:0")
        k["pool"] = B.KVPool(shape.num_layers, shape.block_size, shape.kv_heads, shape.head_dim, 8, nb, k["dev"].data_ptr())
        k["bytes"] = nb * shape.block_bytes
    return k["pool"].kv_host_ptr()[0]


@pytest.fixture(scope="module", autouse=True)
def _release_shared_host():
    yield
    if _KEEPER["pool"] is not None:
        _KEEPER["pool"].destroy()
        _KEEPER["pool"], _KEEPER["dev"], _KEEPER["bytes"] = None, None, 0


class _FullSize:
    def __init__(self, w):
        import torch
        from oracle.kv_definition import TagModel
        from paper_2601_20309_b200 import binding as B
        from paper_2601_20309_b200 import poolfill as F
        self.torch, self.B, self.F, self.w = torch, B, F, w
        shape = w.shape
        free_dev, _ = torch.cuda.mem_get_info()
        if free_dev < w.nb_gpu * shape.block_bytes + (6 << 30):
            pytest.skip("not enough free device memory for this pool")
        self.dev = torch.empty(w.nb_gpu * shape.block_bytes, dtype=torch.uint8, device="cuda:0")
        self.pool = B.KVPool(shape.num_layers, shape.block_size, shape.kv_heads, shape.head_dim, w.nb_gpu, w.nb_host,
                             self.dev.data_ptr(), host_base=_shared_host(w.nb_host * shape.block_bytes),
                             flags=B.KV_FLAG_TIME_KERNELS)
        host_base, _ = self.pool.kv_host_ptr()
        self.lay_g = F.Layout.device(self.dev.data_ptr(), shape, w.nb_gpu)
        self.lay_h = F.Layout.host(host_base, shape, w.nb_host)
        F.fill_blocks(self.lay_g, w.seed, W.POOL_GPU, w.nb_gpu)
        F.fill_blocks(self.lay_h, w.seed, W.POOL_HOST, w.nb_host)
        self.d0 = self.digests()
        self.rng = np.random.default_rng(5)
        # pin the digests (and the GPU fill) to the CPU generator on a sample
        for p, nb in ((W.POOL_GPU, w.nb_gpu), (W.POOL_HOST, w.nb_host)):
            for b in self.rng.choice(nb, 16, replace=False):
                assert self.d0[p][b] == F.checksum_words(W.block_words(w.seed, p, int(b), shape.words_per_block))
        self.tags = TagModel(w.nb_gpu, w.nb_host)

    def digests(self):
        return {W.POOL_GPU: self.F.checksum_blocks(self.lay_g, self.w.nb_gpu),
                W.POOL_HOST: self.F.checksum_blocks(self.lay_h, self.w.nb_host)}

    def swap_out(self, g, h):
        assert self.tags.swap_out(g.tolist(), h.tolist()) == 0 and self.pool.kv_swap_out(g, h) == 0

    def swap_in(self, h, g):
        assert self.tags.swap_in(h.tolist(), g.tolist()) == 0 and self.pool.kv_swap_in(h, g) == 0

    def rotate(self, r):
        assert self.tags.rotate(r.out_gpu.tolist(), r.out_host.tolist(), r.in_host.tolist(), r.in_gpu.tolist()) == 0
        assert self.pool.kv_rotate(r.out_gpu, r.out_host, r.in_host, r.in_gpu) == 0

    def verify(self, what, n_read_back=12):
        w, shape, tags = self.w, self.w.shape, self.tags
        self.pool.kv_sync()
        assert self.pool.kv_get_stats()["device_status"] == 0
        d1 = self.digests()
        g_origin = np.array(tags.g_tag, dtype=np.int64)         # (origin pool, origin block) per slot
        h_origin = np.array(tags.h_tag, dtype=np.int64)
        moved_g = np.flatnonzero((g_origin[:, 0] != W.POOL_GPU) | (g_origin[:, 1] != np.arange(w.nb_gpu)))
        moved_h = np.flatnonzero((h_origin[:, 0] != W.POOL_HOST) | (h_origin[:, 1] != np.arange(w.nb_host)))
        for name, origin, d_after in (("device", g_origin, d1[W.POOL_GPU]), ("host", h_origin, d1[W.POOL_HOST])):
            want = np.where(origin[:, 0] == W.POOL_GPU, self.d0[W.POOL_GPU][np.minimum(origin[:, 1], w.nb_gpu - 1)],
                            self.d0[W.POOL_HOST][np.minimum(origin[:, 1], w.nb_host - 1)])
            bad = np.flatnonzero(want != d_after)
            assert len(bad) == 0, f"{what}: {len(bad)} {name} blocks hold the wrong content, first {bad[:5]}"
        # full read-back of a sample: plain copies, compared with regenerated content of the origin
        planes = 2 * shape.num_layers
        dev3 = self.dev.view(planes, w.nb_gpu, shape.words_per_plane * 2)
        harr = self.pool.host_array()
        pick = lambda moved, nb: np.concatenate([self.rng.choice(moved, min(n_read_back, len(moved)), replace=False),
                                                 self.rng.choice(nb, 4, replace=False)])
        for b in pick(moved_g, w.nb_gpu):
            op, ob = tags.g_tag[int(b)]
            got = dev3[:, int(b), :].contiguous().cpu().numpy().view(np.uint16).reshape(-1)
            assert np.array_equal(got, W.block_words(w.seed, op, ob, shape.words_per_block)), (what, "device", int(b))
        for h in pick(moved_h, w.nb_host):
            op, ob = tags.h_tag[int(h)]
            got = harr[int(h) * shape.block_bytes:(int(h) + 1) * shape.block_bytes].view(np.uint16)
            assert np.array_equal(got, W.block_words(w.seed, op, ob, shape.words_per_block)), (what, "host", int(h))
        return len(moved_g), len(moved_h)

    def close(self):
        self.pool.destroy()
        del self.dev
        self.torch.cuda.empty_cache()


def test_config2_full_size_rotate_single_swaps_and_pairwise_rotations():
    """60 GB device pool, 120 GB pinned host pool: the single swaps, the rotate of 16 requests each way
    (twice, as the bench repeats it), then the one-request-each-way rotations, queued without syncing."""
    shape = W.SHAPE_8B
    nb_gpu = W.blocks_for_bytes(shape, 60e9)
    nb_host = _fit_host_pool(shape, W.blocks_for_bytes(shape, 120e9))
    t = _FullSize(W.config2_8b(nb_gpu=nb_gpu, nb_host=nb_host))
    try:
        w, B = t.w, t.B
        for k in ("median", "longest"):
            t.swap_out(*w.extra["single_out"][k])
            t.swap_in(*w.extra["single_in"][k])
        for _ in range(2):
            t.rotate(w.steps[0])
        t.pool.kv_sync()
        st = t.pool.kv_get_stats()
        assert B.PATH_NAMES[st["last_path_out"]] == "staged" and B.PATH_NAMES[st["last_path_in"]] == "staged"
        assert st["timed_kernels"] > 0                          # the bench's path and kernels ran
        for r in w.extra["pairs"]:                              # small ones may take the zero-copy kernels
            t.rotate(r)
        moved_g, moved_h = t.verify("config 2")
        assert moved_g >= w.steps[0].n_in and moved_h >= w.steps[0].n_out
    finally:
        t.close()


def test_config3_full_size_70b_hundred_steps():
    """70B shape (5 MiB blocks, 160 planes), 60 / 120 GB pools, fragmented device pool, 100 steps of 8
    requests each way (about 8 GB per direction per step), queued back to back; what a step swaps in is
    what an earlier step swapped out.  Verified after step 10 and at the end."""
    shape = W.SHAPE_70B
    nb_gpu = W.blocks_for_bytes(shape, 60e9)
    nb_host = _fit_host_pool(shape, W.blocks_for_bytes(shape, 120e9))
    t = _FullSize(W.config3_70b(nb_gpu=nb_gpu, nb_host=nb_host))
    try:
        for k, r in enumerate(t.w.steps):
            t.rotate(r)
            if k == 9:
                t.verify("config 3 after 10 steps", n_read_back=6)
        t.verify("config 3 after 100 steps")
        st = t.pool.kv_get_stats()
        assert st["bytes_out"] == sum(r.n_out for r in t.w.steps) * shape.block_bytes
        assert st["bytes_in"] == sum(r.n_in for r in t.w.steps) * shape.block_bytes
    finally:
        t.close()


def test_config5_full_shape_replay_2000_steps():
    """Serving replay on the 8B shape at 4 requests/s: 2000 steps interleaving swap-outs, swap-ins,
    growth and empty steps (about 160 000 blocks each way), queued without syncing.  Blocks a request
    grows into keep whatever the pool held; whole blocks move, so the comparison stays exact."""
    w = W.config5_replay(rate=4.0)
    assert w.nb_host * w.shape.block_bytes < 0.70 * _mem_available() or pytest.skip("host pool does not fit")
    t = _FullSize(w)
    try:
        for r in w.steps:
            t.rotate(r)
        t.verify("config 5 replay")
    finally:
        t.close()


@pytest.mark.parametrize("bs,contiguous,payload", [(8, False, 2e9), (64, True, 4e9), (32, False, 4e9), (16, False, 8 << 30)],
                         ids=["block8-random-2GB", "block64-contiguous-4GB", "block32-random-4GB", "block16-random-8GiB"])
def test_config4_sweep_cells_at_full_payload(bs, contiguous, payload):
    """Cells of the block-size / fragmentation sweep at full payload, default path: 1 MiB blocks with random
    tables (four-block lattices and pairs), 8 MiB blocks with contiguous tables (long merged transfers), 4 MiB
    blocks with random tables, and the cell of the paper's bandwidth table
    (section 5.3.3): 2 MiB blocks, random tables, 8 GiB = 32768 tokens of 256 KB each way.  Each direction
    alone, then both at once."""
    w = W.config4_sweep_case(bs, contiguous, payload)
    t = _FullSize(w)
    try:
        r = w.steps[0]
        t.swap_out(r.out_gpu, r.out_host)
        moved = t.verify("swap-out alone", n_read_back=4)
        assert moved == (0, r.n_out)
        t.swap_in(r.in_host, r.in_gpu)
        t.rotate(r)
        moved = t.verify("swap-in alone, then both at once", n_read_back=4)
        assert moved == (r.n_in, r.n_out)
        assert t.B.PATH_NAMES[t.pool.kv_get_stats()["last_path_out"]] == "staged"
    finally:
        t.close()


@pytest.mark.parametrize("bs,kv_heads,contiguous,took", [(16, 1, False, "zerocopy"), (8, 1, True, "staged"), (32, 2, False, "staged")],
                         ids=["tp8-block16-random", "tp8-block8-contiguous", "tp4-block32-random"])
def test_tensor_parallel_shard_cells_at_full_payload(bs, kv_heads, contiguous, took):
    """The shard one rank of a tensor-parallel group holds (1 or 2 of the 8 KV heads: 4 KiB, 2 KiB and 16 KiB
    segments, 256 KiB, 128 KiB and 1 MiB blocks), 2 GB each way, default path: scattered small blocks through the
    zero-copy kernels (several issuing warps per CTA), neighbouring ids and 1 MiB blocks staged."""
    w = W.config4_sweep_case(bs, contiguous, 2e9, kv_heads=kv_heads)
    t = _FullSize(w)
    try:
        r = w.steps[0]
        t.swap_out(r.out_gpu, r.out_host)
        moved = t.verify("swap-out alone", n_read_back=4)
        assert moved == (0, r.n_out)
        t.swap_in(r.in_host, r.in_gpu)
        t.rotate(r)
        moved = t.verify("swap-in alone, then both at once", n_read_back=4)
        assert moved == (r.n_in, r.n_out)
        assert t.B.PATH_NAMES[t.pool.kv_get_stats()["last_path_out"]] == took
    finally:
        t.close()
