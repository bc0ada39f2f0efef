"""Parity at the bench's full size and launch configuration (config 2: 60 GB device pool, 120 GB pinned
host pool, rotate of 16 requests each way through the default path).

Both pools are too large for a second copy, so the expected state comes from the oracle's tag model
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


def test_config2_full_size_rotate_single_swaps_and_pairwise_rotations():
    import torch
    from oracle.kv_definition import TagModel
    from paper_2601_20309_b200 import binding as B
    from paper_2601_20309_b200 import poolfill as F

    shape = W.SHAPE_8B
    nb_gpu = W.blocks_for_bytes(shape, 60e9)
    nb_host = W.blocks_for_bytes(shape, 120e9)
    free_dev, _ = torch.cuda.mem_get_info()
    if free_dev < 70e9:
        pytest.skip("needs 70 GB of free device memory")
    budget = int(0.70 * _mem_available())
    if nb_host * shape.block_bytes > budget:                    # same rule as bench.py
        nb_host = max(8192, budget // shape.block_bytes)
    w = W.config2_8b(nb_gpu=nb_gpu, nb_host=nb_host)
    dev = torch.empty(nb_gpu * shape.block_bytes, dtype=torch.uint8, device="cuda:0")
    pool = B.KVPool(shape.num_layers, shape.block_size, shape.kv_heads, shape.head_dim, nb_gpu, nb_host,
                    dev.data_ptr(), flags=B.KV_FLAG_TIME_KERNELS)
    try:
        host_base, _ = pool.kv_host_ptr()
        lay_g = F.Layout.device(dev.data_ptr(), shape, nb_gpu)
        lay_h = F.Layout.host(host_base, shape, nb_host)
        F.fill_blocks(lay_g, w.seed, W.POOL_GPU, nb_gpu)
        F.fill_blocks(lay_h, w.seed, W.POOL_HOST, nb_host)
        d0 = {W.POOL_GPU: F.checksum_blocks(lay_g, nb_gpu), W.POOL_HOST: F.checksum_blocks(lay_h, nb_host)}

        # pin the digests (and the GPU fill) to the CPU generator on a sample
        rng = np.random.default_rng(5)
        for p, nb in ((W.POOL_GPU, nb_gpu), (W.POOL_HOST, nb_host)):
            for b in rng.choice(nb, 24, replace=False):
                assert d0[p][b] == F.checksum_words(W.block_words(w.seed, p, int(b), shape.words_per_block))

        tags = TagModel(nb_gpu, nb_host)
        rot = w.steps[0]
        for k in ("median", "longest"):
            g, h = w.extra["single_out"][k]
            assert tags.swap_out(g.tolist(), h.tolist()) == 0 and pool.kv_swap_out(g, h) == 0
            h2, g2 = w.extra["single_in"][k]
            assert tags.swap_in(h2.tolist(), g2.tolist()) == 0 and pool.kv_swap_in(h2, g2) == 0
        for _ in range(2):                                      # the bench repeats this very call
            assert tags.rotate(rot.out_gpu.tolist(), rot.out_host.tolist(), rot.in_host.tolist(), rot.in_gpu.tolist()) == 0
            assert pool.kv_rotate(rot.out_gpu, rot.out_host, rot.in_host, rot.in_gpu) == 0
        pool.kv_sync()
        st = pool.kv_get_stats()
        assert B.PATH_NAMES[st["last_path_out"]] == "staged" and B.PATH_NAMES[st["last_path_in"]] == "staged"
        assert st["timed_kernels"] > 0                          # the bench's path and kernels ran
        for r in w.extra["pairs"]:                              # small ones may take the zero-copy kernels
            assert tags.rotate(r.out_gpu.tolist(), r.out_host.tolist(), r.in_host.tolist(), r.in_gpu.tolist()) == 0
            assert pool.kv_rotate(r.out_gpu, r.out_host, r.in_host, r.in_gpu) == 0
        pool.kv_sync()
        st = pool.kv_get_stats()
        assert st["device_status"] == 0

        d1 = {W.POOL_GPU: F.checksum_blocks(lay_g, nb_gpu), W.POOL_HOST: F.checksum_blocks(lay_h, nb_host)}
        g_origin = np.array(tags.g_tag, dtype=np.int64)         # (origin pool, origin block) per slot
        h_origin = np.array(tags.h_tag, dtype=np.int64)
        moved_g = np.flatnonzero((g_origin[:, 0] != W.POOL_GPU) | (g_origin[:, 1] != np.arange(nb_gpu)))
        moved_h = np.flatnonzero((h_origin[:, 0] != W.POOL_HOST) | (h_origin[:, 1] != np.arange(nb_host)))
        assert len(moved_g) >= rot.n_in and len(moved_h) >= rot.n_out
        for origin, d_after in ((g_origin, d1[W.POOL_GPU]), (h_origin, d1[W.POOL_HOST])):
            want = np.where(origin[:, 0] == W.POOL_GPU, d0[W.POOL_GPU][np.minimum(origin[:, 1], nb_gpu - 1)],
                            d0[W.POOL_HOST][np.minimum(origin[:, 1], nb_host - 1)])
            bad = np.flatnonzero(want != d_after)
            assert len(bad) == 0, f"{len(bad)} blocks hold the wrong content, first {bad[:5]}"

        # full read-back of a sample: plain copies, compared with regenerated content of the origin
        planes = 2 * shape.num_layers
        dev3 = dev.view(planes, nb_gpu, shape.words_per_plane * 2)
        harr = pool.host_array()
        pick_g = np.concatenate([rng.choice(moved_g, 12, replace=False), rng.choice(nb_gpu, 4, replace=False)])
        pick_h = np.concatenate([rng.choice(moved_h, 12, replace=False), rng.choice(nb_host, 4, replace=False)])
        for b in pick_g:
            op, ob = tags.g_tag[int(b)]
            got = dev3[:, int(b), :].contiguous().cpu().numpy().view(np.uint16).reshape(-1)
            assert np.array_equal(got, W.block_words(w.seed, op, ob, shape.words_per_block))
        for h in pick_h:
            op, ob = tags.h_tag[int(h)]
            got = harr[int(h) * shape.block_bytes:(int(h) + 1) * shape.block_bytes].view(np.uint16)
            assert np.array_equal(got, W.block_words(w.seed, op, ob, shape.words_per_block))
    finally:
        pool.destroy()
        del dev
        torch.cuda.empty_cache()
