"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle, bit for bit."""
import itertools

import numpy as np
import pytest

from paper_2601_20309_b200 import workload as W

pytestmark = pytest.mark.gpu

PATHS = {"zerocopy": 1, "staged": 2, "ce2d": 3, "naive": 4}


def _pair(*a, **k):
    from gpu_harness import Pair
    return Pair(*a, **k)


@pytest.mark.parametrize("path", list(PATHS))
@pytest.mark.parametrize("flags", [0, 2, 4, 6], ids=["bulk", "ldst", "bulk-fused", "ldst-fused"])
@pytest.mark.parametrize("layout", [0, 1], ids=["hostblockfirst", "hostlayerfirst"])
def test_config1_tiny_rotation(path, flags, layout):
    if path != "zerocopy" and flags & 4:
        pytest.skip("fused launch exists on the zero-copy path only")
    if path in ("ce2d", "naive") and flags:
        pytest.skip("no kernel on this path")
    w = W.config1_tiny()
    p = _pair(w.shape, w.nb_gpu, w.nb_host, seed=w.seed, host_layout=layout, path=PATHS[path], flags=flags)
    try:
        assert p.rotate_both(w.steps[0]) == 0
        p.assert_equal(f"tiny rotate {path}")
        st = p.pool.kv_get_stats()
        assert st["bytes_out"] == w.steps[0].n_out * w.shape.block_bytes
        assert st["bytes_in"] == w.steps[0].n_in * w.shape.block_bytes
        assert st["device_status"] == 0
        if path in ("zerocopy", "staged"):
            assert st["kernel_launches"] >= 1
        # single directions
        r = w.steps[0]
        free_h = np.setdiff1d(np.arange(w.nb_host), np.concatenate([r.out_host, r.in_host]))[:10].astype(np.int32)
        src_g = r.in_gpu[:10]
        assert p.oracle.swap_out(src_g, free_h) == 0
        assert p.pool.kv_swap_out(src_g, free_h) == 0
        p.assert_equal("single swap-out")
        dst_g = r.out_gpu[:10]
        assert p.oracle.swap_in(free_h, dst_g) == 0
        assert p.pool.kv_swap_in(free_h, dst_g) == 0
        p.assert_equal("single swap-in")
    finally:
        p.close()


@pytest.mark.parametrize("dims", [(3, 5, 3, 72), (1, 20, 8, 128), (2, 24, 8, 128), (5, 1, 1, 8), (2, 64, 8, 128)],
                         ids=lambda d: "L%d_bs%d_H%d_D%d" % d)
@pytest.mark.parametrize("flags", [0, 2], ids=["bulk", "ldst"])
@pytest.mark.parametrize("path", ["zerocopy", "staged"])
def test_ragged_segment_sizes(dims, flags, path):
    """Segments that are not a whole number of kernel chunks, a 16-byte segment, and a 128 KiB one."""
    L, bs, H, D = dims
    shape = W.KVShape(L, bs, H, D)
    rng = np.random.default_rng(3)
    nbg, nbh = 37, 53
    p = _pair(shape, nbg, nbh, seed=9, path=PATHS[path], flags=flags, staging_bytes=5 * shape.block_bytes)
    try:
        og = rng.choice(nbg, 17, replace=False).astype(np.int32)
        oh = rng.choice(nbh, 17, replace=False).astype(np.int32)
        ig = np.setdiff1d(np.arange(nbg), og)[:13].astype(np.int32)
        ih = np.setdiff1d(np.arange(nbh), oh)[:13].astype(np.int32)
        r = W.Rotation(og, oh, ih, ig, np.zeros(1), np.zeros(1))
        assert p.rotate_both(r) == 0
        p.assert_equal("ragged")
    finally:
        p.close()


@pytest.mark.parametrize("path", ["zerocopy", "staged", "ce2d"])
def test_config2_scaled_8b(path):
    """8B shape (2 MiB blocks), pools shrunk to 320/448 blocks, request lengths scaled down; the
    paired rotation, the single swaps and the one-pair-at-a-time rotations, compared whole-pool."""
    w = W.config2_8b(nb_gpu=320, nb_host=448, n_req=16, median=96, max_tokens=512, n_rot=4)
    p = _pair(w.shape, w.nb_gpu, w.nb_host, seed=w.seed, path=PATHS[path])
    try:
        for k in ("median", "longest"):
            g, h = w.extra["single_out"][k]
            assert p.oracle.swap_out(g, h) == 0 and p.pool.kv_swap_out(g, h) == 0
            h2, g2 = w.extra["single_in"][k]
            assert p.oracle.swap_in(h2, g2) == 0 and p.pool.kv_swap_in(h2, g2) == 0
        p.assert_equal("single swaps")
        assert p.rotate_both(w.steps[0]) == 0
        p.assert_equal("rotate 4+4 requests")
        for r in w.extra["pairs"]:
            assert p.rotate_both(r) == 0          # no sync in between: calls queue up
        p.assert_equal("pairwise rotations")
    finally:
        p.close()


@pytest.mark.parametrize("flags", [0, 4], ids=["two-streams", "fused"])
def test_config3_scaled_70b_steps(flags):
    """70B shape (5 MiB blocks, 160 planes), fragmented pool, 12 steps of 2 requests each way,
    issued back to back; what step k swaps in is what step k-2 swapped out."""
    w = W.config3_70b(nb_gpu=160, nb_host=240, n_req=8, median=96, max_tokens=256, n_steps=12, per_step=2)
    p = _pair(w.shape, w.nb_gpu, w.nb_host, seed=w.seed, path=1, flags=flags)
    try:
        for k, r in enumerate(w.steps):
            assert p.rotate_both(r) == 0
            if k % 5 == 4:
                p.assert_equal(f"step {k}")
        p.assert_equal("final")
    finally:
        p.close()


@pytest.mark.parametrize("bs", [8, 16, 32, 64])
@pytest.mark.parametrize("contig", [True, False], ids=["contiguous", "permuted"])
def test_config4_sweep_cells_small(bs, contig):
    w = W.config4_sweep_case(bs, contig, 48e6, num_layers=8)
    for path in ("zerocopy", "staged", "ce2d"):
        p = _pair(w.shape, w.nb_gpu, w.nb_host, seed=w.seed, path=PATHS[path], staging_bytes=16 << 20)
        try:
            assert p.rotate_both(w.steps[0]) == 0
            p.assert_equal(f"sweep bs{bs} {path}")
        finally:
            p.close()


def test_config5_replay_scaled():
    """Replay lists (swap-outs, swap-ins, growth, empty steps) on a shrunk shape, queued without
    syncing.  Blocks a request grows into keep whatever bytes the pool held there: whole blocks
    move, filled or not, so the comparison stays bit-exact."""
    w = W.config5_replay(rate=2.0, n_steps=400, shape=W.KVShape(2, 16, 2, 64), duration_s=25.0, max_tokens=1024)
    assert sum(1 for s in w.steps if s.n_out and s.n_in) > 3
    p = _pair(w.shape, w.nb_gpu, w.nb_host, seed=w.seed, path=1)
    try:
        for k, r in enumerate(w.steps):
            assert p.rotate_both(r) == 0
            if k % 100 == 99:
                p.assert_equal(f"replay step {k}")
        p.assert_equal("replay final")
    finally:
        p.close()


@pytest.mark.parametrize("path", ["zerocopy", "staged", "auto"])
def test_back_to_back_calls_with_cross_direction_dependencies(path):
    """swap_out(g->h) immediately followed by swap_in(h->g2) with no sync: the library must order the
    second after the first (the host block is written, then read).  Then the reverse dependency."""
    shape = W.KVShape(4, 16, 8, 128)
    p = _pair(shape, 64, 64, seed=5, path={"auto": 0, **PATHS}[path])
    rng = np.random.default_rng(0)
    try:
        for _ in range(6):
            g = rng.choice(64, 12, replace=False).astype(np.int32)
            h = rng.choice(64, 12, replace=False).astype(np.int32)
            g2 = rng.choice(64, 12, replace=False).astype(np.int32)
            assert p.oracle.swap_out(g, h) == 0 and p.pool.kv_swap_out(g, h) == 0
            assert p.oracle.swap_in(h, g2) == 0 and p.pool.kv_swap_in(h, g2) == 0       # RAW on host blocks
            h3 = rng.choice(64, 12, replace=False).astype(np.int32)
            assert p.oracle.swap_out(g2, h3) == 0 and p.pool.kv_swap_out(g2, h3) == 0   # RAW on device blocks
        p.assert_equal("dependent call chain")
    finally:
        p.close()


@pytest.mark.parametrize("path", ["zerocopy", "staged", "ce2d"])
def test_overlapping_rotate_needs_flag_and_matches_sequential_semantics(path):
    shape = W.KVShape(2, 16, 8, 128)
    rng = np.random.default_rng(2)
    og = np.array([3, 7, 11, 15, 19], np.int32)
    oh = np.array([1, 2, 3, 4, 5], np.int32)
    ih = np.array([20, 2, 21, 4, 22, 23], np.int32)         # 2 and 4 are written by the swap-out
    ig = np.array([7, 30, 31, 15, 32, 33], np.int32)        # 7 and 15 are swap-out sources
    r = W.Rotation(og, oh, ih, ig, np.zeros(1), np.zeros(1))
    p = _pair(shape, 40, 40, seed=6, path=PATHS[path])
    try:
        before_g, before_h = p.gpu_bytes().copy(), p.pool.host_array().copy()
        assert p.rotate_both(r) == -4
        p.pool.kv_sync()
        assert np.array_equal(p.gpu_bytes(), before_g) and np.array_equal(p.pool.host_array(), before_h)
    finally:
        p.close()
    p = _pair(shape, 40, 40, seed=6, path=PATHS[path], flags=1)
    try:
        assert p.rotate_both(r, allow_overlap=True) == 0
        p.assert_equal("overlapping rotate")
    finally:
        p.close()


def test_validation_errors_move_nothing():
    shape = W.KVShape(2, 16, 8, 128)
    p = _pair(shape, 16, 24, seed=7, path=1)
    try:
        g0, h0 = p.gpu_bytes().copy(), p.pool.host_array().copy()
        P = p.pool
        assert P.kv_swap_out([0, 16], [0, 1], check=False) == -2
        assert P.kv_swap_out([0, 1], [0, 24], check=False) == -2
        assert P.kv_swap_out([0, -1], [0, 1], check=False) == -2
        assert P.kv_swap_out([0, 1], [5, 5], check=False) == -3
        assert P.kv_swap_in([0, 1], [5, 5], check=False) == -3
        assert P.kv_rotate([0], [1], [2], [0], check=False) == -4
        assert P.kv_rotate([0], [1], [1], [2], check=False) == -4
        assert "race" in P.kv_last_error()
        assert P.kv_swap_out([1, 1], [2, 3], check=False) == 0       # duplicate sources are fine
        assert p.oracle.swap_out([1, 1], [2, 3]) == 0
        assert P.kv_rotate([], [], [], [], check=False) == 0
        assert P.kv_swap_out([], [], check=False) == 0 and P.kv_swap_in([], [], check=False) == 0
        p.assert_equal("after refused calls")
        assert not np.array_equal(p.pool.host_array(), h0)           # the valid call did move bytes
        assert np.array_equal(p.gpu_bytes(), g0)
    finally:
        p.close()


def test_whole_pool_in_one_call_and_device_leg():
    """n = every block of the device pool; then gather/scatter through a contiguous device buffer."""
    import torch
    shape = W.KVShape(3, 16, 8, 128)
    nbg, nbh = 48, 48
    p = _pair(shape, nbg, nbh, seed=8, path=1)
    try:
        rng = np.random.default_rng(1)
        g = rng.permutation(nbg).astype(np.int32)
        h = rng.permutation(nbh).astype(np.int32)
        assert p.oracle.swap_out(g, h) == 0 and p.pool.kv_swap_out(g, h) == 0
        p.assert_equal("whole pool out")
        g2 = rng.permutation(nbg).astype(np.int32)
        assert p.oracle.swap_in(h, g2) == 0 and p.pool.kv_swap_in(h, g2) == 0
        p.assert_equal("whole pool in")
        # device leg: gather listed blocks into a contiguous block-first buffer
        ids = rng.choice(nbg, 20, replace=False).astype(np.int32)
        buf = torch.zeros(20 * shape.block_bytes, dtype=torch.uint8, device="cuda:0")
        assert p.pool.kv_gather_blocks(ids, buf.data_ptr()) == 0
        p.pool.kv_sync()
        got = buf.cpu().numpy().reshape(20, shape.block_bytes)
        for k, b in enumerate(ids):
            assert np.array_equal(got[k], p.oracle.g_block(int(b)))
        # scatter them back to other ids: equals a swap-in from a block-first host model
        dst = rng.permutation(nbg)[:20].astype(np.int32)
        expect = {int(d): p.oracle.g_block(int(s)).copy() for s, d in zip(ids, dst)}
        assert p.pool.kv_scatter_blocks(buf.data_ptr(), dst) == 0
        p.pool.kv_sync()
        gb = p.gpu_bytes()
        seg = p.oracle.seg
        for d, want in expect.items():
            have = np.concatenate([gb[p.oracle.dev_off(l, kv, d):p.oracle.dev_off(l, kv, d) + seg]
                                   for l in range(shape.num_layers) for kv in range(2)])
            assert np.array_equal(have, want)
        touched = set(int(x) for x in dst)
        for b in range(nbg):
            if b not in touched:
                o = p.oracle.dev_off(1, 1, b)
                assert np.array_equal(gb[o:o + seg], p.oracle.G[o:o + seg])
    finally:
        p.close()


def test_gpu_fill_twin_matches_cpu_generator():
    """The GPU pool-fill helper must write exactly what workload.block_words generates."""
    import torch
    from paper_2601_20309_b200 import poolfill as F
    shape = W.KVShape(3, 8, 2, 64)
    nb = 11
    dev = torch.zeros(nb * shape.block_bytes, dtype=torch.uint8, device="cuda:0")
    lay = F.Layout.device(dev.data_ptr(), shape, nb)
    F.fill_blocks(lay, 77, W.POOL_GPU, nb)
    got = dev.cpu().numpy().view(np.uint16).reshape(2 * shape.num_layers, nb, shape.words_per_plane)
    for b in range(nb):
        want = W.block_words(77, W.POOL_GPU, b, shape.words_per_block).reshape(2 * shape.num_layers, -1)
        assert np.array_equal(got[:, b, :], want)
    sums = F.checksum_blocks(lay, nb)
    for b in range(nb):
        assert sums[b] == F.checksum_words(W.block_words(77, W.POOL_GPU, b, shape.words_per_block))


@pytest.mark.parametrize("layout", [0, 1], ids=["hostblockfirst", "hostlayerfirst"])
def test_staged_transfer_planning_patterns(layout):
    """Host-id patterns that the staged path turns into different copy-engine transfers: long runs,
    equal runs at a constant spacing (one strided transfer of several rows), isolated blocks in
    pairs, a list given in descending order, repeated swap-in sources, and more blocks than one
    staging half holds."""
    shape = W.KVShape(2, 16, 4, 64)              # 16 KiB planes, 64 KiB blocks
    nbg, nbh = 96, 400
    p = _pair(shape, nbg, nbh, seed=11, host_layout=layout, path=PATHS["staged"], staging_bytes=12 * shape.block_bytes)
    rng = np.random.default_rng(4)
    try:
        patterns = {
            "one long run": np.arange(100, 140),
            "runs of 3 every 10": np.concatenate([np.arange(s, s + 3) for s in range(20, 120, 10)]),
            "every 7th": np.arange(3, 3 + 7 * 30, 7),
            "descending": np.arange(300, 260, -1),
            "mixed": np.array([0, 1, 2, 9, 20, 21, 50, 51, 52, 53, 80, 399, 398, 200, 210, 220, 231, 5]),
            "random": rng.choice(nbh, 45, replace=False),
        }
        for name, hid in patterns.items():
            hid = hid.astype(np.int32)
            g = rng.choice(nbg, len(hid), replace=False).astype(np.int32)
            assert p.oracle.swap_out(g, hid) == 0 and p.pool.kv_swap_out(g, hid) == 0
            p.assert_equal(f"staged out, {name}")
            g2 = rng.choice(nbg, len(hid), replace=False).astype(np.int32)
            assert p.oracle.swap_in(hid, g2) == 0 and p.pool.kv_swap_in(hid, g2) == 0
            p.assert_equal(f"staged in, {name}")
        # the same host block as the source of several swap-ins
        hid = np.array([7, 7, 8, 7, 30, 30, 31], np.int32)
        g = rng.choice(nbg, len(hid), replace=False).astype(np.int32)
        assert p.oracle.swap_in(hid, g) == 0 and p.pool.kv_swap_in(hid, g) == 0
        p.assert_equal("staged in, repeated sources")
        # both directions at once, several halves deep, queued twice without a sync
        for _ in range(2):
            og = rng.choice(nbg, 40, replace=False).astype(np.int32)
            ig = np.setdiff1d(np.arange(nbg), og)[:40].astype(np.int32)
            oh = rng.choice(nbh, 40, replace=False).astype(np.int32)
            ih = rng.choice(np.setdiff1d(np.arange(nbh), oh), 40, replace=False).astype(np.int32)
            assert p.rotate_both(W.Rotation(og, oh, ih, ig, np.zeros(1), np.zeros(1))) == 0
        p.assert_equal("staged rotate, queued")
        # one direction with a long run of host ids, the other scattered: both must end up on the same kind
        # of transfers (the plan of one of them is redone), whichever direction has the run
        for flip in (False, True):
            og = rng.choice(nbg, 40, replace=False).astype(np.int32)
            ig = np.setdiff1d(np.arange(nbg), og)[:40].astype(np.int32)
            run = np.arange(150, 190, dtype=np.int32)
            scattered = rng.choice(np.setdiff1d(np.arange(nbh), run), 40, replace=False).astype(np.int32)
            oh, ih = (scattered, run) if flip else (run, scattered)
            assert p.rotate_both(W.Rotation(og, oh, ih, ig, np.zeros(1), np.zeros(1))) == 0
            p.assert_equal(f"staged rotate, mixed host id patterns, flip={flip}")
        st = p.pool.kv_get_stats()
        assert st["device_status"] == 0 and st["kernel_launches"] > 0
    finally:
        p.close()


@pytest.mark.parametrize("path", ["zerocopy", "staged"])
def test_rotate_swap_in_waits_for_an_earlier_swap_out_that_reads_its_destinations(path):
    """A long swap-out is still reading device blocks when a rotate arrives whose swap-in overwrites some
    of them (the blocks were released in between).  The rotate's swap-in must follow the EARLIER
    swap-out, not only the swap-out that travels in the same rotate."""
    shape = W.KVShape(32, 16, 8, 128)             # 2 MiB blocks
    nbg, nbh = 230, 420
    p = _pair(shape, nbg, nbh, seed=13, path=PATHS[path])
    try:
        big_g = np.arange(0, 200, dtype=np.int32)
        big_h = np.arange(0, 200, dtype=np.int32)
        assert p.oracle.swap_out(big_g, big_h) == 0
        og = np.arange(200, 210, dtype=np.int32)          # not part of the long swap-out
        oh = np.arange(300, 310, dtype=np.int32)
        ih = np.arange(400, 420, dtype=np.int32)          # untouched host blocks
        ig = np.arange(180, 200, dtype=np.int32)          # the blocks the long swap-out reads last
        r = W.Rotation(og, oh, ih, ig, np.zeros(1), np.zeros(1))
        assert p.oracle.rotate(og, oh, ih, ig) == 0
        assert p.pool.kv_swap_out(big_g, big_h) == 0      # 400 MiB over the link: several milliseconds
        assert p.pool.kv_rotate(og, oh, ih, ig) == 0      # issued at once, no sync
        p.assert_equal("rotate behind a long swap-out")
    finally:
        p.close()


@pytest.mark.parametrize("path", list(PATHS))
@pytest.mark.parametrize("host_layout", [0, 1], ids=["hostblockfirst", "hostlayerfirst"])
def test_block_first_device_layout(path, host_layout):
    """The paper's redesigned storage order applied to the device pool: all planes of a block contiguous.
    Same calls, same oracle results through the logical accessor; on the copy-engine path with a
    block-first host pool a block is then one plain transfer."""
    w = W.config1_tiny()
    p = _pair(w.shape, w.nb_gpu, w.nb_host, seed=w.seed, host_layout=host_layout, device_layout=1, path=PATHS[path])
    try:
        assert p.rotate_both(w.steps[0]) == 0
        p.assert_equal(f"block-first device, {path}")
        st = p.pool.kv_get_stats()
        if path == "ce2d":
            assert st["ce_copies"] == w.steps[0].n_out + w.steps[0].n_in
    finally:
        p.close()
    w = W.config2_8b(nb_gpu=320, nb_host=448, n_req=16, median=96, max_tokens=512, n_rot=4)
    p = _pair(w.shape, w.nb_gpu, w.nb_host, seed=w.seed, host_layout=host_layout, device_layout=1, path=PATHS[path])
    try:
        assert p.rotate_both(w.steps[0]) == 0
        for r in w.extra["pairs"][:3]:
            assert p.rotate_both(r) == 0
        p.assert_equal(f"block-first device 8B shape, {path}")
    finally:
        p.close()


def test_stream_wait_orders_a_consumer_stream_behind_the_swap_in():
    """No host-side sync: a torch stream that was told to wait for the pool reads swapped-in blocks only
    after they have landed."""
    import torch
    shape = W.KVShape(32, 16, 8, 128)                 # 2 MiB blocks
    nbg, nbh = 260, 300
    p = _pair(shape, nbg, nbh, seed=21, path=PATHS["zerocopy"])
    try:
        ih = np.arange(0, 250, dtype=np.int32)
        ig = np.arange(0, 250, dtype=np.int32)        # 500 MiB over the link: about 10 ms
        assert p.oracle.swap_in(ih, ig) == 0
        snap = torch.empty_like(p.dev)
        consumer = torch.cuda.Stream()
        assert p.pool.kv_swap_in(ih, ig) == 0
        assert p.pool.kv_stream_wait(consumer.cuda_stream, 2) == 0
        with torch.cuda.stream(consumer):
            snap.copy_(p.dev, non_blocking=True)      # would see half-written blocks without the wait
        consumer.synchronize()
        assert np.array_equal(snap.cpu().numpy(), p.oracle.G)
        assert p.pool.kv_stream_wait(None, 0, check=False) == -1
        p.assert_equal("after stream wait")
    finally:
        p.close()


def test_budgeted_replay_matches_the_oracle():
    """The replay lists re-timed under a per-step budget of 24 blocks (work carried over to later steps),
    queued without syncing: same final pools as the oracle fed the same budgeted steps."""
    w = W.config5_replay(rate=2.0, n_steps=300, shape=W.KVShape(2, 16, 2, 64), duration_s=20.0, max_tokens=1024)
    steps = W.budgeted_steps(w.steps, 24)
    assert len(steps) > len(w.steps) and max(s.n_out + s.n_in for s in steps) <= 24
    p = _pair(w.shape, w.nb_gpu, w.nb_host, seed=w.seed)
    try:
        for r in steps:
            assert p.rotate_both(r) == 0
        p.assert_equal("budgeted replay")
    finally:
        p.close()


@pytest.mark.parametrize("path", ["zerocopy", "staged"])
def test_caller_supplied_host_memory_is_page_locked_and_stays_inside_its_bounds(path):
    """host_base given by the caller: the library page-locks it for the pool's lifetime, moves the same
    bytes as with its own allocation, and writes nothing outside the region it was given."""
    import torch
    from oracle.kv_oracle import ByteOracle
    from paper_2601_20309_b200 import binding as B
    shape = W.KVShape(3, 16, 8, 128)
    nbg, nbh = 40, 60
    o = ByteOracle(shape.num_layers, shape.block_size, shape.kv_heads, shape.head_dim, nbg, nbh)
    rng = np.random.default_rng(31)
    o.G[:] = rng.integers(0, 256, o.G.size, dtype=np.uint8)
    o.Hs[:] = rng.integers(0, 256, o.Hs.size, dtype=np.uint8)
    page, size = 4096, nbh * shape.block_bytes
    raw = np.full(size + 3 * page, 0x5A, np.uint8)
    start = (-raw.ctypes.data) % page + page                    # page-aligned, one guard page before
    region = raw[start:start + size]
    region[:] = o.Hs
    dev = torch.from_numpy(o.G.copy()).to("cuda:0")
    pool = B.KVPool(shape.num_layers, shape.block_size, shape.kv_heads, shape.head_dim, nbg, nbh, dev.data_ptr(),
                    host_base=region.ctypes.data, path=PATHS[path])
    try:
        base, nbytes = pool.kv_host_ptr()
        assert base == region.ctypes.data and nbytes == size
        og = rng.choice(nbg, 15, replace=False).astype(np.int32)
        ig = np.setdiff1d(np.arange(nbg), og)[:12].astype(np.int32)
        oh = rng.choice(nbh, 15, replace=False).astype(np.int32)
        ih = rng.choice(np.setdiff1d(np.arange(nbh), oh), 12, replace=False).astype(np.int32)
        assert o.rotate(og, oh, ih, ig) == 0 and pool.kv_rotate(og, oh, ih, ig) == 0
        pool.kv_sync()
        assert np.array_equal(region, o.Hs)
        assert np.array_equal(dev.cpu().numpy(), o.G)
        assert (raw[:start] == 0x5A).all() and (raw[start + size:] == 0x5A).all()
    finally:
        pool.destroy()
    region[:8] = 1                                                # still ordinary memory after the pool is gone
    # a misaligned host_base is refused
    with pytest.raises(B.KVError):
        B.KVPool(shape.num_layers, shape.block_size, shape.kv_heads, shape.head_dim, nbg, nbh, dev.data_ptr(),
                 host_base=region.ctypes.data + 8)


@pytest.mark.parametrize("knobs", [
    dict(path=1, path_in=2), dict(path=2, path_in=1), dict(path=3, path_in=1), dict(path=3, ce_streams=4),
    dict(path=4, ce_streams=2), dict(path=1, ctas_out=3, ctas_in=148), dict(path=1, flags=4, ctas_out=5, ctas_in=9),
    dict(path=2, staging_bytes=1), dict(path=0, flags=8),
    dict(path=1, link_variant=1), dict(path=1, link_variant=2), dict(path=1, flags=2, link_variant=1),
    dict(path=1, flags=4, link_variant=2, ctas_out=7, ctas_in=7),
], ids=lambda k: "-".join(f"{a}{b}" for a, b in k.items()))
def test_tuning_knobs_do_not_change_results(knobs):
    """A different path per direction, several copy-engine streams, odd CTA counts, the smallest staging,
    kernel timing, the other shapes of the zero-copy kernels' transfers (32 and 64 KiB bulk copies, 32-byte
    vectors): every setting must give the oracle's bytes."""
    w = W.config2_8b(nb_gpu=320, nb_host=448, n_req=16, median=96, max_tokens=512, n_rot=4)
    p = _pair(w.shape, w.nb_gpu, w.nb_host, seed=w.seed, **knobs)
    try:
        assert p.rotate_both(w.steps[0]) == 0
        for r in w.extra["pairs"][:4]:
            assert p.rotate_both(r) == 0
        p.assert_equal(f"knobs {knobs}")
        assert p.pool.kv_get_stats()["device_status"] == 0
    finally:
        p.close()


def test_caller_streams_and_link_probe():
    """Streams made by the caller (here: torch) carry the two directions; and the link probe returns
    sensible figures for plain and strided transfers and refuses nonsense."""
    import torch
    from paper_2601_20309_b200 import binding as B
    s_out, s_in = torch.cuda.Stream(), torch.cuda.Stream()
    w = W.config1_tiny()
    p = _pair(w.shape, w.nb_gpu, w.nb_host, seed=w.seed, stream_out=s_out.cuda_stream, stream_in=s_in.cuda_stream, path=2)
    try:
        assert p.rotate_both(w.steps[0]) == 0
        s_out.synchronize()
        s_in.synchronize()                             # the caller's own streams are what the work ran on
        assert np.array_equal(p.pool.host_array(), p.oracle.Hs)
        p.assert_equal("caller streams")
        assert p.pool.kv_pool_progress() == {"out_issued": 1, "out_done": 1, "in_issued": 1, "in_done": 1}
    finally:
        p.close()
    plain = B.kv_probe_link_ex(0, copy_bytes=1 << 20, total_bytes=32 << 20, span_bytes=64 << 20, scattered=True, rounds=1)
    strided = B.kv_probe_link_ex(0, copy_bytes=2 << 20, total_bytes=32 << 20, span_bytes=64 << 20, scattered=True, rounds=1,
                                 rows=2, host_pitch=8 << 20)
    for r in (plain, strided):
        assert 1.0 < r["d2h_gbs"] < 200.0 and 1.0 < r["h2d_gbs"] < 200.0 and r["bi_sum_gbs"] > r["d2h_gbs"] * 0.8
    with pytest.raises(B.KVError):
        B.kv_probe_link_ex(0, copy_bytes=3 << 20, total_bytes=32 << 20, span_bytes=64 << 20, rows=2, host_pitch=1 << 20)
    with pytest.raises(B.KVError):
        B.kv_probe_link_ex(0, copy_bytes=1 << 20, total_bytes=1 << 10, span_bytes=64 << 20)


@pytest.mark.parametrize("path", ["zerocopy", "staged"])
def test_device_leg_is_ordered_against_the_other_direction(path):
    """kv_gather_blocks / kv_scatter_blocks queued right behind (or in front of) a swap of the other
    direction that touches the same device blocks, with no kv_sync in between: 200 blocks of 2 MiB, so
    the first call is still running when the second is issued.  A contiguous device buffer is a
    block-first pool of its own, so the oracle models a gather as a swap-out into it and a scatter as a
    swap-in from it."""
    import torch
    from oracle.kv_oracle import ByteOracle
    shape = W.SHAPE_8B
    n, nbg, nbh = 200, 420, 440
    p = _pair(shape, nbg, nbh, seed=11, path=PATHS[path])
    try:
        rng = np.random.default_rng(4)
        buf_model = ByteOracle(shape.num_layers, shape.block_size, shape.kv_heads, shape.head_dim, nbg, n, alloc=False)
        buf_model.G = p.oracle.G                                  # the same device pool
        buf_model.Hs = rng.integers(0, 256, n * shape.block_bytes, dtype=np.uint8)
        buf = torch.from_numpy(buf_model.Hs.copy()).to("cuda:0")
        slots = np.arange(n, dtype=np.int32)

        def check(what):
            p.assert_equal(what)
            assert np.array_equal(buf.cpu().numpy(), buf_model.Hs), what + ": the device buffer differs"

        ids = rng.choice(nbg, n, replace=False).astype(np.int32)
        h1 = rng.choice(nbh, n, replace=False).astype(np.int32)
        # scatter writes the blocks, the swap-out right behind it must send what the scatter wrote
        assert buf_model.swap_in(slots, ids) == 0 and p.pool.kv_scatter_blocks(buf.data_ptr(), ids) == 0
        assert p.oracle.swap_out(ids, h1) == 0 and p.pool.kv_swap_out(ids, h1) == 0
        check("scatter then swap-out")
        # swap-in writes the blocks, the gather right behind it must read what came in
        h2 = rng.choice(nbh, n, replace=False).astype(np.int32)
        ids2 = rng.choice(nbg, n, replace=False).astype(np.int32)
        assert p.oracle.swap_in(h2, ids2) == 0 and p.pool.kv_swap_in(h2, ids2) == 0
        assert buf_model.swap_out(ids2, slots) == 0 and p.pool.kv_gather_blocks(ids2, buf.data_ptr()) == 0
        check("swap-in then gather")
        # gather reads the blocks, the swap-in right behind it must not overwrite them too early
        h3 = rng.choice(nbh, n, replace=False).astype(np.int32)
        assert buf_model.swap_out(ids, slots) == 0 and p.pool.kv_gather_blocks(ids, buf.data_ptr()) == 0
        assert p.oracle.swap_in(h3, ids) == 0 and p.pool.kv_swap_in(h3, ids) == 0
        check("gather then swap-in")
        # swap-out reads the blocks, the scatter right behind it must wait for it
        h4 = rng.choice(nbh, n, replace=False).astype(np.int32)
        assert p.oracle.swap_out(ids2, h4) == 0 and p.pool.kv_swap_out(ids2, h4) == 0
        assert buf_model.swap_in(slots, ids2) == 0 and p.pool.kv_scatter_blocks(buf.data_ptr(), ids2) == 0
        check("swap-out then scatter")
    finally:
        p.close()


def test_lists_made_by_the_lvf_scheduler_match_the_oracle():
    """Rotation lists that the paper's Largest-VLT-First policy produces on synthetic arrivals (a CPU toy
    that only makes inputs), first 300 steps on a shrunk shape, queued without syncing, AUTO path."""
    w = W.config5_lvf(rate=3.0, n_steps=300, shape=W.KVShape(2, 16, 2, 64), duration_s=20.0, max_tokens=1024,
                      params=W.LVFParams(b_xfer=40))
    assert sum(1 for s in w.steps if s.n_out and s.n_in) > 10
    p = _pair(w.shape, w.nb_gpu, w.nb_host, seed=w.seed, path=0)
    try:
        for k, r in enumerate(w.steps):
            assert p.rotate_both(r) == 0
            if k % 100 == 99:
                p.assert_equal(f"LVF step {k}")
        p.assert_equal("LVF final")
    finally:
        p.close()


@pytest.mark.parametrize("seed", range(12))
def test_random_shapes_lists_and_staging_sizes(seed):
    """Seeded random cases across shapes, pool sizes, list lengths, staging sizes (so that the staged plan
    is cut into one to many chunks, with four-block lattices, pairs and singles in them), paths and host
    layouts: three calls queued without syncing, then both pools against the oracle."""
    rng = np.random.default_rng(1000 + seed)
    shape = W.KVShape(int(rng.choice([1, 2, 3, 5])), int(rng.choice([8, 16, 32])), int(rng.choice([1, 2, 8])), int(rng.choice([64, 128])))
    nbg, nbh = int(rng.integers(60, 260)), int(rng.integers(80, 400))
    path = int(rng.choice([0, 2, 2, 1]))
    layout = int(rng.choice([0, 0, 1]))
    staging = int(rng.choice([2, 5, 8, 16, 33, 1000])) * shape.block_bytes
    p = _pair(shape, nbg, nbh, seed=seed, path=path, host_layout=layout, staging_bytes=staging)
    try:
        for call in range(3):
            n_out = int(rng.integers(1, min(nbg, nbh) // 2))
            n_in = int(rng.integers(1, min(nbg, nbh) // 2))
            og = rng.choice(nbg, n_out, replace=False).astype(np.int32)
            oh = rng.choice(nbh, n_out, replace=False).astype(np.int32)
            ig = np.setdiff1d(np.arange(nbg), og)
            ig = rng.choice(ig, min(n_in, len(ig)), replace=False).astype(np.int32)
            ih = np.setdiff1d(np.arange(nbh), oh)
            ih = rng.choice(ih, len(ig), replace=True).astype(np.int32)         # swap-in sources may repeat
            if call == 1 and rng.random() < 0.5:                                  # every other host id: all lattices
                oh = (2 * np.arange(n_out) % nbh).astype(np.int32)
                oh = np.unique(oh)[:n_out]
                og = og[:len(oh)]
                ih = np.setdiff1d(np.arange(nbh), oh)
                ih = rng.choice(ih, len(ig), replace=True).astype(np.int32) if len(ih) else ih[:0].astype(np.int32)
                ig = ig[:len(ih)]
            r = W.Rotation(og, oh, ih, ig, np.zeros(1), np.zeros(1))
            assert p.rotate_both(r) == 0, (seed, call)
        p.assert_equal(f"random case {seed}: shape {shape}, pools {nbg}/{nbh}, path {path}, layout {layout}, staging {staging}")
        assert p.pool.kv_get_stats()["device_status"] == 0
    finally:
        p.close()


# segment bytes -> (block_size, kv_heads, head_dim): every ring shape of the bulk kernel, from one issuing
# warp with 16 KiB stages down to sixteen warps with 1 KiB stages, plus sizes between the powers of two
SMALL_SEGMENTS = {512: (4, 1, 64), 1024: (8, 1, 64), 1536: (4, 3, 64), 2048: (8, 1, 128), 4096: (16, 1, 128),
                  6144: (8, 3, 128), 8192: (16, 2, 128), 12288: (16, 3, 128), 16384: (16, 4, 128),
                  20480: (16, 5, 128)}


@pytest.mark.parametrize("device_layout", [0, 1], ids=["devlayerfirst", "devblockfirst"])
@pytest.mark.parametrize("path", [1, 2], ids=["zerocopy", "staged"])
@pytest.mark.parametrize("seg", sorted(SMALL_SEGMENTS))
def test_small_segments_take_every_ring_shape(seg, path, device_layout):
    """Shards of a tensor-parallel group and small block sizes have small segments, which the bulk kernel
    moves with several issuing warps per CTA: lists long and short (fewer items than warps in some CTAs),
    gather and scatter on their own, rotations on both paths, all against the oracle.  With a block-first
    device pool the same blocks travel as whole runs of BLK bytes."""
    bs, kv, hd = SMALL_SEGMENTS[seg]
    shape = W.KVShape(3, bs, kv, hd)
    assert shape.words_per_plane * 2 == seg
    nbg, nbh = 700, 900
    p = _pair(shape, nbg, nbh, seed=seg, path=path, device_layout=device_layout)
    try:
        import torch
        rng = np.random.default_rng(seg + path)
        for n in (1, 3, 37, 300):
            og = rng.choice(nbg, n, replace=False).astype(np.int32)
            oh = rng.choice(nbh, n, replace=False).astype(np.int32)
            ig = rng.choice(np.setdiff1d(np.arange(nbg), og), n, replace=False).astype(np.int32)
            ih = rng.choice(np.setdiff1d(np.arange(nbh), oh), n, replace=False).astype(np.int32)
            assert p.rotate_both(W.Rotation(og, oh, ih, ig, np.zeros(1), np.zeros(1))) == 0
            p.assert_equal(f"segment {seg}, path {path}, rotate of {n}")
            # the device leg alone: gather into a buffer, scatter it to other blocks
            buf = torch.zeros(n * shape.block_bytes, dtype=torch.uint8, device="cuda:0")
            assert p.pool.kv_gather_blocks(og, buf.data_ptr()) == 0
            p.pool.kv_sync()
            want = np.concatenate([p.oracle.g_block(int(b)) for b in og])
            assert np.array_equal(buf.cpu().numpy(), want), (seg, n)
            assert p.pool.kv_scatter_blocks(buf.data_ptr(), ig) == 0
            for s_, d_ in zip(og, ig):                      # the model's side of it: plane by plane
                for l in range(shape.num_layers):
                    for plane in range(2):
                        p.oracle.g_seg(l, plane, int(d_))[:] = p.oracle.g_seg(l, plane, int(s_))
            p.assert_equal(f"segment {seg}, path {path}, scatter of {n}")
        assert p.pool.kv_get_stats()["device_status"] == 0
    finally:
        p.close()
