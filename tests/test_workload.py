"""Seeded input generators: determinism, the shapes of the five workloads, and the
block-table bookkeeping (one residency per request, table length, pool-wide unique ids)."""
import numpy as np
import pytest

from paper_2601_20309_b200 import workload as W


def test_lut_is_standard_normal_in_bf16():
    import torch
    t = W.lut()
    assert t.dtype == np.uint16 and t.shape == (65536,)
    v = torch.from_numpy(t.view(np.int16)).view(torch.bfloat16).double()
    assert abs(v.mean().item()) < 1e-3 and abs(v.std().item() - 1.0) < 5e-3
    assert torch.all(v[1:] >= v[:-1])                     # quantiles are monotone
    assert v[32768 - 1].item() <= 0.0 <= v[32768].item()  # median at zero


def test_block_words_is_a_pure_function_of_seed_pool_block():
    n = W.SHAPE_TINY.words_per_block
    a = W.block_words(5, W.POOL_GPU, 17, n)
    assert np.array_equal(a, W.block_words(5, W.POOL_GPU, 17, n))
    assert not np.array_equal(a, W.block_words(5, W.POOL_HOST, 17, n))
    assert not np.array_equal(a, W.block_words(5, W.POOL_GPU, 18, n))
    assert not np.array_equal(a, W.block_words(6, W.POOL_GPU, 17, n))
    # splitmix64 reference values for counter 0 and 1 (state advanced by the golden ratio first)
    z = W.mix64(np.array([0, 1], np.uint64))
    assert int(z[0]) == 0xE220A8397B1DCDAF
    assert int(z[1]) == 0x910A2DEC89025CC1


def test_config1_tiny_shape():
    w = W.config1_tiny()
    r = w.steps[0]
    assert (w.shape.num_layers, w.shape.block_size, w.nb_gpu, w.nb_host) == (2, 16, 256, 512)
    assert w.shape.block_bytes == 128 << 10
    assert len(r.out_req_offsets) == 5 and len(r.in_req_offsets) == 5
    sizes = list(np.diff(r.out_req_offsets)) + list(np.diff(r.in_req_offsets))
    assert all(4 <= s <= 20 for s in sizes)
    assert not set(r.in_gpu) & set(r.out_gpu) and not set(r.in_host) & set(r.out_host)
    assert len(set(r.out_host)) == r.n_out and len(set(r.in_gpu)) == r.n_in
    w.table.check_consistent()
    w2 = W.config1_tiny()
    assert all(np.array_equal(a, b) for a, b in zip(
        (r.out_gpu, r.out_host, r.in_host, r.in_gpu),
        (w2.steps[0].out_gpu, w2.steps[0].out_host, w2.steps[0].in_host, w2.steps[0].in_gpu)))
    # tables are scattered, not runs
    assert np.count_nonzero(np.diff(r.out_gpu) == 1) < r.n_out // 2


def test_config2_8b_full_size_lists():
    w = W.config2_8b()
    assert (w.nb_gpu, w.nb_host) == (28610, 57220)          # 60 GB and 120 GB of 2 MiB blocks
    toks = w.extra["tokens"]
    assert len(toks) == 64 and toks.min() >= 16 and toks.max() <= 8192
    assert 600 < np.median(toks) < 1700
    r = w.steps[0]
    assert len(r.out_req_offsets) == 17 and len(r.in_req_offsets) == 17
    assert abs(r.n_out - r.n_in) < 0.05 * r.n_out            # a rotation frees about what it brings in
    assert not set(r.in_gpu) & set(r.out_gpu)
    pairs = w.extra["pairs"]
    assert len(pairs) == 32                                   # every one of the 64 requests rotates once, pairwise
    moved = sum(len(p.out_req_offsets) - 1 + len(p.in_req_offsets) - 1 for p in pairs)
    assert moved == 64 and all(p.n_out and p.n_in and not set(p.in_gpu) & set(p.out_gpu) for p in pairs)
    assert sum(p.n_out + p.n_in for p in pairs) == sum(-(-int(t) // 16) for t in toks)
    for k in ("median", "longest"):
        src, dst = w.extra["single_out"][k]
        assert len(src) == len(dst) and len(set(dst)) == len(dst)
    w.table.check_consistent()


def test_config3_steps_track_residency():
    w = W.config3_70b(nb_gpu=6000, nb_host=9000, n_steps=12)
    assert w.shape.block_bytes == 5 << 20
    tab = W.RequestTable(w.shape, 1, 1, np.random.default_rng(0))   # only for blocks_for
    for s in w.steps:
        assert len(s.out_req_offsets) == 9 and len(s.in_req_offsets) == 9
        assert not set(s.in_gpu) & set(s.out_gpu) and not set(s.in_host) & set(s.out_host)
        assert len(set(s.in_gpu)) == s.n_in and len(set(s.out_host)) == s.n_out
    w.table.check_consistent()
    # what step k swaps in is what step k-2 swapped out (two queues of two groups)
    assert np.array_equal(np.sort(w.steps[2].in_host), np.sort(w.steps[0].out_host))


@pytest.mark.parametrize("contig", [True, False])
def test_config4_cell(contig):
    w = W.config4_sweep_case(32, contig, 64e6)
    r = w.steps[0]
    assert w.shape.block_bytes == 4 << 20 and r.n_out == r.n_in == 15
    if contig:
        assert np.all(np.diff(r.out_gpu) == 1) and np.all(np.diff(r.in_gpu) == 1)
    w.table.check_consistent()


def test_config5_replay_interleaves_and_stays_consistent():
    w = W.config5_replay(rate=8.0, n_steps=1000)
    assert len(w.steps) == 1000
    assert w.nb_gpu <= 0.41 * w.extra["demand_blocks"] + 600
    both = sum(1 for s in w.steps if s.n_out and s.n_in)
    idle = sum(1 for s in w.steps if not s.n_out and not s.n_in)
    assert both > 10 and idle > 10
    for s in w.steps:
        assert not set(s.in_gpu) & set(s.out_gpu) and not set(s.in_host) & set(s.out_host)
        assert len(set(s.in_gpu)) == s.n_in and len(set(s.out_host)) == s.n_out
    w.table.check_consistent()


def test_budgeted_steps_respect_the_budget_and_change_nothing_else():
    """Re-timing rotations under a per-step block budget: no step moves more than the budget, nothing is
    lost or reordered inside a direction, and the pools end up as with the original steps."""
    from oracle.kv_definition import TagModel
    w = W.config5_replay(rate=2.0, n_steps=300, shape=W.KVShape(2, 16, 2, 64), duration_s=20.0, max_tokens=1024)
    for b_xfer in (7, 24, 10_000):
        steps = W.budgeted_steps(w.steps, b_xfer)
        assert len(steps) >= len(w.steps)
        assert max(s.n_out + s.n_in for s in steps) <= b_xfer
        cat = lambda xs: np.concatenate(xs) if xs else np.empty(0, np.int32)
        for field in ("out_gpu", "out_host", "in_host", "in_gpu"):
            assert np.array_equal(cat([getattr(s, field) for s in steps]), cat([getattr(s, field) for s in w.steps]))
        a, b = TagModel(w.nb_gpu, w.nb_host), TagModel(w.nb_gpu, w.nb_host)
        for s in w.steps:
            assert a.rotate(s.out_gpu.tolist(), s.out_host.tolist(), s.in_host.tolist(), s.in_gpu.tolist()) == 0
        for s in steps:     # every emitted step is itself a valid rotation (no cross-direction overlap)
            assert b.rotate(s.out_gpu.tolist(), s.out_host.tolist(), s.in_host.tolist(), s.in_gpu.tolist()) == 0
        assert a.g_tag == b.g_tag and a.h_tag == b.h_tag
    if True:
        big = W.budgeted_steps(w.steps, 10_000)
        assert len(big) == len(w.steps) and all(x.n_out == y.n_out and x.n_in == y.n_in for x, y in zip(big, w.steps))
