"""The staged path's transfer planner (host logic, no GPU): for any list of host ids the planned
transfers cover every block exactly once, their row geometry matches the ids, no chunk exceeds a staging
half, scattered lists give transfers that all carry two blocks, and long runs are merged."""
import numpy as np
import pytest

from paper_2601_20309_b200 import binding as B

BLK = 2 << 20


def check_plan(host_ids, half_blocks, direction, blk=BLK):
    host_ids = np.asarray(host_ids, np.int32)
    ops, order = B.kv_plan_staged(blk, half_blocks, direction, host_ids)
    n = len(host_ids)
    assert sorted(order.tolist()) == list(range(n))                         # a permutation of the list
    staged_ids = host_ids[order]                                            # host id at every staging position
    pos = 0
    per_chunk = {}
    for op in ops:
        assert op["first_position"] == pos                                  # issue order walks the staging order
        assert op["rows"] >= 1 and op["blocks_per_row"] >= 1 and op["slices"] >= 1
        for s in range(op["slices"]):
            for r in range(op["rows"]):
                for j in range(op["blocks_per_row"]):
                    want = op["host_block"] + s * op["slice_pitch_blocks"] + r * op["pitch_blocks"] + j
                    assert staged_ids[pos] == want, (op, s, r, j)
                    pos += 1
        if op["rows"] > 1:
            assert op["pitch_blocks"] >= op["blocks_per_row"]                # rows do not overlap in host memory
            assert op["pitch_blocks"] * blk <= 2 ** 31 - 1                   # what a strided transfer accepts
        if op["slices"] > 1:
            assert op["rows"] > 1 and op["slice_pitch_blocks"] % op["pitch_blocks"] == 0      # a whole number of row pitches
            assert op["slice_pitch_blocks"] >= op["rows"] * op["pitch_blocks"]                # slices do not interleave
        per_chunk[op["chunk"]] = per_chunk.get(op["chunk"], 0) + op["slices"] * op["rows"] * op["blocks_per_row"]
    assert pos == n                                                          # every block exactly once
    assert sorted(per_chunk) == list(range(len(per_chunk)))                  # chunks numbered in order
    assert all(v <= half_blocks for v in per_chunk.values())                 # a chunk fits a staging half
    if all(op["slices"] == 1 for op in ops):
        assert np.all(np.diff(staged_ids) >= 0)                             # without lattices: ascending host id
    return ops, per_chunk


def _blocks(op):
    return op["slices"] * op["rows"] * op["blocks_per_row"]


@pytest.mark.parametrize("direction", [0, 1])
@pytest.mark.parametrize("seed", range(5))
def test_scattered_ids_travel_four_or_two_per_transfer(seed, direction):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(50, 700))
    ids = rng.choice(60_000, n, replace=False)
    ops, chunks = check_plan(ids, 512, direction)
    sizes = [_blocks(op) for op in ops]
    # lattices of four first, then pairs; ids more than 2 GiB apart cannot share a strided transfer
    far = sum(1 for a, b in zip(np.sort(ids), np.sort(ids)[1:]) if (b - a) * BLK > 2 ** 31 - 1)
    assert set(sizes) <= {4, 2, 1} and sizes.count(1) <= 1 + far
    assert sizes == sorted(sizes, reverse=True) or far                     # four-block transfers are issued first
    assert all(op["slices"] == 2 and op["rows"] == 2 for op in ops if _blocks(op) == 4)
    assert len(ops) <= (n + 1) // 2 + 8


def test_lattices_cover_most_of_a_scattered_list():
    """1844 ids drawn from 57 220 (the density of the 8B-shaped rotation): about three quarters of the
    blocks find a place in a four-block lattice; a denser list does better."""
    rng = np.random.default_rng(11)
    for n, nb, least in ((1844, 57_220, 0.65), (4096, 57_220, 0.85)):
        ids = rng.choice(nb, n, replace=False)
        ops, _ = check_plan(ids, 512, 0)
        in_fours = sum(4 for op in ops if _blocks(op) == 4)
        assert in_fours >= least * n, (n, in_fours)
        assert all(op["pitch_blocks"] <= 256 for op in ops if _blocks(op) == 4)


def test_hand_made_lattice():
    # 10, 13 and 31, 34: gap 3, starts congruent modulo 3 (31 - 10 = 7 * 3): one transfer; the rest go in pairs
    ops, _ = check_plan([34, 500, 10, 900, 31, 13, 77, 70], 64, 0)
    four = [op for op in ops if _blocks(op) == 4]
    assert len(four) == 1
    assert (four[0]["host_block"], four[0]["pitch_blocks"], four[0]["slice_pitch_blocks"]) == (10, 3, 21)
    assert [_blocks(op) for op in ops] == [4, 2, 2]


def test_long_runs_are_merged_and_cut_at_chunk_size():
    ids = np.concatenate([np.arange(1000, 1300), np.arange(5000, 5200), np.arange(9000, 9040)])    # runs of 300, 200, 40
    rng = np.random.default_rng(0)
    ops, chunks = check_plan(rng.permutation(ids), 128, 1)
    assert all(_blocks(op) <= 128 for op in ops)
    assert len(ops) <= 8                                                     # 300 -> 3, 200 -> 2, 40 -> 1 (or merged rows)
    assert sum(chunks.values()) == 540
    one, _ = check_plan(np.arange(77, 77 + 64), 512, 0)                      # 128 MiB or less: one chunk, one transfer
    assert len(one) == 1 and one[0]["blocks_per_row"] == 64
    four, _ = check_plan(np.arange(77, 77 + 200), 512, 0)                    # larger, but fits one half: about four chunks,
    sizes = [_blocks(op) for op in four]                                     # the first of a swap-out half as long
    assert sizes == [26, 52, 52, 52, 18]                                     # equal chunks of a multiple of four blocks
    four_in, _ = check_plan(np.arange(77, 77 + 200), 512, 1)
    assert [_blocks(op) for op in four_in] == [52, 52, 52, 44]


def test_short_runs_are_not_merged_into_uneven_transfers():
    """Runs of 1 to 4 blocks: merging would give transfers of many sizes; the plan keeps them all alike."""
    rng = np.random.default_rng(3)
    ids, at = [], 0
    while len(ids) < 400:
        L = int(rng.integers(1, 5))
        ids += list(range(at, at + L))
        at += L + int(rng.integers(2, 50))
    ops, _ = check_plan(rng.permutation(np.array(ids[:400])), 512, 0)
    assert {_blocks(op) for op in ops} <= {4, 2}
    assert 100 <= len(ops) <= 200


def test_equal_runs_at_a_constant_spacing_share_one_strided_transfer():
    ids = np.concatenate([np.arange(s, s + 16) for s in range(100, 100 + 8 * 40, 40)])            # 8 runs of 16, 40 apart
    ops, _ = check_plan(ids, 512, 0)
    assert any(op["rows"] > 1 and op["blocks_per_row"] == 16 and op["pitch_blocks"] == 40 for op in ops)
    assert len(ops) <= 5                                                     # chunks of 16, 32, 32, 32, 16 blocks


def test_repeated_sources_far_apart_ids_and_tiny_lists():
    check_plan([7, 7, 8, 7, 30, 30, 31], 16, 1)                              # swap-in sources may repeat
    ops, _ = check_plan([0, 5000, 10000, 15000], 16, 0)                      # more than 2 GiB apart: singles
    assert all(op["rows"] == 1 for op in ops)
    ops, _ = check_plan([42], 16, 0)
    assert len(ops) == 1
    ops, order = B.kv_plan_staged(BLK, 16, 0, [])
    assert ops == [] and len(order) == 0
    check_plan(np.arange(50)[::-1], 3, 1)                                    # tiny staging halves
    with pytest.raises(B.KVError):
        B.kv_plan_staged(BLK, 0, 0, [1, 2])
    with pytest.raises(B.KVError):
        B.kv_plan_staged(BLK, 16, 0, [1, -2])


@pytest.mark.parametrize("blk", [128 << 10, 1 << 20, 8 << 20])
def test_other_block_sizes(blk):
    rng = np.random.default_rng(9)
    check_plan(rng.choice(5000, 333, replace=False), max(2, (64 << 20) // blk), 0, blk=blk)
    check_plan(np.arange(10, 410), max(2, (64 << 20) // blk), 1, blk=blk)


def test_lattices_with_repeated_sources_and_dense_ids():
    """Swap-in sources may repeat: the plan must still name every list entry exactly once; and a dense
    scattered list (every other id) is all lattices."""
    rng = np.random.default_rng(5)
    ids = rng.choice(3000, 300, replace=False)
    ids = np.concatenate([ids, ids[:40], ids[:7]])                           # 47 entries repeat earlier ones
    check_plan(rng.permutation(ids), 512, 1)
    ops, _ = check_plan(np.arange(0, 400, 2), 512, 0)                        # 0, 2, 4, ...: gap 2 everywhere
    assert all(_blocks(op) == 4 for op in ops)
    ops, _ = check_plan(np.arange(0, 64, 2), 3, 0)                           # halves too small for a lattice: pairs
    assert all(op["slices"] == 1 for op in ops)


def test_large_blocks_travel_in_pairs_only():
    """A pair of 4 MiB blocks is an 8 MiB transfer already: no lattices, one transfer size."""
    rng = np.random.default_rng(12)
    ids = rng.choice(20_000, 600, replace=False)
    for blk, expect_fours in ((1 << 20, True), (2 << 20, True), (4 << 20, False), (5 << 20, False), (8 << 20, False)):
        ops, _ = check_plan(ids, 4096, 0, blk=blk)
        assert any(_blocks(op) == 4 for op in ops) == expect_fours, blk
