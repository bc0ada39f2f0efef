"""The C-ABI library loads without a GPU and exports every function ``include/duplexkv.h`` declares;
the Python binding names the same set.  No compute call is made here."""
import ctypes as C
import os
import re

from paper_2601_20309_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "duplexkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)                   # drop comments
    return sorted(set(re.findall(r"^\s*(?:const\s+char\s*\*|int32_t|int64_t)\s*(kv_[a-z0-9_]+)\s*\(", text, flags=re.M)))


def test_header_declares_the_named_calls():
    names = declared_functions()
    for must in ("kv_pool_create", "kv_swap_out", "kv_swap_in", "kv_rotate", "kv_sync"):
        assert must in names
    assert len(names) >= 15


def test_library_exports_every_declared_symbol():
    lib = B.lib()
    missing = [n for n in declared_functions() if not hasattr(lib, n)]
    assert not missing, missing


def test_binding_names_match_the_header():
    assert sorted(B.EXPORTS) == declared_functions()


def test_shape_helpers_need_no_device():
    assert B.kv_seg_bytes(16, 8, 128) == 32768
    assert B.kv_blk_bytes(32, 16, 8, 128) == 2 << 20
    assert B.kv_blk_bytes(80, 16, 8, 128) == 5 << 20
    assert B.kv_seg_bytes(0, 8, 128) == 0
    assert B.kv_path_for(2 << 20) == B.KV_PATH_STAGED and B.kv_path_for(1 << 20) == B.KV_PATH_ZEROCOPY


def test_struct_sizes_match_the_header_layout():
    # natural alignment on both sides; a mismatch here means the ctypes mirror drifted from the header
    assert C.sizeof(B.kv_pool_config_t) == 112
    assert C.sizeof(B.kv_stats_t) == 144
    assert C.sizeof(B.kv_link_probe_t) == 56
    assert C.sizeof(B.kv_probe_spec_t) == 72


def test_bounds_predicate_of_the_debug_flag():
    """What the kernels check under KV_FLAG_DEBUG_BOUNDS, as the plain host function it is written as."""
    ok = B.kv_debug_pair_in_bounds
    assert ok(0, 0, 1, 1) and ok(27, 511, 28, 512)
    assert not ok(28, 0, 28, 512) and not ok(0, 512, 28, 512)       # one past the end, either side
    assert not ok(-1, 0, 28, 512) and not ok(0, -1, 28, 512)        # negative ids
    assert not ok(0, 0, 0, 5) and not ok(2 ** 31 - 1, 0, 2 ** 31 - 1, 1)


def test_ring_shape_of_the_bulk_kernel_by_segment_size():
    """Host logic that picks the bulk kernel's ring: an item must fit a stage (a bulk copy that overran its
    stage would write into the next warp's), the shared memory of a CTA must fit an SM, a stage may be
    refilled only after the store that read it (stages >= ahead + 2 with one group allowed pending), and
    smaller items get at least as many issuing warps."""
    table = {  # segment bytes, over the link -> stage, stages, ahead, warps
        (32768, False): (16384, 4, 2, 1), (16384, False): (16384, 4, 2, 1), (8192, False): (8192, 4, 2, 2),
        (4096, False): (4096, 4, 2, 4), (2048, False): (2048, 4, 2, 8), (1024, False): (1024, 3, 1, 16),
        (32768, True): (8192, 8, 6, 1), (8192, True): (8192, 8, 6, 1), (4096, True): (4096, 8, 6, 2),
        (2048, True): (2048, 8, 6, 4), (1024, True): (1024, 8, 6, 8)}
    for (seg, link), want in table.items():
        _, s = B.kv_debug_ring_shape(seg, link)
        assert (s["stage_bytes"], s["stages"], s["ahead"], s["warps"]) == want, (seg, link, s)
    cap = {(False, 0): 16384, (True, 0): 8192, (True, 1): 32768, (True, 2): 65536}
    for (link, variant), biggest in cap.items():
        last_warps = 1 << 30
        for seg in list(range(16, 4208, 16)) + list(range(4208, 70000, 304)):
            _, s = B.kv_debug_ring_shape(seg, link, variant)
            assert s["item_bytes"] == min(seg, biggest)
            assert s["item_bytes"] <= s["stage_bytes"], (seg, link, variant, s)
            assert s["stage_bytes"] % 128 == 0
            assert s["stage_bytes"] * s["stages"] * s["warps"] <= 227 * 1024
            assert 1 <= s["ahead"] and s["ahead"] + 2 <= s["stages"]
            assert 1 <= s["warps"] <= 16
            assert s["warps"] <= last_warps
            last_warps = s["warps"]
    assert B.kv_debug_ring_shape(24, check=False)[0] == B.KV_ERR_INVALID_ARG
    assert B.kv_debug_ring_shape(0, check=False)[0] == B.KV_ERR_INVALID_ARG
    assert B.kv_debug_ring_shape(4096, True, 3, check=False)[0] == B.KV_ERR_INVALID_ARG
