"""Pins for the CPU oracle: things the paper and the mathematics fix, independent of the oracle.

Every model of the rotation path (6-D numpy definition, element-by-element index model, the C
byte model, the symbolic tag model) is checked against closed forms, the paper's worked example,
invariants, an independent indexer (torch), plain numpy slicing on the contiguous special case,
and each other; the last tests plant typical mistakes and show that the pins catch them.
"""
import itertools

import numpy as np
import pytest

from conftest import read_golden
from oracle import kv_definition as D
from oracle.kv_oracle import ByteOracle

RNG = np.random.default_rng(7)


def fill_random(model, rng):
    model.G[...] = rng.integers(0, 65536, size=model.G.shape, dtype=np.uint16)
    model.Hs[...] = rng.integers(0, 65536, size=model.Hs.shape, dtype=np.uint16)


def make_all(L, bs, H, Dm, nbg, nbh, layout, rng):
    """The three byte-carrying models with identical logical content, plus the tag model."""
    d = D.KVDefinition(L, bs, H, Dm, nbg, nbh, layout)
    fill_random(d, rng)
    e = D.ElementwiseModel(L, bs, H, Dm, nbg, nbh, layout)
    e.G[:] = d.G.reshape(-1)
    e.Hs[:] = d.Hs.reshape(-1)
    c = ByteOracle(L, bs, H, Dm, nbg, nbh, layout)
    c.G[:] = d.G.reshape(-1).view(np.uint8)
    c.Hs[:] = d.Hs.reshape(-1).view(np.uint8)
    t = D.TagModel(nbg, nbh)
    return d, e, c, t


def same_state(d, e, c):
    return (np.array_equal(d.G.reshape(-1), e.G) and np.array_equal(d.Hs.reshape(-1), e.Hs)
            and np.array_equal(d.G.reshape(-1).view(np.uint8), c.G)
            and np.array_equal(d.Hs.reshape(-1).view(np.uint8), c.Hs))


# ------------------------------------------------------------------ sizes and strides

def test_paper_worked_example_sizes():
    g = read_golden("paper_sizes.txt")
    L, bs, H, Dm = g["num_layers"], g["block_size"], g["kv_heads"], g["head_dim"]
    # per-token KV per layer = both planes of one token
    assert 2 * D.seg_bytes(1, H, Dm) == g["per_token_bytes_per_layer"]
    # the paper's segment holds K and V; a K-or-V plane is half of it
    assert 2 * D.seg_bytes(bs, H, Dm) == g["segment_bytes_k_plus_v"]
    assert D.blk_bytes(L, bs, H, Dm) == g["block_bytes"]
    blocks = g["tokens_per_direction"] // bs
    assert blocks * D.blk_bytes(L, bs, H, Dm) == g["bytes_per_direction"]
    c = ByteOracle(L, bs, H, Dm, 4, 4, alloc=False)
    assert 2 * c.seg == g["segment_bytes_k_plus_v"] and c.blk == g["block_bytes"]


@pytest.mark.parametrize("L,bs,blk", [(32, 16, 2 << 20), (80, 16, 5 << 20), (2, 16, 128 << 10),
                                      (32, 8, 1 << 20), (32, 64, 8 << 20)])
def test_block_bytes_of_the_configs(L, bs, blk):
    assert D.blk_bytes(L, bs, 8, 128) == blk
    assert ByteOracle(L, bs, 8, 128, 2, 2, alloc=False).blk == blk


def test_stride_formulas():
    """Layer-first: blocks i and j of one layer are (j-i)*S apart, S the contiguous unit.
    Block-first: they are (j-i)*N_L*S_seg apart, S_seg holding K and V, i.e. whole blocks."""
    L, bs, H, Dm, nbg, nbh = 5, 4, 2, 8, 11, 13
    c = ByteOracle(L, bs, H, Dm, nbg, nbh, D.BLOCK_FIRST, alloc=False)
    seg = D.seg_bytes(bs, H, Dm)
    for l, kv, i, j in itertools.product(range(L), range(2), (0, 3), (1, 10)):
        assert c.dev_off(l, kv, j) - c.dev_off(l, kv, i) == (j - i) * seg
        assert c.host_off(j, l, kv) - c.host_off(i, l, kv) == (j - i) * L * (2 * seg)
    # planes follow each other K then V inside a layer, layers follow each other
    assert c.dev_off(0, 1, 0) - c.dev_off(0, 0, 0) == nbg * seg
    assert c.dev_off(1, 0, 0) - c.dev_off(0, 0, 0) == 2 * nbg * seg
    assert c.host_off(0, 0, 1) - c.host_off(0, 0, 0) == seg
    assert c.host_off(0, 1, 0) - c.host_off(0, 0, 0) == 2 * seg
    # offsets tile each pool exactly once
    offs = sorted(c.dev_off(l, kv, b) for l in range(L) for kv in range(2) for b in range(nbg))
    assert offs == list(range(0, 2 * L * nbg * seg, seg))
    offs = sorted(c.host_off(h, l, kv) for l in range(L) for kv in range(2) for h in range(nbh))
    assert offs == list(range(0, 2 * L * nbh * seg, seg))
    lf = ByteOracle(L, bs, H, Dm, nbg, nbh, D.LAYER_FIRST, alloc=False)
    assert lf.host_off(7, 3, 1) == ((3 * 2 + 1) * nbh + 7) * seg


def test_64bit_offsets_at_full_size():
    """60 GB pool of 2 MiB blocks: the last segment starts beyond 2^35."""
    c = ByteOracle(32, 16, 8, 128, 28610, 57220, alloc=False)
    assert c.dev_off(31, 1, 28609) == (63 * 28610 + 28609) * 32768
    assert c.dev_off(31, 1, 28609) + c.seg == 28610 * (2 << 20)
    assert c.host_off(57219, 31, 1) + c.seg == 57220 * (2 << 20)


@pytest.mark.parametrize("layout", [D.BLOCK_FIRST, D.LAYER_FIRST])
def test_torch_as_independent_indexer(layout):
    """A torch tensor of the stated shape, indexed [l, kv, b], must see the bytes that the
    byte model's offset formula names."""
    import torch
    L, bs, H, Dm, nbg, nbh = 3, 2, 2, 4, 5, 6
    d, e, c, _ = make_all(L, bs, H, Dm, nbg, nbh, layout, np.random.default_rng(1))
    tg = torch.from_numpy(c.G.view(np.int16).copy()).view(L, 2, nbg, bs, H, Dm)
    th = (torch.from_numpy(c.Hs.view(np.int16).copy()).view(nbh, L, 2, bs, H, Dm) if layout == D.BLOCK_FIRST
          else torch.from_numpy(c.Hs.view(np.int16).copy()).view(L, 2, nbh, bs, H, Dm))
    for l, kv in itertools.product(range(L), range(2)):
        for b in range(nbg):
            want = tg[l, kv, b].numpy().reshape(-1).view(np.uint16)
            assert np.array_equal(c.g_seg(l, kv, b).view(np.uint16), want)
            assert np.array_equal(d.g_seg(l, kv, b).reshape(-1), want)
            assert e.G[e.g_index(l, kv, b, 1, 1, 3)] == np.uint16(tg[l, kv, b, 1, 1, 3].item() & 0xFFFF)
        for h in range(nbh):
            want = (th[h, l, kv] if layout == D.BLOCK_FIRST else th[l, kv, h]).numpy().reshape(-1).view(np.uint16)
            assert np.array_equal(c.h_seg(l, kv, h).view(np.uint16), want)
            assert np.array_equal(d.h_seg(l, kv, h).reshape(-1), want)


# ------------------------------------------------------------------ invariants

def random_lists(rng, nbg, nbh, n_out, n_in, disjoint=True):
    out_gpu = rng.choice(nbg, n_out, replace=False)
    out_host = rng.choice(nbh, n_out, replace=False)
    if disjoint:
        g_left = np.setdiff1d(np.arange(nbg), out_gpu)
        h_left = np.setdiff1d(np.arange(nbh), out_host)
    else:
        g_left, h_left = np.arange(nbg), np.arange(nbh)
    in_gpu = rng.choice(g_left, n_in, replace=False)
    in_host = rng.choice(h_left, n_in, replace=False)
    return [x.astype(np.int32) for x in (out_gpu, out_host, in_host, in_gpu)]


@pytest.mark.parametrize("layout", [D.BLOCK_FIRST, D.LAYER_FIRST])
def test_round_trip_untouched_and_single_writer(layout):
    rng = np.random.default_rng(11)
    L, bs, H, Dm, nbg, nbh = 3, 4, 2, 8, 24, 40
    d, e, c, t = make_all(L, bs, H, Dm, nbg, nbh, layout, rng)
    G0, H0 = d.G.copy(), d.Hs.copy()
    src = rng.choice(nbg, 6, replace=False)
    via = rng.choice(nbh, 6, replace=False)
    back = rng.choice(np.setdiff1d(np.arange(nbg), src), 6, replace=False)
    for m in (d, c, t):
        assert m.swap_out(src, via) == 0
    # swap-out leaves the device pool alone and writes only the named host blocks
    assert np.array_equal(d.G, G0)
    for h in range(nbh):
        if h not in via:
            assert np.array_equal(d.h_block(h), (H0[h] if layout == D.BLOCK_FIRST else H0[:, :, h]))
    for g, h in zip(src, via):
        assert np.array_equal(d.h_block(h), G0[:, :, g])
    assert all(t.h_writes[h] == (1 if h in via else 0) for h in range(nbh)) and sum(t.g_writes) == 0
    H1 = d.Hs.copy()
    for m in (d, c, t):
        assert m.swap_in(via, back) == 0
    assert np.array_equal(d.Hs, H1)                      # swap-in leaves the host pool alone
    for g, g2 in zip(src, back):                          # round trip to different ids
        assert np.array_equal(d.G[:, :, g2], G0[:, :, g])
        assert t.g_tag[g2] == (0, int(g))
    for g in range(nbg):
        if g not in back:
            assert np.array_equal(d.G[:, :, g], G0[:, :, g])
    assert all(t.g_writes[g] == (1 if g in back else 0) for g in range(nbg)) and sum(t.h_writes) == 0
    # C byte model agrees with the definition
    assert np.array_equal(d.G.reshape(-1).view(np.uint8), c.G)
    assert np.array_equal(d.Hs.reshape(-1).view(np.uint8), c.Hs)


def tags_match_bytes(d, t, G0, H0):
    """Block b of each pool must carry the initial bytes of the block its tag names."""
    def origin(tag):
        pool, b = tag
        if pool == 0:
            return G0[:, :, b]
        return H0[b] if d.host_layout == D.BLOCK_FIRST else H0[:, :, b]
    return (all(np.array_equal(d.g_block(g), origin(t.g_tag[g])) for g in range(d.nb_gpu))
            and all(np.array_equal(d.h_block(h), origin(t.h_tag[h])) for h in range(d.nb_host)))


@pytest.mark.parametrize("layout", [D.BLOCK_FIRST, D.LAYER_FIRST])
def test_models_agree_on_random_rotation_sequences(layout):
    rng = np.random.default_rng(5)
    L, bs, H, Dm, nbg, nbh = 2, 2, 1, 8, 12, 16
    d, e, c, t = make_all(L, bs, H, Dm, nbg, nbh, layout, rng)
    G0, H0 = d.G.copy(), d.Hs.copy()
    for step in range(12):
        n_out, n_in = int(rng.integers(0, 5)), int(rng.integers(0, 5))
        lists = random_lists(rng, nbg, nbh, n_out, n_in)
        for m in (d, e, c, t):
            assert m.rotate(*lists) == 0
        assert same_state(d, e, c)
        assert tags_match_bytes(d, t, G0, H0)
        assert max(t.g_writes + t.h_writes) <= 1


def test_disjoint_rotation_commutes():
    """With no cross-direction overlap, out-then-in equals in-then-out: the condition under
    which the two directions may run concurrently."""
    rng = np.random.default_rng(9)
    L, bs, H, Dm, nbg, nbh = 2, 2, 2, 4, 20, 20
    d1, _, c1, _ = make_all(L, bs, H, Dm, nbg, nbh, D.BLOCK_FIRST, rng)
    d2 = D.KVDefinition(L, bs, H, Dm, nbg, nbh)
    d2.G[...], d2.Hs[...] = d1.G, d1.Hs
    og, oh, ih, ig = random_lists(rng, nbg, nbh, 7, 6)
    assert d1.rotate(og, oh, ih, ig) == 0
    assert d2.swap_in(ih, ig) == 0 and d2.swap_out(og, oh) == 0
    assert np.array_equal(d1.G, d2.G) and np.array_equal(d1.Hs, d2.Hs)
    # threaded C variant equals the sequential one
    c2 = ByteOracle(L, bs, H, Dm, nbg, nbh)
    c2.G[:], c2.Hs[:] = c1.G, c1.Hs
    assert c1.rotate(og, oh, ih, ig) == 0 and c2.rotate(og, oh, ih, ig, threads=3) == 0
    assert np.array_equal(c1.G, c2.G) and np.array_equal(c1.Hs, c2.Hs)
    assert np.array_equal(d1.G.reshape(-1).view(np.uint8), c1.G)


def test_overlapping_rotation_is_out_then_in():
    """The paper's race: a swap-in destination that is a swap-out source.  Sequential semantics
    say the host copy receives the OLD device bytes and the device block then takes the new ones;
    and a swap-in that reads a host block written by the same call's swap-out sees the NEW bytes."""
    rng = np.random.default_rng(3)
    d, e, c, t = make_all(2, 2, 1, 4, 6, 6, D.BLOCK_FIRST, rng)
    G0, H0 = d.G.copy(), d.Hs.copy()
    lists = ([2, 4], [1, 3], [5, 1], [2, 0])     # in_gpu 2 == out_gpu 2 ; in_host 1 == out_host 1
    for m in (d, e, c, t):
        assert m.rotate(*lists) == D.ERR_HAZARD
    assert np.array_equal(d.G, G0) and np.array_equal(d.Hs, H0)     # refused: nothing moved
    assert same_state(d, e, c)
    for m in (d, e, c, t):
        assert m.rotate(*lists, allow_overlap=True) == 0
    assert same_state(d, e, c)
    assert np.array_equal(d.Hs[1], G0[:, :, 2]) and np.array_equal(d.Hs[3], G0[:, :, 4])
    assert np.array_equal(d.G[:, :, 2], H0[5])           # device block 2 overwritten after it was saved
    assert np.array_equal(d.G[:, :, 0], G0[:, :, 2])     # read back what this call had just swapped out
    assert t.g_tag[0] == (0, 2) and t.g_tag[2] == (1, 5) and t.h_tag[1] == (0, 2)


def test_contiguous_special_case_is_plain_slicing():
    """Identity tables over a run of ids: swap-out is, per (layer, plane), one contiguous slab."""
    rng = np.random.default_rng(2)
    L, bs, H, Dm, nbg, nbh = 3, 4, 2, 8, 16, 16
    c = ByteOracle(L, bs, H, Dm, nbg, nbh, D.LAYER_FIRST)
    c.G[:] = rng.integers(0, 256, c.G.size, dtype=np.uint8)
    c.Hs[:] = rng.integers(0, 256, c.Hs.size, dtype=np.uint8)
    G0, H0 = c.G.copy(), c.Hs.copy()
    ids = np.arange(4, 11, dtype=np.int32)
    assert c.swap_out(ids, ids) == 0
    seg = c.seg
    want = H0.copy().reshape(2 * L, nbh * seg)
    want[:, 4 * seg:11 * seg] = G0.reshape(2 * L, nbg * seg)[:, 4 * seg:11 * seg]
    assert np.array_equal(c.Hs, want.reshape(-1)) and np.array_equal(c.G, G0)
    # block-first host: each block is the concatenation of its planes
    b = ByteOracle(L, bs, H, Dm, nbg, nbh, D.BLOCK_FIRST)
    b.G[:], b.Hs[:] = G0, H0
    assert b.swap_out(ids, ids) == 0
    planes = G0.reshape(2 * L, nbg, seg)
    for h in ids:
        assert np.array_equal(b.Hs[h * b.blk:(h + 1) * b.blk], planes[:, h, :].reshape(-1))


def test_validation_codes_and_no_side_effects():
    rng = np.random.default_rng(4)
    d, e, c, t = make_all(1, 2, 1, 4, 5, 5, D.BLOCK_FIRST, rng)
    G0, H0 = d.G.copy(), d.Hs.copy()
    bad = [
        (([0, 5], [0, 1], [], []), D.ERR_RANGE),          # gpu id out of range
        (([0, 1], [0, -1], [], []), D.ERR_RANGE),
        (([0, 1], [2, 2], [], []), D.ERR_DUP_DST),        # same host destination twice
        (([], [], [0, 1], [3, 3]), D.ERR_DUP_DST),        # same device destination twice
        (([0], [1], [2], [0]), D.ERR_HAZARD),             # in-dst is out-src
        (([0], [1], [1], [2]), D.ERR_HAZARD),             # in-src is out-dst
        (([0, 1], [1], [], []), D.ERR_INVALID_ARG),       # ragged pair lists
    ]
    for lists, code in bad:
        for m in (d, e, c, t):
            assert m.rotate(*lists) == code, (lists, code, type(m).__name__)
        assert np.array_equal(d.G, G0) and np.array_equal(d.Hs, H0) and same_state(d, e, c)
    # duplicate SOURCES are fine, and empty lists are no-ops
    for m in (d, e, c, t):
        assert m.rotate([3, 3], [0, 1], [], []) == 0
        assert m.rotate([], [], [], []) == 0
    assert np.array_equal(d.Hs[0], G0[:, :, 3]) and np.array_equal(d.Hs[1], G0[:, :, 3])
    assert same_state(d, e, c)


# ------------------------------------------------------------------ exhaustive tiny pools

@pytest.mark.parametrize("L,bs,nbg,nbh", [(1, 1, 3, 3), (2, 2, 3, 4)])
def test_exhaustive_injective_lists_on_tiny_pools(L, bs, nbg, nbh):
    """Every injective pair list of length <= 2 each way (<= 3 for one direction alone) on pools of
    3-4 blocks: all four models agree and the invariants hold."""
    rng = np.random.default_rng(13)
    H, Dm = 1, 8
    base = make_all(L, bs, H, Dm, nbg, nbh, D.BLOCK_FIRST, rng)
    G0, H0 = base[0].G.copy(), base[0].Hs.copy()

    def pair_lists(n_src, n_dst, maxlen):
        for n in range(maxlen + 1):
            for src in itertools.product(range(n_src), repeat=n):          # sources may repeat
                for dst in itertools.permutations(range(n_dst), n):        # destinations injective
                    yield list(src), list(dst)

    def fresh():
        d = D.KVDefinition(L, bs, H, Dm, nbg, nbh)
        d.G[...], d.Hs[...] = G0, H0
        e = D.ElementwiseModel(L, bs, H, Dm, nbg, nbh)
        e.G[:], e.Hs[:] = G0.reshape(-1), H0.reshape(-1)
        c = ByteOracle(L, bs, H, Dm, nbg, nbh)
        c.G[:], c.Hs[:] = G0.reshape(-1).view(np.uint8), H0.reshape(-1).view(np.uint8)
        return d, e, c, D.TagModel(nbg, nbh)

    count = 0
    outs = list(pair_lists(nbg, nbh, 2))
    ins = list(pair_lists(nbh, nbg, 2))            # (host sources, injective device destinations)
    for (og, oh) in outs:
        for (ih, ig) in ins:
            overlap = bool(set(ig) & set(og)) or bool(set(ih) & set(oh))
            d, e, c, t = fresh()
            for m in (d, e, c, t):
                assert m.rotate(og, oh, ih, ig) == (D.ERR_HAZARD if overlap else 0)
            if overlap:
                assert np.array_equal(d.G, G0) and np.array_equal(d.Hs, H0)
                for m in (d, e, c, t):
                    assert m.rotate(og, oh, ih, ig, allow_overlap=True) == 0
            assert same_state(d, e, c)
            assert tags_match_bytes(d, t, G0, H0)
            assert max(t.g_writes + t.h_writes) <= 1
            touched_g, touched_h = set(ig), set(oh)
            assert all(np.array_equal(d.G[:, :, g], G0[:, :, g]) for g in range(nbg) if g not in touched_g)
            assert all(np.array_equal(d.Hs[h], H0[h]) for h in range(nbh) if h not in touched_h)
            count += 1
    assert count == len(outs) * len(ins)
    # single directions up to length 3
    for (og, oh) in pair_lists(nbg, nbh, 3):
        d, e, c, t = fresh()
        for m in (d, e, c, t):
            assert m.swap_out(og, oh) == 0
        assert same_state(d, e, c) and tags_match_bytes(d, t, G0, H0)


# ------------------------------------------------------------------ the pins have teeth

class _SwappedPlaneOrder(D.ElementwiseModel):
    def h_index(self, h, l, kv, t, hd, d):          # planted: [block][K|V][layer] instead of [block][layer][K|V]
        i = (h * 2 + kv) * self.L + l
        return ((i * self.bs + t) * self.H + hd) * self.D + d


class _LayerStrideOffByOne(D.ElementwiseModel):
    def g_index(self, l, kv, b, t, hd, d):          # planted: stride of nb_gpu-1 blocks per plane
        i = (l * 2 + kv) * (self.nb_gpu - 1) + b
        return ((i * self.bs + t) * self.H + hd) * self.D + d


class _DroppedVPlane(D.KVDefinition):
    def swap_out(self, gpu_ids, host_ids):          # planted: copies K only
        for g, h in zip(gpu_ids, host_ids):
            for l in range(self.L):
                self.h_seg(l, 0, h)[...] = self.g_seg(l, 0, g)
        return 0


class _InBeforeOut(D.KVDefinition):
    def rotate(self, og, oh, ih, ig, allow_overlap=False):     # planted: wrong order
        self.swap_in(ih, ig)
        self.swap_out(og, oh)
        return 0


def test_planted_mistakes_are_caught():
    rng = np.random.default_rng(21)
    L, bs, H, Dm, nbg, nbh = 2, 2, 2, 4, 6, 6
    d, e, c, t = make_all(L, bs, H, Dm, nbg, nbh, D.BLOCK_FIRST, rng)
    G0, H0 = d.G.copy(), d.Hs.copy()
    for cls in (_SwappedPlaneOrder, _LayerStrideOffByOne):
        bad = cls(L, bs, H, Dm, nbg, nbh)
        bad.G[:], bad.Hs[:] = G0.reshape(-1), H0.reshape(-1)
        good = D.KVDefinition(L, bs, H, Dm, nbg, nbh)
        good.G[...], good.Hs[...] = G0, H0
        bad.swap_out([1, 4], [0, 5]); bad.swap_in([0, 5], [2, 3])
        good.swap_out([1, 4], [0, 5]); good.swap_in([0, 5], [2, 3])
        assert not (np.array_equal(good.G.reshape(-1), bad.G) and np.array_equal(good.Hs.reshape(-1), bad.Hs)), cls
    bad = _DroppedVPlane(L, bs, H, Dm, nbg, nbh)
    bad.G[...], bad.Hs[...] = G0, H0
    bad.swap_out([1], [0])
    assert not np.array_equal(bad.h_block(0), G0[:, :, 1])                  # round-trip pin fails
    bad = _InBeforeOut(L, bs, H, Dm, nbg, nbh)
    bad.G[...], bad.Hs[...] = G0, H0
    bad.rotate([2], [1], [1], [0], allow_overlap=True)
    assert not np.array_equal(bad.G[:, :, 0], G0[:, :, 2])                  # sequential-semantics pin fails


# ------------------------------------------------------------ block-first DEVICE layout (the paper's redesign)

def test_block_first_device_layout_strides_and_paper_sizes():
    """Section 4.3.2: with block-first storage all layers of a block are contiguous (64 KB segments merge
    into one 4 MB region for Qwen2.5-32B) and the stride between blocks i and j is (j-i)*N_L*S_seg."""
    g = read_golden("paper_sizes.txt")
    L, bs, H, Dm = g["num_layers"], g["block_size"], g["kv_heads"], g["head_dim"]
    c = ByteOracle(L, bs, H, Dm, 9, 9, alloc=False, dev_layout=1)
    assert c.dev_off(0, 0, 1) - c.dev_off(0, 0, 0) == g["block_bytes"] == L * g["segment_bytes_k_plus_v"]
    assert c.dev_off(1, 0, 0) - c.dev_off(0, 0, 0) == g["segment_bytes_k_plus_v"]      # next layer: next segment
    assert c.dev_off(0, 1, 0) - c.dev_off(0, 0, 0) == g["segment_bytes_k_plus_v"] // 2  # V plane follows K plane
    small = ByteOracle(5, 4, 2, 8, 11, 13, alloc=False, dev_layout=1)
    seg = small.seg
    for l, kv, i, j in itertools.product(range(5), range(2), (0, 3), (1, 10)):
        assert small.dev_off(l, kv, j) - small.dev_off(l, kv, i) == (j - i) * 5 * (2 * seg)
    offs = sorted(small.dev_off(l, kv, b) for l in range(5) for kv in range(2) for b in range(11))
    assert offs == list(range(0, 2 * 5 * 11 * seg, seg))
    # the same rule as the block-first host pool
    assert all(small.dev_off(l, kv, b) == small.host_off(b, l, kv) for l in range(5) for kv in range(2) for b in range(11))


@pytest.mark.parametrize("host_layout", [D.BLOCK_FIRST, D.LAYER_FIRST])
def test_block_first_device_layout_moves_the_same_logical_content(host_layout):
    """Changing where the device pool keeps a plane must not change what a rotation does to the logical
    content: byte oracle and 6-D definition, both on the block-first device layout, against the
    layer-first pair on the same logical data and lists."""
    rng = np.random.default_rng(21)
    L, bs, H, Dm, nbg, nbh = 3, 4, 2, 8, 10, 12
    dl = D.KVDefinition(L, bs, H, Dm, nbg, nbh, host_layout)                       # layer-first device
    db = D.KVDefinition(L, bs, H, Dm, nbg, nbh, host_layout, dev_layout=D.BLOCK_FIRST)
    cb = ByteOracle(L, bs, H, Dm, nbg, nbh, host_layout, dev_layout=1)
    dl.G[...] = rng.integers(0, 65536, dl.G.shape, dtype=np.uint16)
    dl.Hs[...] = rng.integers(0, 65536, dl.Hs.shape, dtype=np.uint16)
    db.G[...] = np.moveaxis(dl.G, 2, 0)                                             # same logical content
    db.Hs[...] = dl.Hs
    cb.G[:] = db.G.reshape(-1).view(np.uint8)                                       # row-major = the byte layout
    cb.Hs[:] = db.Hs.reshape(-1).view(np.uint8)
    for _ in range(5):
        og, oh, ih, ig = random_lists(rng, nbg, nbh, 4, 3)
        assert dl.rotate(og, oh, ih, ig) == db.rotate(og, oh, ih, ig) == cb.rotate(og, oh, ih, ig) == 0
    assert np.array_equal(np.moveaxis(dl.G, 2, 0), db.G) and np.array_equal(dl.Hs, db.Hs)
    assert np.array_equal(cb.G.view(np.uint16), db.G.reshape(-1))
    assert np.array_equal(cb.Hs.view(np.uint16), db.Hs.reshape(-1))
