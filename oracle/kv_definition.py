"""The rotation path's definition, written out.  TEST INFRASTRUCTURE, not product code.

Follows the paper's section 4.3: a request's KV cache is a virtual tensor
(layers, blocks, segment); swap-out copies every segment of each listed HBM
block into its DRAM block, swap-in does the reverse, and a rotation is both.
The device pool is layer-first ``[layer][K|V][block][block_size][kv_heads][head_dim]``;
the host pool is block-first ``[block][layer][K|V][block_size][kv_heads][head_dim]``
(the paper's merged layout: all layers of one block contiguous), or layer-first
when asked.  Values are opaque 16-bit words: nothing is ever interpreted as a float.

Three independent statements of the same thing:

* ``KVDefinition``     6-D numpy arrays, one indexed assignment per (pair, layer, plane).
* ``ElementwiseModel`` flat word arrays, every word moved by a Python loop whose
                       index arithmetic is spelled out term by term (tiny cases only).
* ``TagModel``         no bytes at all: each block slot holds the name of the
                       original block whose content it now carries.
"""
from __future__ import annotations

import numpy as np

OK = 0
ERR_INVALID_ARG = -1
ERR_RANGE = -2
ERR_DUP_DST = -3
ERR_HAZARD = -4

BLOCK_FIRST = 0
LAYER_FIRST = 1


def seg_bytes(block_size: int, kv_heads: int, head_dim: int) -> int:
    """Bytes of one K-or-V plane of one block in one layer (16-bit elements)."""
    return block_size * kv_heads * head_dim * 2


def blk_bytes(num_layers: int, block_size: int, kv_heads: int, head_dim: int) -> int:
    """Bytes of one block over all layers, K and V."""
    return num_layers * 2 * seg_bytes(block_size, kv_heads, head_dim)


def check_lists(nb_gpu, nb_host, out_gpu, out_host, in_host, in_gpu, allow_overlap=False):
    """Validation shared by all three models; returns an error code, touches nothing.

    Order of checks: ranges of both directions' ids, duplicate destinations inside a
    direction, then the cross-direction overlap that the paper's data-race figure shows
    (a swap-in destination that is a swap-out source; likewise on the host side).
    """
    out_gpu, out_host = list(out_gpu), list(out_host)
    in_host, in_gpu = list(in_host), list(in_gpu)
    if len(out_gpu) != len(out_host) or len(in_host) != len(in_gpu):
        return ERR_INVALID_ARG
    for ids, nb in ((out_gpu, nb_gpu), (out_host, nb_host)):
        if any(i < 0 or i >= nb for i in ids):
            return ERR_RANGE
    if len(set(out_host)) != len(out_host):
        return ERR_DUP_DST
    for ids, nb in ((in_gpu, nb_gpu), (in_host, nb_host)):
        if any(i < 0 or i >= nb for i in ids):
            return ERR_RANGE
    if len(set(in_gpu)) != len(in_gpu):
        return ERR_DUP_DST
    if not allow_overlap:
        if set(in_gpu) & set(out_gpu) or set(in_host) & set(out_host):
            return ERR_HAZARD
    return OK


class KVDefinition:
    """Both pools as 6-D ``uint16`` arrays; every move is one indexed assignment."""

    def __init__(self, num_layers, block_size, kv_heads, head_dim,
                 num_gpu_blocks, num_host_blocks, host_layout=BLOCK_FIRST, dev_layout=LAYER_FIRST):
        self.L, self.bs, self.H, self.D = num_layers, block_size, kv_heads, head_dim
        self.nb_gpu, self.nb_host = num_gpu_blocks, num_host_blocks
        self.host_layout = host_layout
        self.dev_layout = dev_layout
        if dev_layout == LAYER_FIRST:
            self.G = np.zeros((num_layers, 2, num_gpu_blocks, block_size, kv_heads, head_dim), np.uint16)
        else:       # the paper's block-first storage order, applied to the device pool
            self.G = np.zeros((num_gpu_blocks, num_layers, 2, block_size, kv_heads, head_dim), np.uint16)
        if host_layout == BLOCK_FIRST:
            self.Hs = np.zeros((num_host_blocks, num_layers, 2, block_size, kv_heads, head_dim), np.uint16)
        else:
            self.Hs = np.zeros((num_layers, 2, num_host_blocks, block_size, kv_heads, head_dim), np.uint16)

    # logical accessors: the (block_size, kv_heads, head_dim) words of one plane of one block
    def g_seg(self, l, kv, b):
        return self.G[l, kv, b] if self.dev_layout == LAYER_FIRST else self.G[b, l, kv]

    def h_seg(self, l, kv, h):
        return self.Hs[h, l, kv] if self.host_layout == BLOCK_FIRST else self.Hs[l, kv, h]

    def g_block(self, b):
        """All 2L planes of device block b, shape (L, 2, bs, H, D)."""
        return self.G[:, :, b] if self.dev_layout == LAYER_FIRST else self.G[b]

    def h_block(self, h):
        return self.Hs[h] if self.host_layout == BLOCK_FIRST else self.Hs[:, :, h]

    def swap_out(self, gpu_ids, host_ids):
        rc = check_lists(self.nb_gpu, self.nb_host, gpu_ids, host_ids, [], [])
        if rc != OK:
            return rc
        for g, h in zip(gpu_ids, host_ids):
            for l in range(self.L):
                for kv in range(2):
                    self.h_seg(l, kv, h)[...] = self.g_seg(l, kv, g)
        return OK

    def swap_in(self, host_ids, gpu_ids):
        rc = check_lists(self.nb_gpu, self.nb_host, [], [], host_ids, gpu_ids)
        if rc != OK:
            return rc
        for h, g in zip(host_ids, gpu_ids):
            for l in range(self.L):
                for kv in range(2):
                    self.g_seg(l, kv, g)[...] = self.h_seg(l, kv, h)
        return OK

    def rotate(self, out_gpu, out_host, in_host, in_gpu, allow_overlap=False):
        """Swap-out of the first pair of lists, then swap-in of the second."""
        rc = check_lists(self.nb_gpu, self.nb_host, out_gpu, out_host, in_host, in_gpu, allow_overlap)
        if rc != OK:
            return rc
        self.swap_out(out_gpu, out_host)
        self.swap_in(in_host, in_gpu)
        return OK


class ElementwiseModel:
    """Flat word arrays; every 16-bit word is moved on its own by explicit index arithmetic.

    Deliberately avoids the "a segment is contiguous" shortcut, so it pins the layout
    strings themselves.  Pure Python loops: use only on pools of a few blocks.
    """

    def __init__(self, num_layers, block_size, kv_heads, head_dim,
                 num_gpu_blocks, num_host_blocks, host_layout=BLOCK_FIRST):
        self.L, self.bs, self.H, self.D = num_layers, block_size, kv_heads, head_dim
        self.nb_gpu, self.nb_host = num_gpu_blocks, num_host_blocks
        self.host_layout = host_layout
        words_per_block = num_layers * 2 * block_size * kv_heads * head_dim
        self.G = np.zeros(num_gpu_blocks * words_per_block, np.uint16)
        self.Hs = np.zeros(num_host_blocks * words_per_block, np.uint16)

    def g_index(self, l, kv, b, t, hd, d):
        # [layer][K|V][block][block_size][kv_heads][head_dim], row-major
        i = l
        i = i * 2 + kv
        i = i * self.nb_gpu + b
        i = i * self.bs + t
        i = i * self.H + hd
        i = i * self.D + d
        return i

    def h_index(self, h, l, kv, t, hd, d):
        if self.host_layout == BLOCK_FIRST:
            # [block][layer][K|V][block_size][kv_heads][head_dim], row-major
            i = h
            i = i * self.L + l
            i = i * 2 + kv
        else:
            i = l
            i = i * 2 + kv
            i = i * self.nb_host + h
        i = i * self.bs + t
        i = i * self.H + hd
        i = i * self.D + d
        return i

    def _each_word(self):
        for l in range(self.L):
            for kv in range(2):
                for t in range(self.bs):
                    for hd in range(self.H):
                        for d in range(self.D):
                            yield l, kv, t, hd, d

    def swap_out(self, gpu_ids, host_ids):
        rc = check_lists(self.nb_gpu, self.nb_host, gpu_ids, host_ids, [], [])
        if rc != OK:
            return rc
        for g, h in zip(gpu_ids, host_ids):
            for l, kv, t, hd, d in self._each_word():
                self.Hs[self.h_index(h, l, kv, t, hd, d)] = self.G[self.g_index(l, kv, g, t, hd, d)]
        return OK

    def swap_in(self, host_ids, gpu_ids):
        rc = check_lists(self.nb_gpu, self.nb_host, [], [], host_ids, gpu_ids)
        if rc != OK:
            return rc
        for h, g in zip(host_ids, gpu_ids):
            for l, kv, t, hd, d in self._each_word():
                self.G[self.g_index(l, kv, g, t, hd, d)] = self.Hs[self.h_index(h, l, kv, t, hd, d)]
        return OK

    def rotate(self, out_gpu, out_host, in_host, in_gpu, allow_overlap=False):
        rc = check_lists(self.nb_gpu, self.nb_host, out_gpu, out_host, in_host, in_gpu, allow_overlap)
        if rc != OK:
            return rc
        self.swap_out(out_gpu, out_host)
        self.swap_in(in_host, in_gpu)
        return OK


class TagModel:
    """Symbolic model: slot -> (origin_pool, origin_block) of the content it carries.

    Origin pools: 0 = the device pool's initial content, 1 = the host pool's.  A move
    copies the tag, exactly as a move of bytes copies the bytes, so after any sequence
    of valid calls block ``b`` of a pool must hold the initial bytes of ``tag[b]``.
    Also counts writes per destination slot inside one call, for the single-writer check.
    """

    def __init__(self, num_gpu_blocks, num_host_blocks):
        self.nb_gpu, self.nb_host = num_gpu_blocks, num_host_blocks
        self.g_tag = [(0, b) for b in range(num_gpu_blocks)]
        self.h_tag = [(1, h) for h in range(num_host_blocks)]
        self.g_writes = [0] * num_gpu_blocks
        self.h_writes = [0] * num_host_blocks

    def _reset_counts(self):
        self.g_writes = [0] * self.nb_gpu
        self.h_writes = [0] * self.nb_host

    def swap_out(self, gpu_ids, host_ids, _keep_counts=False):
        rc = check_lists(self.nb_gpu, self.nb_host, gpu_ids, host_ids, [], [])
        if rc != OK:
            return rc
        if not _keep_counts:
            self._reset_counts()
        for g, h in zip(gpu_ids, host_ids):
            self.h_tag[h] = self.g_tag[g]
            self.h_writes[h] += 1
        return OK

    def swap_in(self, host_ids, gpu_ids, _keep_counts=False):
        rc = check_lists(self.nb_gpu, self.nb_host, [], [], host_ids, gpu_ids)
        if rc != OK:
            return rc
        if not _keep_counts:
            self._reset_counts()
        for h, g in zip(host_ids, gpu_ids):
            self.g_tag[g] = self.h_tag[h]
            self.g_writes[g] += 1
        return OK

    def rotate(self, out_gpu, out_host, in_host, in_gpu, allow_overlap=False):
        rc = check_lists(self.nb_gpu, self.nb_host, out_gpu, out_host, in_host, in_gpu, allow_overlap)
        if rc != OK:
            return rc
        self._reset_counts()
        self.swap_out(out_gpu, out_host, _keep_counts=True)
        self.swap_in(in_host, in_gpu, _keep_counts=True)
        return OK
