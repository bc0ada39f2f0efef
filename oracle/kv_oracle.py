"""ctypes front end of ``kv_oracle.c``.  TEST INFRASTRUCTURE, not product code.

``ByteOracle`` owns two flat ``uint8`` numpy arrays (the device-pool model ``G`` and
the host-pool model ``Hs``) and applies swap-out / swap-in / rotate to them with the
C routines, which copy one segment at a time at byte offsets computed from the
layer-first and block-first stride formulas of the paper's section 4.3.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from . import build as _build

OK = 0
ERR_INVALID_ARG = -1
ERR_RANGE = -2
ERR_DUP_DST = -3
ERR_HAZARD = -4


class _Shape(C.Structure):
    _fields_ = [("num_layers", C.c_int32), ("block_size", C.c_int32),
                ("kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("num_gpu_blocks", C.c_int64), ("num_host_blocks", C.c_int64),
                ("host_layout", C.c_int32), ("dev_layout", C.c_int32)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        sp, i32p, u8p = C.POINTER(_Shape), C.POINTER(C.c_int32), C.c_void_p
        L.kvo_seg_bytes.restype = C.c_int64
        L.kvo_seg_bytes.argtypes = [sp]
        L.kvo_blk_bytes.restype = C.c_int64
        L.kvo_blk_bytes.argtypes = [sp]
        L.kvo_dev_off.restype = C.c_int64
        L.kvo_dev_off.argtypes = [sp, C.c_int64, C.c_int64, C.c_int64]
        L.kvo_host_off.restype = C.c_int64
        L.kvo_host_off.argtypes = [sp, C.c_int64, C.c_int64, C.c_int64]
        L.kvo_swap_out.restype = C.c_int32
        L.kvo_swap_out.argtypes = [sp, u8p, u8p, i32p, i32p, C.c_int64]
        L.kvo_swap_in.restype = C.c_int32
        L.kvo_swap_in.argtypes = [sp, u8p, u8p, i32p, i32p, C.c_int64]
        L.kvo_rotate.restype = C.c_int32
        L.kvo_rotate.argtypes = [sp, u8p, u8p, i32p, i32p, C.c_int64, i32p, i32p, C.c_int64, C.c_int32]
        L.kvo_rotate_mt.restype = C.c_int32
        L.kvo_rotate_mt.argtypes = [sp, u8p, u8p, i32p, i32p, C.c_int64, i32p, i32p, C.c_int64,
                                    C.c_int32, C.c_int32]
        _lib = L
    return _lib


def _ids(a):
    a = np.ascontiguousarray(np.asarray(a, dtype=np.int32))
    return a, a.ctypes.data_as(C.POINTER(C.c_int32))


class ByteOracle:
    def __init__(self, num_layers, block_size, kv_heads, head_dim,
                 num_gpu_blocks, num_host_blocks, host_layout=0, alloc=True, dev_layout=0):
        self.shape = _Shape(num_layers, block_size, kv_heads, head_dim,
                            num_gpu_blocks, num_host_blocks, host_layout, dev_layout)
        self.seg = lib().kvo_seg_bytes(C.byref(self.shape))
        self.blk = lib().kvo_blk_bytes(C.byref(self.shape))
        if alloc:
            self.G = np.zeros(num_gpu_blocks * self.blk, np.uint8)
            self.Hs = np.zeros(num_host_blocks * self.blk, np.uint8)

    def dev_off(self, l, kv, b):
        return lib().kvo_dev_off(C.byref(self.shape), l, kv, b)

    def host_off(self, h, l, kv):
        return lib().kvo_host_off(C.byref(self.shape), h, l, kv)

    def g_seg(self, l, kv, b):
        o = self.dev_off(l, kv, b)
        return self.G[o:o + self.seg]

    def h_seg(self, l, kv, h):
        o = self.host_off(h, l, kv)
        return self.Hs[o:o + self.seg]

    def g_block(self, b):
        """Logical content of device block b: bytes of all planes in (layer, K|V) order."""
        L = self.shape.num_layers
        return np.concatenate([self.g_seg(l, kv, b) for l in range(L) for kv in range(2)])

    def h_block(self, h):
        L = self.shape.num_layers
        return np.concatenate([self.h_seg(l, kv, h) for l in range(L) for kv in range(2)])

    def swap_out(self, gpu_ids, host_ids):
        if len(gpu_ids) != len(host_ids):
            return ERR_INVALID_ARG
        g, gp = _ids(gpu_ids)
        h, hp = _ids(host_ids)
        return lib().kvo_swap_out(C.byref(self.shape), self.G.ctypes.data, self.Hs.ctypes.data, gp, hp, len(g))

    def swap_in(self, host_ids, gpu_ids):
        if len(gpu_ids) != len(host_ids):
            return ERR_INVALID_ARG
        h, hp = _ids(host_ids)
        g, gp = _ids(gpu_ids)
        return lib().kvo_swap_in(C.byref(self.shape), self.G.ctypes.data, self.Hs.ctypes.data, hp, gp, len(g))

    def rotate(self, out_gpu, out_host, in_host, in_gpu, allow_overlap=False, threads=0):
        if len(out_gpu) != len(out_host) or len(in_host) != len(in_gpu):
            return ERR_INVALID_ARG
        og, ogp = _ids(out_gpu)
        oh, ohp = _ids(out_host)
        ih, ihp = _ids(in_host)
        ig, igp = _ids(in_gpu)
        if threads and threads > 0:
            return lib().kvo_rotate_mt(C.byref(self.shape), self.G.ctypes.data, self.Hs.ctypes.data,
                                       ogp, ohp, len(og), ihp, igp, len(ig), int(allow_overlap), threads)
        return lib().kvo_rotate(C.byref(self.shape), self.G.ctypes.data, self.Hs.ctypes.data,
                                ogp, ohp, len(og), ihp, igp, len(ig), int(allow_overlap))
