"""ctypes binding of ``libkvtestutil.so``: seeded pool fill and per-block digests on the GPU.

Input-making and result-checking helpers for tests and the bench.  They are not part of the
rotation path.  ``fill_blocks`` is the GPU twin of ``workload.block_words``.
"""
from __future__ import annotations

import ctypes as C

import numpy as np

from . import build as _build
from . import workload as W

_lib = None


def lib() -> C.CDLL:
    global _lib
    if _lib is None:
        _build.build()
        L = C.CDLL(_build.TESTUTIL_LIB)
        ll, vp = C.c_longlong, C.c_void_p
        L.kvt_fill_blocks.restype = C.c_int
        L.kvt_fill_blocks.argtypes = [vp, ll, ll, ll, C.c_int, vp, ll, ll, C.c_ulonglong, C.c_ulonglong, vp]
        L.kvt_checksum_blocks.restype = C.c_int
        L.kvt_checksum_blocks.argtypes = [vp, ll, ll, ll, C.c_int, vp, ll, ll, vp]
        L.kvt_wait_runs_out.restype = C.c_int
        L.kvt_wait_runs_out.argtypes = [C.c_ulonglong, vp]
        _lib = L
    return _lib


class Layout:
    """Address rule of a pool: address(block, plane) = base + block*blk_stride + plane*plane_stride."""

    def __init__(self, base: int, blk_stride: int, plane_stride: int, shape: W.KVShape):
        self.base, self.blk_stride, self.plane_stride, self.shape = base, blk_stride, plane_stride, shape

    @staticmethod
    def device(base: int, shape: W.KVShape, num_blocks: int, block_first: bool = False) -> "Layout":
        seg = 2 * shape.words_per_plane
        if block_first:
            return Layout(base, shape.block_bytes, seg, shape)
        return Layout(base, seg, num_blocks * seg, shape)

    @staticmethod
    def host(base: int, shape: W.KVShape, num_blocks: int, layer_first: bool = False) -> "Layout":
        seg = 2 * shape.words_per_plane
        if layer_first:
            return Layout(base, seg, num_blocks * seg, shape)
        return Layout(base, shape.block_bytes, seg, shape)


_lut_dev = {}


def _lut(device):
    import torch
    key = str(device)
    if key not in _lut_dev:
        _lut_dev[key] = torch.from_numpy(W.lut().view(np.int16).copy()).to(device)
    return _lut_dev[key]


def fill_blocks(lay: Layout, seed: int, pool: int, n: int, first_id: int = 0, ids=None, device="cuda:0") -> None:
    """Write the seeded content of ``n`` blocks (a run from ``first_id``, or the int32 CUDA tensor ``ids``)."""
    import torch
    s = lay.shape
    ids_ptr = ids.data_ptr() if ids is not None else None
    rc = lib().kvt_fill_blocks(lay.base, lay.blk_stride, lay.plane_stride, s.words_per_plane, 2 * s.num_layers,
                               ids_ptr, first_id, n, seed, pool, _lut(device).data_ptr())
    if rc != 0:
        raise RuntimeError(f"kvt_fill_blocks failed: {rc}")


def checksum_blocks(lay: Layout, n: int, first_id: int = 0, ids=None, device="cuda:0") -> np.ndarray:
    """Position-weighted 64-bit digests of ``n`` blocks, as a numpy uint64 array."""
    import torch
    s = lay.shape
    out = torch.empty(n, dtype=torch.int64, device=device)
    ids_ptr = ids.data_ptr() if ids is not None else None
    rc = lib().kvt_checksum_blocks(lay.base, lay.blk_stride, lay.plane_stride, s.words_per_plane,
                                   2 * s.num_layers, ids_ptr, first_id, n, out.data_ptr())
    if rc != 0:
        raise RuntimeError(f"kvt_checksum_blocks failed: {rc}")
    return out.cpu().numpy().view(np.uint64)


def checksum_words(words: np.ndarray) -> np.uint64:
    """The same digest on the CPU from a block's logical words (uint16, any shape)."""
    w = words.reshape(-1).astype(np.uint64)
    with np.errstate(over="ignore"):
        return (w * (np.uint64(2) * np.arange(len(w), dtype=np.uint64) + np.uint64(1))).sum(dtype=np.uint64)


def wait_runs_out(limit_ns: int, device="cuda:0"):
    """Run the kernels' bounded barrier wait on a barrier nothing completes.  Returns (gave_up, waited_ns)."""
    import torch
    out = torch.zeros(2, dtype=torch.int64, device=device)
    rc = lib().kvt_wait_runs_out(limit_ns, out.data_ptr())
    if rc != 0:
        raise RuntimeError(f"kvt_wait_runs_out failed: {rc}")
    r = out.cpu().numpy()
    return bool(r[0]), int(r[1])
