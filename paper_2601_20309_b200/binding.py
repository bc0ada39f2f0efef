"""ctypes binding of ``libduplexkv.so``: argument marshalling only.

Every function here has the name and the semantics of the C entry point it wraps (see
``include/duplexkv.h``); all data movement happens inside the CUDA library.  If the library
is missing it is built with nvcc; if that fails, importing raises: there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

from . import build as _build

KV_OK = 0
KV_ERR_INVALID_ARG = -1
KV_ERR_RANGE = -2
KV_ERR_DUP_DST = -3
KV_ERR_HAZARD = -4
KV_ERR_CUDA = -5
KV_ERR_TIMEOUT = -6
KV_ERR_NOMEM = -7
KV_ERR_UNSUPPORTED = -8

KV_HOST_BLOCK_FIRST = 0
KV_HOST_LAYER_FIRST = 1

KV_DEV_LAYER_FIRST = 0
KV_DEV_BLOCK_FIRST = 1

KV_PATH_AUTO = 0
KV_PATH_ZEROCOPY = 1
KV_PATH_STAGED = 2
KV_PATH_CE2D = 3
KV_PATH_NAIVE = 4
PATH_NAMES = {0: "auto", 1: "zerocopy", 2: "staged", 3: "ce2d", 4: "naive"}

KV_FLAG_ALLOW_OVERLAP = 1
KV_FLAG_LDST_KERNEL = 2
KV_FLAG_FUSED_ROTATE = 4
KV_FLAG_TIME_KERNELS = 8
KV_FLAG_DEBUG_BOUNDS = 16


class kv_pool_config_t(C.Structure):
    _fields_ = [("num_layers", C.c_int32), ("block_size", C.c_int32), ("kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("num_gpu_blocks", C.c_int64), ("num_host_blocks", C.c_int64),
                ("device_base", C.c_void_p), ("host_base", C.c_void_p), ("host_layout", C.c_int32),
                ("device_id", C.c_int32), ("stream_out", C.c_void_p), ("stream_in", C.c_void_p),
                ("path", C.c_int32), ("flags", C.c_int32), ("ctas_out", C.c_int32), ("ctas_in", C.c_int32),
                ("staging_bytes", C.c_int64), ("path_in", C.c_int32), ("ce_streams", C.c_int32),
                ("device_layout", C.c_int32), ("link_variant", C.c_int32)]


class kv_stats_t(C.Structure):
    _fields_ = [("bytes_out", C.c_int64), ("bytes_in", C.c_int64), ("calls_out", C.c_int64),
                ("calls_in", C.c_int64), ("kernel_launches", C.c_int64), ("ce_copies", C.c_int64),
                ("last_out_ms", C.c_double), ("last_in_ms", C.c_double), ("last_union_ms", C.c_double),
                ("last_path_out", C.c_int32), ("last_path_in", C.c_int32),
                ("device_status", C.c_uint32), ("pad_", C.c_int32),
                ("timed_kernel_ms", C.c_double), ("timed_kernel_bytes", C.c_int64), ("timed_kernels", C.c_int64),
                ("timed_kernel_exec_ms", C.c_double), ("last_in_offset_ms", C.c_double),
                ("requests_out", C.c_int64), ("requests_in", C.c_int64)]


class kv_link_probe_t(C.Structure):
    _fields_ = [("d2h_gbs", C.c_double), ("h2d_gbs", C.c_double), ("bi_d2h_gbs", C.c_double),
                ("bi_h2d_gbs", C.c_double), ("bi_sum_gbs", C.c_double), ("bytes", C.c_int64),
                ("reps", C.c_int32), ("pad_", C.c_int32)]


class kv_probe_spec_t(C.Structure):
    _fields_ = [("copy_bytes", C.c_int64), ("total_bytes", C.c_int64), ("span_bytes", C.c_int64),
                ("scattered", C.c_int32), ("rounds", C.c_int32),
                ("rows", C.c_int64), ("host_pitch", C.c_int64), ("dev_pitch", C.c_int64),
                ("slices", C.c_int64), ("host_slice_rows", C.c_int64)]


class kv_pool_shape_t(C.Structure):
    _fields_ = [("num_layers", C.c_int32), ("block_size", C.c_int32), ("kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("num_gpu_blocks", C.c_int64), ("num_host_blocks", C.c_int64), ("seg_bytes", C.c_int64),
                ("blk_bytes", C.c_int64)]


class kv_req_info_t(C.Structure):
    _fields_ = [("tokens", C.c_int64), ("num_blocks", C.c_int64), ("synced_blocks", C.c_int64),
                ("host_blocks", C.c_int64), ("dirty_blocks", C.c_int64), ("on_gpu", C.c_int32), ("pad_", C.c_int32)]


class kv_table_stats_t(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("eager_blocks", "eager_calls", "preempt_blocks_moved", "discarded_blocks",
                                         "resume_blocks_moved", "preempted_requests", "resumed_requests",
                                         "rotate_calls", "free_gpu_blocks", "free_host_blocks", "free_host_extents",
                                         "requests")]


class kv_plan_op_t(C.Structure):
    _fields_ = [("host_block", C.c_int64), ("first_position", C.c_int64), ("pitch_blocks", C.c_int64),
                ("rows", C.c_int32), ("blocks_per_row", C.c_int32), ("chunk", C.c_int32), ("slices", C.c_int32),
                ("slice_pitch_blocks", C.c_int64)]


EXPORTS = ["kv_pool_create", "kv_pool_destroy", "kv_pool_set_path", "kv_swap_out", "kv_swap_in", "kv_rotate", "kv_sync",
           "kv_gather_blocks", "kv_scatter_blocks", "kv_host_ptr", "kv_get_stats", "kv_last_error",
           "kv_seg_bytes", "kv_blk_bytes", "kv_path_for", "kv_probe_link", "kv_probe_link_ex",
           "kv_gather_blocks_static", "kv_pool_shape", "kv_pool_progress", "kv_stream_wait", "kv_plan_staged",
           "kv_table_create", "kv_table_create_dry", "kv_table_destroy", "kv_table_last_error", "kv_req_add",
           "kv_req_append", "kv_eager_rotate", "kv_req_rotate", "kv_req_preempt", "kv_req_resume", "kv_req_finish",
           "kv_req_info", "kv_req_blocks", "kv_table_get_stats", "kv_table_fail_pool_call",
           "kv_pool_set_wait_limit", "kv_pool_set_call_timing", "kv_completion_event", "kv_pool_set_ctas",
           "kv_debug_pair_in_bounds", "kv_rotate_req", "kv_debug_ring_shape"]

_lib = None


def lib() -> C.CDLL:
    """Load (building first if needed) the CUDA library.  Raises if it cannot be had."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.build()
    L = C.CDLL(path)
    i32p, vp, i64 = C.POINTER(C.c_int32), C.c_void_p, C.c_int64
    L.kv_pool_create.restype = C.c_int32
    L.kv_pool_create.argtypes = [C.POINTER(kv_pool_config_t), C.POINTER(vp)]
    L.kv_pool_destroy.restype = C.c_int32
    L.kv_pool_destroy.argtypes = [vp]
    L.kv_swap_out.restype = C.c_int32
    L.kv_swap_out.argtypes = [vp, i32p, i32p, i64]
    L.kv_swap_in.restype = C.c_int32
    L.kv_swap_in.argtypes = [vp, i32p, i32p, i64]
    L.kv_rotate.restype = C.c_int32
    L.kv_rotate.argtypes = [vp, i32p, i32p, i64, i32p, i32p, i64]
    L.kv_sync.restype = C.c_int32
    L.kv_sync.argtypes = [vp]
    L.kv_pool_set_path.restype = C.c_int32
    L.kv_pool_set_path.argtypes = [vp, C.c_int32, C.c_int32]
    L.kv_gather_blocks.restype = C.c_int32
    L.kv_gather_blocks.argtypes = [vp, i32p, i64, vp]
    L.kv_scatter_blocks.restype = C.c_int32
    L.kv_scatter_blocks.argtypes = [vp, vp, i32p, i64]
    L.kv_host_ptr.restype = C.c_int32
    L.kv_host_ptr.argtypes = [vp, C.POINTER(vp), C.POINTER(i64)]
    L.kv_get_stats.restype = C.c_int32
    L.kv_get_stats.argtypes = [vp, C.POINTER(kv_stats_t)]
    L.kv_last_error.restype = C.c_char_p
    L.kv_last_error.argtypes = [vp]
    L.kv_seg_bytes.restype = i64
    L.kv_seg_bytes.argtypes = [C.c_int32] * 3
    L.kv_blk_bytes.restype = i64
    L.kv_blk_bytes.argtypes = [C.c_int32] * 4
    L.kv_path_for.restype = C.c_int32
    L.kv_path_for.argtypes = [i64]
    L.kv_probe_link.restype = C.c_int32
    L.kv_probe_link.argtypes = [C.c_int32, i64, C.c_int32, C.POINTER(kv_link_probe_t)]
    i64p = C.POINTER(C.c_int64)
    L.kv_pool_shape.restype = C.c_int32
    L.kv_pool_shape.argtypes = [vp, C.POINTER(kv_pool_shape_t)]
    L.kv_plan_staged.restype = C.c_int32
    L.kv_plan_staged.argtypes = [i64, i64, C.c_int32, i32p, i64, C.POINTER(kv_plan_op_t), i64, i64p, i32p]
    L.kv_stream_wait.restype = C.c_int32
    L.kv_stream_wait.argtypes = [vp, vp, C.c_int32]
    L.kv_pool_progress.restype = C.c_int32
    L.kv_pool_progress.argtypes = [vp, i64p, i64p, i64p, i64p]
    L.kv_table_create.restype = C.c_int32
    L.kv_table_create.argtypes = [vp, C.POINTER(vp)]
    L.kv_table_create_dry.restype = C.c_int32
    L.kv_table_create_dry.argtypes = [i64, i64, C.c_int32, C.POINTER(vp)]
    L.kv_table_destroy.restype = C.c_int32
    L.kv_table_destroy.argtypes = [vp]
    L.kv_table_last_error.restype = C.c_char_p
    L.kv_table_last_error.argtypes = [vp]
    L.kv_req_add.restype = C.c_int32
    L.kv_req_add.argtypes = [vp, i64, i64]
    L.kv_req_append.restype = C.c_int32
    L.kv_req_append.argtypes = [vp, i64, i64]
    L.kv_eager_rotate.restype = C.c_int32
    L.kv_eager_rotate.argtypes = [vp, i64, i64p]
    L.kv_req_rotate.restype = C.c_int32
    L.kv_req_rotate.argtypes = [vp, i64p, i64, i64p, i64]
    for name in ("kv_req_preempt", "kv_req_resume", "kv_req_finish"):
        getattr(L, name).restype = C.c_int32
        getattr(L, name).argtypes = [vp, i64]
    L.kv_req_info.restype = C.c_int32
    L.kv_req_info.argtypes = [vp, i64, C.POINTER(kv_req_info_t)]
    L.kv_req_blocks.restype = C.c_int32
    L.kv_req_blocks.argtypes = [vp, i64, i32p, i32p, C.POINTER(C.c_uint8), i64]
    L.kv_table_get_stats.restype = C.c_int32
    L.kv_table_get_stats.argtypes = [vp, C.POINTER(kv_table_stats_t)]
    L.kv_completion_event.restype = C.c_int32
    L.kv_completion_event.argtypes = [vp, C.c_int32, C.POINTER(vp)]
    L.kv_pool_set_ctas.restype = C.c_int32
    L.kv_pool_set_ctas.argtypes = [vp, C.c_int32, C.c_int32]
    L.kv_debug_pair_in_bounds.restype = C.c_int32
    L.kv_debug_pair_in_bounds.argtypes = [C.c_int32] * 4
    L.kv_debug_ring_shape.restype = C.c_int32
    L.kv_debug_ring_shape.argtypes = [C.c_int64, C.c_int32, C.c_int32] + [C.POINTER(C.c_int32)] * 5
    L.kv_rotate_req.restype = C.c_int32
    L.kv_rotate_req.argtypes = [vp, i32p, i32p, i64, C.POINTER(C.c_int64), i64, i32p, i32p, i64, C.POINTER(C.c_int64), i64]
    L.kv_pool_set_call_timing.restype = C.c_int32
    L.kv_pool_set_call_timing.argtypes = [vp, C.c_int32]
    L.kv_pool_set_wait_limit.restype = C.c_int32
    L.kv_pool_set_wait_limit.argtypes = [vp, C.c_uint32, C.c_uint64]
    L.kv_table_fail_pool_call.restype = C.c_int32
    L.kv_table_fail_pool_call.argtypes = [vp, i64, C.c_int32]
    L.kv_gather_blocks_static.restype = C.c_int32
    L.kv_gather_blocks_static.argtypes = [vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, i64, i32p, i64, vp, vp]
    L.kv_probe_link_ex.restype = C.c_int32
    L.kv_probe_link_ex.argtypes = [C.c_int32, C.POINTER(kv_probe_spec_t), C.POINTER(kv_link_probe_t)]
    _lib = L
    return L


def lib_path() -> str:
    return _build.LIB


class KVError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"duplexkv error {code}: {msg}")
        self.code = code


def _ids(a) -> tuple:
    arr = np.ascontiguousarray(np.asarray(a, dtype=np.int32))
    return arr, arr.ctypes.data_as(C.POINTER(C.c_int32))


def kv_seg_bytes(block_size: int, kv_heads: int, head_dim: int) -> int:
    return lib().kv_seg_bytes(block_size, kv_heads, head_dim)


def kv_blk_bytes(num_layers: int, block_size: int, kv_heads: int, head_dim: int) -> int:
    return lib().kv_blk_bytes(num_layers, block_size, kv_heads, head_dim)


def kv_debug_ring_shape(segment_bytes: int, over_link: bool = False, link_variant: int = 0, check: bool = True):
    """(rc, dict): item bytes, stage bytes, stages, loads ahead and issuing warps of the bulk kernel for this segment size."""
    v = [C.c_int32() for _ in range(5)]
    rc = lib().kv_debug_ring_shape(segment_bytes, int(over_link), link_variant, *[C.byref(x) for x in v])
    if check and rc != KV_OK:
        raise KVError(rc, lib().kv_last_error(None).decode())
    return rc, dict(zip(("item_bytes", "stage_bytes", "stages", "ahead", "warps"), (x.value for x in v)))


def kv_debug_pair_in_bounds(src_id: int, dst_id: int, src_blocks: int, dst_blocks: int) -> bool:
    return bool(lib().kv_debug_pair_in_bounds(src_id, dst_id, src_blocks, dst_blocks))


def kv_path_for(blk_bytes: int) -> int:
    return lib().kv_path_for(blk_bytes)


def kv_probe_link(device_id: int = 0, nbytes: int = 256 << 20, reps: int = 4) -> dict:
    out = kv_link_probe_t()
    rc = lib().kv_probe_link(device_id, nbytes, reps, C.byref(out))
    if rc != KV_OK:
        raise KVError(rc, lib().kv_last_error(None).decode())
    return {k: getattr(out, k) for k, _ in kv_link_probe_t._fields_ if k != "pad_"}


def kv_probe_link_ex(device_id: int, copy_bytes: int, total_bytes: int, span_bytes: int,
                     scattered: bool = False, rounds: int = 3, rows: int = 1, host_pitch: int = 0,
                     dev_pitch: int = 0, slices: int = 1, host_slice_rows: int = 0) -> dict:
    spec = kv_probe_spec_t(copy_bytes, total_bytes, span_bytes, int(scattered), rounds, rows, host_pitch, dev_pitch,
                           slices, host_slice_rows)
    out = kv_link_probe_t()
    rc = lib().kv_probe_link_ex(device_id, C.byref(spec), C.byref(out))
    if rc != KV_OK:
        raise KVError(rc, lib().kv_last_error(None).decode())
    return {k: getattr(out, k) for k, _ in kv_link_probe_t._fields_ if k != "pad_"}


def kv_plan_staged(blk_bytes: int, half_blocks: int, direction: int, host_ids):
    """(ops, order): the transfers the STAGED path would make for these host ids, as a list of dicts in
    issue order, and the staging order as a numpy array of indices into ``host_ids``.  Needs no GPU."""
    h, hp = _ids(host_ids)
    n_ops = C.c_int64()
    ops = (kv_plan_op_t * max(1, len(h)))()
    order = np.empty(len(h), np.int32)
    rc = lib().kv_plan_staged(blk_bytes, half_blocks, direction, hp, len(h), ops, len(ops), C.byref(n_ops),
                              order.ctypes.data_as(C.POINTER(C.c_int32)))
    if rc != KV_OK:
        raise KVError(rc, lib().kv_last_error(None).decode())
    fields = [k for k, _ in kv_plan_op_t._fields_ if k != "pad_"]
    return [{k: getattr(ops[a], k) for k in fields} for a in range(n_ops.value)], order


KV_STATIC_MAX_BLOCKS = 8192


def kv_gather_blocks_static(device_base: int, num_layers: int, block_size: int, kv_heads: int, head_dim: int,
                            num_gpu_blocks: int, gpu_ids, dst_device: int, stream: Optional[int] = None,
                            check: bool = True) -> int:
    """The allocation-free gather (no pool needed): see ``kv_gather_blocks_static`` in the header.
    Synchronous; one call at a time per device."""
    g, gp = _ids(gpu_ids)
    rc = lib().kv_gather_blocks_static(device_base, num_layers, block_size, kv_heads, head_dim, num_gpu_blocks,
                                       gp, len(g), dst_device, stream)
    if check and rc != KV_OK:
        raise KVError(rc, lib().kv_last_error(None).decode())
    return rc


class KVPool:
    """Thin owner of a ``kv_pool_t*``.  Methods return the C status code unchanged unless
    ``check=True`` (default), in which case a negative status raises ``KVError``."""

    def __init__(self, num_layers: int, block_size: int, kv_heads: int, head_dim: int,
                 num_gpu_blocks: int, num_host_blocks: int, device_base: int, *,
                 host_base: Optional[int] = None, host_layout: int = KV_HOST_BLOCK_FIRST,
                 device_id: int = 0, stream_out: Optional[int] = None, stream_in: Optional[int] = None,
                 path: int = KV_PATH_AUTO, flags: int = 0, ctas_out: int = 0, ctas_in: int = 0,
                 staging_bytes: int = 0, path_in: int = KV_PATH_AUTO, ce_streams: int = 0,
                 device_layout: int = KV_DEV_LAYER_FIRST, link_variant: int = 0):
        self.cfg = kv_pool_config_t(num_layers, block_size, kv_heads, head_dim, num_gpu_blocks,
                                    num_host_blocks, device_base, host_base, host_layout, device_id,
                                    stream_out, stream_in, path, flags, ctas_out, ctas_in, staging_bytes,
                                    path_in, ce_streams, device_layout, link_variant)
        self._h = C.c_void_p()
        rc = lib().kv_pool_create(C.byref(self.cfg), C.byref(self._h))
        if rc != KV_OK:
            raise KVError(rc, lib().kv_last_error(None).decode())
        self.seg = kv_seg_bytes(block_size, kv_heads, head_dim)
        self.blk = kv_blk_bytes(num_layers, block_size, kv_heads, head_dim)

    # -- lifetime
    def destroy(self) -> None:
        if self._h:
            lib().kv_pool_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.destroy()

    def _ret(self, rc: int, check: bool) -> int:
        if check and rc != KV_OK:
            raise KVError(rc, self.kv_last_error())
        return rc

    # -- the C entry points
    def kv_swap_out(self, gpu_ids, host_ids, check: bool = True) -> int:
        g, gp = _ids(gpu_ids)
        h, hp = _ids(host_ids)
        if len(g) != len(h):
            raise ValueError("gpu_ids and host_ids differ in length")
        return self._ret(lib().kv_swap_out(self._h, gp, hp, len(g)), check)

    def kv_swap_in(self, host_ids, gpu_ids, check: bool = True) -> int:
        h, hp = _ids(host_ids)
        g, gp = _ids(gpu_ids)
        if len(g) != len(h):
            raise ValueError("gpu_ids and host_ids differ in length")
        return self._ret(lib().kv_swap_in(self._h, hp, gp, len(g)), check)

    def kv_rotate(self, out_gpu, out_host, in_host, in_gpu, check: bool = True) -> int:
        og, ogp = _ids(out_gpu)
        oh, ohp = _ids(out_host)
        ih, ihp = _ids(in_host)
        ig, igp = _ids(in_gpu)
        if len(og) != len(oh) or len(ih) != len(ig):
            raise ValueError("paired lists differ in length")
        return self._ret(lib().kv_rotate(self._h, ogp, ohp, len(og), ihp, igp, len(ig)), check)

    def kv_rotate_raw(self, ogp, ohp, n_out, ihp, igp, n_in) -> int:
        """Same call with pre-marshalled ``POINTER(c_int32)`` arguments (for timing loops)."""
        return lib().kv_rotate(self._h, ogp, ohp, n_out, ihp, igp, n_in)

    def kv_pool_set_path(self, path_out: int, path_in: int, check: bool = True) -> int:
        return self._ret(lib().kv_pool_set_path(self._h, path_out, path_in), check)

    def kv_completion_event(self, direction: int) -> Optional[int]:
        """The pool-owned ``cudaEvent_t`` (as an integer handle) of the latest call of ``direction``, or None."""
        ev = C.c_void_p()
        self._ret(lib().kv_completion_event(self._h, direction, C.byref(ev)), True)
        return ev.value

    def kv_pool_set_ctas(self, ctas_out: int, ctas_in: int, check: bool = True) -> int:
        return self._ret(lib().kv_pool_set_ctas(self._h, ctas_out, ctas_in), check)

    def kv_rotate_req(self, out_gpu, out_host, out_req_offsets, in_host, in_gpu, in_req_offsets, check: bool = True) -> int:
        og, ogp = _ids(out_gpu)
        oh, ohp = _ids(out_host)
        ih, ihp = _ids(in_host)
        ig, igp = _ids(in_gpu)
        oo = np.ascontiguousarray(np.asarray(out_req_offsets, dtype=np.int64))
        io = np.ascontiguousarray(np.asarray(in_req_offsets, dtype=np.int64))
        i64p = C.POINTER(C.c_int64)
        return self._ret(lib().kv_rotate_req(self._h, ogp, ohp, len(og), oo.ctypes.data_as(i64p) if len(oo) else None,
                                             max(0, len(oo) - 1), ihp, igp, len(ig),
                                             io.ctypes.data_as(i64p) if len(io) else None, max(0, len(io) - 1)), check)

    def kv_pool_set_call_timing(self, on: bool, check: bool = True) -> int:
        return self._ret(lib().kv_pool_set_call_timing(self._h, int(on)), check)

    def kv_pool_set_wait_limit(self, polls: int, ns: int, check: bool = True) -> int:
        return self._ret(lib().kv_pool_set_wait_limit(self._h, polls, ns), check)

    def kv_sync(self, check: bool = True) -> int:
        return self._ret(lib().kv_sync(self._h), check)

    def kv_gather_blocks(self, gpu_ids, dst_device: int, check: bool = True) -> int:
        g, gp = _ids(gpu_ids)
        return self._ret(lib().kv_gather_blocks(self._h, gp, len(g), dst_device), check)

    def kv_scatter_blocks(self, src_device: int, gpu_ids, check: bool = True) -> int:
        g, gp = _ids(gpu_ids)
        return self._ret(lib().kv_scatter_blocks(self._h, src_device, gp, len(g)), check)

    def kv_host_ptr(self) -> tuple:
        base, nbytes = C.c_void_p(), C.c_int64()
        self._ret(lib().kv_host_ptr(self._h, C.byref(base), C.byref(nbytes)), True)
        return base.value, nbytes.value

    def kv_get_stats(self) -> dict:
        st = kv_stats_t()
        self._ret(lib().kv_get_stats(self._h, C.byref(st)), True)
        return {k: getattr(st, k) for k, _ in kv_stats_t._fields_ if k != "pad_"}

    def kv_last_error(self) -> str:
        return lib().kv_last_error(self._h).decode()

    def kv_stream_wait(self, stream: Optional[int], directions: int = 3, check: bool = True) -> int:
        return self._ret(lib().kv_stream_wait(self._h, stream, directions), check)

    def kv_pool_progress(self) -> dict:
        v = [C.c_int64() for _ in range(4)]
        self._ret(lib().kv_pool_progress(self._h, *[C.byref(x) for x in v]), True)
        return dict(zip(("out_issued", "out_done", "in_issued", "in_done"), (x.value for x in v)))

    def kv_pool_shape(self) -> dict:
        sh = kv_pool_shape_t()
        self._ret(lib().kv_pool_shape(self._h, C.byref(sh)), True)
        return {k: getattr(sh, k) for k, _ in kv_pool_shape_t._fields_}

    # -- convenience for verification (no data path): the host pool as a numpy view
    def host_array(self) -> np.ndarray:
        base, nbytes = self.kv_host_ptr()
        buf = (C.c_uint8 * nbytes).from_address(base)
        return np.frombuffer(buf, dtype=np.uint8)


class KVTable:
    """Thin owner of a ``kv_table_t*`` (block table with eager block rotation).  ``pool`` is a ``KVPool`` or,
    for bookkeeping without a GPU, ``None`` with the sizes given.  Methods return the C status unless
    ``check`` (default) turns a negative one into ``KVError``."""

    def __init__(self, pool: Optional[KVPool] = None, *, num_gpu_blocks: int = 0, num_host_blocks: int = 0,
                 block_size: int = 0):
        self._h = C.c_void_p()
        self.pool = pool
        if pool is not None:
            rc = lib().kv_table_create(pool._h, C.byref(self._h))
        else:
            rc = lib().kv_table_create_dry(num_gpu_blocks, num_host_blocks, block_size, C.byref(self._h))
        if rc != KV_OK:
            raise KVError(rc, "kv_table_create failed")

    def destroy(self) -> None:
        if self._h:
            lib().kv_table_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

    def _ret(self, rc: int, check: bool) -> int:
        if check and rc != KV_OK:
            raise KVError(rc, lib().kv_table_last_error(self._h).decode())
        return rc

    def kv_req_add(self, req: int, tokens: int, check: bool = True) -> int:
        return self._ret(lib().kv_req_add(self._h, req, tokens), check)

    def kv_req_append(self, req: int, new_tokens: int, check: bool = True) -> int:
        return self._ret(lib().kv_req_append(self._h, req, new_tokens), check)

    def kv_eager_rotate(self, max_blocks: int) -> int:
        n = C.c_int64()
        self._ret(lib().kv_eager_rotate(self._h, max_blocks, C.byref(n)), True)
        return n.value

    def kv_req_rotate(self, preempt: Sequence[int], resume: Sequence[int], check: bool = True) -> int:
        p = (C.c_int64 * len(preempt))(*preempt)
        r = (C.c_int64 * len(resume))(*resume)
        return self._ret(lib().kv_req_rotate(self._h, p, len(preempt), r, len(resume)), check)

    def kv_req_preempt(self, req: int, check: bool = True) -> int:
        return self._ret(lib().kv_req_preempt(self._h, req), check)

    def kv_req_resume(self, req: int, check: bool = True) -> int:
        return self._ret(lib().kv_req_resume(self._h, req), check)

    def kv_req_finish(self, req: int, check: bool = True) -> int:
        return self._ret(lib().kv_req_finish(self._h, req), check)

    def kv_req_info(self, req: int) -> dict:
        out = kv_req_info_t()
        self._ret(lib().kv_req_info(self._h, req, C.byref(out)), True)
        return {k: getattr(out, k) for k, _ in kv_req_info_t._fields_ if k != "pad_"}

    def kv_req_blocks(self, req: int):
        """(device ids, host ids, host_valid) as numpy arrays; -1 where a block has no id."""
        n = self.kv_req_info(req)["num_blocks"]
        g, h, v = np.empty(n, np.int32), np.empty(n, np.int32), np.empty(n, np.uint8)
        i32p = C.POINTER(C.c_int32)
        self._ret(lib().kv_req_blocks(self._h, req, g.ctypes.data_as(i32p), h.ctypes.data_as(i32p),
                                      v.ctypes.data_as(C.POINTER(C.c_uint8)), n), True)
        return g, h, v.astype(bool)

    def kv_table_fail_pool_call(self, after_calls: int, code: int) -> int:
        return self._ret(lib().kv_table_fail_pool_call(self._h, after_calls, code), True)

    def kv_table_get_stats(self) -> dict:
        out = kv_table_stats_t()
        self._ret(lib().kv_table_get_stats(self._h, C.byref(out)), True)
        return {k: getattr(out, k) for k, _ in kv_table_stats_t._fields_}
