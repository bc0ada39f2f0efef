#!/usr/bin/env python
"""Benchmark of the KV-block rotation path.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one full-duplex rotation (swap-out of 16 requests' blocks and swap-in of 16 others in one
kv_rotate call, then kv_sync) on the Llama-3-8B-shaped workload: 32 layers, 8 KV heads, head_dim 128,
block_size 16, bf16; 60 GB device pool, 120 GB pinned host pool (shrunk only if the box cannot pin that
much), 64 requests with lognormal lengths (median 1k tokens, max 8k), scattered block tables.

Metric: aggregate GB/s (bytes swapped out + bytes swapped in, per second).
  value  device time from CUDA events recorded by the library on its own two streams.
  e2e    wall time of the same K calls made with host id lists through the C ABI (validation,
         descriptor upload, launches, both transfers, sync).
Denominators are measured in the same process: the host link by a pinned copy-engine probe
(kv_probe_link), HBM from MEASURED_PEAKS.json.  Multi-GPU runs are independent replicas (one pool,
one host link per GPU; the method has no exchange step).
"""
from __future__ import annotations

import argparse
import ctypes as C
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2601_20309_b200 import metrics as M          # noqa: E402
from paper_2601_20309_b200 import workload as W         # noqa: E402

CPU_SAMPLE_BLOCKS = 768      # blocks per direction of the rotation that the CPU oracle is timed on, in both arms
METRIC = "full-duplex KV swap GB/s (out+in)"
UNIT = "GB/s"
WORKLOAD = ("config2 llama-3-8b-shaped KV (32 layers, 8 kv heads, head_dim 128, block 16, bf16): "
            "paired rotate of %d requests each way per step")
# DRAM traffic of one pack / unpack launch, from the ncu capture of an 88-block (184.55 MB) launch on the
# --small case (retaken after the kernel's last change: same figures): dram__bytes_read.sum = 1.0001 x
# payload (no byte read twice); dram__bytes_write.sum = payload - 45 to 50 MB, the lines still in L2 when the
# kernel ends.  Reads scale with the payload, the L2 tail does not.
def ncu_traffic_per_launch(payload_bytes: float) -> float:
    return 1.00005 * payload_bytes + max(0.0, payload_bytes - 48.5e6)


# ------------------------------------------------------------------------------------------------ helpers

def mem_available_bytes() -> int:
    try:
        with open("/proc/meminfo") as f:
            for line in f:
                if line.startswith("MemAvailable:"):
                    return int(line.split()[1]) * 1024
    except OSError:
        pass
    return 0


def measured_peaks() -> dict:
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi polled every 200 ms while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "200",
                 "-i", str(self.index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def ptr(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_int32))


def compact_lists(rot: W.Rotation):
    """The same rotation with ids renumbered densely (order preserved), so that the CPU oracle can run
    it in pools just large enough to hold the blocks it names."""
    def renum(a, b):
        u, inv = np.unique(np.concatenate([a, b]), return_inverse=True)
        return inv[:len(a)].astype(np.int32), inv[len(a):].astype(np.int32), len(u)
    og, ig, nbg = renum(rot.out_gpu, rot.in_gpu)
    oh, ih, nbh = renum(rot.out_host, rot.in_host)
    return og, oh, ih, ig, nbg, nbh


def time_oracle(shape: W.KVShape, rot: W.Rotation, max_blocks: int, threads: int, reps: int, warmup: int = 1):
    """Time the CPU oracle's rotate on the first ``max_blocks`` pairs of each direction."""
    from oracle.kv_oracle import ByteOracle
    sub = W.Rotation(rot.out_gpu[:max_blocks], rot.out_host[:max_blocks], rot.in_host[:max_blocks],
                     rot.in_gpu[:max_blocks], np.zeros(1), np.zeros(1))
    og, oh, ih, ig, nbg, nbh = compact_lists(sub)
    o = ByteOracle(shape.num_layers, shape.block_size, shape.kv_heads, shape.head_dim, nbg, nbh)
    o.G[:] = 1                    # touch every page before timing
    o.Hs[:] = 2
    nbytes = (len(og) + len(ig)) * shape.block_bytes
    times = []
    for it in range(warmup + reps):
        t0 = time.perf_counter()
        rc = o.rotate(og, oh, ih, ig, threads=threads)
        dt = time.perf_counter() - t0
        assert rc == 0
        if it >= warmup:
            times.append(dt)
    return nbytes, times, f"first {len(og)} out + {len(ig)} in blocks of the rotation ({nbytes / 1e9:.2f} GB per step)"


def overlap_of(windows) -> dict:
    """How much of each timed step had both directions in flight, from the library's per-direction
    start / end events (swap-out window [0, out], swap-in window [off, off + in])."""
    fr = []
    for out_ms, off, in_ms in windows:
        lo, hi = max(0.0, off), min(out_ms, off + in_ms)
        union = max(out_ms, off + in_ms) - min(0.0, off)
        fr.append(max(0.0, hi - lo) / union if union > 0 else 0.0)
    return {"both_in_flight_share_of_step": float(np.mean(fr)), "min": float(np.min(fr)), "max": float(np.max(fr)),
            "source": "per-direction start/end events on the library's streams (no nsys on the image)"}


def write_trace(path: str, windows) -> None:
    """Chrome-trace (about://tracing, Perfetto) file of the timed steps: one track per direction."""
    ev, t = [], 0.0
    for k, (out_ms, off, in_ms) in enumerate(windows):
        base = t - min(0.0, off) * 1e3
        ev.append({"name": f"swap-out step {k}", "ph": "X", "pid": 0, "tid": 0, "ts": base, "dur": out_ms * 1e3})
        ev.append({"name": f"swap-in step {k}", "ph": "X", "pid": 0, "tid": 1, "ts": base + off * 1e3, "dur": in_ms * 1e3})
        t = base + max(out_ms, off + in_ms) * 1e3 + 50.0
    meta = [{"name": "thread_name", "ph": "M", "pid": 0, "tid": 0, "args": {"name": "device to host (swap-out stream)"}},
            {"name": "thread_name", "ph": "M", "pid": 0, "tid": 1, "args": {"name": "host to device (swap-in stream)"}}]
    with open(path, "w") as f:
        json.dump({"traceEvents": meta + ev, "displayTimeUnit": "ms"}, f)


# ------------------------------------------------------------------------------------------------ arms

def run_reference(args, rank: int) -> None:
    """The CPU oracle, as it stands, on the host cores: a deliberately plain program."""
    if rank != 0:
        return
    w = W.config2_8b()
    threads = os.cpu_count() or 1
    nbytes, times, sample = time_oracle(w.shape, w.steps[0], CPU_SAMPLE_BLOCKS, threads, reps=args.steps, warmup=args.warmup)
    ms = float(np.mean(times)) * 1e3
    val = M.gbs(nbytes, ms)
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u16", "data": "synthetic",
            "config": {"workload": WORKLOAD % 16, "cpu_sample": sample},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_ours(args, rank: int, local_rank: int, world: int) -> None:
    import torch
    from paper_2601_20309_b200 import binding as B
    from paper_2601_20309_b200 import poolfill as F

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the rotation path has no CPU fallback")
    if local_rank >= torch.cuda.device_count():
        raise SystemExit(f"bench.py: rank {rank} wants cuda:{local_rank} but the node has {torch.cuda.device_count()} GPUs")
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    # the other workloads in the line are measured at N = 1: with more ranks every GPU of the job would be
    # held while rank 0 runs them
    args.quick = args.quick or world > 1
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device(dev))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def reduce(x: float, op: str) -> float:
        return M.reduce_over_ranks(x, op, dist, dev)

    # ---- host-link denominators, measured in this process (again after the timed region)
    probe = B.kv_probe_link(local_rank, 256 << 20, 4)
    peaks = measured_peaks()

    # ---- workload: config 2 at full size; the host pool shrinks only if the box cannot pin 120 GB per rank
    shape = W.SHAPE_8B
    nb_gpu = W.blocks_for_bytes(shape, 60e9)
    nb_host = W.blocks_for_bytes(shape, 120e9)
    avail = mem_available_bytes()
    budget = int(0.70 * avail / max(1, world)) if avail else nb_host * shape.block_bytes
    shrunk = False
    if nb_host * shape.block_bytes > budget:
        nb_host = max(8192, budget // shape.block_bytes)
        shrunk = True
    if args.small:
        nb_gpu, nb_host, shrunk = W.blocks_for_bytes(shape, 6e9), W.blocks_for_bytes(shape, 8e9), True
        w = W.config2_8b(nb_gpu=nb_gpu, nb_host=nb_host, n_req=16, n_rot=4)
    else:
        w = W.config2_8b(nb_gpu=nb_gpu, nb_host=nb_host)
    rot = w.steps[0]
    bytes_out, bytes_in = rot.n_out * shape.block_bytes, rot.n_in * shape.block_bytes

    device_pool = torch.empty(nb_gpu * shape.block_bytes, dtype=torch.uint8, device=dev)
    t0 = time.perf_counter()
    pool = B.KVPool(shape.num_layers, shape.block_size, shape.kv_heads, shape.head_dim, nb_gpu, nb_host,
                    device_pool.data_ptr(), device_id=local_rank, path=args.path,
                    flags=args.flags | B.KV_FLAG_TIME_KERNELS, ctas_out=args.ctas, ctas_in=args.ctas,
                    staging_bytes=args.staging_mib << 20, link_variant=args.link_variant)
    pin_s = time.perf_counter() - t0
    host_base, host_bytes = pool.kv_host_ptr()
    # seeded content in both pools (GPU twin of the CPU generator; verified against it in the tests);
    # mapped pinned memory has the same address on the device (unified addressing)
    F.fill_blocks(F.Layout.device(device_pool.data_ptr(), shape, nb_gpu), w.seed, W.POOL_GPU, nb_gpu, device=dev)
    F.fill_blocks(F.Layout.host(host_base, shape, nb_host), w.seed, W.POOL_HOST, nb_host, device=dev)

    og, oh, ih, ig = (np.ascontiguousarray(x, np.int32) for x in (rot.out_gpu, rot.out_host, rot.in_host, rot.in_gpu))
    args_raw = (ptr(og), ptr(oh), len(og), ptr(ih), ptr(ig), len(ig))

    issue_s = []                        # host time inside kv_rotate (validation, planning, launches, transfers queued)

    def step():
        t_call = time.perf_counter()
        rc = pool.kv_rotate_raw(*args_raw)
        issue_s.append(time.perf_counter() - t_call)
        if rc != 0:
            raise RuntimeError(f"kv_rotate failed: {rc} {pool.kv_last_error()}")
        pool.kv_sync()

    for _ in range(args.warmup):
        step()
    st0 = pool.kv_get_stats()
    sampler = ClockSampler(local_rank)
    sampler.start()
    barrier()
    dev_ms, windows = [], []
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
        s_ = pool.kv_get_stats()
        dev_ms.append(s_["last_union_ms"])
        windows.append((s_["last_out_ms"], s_["last_in_offset_ms"], s_["last_in_ms"]))
    barrier()
    wall_s = time.perf_counter() - t0
    clocks = sampler.stop()
    st = pool.kv_get_stats()
    launches = st["kernel_launches"] - st0["kernel_launches"]
    ce_copies = st["ce_copies"] - st0["ce_copies"]
    k_ms = st["timed_kernel_ms"] - st0["timed_kernel_ms"]
    k_bytes = st["timed_kernel_bytes"] - st0["timed_kernel_bytes"]
    k_n = st["timed_kernels"] - st0["timed_kernels"]
    k_exec_ms = st["timed_kernel_exec_ms"] - st0["timed_kernel_exec_ms"]

    if args.trace and rank == 0:
        write_trace(args.trace, windows)
    dev_total_ms = reduce(float(np.sum(dev_ms)), "max")
    wall_total_s = reduce(wall_s, "max")
    job_bytes = reduce(float(bytes_out + bytes_in), "sum") * args.steps
    value = M.gbs(job_bytes, dev_total_ms)
    e2e_value = job_bytes / wall_total_s / 1e9

    extra = {}
    if rank == 0:
        def timed(fn, reps=3):
            ts = []
            for _ in range(reps):
                fn()
                pool.kv_sync()
                ts.append(pool.kv_get_stats()["last_union_ms"])
            return min(ts)

        probe2 = B.kv_probe_link(local_rank, 256 << 20, 4)
        # ---- every path on the same lists: each direction alone ("u") and both at once ("b"),
        #      the conventions of the paper's bandwidth table
        paths = {}
        path_list = [("staged", B.KV_PATH_STAGED), ("zerocopy", B.KV_PATH_ZEROCOPY), ("ce2d", B.KV_PATH_CE2D)]
        if not args.quick:
            path_list.append(("naive", B.KV_PATH_NAIVE))
        for name, pid in path_list:
            pool.kv_pool_set_path(pid, pid)
            reps = 1 if name == "naive" else 3
            # the per-segment path is measured on the first 256 blocks of each list (16 384 transfers each way)
            cut = 256 if name == "naive" else None
            a = (og[:cut], oh[:cut], ih[:cut], ig[:cut])
            bo, bi_ = len(a[0]) * shape.block_bytes, len(a[3]) * shape.block_bytes
            t_o = timed(lambda: pool.kv_swap_out(a[0], a[1]), reps)
            t_i = timed(lambda: pool.kv_swap_in(a[2], a[3]), reps)
            t_b = timed(lambda: pool.kv_rotate(*a), reps)
            paths[name] = {"out_u_gbs": M.gbs(bo, t_o), "in_u_gbs": M.gbs(bi_, t_i), "both_b_gbs": M.gbs(bo + bi_, t_b),
                           "e2e_ms_serial_u": t_o + t_i, "e2e_ms_concurrent_b": t_b, "blocks_each_way": len(a[0])}
        pool.kv_pool_set_path(args.path, args.path)
        # ---- the same payload with neighbouring host ids (what a run-based host allocator would hand out)
        oh_c = np.arange(len(og), dtype=np.int32)
        ih_c = np.arange(nb_host - len(ig), nb_host, dtype=np.int32)
        t_c = timed(lambda: pool.kv_rotate(og, oh_c, ih_c, ig))
        contiguous_host = M.gbs(bytes_out + bytes_in, t_c)
        F.fill_blocks(F.Layout.host(host_base, shape, nb_host), w.seed, W.POOL_HOST, len(og), device=dev)   # restore what it overwrote
        # ---- the same 16 + 16 requests through the block table (run-based host ids, eager block rotation)
        table = B.KVTable(pool)
        len_a = np.diff(rot.out_req_offsets).astype(int)
        len_b = np.diff(rot.in_req_offsets).astype(int)
        ids_a, ids_b = list(range(len(len_a))), list(range(100, 100 + len(len_b)))
        for rid, nb in zip(ids_a + ids_b, list(len_a) + list(len_b)):
            table.kv_req_add(rid, int(nb) * shape.block_size - 5)          # last block partly filled
        table.kv_req_rotate(ids_b, [])                                      # B leaves the GPU: everything is sent
        pool.kv_sync()

        def table_rotate(pre, res):
            s0, p0 = table.kv_table_get_stats(), pool.kv_get_stats()
            table.kv_req_rotate(pre, res)
            pool.kv_sync()
            s1, p1 = table.kv_table_get_stats(), pool.kv_get_stats()
            nbytes = (p1["bytes_out"] - p0["bytes_out"]) + (p1["bytes_in"] - p0["bytes_in"])
            return {"ms": p1["last_union_ms"], "gbs": M.gbs(nbytes, p1["last_union_ms"]),
                    "blocks_out": s1["preempt_blocks_moved"] - s0["preempt_blocks_moved"],
                    "blocks_discarded": s1["discarded_blocks"] - s0["discarded_blocks"],
                    "blocks_in": s1["resume_blocks_moved"] - s0["resume_blocks_moved"]}
        tb = {}
        tb["rotate_nothing_copied_beforehand"] = table_rotate(ids_a, ids_b)    # A out (all blocks), B in
        tb["rotate_back_host_copies_still_valid"] = table_rotate(ids_b, ids_a)  # B out (nothing to send), A in
        for rid in ids_a:
            table.kv_req_append(rid, 1)                                        # A generated a token each
        tb["rotate_after_one_token_each"] = table_rotate(ids_a, ids_b)          # A out (one dirty block each), B in
        table.destroy()
        # ---- single swaps of the median-length and the longest request
        singles = {}
        for key, which in (("single_out", "out"), ("single_in", "in")):
            for k, (a, b) in w.extra[key].items():
                t = timed((lambda a=a, b=b: pool.kv_swap_out(a, b)) if which == "out" else (lambda a=a, b=b: pool.kv_swap_in(a, b)))
                singles[f"{which}_{k}"] = {"blocks": len(a), "gbs": M.gbs(len(a) * shape.block_bytes, t), "ms": t}
        # ---- per-request rotate latency: one request out + one in per call, call entry to completion, host
        #      clock around the C-ABI calls; all 64 requests (32 pairs), one warm-up pass, then 5 timed passes
        pair_raw = []
        for r in w.extra["pairs"]:
            a = tuple(np.ascontiguousarray(x, np.int32) for x in (r.out_gpu, r.out_host, r.in_host, r.in_gpu))
            pair_raw.append((a, (ptr(a[0]), ptr(a[1]), len(a[0]), ptr(a[2]), ptr(a[3]), len(a[3]))))
        lat_us, lat_blocks, lat_paths = [], [], {}
        for rep in range(6):
            if rep == 1:
                pool.kv_pool_set_call_timing(False)     # timed by the host clock here: no per-call start events
            for a, raw in pair_raw:
                t1 = time.perf_counter()
                pool.kv_rotate_raw(*raw)
                pool.kv_sync()
                dt = (time.perf_counter() - t1) * 1e6
                if rep:
                    lat_us.append(dt)
                    lat_blocks.append(len(a[0]) + len(a[3]))
                else:
                    nm = B.PATH_NAMES[pool.kv_get_stats()["last_path_out"]]
                    lat_paths[nm] = lat_paths.get(nm, 0) + 1
        # ... and the fixed cost alone: one block each way
        one = tuple(np.ascontiguousarray(x[:1], np.int32) for x in (og, oh, ih, ig))
        one_raw = (ptr(one[0]), ptr(one[1]), 1, ptr(one[2]), ptr(one[3]), 1)
        one_us = []
        for rep in range(50):
            t1 = time.perf_counter()
            pool.kv_rotate_raw(*one_raw)
            pool.kv_sync()
            if rep >= 10:
                one_us.append((time.perf_counter() - t1) * 1e6)
        pool.kv_pool_set_call_timing(True)
        # ---- device-side gather / scatter on their own (HBM <-> contiguous HBM), whole list in one launch
        stage = torch.empty(len(og) * shape.block_bytes, dtype=torch.uint8, device=dev)
        leg = {}
        for name, fn in (("gather", lambda: pool.kv_gather_blocks(og, stage.data_ptr())),
                         ("scatter", lambda: pool.kv_scatter_blocks(stage.data_ptr(), ig[:len(og)]))):
            ts = []
            for _ in range(8):
                fn()
                pool.kv_sync()
                ts.append(pool.kv_get_stats()["last_union_ms"])
            leg[name] = float(np.mean(ts[3:]))
        leg_bytes = 2.0 * len(og) * shape.block_bytes          # read + write
        del stage
        p_bi_now = max(probe["bi_sum_gbs"], probe2["bi_sum_gbs"])

        table1, cfg5, cfg3 = None, None, None
        if not args.quick:
            # ---- config 4, the cell of the paper's bandwidth table (section 5.3.3): block 16, 8 GiB (32768 tokens
            #      of the paper's 256 KB per token) each way, tables random and contiguous; each direction alone
            #      ("u", end-to-end = the sum) and both at once ("b", end-to-end = the slower one)
            def table1_cell(contiguous: bool) -> dict:
                n = int(min(4096, (nb_gpu - 16) // 2, (nb_host - 16) // 2))
                w4 = W.config4_sweep_case(16, contiguous, n * shape.block_bytes, nb_gpu=nb_gpu, nb_host=nb_host)
                r4 = w4.steps[0]
                nb4 = r4.n_out * shape.block_bytes
                t_o = timed(lambda: pool.kv_swap_out(r4.out_gpu, r4.out_host))
                t_i = timed(lambda: pool.kv_swap_in(r4.in_host, r4.in_gpu))
                best = None
                for _ in range(3):
                    pool.kv_rotate(r4.out_gpu, r4.out_host, r4.in_host, r4.in_gpu)
                    pool.kv_sync()
                    s4 = pool.kv_get_stats()
                    if best is None or s4["last_union_ms"] < best["last_union_ms"]:
                        best = s4
                return {"blocks_each_way": int(r4.n_out), "bytes_each_way": nb4,
                        "d2h_u_gbs": M.gbs(nb4, t_o), "h2d_u_gbs": M.gbs(nb4, t_i), "e2e_ms_serial_u": t_o + t_i,
                        "d2h_b_gbs": M.gbs(nb4, best["last_out_ms"]), "h2d_b_gbs": M.gbs(nb4, best["last_in_ms"]),
                        "e2e_ms_concurrent_b": best["last_union_ms"], "both_gbs": M.gbs(2 * nb4, best["last_union_ms"]),
                        "frac_of_probe": M.gbs(2 * nb4, best["last_union_ms"]) / p_bi_now,
                        "path": B.PATH_NAMES[best["last_path_out"]]}
            table1 = {"random_tables": table1_cell(False), "contiguous_tables": table1_cell(True),
                      "paper_gh200_context": "DuplexKV 180.99 / 179.37 GB/s (b), 46.80 ms; naive 10.75 / 9.86 GB/s (u), 1556.15 ms (Table 1)"}

            # ---- config 5: the serving replay at 8 requests/s under the paper's per-iteration budget of 2400
            #      blocks; the first 200 steps that move anything, each against the 70 ms of a model step
            try:
                w5 = W.config5_replay(rate=8.0, nb_host=min(nb_host, 52888))
                if w5.nb_gpu > nb_gpu:
                    raise MemoryError("device pool smaller than the replay's")
                moving = [r5 for r5 in W.budgeted_steps(w5.steps, 2400) if r5.n_out + r5.n_in][:200]
                ms5, blocks5 = [], []
                for r5 in moving:
                    pool.kv_rotate(r5.out_gpu, r5.out_host, r5.in_host, r5.in_gpu)
                    pool.kv_sync()
                    ms5.append(pool.kv_get_stats()["last_union_ms"])
                    blocks5.append(r5.n_out + r5.n_in)
                cfg5 = {"steps_timed": len(ms5), "b_xfer_blocks": 2400, "ms_median": float(np.median(ms5)),
                        "ms_worst": float(np.max(ms5)), "blocks_median": float(np.median(blocks5)),
                        "blocks_worst_step": int(blocks5[int(np.argmax(ms5))]),
                        "gbs_overall": M.gbs(float(np.sum(blocks5)) * shape.block_bytes, float(np.sum(ms5))),
                        "steps_over_70ms_model_step": int(np.sum(np.array(ms5) > 70.0)),
                        "model_step_ms_paper": 69.82}
            except MemoryError as e:
                cfg5 = {"skipped": f"pools too small on this box: {e}"}

            # ---- config 3: 70B shape (5 MiB blocks, 160 planes), fragmented pool, 8 requests each way per step; a
            #      second pool over the same device and host memory (already page-locked: no second pinning)
            cfg3 = None
            try:
                s3 = W.SHAPE_70B
                nb_gpu3 = (nb_gpu * shape.block_bytes) // s3.block_bytes
                nb_host3 = host_bytes // s3.block_bytes
                n3 = 12
                w3 = W.config3_70b(nb_gpu=nb_gpu3, nb_host=nb_host3, n_steps=3 + n3)
                pool3 = B.KVPool(s3.num_layers, s3.block_size, s3.kv_heads, s3.head_dim, nb_gpu3, nb_host3,
                                 device_pool.data_ptr(), host_base=host_base, device_id=local_rank, path=args.path,
                                 flags=args.flags, staging_bytes=args.staging_mib << 20)
                ms3, by3 = [], []
                for k3, r3 in enumerate(w3.steps):
                    pool3.kv_rotate(r3.out_gpu, r3.out_host, r3.in_host, r3.in_gpu)
                    pool3.kv_sync()
                    if k3 >= 3:
                        ms3.append(pool3.kv_get_stats()["last_union_ms"])
                        by3.append((r3.n_out + r3.n_in) * s3.block_bytes)
                st3 = pool3.kv_get_stats()
                g3 = [M.gbs(b, t) for b, t in zip(by3, ms3)]
                cfg3 = {"steps_timed": len(ms3), "gpu_pool_blocks": int(nb_gpu3), "host_pool_blocks": int(nb_host3),
                        "block_bytes": s3.block_bytes, "bytes_per_step_median": float(np.median(by3)),
                        "ms_per_step_median": float(np.median(ms3)), "gbs_median": float(np.median(g3)),
                        "gbs_min": float(np.min(g3)), "gbs_max": float(np.max(g3)),
                        "frac_of_probe": float(np.median(g3)) / p_bi_now, "path": B.PATH_NAMES[st3["last_path_out"]]}
                pool3.destroy()
            except (MemoryError, B.KVError) as e:
                cfg3 = {"skipped": f"not run on this box: {e}"}

            # ---- the device leg against segment size: the 8B shape whole and as the shard one rank holds at
            #      tensor-parallel degree 4 and 8 (block 16 and 8), 4 GiB pools, half of the blocks gathered
            by_seg = []
            for kv_h, bs_h, hd_h in ((8, 16, 128), (2, 16, 128), (1, 16, 128), (1, 8, 128), (1, 8, 64)):
                sh = W.KVShape(shape.num_layers, bs_h, kv_h, hd_h)
                nb_s = ((1 if args.small else 4) << 30) // sh.block_bytes - 37
                ids_s = np.random.default_rng(3).permutation(nb_s)[:nb_s // 2].astype(np.int32)
                dev_s = torch.empty(nb_s * sh.block_bytes, dtype=torch.uint8, device=dev)
                out_s = torch.empty(len(ids_s) * sh.block_bytes, dtype=torch.uint8, device=dev)
                pool_s = B.KVPool(sh.num_layers, bs_h, kv_h, hd_h, nb_s, 16, dev_s.data_ptr(), device_id=local_rank)
                ts = []
                for _ in range(8):
                    pool_s.kv_gather_blocks(ids_s, out_s.data_ptr())
                    pool_s.kv_sync()
                    ts.append(pool_s.kv_get_stats()["last_union_ms"])
                pool_s.destroy()
                g_s = M.gbs(2.0 * len(ids_s) * sh.block_bytes, float(np.mean(ts[3:])))
                by_seg.append({"kv_heads": kv_h, "block_size": bs_h, "head_dim": hd_h, "segment_bytes": sh.words_per_plane * 2,
                               "gather_gbs": g_s, "frac_of_measured_hbm": g_s / peaks["hbm_gbs"]})
                del dev_s, out_s

        extra = {"paths": paths, "singles": singles, "lat_us": lat_us, "lat_blocks": lat_blocks, "leg": leg,
                 "leg_bytes": leg_bytes, "probe2": probe2, "contiguous_host": contiguous_host, "table": tb,
                 "lat_paths": lat_paths, "one_us": one_us, "table1": table1, "cfg5": cfg5, "cfg3": cfg3,
                 "by_seg": by_seg if not args.quick else None}

    pool.destroy()
    del device_pool
    torch.cuda.empty_cache()

    if rank == 0:
        # ---- CPU oracle on the host cores, bounded sample of the same rotation
        threads = os.cpu_count() or 1
        cpu_line = None
        if world == 1:                 # with more ranks the other GPUs would be held while the host cores work
            nb_s, t_mt, sample = time_oracle(shape, rot, CPU_SAMPLE_BLOCKS, threads, reps=20, warmup=2)
            _, t_1, _ = time_oracle(shape, rot, 256, 1, reps=5)
            cpu_line = {"value": M.gbs(nb_s, float(np.mean(t_mt)) * 1e3), "unit": UNIT, "cores": threads, "kind": "oracle",
                        "sample": sample,
                        "single_thread_value": M.gbs(2 * 256 * shape.block_bytes, float(np.mean(t_1)) * 1e3)}

        step_ms = dev_total_ms / args.steps
        probe2 = extra["probe2"]
        p_bi = max(probe["bi_sum_gbs"], probe2["bi_sum_gbs"])
        p_d2h = max(probe["d2h_gbs"], probe2["d2h_gbs"])
        p_h2d = max(probe["h2d_gbs"], probe2["h2d_gbs"])
        ideal_ms = M.duplex_ideal_ms(bytes_out, bytes_in, p_d2h, p_h2d, p_bi)
        paths = extra["paths"]
        mine = B.PATH_NAMES[st["last_path_out"]]
        uni = paths.get(mine, paths["staged"])
        link = {"bound": "host_link", "achieved": value / world, "peak": p_bi, "unit": "GB/s",
                "frac": value / world / p_bi,
                "peak_source": "pinned copy-engine probe in this process, 256 MiB transfers, both directions at once; "
                               "the larger of the readings taken before and after the timed region (of measured)",
                "probe_before": probe, "probe_after": probe2, "ideal_ms_per_step": ideal_ms}
        leg_ach = M.gbs(extra["leg_bytes"], extra["leg"]["gather"])
        if k_n > 0:
            k_avg_ms = k_ms / k_n
            k_ach = M.gbs(2.0 * k_bytes, k_ms)
            roofline = {"bound": "hbm", "achieved": k_ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": k_ach / peaks["hbm_gbs"], "traffic": ncu_traffic_per_launch(k_bytes / k_n),
                        "traffic_source": "ncu capture on the --small case, scaled to this run's average launch",
                        "kernel": "kv_copy_bulk (pack: scattered HBM planes -> contiguous HBM staging; unpack: the reverse)",
                        "launches_timed": int(k_n), "avg_launch_us": k_avg_ms * 1e3,
                        "algorithmic_bytes_per_launch": 2.0 * k_bytes / k_n,
                        "peak_source": f"MEASURED_PEAKS.json hbm_gbs ({peaks['source']}; burst copy figure)",
                        "frac_of_nominal_8TBs": k_ach / 8000.0,
                        "how": "CUDA events around every pack / unpack launch on the stream it runs on, inside the timed steps. "
                               "The step itself is bound by the host link, not by this kernel (its launches take "
                               f"{100.0 * k_ms / dev_total_ms:.1f} % of the step): the step's own fraction is "
                               f"roofline_link.frac = {value / world / p_bi:.3f} of the probed both-directions rate",
                        # the same launches timed from inside the kernel (first CTA start to last CTA end): the
                        # events also see the wait for the launch, which is long while the link is busy
                        "exec_only": {"achieved": M.gbs(2.0 * k_bytes, k_exec_ms), "avg_launch_us": k_exec_ms / k_n * 1e3,
                                      "frac": M.gbs(2.0 * k_bytes, k_exec_ms) / peaks["hbm_gbs"]} if k_exec_ms > 0 else None}
        else:
            # zero-copy path: the dominant kernel crosses the host link, which is what bounds it
            roofline = dict(link, kernel="kv_copy_bulk (zero-copy rotate)", traffic=None)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "u16", "data": "synthetic",
            "config": {"workload": ("SMALL profiling case of " if args.small else "") +
                                   WORKLOAD % (len(rot.out_req_offsets) - 1),
                       "gpu_pool_blocks": nb_gpu, "host_pool_blocks": nb_host, "host_pool_shrunk": shrunk,
                       "blocks_out": int(rot.n_out), "blocks_in": int(rot.n_in), "block_bytes": shape.block_bytes,
                       "bytes_out_per_step": bytes_out, "bytes_in_per_step": bytes_in,
                       "path_out": B.PATH_NAMES[st["last_path_out"]], "path_in": B.PATH_NAMES[st["last_path_in"]],
                       "block_tables": "scattered ids in both pools (seeded free-list allocator)",
                       "l2": "inputs larger than L2 (3.9 GB per direction per step)", "replicas": world,
                       "pin_seconds": round(pin_s, 1)},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": bytes_in + 8 * (rot.n_out + rot.n_in),
                    "d2h_bytes_per_step": bytes_out, "ms_per_step": wall_total_s * 1e3 / args.steps,
                    "host_ms_inside_kv_rotate": float(np.median(issue_s[-args.steps:])) * 1e3},
            "gpu_launches": int(launches), "ce_transfers": int(ce_copies),
            "overlap": overlap_of(windows),
            "clocks": clocks,
            "roofline": roofline,
            "roofline_link": link,
            "roofline_hbm_standalone": {"bound": "hbm", "achieved": leg_ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                        "frac": leg_ach / peaks["hbm_gbs"], "frac_of_nominal_8TBs": leg_ach / 8000.0,
                                        "kernel": "kv_copy_bulk via kv_gather_blocks / kv_scatter_blocks, the whole "
                                                  "out list in one launch",
                                        "gather_ms": extra["leg"]["gather"], "scatter_ms": extra["leg"]["scatter"],
                                        "algorithmic_bytes": extra["leg_bytes"]},
            "directions": {"rotate_out_gbs": M.gbs(bytes_out * args.steps, dev_total_ms),
                           "rotate_in_gbs": M.gbs(bytes_in * args.steps, dev_total_ms),
                           "out_alone_gbs": uni["out_u_gbs"], "in_alone_gbs": uni["in_u_gbs"],
                           "out_alone_frac_of_d2h": uni["out_u_gbs"] / p_d2h,
                           "in_alone_frac_of_h2d": uni["in_u_gbs"] / p_h2d,
                           "e2e_ms_serial_u": uni["e2e_ms_serial_u"], "e2e_ms_concurrent_b": step_ms},
            "paths_on_same_lists": paths,
            "rotate_with_neighbouring_host_ids_gbs": extra["contiguous_host"],
            "block_table": extra["table"],
            "single_swaps": extra["singles"],
            "request_rotate_us": {"p50": M.percentile(extra["lat_us"], 0.5), "p99": M.percentile(extra["lat_us"], 0.99),
                                  "n": len(extra["lat_us"]), "requests": 2 * len(w.extra["pairs"]), "passes": 5,
                                  "median_blocks_per_call": float(np.median(extra["lat_blocks"])),
                                  "paths_taken": extra["lat_paths"],
                                  "how": "host clock from kv_rotate entry to kv_sync return, one request out + one in per call"},
            "one_block_rotate_us": {"p50": M.percentile(extra["one_us"], 0.5), "p99": M.percentile(extra["one_us"], 0.99),
                                    "n": len(extra["one_us"]),
                                    "link_time_us": shape.block_bytes / (p_d2h * 1e9) * 1e6},
            "config3": extra["cfg3"],
            "config4_table1": extra["table1"],
            "config5": extra["cfg5"],
            "device_leg_by_segment": extra["by_seg"],
            "cpu_baseline": cpu_line,
        }
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--path", type=int, default=0, help="KV_PATH_* (0 = auto)")
    ap.add_argument("--flags", type=int, default=0, help="KV_FLAG_* bits")
    ap.add_argument("--ctas", type=int, default=0, help="CTAs per direction (0 = default)")
    ap.add_argument("--staging-mib", type=int, default=0, help="per-direction staging of the staged path (0 = library default)")
    ap.add_argument("--link-variant", type=int, default=0, help="shape of the zero-copy kernels' transfers (0, 1, 2)")
    ap.add_argument("--quick", action="store_true", help="skip the per-segment comparator path")
    ap.add_argument("--trace", default=None, help="write a Chrome-trace JSON of the timed steps' two directions here")
    ap.add_argument("--small", action="store_true",
                    help="profiling case: same shape and kernels, 16 requests, 4 rotated each way, 6 GB + 8 GB pools")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        # not started by a launcher: start the N replicas here, one process per GPU
        import torch
        if torch.cuda.is_available() and torch.cuda.device_count() < args.gpus:
            raise SystemExit(f"bench.py: --gpus {args.gpus} asked for, the node has {torch.cuda.device_count()} GPUs")
        from paper_2601_20309_b200 import replicas as R
        sys.exit(R.main_spawn(args.gpus))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
    else:
        run_ours(args, rank, local_rank, world)


if __name__ == "__main__":
    main()
