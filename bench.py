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

METRIC = "full-duplex KV swap GB/s (out+in)"
UNIT = "GB/s"


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


# ------------------------------------------------------------------------------------------------ arms

def run_reference(args, rank: int) -> None:
    """The CPU oracle, as it stands, on the host cores: a deliberately plain program."""
    if rank != 0:
        return
    w = W.config2_8b()
    threads = os.cpu_count() or 1
    nbytes, times, sample = time_oracle(w.shape, w.steps[0], 512, threads, reps=args.steps, warmup=args.warmup)
    ms = float(np.mean(times)) * 1e3
    val = M.gbs(nbytes, ms)
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u16", "data": "synthetic",
            "config": {"workload": "config2 llama-3-8b-shaped KV, paired rotate 16 requests each way (CPU sample)"},
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
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device(dev))

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x: float) -> float:
        if dist is None:
            return x
        t = torch.tensor([x], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def sum_over_ranks(x: float) -> float:
        if dist is None:
            return x
        t = torch.tensor([x], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        return float(t.item())

    # ---- roofline denominators, measured here
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
                    device_pool.data_ptr(), device_id=local_rank, path=args.path, flags=args.flags,
                    ctas_out=args.ctas, ctas_in=args.ctas)
    pin_s = time.perf_counter() - t0
    host_base, host_bytes = pool.kv_host_ptr()
    # seeded content in both pools (GPU twin of the CPU generator; verified against it in the tests)
    F.fill_blocks(F.Layout.device(device_pool.data_ptr(), shape, nb_gpu), w.seed, W.POOL_GPU, nb_gpu, device=dev)
    host_dev_ptr = host_base       # unified addressing: mapped pinned memory has the same address on the device
    F.fill_blocks(F.Layout.host(host_dev_ptr, shape, nb_host), w.seed, W.POOL_HOST, nb_host, device=dev)

    og, oh, ih, ig = (np.ascontiguousarray(x, np.int32) for x in (rot.out_gpu, rot.out_host, rot.in_host, rot.in_gpu))
    args_raw = (ptr(og), ptr(oh), len(og), ptr(ih), ptr(ig), len(ig))

    def step():
        rc = pool.kv_rotate_raw(*args_raw)
        if rc != 0:
            raise RuntimeError(f"kv_rotate failed: {rc} {pool.kv_last_error()}")
        pool.kv_sync()

    for _ in range(args.warmup):
        step()
    launches0 = pool.kv_get_stats()["kernel_launches"]
    sampler = ClockSampler(local_rank)
    sampler.start()
    barrier()
    dev_ms = []
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
        dev_ms.append(pool.kv_get_stats()["last_union_ms"])
    barrier()
    wall_s = time.perf_counter() - t0
    clocks = sampler.stop()
    st = pool.kv_get_stats()
    launches = st["kernel_launches"] - launches0

    dev_total_ms = max_over_ranks(float(np.sum(dev_ms)))
    wall_total_s = max_over_ranks(wall_s)
    job_bytes = sum_over_ranks(float(bytes_out + bytes_in)) * args.steps
    value = M.gbs(job_bytes, dev_total_ms)
    e2e_value = job_bytes / wall_total_s / 1e9

    extra = {}
    if rank == 0:
        # ---- each direction alone (Table 1's "u" rows): the same lists, one direction per call
        uni = {}
        for name, fn, nb in (("out", lambda: pool.kv_swap_out(og, oh), bytes_out),
                             ("in", lambda: pool.kv_swap_in(ih, ig), bytes_in)):
            ts = []
            for _ in range(3):
                fn()
                pool.kv_sync()
                ts.append(pool.kv_get_stats()["last_union_ms"])
            uni[name] = M.gbs(nb, min(ts))
        # ---- single swaps of the median-length and the longest request
        singles = {}
        for key, which in (("single_out", "out"), ("single_in", "in")):
            for k, (a, b) in w.extra[key].items():
                ts = []
                for _ in range(3):
                    (pool.kv_swap_out(a, b) if which == "out" else pool.kv_swap_in(a, b))
                    pool.kv_sync()
                    ts.append(pool.kv_get_stats()["last_union_ms"])
                singles[f"{which}_{k}"] = {"blocks": len(a), "gbs": M.gbs(len(a) * shape.block_bytes, min(ts)),
                                           "ms": min(ts)}
        # ---- per-request rotate latency: one request out + one in per call, call entry to completion
        lat_us, lat_blocks = [], []
        for r in w.extra["pairs"] * 2:
            a = tuple(np.ascontiguousarray(x, np.int32) for x in (r.out_gpu, r.out_host, r.in_host, r.in_gpu))
            raw = (ptr(a[0]), ptr(a[1]), len(a[0]), ptr(a[2]), ptr(a[3]), len(a[3]))
            t1 = time.perf_counter()
            pool.kv_rotate_raw(*raw)
            pool.kv_sync()
            lat_us.append((time.perf_counter() - t1) * 1e6)
            lat_blocks.append(len(a[0]) + len(a[3]))
        lat_us = lat_us[len(lat_us) // 2:]       # second pass (first pass warms the path)
        # ---- device-side gather/scatter (HBM <-> contiguous HBM), the kernel half of the staged path
        ids = og
        stage = torch.empty(len(ids) * shape.block_bytes, dtype=torch.uint8, device=dev)
        leg = {}
        for name, fn in (("gather", lambda: pool.kv_gather_blocks(ids, stage.data_ptr())),
                         ("scatter", lambda: pool.kv_scatter_blocks(stage.data_ptr(), ig[:len(ids)]))):
            ts = []
            for _ in range(8):
                fn()
                pool.kv_sync()
                ts.append(pool.kv_get_stats()["last_union_ms"])
            leg[name] = float(np.mean(ts[3:]))
        n_leg = min(len(ids), len(ig))
        leg_bytes = 2.0 * len(ids) * shape.block_bytes          # read + write
        hbm_ach = M.gbs(leg_bytes, leg["gather"])
        del stage
        extra = {"uni": uni, "singles": singles, "lat_us": lat_us, "lat_blocks": lat_blocks[len(lat_blocks) // 2:],
                 "leg": leg, "hbm_ach": hbm_ach, "leg_bytes": leg_bytes, "n_leg": n_leg}

    pool.destroy()
    del device_pool
    torch.cuda.empty_cache()

    if rank == 0:
        # ---- CPU oracle on the host cores, bounded sample of the same rotation
        threads = os.cpu_count() or 1
        nb_s, t_mt, sample = time_oracle(shape, rot, 768, threads, reps=3)
        _, t_1, _ = time_oracle(shape, rot, 256, 1, reps=2)
        cpu_val = M.gbs(nb_s, float(np.mean(t_mt)) * 1e3)
        cpu_1 = M.gbs(2 * 256 * shape.block_bytes, float(np.mean(t_1)) * 1e3)

        step_ms = dev_total_ms / args.steps
        p_bi = probe["bi_sum_gbs"]
        ideal_ms = M.duplex_ideal_ms(bytes_out, bytes_in, probe["d2h_gbs"], probe["h2d_gbs"], p_bi)
        uni = extra["uni"]
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "u16", "data": "synthetic",
            "config": {"workload": ("SMALL profiling case of " if args.small else "") +
                                   "config2 llama-3-8b-shaped KV (32 layers, 8 kv heads, head_dim 128, block 16, bf16): "
                                   "paired rotate of %d requests each way per step" % (len(rot.out_req_offsets) - 1),
                       "gpu_pool_blocks": nb_gpu, "host_pool_blocks": nb_host, "host_pool_shrunk": shrunk,
                       "blocks_out": int(rot.n_out), "blocks_in": int(rot.n_in), "block_bytes": shape.block_bytes,
                       "bytes_out_per_step": bytes_out, "bytes_in_per_step": bytes_in,
                       "path_out": B.PATH_NAMES[st["last_path_out"]], "path_in": B.PATH_NAMES[st["last_path_in"]],
                       "l2": "inputs larger than L2 (3.9 GB per direction per step)", "replicas": world,
                       "pin_seconds": round(pin_s, 1)},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": bytes_in + 8 * (rot.n_out + rot.n_in),
                    "d2h_bytes_per_step": bytes_out, "ms_per_step": wall_total_s * 1e3 / args.steps},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "roofline": {"bound": "host_link", "achieved": value / world, "peak": p_bi, "unit": "GB/s",
                         "frac": value / world / p_bi, "traffic": None,
                         "peak_source": "pinned copy-engine probe in this process (256 MiB x 4, both directions at once)",
                         "kernel": "kv_copy_bulk (zero-copy rotate)", "ideal_ms_per_step": ideal_ms},
            "roofline_hbm": {"bound": "hbm", "achieved": extra["hbm_ach"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                             "frac": extra["hbm_ach"] / peaks["hbm_gbs"], "traffic": None,
                             "peak_source": f"MEASURED_PEAKS.json ({peaks['source']})",
                             "frac_of_nominal_8TBs": extra["hbm_ach"] / 8000.0,
                             "kernel": "kv_copy_bulk (device-side gather, HBM to contiguous HBM)",
                             "gather_ms": extra["leg"]["gather"], "scatter_ms": extra["leg"]["scatter"],
                             "algorithmic_bytes": extra["leg_bytes"]},
            "link_probe": probe,
            "directions": {"rotate_out_gbs": M.gbs(bytes_out * args.steps, dev_total_ms),
                           "rotate_in_gbs": M.gbs(bytes_in * args.steps, dev_total_ms),
                           "out_alone_gbs": uni["out"], "in_alone_gbs": uni["in"],
                           "out_alone_frac_of_d2h": uni["out"] / probe["d2h_gbs"],
                           "in_alone_frac_of_h2d": uni["in"] / probe["h2d_gbs"],
                           "e2e_ms_serial_u": M.e2e_ms(bytes_out, bytes_in, uni["out"], uni["in"], False),
                           "e2e_ms_concurrent_b": step_ms},
            "single_swaps": extra["singles"],
            "request_rotate_us": {"p50": M.percentile(extra["lat_us"], 0.5), "p99": M.percentile(extra["lat_us"], 0.99),
                                  "n": len(extra["lat_us"]),
                                  "median_blocks_per_call": float(np.median(extra["lat_blocks"]))},
            "cpu_baseline": {"value": cpu_val, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample,
                             "single_thread_value": cpu_1},
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
    ap.add_argument("--small", action="store_true",
                    help="profiling case: same shape and kernels, 16 requests, 4 rotated each way, 6 GB + 8 GB pools")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
    else:
        run_ours(args, rank, local_rank, world)


if __name__ == "__main__":
    main()
