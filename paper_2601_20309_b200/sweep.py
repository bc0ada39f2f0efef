"""Measurement sweeps on the GPU machine (need a CUDA device).

    python -m paper_2601_20309_b200.sweep probe [--out FILE]
        The host link's bandwidth against the shape of copy-engine transfers: plain transfers of
        32 KiB .. 1 GiB, and strided 2-D transfers (rows x row bytes), each direction alone and both
        at once, at scattered offsets of 4 GiB pinned buffers.  The analogue of the paper's
        bandwidth-versus-segment-size figure (section 3.3) on this machine.

    python -m paper_2601_20309_b200.sweep paths [--max-payload-gb G] [--out FILE]
        Block-size and fragmentation sweep on the 8B shape: block_size 8/16/32/64, block tables
        contiguous or uniformly random, payload 64 MB .. G GB per direction, each direction alone
        and both at once, on every transfer path.  Its result is the table behind kv_path_for.

    python -m paper_2601_20309_b200.sweep paths --kv-heads H ...
        The same sweep for the shard one rank of a tensor-parallel group holds (H = 4, 2 or 1 of the 8 KV
        heads): segments and blocks shrink by 8 / H.

    python -m paper_2601_20309_b200.sweep segments [--pool-gib P] [--out FILE]
        Rates against segment size, 32 KiB (the 8B shape) down to 1 KiB (small shards): gather and scatter
        of half of a P GiB pool's blocks (P = 4: 2 GiB), scattered, HBM to HBM, and the zero-copy kernels over
        the link, P/8 GiB each way.

    python -m paper_2601_20309_b200.sweep overlap [--out FILE]
        Rotation beside compute (the paper's cross-iteration pipeline, section 4.3.2, hides transfers
        behind model execution): a rotation of 2 GiB each way runs while a stand-in for a decode step
        (back-to-back element-wise kernels over 1 GiB on a third stream: HBM-bound, every SM busy) runs too.  Reports
        how much each slows the other, for the staged path and for the zero-copy path with 8, 16, 32 and
        64 CTAs per direction (how many SMs the rotation needs beside compute).

    python -m paper_2601_20309_b200.sweep latency [--out FILE]
        Call-to-completion time of small rotations (1 .. 256 blocks each way, 8B shape, scattered ids):
        host clock around kv_rotate + kv_sync through the C ABI with ready-made id arrays, median of 40,
        per path, and how much of it the call itself takes before it returns.  What a per-request
        rotate costs when the link is not the limit, and whether AUTO picks the quickest path.

    python -m paper_2601_20309_b200.sweep budget [--b-xfer N] [--out FILE]
        The serving replay (8B shape, 8 requests/s, 2000 steps) re-timed under the paper's per-iteration
        transfer budget (B_xfer blocks per step, 2400 in the paper's main runs; remainder carried over):
        device time of every step's rotation, against the 70 ms a model step takes in the paper
        (section 5.3.4), i.e. how often the transfer would not hide behind the step.

    python -m paper_2601_20309_b200.sweep lvf [--b-xfer N] [--steps K] [--out FILE]
        Rotation lists made by the paper's Largest-VLT-First policy (section 4.2, Algorithm 1) on the serving
        replay (8B shape, 8 requests/s, the paper's scheduler settings) under a transfer budget of N blocks:
        device time of the first K steps that move blocks, against the 70 ms of a model step.  The policy
        rotates hard; this shows what budget a PCIe link can hide.

    python -m paper_2601_20309_b200.sweep lvf-table [--b-xfer N] [--steps K] [--eager-blocks E] [--out FILE]
        The same replay and policy driven through the library's block table (kv_req_add / kv_req_append /
        kv_eager_rotate / kv_req_rotate / kv_req_finish), which hands out the blocks itself: with E > 0 up
        to E full blocks per step are copied to host memory in the background (the paper's eager block
        rotation, section 4.3.2), so a preemption sends only what has no valid host copy and its device
        blocks serve the requests resuming in the same rotation.  Reports, per step, the blocks moved at
        rotation time and the rotation's device time, with and without the background copies.

    python -m paper_2601_20309_b200.sweep handoff [--out FILE]
        What a hand-off between the copy engine and a kernel costs while the host link is busy (plain torch
        streams, no library call): a host-to-device copy followed by a tiny kernel that waits for it, and a
        tiny kernel followed by a device-to-host copy that waits for it, on one stream or across two, with
        the other direction idle or saturated.  This is the price of every chunk boundary of the staged path.

All print one JSON object per line and, at the end, a markdown table.
"""
from __future__ import annotations

import argparse
import json
import sys

from . import binding as B
from . import workload as W

K, M, G = 1 << 10, 1 << 20, 1 << 30


def _emit(rec, out):
    line = json.dumps(rec)
    print(line, flush=True)
    if out:
        out.write(line + "\n")
        out.flush()


def probe(out) -> None:
    rows = []
    base = B.kv_probe_link(0, 256 * M, 4)
    _emit({"case": "reference: 256 MiB plain transfers, same buffer", **base}, out)
    shapes = [(f"plain {s // K} KiB" if s < M else f"plain {s // M} MiB", dict(copy_bytes=s))
              for s in (32 * K, 64 * K, 256 * K, 1 * M, 2 * M, 4 * M, 8 * M, 16 * M, 64 * M, 256 * M, 1 * G)]
    shapes += [
        ("64 rows x 32 KiB, packed both sides", dict(copy_bytes=2 * M, rows=64)),
        ("64 rows x 32 KiB, device pitch 32 MiB (one block-16 block of a layer-first pool)",
         dict(copy_bytes=2 * M, rows=64, dev_pitch=32 * M)),
        ("64 rows x 16 KiB, device pitch 32 MiB (block 8)", dict(copy_bytes=1 * M, rows=64, dev_pitch=32 * M)),
        ("64 rows x 64 KiB, device pitch 32 MiB (block 32)", dict(copy_bytes=4 * M, rows=64, dev_pitch=32 * M)),
        ("64 rows x 128 KiB, device pitch 32 MiB (block 64)", dict(copy_bytes=8 * M, rows=64, dev_pitch=32 * M)),
        ("2 rows x 1 MiB, host pitch 64 MiB", dict(copy_bytes=2 * M, rows=2, host_pitch=64 * M)),
        ("2 rows x 2 MiB, host pitch 64 MiB", dict(copy_bytes=4 * M, rows=2, host_pitch=64 * M)),
        ("2 rows x 2 MiB, host pitch 1 GiB", dict(copy_bytes=4 * M, rows=2, host_pitch=1024 * M)),
        ("2 rows x 4 MiB, host pitch 64 MiB", dict(copy_bytes=8 * M, rows=2, host_pitch=64 * M)),
        ("4 rows x 2 MiB, host pitch 64 MiB", dict(copy_bytes=8 * M, rows=4, host_pitch=64 * M)),
        ("8 rows x 2 MiB, host pitch 64 MiB", dict(copy_bytes=16 * M, rows=8, host_pitch=64 * M)),
        # four blocks whose host addresses form a 2 x 2 lattice (a, a+g, a+kg, a+kg+g) as one 3-D transfer
        ("2 slices x 2 rows x 2 MiB (3-D), row pitch 64 MiB, slices 448 MiB apart",
         dict(copy_bytes=8 * M, rows=2, host_pitch=64 * M, slices=2, host_slice_rows=7)),
        ("2 slices x 2 rows x 1 MiB (3-D), row pitch 64 MiB, slices 448 MiB apart",
         dict(copy_bytes=4 * M, rows=2, host_pitch=64 * M, slices=2, host_slice_rows=7)),
    ]
    for name, kw in shapes:
        total = G if kw["copy_bytes"] >= 256 * K else G // 4
        r = B.kv_probe_link_ex(0, total_bytes=max(total, kw["copy_bytes"]), span_bytes=4 * G, scattered=True,
                               rounds=2, **kw)
        rec = {"case": name, **{k: round(v, 2) for k, v in r.items() if k.endswith("gbs")},
               "transfers_per_round": r["reps"]}
        rows.append(rec)
        _emit(rec, out)
    print("\n| transfer shape | D2H alone | H2D alone | both: D2H | both: H2D | both: sum |\n|---|---|---|---|---|---|")
    for r in rows:
        print(f"| {r['case']} | {r['d2h_gbs']} | {r['h2d_gbs']} | {r['bi_d2h_gbs']} | {r['bi_h2d_gbs']} | {r['bi_sum_gbs']} |")


PATHS = [("staged", B.KV_PATH_STAGED), ("zerocopy", B.KV_PATH_ZEROCOPY), ("ce2d", B.KV_PATH_CE2D),
         ("naive", B.KV_PATH_NAIVE), ("auto", B.KV_PATH_AUTO)]


def paths(out, max_payload_gb: float, device_layout: int = 0, kv_heads: int = 8) -> None:
    import torch
    rows = []
    payloads = [p for p in (64e6, 256e6, 1e9, 4e9, 8e9) if p <= max_payload_gb * 1e9 + 1]
    for bs in (8, 16, 32, 64):
        for contiguous in (True, False):
            for payload in payloads:
                shape = W.KVShape(32, bs, kv_heads)
                n = max(1, int(payload // shape.block_bytes))
                # random tables: a host pool much larger than the payload, so that ids are truly scattered
                nb_host = 2 * n + 16 if contiguous else int(min(16 * n, 40e9 // shape.block_bytes))
                w = W.config4_sweep_case(bs, contiguous, payload, nb_host=max(nb_host, 2 * n + 16), kv_heads=kv_heads)
                rot = w.steps[0]
                dev = torch.empty(w.nb_gpu * shape.block_bytes, dtype=torch.uint8, device="cuda:0")
                probe_bi = B.kv_probe_link(0, 256 * M, 2)["bi_sum_gbs"]
                pool = B.KVPool(shape.num_layers, shape.block_size, shape.kv_heads, shape.head_dim, w.nb_gpu,
                                w.nb_host, dev.data_ptr(), device_layout=device_layout)
                nbytes = rot.n_out * shape.block_bytes

                def best(fn, reps):
                    ts = []
                    for k in range(reps + 1):
                        fn()
                        pool.kv_sync()
                        if k:
                            ts.append(pool.kv_get_stats()["last_union_ms"])
                    return min(ts)

                rec = {"block_size": bs, "seg_kib": shape.words_per_plane * 2 // K, "blk_mib": shape.block_bytes / M,
                       "tables": "contiguous" if contiguous else "random", "payload_mb": round(nbytes / 1e6),
                       "blocks": rot.n_out, "probe_bi_gbs": round(probe_bi, 1)}
                for name, pid in PATHS:
                    if name == "naive" and payload > 300e6:
                        continue
                    pool.kv_pool_set_path(pid, pid)
                    reps = 1 if name == "naive" else 3
                    t_o = best(lambda: pool.kv_swap_out(rot.out_gpu, rot.out_host), reps)
                    t_i = best(lambda: pool.kv_swap_in(rot.in_host, rot.in_gpu), reps)
                    t_b = best(lambda: pool.kv_rotate(rot.out_gpu, rot.out_host, rot.in_host, rot.in_gpu), reps)
                    rec[name] = {"out": round(nbytes / t_o / 1e6, 1), "in": round(nbytes / t_i / 1e6, 1),
                                 "both": round(2 * nbytes / t_b / 1e6, 1)}
                    if name == "auto":
                        rec["auto_took"] = B.PATH_NAMES[pool.kv_get_stats()["last_path_out"]]
                pool.destroy()
                del dev
                torch.cuda.empty_cache()
                rows.append(rec)
                _emit(rec, out)
    print("\n| block | BLK MiB | tables | payload MB | probe both | staged out/in/both | zero-copy out/in/both | "
          "2-D per block out/in/both | per segment out/in/both | AUTO out/in/both | AUTO took |\n|---|---|---|---|---|---|---|---|---|---|---|")
    for r in rows:
        f = lambda k: "%s / %s / %s" % (r[k]["out"], r[k]["in"], r[k]["both"]) if k in r else "-"
        print(f"| {r['block_size']} | {r['blk_mib']:g} | {r['tables']} | {r['payload_mb']} | {r['probe_bi_gbs']} | "
              f"{f('staged')} | {f('zerocopy')} | {f('ce2d')} | {f('naive')} | {f('auto')} | {r['auto_took']} |")


def segments(out, pool_gib: int = 4) -> None:
    """Rates against segment size: the device leg (gather / scatter of 2 GiB of scattered blocks, HBM to
    HBM) and the zero-copy kernels (an eighth of the pool size each way over the link), for the 8B shape and the shards of it
    that one rank of a tensor-parallel group holds, down to 1 KiB segments."""
    import numpy as np
    import torch
    rows = []
    for kv, bs, hd in ((8, 16, 128), (4, 16, 128), (2, 16, 128), (1, 32, 128), (1, 16, 128), (1, 8, 128), (1, 8, 64)):
        shape = W.KVShape(32, bs, kv, hd)
        blk = shape.block_bytes
        nbg, nbh = pool_gib * G // blk - 37, pool_gib * G // 2 // blk
        n = nbg // 2
        dev = torch.empty(nbg * blk, dtype=torch.uint8, device="cuda:0")
        stage = torch.empty(n * blk, dtype=torch.uint8, device="cuda:0")
        pool = B.KVPool(shape.num_layers, bs, kv, hd, nbg, nbh, dev.data_ptr(), path=B.KV_PATH_ZEROCOPY)
        rng = np.random.default_rng(3)
        gp, hp = rng.permutation(nbg).astype(np.int32), rng.permutation(nbh).astype(np.int32)
        ids = gp[:n]

        def mean_ms(fn, reps=7, skip=3):
            ts = []
            for _ in range(reps):
                fn()
                pool.kv_sync()
                ts.append(pool.kv_get_stats()["last_union_ms"])
            return float(np.mean(ts[skip:]))

        rec = {"kv_heads": kv, "block_size": bs, "head_dim": hd, "seg_kib": shape.words_per_plane * 2 / K,
               "blk_kib": blk / K, "blocks_gathered": int(n),
               "gather_tbs": round(2.0 * n * blk / mean_ms(lambda: pool.kv_gather_blocks(ids, stage.data_ptr())) / 1e9, 3),
               "scatter_tbs": round(2.0 * n * blk / mean_ms(lambda: pool.kv_scatter_blocks(stage.data_ptr(), ids)) / 1e9, 3)}
        m = (pool_gib * 128 * M) // blk
        og, ig, oh, ih = gp[:m], gp[m:2 * m], hp[:m], hp[m:2 * m]
        rec["zerocopy_out_gbs"] = round(m * blk / mean_ms(lambda: pool.kv_swap_out(og, oh), 4, 1) / 1e6, 1)
        rec["zerocopy_in_gbs"] = round(m * blk / mean_ms(lambda: pool.kv_swap_in(ih, ig), 4, 1) / 1e6, 1)
        rec["zerocopy_both_gbs"] = round(2 * m * blk / mean_ms(lambda: pool.kv_rotate(og, oh, ih, ig), 4, 1) / 1e6, 1)
        pool.destroy()
        del dev, stage
        torch.cuda.empty_cache()
        rows.append(rec)
        _emit(rec, out)
    print("\n| KV heads | block | head dim | SEG KiB | BLK KiB | gather TB/s | scatter TB/s | zero-copy out / in / both GB/s |\n|---|---|---|---|---|---|---|---|")
    for r in rows:
        print(f"| {r['kv_heads']} | {r['block_size']} | {r['head_dim']} | {r['seg_kib']:g} | {r['blk_kib']:g} | {r['gather_tbs']} | "
              f"{r['scatter_tbs']} | {r['zerocopy_out_gbs']} / {r['zerocopy_in_gbs']} / {r['zerocopy_both_gbs']} |")


def overlap(out) -> None:
    import torch
    shape = W.SHAPE_8B
    n = 1024                                                   # 2 GiB each way
    w = W.config4_sweep_case(16, False, n * shape.block_bytes, nb_host=16 * n)
    rot = w.steps[0]
    dev = torch.empty(w.nb_gpu * shape.block_bytes, dtype=torch.uint8, device="cuda:0")
    src = torch.empty(1 << 30, dtype=torch.uint8, device="cuda:0")
    dst = torch.empty_like(src)
    side = torch.cuda.Stream()
    pool = B.KVPool(shape.num_layers, shape.block_size, shape.kv_heads, shape.head_dim, w.nb_gpu, w.nb_host,
                    dev.data_ptr())
    nbytes = 2 * rot.n_out * shape.block_bytes

    def compute(k):
        """k stand-in decode steps on the side stream; returns (start, end) events."""
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(side):
            e0.record()
            for _ in range(k):
                torch.add(src, 1, out=dst)                     # an SM kernel (a plain copy could go to a copy engine)
            e1.record()
        return e0, e1

    rows = []
    # the zero-copy kernels occupy SMs for the whole transfer: how many CTAs per direction they need beside
    # compute is the sizing question (the staged path's pack / unpack kernels run for about 1 % of the time)
    cases = [("staged", B.KV_PATH_STAGED, 0)] + [("zerocopy", B.KV_PATH_ZEROCOPY, c) for c in (8, 16, 32, 64)]
    for name, pid, ctas in cases:
        pool.kv_pool_set_path(pid, pid)
        pool.kv_pool_set_ctas(ctas, ctas)
        for _ in range(2):                                     # warm-up
            pool.kv_rotate(rot.out_gpu, rot.out_host, rot.in_host, rot.in_gpu)
            pool.kv_sync()
        t_rot = []
        for _ in range(3):
            pool.kv_rotate(rot.out_gpu, rot.out_host, rot.in_host, rot.in_gpu)
            pool.kv_sync()
            t_rot.append(pool.kv_get_stats()["last_union_ms"])
        rot_alone = min(t_rot)
        alone = []
        for _ in range(3):                                     # first round warms the kernel up
            e0, e1 = compute(40)
            torch.cuda.synchronize()
            alone.append(e0.elapsed_time(e1) / 40)
        step_alone = min(alone[1:])                            # ms per 1 GiB pass with nothing else running
        k = max(4, int(1.3 * rot_alone / step_alone))          # compute outlasts the rotation a little
        both_rot, both_step = [], []
        for _ in range(3):
            e0, e1 = compute(k)
            pool.kv_rotate(rot.out_gpu, rot.out_host, rot.in_host, rot.in_gpu)
            pool.kv_sync()
            both_rot.append(pool.kv_get_stats()["last_union_ms"])
            torch.cuda.synchronize()
            both_step.append(e0.elapsed_time(e1) / k)
        # the compute ran beside the rotation for rot/(k*step) of its time; scale its slowdown to that share
        r_ms, s_ms = min(both_rot), min(both_step)
        share = min(1.0, r_ms / (k * s_ms))
        rec = {"path": name, "ctas_per_direction": ctas if ctas else None, "rotate_alone_gbs": round(nbytes / rot_alone / 1e6, 1), "rotate_beside_compute_gbs": round(nbytes / r_ms / 1e6, 1),
               "compute_alone_tbs": round(2 * (1 << 30) / step_alone / 1e9, 2), "compute_beside_rotate_tbs": round(2 * (1 << 30) / s_ms / 1e9, 2),
               "compute_slowdown_pct_over_whole_run": round(100 * (s_ms / step_alone - 1), 2),
               "compute_slowdown_pct_while_rotating": round(100 * (s_ms / step_alone - 1) / share, 2),
               "rotate_slowdown_pct": round(100 * (r_ms / rot_alone - 1), 2), "decode_steps": k}
        rows.append(rec)
        _emit(rec, out)
    pool.destroy()
    print("\n| path | CTAs per direction | rotate alone GB/s | rotate beside compute GB/s | compute alone TB/s | compute beside rotate TB/s | "
          "compute slowdown while rotating | rotate slowdown |\n|---|---|---|---|---|---|---|---|")
    for r in rows:
        print(f"| {r['path']} | {r['ctas_per_direction'] or '-'} | {r['rotate_alone_gbs']} | {r['rotate_beside_compute_gbs']} | {r['compute_alone_tbs']} | "
              f"{r['compute_beside_rotate_tbs']} | {r['compute_slowdown_pct_while_rotating']} % | {r['rotate_slowdown_pct']} % |")


def latency(out, block_size: int = 16, kv_heads: int = 8) -> None:
    import time
    import numpy as np
    import torch
    shape = W.KVShape(32, block_size, kv_heads)
    nb = 4096 * 16 // block_size if block_size < 16 else 4096
    dev = torch.empty(nb * shape.block_bytes, dtype=torch.uint8, device="cuda:0")
    pool = B.KVPool(shape.num_layers, shape.block_size, shape.kv_heads, shape.head_dim, nb, nb, dev.data_ptr())
    rng = np.random.default_rng(3)
    i32p = B.C.POINTER(B.C.c_int32)
    rows = []
    for n in (1, 2, 4, 8, 16, 32, 64, 128, 256):
        pg, ph = rng.permutation(nb).astype(np.int32), rng.permutation(nb).astype(np.int32)
        og, ig, oh, ih = (np.ascontiguousarray(x) for x in (pg[:n], pg[n:2 * n], ph[:n], ph[n:2 * n]))
        raw = (og.ctypes.data_as(i32p), oh.ctypes.data_as(i32p), n, ih.ctypes.data_as(i32p), ig.ctypes.data_as(i32p), n)
        rec = {"blocks_each_way": n, "mib_each_way": n * shape.block_bytes / M}
        for name, pid in (("auto", B.KV_PATH_AUTO), ("staged", B.KV_PATH_STAGED), ("zerocopy", B.KV_PATH_ZEROCOPY),
                          ("ce2d", B.KV_PATH_CE2D), ("auto_untimed", B.KV_PATH_AUTO)):
            pool.kv_pool_set_path(pid, pid)
            pool.kv_pool_set_call_timing(name != "auto_untimed")       # last column: no per-call start events
            ts, issue = [], []
            for k in range(45):
                t0 = time.perf_counter()
                pool.kv_rotate_raw(*raw)
                t1 = time.perf_counter()
                pool.kv_sync()
                t2 = time.perf_counter()
                if k >= 5:
                    ts.append((t2 - t0) * 1e6)
                    issue.append((t1 - t0) * 1e6)
            rec[name + "_us"] = round(float(np.median(ts)), 1)
            rec[name + "_issue_us"] = round(float(np.median(issue)), 1)
            if name == "auto":
                rec["auto_took"] = B.PATH_NAMES[pool.kv_get_stats()["last_path_out"]]
        rec["link_floor_us"] = round(n * shape.block_bytes / 50e9 * 1e6, 1)       # payload at 50 GB/s per direction
        best = min(rec[k + "_us"] for k in ("staged", "zerocopy", "ce2d"))
        rec["auto_over_best_pct"] = round(100 * (rec["auto_us"] / best - 1), 1)
        rows.append(rec)
        _emit(rec, out)
    pool.destroy()
    print("\n| blocks each way | MiB each way | AUTO us (took; of which issuing) | staged us | zero-copy us | 2-D per block us | "
          "AUTO over the best fixed path | AUTO, call timing off, us | payload at 50 GB/s per direction, us |\n|---|---|---|---|---|---|---|---|---|")
    for r in rows:
        print(f"| {r['blocks_each_way']} | {r['mib_each_way']:g} | {r['auto_us']} ({r['auto_took']}; {r['auto_issue_us']}) | {r['staged_us']} | "
              f"{r['zerocopy_us']} | {r['ce2d_us']} | {r['auto_over_best_pct']} % | {r['auto_untimed_us']} | {r['link_floor_us']} |")


def lvf(out, b_xfer: int, n_steps: int) -> None:
    import numpy as np
    import torch
    w = W.config5_lvf(rate=8.0, params=W.LVFParams(b_xfer=b_xfer))
    shape = w.shape
    moving = [r for r in w.steps if r.n_out + r.n_in][:n_steps]
    dev = torch.empty(w.nb_gpu * shape.block_bytes, dtype=torch.uint8, device="cuda:0")
    pool = B.KVPool(shape.num_layers, shape.block_size, shape.kv_heads, shape.head_dim, w.nb_gpu, w.nb_host,
                    dev.data_ptr())
    ms, blocks, outs = [], [], []
    for r in moving:
        pool.kv_rotate(r.out_gpu, r.out_host, r.in_host, r.in_gpu)
        pool.kv_sync()
        ms.append(pool.kv_get_stats()["last_union_ms"])
        blocks.append(r.n_out + r.n_in)
        outs.append(r.n_out)
    pool.destroy()
    ms, blocks, outs = np.array(ms), np.array(blocks), np.array(outs)
    e = w.extra
    rec = {"b_xfer": b_xfer, "steps_total": len(w.steps), "steps_that_move_blocks": int(sum(1 for r in w.steps if r.n_out + r.n_in)),
           "steps_timed": len(ms), "blocks_per_step_median": float(np.median(blocks)), "blocks_per_step_max": int(blocks.max()),
           "blocks_out_per_step_max": int(outs.max()), "ms_median": round(float(np.median(ms)), 2),
           "ms_p99": round(float(np.percentile(ms, 99)), 2), "ms_max": round(float(ms.max()), 2),
           "gbs_overall": round(float(blocks.sum() * shape.block_bytes / ms.sum() / 1e6), 1),
           "steps_over_70ms": int((ms > 70.0).sum()), "share_over_70ms": round(float((ms > 70.0).mean()), 4),
           "preempted_requests": int(e["preempted"].sum()), "resumed_requests": int(e["resumed"].sum()),
           "admitted_requests": int(e["admitted"].sum()), "arrivals": int(e["arrivals"])}
    _emit(rec, out)
    print("\n| B_xfer | steps that move blocks (of 2000) | timed | blocks per step, median / max | ms median | ms p99 | ms max | GB/s overall | steps over 70 ms | requests preempted / resumed / admitted |\n|---|---|---|---|---|---|---|---|---|---|")
    print(f"| {b_xfer} | {rec['steps_that_move_blocks']} | {rec['steps_timed']} | {rec['blocks_per_step_median']:.0f} / {rec['blocks_per_step_max']} | {rec['ms_median']} | "
          f"{rec['ms_p99']} | {rec['ms_max']} | {rec['gbs_overall']} | {rec['steps_over_70ms']} ({100 * rec['share_over_70ms']:.1f} %) | "
          f"{rec['preempted_requests']} / {rec['resumed_requests']} / {rec['admitted_requests']} |")


def lvf_table(out, b_xfer: int, n_steps: int, eager_blocks: int) -> None:
    import numpy as np
    import torch
    shape = W.SHAPE_8B
    bs = shape.block_size
    params = W.LVFParams(b_xfer=b_xfer)
    # the arrivals, lengths and pool sizes of workload.config5_lvf (same seed, same draws)
    rng = np.random.default_rng(W.MASTER_SEED + 6)
    rate, duration_s, step_s, max_tokens = 8.0, 120.0, 0.070, 8192
    n_arr = max(1, int(rng.poisson(rate * duration_s)))
    arrive = np.sort(rng.uniform(0.0, duration_s, size=n_arr))
    prompt = W.lognormal_tokens(rng, n_arr, 512, 1, max_tokens)
    output = W.lognormal_tokens(rng, n_arr, 256, 1, max_tokens)
    nblk = lambda tokens: -(-int(tokens) // bs)
    a_step = np.floor(arrive / step_s).astype(np.int64)
    horizon = int(a_step.max() + output.max() + 2)
    delta = np.zeros(horizon + 1, np.int64)
    for s_, p_, o_ in zip(a_step, prompt, output):
        delta[s_] += nblk(p_ + o_)
        delta[min(horizon, s_ + int(o_))] -= nblk(p_ + o_)
    demand = int(np.cumsum(delta).max())
    nb_gpu = max(int(0.40 * demand), nblk((prompt + output).max()) + 8)
    nb_host = max(2 * demand, 64)
    dev = torch.empty(nb_gpu * shape.block_bytes, dtype=torch.uint8, device="cuda:0")
    pool = B.KVPool(shape.num_layers, shape.block_size, shape.kv_heads, shape.head_dim, nb_gpu, nb_host, dev.data_ptr())
    table = B.KVTable(pool)
    running, rotary, waiting, remaining = {}, {}, [], {}
    ms, moved_out, moved_in, discarded, eager_sent, eager_ms = [], [], [], [], [], []
    nxt, step = 0, 0
    while len(ms) < n_steps and step < 2000:
        t_now = step * step_s
        while nxt < n_arr and a_step[nxt] <= step:
            waiting.append(nxt)
            nxt += 1
        for rid in [r for r in running if remaining[r] <= 0]:
            del running[rid]
            table.kv_req_finish(rid)
        info = {r: table.kv_req_info(r) for r in list(running) + list(rotary)}
        grow_need = sum(1 for r in running if info[r]["tokens"] % bs == 0)
        st0 = table.kv_table_get_stats()
        b_hbm = max(0, st0["free_gpu_blocks"] - grow_need)
        reqs = [(r, "running", W.vlt("running", t_now, t0, params), info[r]["num_blocks"]) for r, t0 in running.items()]
        reqs += [(r, "waiting", W.vlt("waiting", t_now, float(arrive[r]), params), nblk(prompt[r])) for r in waiting]
        reqs += [(r, "rotary", W.vlt("rotary", t_now, t0, params), info[r]["num_blocks"]) for r, t0 in rotary.items()]
        preempt, prio = W.lvf_select(reqs, b_hbm, params.b_xfer)
        resume = [r for r in prio if r in rotary]
        admit = [r for r in prio if r not in rotary]
        # the table lets resuming requests take what the preempted ones release; it refuses what does not fit
        while True:
            rc = table.kv_req_rotate(preempt, resume, check=False)
            if rc == B.KV_OK or not resume:
                break
            resume.pop()
        if rc != B.KV_OK:
            raise RuntimeError(f"kv_req_rotate failed: {rc}")
        pool.kv_sync()
        st1 = table.kv_table_get_stats()
        out_b = st1["preempt_blocks_moved"] - st0["preempt_blocks_moved"]
        in_b = st1["resume_blocks_moved"] - st0["resume_blocks_moved"]
        if out_b + in_b:
            ms.append(pool.kv_get_stats()["last_union_ms"])
            moved_out.append(out_b)
            moved_in.append(in_b)
            discarded.append(st1["discarded_blocks"] - st0["discarded_blocks"])
        for rid in preempt:
            del running[rid]
            rotary[rid] = t_now
        for rid in resume:
            del rotary[rid]
            running[rid] = t_now
        for rid in admit:
            if table.kv_req_add(rid, int(prompt[rid]), check=False) == B.KV_OK:
                waiting.remove(rid)
                remaining[rid] = int(output[rid])
                running[rid] = t_now
        for rid in running:
            if table.kv_req_append(rid, 1, check=False) == B.KV_OK:
                remaining[rid] -= 1
        if eager_blocks > 0:
            n_sent = table.kv_eager_rotate(eager_blocks)
            pool.kv_sync()
            if n_sent:
                eager_sent.append(n_sent)
                eager_ms.append(pool.kv_get_stats()["last_union_ms"])
        step += 1
    table.destroy()
    pool.destroy()
    ms, mo, mi, dc = (np.array(x, float) for x in (ms, moved_out, moved_in, discarded))
    rec = {"b_xfer": b_xfer, "eager_blocks_per_step": eager_blocks, "steps_run": step, "rotations_timed": len(ms),
           "blocks_out_per_rotation_median": float(np.median(mo)), "blocks_in_per_rotation_median": float(np.median(mi)),
           "blocks_discarded_per_rotation_median": float(np.median(dc)),
           "blocks_out_total": int(mo.sum()), "blocks_discarded_total": int(dc.sum()), "blocks_in_total": int(mi.sum()),
           "rotation_ms_median": round(float(np.median(ms)), 2), "rotation_ms_p99": round(float(np.percentile(ms, 99)), 2),
           "rotation_ms_max": round(float(ms.max()), 2), "rotations_over_70ms": int((ms > 70.0).sum()),
           "background_blocks_total": int(np.sum(eager_sent)) if eager_sent else 0,
           "background_ms_median": round(float(np.median(eager_ms)), 2) if eager_ms else None}
    _emit(rec, out)
    print("\n| B_xfer | background blocks per step | rotations timed | blocks out / discarded / in per rotation (median) | blocks out / discarded / in, total | "
          "rotation ms median | p99 | max | over 70 ms | background copies: blocks, median ms per step |\n|---|---|---|---|---|---|---|---|---|---|")
    print(f"| {b_xfer} | {eager_blocks} | {rec['rotations_timed']} | {rec['blocks_out_per_rotation_median']:.0f} / {rec['blocks_discarded_per_rotation_median']:.0f} / "
          f"{rec['blocks_in_per_rotation_median']:.0f} | {rec['blocks_out_total']} / {rec['blocks_discarded_total']} / {rec['blocks_in_total']} | {rec['rotation_ms_median']} | "
          f"{rec['rotation_ms_p99']} | {rec['rotation_ms_max']} | {rec['rotations_over_70ms']} | {rec['background_blocks_total']}, {rec['background_ms_median']} |")


def handoff(out) -> None:
    import torch
    dev = "cuda:0"
    hsrc = torch.empty(256 * M, dtype=torch.uint8).pin_memory()
    hdst = torch.empty(1024 * M, dtype=torch.uint8).pin_memory()
    dsrc = torch.empty(1024 * M, dtype=torch.uint8, device=dev)
    ddst = torch.empty(256 * M, dtype=torch.uint8, device=dev)
    small = torch.zeros(1024, device=dev)
    s_a, s_b, s_k = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()

    def median_of(fn, reps=7):
        res = sorted((fn() for _ in range(reps)), key=lambda r: r[1])
        return res[len(res) // 2]

    def copy_then_kernel(size_mib, busy, same_stream):
        torch.cuda.synchronize()
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        if busy:
            with torch.cuda.stream(s_b):
                hdst.copy_(dsrc, non_blocking=True)                # 1 GiB device to host: outlasts everything below
        with torch.cuda.stream(s_a):
            e0.record()
            ddst[:size_mib * M].copy_(hsrc[:size_mib * M], non_blocking=True)
            e1.record()
            if same_stream:
                small.add_(1)
                e2.record()
        if not same_stream:
            s_k.wait_event(e1)
            with torch.cuda.stream(s_k):
                small.add_(1)
                e2.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1), e1.elapsed_time(e2)

    def kernel_then_copy(size_mib, busy, same_stream):
        torch.cuda.synchronize()
        e0, e1, e2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        if busy:
            with torch.cuda.stream(s_b):
                for _ in range(4):
                    ddst.copy_(hsrc, non_blocking=True)            # 1 GiB host to device in all
        with torch.cuda.stream(s_a if same_stream else s_k):
            e0.record()
            small.add_(1)
            e1.record()
        if not same_stream:
            s_a.wait_event(e1)
        with torch.cuda.stream(s_a):
            hdst[:size_mib * M].copy_(dsrc[:size_mib * M], non_blocking=True)
            e2.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1), e1.elapsed_time(e2)

    rows = []
    for size in (16, 64):
        for busy in (False, True):
            for same in (False, True):
                c, h = median_of(lambda: copy_then_kernel(size, busy, same))
                k, t = median_of(lambda: kernel_then_copy(size, busy, same))
                rate = (55.5e9 if not busy else 49.5e9), (57.2e9 if not busy else 49.5e9)
                rec = {"copy_mib": size, "other_direction_busy": busy, "same_stream": same,
                       "h2d_copy_ms": round(c, 3), "h2d_copy_end_to_kernel_end_us": round(h * 1e3, 1),
                       "kernel_end_to_d2h_copy_end_ms": round(t, 3),
                       "of_which_before_the_copy_starts_us": round((t - size * M / rate[1] * 1e3) * 1e3, 1)}
                rows.append(rec)
                _emit(rec, out)
    print("\n| copy MiB | other direction | streams | H2D copy ms | copy end to kernel end us | kernel end to D2H copy end ms | of which before the copy starts, us (copy at the probe's rate) |\n|---|---|---|---|---|---|---|")
    for r in rows:
        print(f"| {r['copy_mib']} | {'saturated' if r['other_direction_busy'] else 'idle'} | {'one' if r['same_stream'] else 'two'} | {r['h2d_copy_ms']} | "
              f"{r['h2d_copy_end_to_kernel_end_us']} | {r['kernel_end_to_d2h_copy_end_ms']} | {r['of_which_before_the_copy_starts_us']} |")


def budget(out, b_xfer: int) -> None:
    import numpy as np
    import torch
    w = W.config5_replay(rate=8.0)
    shape = w.shape
    steps = W.budgeted_steps(w.steps, b_xfer)
    dev = torch.empty(w.nb_gpu * shape.block_bytes, dtype=torch.uint8, device="cuda:0")
    pool = B.KVPool(shape.num_layers, shape.block_size, shape.kv_heads, shape.head_dim, w.nb_gpu, w.nb_host,
                    dev.data_ptr())
    ms, blocks = [], []
    for r in steps:
        if r.n_out + r.n_in == 0:
            continue
        pool.kv_rotate(r.out_gpu, r.out_host, r.in_host, r.in_gpu)
        pool.kv_sync()
        ms.append(pool.kv_get_stats()["last_union_ms"])
        blocks.append(r.n_out + r.n_in)
    pool.destroy()
    ms, blocks = np.array(ms), np.array(blocks)
    full = blocks >= b_xfer
    rec = {"b_xfer": b_xfer, "original_steps": len(w.steps), "emitted_steps": len(steps), "steps_that_move_blocks": len(ms),
           "blocks_moved": int(blocks.sum()), "steps_at_budget": int(full.sum()),
           "ms_median": round(float(np.median(ms)), 2), "ms_p99": round(float(np.percentile(ms, 99)), 2),
           "ms_max": round(float(ms.max()), 2), "ms_median_at_budget": round(float(np.median(ms[full])), 2) if full.any() else None,
           "gbs_at_budget": round(float(np.median(blocks[full] * shape.block_bytes / ms[full] / 1e6)), 1) if full.any() else None,
           "steps_over_70ms": int((ms > 70.0).sum()), "share_over_70ms": round(float((ms > 70.0).mean()), 4)}
    _emit(rec, out)
    print("\n| B_xfer | emitted steps | steps that move blocks | at budget | median ms | p99 ms | max ms | median ms at budget | "
          "GB/s at budget | steps over 70 ms |\n|---|---|---|---|---|---|---|---|---|---|")
    print(f"| {b_xfer} | {rec['emitted_steps']} | {rec['steps_that_move_blocks']} | {rec['steps_at_budget']} | {rec['ms_median']} | "
          f"{rec['ms_p99']} | {rec['ms_max']} | {rec['ms_median_at_budget']} | {rec['gbs_at_budget']} | "
          f"{rec['steps_over_70ms']} ({100 * rec['share_over_70ms']:.2f} %) |")


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("what", choices=["probe", "paths", "segments", "overlap", "latency", "budget", "handoff", "lvf", "lvf-table"])
    ap.add_argument("--eager-blocks", type=int, default=0, help="lvf-table: full blocks copied out in the background per step")
    ap.add_argument("--steps", type=int, default=300, help="lvf: steps to time")
    ap.add_argument("--out", default=None)
    ap.add_argument("--max-payload-gb", type=float, default=4.0)
    ap.add_argument("--b-xfer", type=int, default=2400, help="budget: blocks per step, both directions together")
    ap.add_argument("--block-size", type=int, default=16, help="latency: tokens per block (8 = 1 MiB blocks, 16 = 2 MiB, 32 = 4 MiB)")
    ap.add_argument("--device-layout", choices=["layer-first", "block-first"], default="layer-first",
                    help="paths: device pool layout (block-first = the paper's redesigned storage order)")
    ap.add_argument("--pool-gib", type=int, default=4, help="segments: device pool size in GiB")
    ap.add_argument("--kv-heads", type=int, default=8,
                    help="paths, latency: KV heads held by this GPU (8 = the whole 8B shape; 1, 2 or 4 = one rank's shard under tensor parallelism)")
    a = ap.parse_args()
    import torch
    if not torch.cuda.is_available():
        sys.exit("sweep needs a CUDA device")
    out = open(a.out, "w") if a.out else None
    if a.what == "probe":
        probe(out)
    elif a.what == "paths":
        paths(out, a.max_payload_gb, 1 if a.device_layout == "block-first" else 0, a.kv_heads)
    elif a.what == "segments":
        segments(out, a.pool_gib)
    elif a.what == "overlap":
        overlap(out)
    elif a.what == "latency":
        latency(out, a.block_size, a.kv_heads)
    elif a.what == "handoff":
        handoff(out)
    elif a.what == "lvf":
        lvf(out, a.b_xfer, a.steps)
    elif a.what == "lvf-table":
        lvf_table(out, a.b_xfer, a.steps, a.eager_blocks)
    else:
        budget(out, a.b_xfer)


if __name__ == "__main__":
    main()
