"""Seeded synthetic inputs for the KV rotation path: pool contents and rotation lists.

This module only *makes inputs*.  It holds none of the path's address arithmetic or
data movement, imports neither the CUDA binding nor the CPU oracle, and is the one
piece both of them are fed from.

Two kinds of input:

* Pool contents.  ``block_words(seed, pool, b, words)`` is a counter-based generator:
  the logical content of block ``b`` of pool ``pool`` is a pure function of
  ``(seed, pool, b)``, independent of where the block sits in memory.  Each 64-bit
  hash output selects four entries of a 65 536-entry table of bf16 bit patterns whose
  values follow N(0, 1) (``normal_bf16_lut``).  Integer-only, so the same generator
  written again for the GPU gives identical bits.

* Rotation lists.  Requests with skewed lengths own scattered block ids handed out by
  a seeded free-list allocator; a rotation names the blocks of the requests that leave
  the GPU (with fresh host ids) and of those that come back (with GPU ids taken from
  the free list *before* the leaving requests' blocks are released, so that swap-in
  destinations never alias swap-out sources).  The paper drives its engine with a
  scheduler over ShareGPT / LMSYS-Chat-1M traces at Poisson arrivals; those traces are
  not used here, only their shape: many requests, lognormal lengths, scattered blocks.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

MASTER_SEED = 20260120

POOL_GPU = 0
POOL_HOST = 1

_M64 = np.uint64(0xFFFFFFFFFFFFFFFF)
_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_POOLMUL = np.uint64(0xD1B54A32D192ED03)
_C1 = np.uint64(0xBF58476D1CE4E5B9)
_C2 = np.uint64(0x94D049BB133111EB)


# --------------------------------------------------------------------------- pool contents

def normal_bf16_lut() -> np.ndarray:
    """65 536 bf16 bit patterns: entry k is the normal quantile of (k + 1/2) / 65536.

    Quantiles are computed in float64, narrowed to float32, then to bf16 with
    round-to-nearest-even on the bit pattern.
    """
    from scipy.special import ndtri
    k = np.arange(65536, dtype=np.float64)
    q = ndtri((k + 0.5) / 65536.0).astype(np.float32)
    u = q.view(np.uint32).astype(np.uint64)
    r = (u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) >> np.uint64(16)
    return r.astype(np.uint16)


_LUT: Optional[np.ndarray] = None


def lut() -> np.ndarray:
    global _LUT
    if _LUT is None:
        _LUT = normal_bf16_lut()
    return _LUT


def mix64(key: np.ndarray) -> np.ndarray:
    """splitmix64 output function applied to an array of 64-bit counters."""
    with np.errstate(over="ignore"):
        z = (key + _GOLDEN) & _M64
        z = ((z ^ (z >> np.uint64(30))) * _C1) & _M64
        z = ((z ^ (z >> np.uint64(27))) * _C2) & _M64
        z = z ^ (z >> np.uint64(31))
    return z


def block_key_base(seed: int, pool: int, b: int, words_per_block: int) -> np.uint64:
    """Counter of the first 4-word group of block ``b``; group q adds q."""
    groups = words_per_block // 4
    with np.errstate(over="ignore"):
        return (np.uint64(seed) * _GOLDEN + np.uint64(pool) * _POOLMUL
                + np.uint64(b) * np.uint64(groups)) & _M64


def block_words(seed: int, pool: int, b: int, words_per_block: int,
                table: Optional[np.ndarray] = None) -> np.ndarray:
    """Logical content of one block: ``words_per_block`` uint16 in (layer, K|V, token, head, dim) order."""
    assert words_per_block % 4 == 0
    table = lut() if table is None else table
    groups = words_per_block // 4
    with np.errstate(over="ignore"):
        key = block_key_base(seed, pool, b, words_per_block) + np.arange(groups, dtype=np.uint64)
    z = mix64(key)
    out = np.empty((groups, 4), np.uint16)
    for k in range(4):
        out[:, k] = table[((z >> np.uint64(16 * k)) & np.uint64(0xFFFF)).astype(np.int64)]
    return out.reshape(-1)


def blocks_words(seed: int, pool: int, ids: Sequence[int], words_per_block: int) -> np.ndarray:
    """Stack of ``block_words`` for several blocks, shape (len(ids), words_per_block)."""
    return np.stack([block_words(seed, pool, int(b), words_per_block) for b in ids]) if len(ids) else \
        np.empty((0, words_per_block), np.uint16)


# --------------------------------------------------------------------------- shapes

@dataclass(frozen=True)
class KVShape:
    num_layers: int
    block_size: int
    kv_heads: int = 8
    head_dim: int = 128

    @property
    def words_per_plane(self) -> int:
        return self.block_size * self.kv_heads * self.head_dim

    @property
    def words_per_block(self) -> int:
        return 2 * self.num_layers * self.words_per_plane

    @property
    def block_bytes(self) -> int:
        return 2 * self.words_per_block


SHAPE_TINY = KVShape(2, 16)
SHAPE_8B = KVShape(32, 16)
SHAPE_70B = KVShape(80, 16)


def blocks_for_bytes(shape: KVShape, pool_bytes: float) -> int:
    return int(pool_bytes // shape.block_bytes)


# --------------------------------------------------------------------------- allocator and request table

class FreeList:
    """Free block ids of one pool.

    Scattered mode keeps the free ids in a uniformly random order: ``take`` pops from the
    end, ``give`` inserts each returned id at a random position, so every table handed out
    is a random sample with no locality.  Contiguous mode keeps them ascending and hands
    out the lowest ids.
    """

    def __init__(self, num_blocks: int, rng: np.random.Generator, scattered: bool = True):
        self.num_blocks = num_blocks
        self.rng = rng
        self.scattered = scattered
        self._buf = np.arange(num_blocks, dtype=np.int32)
        self._n = num_blocks
        if scattered:
            rng.shuffle(self._buf)

    def __len__(self):
        return self._n

    @property
    def free(self) -> np.ndarray:
        return self._buf[:self._n]

    def take(self, n: int) -> np.ndarray:
        if n > self._n:
            raise MemoryError(f"pool exhausted: want {n}, have {self._n}")
        if self.scattered:
            ids = self._buf[self._n - n:self._n][::-1].copy()
            self._n -= n
        else:
            ids = self._buf[:n].copy()
            self._buf[:self._n - n] = self._buf[n:self._n]
            self._n -= n
        return ids

    def give(self, ids: np.ndarray) -> None:
        ids = np.asarray(ids, np.int32)
        k = len(ids)
        assert self._n + k <= self.num_blocks
        if not self.scattered:
            self._buf[self._n:self._n + k] = ids
            self._n += k
            self._buf[:self._n].sort()
            return
        pos = self.rng.integers(0, self._n + 1 + np.arange(k))      # insertion point of each id
        for b, j in zip(ids.tolist(), pos.tolist()):
            self._buf[self._n] = self._buf[j]
            self._buf[j] = b
            self._n += 1

    def fragment(self, rounds: int = 4) -> None:
        """Allocate and release random subsets a few times.  The free *set* is unchanged by
        construction; what this models is a pool whose free ids are an arbitrary subset in
        arbitrary order, so the tables handed out afterwards have no locality."""
        for _ in range(rounds):
            n = int(self.rng.integers(self._n // 4, self._n // 2 + 1))
            held = self.take(n)
            self.give(held)


@dataclass
class Request:
    rid: int
    tokens: int
    where: str                      # "gpu" | "host" | "none"
    blocks: np.ndarray              # ids in the pool named by ``where``
    origin: List[Tuple[int, int]] = field(default_factory=list)   # (origin pool, origin block) per block


@dataclass
class Rotation:
    """Paired lists of one rotate call, plus request boundaries (for per-request statistics)."""
    out_gpu: np.ndarray
    out_host: np.ndarray
    in_host: np.ndarray
    in_gpu: np.ndarray
    out_req_offsets: np.ndarray
    in_req_offsets: np.ndarray

    @property
    def n_out(self) -> int:
        return len(self.out_gpu)

    @property
    def n_in(self) -> int:
        return len(self.in_gpu)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _empty_rotation() -> Rotation:
    e = np.empty(0, np.int32)
    z = np.zeros(1, np.int64)
    return Rotation(e, e.copy(), e.copy(), e.copy(), z, z.copy())


class RequestTable:
    """Requests, their residency and block tables over two pools.

    ``rotate(out_rids, in_rids)`` moves whole requests: incoming requests get GPU ids from
    the free list first, outgoing requests get fresh host ids, and only then are the old
    ids of both released.  Returns the lists that describe the move.
    """

    def __init__(self, shape: KVShape, nb_gpu: int, nb_host: int, rng: np.random.Generator,
                 scattered: bool = True):
        self.shape = shape
        self.nb_gpu, self.nb_host = nb_gpu, nb_host
        self.rng = rng
        self.gpu_free = FreeList(nb_gpu, rng, scattered)
        self.host_free = FreeList(nb_host, rng, scattered)
        self.requests: Dict[int, Request] = {}

    def blocks_for(self, tokens: int) -> int:
        return -(-tokens // self.shape.block_size)

    def add(self, rid: int, tokens: int, where: str) -> Request:
        n = self.blocks_for(tokens)
        fl = self.gpu_free if where == "gpu" else self.host_free
        ids = fl.take(n)
        pool = POOL_GPU if where == "gpu" else POOL_HOST
        r = Request(rid, tokens, where, ids, [(pool, int(b)) for b in ids])
        self.requests[rid] = r
        return r

    def grow(self, rid: int, new_tokens: int) -> None:
        """Decode-length growth of a GPU-resident request; a new block holds whatever the pool held."""
        r = self.requests[rid]
        assert r.where == "gpu"
        need = self.blocks_for(new_tokens) - len(r.blocks)
        if need > 0:
            ids = self.gpu_free.take(need)
            r.blocks = np.concatenate([r.blocks, ids])
            r.origin += [None] * need          # content undefined until written by the model
        r.tokens = new_tokens

    def finish(self, rid: int) -> None:
        r = self.requests.pop(rid)
        (self.gpu_free if r.where == "gpu" else self.host_free).give(r.blocks)

    def rotate(self, out_rids: Sequence[int], in_rids: Sequence[int]) -> Rotation:
        in_gpu, in_host, in_off = [], [], [0]
        new_gpu = {}
        for rid in in_rids:
            r = self.requests[rid]
            assert r.where == "host"
            ids = self.gpu_free.take(len(r.blocks))
            new_gpu[rid] = ids
            in_host.append(r.blocks)
            in_gpu.append(ids)
            in_off.append(in_off[-1] + len(ids))
        out_gpu, out_host, out_off = [], [], [0]
        new_host = {}
        for rid in out_rids:
            r = self.requests[rid]
            assert r.where == "gpu"
            ids = self.host_free.take(len(r.blocks))
            new_host[rid] = ids
            out_gpu.append(r.blocks)
            out_host.append(ids)
            out_off.append(out_off[-1] + len(ids))
        for rid in in_rids:
            r = self.requests[rid]
            self.host_free.give(r.blocks)
            r.blocks, r.where = new_gpu[rid], "gpu"
        for rid in out_rids:
            r = self.requests[rid]
            self.gpu_free.give(r.blocks)
            r.blocks, r.where = new_host[rid], "host"
        cat = lambda xs: _i32(np.concatenate(xs)) if xs else np.empty(0, np.int32)
        return Rotation(cat(out_gpu), cat(out_host), cat(in_host), cat(in_gpu),
                        np.asarray(out_off, np.int64), np.asarray(in_off, np.int64))

    def check_consistent(self) -> None:
        """Every request has one residency, the right table length, pool-wide unique ids,
        and free + used covers each pool exactly once."""
        for pool, fl, nb in (("gpu", self.gpu_free, self.nb_gpu), ("host", self.host_free, self.nb_host)):
            used = [r.blocks for r in self.requests.values() if r.where == pool]
            allids = np.concatenate(used + [fl.free]) if used else fl.free
            assert len(allids) == nb, (pool, len(allids), nb)
            assert len(np.unique(allids)) == nb, pool
        for r in self.requests.values():
            assert r.where in ("gpu", "host")
            assert len(r.blocks) == self.blocks_for(r.tokens)


def lognormal_tokens(rng: np.random.Generator, n: int, median: float, lo: int, hi: int,
                     sigma: float = 1.0) -> np.ndarray:
    t = np.rint(np.exp(rng.normal(np.log(median), sigma, size=n)))
    return np.clip(t, lo, hi).astype(np.int64)


# --------------------------------------------------------------------------- the five workloads

@dataclass
class Workload:
    name: str
    shape: KVShape
    nb_gpu: int
    nb_host: int
    seed: int
    table: RequestTable
    steps: List[Rotation]
    extra: dict = field(default_factory=dict)


def config1_tiny(seed: int = MASTER_SEED + 1) -> Workload:
    """2 layers, block_size 16; GPU pool 256 blocks, host pool 512; 8 requests of 4-20 blocks,
    four resident on each side, random-permuted tables; one rotation moving 4 out and 4 in."""
    rng = np.random.default_rng(seed)
    shape = SHAPE_TINY
    tab = RequestTable(shape, 256, 512, rng)
    nblocks = rng.integers(4, 21, size=8)
    for rid in range(8):
        tab.add(rid, int(nblocks[rid]) * shape.block_size, "gpu" if rid < 4 else "host")
    rot = tab.rotate([0, 1, 2, 3], [4, 5, 6, 7])
    return Workload("tiny", shape, 256, 512, seed, tab, [rot])


def deal_balanced(lengths: Sequence[int], n_groups: int) -> List[List[int]]:
    """Split items into ``n_groups`` groups of equal count and similar total: longest first, each
    to the group with the smallest total that still has room.  A rotation frees about as many
    blocks as it brings in (that is what a scheduler preempts for), so the groups of requests
    that swap places should carry similar payloads."""
    lengths = np.asarray(lengths)
    cap = -(-len(lengths) // n_groups)
    order = np.argsort(-lengths, kind="stable")
    groups: List[List[int]] = [[] for _ in range(n_groups)]
    totals = [0] * n_groups
    for idx in order:
        open_groups = [g for g in range(n_groups) if len(groups[g]) < cap]
        g = min(open_groups, key=lambda q: (totals[q], q))
        groups[g].append(int(idx))
        totals[g] += int(lengths[idx])
    return groups


def config2_8b(seed: int = MASTER_SEED + 2, nb_gpu: Optional[int] = None, nb_host: Optional[int] = None,
               shape: KVShape = SHAPE_8B, n_req: int = 64, median: int = 1024, max_tokens: int = 8192,
               n_rot: int = 16) -> Workload:
    """8B-shaped KV; 64 requests with lognormal lengths (median 1k tokens, max 8k), half resident
    on each side.  ``steps[0]`` is the paired rotation of 16 requests each way; ``extra`` holds the
    single swap-out / swap-in lists (median-length and longest request) and one-pair-at-a-time
    rotations of every request (first the other 32, then the 32 of the paired rotation on their way
    back) for per-request latency."""
    rng = np.random.default_rng(seed)
    nb_gpu = blocks_for_bytes(shape, 60e9) if nb_gpu is None else nb_gpu
    nb_host = blocks_for_bytes(shape, 120e9) if nb_host is None else nb_host
    tab = RequestTable(shape, nb_gpu, nb_host, rng)
    toks = lognormal_tokens(rng, n_req, median, shape.block_size, max_tokens)
    # four groups: two resident on the GPU, two on the host; the first of each pair rotates
    g_rot, h_rot, g_rest, h_rest = deal_balanced(toks, 4)
    g_rot, h_rot = g_rot[:n_rot], h_rot[:n_rot]
    gpu_rids = g_rot + g_rest
    host_rids = h_rot + h_rest
    for rid in range(n_req):
        tab.add(rid, int(toks[rid]), "gpu" if rid in gpu_rids else "host")

    # single swaps: median-length and longest request of each side (lists only; residency unchanged,
    # destinations drawn from the free lists and returned at once)
    def single(rids, side):
        lens = [len(tab.requests[r].blocks) for r in rids]
        order = np.argsort(lens, kind="stable")
        picks = {"median": rids[int(order[len(order) // 2])], "longest": rids[int(order[-1])]}
        out = {}
        for k, rid in picks.items():
            r = tab.requests[rid]
            fl = tab.host_free if side == "gpu" else tab.gpu_free
            dst = fl.take(len(r.blocks))
            fl.give(dst)
            out[k] = (_i32(r.blocks), _i32(dst))
        return out
    extra = {"single_out": single(gpu_rids, "gpu"), "single_in": single(host_rids, "host")}
    rot = tab.rotate(g_rot, h_rot)
    extra["pairs"] = [tab.rotate([a], [b]) for a, b in zip(g_rest, h_rest)]
    # ... and the requests of the paired rotation change places once more, one pair at a time, so that
    # all ``n_req`` requests take part in a one-request-each-way rotation (per-request latency sample)
    extra["pairs"] += [tab.rotate([b], [a]) for a, b in zip(g_rot, h_rot)]
    extra["tokens"] = toks
    return Workload("8b", shape, nb_gpu, nb_host, seed, tab, [rot], extra)


def config3_70b(seed: int = MASTER_SEED + 3, nb_gpu: Optional[int] = None, nb_host: Optional[int] = None,
                shape: KVShape = SHAPE_70B, n_req: int = 32, median: int = 2048, max_tokens: int = 16384,
                n_steps: int = 100, per_step: int = 8) -> Workload:
    """70B-shaped KV; 32 requests (median 2k tokens, max 16k); GPU pool fragmented by random
    allocation; every step rotates 8 requests out and 8 in, round-robin: each side is a queue,
    the 8 at the front change sides and join the back of the other queue."""
    rng = np.random.default_rng(seed)
    nb_gpu = blocks_for_bytes(shape, 60e9) if nb_gpu is None else nb_gpu
    nb_host = blocks_for_bytes(shape, 120e9) if nb_host is None else nb_host
    tab = RequestTable(shape, nb_gpu, nb_host, rng)
    tab.gpu_free.fragment()
    toks = lognormal_tokens(rng, n_req, median, shape.block_size, max_tokens)
    groups = deal_balanced(toks, max(2, n_req // per_step))
    half = len(groups) // 2
    gpu_q = [rid for g in groups[:half] for rid in g]
    host_q = [rid for g in groups[half:] for rid in g]
    for rid in range(n_req):
        tab.add(rid, int(toks[rid]), "gpu" if rid in gpu_q else "host")
    steps = []
    for _ in range(n_steps):
        outs, gpu_q = gpu_q[:per_step], gpu_q[per_step:]
        ins, host_q = host_q[:per_step], host_q[per_step:]
        steps.append(tab.rotate(outs, ins))
        gpu_q += ins
        host_q += outs
    return Workload("70b", shape, nb_gpu, nb_host, seed, tab, steps, {"tokens": toks})


def config4_sweep_case(block_size: int, contiguous: bool, payload_bytes: float,
                       seed: int = MASTER_SEED + 4, nb_gpu: Optional[int] = None,
                       nb_host: Optional[int] = None, num_layers: int = 32, kv_heads: int = 8) -> Workload:
    """One cell of the block-size / fragmentation sweep on the 8B shape: ``payload_bytes`` per
    direction, block tables either ascending runs of ids or a uniformly random permutation.
    ``kv_heads`` below 8 gives the shard one rank of a tensor-parallel group would hold."""
    rng = np.random.default_rng(seed + block_size + (0 if contiguous else 1000))
    shape = KVShape(num_layers, block_size, kv_heads)
    n = max(1, int(payload_bytes // shape.block_bytes))
    nb_gpu = 2 * n + 16 if nb_gpu is None else nb_gpu
    nb_host = 2 * n + 16 if nb_host is None else nb_host
    tab = RequestTable(shape, nb_gpu, nb_host, rng, scattered=not contiguous)
    tab.add(0, n * block_size, "gpu")
    tab.add(1, n * block_size, "host")
    rot = tab.rotate([0], [1])
    return Workload(f"sweep_bs{block_size}_{'contig' if contiguous else 'random'}", shape,
                    nb_gpu, nb_host, seed, tab, [rot])


def config5_replay(seed: int = MASTER_SEED + 5, rate: float = 16.0, n_steps: int = 2000,
                   shape: KVShape = SHAPE_8B, duration_s: float = 120.0, step_s: float = 0.070,
                   nb_host: Optional[int] = None, cap: float = 0.40, max_tokens: int = 8192,
                   patience: int = 16) -> Workload:
    """Serving replay on the 8B shape: Poisson arrivals, lognormal prompt (median 512) and output
    (median 256) lengths, one token of growth per running request per step of 70 ms, GPU pool capped
    at 40 % of the peak demand an unconstrained run would have.  When free GPU blocks fall short of
    what the step needs (growth plus the prompts that arrived), the longest-running requests are
    swapped out in turn until a small reserve of free blocks is restored; parked requests return
    oldest first when there is room beyond the reserve, and one that has waited ``patience`` steps
    returns into the reserve while a running request is swapped out in the same step (a rotation).  No scheduling policy
    from the paper is used: this is a seeded list maker.  Steps with nothing to move are kept."""
    rng = np.random.default_rng(seed)
    n_arr = max(1, int(rng.poisson(rate * duration_s)))
    arrive = np.sort(rng.uniform(0.0, duration_s, size=n_arr))
    prompt = lognormal_tokens(rng, n_arr, 512, 1, max_tokens)
    output = lognormal_tokens(rng, n_arr, 256, 1, max_tokens)
    bs = shape.block_size
    nblk = lambda tokens: -(-int(tokens) // bs)
    # peak demand with nothing swapped: a request holds its final block count from arrival to finish
    a_step = np.floor(arrive / step_s).astype(np.int64)
    horizon = int(a_step.max() + output.max() + 2)
    delta = np.zeros(horizon + 1, np.int64)
    for s, p, o in zip(a_step, prompt, output):
        delta[s] += nblk(p + o)
        delta[min(horizon, s + int(o))] -= nblk(p + o)
    demand = int(np.cumsum(delta).max())
    nb_gpu = max(int(cap * demand), nblk((prompt + output).max()) + 8)
    nb_host = max(2 * demand, 64) if nb_host is None else nb_host
    tab = RequestTable(shape, nb_gpu, nb_host, rng)
    running: List[int] = []            # oldest-run first
    parked: List[Tuple[int, int]] = [] # (rid, step parked), oldest first
    waiting: List[int] = []
    remaining: Dict[int, int] = {}
    steps: List[Rotation] = []
    nxt = 0
    blocks_of = lambda rid: len(tab.requests[rid].blocks)
    reserve = max(nblk(max_tokens) // 2, nb_gpu // 25)
    for step in range(n_steps):
        while nxt < n_arr and a_step[nxt] <= step:
            waiting.append(nxt)
            nxt += 1
        for rid in [r for r in running if remaining[r] <= 0]:
            running.remove(rid)
            tab.finish(rid)
        grow_need = sum(1 for r in running if tab.requests[r].tokens % bs == 0)
        need = grow_need + sum(nblk(prompt[r]) for r in waiting)
        avail = len(tab.gpu_free) - need
        ins: List[int] = []
        # a parked request returns when there is true spare room, or, once it has waited
        # ``patience`` steps, by dipping into the reserve (the eviction below refills it)
        while parked and avail >= blocks_of(parked[0][0]) + 1 and (
                avail - reserve >= blocks_of(parked[0][0]) + 1 or step - parked[0][1] > patience):
            rid, _ = parked.pop(0)
            ins.append(rid)
            avail -= blocks_of(rid) + 1
        short = max(0, reserve - avail)
        outs: List[int] = []
        while short > 0 and len(outs) < len(running) - 1:
            rid = running[len(outs)]
            outs.append(rid)
            short -= blocks_of(rid)
        steps.append(tab.rotate(outs, ins) if (outs or ins) else _empty_rotation())
        for rid in outs:
            running.remove(rid)
            parked.append((rid, step))
        running.extend(ins)
        grow_need = sum(1 for r in running if tab.requests[r].tokens % bs == 0)
        while waiting and len(tab.gpu_free) - grow_need >= nblk(prompt[waiting[0]]):
            rid = waiting.pop(0)
            tab.add(rid, int(prompt[rid]), "gpu")
            remaining[rid] = int(output[rid])
            running.append(rid)
        for rid in running:
            if tab.requests[rid].tokens % bs == 0 and len(tab.gpu_free) == 0:
                continue                       # stalled this step: no block to grow into
            tab.grow(rid, tab.requests[rid].tokens + 1)
            remaining[rid] -= 1
    return Workload(f"replay_{rate:g}rps", shape, nb_gpu, nb_host, seed, tab, steps,
                    {"demand_blocks": demand, "arrivals": n_arr})


# --------------------------------------------------------------------------- transfer budget per step

def budgeted_steps(steps: Sequence[Rotation], b_xfer: int) -> List[Rotation]:
    """Re-time a list of rotations under a per-step transfer budget of ``b_xfer`` blocks (both directions
    together; the paper's scheduler bounds what one iteration may move by such a budget, 2400 blocks in
    its main runs, so that the transfer hides behind one model step).  Work that does not fit a step is
    carried over: the pairs of the incoming rotations are queued in arrival order (inside one rotation
    swap-outs and swap-ins alternate, so both directions stay busy) and every emitted step takes pairs
    from the front of the queue until the budget is used up, or until the next pair names a block that
    a pair of the other direction already taken for this step names too, or a destination already
    taken (a swap-in into device blocks that an earlier rotation's swap-out releases has to wait for the
    next step: one rotate call must not overlap across directions, nor write a block twice).  The queue is never reordered, so the emitted steps do to the pools
    exactly what the original ones did.  One emitted step per original step at least (idle steps stay),
    more at the end until the queue is empty."""
    assert b_xfer >= 1
    queue: List[Tuple[int, int, int]] = []     # (direction 0 = out / 1 = in, gpu id, host id)
    out: List[Rotation] = []

    def emit():
        taken = 0
        g_used = (set(), set())                # device / host ids named so far, per direction
        h_used = (set(), set())
        while taken < len(queue) and taken < b_xfer:
            d, g, h = queue[taken]
            if g in g_used[1 - d] or h in h_used[1 - d] or (h in h_used[0] if d == 0 else g in g_used[1]):
                break                          # other direction names it too, or a destination would repeat
            g_used[d].add(g)
            h_used[d].add(h)
            taken += 1
        part = queue[:taken]
        del queue[:taken]
        po = [p for p in part if p[0] == 0]
        pi = [p for p in part if p[0] == 1]
        z = np.zeros(1, np.int64)
        out.append(Rotation(_i32([p[1] for p in po]), _i32([p[2] for p in po]), _i32([p[2] for p in pi]),
                            _i32([p[1] for p in pi]), z, z.copy()))

    for r in steps:
        outs = [(0, int(g), int(h)) for g, h in zip(r.out_gpu, r.out_host)]
        ins = [(1, int(g), int(h)) for h, g in zip(r.in_host, r.in_gpu)]
        k = min(len(outs), len(ins))
        queue += [p for pair in zip(outs[:k], ins[:k]) for p in pair] + outs[k:] + ins[k:]
        emit()
    while queue:
        emit()
    return out


# --------------------------------------------------------------------------- lists made by the paper's scheduler
#
# The paper drives its rotation engine with a scheduler (section 4.2): every request has a Virtual Lag
# Time (VLT), and each engine iteration the Largest-VLT-First policy (Algorithm 1) picks the requests to
# bring onto the GPU and the running requests to preempt for them.  Here the policy is only a maker of
# rotation lists: a seeded toy loop over synthetic arrivals, no SLO study.

@dataclass(frozen=True)
class LVFParams:
    """Scheduler settings of the paper's evaluation (section 5.2): alpha = 3, beta_B = 0, beta_F = 0.5,
    B_xfer = 2400 blocks, first-token SLO 5 s, between-token SLO 100 ms.  ``slo_first_s`` is the S_F and
    ``slo_between_s`` the S_B of the VLT definition (F: first token, B: between tokens)."""
    alpha: float = 3.0
    beta_b: float = 0.0
    beta_f: float = 0.5
    slo_first_s: float = 5.0
    slo_between_s: float = 0.100
    b_xfer: int = 2400


def vlt(state: str, t_now: float, t_ref: float, p: LVFParams = LVFParams()) -> float:
    """Virtual Lag Time of one request (section 4.2, the piecewise definition).  ``t_ref`` is the time of
    the last generated token for a rotary request, the arrival time for a waiting one, and the time it
    entered the running state for a running one."""
    if state == "rotary":
        return p.alpha * max(0.0, t_now - t_ref - p.beta_b * p.slo_between_s)
    if state == "waiting":
        return max(0.0, t_now - t_ref - p.beta_f * p.slo_first_s)
    if state == "running":
        return -(t_now - t_ref)
    raise ValueError(state)


def lvf_select(requests: Sequence[Tuple[int, str, float, int]], b_hbm: int, b_xfer: int) -> Tuple[List[int], List[int]]:
    """One decision of Largest-VLT-First (Algorithm 1).  ``requests`` holds (id, state, VLT, blocks) with
    state in {"running", "waiting", "rotary"}; ``b_hbm`` is the number of free device blocks.  Returns
    (preempted ids, prioritized ids), each in the order the algorithm picks them.

    Steps, as the paper numbers them: (1) if the free blocks hold every waiting and rotary request, nothing
    is preempted and all of them are prioritized; (2) sort everything by VLT, largest first; (3) from the
    head, take waiting / rotary requests whose blocks still fit into ``b_hbm + b_xfer``; (4) the blocks
    needed beyond the free ones are ``B_swap``: from the tail, preempt running requests until that many
    are freed.  Equal VLTs keep the order of ``requests`` (a stable sort)."""
    idle = [r for r in requests if r[1] != "running"]
    if b_hbm >= sum(r[3] for r in idle):
        return [], [r[0] for r in idle]
    order = sorted(requests, key=lambda r: -r[2])
    left = b_hbm + b_xfer
    prioritized = []
    for rid, state, v, blk in order:
        if state != "running" and v >= 0 and blk <= left:
            prioritized.append(rid)
            left -= blk
    swap = b_xfer - left
    preempted = []
    for rid, state, v, blk in reversed(order):
        if state == "running" and v < 0 and swap > 0:
            preempted.append(rid)
            swap -= blk
    return preempted, prioritized


def config5_lvf(seed: int = MASTER_SEED + 6, rate: float = 8.0, n_steps: int = 2000, shape: KVShape = SHAPE_8B,
                duration_s: float = 120.0, step_s: float = 0.070, nb_host: Optional[int] = None, cap: float = 0.40,
                max_tokens: int = 8192, params: LVFParams = LVFParams()) -> Workload:
    """The serving replay of ``config5_replay`` (same arrivals, lengths, growth of one token per running
    request per 70 ms step, device pool at 40 % of the unconstrained demand) with the paper's scheduler
    choosing who moves: each step computes every request's VLT and runs one Largest-VLT-First decision
    under the free-block count and ``params.b_xfer``.

    What a decision turns into.  Preempted requests are swapped out in this step.  A prioritized rotary
    request is swapped in, and a prioritized waiting request is admitted (its prompt blocks allocated, no
    transfer), only as far as blocks are free *before* this step's swap-out releases any: the lists take
    swap-in destinations from the free list first, so no rotation ever names a block in both directions
    (the paper gets the same freedom from eager block rotation; without it the blocks a preemption frees
    serve the next step).  Requests left over stay in their queue and are decided on again next step.
    ``extra`` reports how many requests each step preempted / resumed / admitted."""
    rng = np.random.default_rng(seed)
    n_arr = max(1, int(rng.poisson(rate * duration_s)))
    arrive = np.sort(rng.uniform(0.0, duration_s, size=n_arr))
    prompt = lognormal_tokens(rng, n_arr, 512, 1, max_tokens)
    output = lognormal_tokens(rng, n_arr, 256, 1, max_tokens)
    bs = shape.block_size
    nblk = lambda tokens: -(-int(tokens) // bs)
    a_step = np.floor(arrive / step_s).astype(np.int64)
    horizon = int(a_step.max() + output.max() + 2)
    delta = np.zeros(horizon + 1, np.int64)
    for s, p_, o in zip(a_step, prompt, output):
        delta[s] += nblk(p_ + o)
        delta[min(horizon, s + int(o))] -= nblk(p_ + o)
    demand = int(np.cumsum(delta).max())
    nb_gpu = max(int(cap * demand), nblk((prompt + output).max()) + 8)
    nb_host = max(2 * demand, 64) if nb_host is None else nb_host
    tab = RequestTable(shape, nb_gpu, nb_host, rng)
    running: Dict[int, float] = {}         # rid -> time it entered the running state
    rotary: Dict[int, float] = {}          # rid -> time of its last generated token
    waiting: List[int] = []                # arrival order
    remaining: Dict[int, int] = {}
    steps: List[Rotation] = []
    log = {"preempted": [], "resumed": [], "admitted": [], "deferred": []}
    nxt = 0
    for step in range(n_steps):
        t_now = step * step_s
        while nxt < n_arr and a_step[nxt] <= step:
            waiting.append(nxt)
            nxt += 1
        for rid in [r for r in running if remaining[r] <= 0]:
            del running[rid]
            tab.finish(rid)
        grow_need = sum(1 for r in running if tab.requests[r].tokens % bs == 0)
        b_hbm = max(0, len(tab.gpu_free) - grow_need)
        reqs = [(r, "running", vlt("running", t_now, t0, params), len(tab.requests[r].blocks)) for r, t0 in running.items()]
        reqs += [(r, "waiting", vlt("waiting", t_now, float(arrive[r]), params), nblk(prompt[r])) for r in waiting]
        reqs += [(r, "rotary", vlt("rotary", t_now, t0, params), len(tab.requests[r].blocks)) for r, t0 in rotary.items()]
        preempt, prio = lvf_select(reqs, b_hbm, params.b_xfer)
        blk_of = {r[0]: r[3] for r in reqs}
        free_now = b_hbm
        ins, admit, deferred = [], [], 0
        for rid in prio:
            if blk_of[rid] > free_now:
                deferred += 1
                continue
            free_now -= blk_of[rid]
            (ins if rid in rotary else admit).append(rid)
        steps.append(tab.rotate(preempt, ins) if (preempt or ins) else _empty_rotation())
        for rid in preempt:
            del running[rid]
            rotary[rid] = t_now
        for rid in ins:
            del rotary[rid]
            running[rid] = t_now
        for rid in admit:
            waiting.remove(rid)
            tab.add(rid, int(prompt[rid]), "gpu")
            remaining[rid] = int(output[rid])
            running[rid] = t_now
        for k, v in (("preempted", len(preempt)), ("resumed", len(ins)), ("admitted", len(admit)), ("deferred", deferred)):
            log[k].append(v)
        for rid in running:
            if tab.requests[rid].tokens % bs == 0 and len(tab.gpu_free) == 0:
                continue                       # stalled this step: no block to grow into
            tab.grow(rid, tab.requests[rid].tokens + 1)
            remaining[rid] -= 1
    return Workload(f"lvf_{rate:g}rps", shape, nb_gpu, nb_host, seed, tab, steps,
                    {"demand_blocks": demand, "arrivals": n_arr, **{k: np.asarray(v) for k, v in log.items()}})
