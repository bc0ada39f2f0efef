"""Eager block rotation: the plain model against what the paper states, and the library's block table
(bookkeeping only, no GPU) against the model over long random histories."""
import ctypes as C

import numpy as np
import pytest

from oracle.kv_block_table import BlockTableModel, OK, ERR_NOMEM, ERR_INVALID_ARG
from paper_2601_20309_b200 import binding as B


# ---------------------------------------------------------------------------------- pins of the model

def test_after_eager_rotation_a_preemption_sends_only_the_dirty_block():
    """Section 4.3.2: with the synced blocks already in host memory, only the last dirty block needs
    swap-out when the request is preempted; the synced device blocks are discarded."""
    m = BlockTableModel(100, 200, 16)
    assert m.add(1, 16 * 9 + 5) == OK                       # 9 full blocks + a dirty one
    assert len(m.eager(1000)) == 9                          # the dirty block is never copied early
    st, sent, brought = m.rotate([1], [])
    assert (st, sent, brought) == (OK, 1, 0)
    assert m.discarded_blocks == 9 and m.free_gpu == 100


def test_without_eager_rotation_every_block_is_sent():
    m = BlockTableModel(100, 200, 16)
    m.add(1, 16 * 9 + 5)
    assert m.rotate([1], []) == (OK, 10, 0)
    assert m.discarded_blocks == 0


def test_a_request_whose_last_block_is_full_sends_nothing():
    m = BlockTableModel(100, 200, 16)
    m.add(1, 16 * 4)
    assert len(m.eager(10)) == 4
    assert m.rotate([1], []) == (OK, 0, 0)


def test_host_copies_survive_a_resume_until_tokens_are_written():
    m = BlockTableModel(100, 200, 16)
    m.add(1, 16 * 3 + 2)
    m.rotate([1], [])
    assert m.rotate([], [1]) == (OK, 0, 4)                  # all four blocks come back
    assert m.info(1)["synced_blocks"] == 4                  # host duplicates are kept
    assert m.rotate([1], []) == (OK, 0, 0)                  # nothing was written meanwhile: nothing to send
    m.rotate([], [1])
    m.append(1, 1)                                          # one token into the dirty block
    assert m.info(1)["synced_blocks"] == 3
    assert m.rotate([1], []) == (OK, 1, 0)
    assert m.free_host == 200 - 4                           # the stale copy's host block was reused


def test_append_fills_the_dirty_block_then_takes_new_ones():
    m = BlockTableModel(100, 200, 16)
    m.add(1, 10)
    assert m.info(1) == {"tokens": 10, "num_blocks": 1, "on_gpu": 1, "synced_blocks": 0, "host_blocks": 0, "dirty_blocks": 1}
    m.append(1, 6)
    assert m.info(1)["num_blocks"] == 1 and m.info(1)["dirty_blocks"] == 0
    m.append(1, 33)
    assert m.info(1)["num_blocks"] == 4 and m.info(1)["dirty_blocks"] == 1 and m.free_gpu == 96
    assert [i for _, i in m.eager(10)] == [0, 1, 2]


def test_discarded_blocks_are_at_once_free_for_the_requests_that_resume():
    """The point of the mechanism: a rotation's swap-in does not wait for its swap-out."""
    m = BlockTableModel(10, 100, 16)
    m.add(1, 16 * 5)
    m.add(2, 16 * 5)
    m.eager(100)
    assert m.rotate([2], []) == (OK, 0, 0) and m.free_gpu == 5
    m.add(3, 16 * 5)
    assert m.free_gpu == 0
    m.eager(100)
    assert m.rotate([1], [2]) == (OK, 0, 5)                 # 2 comes back into the blocks 1 gives up
    m2 = BlockTableModel(10, 100, 16)                       # without the background copies it cannot
    m2.add(1, 16 * 5); m2.add(2, 16 * 5)
    m2.rotate([2], []); m2.add(3, 16 * 5)
    assert m2.rotate([1], [2])[0] == ERR_NOMEM
    assert m2.info(1)["on_gpu"] == 1 and m2.free_gpu == 0   # refused: nothing changed


def test_background_step_walks_requests_round_robin_and_respects_its_budget():
    m = BlockTableModel(100, 100, 4)
    for rid in (1, 2, 3):
        m.add(rid, 4 * 4)
    assert m.eager(6) == [(1, 0), (1, 1), (1, 2), (1, 3), (2, 0), (2, 1)]
    assert m.eager(6) == [(3, 0), (3, 1), (3, 2), (3, 3), (2, 2), (2, 3)]    # goes on after request 2, returns to it
    assert m.eager(6) == []
    m.rotate([1], [])
    m.append(2, 4)
    assert m.eager(6) == [(2, 4)]                           # preempted requests have nothing to copy


def test_model_invalid_calls_change_nothing():
    m = BlockTableModel(4, 4, 16)
    assert m.add(1, 16 * 5) == ERR_NOMEM and m.free_gpu == 4
    m.add(1, 16)
    assert m.add(1, 16) == ERR_INVALID_ARG
    assert m.rotate([], [1])[0] == ERR_INVALID_ARG          # not preempted
    assert m.rotate([1, 1], [])[0] == ERR_INVALID_ARG
    assert m.append(7, 1) == ERR_INVALID_ARG
    m.rotate([1], [])
    assert m.append(1, 1) == ERR_INVALID_ARG                # a preempted request generates nothing
    assert m.rotate([1], [])[0] == ERR_INVALID_ARG


# ------------------------------------------------------------------- pins of the model's finish()
#
# Section 4.3.2: a full block never changes again "until its request finishes", and the host-side
# duplicates exist only for the request's sake, so finishing a request frees every block it owns in
# either pool.  The background step's policy (requests in arrival order, going on after the last request
# the previous step looked at) fixes where the next step starts once a request has left the order.  All
# expected values below are worked out by hand from those two statements.

def pin_finish_of_a_running_request_frees_both_pools(Model):
    m = Model(10, 20, 4)
    m.add(1, 10)                                  # 2 full blocks + a dirty one: 3 device blocks
    assert (m.free_gpu, m.free_host) == (7, 20)
    assert len(m.eager(10)) == 2                  # the two full blocks get host copies
    m.rotate([1], [])                             # the dirty block is sent too: 3 host blocks owned
    m.rotate([], [1])                             # back on the GPU, the three host copies kept
    m.append(1, 1)                                # the dirty block's host copy goes stale, its host block stays owned
    assert (m.free_gpu, m.free_host) == (7, 17)
    assert m.info(1)["synced_blocks"] == 2 and m.info(1)["host_blocks"] == 3
    assert m.finish(1) == OK
    assert (m.free_gpu, m.free_host) == (10, 20)  # 3 device blocks and 3 host blocks (2 valid + 1 stale) return
    assert m.finish(1) == ERR_INVALID_ARG         # gone
    assert m.add(1, 40) == OK                     # the id and the whole pool can be used again


def pin_finish_of_a_preempted_request_frees_host_blocks_only(Model):
    m = Model(10, 20, 4)
    m.add(1, 10)
    m.add(2, 8)
    m.rotate([1], [])                             # nothing copied beforehand: all 3 blocks are sent
    assert (m.free_gpu, m.free_host) == (8, 17)   # request 1 holds no device block any more
    assert m.finish(1) == OK
    assert (m.free_gpu, m.free_host) == (8, 20)   # its device blocks were released at preemption, not again
    assert m.finish(2) == OK
    assert (m.free_gpu, m.free_host) == (10, 20)


def _four_requests_cursor_at_the_second(Model):
    m = Model(100, 100, 4)
    for rid in (1, 2, 3, 4):
        m.add(rid, 8)                             # two full blocks each
    assert m.eager(2) == [(1, 0), (1, 1)]         # request 1 done; the next step would start at request 2
    return m


def pin_finish_before_at_and_after_the_background_cursor(Model):
    m = _four_requests_cursor_at_the_second(Model)
    m.finish(1)                                   # a request the step has already passed
    assert m.eager(2) == [(2, 0), (2, 1)]         # still starts at request 2
    m = _four_requests_cursor_at_the_second(Model)
    m.finish(2)                                   # the very request the next step would start at
    assert m.eager(2) == [(3, 0), (3, 1)]         # its successor in arrival order takes its place
    m = _four_requests_cursor_at_the_second(Model)
    m.finish(3)                                   # a request further on
    assert m.eager(4) == [(2, 0), (2, 1), (4, 0), (4, 1)]
    m = _four_requests_cursor_at_the_second(Model)
    assert len(m.eager(4)) == 4                   # requests 2 and 3 done; the next step would start at request 4
    m.finish(4)                                   # the last in arrival order, at the cursor: the walk wraps to request 1
    m.append(1, 4)                                # gives request 1 a new full block
    m.append(2, 4)
    assert m.eager(1) == [(1, 2)]
    assert m.eager(1) == [(2, 2)]
    m.finish(1); m.finish(2); m.finish(3)         # nothing left: the step is a no-op and the model stays usable
    assert m.eager(5) == [] and m.add(9, 4) == OK and m.eager(5) == [(9, 0)]
    # a request the walk has passed may still have blocks to copy (the step's budget ran out inside it):
    # a finish elsewhere must not send the walk back to it before the others had their turn
    m = Model(100, 100, 4)
    for rid in (1, 2, 3):
        m.add(rid, 16)                            # four full blocks each
    assert m.eager(2) == [(1, 0), (1, 1)]
    m.finish(3)
    assert m.eager(2) == [(2, 0), (2, 1)]
    assert m.eager(4) == [(1, 2), (1, 3), (2, 2), (2, 3)]


FINISH_PINS = [pin_finish_of_a_running_request_frees_both_pools, pin_finish_of_a_preempted_request_frees_host_blocks_only,
               pin_finish_before_at_and_after_the_background_cursor]


@pytest.mark.parametrize("pin", FINISH_PINS, ids=lambda f: f.__name__)
def test_model_finish(pin):
    pin(BlockTableModel)


def test_finish_pins_catch_planted_mistakes():
    """Each plausible slip in finish() fails at least one of the pins above."""
    class FreesDeviceBlocksOfPreempted(BlockTableModel):
        def finish(self, rid):
            r = self.reqs.get(rid)
            extra = len(r.version) if r is not None and not r.on_gpu else 0
            rc = super().finish(rid)
            self.free_gpu += extra
            return rc

    class KeepsStaleHostBlocks(BlockTableModel):
        def finish(self, rid):
            r = self.reqs.get(rid)
            stale = sum(1 for i, v in enumerate(r.host_version) if v is not None and not r.host_valid(i)) if r else 0
            rc = super().finish(rid)
            self.free_host -= stale
            return rc

    class ForgetsTheCursor(BlockTableModel):
        def finish(self, rid):
            c = self.cursor
            rc = super().finish(rid)
            self.cursor = c % len(self.order) if self.order else 0
            return rc

    class RestartsTheWalk(BlockTableModel):
        def finish(self, rid):
            rc = super().finish(rid)
            self.cursor = 0
            return rc

    for Broken in (FreesDeviceBlocksOfPreempted, KeepsStaleHostBlocks, ForgetsTheCursor, RestartsTheWalk):
        caught = 0
        for pin in FINISH_PINS:
            try:
                pin(Broken)
            except AssertionError:
                caught += 1
        assert caught >= 1, Broken.__name__


# ------------------------------------------------------------- the library's table (no GPU) vs the model

def _random_history(seed, steps, nb_gpu, nb_host, bs):
    rng = np.random.default_rng(seed)
    m = BlockTableModel(nb_gpu, nb_host, bs)
    t = B.KVTable(num_gpu_blocks=nb_gpu, num_host_blocks=nb_host, block_size=bs)
    next_id, live = 0, []
    for step in range(steps):
        op = rng.choice(["add", "append", "eager", "rotate", "finish", "bad"], p=[0.2, 0.3, 0.15, 0.22, 0.1, 0.03])
        if op == "add":
            tokens = int(rng.integers(1, 12 * bs))
            rc_m, rc_t = m.add(next_id, tokens), t.kv_req_add(next_id, tokens, check=False)
            assert rc_m == rc_t, (step, op)
            if rc_m == OK:
                live.append(next_id)
            next_id += 1
        elif op == "append" and live:
            rid, k = int(rng.choice(live)), int(rng.integers(1, 3 * bs))
            assert m.append(rid, k) == t.kv_req_append(rid, k, check=False), (step, op)
        elif op == "eager":
            budget = int(rng.integers(0, 20))
            assert len(m.eager(budget)) == t.kv_eager_rotate(budget), (step, op)
        elif op == "rotate" and live:
            on = [r for r in live if m.reqs[r].on_gpu]
            off = [r for r in live if not m.reqs[r].on_gpu]
            p = [int(x) for x in rng.permutation(on)[:rng.integers(0, 3)]]
            r = [int(x) for x in rng.permutation(off)[:rng.integers(0, 3)]]
            rc_m, sent, brought = m.rotate(p, r)
            before = t.kv_table_get_stats()
            assert rc_m == t.kv_req_rotate(p, r, check=False), (step, op, p, r)
            after = t.kv_table_get_stats()
            assert after["preempt_blocks_moved"] - before["preempt_blocks_moved"] == sent
            assert after["resume_blocks_moved"] - before["resume_blocks_moved"] == brought
        elif op == "finish" and live:
            rid = int(rng.choice(live))
            assert m.finish(rid) == t.kv_req_finish(rid, check=False) == OK
            live.remove(rid)
        elif op == "bad":
            assert t.kv_req_rotate([10 ** 9], [], check=False) == ERR_INVALID_ARG
            assert m.rotate([10 ** 9], [])[0] == ERR_INVALID_ARG
        # everything the model says must hold in the table
        st = t.kv_table_get_stats()
        assert (st["free_gpu_blocks"], st["free_host_blocks"]) == (m.free_gpu, m.free_host), (step, op)
        assert (st["eager_blocks"], st["preempt_blocks_moved"], st["discarded_blocks"], st["resume_blocks_moved"]) == \
               (m.eager_blocks, m.preempt_blocks_moved, m.discarded_blocks, m.resume_blocks_moved), (step, op)
        used_g, used_h = [], []
        for rid in live:
            assert t.kv_req_info(rid) == m.info(rid), (step, op, rid)
            g, h, valid = t.kv_req_blocks(rid)
            mr = m.reqs[rid]
            assert list(valid) == [mr.host_valid(i) for i in range(len(g))]
            assert list(h >= 0) == [v is not None for v in mr.host_version]
            assert all(g >= 0) if mr.on_gpu else all(g < 0)
            used_g += list(g[g >= 0])
            used_h += list(h[h >= 0])
        assert len(set(used_g)) == len(used_g) == nb_gpu - m.free_gpu          # ids unique, free + used = pool
        assert len(set(used_h)) == len(used_h) == nb_host - m.free_host
        assert all(0 <= x < nb_gpu for x in used_g) and all(0 <= x < nb_host for x in used_h)
    t.destroy()
    return m


@pytest.mark.parametrize("seed", range(6))
def test_library_table_follows_the_model_over_random_histories(seed):
    _random_history(seed, 500, nb_gpu=120, nb_host=400, bs=16)


def test_library_table_under_pressure_small_pools():
    m = _random_history(99, 800, nb_gpu=30, nb_host=40, bs=4)
    assert m.discarded_blocks > 0 and m.preempt_blocks_moved > 0


def test_host_blocks_come_in_runs():
    """Blocks a request sends out together are neighbours in host memory while the pool has room."""
    t = B.KVTable(num_gpu_blocks=1000, num_host_blocks=4000, block_size=16)
    for rid in range(10):
        t.kv_req_add(rid, 16 * 50)
    assert t.kv_eager_rotate(10_000) == 500
    for rid in range(10):
        _, h, _ = t.kv_req_blocks(rid)
        assert np.array_equal(h, np.arange(h[0], h[0] + 50))
    for rid in (1, 3, 5):
        t.kv_req_finish(rid)
    assert t.kv_table_get_stats()["free_host_extents"] == 4                 # three holes of 50 and the tail
    t.kv_req_add(20, 16 * 120)
    t.kv_eager_rotate(10_000)
    _, h, _ = t.kv_req_blocks(20)
    assert np.array_equal(h, np.arange(h[0], h[0] + 120))                   # does not fit a hole: one run from the tail
    t.kv_req_add(21, 16 * 30)
    t.kv_eager_rotate(10_000)
    _, h, _ = t.kv_req_blocks(21)
    assert np.array_equal(h, np.arange(50, 80))                             # first hole that fits
    t.destroy()


# ------------------------------------------------- all or nothing when the pool refuses (host-side injection)

def _snapshot(t, live):
    """Everything observable of a table: statistics, and per request its info and every block's ids."""
    snap = {"stats": t.kv_table_get_stats()}
    for rid in live:
        g, h, v = t.kv_req_blocks(rid)
        snap[rid] = (t.kv_req_info(rid), g.tolist(), h.tolist(), v.tolist())
    return snap


def _table_in_mid_history():
    t = B.KVTable(num_gpu_blocks=40, num_host_blocks=60, block_size=4)
    for rid, tokens in ((1, 18), (2, 9), (3, 16), (4, 7)):
        t.kv_req_add(rid, tokens)
    assert t.kv_eager_rotate(3) == 3                          # request 1 partly copied
    t.kv_req_rotate([3, 4], [])                               # two requests parked in host memory
    t.kv_req_add(5, 30)
    return t, [1, 2, 3, 4, 5]


@pytest.mark.parametrize("code", [B.KV_ERR_CUDA, B.KV_ERR_NOMEM])
def test_rotate_refused_by_the_pool_leaves_the_table_unchanged(code):
    """kv_req_rotate promises all or nothing; the pool call is made to fail on the host, nothing else."""
    t, live = _table_in_mid_history()
    before = _snapshot(t, live)
    t.kv_table_fail_pool_call(0, code)
    assert t.kv_req_rotate([1, 2], [3, 4], check=False) == code
    assert _snapshot(t, live) == before
    # the same call goes through afterwards, and leaves what a table that never saw the failure has
    assert t.kv_req_rotate([1, 2], [3, 4], check=False) == B.KV_OK
    u, _ = _table_in_mid_history()
    u.kv_req_rotate([1, 2], [3, 4])
    assert _snapshot(t, live) == _snapshot(u, live)
    t.destroy(); u.destroy()


def test_background_copy_refused_by_the_pool_leaves_the_table_unchanged():
    t, live = _table_in_mid_history()
    before = _snapshot(t, live)
    t.kv_table_fail_pool_call(0, B.KV_ERR_CUDA)
    n = C.c_int64(-1)
    assert B.lib().kv_eager_rotate(t._h, 100, C.byref(n)) == B.KV_ERR_CUDA and n.value == 0
    assert _snapshot(t, live) == before                       # host ids handed back, the walk has not moved on
    u, _ = _table_in_mid_history()
    assert t.kv_eager_rotate(100) == u.kv_eager_rotate(100) > 0
    assert _snapshot(t, live) == _snapshot(u, live)
    t.destroy(); u.destroy()


def test_injected_failure_hits_the_call_it_names_only():
    t, live = _table_in_mid_history()
    t.kv_table_fail_pool_call(1, B.KV_ERR_CUDA)               # the second pool call from now
    assert t.kv_req_rotate([1], [], check=False) == B.KV_OK
    before = _snapshot(t, live)
    assert t.kv_req_rotate([2], [3], check=False) == B.KV_ERR_CUDA
    assert _snapshot(t, live) == before
    assert t.kv_req_rotate([2], [3], check=False) == B.KV_OK  # disarmed again
    t.destroy()
