"""The block table with eager block rotation on the GPU: random histories of add / append / background
copies / preempt-and-resume rotations / finish, with real content written into the device blocks the
table hands out.  The plain model (oracle/kv_block_table.py) says which copies of every logical block
must exist and which version of its content each one holds; every one of them is read back and compared
bit for bit."""
import numpy as np
import pytest

from paper_2601_20309_b200 import workload as W

pytestmark = pytest.mark.gpu


def _content(rid, i, version, shape):
    """Content of logical block i of request rid after its version-th write: (planes, SEG bytes) uint8."""
    words = W.block_words(4242, 1000 * version + 7, rid * 4096 + i, shape.words_per_block)
    return words.view(np.uint8).reshape(2 * shape.num_layers, -1)


@pytest.mark.parametrize("seed,path", [(0, 0), (1, 0), (2, 1), (3, 2)], ids=["auto-a", "auto-b", "zerocopy", "staged"])
def test_block_table_history_keeps_every_copy_exact(seed, path):
    import torch
    from oracle.kv_block_table import BlockTableModel, OK
    from paper_2601_20309_b200 import binding as B

    shape = W.KVShape(4, 16, 8, 128)                  # 32 KiB planes, 256 KiB blocks
    nb_gpu, nb_host, bs = 160, 520, shape.block_size
    planes, seg = 2 * shape.num_layers, 2 * shape.words_per_plane
    rng = np.random.default_rng(seed)
    dev = torch.zeros(nb_gpu * shape.block_bytes, dtype=torch.uint8, device="cuda:0")
    dev3 = dev.view(planes, nb_gpu, seg)
    pool = B.KVPool(shape.num_layers, bs, shape.kv_heads, shape.head_dim, nb_gpu, nb_host, dev.data_ptr(), path=path,
                    staging_bytes=24 * shape.block_bytes)
    table = B.KVTable(pool)
    model = BlockTableModel(nb_gpu, nb_host, bs)
    live, next_id = [], 0

    def write(rid, idx, settle):
        """Play the model: put the current version of the given logical blocks into their device blocks."""
        if settle:
            pool.kv_sync()        # the request's own swap-in has to land before tokens are written over it
        g, _, _ = table.kv_req_blocks(rid)
        for i in idx:
            dev3[:, int(g[i]), :] = torch.from_numpy(_content(rid, i, model.reqs[rid].version[i], shape)).to("cuda:0")
        torch.cuda.synchronize()  # the writes are done before the library is asked to move these blocks

    def verify(what):
        pool.kv_sync()
        harr = pool.host_array()
        for rid in live:
            mr = model.reqs[rid]
            g, h, valid = table.kv_req_blocks(rid)
            for i in range(len(g)):
                if mr.on_gpu:
                    got = dev3[:, int(g[i]), :].cpu().numpy()
                    assert np.array_equal(got, _content(rid, i, mr.version[i], shape)), (what, rid, i, "device")
                if mr.host_version[i] is not None:     # valid or stale: the model knows which version it holds
                    off = int(h[i]) * shape.block_bytes
                    got = harr[off:off + shape.block_bytes].reshape(planes, seg)
                    assert np.array_equal(got, _content(rid, i, mr.host_version[i], shape)), (what, rid, i, "host")
                assert bool(valid[i]) == mr.host_valid(i)

    try:
        for step in range(260):
            op = rng.choice(["add", "append", "eager", "rotate", "finish"], p=[0.2, 0.3, 0.15, 0.25, 0.1])
            if op == "add":
                tokens = int(rng.integers(1, 14 * bs))
                rc = model.add(next_id, tokens)
                assert rc == table.kv_req_add(next_id, tokens, check=False)
                if rc == OK:
                    live.append(next_id)
                    write(next_id, range(model.nblocks(tokens)), settle=False)   # fresh blocks: written at once
                next_id += 1
            elif op == "append" and live:
                on = [r for r in live if model.reqs[r].on_gpu]
                if not on:
                    continue
                rid, k = int(rng.choice(on)), int(rng.integers(1, 3 * bs))
                had, was_dirty = len(model.reqs[rid].version), model.reqs[rid].tokens % bs != 0
                rc = model.append(rid, k)
                assert rc == table.kv_req_append(rid, k, check=False)
                if rc == OK:
                    if was_dirty:
                        write(rid, [had - 1], settle=True)
                    write(rid, range(had, len(model.reqs[rid].version)), settle=False)
            elif op == "eager":
                budget = int(rng.integers(0, 40))
                assert len(model.eager(budget)) == table.kv_eager_rotate(budget)
            elif op == "rotate" and live:
                on = [r for r in live if model.reqs[r].on_gpu]
                off = [r for r in live if not model.reqs[r].on_gpu]
                p = [int(x) for x in rng.permutation(on)[:rng.integers(0, 4)]]
                r = [int(x) for x in rng.permutation(off)[:rng.integers(0, 4)]]
                rc, sent, brought = model.rotate(p, r)
                assert rc == table.kv_req_rotate(p, r, check=False), table._h and B.lib().kv_table_last_error(table._h)
            elif op == "finish" and live:
                rid = int(rng.choice(live))
                assert model.finish(rid) == table.kv_req_finish(rid, check=False) == OK
                live.remove(rid)
            if step % 40 == 39:
                verify(f"step {step}")
        verify("end")
        st = table.kv_table_get_stats()
        assert (st["eager_blocks"], st["preempt_blocks_moved"], st["discarded_blocks"], st["resume_blocks_moved"]) == \
               (model.eager_blocks, model.preempt_blocks_moved, model.discarded_blocks, model.resume_blocks_moved)
        assert st["discarded_blocks"] > 0 and st["resume_blocks_moved"] > 0
        ps = pool.kv_get_stats()
        assert ps["device_status"] == 0
        assert ps["bytes_out"] == (model.eager_blocks + model.preempt_blocks_moved) * shape.block_bytes
        assert ps["bytes_in"] == model.resume_blocks_moved * shape.block_bytes
    finally:
        table.destroy()
        pool.destroy()


def test_eager_rotation_leaves_one_block_per_request_to_send():
    """The paper's claim in numbers: after the background copies, preempting requests of 40-odd blocks
    moves one block each; and the requests that resume in the same rotation land in the device blocks
    the preempted ones gave up, with no hazard refusal from the pool."""
    import torch
    from paper_2601_20309_b200 import binding as B

    shape = W.KVShape(4, 16, 8, 128)
    nb_gpu, nb_host, bs = 200, 800, shape.block_size
    dev = torch.zeros(nb_gpu * shape.block_bytes, dtype=torch.uint8, device="cuda:0")
    pool = B.KVPool(shape.num_layers, bs, shape.kv_heads, shape.head_dim, nb_gpu, nb_host, dev.data_ptr())
    table = B.KVTable(pool)
    try:
        for rid in range(4):
            table.kv_req_add(rid, 45 * bs + 3)                  # 45 full blocks and a dirty one: 184 of 200 device blocks
        table.kv_req_rotate([2, 3], [])                        # no background copies yet: everything is sent
        assert table.kv_table_get_stats()["preempt_blocks_moved"] == 92
        assert table.kv_eager_rotate(10_000) == 90             # requests 0 and 1, full blocks only
        before = pool.kv_get_stats()["bytes_out"]
        table.kv_req_rotate([0, 1], [2, 3])                    # 92 blocks come in, into 90 discarded + 16 free ones
        pool.kv_sync()
        st = table.kv_table_get_stats()
        assert st["preempt_blocks_moved"] == 92 + 2 and st["discarded_blocks"] == 90 and st["resume_blocks_moved"] == 92
        assert pool.kv_get_stats()["bytes_out"] - before == 2 * shape.block_bytes
        assert st["free_gpu_blocks"] == nb_gpu - 92
    finally:
        table.destroy()
        pool.destroy()
