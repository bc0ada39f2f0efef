"""The allocation-free gather, for callers that may not allocate CUDA memory.

Some users of the library run where an allocation is not an option: a serving loop that cannot
afford the device-wide synchronisation of cudaMalloc / cudaFree, a process whose GPU memory is
already owned entirely by another allocator, a component that only gets buffers handed to it.
``kv_gather_blocks_static`` serves them: no pool object, the id list and the kernel's status word
live in an array built into the library.  It must give exactly what ``kv_gather_blocks`` gives.

This file sorts last on purpose: a run that stops at the first failure has then already been
through every other test.  It also has to pass on its own in a fresh process, so it sets up
everything it uses itself.
"""
import numpy as np
import pytest

from paper_2601_20309_b200 import workload as W

pytestmark = pytest.mark.gpu


def test_static_gather_matches_pool_gather_on_two_calls_in_a_row():
    import torch
    from paper_2601_20309_b200 import binding as B

    shape = W.KVShape(3, 16, 8, 128)                  # 32 KiB planes, 192 KiB blocks
    nbg = 300
    rng = np.random.default_rng(17)
    dev = torch.from_numpy(rng.integers(0, 256, nbg * shape.block_bytes, dtype=np.uint8)).to("cuda:0")
    before = dev.clone()

    # two different lists, the second one shorter, so that ids left in the built-in array by the first
    # call would show if they were used
    lists = [rng.integers(0, nbg, 211).astype(np.int32),      # repeats allowed
             rng.permutation(nbg)[:57].astype(np.int32)]
    # the two gathers through the allocation-free entry point first, back to back, before any pool exists in
    # this test (run alone in a fresh process, this is the library's first CUDA work)
    got = []
    outs = [torch.full((len(ids) * shape.block_bytes,), 0xA5, dtype=torch.uint8, device="cuda:0") for ids in lists]
    torch.cuda.synchronize()
    for ids, out in zip(lists, outs):
        rc = B.kv_gather_blocks_static(dev.data_ptr(), shape.num_layers, shape.block_size, shape.kv_heads,
                                       shape.head_dim, nbg, ids, out.data_ptr())
        assert rc == 0
        got.append(out.cpu().numpy())                 # the call is synchronous: the result is there
    # the same two gathers through the existing entry point
    want = []
    with B.KVPool(shape.num_layers, shape.block_size, shape.kv_heads, shape.head_dim, nbg, 8, dev.data_ptr()) as pool:
        for ids in lists:
            buf = torch.zeros(len(ids) * shape.block_bytes, dtype=torch.uint8, device="cuda:0")
            pool.kv_gather_blocks(ids, buf.data_ptr())
            pool.kv_sync()
            want.append(buf.cpu().numpy())

    for k in range(2):
        assert np.array_equal(got[k], want[k]), f"call {k}: allocation-free gather differs from kv_gather_blocks"
    assert torch.equal(dev, before)                   # the pool is only read

    # and against the layout itself: block i of the output is block ids[i], planes in (layer, K|V) order
    g = before.cpu().numpy().reshape(2 * shape.num_layers, nbg, 2 * shape.words_per_plane)
    ids = lists[1]
    out = got[1].reshape(len(ids), 2 * shape.num_layers, 2 * shape.words_per_plane)
    for i in (0, 13, len(ids) - 1):
        assert np.array_equal(out[i], g[:, ids[i], :])

    # on a caller-made stream as well
    s = torch.cuda.Stream()
    out = torch.zeros(len(lists[0]) * shape.block_bytes, dtype=torch.uint8, device="cuda:0")
    torch.cuda.synchronize()
    assert B.kv_gather_blocks_static(dev.data_ptr(), shape.num_layers, shape.block_size, shape.kv_heads,
                                     shape.head_dim, nbg, lists[0], out.data_ptr(), stream=s.cuda_stream) == 0
    assert np.array_equal(out.cpu().numpy(), want[0])


def test_static_gather_refuses_what_it_cannot_hold():
    import torch
    from paper_2601_20309_b200 import binding as B

    shape = W.KVShape(1, 1, 1, 8)                     # 16-byte planes
    nbg = 64
    dev = torch.zeros(nbg * shape.block_bytes, dtype=torch.uint8, device="cuda:0")
    out = torch.full(((B.KV_STATIC_MAX_BLOCKS + 1) * shape.block_bytes,), 7, dtype=torch.uint8, device="cuda:0")
    a = (dev.data_ptr(), shape.num_layers, shape.block_size, shape.kv_heads, shape.head_dim, nbg)
    too_many = np.zeros(B.KV_STATIC_MAX_BLOCKS + 1, np.int32)
    assert B.kv_gather_blocks_static(*a, too_many, out.data_ptr(), check=False) == B.KV_ERR_INVALID_ARG
    assert "KV_STATIC_MAX_BLOCKS" in B.lib().kv_last_error(None).decode()
    assert B.kv_gather_blocks_static(*a, [0, nbg], out.data_ptr(), check=False) == B.KV_ERR_RANGE
    assert B.kv_gather_blocks_static(*a, [0, -1], out.data_ptr(), check=False) == B.KV_ERR_RANGE
    assert B.kv_gather_blocks_static(*a, [], out.data_ptr(), check=False) == 0
    torch.cuda.synchronize()
    assert int(out.min()) == 7 and int(out.max()) == 7           # refused calls wrote nothing
    # the largest list it accepts
    full = (np.arange(B.KV_STATIC_MAX_BLOCKS) % nbg).astype(np.int32)
    dev.copy_(torch.arange(nbg * shape.block_bytes, device="cuda:0").to(torch.uint8))
    assert B.kv_gather_blocks_static(*a, full, out.data_ptr()) == 0
    g = dev.cpu().numpy().reshape(2, nbg, 16)
    o = out.cpu().numpy()[:B.KV_STATIC_MAX_BLOCKS * shape.block_bytes].reshape(B.KV_STATIC_MAX_BLOCKS, 2, 16)
    assert np.array_equal(o, g[:, full, :].transpose(1, 0, 2))
