"""Shared plumbing of the GPU parity tests: build the same initial state on the GPU (through
torch copies) and in the CPU oracle, run calls on both, compare both pools byte for byte."""
import numpy as np

from oracle.kv_oracle import ByteOracle
from paper_2601_20309_b200 import binding as B
from paper_2601_20309_b200 import workload as W


# initial content of the pools of the last Pair built (one entry): many tests start from the same pools, and
# generating a block's content on the CPU is the slow part of building them
_INITIAL = {}


class Pair:
    """A GPU pool (through the C ABI) and the byte oracle holding the same logical content."""

    def __init__(self, shape, nb_gpu, nb_host, seed=1, host_layout=0, device_layout=0, **pool_kw):
        import torch
        self.torch = torch
        self.shape, self.nb_gpu, self.nb_host, self.seed = shape, nb_gpu, nb_host, seed
        s = shape
        self.oracle = ByteOracle(s.num_layers, s.block_size, s.kv_heads, s.head_dim, nb_gpu, nb_host, host_layout,
                                 dev_layout=device_layout)
        o = self.oracle
        wpp = s.words_per_plane
        key = (s, nb_gpu, nb_host, seed, host_layout, device_layout)
        if _INITIAL.get("key") == key:                      # the previous test started from the same pools
            o.G[:] = _INITIAL["G"]
            o.Hs[:] = _INITIAL["Hs"]
        else:
            G16 = o.G.view(np.uint16)
            H16 = o.Hs.view(np.uint16)
            for b in range(nb_gpu):
                words = W.block_words(seed, W.POOL_GPU, b, s.words_per_block).reshape(2 * s.num_layers, wpp)
                for pl in range(2 * s.num_layers):
                    off = o.dev_off(pl // 2, pl % 2, b) // 2
                    G16[off:off + wpp] = words[pl]
            for h in range(nb_host):
                words = W.block_words(seed, W.POOL_HOST, h, s.words_per_block).reshape(2 * s.num_layers, wpp)
                for pl in range(2 * s.num_layers):
                    off = o.host_off(h, pl // 2, pl % 2) // 2
                    H16[off:off + wpp] = words[pl]
            _INITIAL.clear()
            if o.G.size + o.Hs.size <= (4 << 30):
                _INITIAL.update(key=key, G=o.G.copy(), Hs=o.Hs.copy())
        # the device pool sits between two guard areas of one block each, which no call may touch
        self.guard = -(-max(256, s.block_bytes) // 256) * 256
        self.buf = torch.full((o.G.size + 2 * self.guard,), 0xC3, dtype=torch.uint8, device="cuda:0")
        self.dev = self.buf[self.guard:self.guard + o.G.size]
        self.dev.copy_(torch.from_numpy(o.G))
        self.pool = B.KVPool(s.num_layers, s.block_size, s.kv_heads, s.head_dim, nb_gpu, nb_host,
                             self.dev.data_ptr(), host_layout=host_layout, device_layout=device_layout, **pool_kw)
        self.pool.host_array()[:] = o.Hs

    def gpu_bytes(self):
        self.torch.cuda.synchronize()
        return self.dev.cpu().numpy()

    def assert_equal(self, what=""):
        self.pool.kv_sync()
        g = self.gpu_bytes()
        h = self.pool.host_array()
        lo, hi = self.buf[:self.guard], self.buf[self.guard + g.size:]
        if not (bool((lo == 0xC3).all()) and bool((hi == 0xC3).all())):
            raise AssertionError(f"{what}: bytes outside the device pool were written")
        if not np.array_equal(g, self.oracle.G):
            bad = np.flatnonzero(g != self.oracle.G)
            raise AssertionError(f"{what}: device pool differs at {len(bad)} bytes, first {bad[:4]}")
        if not np.array_equal(h, self.oracle.Hs):
            bad = np.flatnonzero(h != self.oracle.Hs)
            raise AssertionError(f"{what}: host pool differs at {len(bad)} bytes, first {bad[:4]}")

    def rotate_both(self, r, allow_overlap=False):
        rc_o = self.oracle.rotate(r.out_gpu, r.out_host, r.in_host, r.in_gpu, allow_overlap=allow_overlap)
        rc_g = self.pool.kv_rotate(r.out_gpu, r.out_host, r.in_host, r.in_gpu, check=False)
        assert rc_o == rc_g, (rc_o, rc_g, self.pool.kv_last_error())
        return rc_g

    def close(self):
        self.pool.destroy()
