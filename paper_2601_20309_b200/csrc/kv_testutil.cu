// Input-making and result-digesting helpers for tests and the bench.  NOT part of the rotation
// path and not linked into it: a separate shared library.
//
// kvt_fill_blocks      writes the seeded synthetic content of whole blocks into a pool.  It is the
//                      GPU twin of the counter-based generator in workload.py: the content of
//                      block b of pool `pool` is LUT[16-bit slices of splitmix64(counter)], with
//                      counter = seed*GOLDEN + pool*POOLMUL + b*groups + q for the q-th group of
//                      four words, in logical (layer, K|V, token, head, dim) order.  Integer-only.
// kvt_checksum_blocks  position-weighted 64-bit sum of the logical content of listed blocks:
//                      sum over words w at logical index q of w*(2q+1), modulo 2^64.
//
// kvt_wait_runs_out    runs the rotation kernels' bounded barrier wait (kv_mbar_wait of kv_kernels.cuh) on
//                      a barrier that expects bytes nobody sends, with a short limit: the wait must
//                      give up after about that long and the kernel must return normally.  This is how
//                      the give-up branch of the wait is executed without any fault or hang.
//
// The first two take an address rule  address(block, plane) = base + block*blk_stride + plane*plane_stride
// so that they work on the layer-first device pool, the block-first host pool and the
// layer-first host pool alike.  `base` must be reachable from the device (device memory or
// mapped pinned host memory).
#include <cuda_runtime.h>
#include <stdint.h>

#include "kv_kernels.cuh"

namespace {

// out[0] = 1 if the wait returned "ran out" (else 0), out[1] = nanoseconds the wait took
__global__ void wait_runs_out_kernel(unsigned long long limit_ns, unsigned long long *out)
{
    __shared__ __align__(8) unsigned long long bar;
    if (threadIdx.x != 0) return;
    const uint32_t b = kv_smem_u32(&bar);
    kv_mbar_init(b, 1);
    kv_fence_mbar_init();
    kv_mbar_expect_tx(b, 16);                       // the one arrival, and 16 bytes that no copy will ever deliver
    const unsigned long long t0 = kv_globaltimer();
    const bool done = kv_mbar_wait(b, 0, KV_WAIT_POLLS, limit_ns);
    out[1] = kv_globaltimer() - t0;
    out[0] = done ? 0ull : 1ull;
    asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(b) : "memory");
}

__device__ __forceinline__ unsigned long long mix64(unsigned long long key)
{
    unsigned long long z = key + 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

__global__ void fill_kernel(unsigned char *base, long long blk_stride, long long plane_stride,
                            long long words_per_plane, long long groups_per_block,
                            const int *ids, long long first_id, long long n_blocks,
                            unsigned long long seed, unsigned long long pool, const unsigned short *lut)
{
    const long long total = n_blocks * groups_per_block;
    for (long long t = blockIdx.x * (long long)blockDim.x + threadIdx.x; t < total;
         t += (long long)gridDim.x * blockDim.x) {
        const long long k = t / groups_per_block;
        const long long q = t - k * groups_per_block;
        const long long b = ids ? (long long)ids[k] : first_id + k;
        const unsigned long long z = mix64(seed * 0x9E3779B97F4A7C15ull + pool * 0xD1B54A32D192ED03ull +
                                           (unsigned long long)b * (unsigned long long)groups_per_block +
                                           (unsigned long long)q);
        const long long w = 4 * q;
        const long long plane = w / words_per_plane;
        const long long inner = w - plane * words_per_plane;
        ushort4 v;
        v.x = lut[z & 0xFFFF];
        v.y = lut[(z >> 16) & 0xFFFF];
        v.z = lut[(z >> 32) & 0xFFFF];
        v.w = lut[(z >> 48) & 0xFFFF];
        *reinterpret_cast<ushort4 *>(base + b * blk_stride + plane * plane_stride + inner * 2) = v;
    }
}

__global__ void checksum_kernel(const unsigned char *base, long long blk_stride, long long plane_stride,
                                long long words_per_plane, long long groups_per_block,
                                const int *ids, long long first_id, unsigned long long *out)
{
    const long long b = ids ? (long long)ids[blockIdx.x] : first_id + blockIdx.x;
    unsigned long long acc = 0;
    for (long long q = threadIdx.x; q < groups_per_block; q += blockDim.x) {
        const long long w = 4 * q;
        const long long plane = w / words_per_plane;
        const long long inner = w - plane * words_per_plane;
        const ushort4 v = *reinterpret_cast<const ushort4 *>(base + b * blk_stride + plane * plane_stride + inner * 2);
        const unsigned long long i = (unsigned long long)w;
        acc += (unsigned long long)v.x * (2 * i + 1) + (unsigned long long)v.y * (2 * i + 3) +
               (unsigned long long)v.z * (2 * i + 5) + (unsigned long long)v.w * (2 * i + 7);
    }
    __shared__ unsigned long long part[256];
    part[threadIdx.x] = acc;
    __syncthreads();
    for (int s = blockDim.x / 2; s > 0; s >>= 1) {
        if ((int)threadIdx.x < s) part[threadIdx.x] += part[threadIdx.x + s];
        __syncthreads();
    }
    if (threadIdx.x == 0) out[blockIdx.x] = part[0];
}

}  // namespace

extern "C" {

// ids: DEVICE pointer to n int32 block ids, or NULL for the run first_id .. first_id+n-1.
// lut: DEVICE pointer to 65536 uint16.  words_per_plane must be a multiple of 4.  Synchronous.
int kvt_fill_blocks(void *base, long long blk_stride, long long plane_stride, long long words_per_plane,
                    int planes, const int *ids, long long first_id, long long n,
                    unsigned long long seed, unsigned long long pool, const unsigned short *lut)
{
    if (!base || !lut || n < 0 || words_per_plane <= 0 || words_per_plane % 4 || planes <= 0) return -1;
    if (n == 0) return 0;
    const long long groups = words_per_plane * planes / 4;
    const long long total = n * groups;
    const int threads = 256;
    const long long want = (total + threads - 1) / threads;
    const int grid = (int)(want < 148 * 16 ? want : 148 * 16);
    fill_kernel<<<grid, threads>>>((unsigned char *)base, blk_stride, plane_stride, words_per_plane, groups,
                                   ids, first_id, n, seed, pool, lut);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    return e == cudaSuccess ? 0 : -(int)e - 1000;
}

// out: DEVICE pointer to n uint64.  Synchronous.
int kvt_checksum_blocks(const void *base, long long blk_stride, long long plane_stride, long long words_per_plane,
                        int planes, const int *ids, long long first_id, long long n, unsigned long long *out)
{
    if (!base || !out || n < 0 || words_per_plane <= 0 || words_per_plane % 4 || planes <= 0) return -1;
    if (n == 0) return 0;
    const long long groups = words_per_plane * planes / 4;
    for (long long lo = 0; lo < n; lo += 32768) {
        const long long cnt = (n - lo < 32768) ? n - lo : 32768;
        checksum_kernel<<<(int)cnt, 256>>>((const unsigned char *)base, blk_stride, plane_stride, words_per_plane,
                                          groups, ids ? ids + lo : nullptr, first_id + lo, out + lo);
    }
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    return e == cudaSuccess ? 0 : -(int)e - 1000;
}

// out: DEVICE pointer to 2 uint64 (see wait_runs_out_kernel).  limit_ns is clamped to 100 ms.  Synchronous.
int kvt_wait_runs_out(unsigned long long limit_ns, unsigned long long *out)
{
    if (!out) return -1;
    if (limit_ns > 100000000ull) limit_ns = 100000000ull;
    wait_runs_out_kernel<<<1, 32>>>(limit_ns, out);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) e = cudaDeviceSynchronize();
    return e == cudaSuccess ? 0 : -(int)e - 1000;
}

}  // extern "C"
