// Device code of the KV-block rotation engine: two copy kernels over one job description.
//
// A job names up to two directions (swap-out and swap-in).  Each direction is a list of
// (source block id, destination block id) pairs plus an address rule per side:
//     address(id, plane) = base + id * blk_stride + plane * plane_stride
// which covers the layer-first device pool (blk_stride = SEG, plane_stride = num_blocks*SEG),
// the block-first host pool or staging buffer (blk_stride = BLK, plane_stride = SEG) and the
// layer-first host pool.  A plane of one block (SEG bytes, contiguous on both sides) is cut into
// chunks of at most `chunk` bytes; the work items of a direction are (pair, plane, chunk) in that
// order, and every CTA of the direction takes one contiguous range of items, so each CTA streams
// through consecutive destination addresses and re-reads the pair list only when it moves to the
// next block.
//
// kv_copy_bulk  one thread per warp drives bulk asynchronous copies (global -> shared -> global)
//               through a ring of shared-memory stages guarded by mbarriers; no registers are
//               spent on the payload.  One warp per CTA when segments are large, up to 16 when
//               they are small.  Used for HBM<->HBM gather/scatter and for HBM<->mapped host memory.
// kv_copy_ldst  every thread moves 16-byte (or 32-byte) vectors with streaming loads/stores, all loads of a
//               chunk issued before its stores; each warp walks the pair list cooperatively
//               (one coalesced load of up to 32 pairs, then shuffles).
//
// Every wait on an mbarrier is bounded (the job carries the bound of the main-loop waits): when one
// runs out the thread sets KV_DEV_TIMEOUT in the job's status word, waits -- again bounded -- for the
// loads it has in flight, drains its stores and returns.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#define KV_DEV_TIMEOUT 1u   // a bounded wait ran out
#define KV_DEV_BAD_ID  2u   // KvJob::check_ids: a pair named a block outside its pool; the pair was skipped

// The check behind KvJob::check_ids, as a plain function of the ids and the pool sizes (host and device).
__host__ __device__ inline bool kv_pair_in_bounds(int src_id, int dst_id, int src_blocks, int dst_blocks)
{
    return src_id >= 0 && src_id < src_blocks && dst_id >= 0 && dst_id < dst_blocks;
}

struct KvSide {
    unsigned long long base;
    long long blk_stride;
    long long plane_stride;
};

struct KvDir {
    KvSide src, dst;
    const int2 *pairs;   // x = source block id, y = destination block id (device memory);
                         // nullptr = the list is short and travels with the launch (KvJob::inl)
    int n;               // pairs
    int ctas;            // CTAs assigned to this direction (0 = direction absent)
    int src_blocks, dst_blocks;   // blocks each side holds (what KvJob::check_ids compares the ids with)
};

#define KV_INLINE_PAIRS 64   // longest pair list carried in the kernel parameters (1 KiB for both directions)

struct KvJob {
    KvDir dir[2];
    int planes;          // 2 * num_layers
    int seg;             // bytes of one plane of one block
    int chunk;           // bytes per work item (last chunk of a plane may be shorter)
    int cps;             // chunks per plane
    unsigned int *status;
    // bound of every wait for a load in the kernels' main loops: `wait_polls` immediate polls, then polls
    // 200 ns apart for at most `wait_ns` nanoseconds (0 = give up right after the immediate polls)
    unsigned int wait_polls;
    unsigned long long wait_ns;
    // non-zero: before an address is formed from a pair, its ids are compared with src_blocks / dst_blocks;
    // a pair out of bounds sets KV_DEV_BAD_ID in the status word and none of its bytes is touched
    int check_ids;
    // optional: device words that receive the earliest start and the latest end of the launch's CTAs
    // (%globaltimer, ns); nullptr = not wanted.  The host presets them to ~0 and 0.
    unsigned long long *t_first, *t_last;
    // pair lists of at most KV_INLINE_PAIRS entries ride in the launch parameters: a small rotation then
    // needs no separate copy of its ids, and the kernel no read from memory to find its first block
    int2 inl[2][KV_INLINE_PAIRS];
};

__device__ __forceinline__ int2 kv_pair(const KvJob &job, int dsel, int i)
{
    const int2 *pairs = job.dir[dsel].pairs;
    return pairs ? pairs[i] : job.inl[dsel][i];
}

// ------------------------------------------------------------------------------------------------
// work-item cursor: (pair i, plane p, chunk c), advanced one item at a time
struct KvCursor {
    int i, p, c;
    int2 pr;
    bool ok;             // the current pair passed the bounds check (always true when the job does not ask for it)

    __device__ __forceinline__ void load_pair(const KvJob &job, int dsel)
    {
        const KvDir &d = job.dir[dsel];
        pr = kv_pair(job, dsel, i);
        ok = !job.check_ids || kv_pair_in_bounds(pr.x, pr.y, d.src_blocks, d.dst_blocks);
        if (!ok) atomicOr(job.status, KV_DEV_BAD_ID);
    }

    __device__ __forceinline__ void seek(const KvJob &job, int dsel, long long item)
    {
        const KvDir &d = job.dir[dsel];
        const long long per = (long long)job.planes * job.cps;
        i = (int)(item / per);
        const int r = (int)(item - (long long)i * per);
        p = r / job.cps;
        c = r - p * job.cps;
        pr = make_int2(0, 0);
        ok = true;
        if (i < d.n) load_pair(job, dsel);
    }
    __device__ __forceinline__ void step(const KvJob &job, int dsel)
    {
        const KvDir &d = job.dir[dsel];
        if (++c == job.cps) {
            c = 0;
            if (++p == job.planes) {
                p = 0;
                ++i;
                if (i < d.n) load_pair(job, dsel);
            }
        }
    }
    __device__ __forceinline__ unsigned long long src(const KvJob &job, const KvDir &d) const
    {
        return d.src.base + (long long)pr.x * d.src.blk_stride + (long long)p * d.src.plane_stride +
               (long long)c * job.chunk;
    }
    __device__ __forceinline__ unsigned long long dst(const KvJob &job, const KvDir &d) const
    {
        return d.dst.base + (long long)pr.y * d.dst.blk_stride + (long long)p * d.dst.plane_stride +
               (long long)c * job.chunk;
    }
    __device__ __forceinline__ int bytes(const KvJob &job) const
    {
        const int left = job.seg - c * job.chunk;
        return left < job.chunk ? left : job.chunk;
    }
};

// which direction this CTA serves and its item range [lo, hi)
__device__ __forceinline__ bool kv_my_range(const KvJob &job, int &dsel, long long &lo, long long &hi)
{
    int b = blockIdx.x;
    dsel = 0;
    if (b >= job.dir[0].ctas) {
        b -= job.dir[0].ctas;
        dsel = 1;
    }
    const KvDir &d = job.dir[dsel];
    if (b >= d.ctas) return false;
    const long long total = (long long)d.n * job.planes * job.cps;
    lo = total * b / d.ctas;
    hi = total * (b + 1) / d.ctas;
    return hi > lo;
}

// ------------------------------------------------------------------------------------------------
// PTX wrappers (sm_100a): mbarrier + bulk asynchronous copy, no multicast, no cluster
__device__ __forceinline__ uint32_t kv_smem_u32(const void *p)
{
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void kv_mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void kv_mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t kv_mbar_try_wait(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok;
}
__device__ __forceinline__ unsigned long long kv_globaltimer()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// bounded wait: `polls` immediate polls, then polls 200 ns apart until about limit_ns have passed.  The
// short burst catches HBM-latency waits; after that the thread sleeps between polls, so a CTA that waits
// on the host link for microseconds at a time does not take issue slots from whatever else runs on its
// SM.  Returns false when the wait ran out (with polls == 0 and limit_ns == 0: without looking at all).
#define KV_WAIT_POLLS 16u
#define KV_WAIT_NS 2000000000ull       // 2 s
__device__ __forceinline__ bool kv_mbar_wait(uint32_t bar, uint32_t parity, unsigned int polls, unsigned long long limit_ns)
{
#pragma unroll 1
    for (unsigned int k = 0; k < polls; ++k)
        if (kv_mbar_try_wait(bar, parity)) return true;
    if (limit_ns == 0) return false;
    const unsigned long long t0 = kv_globaltimer();
    for (;;) {
#pragma unroll 1
        for (int k = 0; k < 64; ++k) {
            __nanosleep(200);
            if (kv_mbar_try_wait(bar, parity)) return true;
        }
        if (kv_globaltimer() - t0 > limit_ns) return false;
    }
}
__device__ __forceinline__ void kv_bulk_load(uint32_t smem_dst, unsigned long long gsrc, uint32_t bytes, uint32_t bar)
{
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(smem_dst),
                 "l"(gsrc), "r"(bytes), "r"(bar)
                 : "memory");
}
__device__ __forceinline__ void kv_bulk_store(unsigned long long gdst, uint32_t smem_src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_src), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void kv_bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void kv_bulk_wait_read()
{
    asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void kv_bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void kv_fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void kv_fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

// ------------------------------------------------------------------------------------------------
// Bulk-copy kernel.  STAGE bytes per stage, NS stages, loads run AHEAD items in front of stores.
// Stage s is refilled only after the store that last read it has finished reading: stores are
// committed one group per item, in order, so allowing NS-AHEAD-1 newer groups to be pending
// guarantees that.
// The first thread of every warp of the CTA runs such a ring of its own (its own stages and barriers)
// over its share of the CTA's items: one warp when the items are large, several when segments are
// small, where one thread cannot issue copies fast enough and AHEAD small items are too few bytes in
// flight.  Dynamic shared memory: STAGE * NS bytes per warp.
#define KV_BULK_MAX_WARPS 16
template <int STAGE, int NS, int AHEAD>
__global__ void __launch_bounds__(32 * KV_BULK_MAX_WARPS, 1) kv_copy_bulk(const __grid_constant__ KvJob job)
{
    static_assert(AHEAD >= 1 && AHEAD < NS, "AHEAD must be in [1, NS)");
    extern __shared__ __align__(128) unsigned char kv_smem[];
    __shared__ __align__(8) unsigned long long full_bar[KV_BULK_MAX_WARPS][NS];
    if ((threadIdx.x & 31) != 0) return;
    const int warp = (int)(threadIdx.x >> 5), nwarps = (int)(blockDim.x >> 5);

    int dsel;
    long long lo, hi;
    if (!kv_my_range(job, dsel, lo, hi)) return;
    {
        const long long span = hi - lo;
        hi = lo + span * (warp + 1) / nwarps;
        lo = lo + span * warp / nwarps;
        if (hi <= lo) return;
    }
    const KvDir &d = job.dir[dsel];
    if (job.t_first) atomicMin(job.t_first, kv_globaltimer());

    const uint32_t smem0 = kv_smem_u32(kv_smem) + (uint32_t)warp * (uint32_t)(STAGE * NS);
    const uint32_t bar0 = kv_smem_u32(full_bar[warp]);
#pragma unroll
    for (int s = 0; s < NS; ++s) kv_mbar_init(bar0 + 8 * s, 1);
    kv_fence_mbar_init();
    kv_fence_async_smem();

    KvCursor ld, st;
    ld.seek(job, dsel, lo);
    st = ld;
    const long long n_items = hi - lo;
    long long loads_issued = 0, loads_seen = 0;
    bool ok = true;

    for (long long k = 0; k < n_items + AHEAD && ok; ++k) {
        if (k < n_items) {
            const int s = (int)(k % NS);
            if (k >= NS) kv_bulk_wait_read<NS - AHEAD - 1>();
            const uint32_t nbytes = ld.ok ? (uint32_t)ld.bytes(job) : 0u;
            kv_mbar_expect_tx(bar0 + 8 * s, nbytes);        // a skipped item arrives with no bytes to wait for
            if (ld.ok) kv_bulk_load(smem0 + s * STAGE, ld.src(job, d), nbytes, bar0 + 8 * s);
            ld.step(job, dsel);
            ++loads_issued;
        }
        const long long j = k - AHEAD;
        if (j >= 0) {
            const int s = (int)(j % NS);
            const uint32_t parity = (uint32_t)((j / NS) & 1);
            ok = kv_mbar_wait(bar0 + 8 * s, parity, job.wait_polls, job.wait_ns);
            if (!ok) break;
            ++loads_seen;
            kv_fence_async_smem();
            if (st.ok) kv_bulk_store(st.dst(job, d), smem0 + s * STAGE, (uint32_t)st.bytes(job));
            kv_bulk_commit();                               // one group per item, empty for a skipped one
            st.step(job, dsel);
        }
    }
    if (!ok) {
        atomicOr(job.status, KV_DEV_TIMEOUT);
        // loads still in flight write into this CTA's shared memory: give each one more bounded wait (the
        // fixed bound, whatever the job says) so that none lands after the CTA has gone
        for (long long j = loads_seen; j < loads_issued; ++j)
            kv_mbar_wait(bar0 + 8 * (int)(j % NS), (uint32_t)((j / NS) & 1), KV_WAIT_POLLS, KV_WAIT_NS);
    }
    kv_bulk_wait_all();
    if (job.t_last) atomicMax(job.t_last, kv_globaltimer());
}

// ------------------------------------------------------------------------------------------------
// 32-byte vectors (sm_100: 256-bit global loads and stores).  Addresses must be 32-byte aligned.
struct KvVec32 {
    unsigned int w[8];
};
__device__ __forceinline__ KvVec32 kv_ld32(const void *p)
{
    KvVec32 r;
    asm volatile("ld.global.cs.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(r.w[0]), "=r"(r.w[1]), "=r"(r.w[2]), "=r"(r.w[3]), "=r"(r.w[4]), "=r"(r.w[5]), "=r"(r.w[6]), "=r"(r.w[7])
                 : "l"(p)
                 : "memory");
    return r;
}
__device__ __forceinline__ void kv_st32(void *p, const KvVec32 &r)
{
    asm volatile("st.global.cs.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(r.w[0]), "r"(r.w[1]), "r"(r.w[2]),
                 "r"(r.w[3]), "r"(r.w[4]), "r"(r.w[5]), "r"(r.w[6]), "r"(r.w[7])
                 : "memory");
}

// Load/store kernel: THREADS threads, each moving up to UNROLL vectors of VEC bytes (16 or 32) per item.
template <int THREADS, int UNROLL, int VEC>
__global__ void __launch_bounds__(THREADS) kv_copy_ldst(const __grid_constant__ KvJob job)
{
    static_assert(VEC == 16 || VEC == 32, "16- or 32-byte vectors");
    int dsel;
    long long lo, hi;
    if (!kv_my_range(job, dsel, lo, hi)) return;
    const KvDir &d = job.dir[dsel];
    const int lane = threadIdx.x & 31;

    // warp-cooperative walk of the pair list: lane q holds pair (win + q)
    const long long per = (long long)job.planes * job.cps;
    int i = (int)(lo / per);
    int r = (int)(lo - (long long)i * per);
    int p = r / job.cps;
    int c = r - p * job.cps;
    int win = i;
    int2 mine = (win + lane < d.n) ? kv_pair(job, dsel, win + lane) : make_int2(0, 0);

    for (long long item = lo; item < hi; ++item) {
        if (i >= win + 32) {
            win = i;
            mine = (win + lane < d.n) ? kv_pair(job, dsel, win + lane) : make_int2(0, 0);
        }
        const int sid = __shfl_sync(0xffffffffu, mine.x, i - win);
        const int did = __shfl_sync(0xffffffffu, mine.y, i - win);
        const bool ok = !job.check_ids || kv_pair_in_bounds(sid, did, d.src_blocks, d.dst_blocks);
        if (!ok && threadIdx.x == 0) atomicOr(job.status, KV_DEV_BAD_ID);
        const long long inner = (long long)c * job.chunk;
        const unsigned char *src = reinterpret_cast<const unsigned char *>(d.src.base + (long long)sid * d.src.blk_stride +
                                                                          (long long)p * d.src.plane_stride + inner);
        unsigned char *dst = reinterpret_cast<unsigned char *>(d.dst.base + (long long)did * d.dst.blk_stride +
                                                               (long long)p * d.dst.plane_stride + inner);
        const int left = job.seg - c * job.chunk;
        const int nvec = ok ? (left < job.chunk ? left : job.chunk) / VEC : 0;      // a pair out of bounds moves nothing
        if constexpr (VEC == 16) {
            uint4 v[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int q = u * THREADS + (int)threadIdx.x;
                if (q < nvec) v[u] = __ldcs(reinterpret_cast<const uint4 *>(src) + q);
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int q = u * THREADS + (int)threadIdx.x;
                if (q < nvec) __stcs(reinterpret_cast<uint4 *>(dst) + q, v[u]);
            }
        } else {
            KvVec32 v[UNROLL];
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int q = u * THREADS + (int)threadIdx.x;
                if (q < nvec) v[u] = kv_ld32(src + (size_t)q * 32);
            }
#pragma unroll
            for (int u = 0; u < UNROLL; ++u) {
                const int q = u * THREADS + (int)threadIdx.x;
                if (q < nvec) kv_st32(dst + (size_t)q * 32, v[u]);
            }
        }
        if (++c == job.cps) {
            c = 0;
            if (++p == job.planes) {
                p = 0;
                ++i;
            }
        }
    }
}
