// Host side of the KV-block rotation engine: the C ABI declared in include/duplexkv.h.
//
// What runs where
//   validation, hazard tracking, descriptor staging, stream/event orchestration   -> this file (host)
//   every byte of payload                                                         -> kernels in
//   kv_kernels.cuh, or the GPU's copy engines on the CE paths
//
// There is no CPU data path: when CUDA is unavailable every entry point fails with KV_ERR_CUDA.
#include "../../include/duplexkv.h"
#include "kv_kernels.cuh"

#include <algorithm>
#include <chrono>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <thread>
#include <vector>

#include <sys/mman.h>
#include <sys/syscall.h>
#include <unistd.h>

namespace {

constexpr int KV_SLOTS = 8;            // descriptor / event ring depth per direction
constexpr int KV_MAX_CE_STREAMS = 4;
constexpr int64_t KV_AUTO_MIN_TRANSFER = 5ll << 19;   // AUTO: staged when its transfers average 2.5 MiB or more
// AUTO, calls bound by fixed costs rather than by the link (measured on scattered ids, call to completion):
// one copy-engine transfer per block is the quickest up to 8 MiB per direction of 2 MiB blocks (65 / 111 /
// 212 us for 1 / 2 / 4 blocks each way against 85 / 141 / 231 us staged and 87 / 143 / 247 us for the
// zero-copy kernels); from 16 MiB on the staged path (one chunk, ids in the launch parameters, four-block
// lattices) is ahead (406 / 789 us at 8 / 16 blocks against 451 / 847 and 463 / 908) and the transfer-size
// rule decides.  With smaller blocks one transfer per block wins only for one or two blocks per direction
// (1 MiB blocks: 44 / 70 us for 1 / 2 blocks against 59 / 90 zero-copy, but 161 against 144 for 4; 256 KiB
// blocks: 28 / 43-48 against 43 / 43, but 69 / 122 against 60 / 90 for 4 / 8); above that the transfer-size
// rule picks the zero-copy kernels, which lead up to ~128 MiB.
constexpr int64_t KV_AUTO_TINY_BYTES = 8ll << 20;
constexpr int64_t KV_AUTO_TINY_BYTES_SMALL_BLOCKS = 2ll << 20;
constexpr int64_t KV_AUTO_TINY_COUNT_SMALL_BLOCKS = 2;
constexpr int64_t KV_MERGE_MIN_MEAN_RUN = 8;
constexpr int64_t KV_QUAD_MAX_GAP = 256;              // STAGED, scattered ids: largest row gap (blocks) of a four-block lattice
constexpr int64_t KV_QUAD_ENOUGH_BYTES = 8ll << 20;  //         no lattices when a pair of blocks already carries this much
constexpr int KV_QUAD_PARTNERS = 6;                   //         partners tried per block when looking for lattices
constexpr int64_t KV_PLAN_CHUNKS = 4;                 // STAGED: a call that fits one staging half is still cut into about this many chunks ...
constexpr int64_t KV_PLAN_ONE_CHUNK_BYTES = 128ll << 20;   // ... unless it moves this much or less per direction: then it is one chunk          // STAGED: merge runs of host ids when they average 8 blocks or more
// HBM-to-HBM shape of the bulk kernel's ring.  Measured on the 3.87 GB gather (148 CTAs): the rate peaks with
// about 32 KiB of loads in flight per SM and falls with more -- 16 KiB x 2 ahead 6.42-6.45 TB/s, 32 KiB x 1
// ahead 6.43, 8 KiB x 5 ahead 6.40, 16 KiB x 3 ahead 6.32, 16 KiB x 5 ahead (the first choice) 6.09-6.15, one
// load ahead 5.56; 4 KiB copies are bound by the one thread that issues them (3.8); two CTAs per SM lose 5 %.
constexpr int BULK_STAGE = 16384;      // bytes per shared-memory stage of the bulk kernel
constexpr int BULK_NS = 4;             // stages
constexpr int BULK_AHEAD = 2;          // loads in flight ahead of the stores
// the same kernel when one side is mapped host memory: the link needs far fewer bytes in flight than
// HBM does, and a small shared-memory footprint leaves the SMs' L1 to whatever else runs on them
constexpr int LINK_STAGE = 8192;
constexpr int LINK_NS = 8;
constexpr int LINK_AHEAD = 6;
// other shapes of the same ring for the link (kv_pool_config_t.link_variant 1 and 2): fewer, larger bulk copies
constexpr int LINK1_STAGE = 32768, LINK1_NS = 4, LINK1_AHEAD = 2;
constexpr int LINK2_STAGE = 65536, LINK2_NS = 3, LINK2_AHEAD = 1;
// Small segments (the shard of one rank under tensor parallelism, small block sizes): an item is a whole
// segment, so with the large ring too few bytes are in flight and one thread issues too few copies per
// second (measured on a 2 GiB gather: 5.1 / 3.4 / 1.8 / 0.9 TB/s for segments of 8 / 4 / 2 / 1 KiB against 6.4
// for 16 KiB and more).  Such launches take a ring of smaller stages per warp and more issuing warps per
// CTA.  HBM to HBM, what counts is many warps with few loads ahead each, 32 KiB in flight per SM as in the
// large ring: 2 / 4 / 8 warps x 2 ahead reach 6.43 / 6.24 / 5.98 TB/s at 8 / 4 / 2 KiB and 16 warps x 1 ahead
// 6.04 at 1 KiB, while 4 or 8 loads ahead on half as many warps stay at 4.9-5.0.  Over the link every shape
// with 48 KiB in flight per CTA reaches the zero-copy ceiling (80.4-80.7 GB/s both ways, where the 8 KiB ring
// gave 79.5 / 74.2 / 63.5 at 4 / 2 / 1 KiB).
constexpr int SMALL_NS = 4, SMALL_AHEAD = 2;           // HBM to HBM: stages of 8 / 4 / 2 KiB on 2 / 4 / 8 warps
constexpr int TINY_NS = 3, TINY_AHEAD = 1;             //             stages of 1 KiB on 16 warps
constexpr int SMALL_LINK_NS = 8, SMALL_LINK_AHEAD = 6; // over the link: stages of 4 / 2 / 1 KiB on 2 / 4 / 8 warps
constexpr int LDST_THREADS = 512;
constexpr int LDST_UNROLL = 4;         // 512 threads * 4 * 16 B = 32 KiB per item
constexpr int LDST_CHUNK = LDST_THREADS * LDST_UNROLL * 16;
constexpr int LDST32_UNROLL = 2;       // 512 threads * 2 * 32 B = 32 KiB per item

thread_local char g_err[256] = "";

// One copy-engine transfer of the STAGED path: `rows` rows of `width` bytes, packed back to back in
// the staging half, `host_pitch` bytes apart on the host (rows == 1: a plain transfer).
struct CeOp {
    int64_t host_off, stage_off, width, host_pitch;
    int32_t rows;
    int64_t pos;        // planning: the staging position (place in the staging order) of its first block
    int32_t nblk;       // blocks it moves (slices x rows x blocks per row)
    int32_t slices = 1; // > 1: a 3-D transfer of `slices` groups of `rows` rows, packed in staging,
    int64_t slice_rows = 0;   //  slice_rows * host_pitch bytes apart on the host
};
// Staging positions [lo, hi) go through one staging half; ops [op_lo, op_hi) move them.
struct CeChunk {
    int64_t lo, hi;
    int32_t op_lo, op_hi;
};

struct DirState {
    cudaStream_t stream = nullptr;
    bool owns_stream = false;
    int2 *ring_host = nullptr;         // pinned: KV_SLOTS slots of 2*cap pairs
    int2 *ring_dev = nullptr;          // device mirror
    cudaEvent_t ev_start[KV_SLOTS] = {};
    cudaEvent_t ev_end[KV_SLOTS] = {};
    uint64_t issued = 0;               // calls issued on this direction (sequence number of the latest)
    uint64_t done = 0;                 // latest call known to be complete
    // STAGED path: two staging halves in HBM (allocated on first use) worked as a double buffer: the
    // pack/unpack kernels run on `kstream`, the copy-engine transfers on `stream`
    uint8_t *stage = nullptr;
    int64_t half_blocks = 0;           // blocks per half
    cudaStream_t kstream = nullptr;
    cudaEvent_t kfork_ev = nullptr;
    cudaEvent_t ev_a[2] = {};          // half filled   (out: packed by the kernel;   in: landed from the host)
    cudaEvent_t ev_b[2] = {};          // half drained  (out: copied to the host;     in: scattered by the kernel)
    // optional timing of the pack / unpack kernels (KV_FLAG_TIME_KERNELS): event pairs on kstream
    std::vector<cudaEvent_t> kev;
    std::vector<int64_t> kev_bytes;
    int kev_used = 0;
    unsigned long long *ktime_dev = nullptr;   // 2 words per timed launch: earliest CTA start, latest CTA end
    std::vector<int32_t> order;        // list positions sorted by host id (= staging order)
    std::vector<CeOp> ops;             // transfers of the current call, in issue order
    std::vector<CeChunk> chunks;       // the call cut into staging-half-sized pieces
    int ctas = 0;
    int path = 0;                      // configured path of this direction (may be KV_PATH_AUTO)
    // copy-engine paths spread their transfers over nsub streams: sub[0] is `stream`, the others
    // are forked from it and joined back with events, so per-transfer start-up gaps overlap
    int nsub = 1;
    cudaStream_t sub[KV_MAX_CE_STREAMS] = {};
    cudaEvent_t fork_ev = nullptr;
    cudaEvent_t join_ev[KV_MAX_CE_STREAMS] = {};
};

}  // namespace

struct kv_pool {
    kv_pool_config_t cfg;
    int64_t seg = 0, blk = 0;
    int planes = 0;
    int64_t cap = 0;                   // most pairs one direction of one call may carry
    uint8_t *dev = nullptr;
    uint8_t *host = nullptr;           // host address of the host pool
    uint8_t *host_dev = nullptr;       // the same memory as the device sees it
    bool owns_host = false, registered_host = false;
    void *host_map = nullptr;           // anonymous mapping behind `host` when the library made it that way
    size_t host_map_len = 0;
    int sm_count = 0;
    int64_t max_pitch = 0;             // largest row pitch a 2-D copy-engine transfer accepts
    DirState dir[2];                   // 0 = out, 1 = in
    unsigned int *status_host = nullptr, *status_dev = nullptr;   // mapped pinned status word
    // per-block bookkeeping for validation and cross-direction ordering
    std::vector<uint32_t> g_mark, h_mark, g_mark2, h_mark2;
    uint32_t epoch = 0;
    std::vector<uint64_t> g_read_by_out, g_written_by_in, h_written_by_out, h_read_by_in;
    kv_stats_t stats;
    bool union_valid = false;          // the latest call's events have not been turned into statistics yet
    bool union_synced = false;         // ... and kv_sync has seen that call complete
    int union_slot[2] = {-1, -1};      // slots of the latest call (per direction; -1 = not part of it)
    int32_t sticky = KV_OK;
    bool call_timing = true;           // record per-call start events and keep the last_* statistics (kv_pool_set_call_timing)
    unsigned int wait_polls = KV_WAIT_POLLS;            // bound of the kernels' main-loop waits (kv_pool_set_wait_limit)
    unsigned long long wait_ns = KV_WAIT_NS;
    char err[256];
};

namespace {

int32_t fail(kv_pool *p, int32_t code, const char *msg)
{
    char *dst = p ? p->err : g_err;
    snprintf(dst, 256, "%s", msg);
    return code;
}

int32_t fail_cuda(kv_pool *p, cudaError_t e, const char *what)
{
    char *dst = p ? p->err : g_err;
    snprintf(dst, 256, "%s: %s", what, cudaGetErrorString(e));
    if (p && p->sticky == KV_OK) p->sticky = KV_ERR_CUDA;
    return KV_ERR_CUDA;
}

#define KV_CUDA(p, expr)                                          \
    do {                                                          \
        cudaError_t e_ = (expr);                                  \
        if (e_ != cudaSuccess) return fail_cuda((p), e_, #expr);  \
    } while (0)

bool dev_block_first(const kv_pool *p) { return p->cfg.device_layout == KV_DEV_BLOCK_FIRST; }

KvSide device_side(const kv_pool *p)
{
    if (dev_block_first(p)) return KvSide{(unsigned long long)p->dev, p->blk, p->seg};
    return KvSide{(unsigned long long)p->dev, p->seg, p->cfg.num_gpu_blocks * p->seg};
}

// device address of the first plane of block g, and the distance between its planes
inline uint8_t *dev_block_ptr(const kv_pool *p, int32_t g)
{
    return p->dev + (int64_t)g * (dev_block_first(p) ? p->blk : p->seg);
}
inline size_t dev_pitch(const kv_pool *p)
{
    return (size_t)(dev_block_first(p) ? p->seg : p->cfg.num_gpu_blocks * p->seg);
}

KvSide host_side(const kv_pool *p)
{
    if (p->cfg.host_layout == KV_HOST_LAYER_FIRST)
        return KvSide{(unsigned long long)p->host_dev, p->seg, p->cfg.num_host_blocks * p->seg};
    return KvSide{(unsigned long long)p->host_dev, p->blk, p->seg};
}

// contiguous block-first buffer whose block k sits at base + k*BLK
KvSide packed_side(const kv_pool *p, const void *base)
{
    return KvSide{(unsigned long long)base, p->blk, p->seg};
}

bool use_ldst(const kv_pool *p) { return (p->cfg.flags & KV_FLAG_LDST_KERNEL) != 0; }

// which shape of the bulk kernel's ring a zero-copy launch uses
int link_stage(const kv_pool *p)
{
    return p->cfg.link_variant == 1 ? LINK1_STAGE : (p->cfg.link_variant == 2 ? LINK2_STAGE : LINK_STAGE);
}

// 32-byte vectors in the load/store kernel: zero-copy launches of a pool that asks for them, when every
// address they form is 32-byte aligned
bool ldst32(const kv_pool *p, bool link)
{
    return link && use_ldst(p) && p->cfg.link_variant == 1 && p->seg % 32 == 0 && ((uintptr_t)p->dev & 31) == 0 &&
           ((uintptr_t)p->host_dev & 31) == 0;
}

void fill_geometry(const kv_pool *p, KvJob &job, bool link = false)
{
    const int max_chunk = use_ldst(p) ? LDST_CHUNK : (link ? link_stage(p) : BULK_STAGE);
    // With a block-first device pool against staging, a packed buffer or a block-first host pool, both
    // sides hold a block's planes back to back: the block is one run of BLK bytes and is moved as such,
    // however small its segments are.
    const bool whole_blocks = dev_block_first(p) && (!link || p->cfg.host_layout == KV_HOST_BLOCK_FIRST) &&
                              p->blk <= (int64_t)INT32_MAX;
    const int64_t run = whole_blocks ? p->blk : p->seg;
    job.planes = whole_blocks ? 1 : p->planes;
    job.seg = (int)run;
    job.chunk = (int)std::min<int64_t>(run, max_chunk);
    job.cps = (int)((run + job.chunk - 1) / job.chunk);
    job.status = p->status_dev;
    job.wait_polls = p->wait_polls;
    job.wait_ns = p->wait_ns;
    job.check_ids = (p->cfg.flags & KV_FLAG_DEBUG_BOUNDS) ? 1 : 0;
    job.t_first = job.t_last = nullptr;
}

int clamp_ctas(const KvJob &job, const KvDir &d, int want)
{
    const long long items = (long long)d.n * job.planes * job.cps;
    return (int)std::max<long long>(1, std::min<long long>(want, items));
}

// one shape of the bulk kernel: ring geometry and issuing warps per CTA
template <int STAGE, int NS, int AHEAD, int WARPS>
struct Bulk {
    static_assert(WARPS >= 1 && WARPS <= KV_BULK_MAX_WARPS, "issuing warps per CTA");
    static constexpr int smem = STAGE * NS * WARPS;
    static cudaError_t prepare()
    {
        return cudaFuncSetAttribute(kv_copy_bulk<STAGE, NS, AHEAD>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    }
    static void launch(int grid, cudaStream_t stream, const KvJob &job)
    {
        kv_copy_bulk<STAGE, NS, AHEAD><<<grid, 32 * WARPS, smem, stream>>>(job);
    }
};
// every shape of the bulk kernel that a launch can take, in one table: geometry, and how to prepare and launch it
struct BulkShape {
    int stage, stages, ahead, warps;
    cudaError_t (*prepare)();
    void (*launch)(int grid, cudaStream_t stream, const KvJob &job);
};
template <typename B, int STAGE, int NS, int AHEAD, int WARPS>
constexpr BulkShape bulk_shape()
{
    return BulkShape{STAGE, NS, AHEAD, WARPS, B::prepare, B::launch};
}
#define KV_BULK_SHAPE(STAGE, NS, AHEAD, WARPS) bulk_shape<Bulk<STAGE, NS, AHEAD, WARPS>, STAGE, NS, AHEAD, WARPS>()
const BulkShape g_bulk_shapes[] = {
    /* 0..4: HBM to HBM, by item size */
    KV_BULK_SHAPE(BULK_STAGE, BULK_NS, BULK_AHEAD, 1), KV_BULK_SHAPE(8192, SMALL_NS, SMALL_AHEAD, 2),
    KV_BULK_SHAPE(4096, SMALL_NS, SMALL_AHEAD, 4),     KV_BULK_SHAPE(2048, SMALL_NS, SMALL_AHEAD, 8),
    KV_BULK_SHAPE(1024, TINY_NS, TINY_AHEAD, 16),
    /* 5..7: over the link, link_variant 0 / 1 / 2 */
    KV_BULK_SHAPE(LINK_STAGE, LINK_NS, LINK_AHEAD, 1), KV_BULK_SHAPE(LINK1_STAGE, LINK1_NS, LINK1_AHEAD, 1),
    KV_BULK_SHAPE(LINK2_STAGE, LINK2_NS, LINK2_AHEAD, 1),
    /* 8..10: over the link, small items */
    KV_BULK_SHAPE(4096, SMALL_LINK_NS, SMALL_LINK_AHEAD, 2), KV_BULK_SHAPE(2048, SMALL_LINK_NS, SMALL_LINK_AHEAD, 4),
    KV_BULK_SHAPE(1024, SMALL_LINK_NS, SMALL_LINK_AHEAD, 8)};
#undef KV_BULK_SHAPE

cudaError_t prepare_bulk_kernels()
{
    for (const BulkShape &b : g_bulk_shapes) {
        const cudaError_t rc = b.prepare();
        if (rc != cudaSuccess) return rc;
    }
    return cudaSuccess;
}

// the bulk kernel's shape for items of `chunk` bytes (never smaller than an item: a stage holds one)
const BulkShape &bulk_shape_for(int chunk, bool link, int link_variant)
{
    if (link) {
        if (chunk <= 1024) return g_bulk_shapes[10];
        if (chunk <= 2048) return g_bulk_shapes[9];
        if (chunk <= 4096) return g_bulk_shapes[8];
        return g_bulk_shapes[link_variant == 1 ? 6 : (link_variant == 2 ? 7 : 5)];
    }
    if (chunk <= 1024) return g_bulk_shapes[4];
    if (chunk <= 2048) return g_bulk_shapes[3];
    if (chunk <= 4096) return g_bulk_shapes[2];
    if (chunk <= 8192) return g_bulk_shapes[1];
    return g_bulk_shapes[0];
}

void launch_bulk(const kv_pool *p, const KvJob &job, int grid, cudaStream_t stream, bool link)
{
    bulk_shape_for(job.chunk, link, p ? p->cfg.link_variant : 0).launch(grid, stream, job);
}

cudaError_t launch_job(kv_pool *p, const KvJob &job, cudaStream_t stream, bool link = false)
{
    const int grid = job.dir[0].ctas + job.dir[1].ctas;
    if (grid <= 0) return cudaSuccess;
    if (use_ldst(p)) {
        if (ldst32(p, link)) kv_copy_ldst<LDST_THREADS, LDST32_UNROLL, 32><<<grid, LDST_THREADS, 0, stream>>>(job);
        else kv_copy_ldst<LDST_THREADS, LDST_UNROLL, 16><<<grid, LDST_THREADS, 0, stream>>>(job);
    } else {
        launch_bulk(p, job, grid, stream, link);
    }
    p->stats.kernel_launches++;
    return cudaGetLastError();
}

constexpr int KV_MAX_TIMED = 2048;     // kernel launches per direction timed between two kv_sync calls

// earliest-start words to all ones, latest-end words to zero (a strided 2-D memset each)
cudaError_t preset_ktime(DirState &s, cudaStream_t stream)
{
    cudaError_t rc = cudaMemset2DAsync(s.ktime_dev, 16, 0xFF, 8, KV_MAX_TIMED, stream);
    if (rc != cudaSuccess) return rc;
    return cudaMemset2DAsync(s.ktime_dev + 1, 16, 0x00, 8, KV_MAX_TIMED, stream);
}

// HBM-to-HBM gather / scatter launch, bracketed by events on its stream when kernel timing is on, and
// then also timed from inside (first CTA start to last CTA end), which leaves out the wait for the launch
cudaError_t launch_timed(kv_pool *p, DirState &s, cudaStream_t stream, KvJob job, int64_t payload_bytes)
{
    const bool timed = (p->cfg.flags & KV_FLAG_TIME_KERNELS) && s.kev_used < KV_MAX_TIMED;
    if (timed) {
        if (!s.ktime_dev) {
            // allocated and preset once; kv_sync presets the slots again after reading them
            cudaError_t rc = cudaMalloc((void **)&s.ktime_dev, (size_t)KV_MAX_TIMED * 2 * sizeof(unsigned long long));
            if (rc != cudaSuccess) return rc;
            rc = preset_ktime(s, stream);
            if (rc == cudaSuccess) rc = cudaStreamSynchronize(stream);   // once: later launches may come from another stream
            if (rc != cudaSuccess) return rc;
        }
        job.t_first = s.ktime_dev + 2 * (size_t)s.kev_used;
        job.t_last = job.t_first + 1;
        while ((int)s.kev.size() < 2 * (s.kev_used + 1)) {
            cudaEvent_t e;
            cudaError_t rc = cudaEventCreate(&e);
            if (rc != cudaSuccess) return rc;
            s.kev.push_back(e);
        }
        if ((int)s.kev_bytes.size() <= s.kev_used) s.kev_bytes.resize((size_t)s.kev_used + 1);
        cudaError_t rc = cudaEventRecord(s.kev[2 * (size_t)s.kev_used], stream);
        if (rc != cudaSuccess) return rc;
    }
    cudaError_t rc = launch_job(p, job, stream);
    if (rc != cudaSuccess) return rc;
    if (timed) {
        rc = cudaEventRecord(s.kev[2 * (size_t)s.kev_used + 1], stream);
        if (rc != cudaSuccess) return rc;
        s.kev_bytes[(size_t)s.kev_used] = payload_bytes;
        s.kev_used++;
    }
    return cudaSuccess;
}

// ---------------------------------------------------------------------------------------------
// validation

int32_t check_ids(kv_pool *p, const int32_t *ids, int64_t n, int64_t nb, const char *what)
{
    for (int64_t i = 0; i < n; ++i)
        if (ids[i] < 0 || (int64_t)ids[i] >= nb) {
            snprintf(p->err, 256, "%s[%lld] = %d outside [0, %lld)", what, (long long)i, ids[i], (long long)nb);
            return KV_ERR_RANGE;
        }
    return KV_OK;
}

int32_t check_unique(kv_pool *p, const int32_t *ids, int64_t n, std::vector<uint32_t> &mark, const char *what)
{
    const uint32_t e = ++p->epoch;
    for (int64_t i = 0; i < n; ++i) {
        if (mark[ids[i]] == e) {
            snprintf(p->err, 256, "%s: destination block %d listed twice", what, ids[i]);
            return KV_ERR_DUP_DST;
        }
        mark[ids[i]] = e;
    }
    return KV_OK;
}

int32_t check_direction(kv_pool *p, const int32_t *gpu_ids, const int32_t *host_ids, int64_t n, bool out)
{
    if (n < 0) return fail(p, KV_ERR_INVALID_ARG, "negative count");
    if (n == 0) return KV_OK;
    if (!gpu_ids || !host_ids) return fail(p, KV_ERR_INVALID_ARG, "null id list");
    if (n > p->cap) return fail(p, KV_ERR_INVALID_ARG, "more pairs than the pools have blocks");
    int32_t rc = check_ids(p, gpu_ids, n, p->cfg.num_gpu_blocks, out ? "swap-out gpu_ids" : "swap-in gpu_ids");
    if (rc != KV_OK) return rc;
    rc = check_ids(p, host_ids, n, p->cfg.num_host_blocks, out ? "swap-out host_ids" : "swap-in host_ids");
    if (rc != KV_OK) return rc;
    return out ? check_unique(p, host_ids, n, p->h_mark, "swap-out")
               : check_unique(p, gpu_ids, n, p->g_mark, "swap-in");
}

// ---------------------------------------------------------------------------------------------
// ordering between the two directions

void poll_done(kv_pool *p)
{
    for (int d = 0; d < 2; ++d) {
        DirState &s = p->dir[d];
        if (s.done < s.issued && cudaEventQuery(s.ev_end[s.issued % KV_SLOTS]) == cudaSuccess) s.done = s.issued;
    }
}

// does a new call of direction `d` touch a block that an unfinished call of the other direction uses?
// (host_ids == nullptr: a device-side gather / scatter, which names device blocks only)
bool conflicts_with_other(kv_pool *p, int d, const int32_t *gpu_ids, const int32_t *host_ids, int64_t n)
{
    const DirState &o = p->dir[1 - d];
    if (o.done >= o.issued) return false;
    const std::vector<uint64_t> &gside = (d == 0) ? p->g_written_by_in : p->g_read_by_out;
    const std::vector<uint64_t> &hside = (d == 0) ? p->h_read_by_in : p->h_written_by_out;
    for (int64_t i = 0; i < n; ++i)
        if (gside[gpu_ids[i]] > o.done || (host_ids && hside[host_ids[i]] > o.done)) return true;
    return false;
}

void note_use(kv_pool *p, int d, const int32_t *gpu_ids, const int32_t *host_ids, int64_t n, uint64_t seq)
{
    std::vector<uint64_t> &gside = (d == 0) ? p->g_read_by_out : p->g_written_by_in;
    std::vector<uint64_t> &hside = (d == 0) ? p->h_written_by_out : p->h_read_by_in;
    for (int64_t i = 0; i < n; ++i) {
        gside[gpu_ids[i]] = seq;
        if (host_ids) hside[host_ids[i]] = seq;
    }
}

// ---------------------------------------------------------------------------------------------
// one direction of one call

struct DirCall {
    int d;                      // 0 out, 1 in
    const int32_t *gpu_ids;
    const int32_t *host_ids;
    int64_t n;
    int slot;
    int2 *pairs_host, *pairs_dev;      // (src id, dst id)
    int2 *aux_host, *aux_dev;          // (gpu id, position in list) for pack/unpack
    int path;
    // copy-engine issue state (CE paths are issued in slices so the two directions interleave)
    int64_t ce_next = 0;
    bool planned = false;              // STAGED: plan_staged has run for this call
    int64_t plan_nruns = 0;            //         runs of consecutive host ids in its list
    bool plan_uniform = false;         //         the plan uses uniform two-block transfers
    int chunk_idx = 0;                 // STAGED: chunk being issued, next op of it
    int op_next = 0;
    bool chunk_open = false;
    unsigned rr = 0;                   // round-robin cursor over the direction's CE streams
};

// fork: the extra streams of a CE direction wait for everything issued so far on its main stream
int32_t ce_fork(kv_pool *p, DirState &s)
{
    if (s.nsub <= 1) return KV_OK;
    KV_CUDA(p, cudaEventRecord(s.fork_ev, s.stream));
    for (int k = 1; k < s.nsub; ++k) KV_CUDA(p, cudaStreamWaitEvent(s.sub[k], s.fork_ev, 0));
    return KV_OK;
}

// join: the main stream waits for everything issued on the extra streams
int32_t ce_join(kv_pool *p, DirState &s)
{
    for (int k = 1; k < s.nsub; ++k) {
        KV_CUDA(p, cudaEventRecord(s.join_ev[k], s.sub[k]));
        KV_CUDA(p, cudaStreamWaitEvent(s.stream, s.join_ev[k], 0));
    }
    return KV_OK;
}

// STAGED path, host side of one direction of one call: sort the pairs by host id, turn the sorted list
// into copy-engine transfers (long ones where the host ids form long runs, uniform two-block ones
// otherwise), and cut that sequence into chunks of at most a staging half.
//   - a run of consecutive host ids is one plain transfer;
//   - runs of equal length whose starts are equally spaced become one strided 2-D transfer (any two
//     runs are "equally spaced", so isolated blocks still travel two per transfer).
// The cost of a transfer on the copy engine is a fixed start-up plus its bytes, so fewer and larger
// transfers are what keeps the link busy.
struct PlanParams {
    int64_t blk, seg, half_blocks, max_pitch, num_host_blocks;
    int planes;
    bool layer_first;           // host pool layout
};

// Where the sorted list is cut into chunks: chunk number k holds `first` blocks, then twice as much each
// time, up to `chunk`; the boundaries depend on n alone and no transfer crosses one.  With `even`, chunks
// hold an even number of blocks (two-block transfers are never split into singles).
std::vector<int64_t> chunk_bounds(int64_t n, int64_t first, int64_t chunk, bool even)
{
    std::vector<int64_t> bounds{0};
    while (bounds.back() < n) {
        const size_t k = bounds.size() - 1;
        int64_t take = k < 40 ? std::min(chunk, first << k) : chunk;
        if (even && take > 1) take &= ~(int64_t)1;
        bounds.push_back(std::min(n, bounds.back() + take));
    }
    return bounds;
}

// Scattered host ids, four blocks per transfer.  Four blocks whose host ids form a 2 x 2 lattice
// (a, a+g, a+kg, a+kg+g) are one 3-D copy-engine transfer: two rows g blocks apart, two slices k rows apart,
// and a transfer of four blocks runs at the rate of one twice as long as a pair's (measured both ways: 97
// against 94 GB/s for 2 MiB blocks).  Two pairs (x, x+g) and (x', x'+g) form such a lattice exactly when
// their starts are congruent modulo g, so one sweep over the sorted ids keeps, per (g, x mod g), one pair
// still waiting for a partner and closes a lattice whenever a second one turns up: a few probes per
// block, and about three quarters of a uniformly scattered list find a place (95 % of a denser one).  The
// blocks left over travel as before, two per transfer.  `order` comes in sorted by host id and leaves as the
// staging order: the blocks of each transfer next to one another, transfers in issue order (lattices first).
// Returns false, touching nothing, when no lattice is found.
bool plan_lattices(const PlanParams &pp, const int32_t *host_ids, int64_t n, int64_t first, int64_t chunk,
                   std::vector<int32_t> &order, std::vector<CeOp> &ops, std::vector<CeChunk> &chunks)
{
    const std::vector<int32_t> sorted = order;
    auto hid = [&](int64_t q) { return (int64_t)host_ids[sorted[(size_t)q]]; };
    const int64_t gmax = std::min<int64_t>(KV_QUAD_MAX_GAP, pp.max_pitch / pp.blk);
    // blocks of 4 MiB and more already travel in pairs of 8 MiB and more, which run at the link's rate:
    // lattices would only add a second transfer size (measured with 8 MiB blocks: 92 GB/s against 96-99)
    if (gmax < 1 || chunk < 4 || n < 8 || 2 * pp.blk >= KV_QUAD_ENOUGH_BYTES) return false;
    struct Slot {
        uint64_t key;
        int32_t i, j;
    };
    int bits = 6;
    while (((size_t)1 << bits) < (size_t)(2 * KV_QUAD_PARTNERS * n)) ++bits;
    const size_t cap = (size_t)1 << bits;
    std::vector<Slot> table(cap, Slot{~0ull, -1, -1});
    std::vector<uint8_t> used((size_t)n, 0);
    struct Quad {
        int32_t q[4];
        int64_t g, k;
    };
    std::vector<Quad> quads;
    for (int64_t i = 0; i < n; ++i) {
        if (used[(size_t)i]) continue;
        const int64_t x = hid(i);
        int tried = 0;
        for (int64_t j = i + 1; j < n && tried < KV_QUAD_PARTNERS; ++j) {
            const int64_t g = hid(j) - x;
            if (g > gmax) break;
            if (g == 0 || used[(size_t)j]) continue;
            ++tried;
            const uint64_t key = ((uint64_t)g << 32) | (uint64_t)(x % g);
            size_t h = (size_t)((key * 0x9E3779B97F4A7C15ull) >> (64 - bits));
            while (table[h].key != ~0ull && table[h].key != key) h = (h + 1) & (cap - 1);
            Slot &w = table[h];
            const bool waiting = w.key == key && w.i >= 0 && !used[(size_t)w.i] && !used[(size_t)w.j];
            if (waiting && x - hid(w.i) >= 2 * g) {
                quads.push_back(Quad{{w.i, w.j, (int32_t)i, (int32_t)j}, g, (x - hid(w.i)) / g});
                used[(size_t)w.i] = used[(size_t)w.j] = used[(size_t)i] = used[(size_t)j] = 1;
                w.i = w.j = -1;
                break;
            }
            if (waiting) continue;       // the waiting pair ends where this one starts (an arithmetic run): it keeps waiting
            w.key = key;
            w.i = (int32_t)i;
            w.j = (int32_t)j;
        }
    }
    if (quads.empty()) return false;
    ops.clear();
    chunks.clear();
    int64_t pos = 0;
    for (const Quad &qd : quads) {
        CeOp op{hid(qd.q[0]) * pp.blk, 0, pp.blk, qd.g * pp.blk, 2, pos, 4};
        op.slices = 2;
        op.slice_rows = qd.k;
        for (int t = 0; t < 4; ++t) order[(size_t)(pos + t)] = sorted[(size_t)qd.q[t]];
        ops.push_back(op);
        pos += 4;
    }
    // the rest, ascending, two per transfer (a single where the gap does not fit a row pitch, or at the end)
    std::vector<int64_t> rest;
    for (int64_t i = 0; i < n; ++i)
        if (!used[(size_t)i]) rest.push_back(i);
    for (size_t t = 0; t < rest.size();) {
        CeOp op{hid(rest[t]) * pp.blk, 0, pp.blk, pp.blk, 1, pos, 1};
        order[(size_t)pos] = sorted[(size_t)rest[t]];
        if (t + 1 < rest.size()) {
            const int64_t pitch = (hid(rest[t + 1]) - hid(rest[t])) * pp.blk;
            if (pitch >= op.width && pitch <= pp.max_pitch) {
                op.host_pitch = pitch;
                op.rows = 2;
                op.nblk = 2;
                order[(size_t)(pos + 1)] = sorted[(size_t)rest[t + 1]];
            }
        }
        ops.push_back(op);
        pos += op.nblk;
        t += (size_t)op.nblk;
    }
    // chunks: filled transfer by transfer up to the size the doubling rule gives chunk number k (a multiple
    // of four blocks, so that lattices fill it exactly)
    CeChunk ch{0, 0, 0, 0};
    for (size_t a = 0; a < ops.size(); ++a) {
        const size_t k = chunks.size();
        const int64_t base = k < 40 ? std::min(chunk, first << k) : chunk;
        const int64_t cap_k = base >= n ? n : std::max<int64_t>(4, base & ~(int64_t)3);
        if (ops[a].pos > ch.lo && ops[a].pos - ch.lo + ops[a].nblk > cap_k) {
            ch.hi = ops[a].pos;
            ch.op_hi = (int32_t)a;
            chunks.push_back(ch);
            ch = CeChunk{ops[a].pos, ops[a].pos, (int32_t)a, 0};
        }
        ops[a].stage_off = (ops[a].pos - ch.lo) * pp.blk;
    }
    ch.hi = n;
    ch.op_hi = (int32_t)ops.size();
    chunks.push_back(ch);
    return true;
}

// Pure planning (no pool, no CUDA): order, transfers and chunks for n pairs of direction d (0 out, 1 in)
// whose host block ids are host_ids.  May throw std::bad_alloc.
// mode: -1 = decide from this list's runs, 0 = merge runs, 1 = uniform two-block transfers;
// *nruns_out / *uniform_out (may be null) report the list's runs of consecutive host ids and the mode taken.
void plan_transfers(const PlanParams &pp, int d, const int32_t *host_ids, int64_t n, std::vector<int32_t> &order,
                    std::vector<CeOp> &ops, std::vector<CeChunk> &chunks, int mode = -1, int64_t *nruns_out = nullptr,
                    bool *uniform_out = nullptr)
{
    {
        order.resize((size_t)n);
        for (int64_t i = 0; i < n; ++i) order[(size_t)i] = (int32_t)i;
        if (!pp.layer_first)
            std::sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return host_ids[a] < host_ids[b]; });
        ops.clear();
        chunks.clear();
        // A small call (KV_PLAN_ONE_CHUNK_BYTES or less) goes through staging as one chunk: every chunk
        // boundary is a hand-off between the kernel stream and the copy stream, which costs about 65 us while
        // the other direction keeps the link busy, and packing 128 MiB takes 20 us (measured with both
        // directions busy, 64 MB each way: 88-92 GB/s in one chunk against 80-85 in four).  A larger call
        // that would fit one half is still cut into about four chunks, so that its own packing, transfers and
        // unpacking overlap instead of following one another, and the first chunk of a swap-out is half as
        // long as the rest: its first transfer starts sooner.
        const int64_t min_chunk = std::max<int64_t>(1, (8ll << 20) / pp.blk);
        const bool one_chunk = n * pp.blk <= KV_PLAN_ONE_CHUNK_BYTES;
        int64_t chunk = std::min(pp.half_blocks, one_chunk ? n : std::max(min_chunk, (n + KV_PLAN_CHUNKS - 1) / KV_PLAN_CHUNKS));
        {
            // as many chunks as that size needs, but of equal size (a multiple of four blocks where the half
            // allows it), so that no call ends on a chunk of a few blocks and a hand-off of its own
            const int64_t pieces = (n + chunk - 1) / chunk;
            const int64_t even = (((n + pieces - 1) / pieces) + 3) & ~(int64_t)3;
            chunk = std::min(pp.half_blocks, std::max(chunk, even));
        }
        const int64_t first = (d == 0 && n > chunk && !one_chunk) ? std::max<int64_t>(1, chunk / 2) : chunk;
        if (pp.layer_first) {
            // one strided transfer per block: `planes` rows of SEG bytes, a whole host plane apart
            const std::vector<int64_t> bounds = chunk_bounds(n, first, chunk, false);
            for (size_t q = 0; q + 1 < bounds.size(); ++q) {
                const int64_t lo = bounds[q], hi = bounds[q + 1];
                CeChunk ch{lo, hi, (int32_t)ops.size(), 0};
                for (int64_t k = lo; k < hi; ++k)
                    ops.push_back(CeOp{(int64_t)host_ids[order[(size_t)k]] * pp.seg, (k - lo) * pp.blk, pp.seg,
                                         pp.num_host_blocks * pp.seg, pp.planes, k, 1});
                ch.op_hi = (int32_t)ops.size();
                chunks.push_back(ch);
            }
            return;
        }
        // Transfers over the sorted list, chunk by chunk.
        // Measured with both directions busy: transfers that all carry the same number of bytes keep the
        // two copy engines in step and share the link evenly (2 x 2 MiB everywhere: 93.9 GB/s), while a
        // mix of sizes loses 8 % (85.6 GB/s for mostly pairs with a few singles and triples), whatever
        // the order of issue.  Merging neighbouring host blocks into long transfers only pays once the
        // runs are long (mean of 8 blocks and more: 89 to 99 GB/s); below that every block is treated
        // as a single and sent with its neighbour in the sorted list, two per transfer, all alike.
        auto hid = [&](int64_t q) { return (int64_t)host_ids[order[(size_t)q]]; };
        int64_t nruns = 1;
        for (int64_t q = 1; q < n; ++q)
            if (hid(q) != hid(q - 1) + 1) ++nruns;
        const bool uniform = mode < 0 ? n < KV_MERGE_MIN_MEAN_RUN * nruns : mode == 1;
        if (nruns_out) *nruns_out = nruns;
        if (uniform_out) *uniform_out = uniform;
        if (uniform && plan_lattices(pp, host_ids, n, first, chunk, order, ops, chunks)) return;
        const std::vector<int64_t> bounds = chunk_bounds(n, first, chunk, uniform);
        for (size_t q = 0; q + 1 < bounds.size(); ++q) {
            const int64_t lo = bounds[q], hi = bounds[q + 1];
            auto run_len = [&](int64_t k) {
                int64_t r = 1;
                if (uniform) return r;
                while (k + r < hi && hid(k + r) == hid(k) + r) ++r;
                return r;
            };
            CeChunk ch{lo, hi, (int32_t)ops.size(), 0};
            for (int64_t k = lo; k < hi;) {
                const int64_t r = run_len(k);
                // the staging slot of sorted position k is (k - lo) * BLK into the chunk's half
                CeOp op{hid(k) * pp.blk, (k - lo) * pp.blk, r * pp.blk, r * pp.blk, 1, k, (int32_t)r};
                int64_t nxt = k + r;
                // further runs of the same length at a constant spacing join as extra rows (uniform mode: one)
                while (nxt < hi && run_len(nxt) == r && nxt + r <= hi && !(uniform && op.rows >= 2)) {
                    const int64_t pitch = (hid(nxt) - hid(nxt - r)) * pp.blk;
                    if (pitch < op.width || pitch > pp.max_pitch || (op.rows > 1 && pitch != op.host_pitch)) break;
                    op.host_pitch = pitch;
                    op.rows++;
                    op.nblk += (int32_t)r;
                    nxt += r;
                }
                ops.push_back(op);
                k = nxt;
            }
            ch.op_hi = (int32_t)ops.size();
            chunks.push_back(ch);
        }
    }
}

int32_t plan_staged(kv_pool *p, DirCall &c, int mode = -1)
{
    DirState &s = p->dir[c.d];
    const PlanParams pp{p->blk, p->seg, s.half_blocks, p->max_pitch, p->cfg.num_host_blocks, p->planes,
                        p->cfg.host_layout == KV_HOST_LAYER_FIRST};
    try {
        plan_transfers(pp, c.d, c.host_ids, c.n, s.order, s.ops, s.chunks, mode, &c.plan_nruns, &c.plan_uniform);
    } catch (...) {
        return fail(p, KV_ERR_NOMEM, "out of host memory");
    }
    c.planned = true;
    return KV_OK;
}

// Everything about a direction of a call that can be refused for lack of memory (the staging buffer, the
// transfer plan).  Runs for every direction of a call before any of them is begun, so that a refusal
// leaves no direction half issued: no sequence number taken, no block marked as in use.
int32_t prepare_dir(kv_pool *p, DirCall &c)
{
    DirState &s = p->dir[c.d];
    if (c.path != KV_PATH_STAGED) return KV_OK;
    if (!s.stage) {
        cudaError_t e = cudaMalloc((void **)&s.stage, (size_t)(2 * s.half_blocks * p->blk));
        if (e != cudaSuccess) {
            s.stage = nullptr;
            (void)cudaGetLastError();
            return fail(p, KV_ERR_NOMEM, "staging buffer allocation failed");
        }
    }
    if (!c.planned) return plan_staged(p, c);
    return KV_OK;
}

// wait_for: end event of the other direction's call this one must follow, or nullptr
int32_t begin_dir(kv_pool *p, DirCall &c, cudaEvent_t wait_for)
{
    DirState &s = p->dir[c.d];
    const uint64_t seq = s.issued + 1;
    c.slot = (int)(seq % KV_SLOTS);
    if (seq > KV_SLOTS && s.done + KV_SLOTS < seq) KV_CUDA(p, cudaEventSynchronize(s.ev_end[c.slot]));   // slot's previous user
    c.pairs_host = s.ring_host + (size_t)c.slot * 2 * p->cap;
    c.pairs_dev = s.ring_dev + (size_t)c.slot * 2 * p->cap;
    c.aux_host = c.pairs_host + p->cap;
    c.aux_dev = c.pairs_dev + p->cap;
    if (c.path == KV_PATH_STAGED) {
        // the kernel sees (device block id, position in the sorted list)
        for (int64_t k = 0; k < c.n; ++k) {
            const int32_t g = c.gpu_ids[s.order[(size_t)k]];
            c.aux_host[k] = (c.d == 0) ? make_int2(g, (int)k) : make_int2((int)k, g);
        }
    } else if (c.path == KV_PATH_ZEROCOPY && c.n > KV_INLINE_PAIRS) {
        for (int64_t i = 0; i < c.n; ++i)
            c.pairs_host[i] = (c.d == 0) ? make_int2(c.gpu_ids[i], c.host_ids[i]) : make_int2(c.host_ids[i], c.gpu_ids[i]);
    }
    if (wait_for) KV_CUDA(p, cudaStreamWaitEvent(s.stream, wait_for, 0));
    if (p->call_timing) KV_CUDA(p, cudaEventRecord(s.ev_start[c.slot], s.stream));
    if (c.path == KV_PATH_ZEROCOPY) {
        // a short list travels in the launch parameters instead (zerocopy_dir)
        if (c.n > KV_INLINE_PAIRS)
            KV_CUDA(p, cudaMemcpyAsync(c.pairs_dev, c.pairs_host, (size_t)c.n * sizeof(int2), cudaMemcpyHostToDevice, s.stream));
    } else if (c.path == KV_PATH_STAGED) {
        // chunks of KV_INLINE_PAIRS blocks or fewer carry their ids in the launch parameters (ce_issue_some)
        bool ids_on_device = false;
        for (const CeChunk &ch : s.chunks) ids_on_device = ids_on_device || ch.hi - ch.lo > KV_INLINE_PAIRS;
        if (ids_on_device)
            KV_CUDA(p, cudaMemcpyAsync(c.aux_dev, c.aux_host, (size_t)c.n * sizeof(int2), cudaMemcpyHostToDevice, s.stream));
        // the kernel stream starts after everything issued so far on this direction
        KV_CUDA(p, cudaEventRecord(s.kfork_ev, s.stream));
        KV_CUDA(p, cudaStreamWaitEvent(s.kstream, s.kfork_ev, 0));
    }
    if (c.path == KV_PATH_CE2D || c.path == KV_PATH_NAIVE) {
        int32_t rc = ce_fork(p, s);
        if (rc != KV_OK) return rc;
    }
    s.issued = seq;
    note_use(p, c.d, c.gpu_ids, c.host_ids, c.n, seq);
    return KV_OK;
}

int32_t end_dir(kv_pool *p, DirCall &c)
{
    DirState &s = p->dir[c.d];
    if (c.path == KV_PATH_CE2D || c.path == KV_PATH_NAIVE) {
        int32_t rc = ce_join(p, s);
        if (rc != KV_OK) return rc;
    }
    if (c.path == KV_PATH_STAGED && c.d == 1) {
        // the call ends when the last unpack kernels have run (they are on the kernel stream)
        const int nch = (int)s.chunks.size();
        for (int q = std::max(0, nch - 2); q < nch; ++q) KV_CUDA(p, cudaStreamWaitEvent(s.stream, s.ev_b[q & 1], 0));
    }
    KV_CUDA(p, cudaEventRecord(s.ev_end[c.slot], s.stream));
    const int64_t bytes = c.n * p->blk;
    if (c.d == 0) {
        p->stats.bytes_out += bytes;
        p->stats.calls_out++;
        p->stats.last_path_out = c.path;
    } else {
        p->stats.bytes_in += bytes;
        p->stats.calls_in++;
        p->stats.last_path_in = c.path;
    }
    return KV_OK;
}

// direction `k` of `job` := the zero-copy description of call c
void zerocopy_dir(kv_pool *p, const DirCall &c, KvJob &job, int k)
{
    KvDir &d = job.dir[k];
    d.src = (c.d == 0) ? device_side(p) : host_side(p);
    d.dst = (c.d == 0) ? host_side(p) : device_side(p);
    d.n = (int)c.n;
    d.ctas = 0;
    d.src_blocks = (int)(c.d == 0 ? p->cfg.num_gpu_blocks : p->cfg.num_host_blocks);
    d.dst_blocks = (int)(c.d == 0 ? p->cfg.num_host_blocks : p->cfg.num_gpu_blocks);
    if (c.n <= KV_INLINE_PAIRS) {
        d.pairs = nullptr;
        for (int64_t i = 0; i < c.n; ++i)
            job.inl[k][i] = (c.d == 0) ? make_int2(c.gpu_ids[i], c.host_ids[i]) : make_int2(c.host_ids[i], c.gpu_ids[i]);
    } else {
        d.pairs = c.pairs_dev;
    }
}

// host address of the start of host block h (block-first) or of its first plane (layer-first)
inline uint8_t *host_block_ptr(const kv_pool *p, int32_t h)
{
    return p->host + (int64_t)h * (p->cfg.host_layout == KV_HOST_LAYER_FIRST ? p->seg : p->blk);
}
inline size_t host_pitch(const kv_pool *p)
{
    return (size_t)(p->cfg.host_layout == KV_HOST_LAYER_FIRST ? p->cfg.num_host_blocks * p->seg : p->seg);
}

// Issue up to `budget` copy-engine operations of a CE-path direction; returns true when the
// direction has nothing left to issue.
int32_t ce_issue_some(kv_pool *p, DirCall &c, int budget, bool &finished)
{
    DirState &s = p->dir[c.d];
    const cudaMemcpyKind kind = (c.d == 0) ? cudaMemcpyDeviceToHost : cudaMemcpyHostToDevice;
    finished = false;
    if (c.path == KV_PATH_NAIVE) {
        // one transfer per segment
        const int64_t total = c.n * p->planes;
        while (budget-- > 0 && c.ce_next < total) {
            const int64_t i = c.ce_next / p->planes, pl = c.ce_next % p->planes;
            uint8_t *dv = dev_block_ptr(p, c.gpu_ids[i]) + pl * (int64_t)dev_pitch(p);
            uint8_t *hv = host_block_ptr(p, c.host_ids[i]) + pl * (int64_t)host_pitch(p);
            KV_CUDA(p, cudaMemcpyAsync(c.d == 0 ? hv : dv, c.d == 0 ? dv : hv, (size_t)p->seg, kind, s.sub[i % s.nsub]));
            p->stats.ce_copies++;
            c.ce_next++;
        }
        finished = c.ce_next >= total;
        return KV_OK;
    }
    if (c.path == KV_PATH_CE2D) {
        // one transfer per block: `planes` rows of SEG bytes, strided where a pool is layer-first; a
        // plain BLK-byte transfer when both pools are block-first (the paper's one-copy-per-merged-region)
        while (budget-- > 0 && c.ce_next < c.n) {
            const int64_t i = c.ce_next;
            uint8_t *dv = dev_block_ptr(p, c.gpu_ids[i]);
            uint8_t *hv = host_block_ptr(p, c.host_ids[i]);
            const size_t dpitch = dev_pitch(p);
            cudaStream_t cs = s.sub[i % s.nsub];
            if (dpitch == (size_t)p->seg && host_pitch(p) == (size_t)p->seg)
                KV_CUDA(p, cudaMemcpyAsync(c.d == 0 ? hv : dv, c.d == 0 ? dv : hv, (size_t)p->blk, kind, cs));
            else if (c.d == 0)
                KV_CUDA(p, cudaMemcpy2DAsync(hv, host_pitch(p), dv, dpitch, (size_t)p->seg, (size_t)p->planes, kind, cs));
            else
                KV_CUDA(p, cudaMemcpy2DAsync(dv, dpitch, hv, host_pitch(p), (size_t)p->seg, (size_t)p->planes, kind, cs));
            p->stats.ce_copies++;
            c.ce_next++;
        }
        finished = c.ce_next >= c.n;
        return KV_OK;
    }
    // STAGED: chunk q of the sorted list goes through staging half q & 1.
    //   out: kernel stream packs the half, then the transfers drain it on the direction's stream;
    //   in:  the transfers fill the half, then the kernel stream unpacks it.
    // While one half is on the link the other is being packed / unpacked.
    while (budget > 0 && c.chunk_idx < (int)s.chunks.size()) {
        const CeChunk &ch = s.chunks[(size_t)c.chunk_idx];
        const int b = c.chunk_idx & 1;
        uint8_t *half = s.stage + (size_t)b * (size_t)(s.half_blocks * p->blk);
        KvJob job;
        fill_geometry(p, job);
        job.dir[1] = KvDir{};
        KvDir &kd = job.dir[0];
        // the staging slot of sorted position k is half + (k - lo)*BLK
        const KvSide st = packed_side(p, half - ch.lo * p->blk);
        kd.src = (c.d == 0) ? device_side(p) : st;
        kd.dst = (c.d == 0) ? st : device_side(p);
        kd.pairs = c.aux_dev + ch.lo;
        kd.n = (int)(ch.hi - ch.lo);
        if (kd.n <= KV_INLINE_PAIRS) {
            kd.pairs = nullptr;
            for (int q = 0; q < kd.n; ++q) job.inl[0][q] = c.aux_host[ch.lo + q];
        }
        // staging-side "ids" are positions of the sorted list, below ch.hi
        kd.src_blocks = (int)(c.d == 0 ? p->cfg.num_gpu_blocks : ch.hi);
        kd.dst_blocks = (int)(c.d == 0 ? ch.hi : p->cfg.num_gpu_blocks);
        kd.ctas = clamp_ctas(job, kd, p->sm_count);
        if (!c.chunk_open) {
            if (c.d == 0) {
                if (c.chunk_idx >= 2) KV_CUDA(p, cudaStreamWaitEvent(s.kstream, s.ev_b[b], 0));
                KV_CUDA(p, launch_timed(p, s, s.kstream, job, (ch.hi - ch.lo) * p->blk));
                KV_CUDA(p, cudaEventRecord(s.ev_a[b], s.kstream));
                KV_CUDA(p, cudaStreamWaitEvent(s.stream, s.ev_a[b], 0));
            } else if (c.chunk_idx >= 2) {
                KV_CUDA(p, cudaStreamWaitEvent(s.stream, s.ev_b[b], 0));
            }
            c.chunk_open = true;
            c.op_next = ch.op_lo;
        }
        while (budget > 0 && c.op_next < ch.op_hi) {
            const CeOp &op = s.ops[(size_t)c.op_next];
            uint8_t *hv = p->host + op.host_off, *sv = half + op.stage_off;
            if (op.slices > 1) {
                cudaMemcpy3DParms p3 = {};
                const cudaPitchedPtr hpp = make_cudaPitchedPtr(hv, (size_t)op.host_pitch, (size_t)op.width, (size_t)op.slice_rows);
                const cudaPitchedPtr spp = make_cudaPitchedPtr(sv, (size_t)op.width, (size_t)op.width, (size_t)op.rows);
                p3.srcPtr = c.d == 0 ? spp : hpp;
                p3.dstPtr = c.d == 0 ? hpp : spp;
                p3.extent = make_cudaExtent((size_t)op.width, (size_t)op.rows, (size_t)op.slices);
                p3.kind = kind;
                KV_CUDA(p, cudaMemcpy3DAsync(&p3, s.stream));
            } else if (op.rows == 1) {
                KV_CUDA(p, cudaMemcpyAsync(c.d == 0 ? hv : sv, c.d == 0 ? sv : hv, (size_t)op.width, kind, s.stream));
            } else if (c.d == 0) {
                KV_CUDA(p, cudaMemcpy2DAsync(hv, (size_t)op.host_pitch, sv, (size_t)op.width, (size_t)op.width, (size_t)op.rows, kind, s.stream));
            } else {
                KV_CUDA(p, cudaMemcpy2DAsync(sv, (size_t)op.width, hv, (size_t)op.host_pitch, (size_t)op.width, (size_t)op.rows, kind, s.stream));
            }
            p->stats.ce_copies++;
            c.op_next++;
            --budget;
        }
        if (c.op_next >= ch.op_hi) {
            if (c.d == 0) {
                KV_CUDA(p, cudaEventRecord(s.ev_b[b], s.stream));
            } else {
                KV_CUDA(p, cudaEventRecord(s.ev_a[b], s.stream));
                KV_CUDA(p, cudaStreamWaitEvent(s.kstream, s.ev_a[b], 0));
                KV_CUDA(p, launch_timed(p, s, s.kstream, job, (ch.hi - ch.lo) * p->blk));
                KV_CUDA(p, cudaEventRecord(s.ev_b[b], s.kstream));
            }
            c.chunk_idx++;
            c.chunk_open = false;
        }
    }
    finished = c.chunk_idx >= (int)s.chunks.size();
    return KV_OK;
}

// Issue the payload movement of up to two prepared directions.
int32_t issue_calls(kv_pool *p, DirCall *calls, int ncalls, bool fused)
{
    // kernel (zero-copy) directions
    if (fused && ncalls == 2 && calls[0].path == KV_PATH_ZEROCOPY && calls[1].path == KV_PATH_ZEROCOPY) {
        KvJob job;
        fill_geometry(p, job, true);
        zerocopy_dir(p, calls[0], job, 0);
        zerocopy_dir(p, calls[1], job, 1);
        job.dir[0].ctas = clamp_ctas(job, job.dir[0], p->dir[0].ctas);
        job.dir[1].ctas = clamp_ctas(job, job.dir[1], p->dir[1].ctas);
        KV_CUDA(p, launch_job(p, job, p->dir[0].stream, true));
        return KV_OK;
    }
    for (int k = 0; k < ncalls; ++k) {
        DirCall &c = calls[k];
        if (c.path != KV_PATH_ZEROCOPY) continue;
        KvJob job;
        fill_geometry(p, job, true);
        zerocopy_dir(p, c, job, 0);
        job.dir[1] = KvDir{};
        job.dir[0].ctas = clamp_ctas(job, job.dir[0], p->dir[c.d].ctas);
        KV_CUDA(p, launch_job(p, job, p->dir[c.d].stream, true));
    }
    // copy-engine directions, interleaved in slices so that both streams are fed from the start
    bool fin[2] = {true, true};
    for (int k = 0; k < ncalls; ++k) fin[k] = (calls[k].path == KV_PATH_ZEROCOPY);
    while (!(fin[0] && fin[1])) {
        for (int k = 0; k < ncalls; ++k) {
            if (fin[k]) continue;
            int32_t rc = ce_issue_some(p, calls[k], 8, fin[k]);
            if (rc != KV_OK) return rc;
        }
    }
    return KV_OK;
}

// may_fuse: the caller (kv_rotate with lists that do not overlap and wait for nothing) allows both
// directions to share one launch; whether they do is decided here, once the paths are known.
int32_t run_calls(kv_pool *p, DirCall *calls, int ncalls, const bool *wait_other, bool may_fuse)
{
    p->union_slot[0] = p->union_slot[1] = -1;
    // The event each call has to wait for is the end of the other direction's latest EARLIER call.  It is
    // looked up here, before any direction of this call is begun: beginning the swap-out advances that
    // direction's call counter, and the swap-in of the same rotate must not mistake the swap-out it
    // travels with (whose end event is not recorded yet) for the earlier call it depends on.
    cudaEvent_t wait_ev[2] = {nullptr, nullptr};
    for (int k = 0; k < ncalls; ++k)
        if (wait_other[k]) {
            const DirState &o = p->dir[1 - calls[k].d];
            wait_ev[k] = o.ev_end[o.issued % KV_SLOTS];
        }
    // KV_PATH_AUTO is settled per call.  A call that moves very little (KV_AUTO_TINY_BYTES per direction; for
    // blocks under 2 MiB at most two blocks and 2 MiB) is all fixed cost and goes as one copy-engine transfer per block.  Otherwise the
    // staged transfers are planned first (cheap: a sort of the ids and one sweep over them) and the staged
    // path is taken when its transfers would carry KV_AUTO_MIN_TRANSFER bytes or more on average, the
    // zero-copy kernels when not.  Both directions of a rotate take the same path (a kernel on one direction
    // starves the copy engine on the other).
    {
        int64_t largest = 0;
        for (int k = 0; k < ncalls; ++k) {
            calls[k].path = p->dir[calls[k].d].path;
            if (calls[k].path == KV_PATH_AUTO) largest = std::max(largest, calls[k].n * p->blk);
        }
        const bool tiny = p->blk >= (2ll << 20)
                              ? largest <= KV_AUTO_TINY_BYTES
                              : largest <= KV_AUTO_TINY_BYTES_SMALL_BLOCKS && largest <= KV_AUTO_TINY_COUNT_SMALL_BLOCKS * p->blk;
        int chosen;
        if (tiny) {
            chosen = KV_PATH_CE2D;
        } else {
            int64_t bytes = 0, ops = 0;
            for (int k = 0; k < ncalls; ++k) {
                if (calls[k].path != KV_PATH_AUTO) continue;
                int32_t rc = plan_staged(p, calls[k]);
                if (rc != KV_OK) return rc;
                bytes += calls[k].n * p->blk;
                ops += (int64_t)p->dir[calls[k].d].ops.size();
            }
            chosen = (ops > 0 && bytes >= ops * KV_AUTO_MIN_TRANSFER) ? KV_PATH_STAGED : KV_PATH_ZEROCOPY;
        }
        for (int k = 0; k < ncalls; ++k)
            if (calls[k].path == KV_PATH_AUTO) calls[k].path = chosen;
    }
    // One launch for both directions of a zero-copy rotate: always when the pool asks for it
    // (KV_FLAG_FUSED_ROTATE), and by itself when both lists are short and nothing else is in flight on
    // the pool -- then the call is all fixed cost, and one launch on one stream is the least of it.
    bool fused = false;
    if (may_fuse && ncalls == 2 && calls[0].path == KV_PATH_ZEROCOPY && calls[1].path == KV_PATH_ZEROCOPY) {
        const bool small = calls[0].n <= KV_INLINE_PAIRS && calls[1].n <= KV_INLINE_PAIRS;
        const bool idle = p->dir[0].done >= p->dir[0].issued && p->dir[1].done >= p->dir[1].issued;
        fused = (p->cfg.flags & KV_FLAG_FUSED_ROTATE) || (small && idle);
    }
    // Both directions of a staged rotate use the same kind of transfers: two-block transfers one way and
    // long merged ones the other way fall out of step (74 GB/s measured against 88 to 95 when alike).
    if (ncalls == 2 && calls[0].path == KV_PATH_STAGED && calls[1].path == KV_PATH_STAGED &&
        p->cfg.host_layout == KV_HOST_BLOCK_FIRST) {
        for (int k = 0; k < 2; ++k)
            if (!calls[k].planned) {
                int32_t rc = plan_staged(p, calls[k]);
                if (rc != KV_OK) return rc;
            }
        if (calls[0].plan_uniform != calls[1].plan_uniform) {
            const bool joint = calls[0].n + calls[1].n < KV_MERGE_MIN_MEAN_RUN * (calls[0].plan_nruns + calls[1].plan_nruns);
            for (int k = 0; k < 2; ++k)
                if (calls[k].plan_uniform != joint) {
                    int32_t rc = plan_staged(p, calls[k], joint ? 1 : 0);
                    if (rc != KV_OK) return rc;
                }
        }
    }
    for (int k = 0; k < ncalls; ++k) {
        int32_t rc = prepare_dir(p, calls[k]);
        if (rc != KV_OK) return rc;
    }
    for (int k = 0; k < ncalls; ++k) {
        if (fused && calls[k].d == 1) {
            // the fused launch runs on the out stream: order it after earlier swap-ins, and later swap-ins after it
            DirState &in = p->dir[1];
            if (in.issued > in.done)
                KV_CUDA(p, cudaStreamWaitEvent(p->dir[0].stream, in.ev_end[in.issued % KV_SLOTS], 0));
        }
    }
    if (fused) {
        // both directions share the out stream for this call
        cudaStream_t keep = p->dir[1].stream;
        p->dir[1].stream = p->dir[0].stream;
        int32_t rc = KV_OK;
        for (int k = 0; k < ncalls && rc == KV_OK; ++k) rc = begin_dir(p, calls[k], wait_ev[k]);
        if (rc == KV_OK) rc = issue_calls(p, calls, ncalls, true);
        for (int k = 0; k < ncalls && rc == KV_OK; ++k) rc = end_dir(p, calls[k]);
        p->dir[1].stream = keep;
        if (rc != KV_OK) return rc;
        KV_CUDA(p, cudaStreamWaitEvent(keep, p->dir[1].ev_end[calls[1].slot], 0));
    } else {
        for (int k = 0; k < ncalls; ++k) {
            int32_t rc = begin_dir(p, calls[k], wait_ev[k]);
            if (rc != KV_OK) return rc;
        }
        int32_t rc = issue_calls(p, calls, ncalls, false);
        if (rc != KV_OK) return rc;
        for (int k = 0; k < ncalls; ++k) {
            rc = end_dir(p, calls[k]);
            if (rc != KV_OK) return rc;
        }
    }
    for (int k = 0; k < ncalls; ++k) p->union_slot[calls[k].d] = calls[k].slot;
    p->union_valid = true;
    return KV_OK;
}

// Turn the start / end events of the latest call into the last_* statistics.  Done when the statistics
// are read, not in kv_sync: four event queries are a measurable part of a small rotation's latency.
void harvest_call_timing(kv_pool *p)
{
    if (!p->union_valid || !p->union_synced) return;
    float t_out = 0.f, t_in = 0.f, off = 0.f;
    const int so = p->union_slot[0], si = p->union_slot[1];
    if (so >= 0) (void)cudaEventElapsedTime(&t_out, p->dir[0].ev_start[so], p->dir[0].ev_end[so]);
    if (si >= 0) (void)cudaEventElapsedTime(&t_in, p->dir[1].ev_start[si], p->dir[1].ev_end[si]);
    if (so >= 0) p->stats.last_out_ms = t_out;
    if (si >= 0) p->stats.last_in_ms = t_in;
    if (so >= 0 && si >= 0) {
        // position of the in-window relative to the out-window; either may start first
        float a = 0.f, b = 0.f;
        const bool fwd = cudaEventElapsedTime(&a, p->dir[0].ev_start[so], p->dir[1].ev_start[si]) == cudaSuccess;
        const bool bwd = cudaEventElapsedTime(&b, p->dir[1].ev_start[si], p->dir[0].ev_start[so]) == cudaSuccess;
        off = (fwd && a > 0.f) ? a : ((bwd && b > 0.f) ? -b : 0.f);
        const float lo = std::min(0.f, off), hi = std::max(t_out, off + t_in);
        p->stats.last_union_ms = hi - lo;
        p->stats.last_in_offset_ms = off;
    } else {
        p->stats.last_union_ms = so >= 0 ? t_out : t_in;
        p->stats.last_in_offset_ms = 0.0;
    }
    (void)cudaGetLastError();
    p->union_valid = p->union_synced = false;
}

// Host pool made by the library: an anonymous mapping, asked to be backed by transparent huge pages,
// touched by several threads and then page-locked with cudaHostRegister.  Page-locking 120 GB this way
// takes a fraction of what cudaHostAlloc takes for it (measured on 4 GiB: 0.6 s against 2.0 s, single
// thread; the copy engines' rates are the same either way).  Returns nullptr when the mapping cannot be
// made, when the system (or the process's memory control group) does not have that much memory available, or
// when CUDA refuses to register it; the caller then falls back to cudaHostAlloc.
int64_t mem_available_bytes()
{
    FILE *f = fopen("/proc/meminfo", "r");
    if (!f) return -1;
    char line[256];
    long long kb = -1;
    while (fgets(line, sizeof line, f))
        if (sscanf(line, "MemAvailable: %lld kB", &kb) == 1) break;
    fclose(f);
    return kb < 0 ? -1 : (int64_t)kb * 1024;
}

// bytes this process may still take under its memory control group (v2, else v1), or -1 when there is no limit
int64_t cgroup_headroom_bytes()
{
    auto read_ll = [](const char *path, long long &v) {
        FILE *f = fopen(path, "r");
        if (!f) return false;
        char buf[64] = "";
        const bool ok = fgets(buf, sizeof buf, f) != nullptr && sscanf(buf, "%lld", &v) == 1;   // "max" does not parse
        fclose(f);
        return ok;
    };
    long long limit = 0, used = 0;
    if (read_ll("/sys/fs/cgroup/memory.max", limit) && read_ll("/sys/fs/cgroup/memory.current", used))
        return std::max<long long>(0, limit - used);
    if (read_ll("/sys/fs/cgroup/memory/memory.limit_in_bytes", limit) &&
        read_ll("/sys/fs/cgroup/memory/memory.usage_in_bytes", used) && limit < (1ll << 60))
        return std::max<long long>(0, limit - used);
    return -1;
}

// Ask the kernel to take the pages of [base, base + bytes) from the memory node the GPU hangs off, where
// the box has more than one (the node is read from the GPU's PCI entry in sysfs): transfers to the other
// socket's memory cross the sockets' interconnect.  A preference, not a binding; every failure is ignored.
void prefer_memory_node_of_gpu(void *base, size_t bytes, int device_id)
{
    char bdf[32] = "";
    if (cudaDeviceGetPCIBusId(bdf, (int)sizeof bdf, device_id) != cudaSuccess) {
        (void)cudaGetLastError();
        return;
    }
    for (char *c = bdf; *c; ++c)
        if (*c >= 'A' && *c <= 'F') *c = (char)(*c - 'A' + 'a');
    char path[96];
    snprintf(path, sizeof path, "/sys/bus/pci/devices/%s/numa_node", bdf);
    FILE *f = fopen(path, "r");
    if (!f) return;
    int node = -1;
    const bool ok = fscanf(f, "%d", &node) == 1;
    fclose(f);
    if (!ok || node < 0 || node >= 1024) return;
    unsigned long mask[1024 / (8 * sizeof(unsigned long))] = {};
    mask[(size_t)node / (8 * sizeof(unsigned long))] |= 1ul << ((size_t)node % (8 * sizeof(unsigned long)));
#ifdef SYS_mbind
    (void)syscall(SYS_mbind, base, bytes, 1 /* MPOL_PREFERRED */, mask, 1024ul + 1, 0u);
#endif
}

uint8_t *map_host_pool(size_t bytes, int device_id, void *&map, size_t &map_len)
{
    const char *how = getenv("DUPLEXKV_HOST_ALLOC");
    if (how && strcmp(how, "cuda") == 0) return nullptr;
    // never touch more than the box, or this process's control group, can give: touching is what takes the memory
    const int64_t avail = mem_available_bytes(), room = cgroup_headroom_bytes();
    if (avail >= 0 && (double)bytes > 0.95 * (double)avail) return nullptr;
    if (room >= 0 && (double)bytes > 0.95 * (double)room) return nullptr;
    const size_t huge = (size_t)2 << 20;
    map_len = bytes + huge;
    map = mmap(nullptr, map_len, PROT_READ | PROT_WRITE, MAP_PRIVATE | MAP_ANONYMOUS, -1, 0);
    if (map == MAP_FAILED) {
        map = nullptr;
        return nullptr;
    }
    uint8_t *base = (uint8_t *)(((uintptr_t)map + huge - 1) & ~(uintptr_t)(huge - 1));
    (void)madvise(base, bytes, MADV_HUGEPAGE);            // a hint: ordinary pages do as well, only slower to lock
    (void)madvise(base, bytes, MADV_DONTFORK);            // a forked child must not share (and copy-on-write) pages the GPU writes
    prefer_memory_node_of_gpu(base, bytes, device_id);
    // first touch, one byte per 4 KiB page, slices of whole huge pages per thread
    unsigned threads = std::thread::hardware_concurrency();
    threads = std::max(1u, std::min(threads, 16u));
    if (bytes < ((size_t)256 << 20)) threads = 1;
    const size_t pages = (bytes + huge - 1) / huge;
    auto touch = [&](unsigned t) {
        const size_t lo = pages * t / threads * huge, hi = std::min(bytes, pages * (t + 1) / threads * huge);
        for (size_t o = lo; o < hi; o += 4096) ((volatile uint8_t *)base)[o] = 0;
    };
    try {
        std::vector<std::thread> pool;
        for (unsigned t = 1; t < threads; ++t) pool.emplace_back(touch, t);
        touch(0);
        for (auto &th : pool) th.join();
    } catch (...) {
        munmap(map, map_len);
        map = nullptr;
        return nullptr;
    }
    if (cudaHostRegister(base, bytes, cudaHostRegisterMapped | cudaHostRegisterPortable) != cudaSuccess) {
        (void)cudaGetLastError();
        munmap(map, map_len);
        map = nullptr;
        return nullptr;
    }
    return base;
}

}  // namespace

// =================================================================================================
// C ABI
extern "C" {

int64_t kv_seg_bytes(int32_t block_size, int32_t kv_heads, int32_t head_dim)
{
    if (block_size <= 0 || kv_heads <= 0 || head_dim <= 0) return 0;
    return (int64_t)block_size * kv_heads * head_dim * 2;
}

int64_t kv_blk_bytes(int32_t num_layers, int32_t block_size, int32_t kv_heads, int32_t head_dim)
{
    if (num_layers <= 0) return 0;
    return 2 * (int64_t)num_layers * kv_seg_bytes(block_size, kv_heads, head_dim);
}

int32_t kv_path_for(int64_t blk_bytes)
{
    // Measured on B200 behind PCIe Gen5 x16, both directions busy: a copy-engine transfer costs a fixed
    // start-up (about 10 us with the other direction busy) plus its bytes, so the staged path wins once its
    // transfers carry 2.5 MiB or more; below that the zero-copy kernels, which pay no per-transfer cost,
    // are ahead.  Blocks with no neighbours in host memory travel at least two per transfer, hence this rule
    // for the worst case; a pool on KV_PATH_AUTO applies the same threshold to the transfers each call
    // actually needs, so lists whose host ids form runs or four-block lattices go staged at any block size.
    return 2 * blk_bytes >= KV_AUTO_MIN_TRANSFER ? KV_PATH_STAGED : KV_PATH_ZEROCOPY;
}

const char *kv_last_error(kv_pool_t *pool) { return pool ? pool->err : g_err; }

int32_t kv_pool_create(const kv_pool_config_t *cfg, kv_pool_t **out)
{
    if (out) *out = nullptr;
    if (!cfg || !out) return fail(nullptr, KV_ERR_INVALID_ARG, "null argument");
    const int64_t seg = kv_seg_bytes(cfg->block_size, cfg->kv_heads, cfg->head_dim);
    const int64_t blk = kv_blk_bytes(cfg->num_layers, cfg->block_size, cfg->kv_heads, cfg->head_dim);
    if (seg <= 0 || blk <= 0 || cfg->num_gpu_blocks <= 0 || cfg->num_host_blocks <= 0)
        return fail(nullptr, KV_ERR_INVALID_ARG, "non-positive shape or pool size");
    if (cfg->num_gpu_blocks > INT32_MAX || cfg->num_host_blocks > INT32_MAX || seg > (1 << 30) ||
        2 * (int64_t)cfg->num_layers > (1 << 20))
        return fail(nullptr, KV_ERR_INVALID_ARG, "shape or pool size beyond 32-bit ids");
    if (seg % 16 != 0) return fail(nullptr, KV_ERR_UNSUPPORTED, "segment size must be a multiple of 16 bytes");
    if (!cfg->device_base || ((uintptr_t)cfg->device_base & 255))
        return fail(nullptr, KV_ERR_INVALID_ARG, "device_base must be a 256-byte aligned device pointer");
    if (cfg->host_base && ((uintptr_t)cfg->host_base & 4095))
        return fail(nullptr, KV_ERR_INVALID_ARG, "host_base must be 4096-byte aligned");
    if (cfg->host_layout != KV_HOST_BLOCK_FIRST && cfg->host_layout != KV_HOST_LAYER_FIRST)
        return fail(nullptr, KV_ERR_INVALID_ARG, "unknown host_layout");
    if (cfg->device_layout != KV_DEV_LAYER_FIRST && cfg->device_layout != KV_DEV_BLOCK_FIRST)
        return fail(nullptr, KV_ERR_INVALID_ARG, "unknown device_layout");
    if (cfg->path < KV_PATH_AUTO || cfg->path > KV_PATH_NAIVE || cfg->path_in < KV_PATH_AUTO || cfg->path_in > KV_PATH_NAIVE)
        return fail(nullptr, KV_ERR_INVALID_ARG, "unknown path");
    if (cfg->ctas_out < 0 || cfg->ctas_in < 0 || cfg->staging_bytes < 0 || cfg->ce_streams < 0 ||
        cfg->ce_streams > KV_MAX_CE_STREAMS || cfg->link_variant < 0 || cfg->link_variant > 2)
        return fail(nullptr, KV_ERR_INVALID_ARG, "tuning value out of range");

    // environment overrides of the path and of the zero-copy CTA counts (for trying settings on a program
    // that cannot be rebuilt); a value that does not parse is an error, not ignored
    kv_pool_config_t eff = *cfg;
    {
        static const char *names[] = {"auto", "zerocopy", "staged", "ce2d", "naive"};
        if (const char *v = getenv("DUPLEXKV_PATH")) {
            int found = -1;
            for (int k = 0; k < 5; ++k)
                if (!strcmp(v, names[k])) found = k;
            if (found < 0) return fail(nullptr, KV_ERR_INVALID_ARG, "DUPLEXKV_PATH must be auto, zerocopy, staged, ce2d or naive");
            eff.path = found;
            eff.path_in = KV_PATH_AUTO;        // "same as path"
        }
        const char *keys[2] = {"DUPLEXKV_SMS_OUT", "DUPLEXKV_SMS_IN"};
        int32_t *dst[2] = {&eff.ctas_out, &eff.ctas_in};
        for (int k = 0; k < 2; ++k)
            if (const char *v = getenv(keys[k])) {
                char *end = nullptr;
                const long x = strtol(v, &end, 10);
                if (end == v || *end || x < 0 || x > 65535) return fail(nullptr, KV_ERR_INVALID_ARG, "DUPLEXKV_SMS_OUT / DUPLEXKV_SMS_IN must be a CTA count");
                *dst[k] = (int32_t)x;
            }
    }
    cfg = &eff;
    KV_CUDA(nullptr, cudaSetDevice(cfg->device_id));
    kv_pool *p = new (std::nothrow) kv_pool();
    if (!p) return fail(nullptr, KV_ERR_NOMEM, "out of host memory");
    p->cfg = *cfg;
    p->seg = seg;
    p->blk = blk;
    p->planes = 2 * cfg->num_layers;
    p->cap = std::max(cfg->num_gpu_blocks, cfg->num_host_blocks);
    p->dev = (uint8_t *)cfg->device_base;
    p->err[0] = 0;
    memset(&p->stats, 0, sizeof(p->stats));
    // default staging: 2 GiB per direction, but no more than a sixteenth of the device pool -- or 128 MiB (the
    // whole pool's size if that is less) when the pool is small: halves of a few blocks would turn every
    // call into a chain of tiny chunks with an event hand-off between each
    if (p->cfg.staging_bytes == 0) {
        const int64_t pool_bytes = cfg->num_gpu_blocks * blk;
        p->cfg.staging_bytes = std::min<int64_t>(2ll << 30, std::max<int64_t>(pool_bytes / 16, std::min<int64_t>(pool_bytes, 128ll << 20)));
    }
    if (p->cfg.staging_bytes < 2 * blk) p->cfg.staging_bytes = 2 * blk;

#define KV_CREATE_CUDA(expr)                                   \
    do {                                                       \
        cudaError_t e_ = (expr);                               \
        if (e_ != cudaSuccess) {                               \
            int32_t rc_ = fail_cuda(nullptr, e_, #expr);       \
            kv_pool_destroy(p);                                \
            return rc_;                                        \
        }                                                      \
    } while (0)

    cudaDeviceProp prop;
    KV_CREATE_CUDA(cudaGetDeviceProperties(&prop, cfg->device_id));
    p->sm_count = prop.multiProcessorCount;
    p->max_pitch = (int64_t)std::min<size_t>(prop.memPitch, (size_t)INT32_MAX);

    const size_t host_bytes = (size_t)cfg->num_host_blocks * (size_t)blk;
    if (cfg->host_base) {
        p->host = (uint8_t *)cfg->host_base;
        // Memory that CUDA knows as page-locked already (allocated by cudaHostAlloc, registered by the caller,
        // or the host memory of another pool) is used as it is and left page-locked at destroy; the first
        // and the last byte are looked up.
        auto pinned = [](const void *q) {
            cudaPointerAttributes a;
            if (cudaPointerGetAttributes(&a, q) != cudaSuccess) {
                (void)cudaGetLastError();
                return false;
            }
            return a.type == cudaMemoryTypeHost;
        };
        if (!(pinned(p->host) && pinned(p->host + host_bytes - 1))) {
            cudaError_t e = cudaHostRegister(p->host, host_bytes, cudaHostRegisterMapped | cudaHostRegisterPortable);
            if (e != cudaSuccess) {
                (void)cudaGetLastError();
                int32_t rc = fail(nullptr, KV_ERR_NOMEM, "cudaHostRegister of host_base failed");
                kv_pool_destroy(p);
                return rc;
            }
            p->registered_host = true;
        }
    } else if ((p->host = map_host_pool(host_bytes, cfg->device_id, p->host_map, p->host_map_len)) != nullptr) {
        p->registered_host = true;      // unregistered and unmapped at destroy
    } else {
        cudaError_t e = cudaHostAlloc((void **)&p->host, host_bytes, cudaHostAllocMapped | cudaHostAllocPortable);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            p->host = nullptr;
            int32_t rc = fail(nullptr, KV_ERR_NOMEM, "pinned host pool allocation failed");
            kv_pool_destroy(p);
            return rc;
        }
        p->owns_host = true;
    }
    KV_CREATE_CUDA(cudaHostGetDevicePointer((void **)&p->host_dev, p->host, 0));
    KV_CREATE_CUDA(cudaHostAlloc((void **)&p->status_host, 64, cudaHostAllocMapped));
    *p->status_host = 0;
    KV_CREATE_CUDA(cudaHostGetDevicePointer((void **)&p->status_dev, p->status_host, 0));

    void *streams[2] = {cfg->stream_out, cfg->stream_in};
    const int want_ctas[2] = {cfg->ctas_out, cfg->ctas_in};
    for (int d = 0; d < 2; ++d) {
        DirState &s = p->dir[d];
        if (streams[d]) {
            s.stream = (cudaStream_t)streams[d];
        } else {
            KV_CREATE_CUDA(cudaStreamCreateWithFlags(&s.stream, cudaStreamNonBlocking));
            s.owns_stream = true;
        }
        const size_t ring_bytes = (size_t)KV_SLOTS * 2 * (size_t)p->cap * sizeof(int2);
        KV_CREATE_CUDA(cudaHostAlloc((void **)&s.ring_host, ring_bytes, cudaHostAllocDefault));
        KV_CREATE_CUDA(cudaMalloc((void **)&s.ring_dev, ring_bytes));
        for (int k = 0; k < KV_SLOTS; ++k) {
            KV_CREATE_CUDA(cudaEventCreate(&s.ev_start[k]));
            KV_CREATE_CUDA(cudaEventCreate(&s.ev_end[k]));
        }
        s.ctas = want_ctas[d] > 0 ? want_ctas[d] : 64;
        s.half_blocks = std::max<int64_t>(1, p->cfg.staging_bytes / 2 / blk);
        s.path = (d == 1 && cfg->path_in != KV_PATH_AUTO) ? cfg->path_in : cfg->path;
        s.nsub = cfg->ce_streams > 0 ? cfg->ce_streams : 1;
        s.sub[0] = s.stream;
        KV_CREATE_CUDA(cudaEventCreateWithFlags(&s.fork_ev, cudaEventDisableTiming));
        KV_CREATE_CUDA(cudaStreamCreateWithFlags(&s.kstream, cudaStreamNonBlocking));
        KV_CREATE_CUDA(cudaEventCreateWithFlags(&s.kfork_ev, cudaEventDisableTiming));
        for (int k = 0; k < 2; ++k) {
            KV_CREATE_CUDA(cudaEventCreateWithFlags(&s.ev_a[k], cudaEventDisableTiming));
            KV_CREATE_CUDA(cudaEventCreateWithFlags(&s.ev_b[k], cudaEventDisableTiming));
        }
        for (int k = 1; k < s.nsub; ++k) {
            KV_CREATE_CUDA(cudaStreamCreateWithFlags(&s.sub[k], cudaStreamNonBlocking));
            KV_CREATE_CUDA(cudaEventCreateWithFlags(&s.join_ev[k], cudaEventDisableTiming));
        }
    }
    KV_CREATE_CUDA(prepare_bulk_kernels());
#undef KV_CREATE_CUDA

    try {
        p->g_mark.assign((size_t)cfg->num_gpu_blocks, 0);
        p->h_mark.assign((size_t)cfg->num_host_blocks, 0);
        p->g_mark2.assign((size_t)cfg->num_gpu_blocks, 0);
        p->h_mark2.assign((size_t)cfg->num_host_blocks, 0);
        p->g_read_by_out.assign((size_t)cfg->num_gpu_blocks, 0);
        p->g_written_by_in.assign((size_t)cfg->num_gpu_blocks, 0);
        p->h_written_by_out.assign((size_t)cfg->num_host_blocks, 0);
        p->h_read_by_in.assign((size_t)cfg->num_host_blocks, 0);
    } catch (...) {
        kv_pool_destroy(p);
        return fail(nullptr, KV_ERR_NOMEM, "out of host memory");
    }
    *out = p;
    return KV_OK;
}

int32_t kv_pool_destroy(kv_pool_t *p)
{
    if (!p) return KV_ERR_INVALID_ARG;
    for (int d = 0; d < 2; ++d)
        if (p->dir[d].stream) (void)cudaStreamSynchronize(p->dir[d].stream);
    for (int d = 0; d < 2; ++d) {
        DirState &s = p->dir[d];
        for (int k = 0; k < KV_SLOTS; ++k) {
            if (s.ev_start[k]) (void)cudaEventDestroy(s.ev_start[k]);
            if (s.ev_end[k]) (void)cudaEventDestroy(s.ev_end[k]);
        }
        for (int k = 1; k < KV_MAX_CE_STREAMS; ++k) {
            if (s.sub[k]) (void)cudaStreamSynchronize(s.sub[k]);
            if (s.sub[k]) (void)cudaStreamDestroy(s.sub[k]);
            if (s.join_ev[k]) (void)cudaEventDestroy(s.join_ev[k]);
        }
        if (s.fork_ev) (void)cudaEventDestroy(s.fork_ev);
        if (s.kstream) {
            (void)cudaStreamSynchronize(s.kstream);
            (void)cudaStreamDestroy(s.kstream);
        }
        if (s.kfork_ev) (void)cudaEventDestroy(s.kfork_ev);
        for (cudaEvent_t e : s.kev) (void)cudaEventDestroy(e);
        if (s.ktime_dev) (void)cudaFree(s.ktime_dev);
        for (int k = 0; k < 2; ++k) {
            if (s.ev_a[k]) (void)cudaEventDestroy(s.ev_a[k]);
            if (s.ev_b[k]) (void)cudaEventDestroy(s.ev_b[k]);
        }
        if (s.ring_host) (void)cudaFreeHost(s.ring_host);
        if (s.ring_dev) (void)cudaFree(s.ring_dev);
        if (s.stage) (void)cudaFree(s.stage);
        if (s.owns_stream && s.stream) (void)cudaStreamDestroy(s.stream);
    }
    if (p->status_host) (void)cudaFreeHost(p->status_host);
    if (p->owns_host && p->host) (void)cudaFreeHost(p->host);
    if (p->registered_host) (void)cudaHostUnregister(p->host);
    if (p->host_map) (void)munmap(p->host_map, p->host_map_len);
    (void)cudaGetLastError();
    delete p;
    return KV_OK;
}

int32_t kv_swap_out(kv_pool_t *p, const int32_t *gpu_ids, const int32_t *host_ids, int64_t n)
{
    if (!p) return KV_ERR_INVALID_ARG;
    int32_t rc = check_direction(p, gpu_ids, host_ids, n, true);
    if (rc != KV_OK || n == 0) return rc;
    poll_done(p);
    DirCall c{};
    c.d = 0;
    c.gpu_ids = gpu_ids;
    c.host_ids = host_ids;
    c.n = n;
    const bool wait = conflicts_with_other(p, 0, gpu_ids, host_ids, n);
    return run_calls(p, &c, 1, &wait, false);
}

int32_t kv_swap_in(kv_pool_t *p, const int32_t *host_ids, const int32_t *gpu_ids, int64_t n)
{
    if (!p) return KV_ERR_INVALID_ARG;
    int32_t rc = check_direction(p, gpu_ids, host_ids, n, false);
    if (rc != KV_OK || n == 0) return rc;
    poll_done(p);
    DirCall c{};
    c.d = 1;
    c.gpu_ids = gpu_ids;
    c.host_ids = host_ids;
    c.n = n;
    const bool wait = conflicts_with_other(p, 1, gpu_ids, host_ids, n);
    return run_calls(p, &c, 1, &wait, false);
}

int32_t kv_rotate(kv_pool_t *p, const int32_t *out_gpu, const int32_t *out_host, int64_t n_out,
                  const int32_t *in_host, const int32_t *in_gpu, int64_t n_in)
{
    if (!p) return KV_ERR_INVALID_ARG;
    int32_t rc = check_direction(p, out_gpu, out_host, n_out, true);
    if (rc != KV_OK) return rc;
    rc = check_direction(p, in_gpu, in_host, n_in, false);
    if (rc != KV_OK) return rc;
    if (n_out == 0 && n_in == 0) return KV_OK;
    if (n_out == 0) return kv_swap_in(p, in_host, in_gpu, n_in);
    if (n_in == 0) return kv_swap_out(p, out_gpu, out_host, n_out);

    // cross-direction overlap inside this call: mark the swap-out's blocks, then look the swap-in's up
    const uint32_t e = ++p->epoch;
    for (int64_t i = 0; i < n_out; ++i) {
        p->g_mark2[out_gpu[i]] = e;
        p->h_mark2[out_host[i]] = e;
    }
    int64_t n_conf = 0;
    for (int64_t j = 0; j < n_in; ++j)
        if (p->g_mark2[in_gpu[j]] == e || p->h_mark2[in_host[j]] == e) ++n_conf;
    if (n_conf > 0 && !(p->cfg.flags & KV_FLAG_ALLOW_OVERLAP))
        return fail(p, KV_ERR_HAZARD, "swap-in and swap-out lists name the same block (data race); nothing moved");

    poll_done(p);
    if (n_conf == 0) {
        DirCall calls[2] = {};
        calls[0].d = 0;
        calls[0].gpu_ids = out_gpu;
        calls[0].host_ids = out_host;
        calls[0].n = n_out;
        calls[1].d = 1;
        calls[1].gpu_ids = in_gpu;
        calls[1].host_ids = in_host;
        calls[1].n = n_in;
        const bool wait[2] = {conflicts_with_other(p, 0, out_gpu, out_host, n_out),
                              conflicts_with_other(p, 1, in_gpu, in_host, n_in)};
        return run_calls(p, calls, 2, wait, !wait[0] && !wait[1]);
    }
    // overlap allowed: the conflict-free swap-ins run beside the swap-out, the others after it
    std::vector<int32_t> free_h, free_g, conf_h, conf_g;
    try {
        free_h.reserve((size_t)(n_in - n_conf));
        free_g.reserve((size_t)(n_in - n_conf));
        conf_h.reserve((size_t)n_conf);
        conf_g.reserve((size_t)n_conf);
    } catch (...) {
        return fail(p, KV_ERR_NOMEM, "out of host memory");
    }
    for (int64_t j = 0; j < n_in; ++j) {
        const bool cf = p->g_mark2[in_gpu[j]] == e || p->h_mark2[in_host[j]] == e;
        (cf ? conf_h : free_h).push_back(in_host[j]);
        (cf ? conf_g : free_g).push_back(in_gpu[j]);
    }
    {
        DirCall calls[2] = {};
        calls[0].d = 0;
        calls[0].gpu_ids = out_gpu;
        calls[0].host_ids = out_host;
        calls[0].n = n_out;
        calls[1].d = 1;
        calls[1].gpu_ids = free_g.data();
        calls[1].host_ids = free_h.data();
        calls[1].n = (int64_t)free_g.size();
        const bool wait[2] = {conflicts_with_other(p, 0, out_gpu, out_host, n_out),
                              calls[1].n ? conflicts_with_other(p, 1, calls[1].gpu_ids, calls[1].host_ids, calls[1].n) : false};
        rc = run_calls(p, calls, calls[1].n ? 2 : 1, wait, false);
        if (rc != KV_OK) return rc;
    }
    const int out_slot = p->union_slot[0];
    DirCall late{};
    late.d = 1;
    late.gpu_ids = conf_g.data();
    late.host_ids = conf_h.data();
    late.n = n_conf;
    const bool wait_late = true;   // after this call's swap-out
    rc = run_calls(p, &late, 1, &wait_late, false);
    p->union_slot[0] = out_slot;
    return rc;
}

int32_t kv_plan_staged(int64_t blk_bytes, int64_t half_blocks, int32_t direction, const int32_t *host_ids, int64_t n,
                       kv_plan_op_t *ops, int64_t ops_cap, int64_t *n_ops, int32_t *order)
{
    if (n_ops) *n_ops = 0;
    if (blk_bytes <= 0 || half_blocks <= 0 || (direction != 0 && direction != 1) || n < 0 || (n && !host_ids) || !n_ops ||
        (ops_cap && !ops))
        return fail(nullptr, KV_ERR_INVALID_ARG, "bad planning arguments");
    for (int64_t i = 0; i < n; ++i)
        if (host_ids[i] < 0) return fail(nullptr, KV_ERR_RANGE, "negative host id");
    std::vector<int32_t> ord;
    std::vector<CeOp> v;
    std::vector<CeChunk> ch;
    const PlanParams pp{blk_bytes, blk_bytes, half_blocks, (int64_t)INT32_MAX, 0, 1, false};
    try {
        if (n) plan_transfers(pp, direction, host_ids, n, ord, v, ch);
    } catch (...) {
        return fail(nullptr, KV_ERR_NOMEM, "out of host memory");
    }
    *n_ops = (int64_t)v.size();
    if ((int64_t)v.size() > ops_cap) return ops_cap ? fail(nullptr, KV_ERR_INVALID_ARG, "ops array too short") : KV_OK;
    for (size_t q = 0; q < ch.size(); ++q)
        for (int32_t a = ch[q].op_lo; a < ch[q].op_hi; ++a) {
            const CeOp &o = v[(size_t)a];
            kv_plan_op_t &r = ops[a];
            r.host_block = o.host_off / blk_bytes;
            r.first_position = o.pos;
            r.rows = o.rows;
            r.blocks_per_row = (int32_t)(o.width / blk_bytes);
            r.pitch_blocks = o.rows > 1 ? o.host_pitch / blk_bytes : r.blocks_per_row;
            r.chunk = (int32_t)q;
            r.slices = o.slices;
            r.slice_pitch_blocks = o.slices > 1 ? o.slice_rows * (o.host_pitch / blk_bytes) : 0;
        }
    if (order)
        for (int64_t i = 0; i < n; ++i) order[i] = ord[(size_t)i];
    return KV_OK;
}

int32_t kv_pool_set_path(kv_pool_t *p, int32_t path_out, int32_t path_in)
{
    if (!p) return KV_ERR_INVALID_ARG;
    if (path_out < KV_PATH_AUTO || path_out > KV_PATH_NAIVE || path_in < KV_PATH_AUTO || path_in > KV_PATH_NAIVE)
        return fail(p, KV_ERR_INVALID_ARG, "unknown path");
    int32_t rc = kv_sync(p);
    if (rc != KV_OK) return rc;
    p->dir[0].path = path_out;
    p->dir[1].path = path_in;
    return KV_OK;
}

int32_t kv_pool_set_call_timing(kv_pool_t *p, int32_t on)
{
    if (!p) return KV_ERR_INVALID_ARG;
    int32_t rc = kv_sync(p);
    if (rc != KV_OK) return rc;
    p->call_timing = on != 0;
    p->union_valid = p->union_synced = false;
    return KV_OK;
}

int32_t kv_pool_set_wait_limit(kv_pool_t *p, uint32_t polls, uint64_t ns)
{
    if (!p) return KV_ERR_INVALID_ARG;
    if (ns > 60ull * 1000000000ull) return fail(p, KV_ERR_INVALID_ARG, "wait limit beyond 60 s");
    p->wait_polls = polls;
    p->wait_ns = ns;
    return KV_OK;
}

int32_t kv_sync(kv_pool_t *p)
{
    if (!p) return KV_ERR_INVALID_ARG;
    for (int d = 0; d < 2; ++d) {
        cudaError_t e = cudaStreamSynchronize(p->dir[d].stream);
        if (e != cudaSuccess) return fail_cuda(p, e, "cudaStreamSynchronize");
        p->dir[d].done = p->dir[d].issued;
    }
    if (p->union_valid) p->union_synced = true;     // kv_get_stats turns the events into the last_* fields
    for (int d = 0; d < 2; ++d) {
        DirState &s = p->dir[d];
        if (s.kev_used > 0 && s.ktime_dev) {
            std::vector<unsigned long long> t((size_t)2 * s.kev_used);
            if (cudaMemcpy(t.data(), s.ktime_dev, t.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost) == cudaSuccess) {
                for (int k = 0; k < s.kev_used; ++k)
                    if (t[2 * (size_t)k + 1] > t[2 * (size_t)k]) p->stats.timed_kernel_exec_ms += (double)(t[2 * (size_t)k + 1] - t[2 * (size_t)k]) * 1e-6;
                (void)preset_ktime(s, s.kstream);
                (void)cudaStreamSynchronize(s.kstream);
            }
        }
        for (int k = 0; k < s.kev_used; ++k) {
            float ms = 0.f;
            if (cudaEventElapsedTime(&ms, s.kev[2 * (size_t)k], s.kev[2 * (size_t)k + 1]) == cudaSuccess) {
                p->stats.timed_kernel_ms += ms;
                p->stats.timed_kernel_bytes += s.kev_bytes[(size_t)k];
                p->stats.timed_kernels++;
            }
        }
        s.kev_used = 0;
    }
    (void)cudaGetLastError();
    const unsigned int st = *(volatile unsigned int *)p->status_host;
    p->stats.device_status = st;
    if (st & KV_DEV_TIMEOUT) {
        if (p->sticky == KV_OK) p->sticky = KV_ERR_TIMEOUT;
        snprintf(p->err, 256, "a device-side wait ran out (status 0x%x)", st);
    } else if (st & KV_DEV_BAD_ID) {
        if (p->sticky == KV_OK) p->sticky = KV_ERR_RANGE;
        snprintf(p->err, 256, "a kernel met a block id outside its pool and skipped it (status 0x%x)", st);
    }
    return p->sticky;
}

static int32_t device_leg(kv_pool_t *p, const int32_t *gpu_ids, int64_t n, const void *buf, int d)
{
    if (!p) return KV_ERR_INVALID_ARG;
    if (n < 0) return fail(p, KV_ERR_INVALID_ARG, "negative count");
    if (n == 0) return KV_OK;
    if (!gpu_ids || !buf) return fail(p, KV_ERR_INVALID_ARG, "null argument");
    if (n > p->cap) return fail(p, KV_ERR_INVALID_ARG, "more blocks than the pools have");
    if ((uintptr_t)buf & 15) return fail(p, KV_ERR_INVALID_ARG, "buffer must be 16-byte aligned");
    int32_t rc = check_ids(p, gpu_ids, n, p->cfg.num_gpu_blocks, "gpu_ids");
    if (rc != KV_OK) return rc;
    if (d == 1) {
        rc = check_unique(p, gpu_ids, n, p->g_mark, "scatter");
        if (rc != KV_OK) return rc;
    }
    DirState &s = p->dir[d];
    // Ordered like a swap call of its direction: a gather reads device blocks (as a swap-out does), a
    // scatter writes them (as a swap-in does), so it waits for an unfinished call of the other direction
    // that writes / reads one of its blocks, and later calls of the other direction wait for it.
    poll_done(p);
    cudaEvent_t wait_for = nullptr;
    if (conflicts_with_other(p, d, gpu_ids, nullptr, n)) {
        const DirState &o = p->dir[1 - d];
        wait_for = o.ev_end[o.issued % KV_SLOTS];
    }
    const uint64_t seq = s.issued + 1;
    const int slot = (int)(seq % KV_SLOTS);
    if (seq > KV_SLOTS && s.done + KV_SLOTS < seq) KV_CUDA(p, cudaEventSynchronize(s.ev_end[slot]));
    int2 *ph = s.ring_host + (size_t)slot * 2 * p->cap;
    int2 *pd = s.ring_dev + (size_t)slot * 2 * p->cap;
    for (int64_t i = 0; i < n; ++i) ph[i] = (d == 0) ? make_int2(gpu_ids[i], (int)i) : make_int2((int)i, gpu_ids[i]);
    if (wait_for) KV_CUDA(p, cudaStreamWaitEvent(s.stream, wait_for, 0));
    KV_CUDA(p, cudaEventRecord(s.ev_start[slot], s.stream));
    KV_CUDA(p, cudaMemcpyAsync(pd, ph, (size_t)n * sizeof(int2), cudaMemcpyHostToDevice, s.stream));
    KvJob job;
    fill_geometry(p, job);
    job.dir[1] = KvDir{};
    KvDir &kd = job.dir[0];
    kd.src = (d == 0) ? device_side(p) : packed_side(p, buf);
    kd.dst = (d == 0) ? packed_side(p, buf) : device_side(p);
    kd.pairs = pd;
    kd.n = (int)n;
    kd.src_blocks = (int)(d == 0 ? p->cfg.num_gpu_blocks : n);
    kd.dst_blocks = (int)(d == 0 ? n : p->cfg.num_gpu_blocks);
    const int want = (d == 0 ? p->cfg.ctas_out : p->cfg.ctas_in);
    kd.ctas = clamp_ctas(job, kd, want > 0 ? want : p->sm_count);
    KV_CUDA(p, launch_timed(p, s, s.stream, job, n * p->blk));
    KV_CUDA(p, cudaEventRecord(s.ev_end[slot], s.stream));
    s.issued = seq;
    note_use(p, d, gpu_ids, nullptr, n, seq);
    p->union_slot[d] = slot;
    p->union_slot[1 - d] = -1;
    p->union_valid = true;
    p->union_synced = false;
    return KV_OK;
}

int32_t kv_gather_blocks(kv_pool_t *p, const int32_t *gpu_ids, int64_t n, void *dst_device)
{
    return device_leg(p, gpu_ids, n, dst_device, 0);
}

int32_t kv_scatter_blocks(kv_pool_t *p, const void *src_device, const int32_t *gpu_ids, int64_t n)
{
    return device_leg(p, gpu_ids, n, src_device, 1);
}

int32_t kv_stream_wait(kv_pool_t *p, void *stream, int32_t directions)
{
    if (!p || (directions & ~3) || directions == 0) return KV_ERR_INVALID_ARG;
    for (int d = 0; d < 2; ++d) {
        DirState &s = p->dir[d];
        if (!(directions & (1 << d)) || s.issued == 0) continue;
        KV_CUDA(p, cudaStreamWaitEvent((cudaStream_t)stream, s.ev_end[s.issued % KV_SLOTS], 0));
    }
    return KV_OK;
}

int32_t kv_completion_event(kv_pool_t *p, int32_t direction, void **event)
{
    if (!p || !event || (direction != 0 && direction != 1)) return KV_ERR_INVALID_ARG;
    const DirState &s = p->dir[direction];
    *event = s.issued ? (void *)s.ev_end[s.issued % KV_SLOTS] : nullptr;
    return KV_OK;
}

int32_t kv_pool_set_ctas(kv_pool_t *p, int32_t ctas_out, int32_t ctas_in)
{
    if (!p) return KV_ERR_INVALID_ARG;
    if (ctas_out < 0 || ctas_in < 0) return fail(p, KV_ERR_INVALID_ARG, "negative CTA count");
    int32_t rc = kv_sync(p);
    if (rc != KV_OK) return rc;
    p->cfg.ctas_out = ctas_out;
    p->cfg.ctas_in = ctas_in;
    p->dir[0].ctas = ctas_out > 0 ? ctas_out : 64;
    p->dir[1].ctas = ctas_in > 0 ? ctas_in : 64;
    return KV_OK;
}

int32_t kv_debug_ring_shape(int64_t segment_bytes, int32_t over_link, int32_t link_variant, int32_t *item_bytes,
                            int32_t *stage_bytes, int32_t *stages, int32_t *ahead, int32_t *warps)
{
    if (segment_bytes <= 0 || segment_bytes % 16 != 0 || link_variant < 0 || link_variant > 2)
        return fail(nullptr, KV_ERR_INVALID_ARG, "segment_bytes must be a positive multiple of 16, link_variant 0..2");
    // as fill_geometry and launch_bulk decide it
    const int max_chunk = over_link ? (link_variant == 1 ? LINK1_STAGE : (link_variant == 2 ? LINK2_STAGE : LINK_STAGE)) : BULK_STAGE;
    const int chunk = (int)std::min<int64_t>(segment_bytes, max_chunk);
    const BulkShape &b = bulk_shape_for(chunk, over_link != 0, link_variant);
    if (item_bytes) *item_bytes = chunk;
    if (stage_bytes) *stage_bytes = b.stage;
    if (stages) *stages = b.stages;
    if (ahead) *ahead = b.ahead;
    if (warps) *warps = b.warps;
    return KV_OK;
}

int32_t kv_debug_pair_in_bounds(int32_t src_id, int32_t dst_id, int32_t src_blocks, int32_t dst_blocks)
{
    return kv_pair_in_bounds(src_id, dst_id, src_blocks, dst_blocks) ? 1 : 0;
}

static int32_t check_offsets(kv_pool_t *p, const int64_t *off, int64_t n_req, int64_t n, const char *what)
{
    if (n_req < 0 || (n_req > 0 && !off)) return fail(p, KV_ERR_INVALID_ARG, "bad request offsets");
    if (n_req == 0) return n == 0 ? KV_OK : fail(p, KV_ERR_INVALID_ARG, "blocks listed but no request offsets");
    if (off[0] != 0 || off[n_req] != n) {
        snprintf(p->err, 256, "%s request offsets must start at 0 and end at the list length", what);
        return KV_ERR_INVALID_ARG;
    }
    for (int64_t k = 0; k < n_req; ++k)
        if (off[k + 1] < off[k]) {
            snprintf(p->err, 256, "%s request offsets must not decrease", what);
            return KV_ERR_INVALID_ARG;
        }
    return KV_OK;
}

int32_t kv_rotate_req(kv_pool_t *p, const int32_t *out_gpu, const int32_t *out_host, int64_t n_out,
                      const int64_t *out_req_offsets, int64_t n_out_req,
                      const int32_t *in_host, const int32_t *in_gpu, int64_t n_in,
                      const int64_t *in_req_offsets, int64_t n_in_req)
{
    if (!p) return KV_ERR_INVALID_ARG;
    if (n_out < 0 || n_in < 0) return fail(p, KV_ERR_INVALID_ARG, "negative count");
    int32_t rc = check_offsets(p, out_req_offsets, n_out_req, n_out, "swap-out");
    if (rc != KV_OK) return rc;
    rc = check_offsets(p, in_req_offsets, n_in_req, n_in, "swap-in");
    if (rc != KV_OK) return rc;
    rc = kv_rotate(p, out_gpu, out_host, n_out, in_host, in_gpu, n_in);
    if (rc != KV_OK) return rc;
    p->stats.requests_out += n_out_req;
    p->stats.requests_in += n_in_req;
    return KV_OK;
}

int32_t kv_pool_progress(kv_pool_t *p, int64_t *out_issued, int64_t *out_done, int64_t *in_issued, int64_t *in_done)
{
    if (!p) return KV_ERR_INVALID_ARG;
    poll_done(p);
    if (out_issued) *out_issued = (int64_t)p->dir[0].issued;
    if (out_done) *out_done = (int64_t)p->dir[0].done;
    if (in_issued) *in_issued = (int64_t)p->dir[1].issued;
    if (in_done) *in_done = (int64_t)p->dir[1].done;
    return KV_OK;
}

int32_t kv_pool_shape(kv_pool_t *p, kv_pool_shape_t *out)
{
    if (!p || !out) return KV_ERR_INVALID_ARG;
    out->num_layers = p->cfg.num_layers;
    out->block_size = p->cfg.block_size;
    out->kv_heads = p->cfg.kv_heads;
    out->head_dim = p->cfg.head_dim;
    out->num_gpu_blocks = p->cfg.num_gpu_blocks;
    out->num_host_blocks = p->cfg.num_host_blocks;
    out->seg_bytes = p->seg;
    out->blk_bytes = p->blk;
    return KV_OK;
}

int32_t kv_host_ptr(kv_pool_t *p, void **base, int64_t *bytes)
{
    if (!p || !base || !bytes) return KV_ERR_INVALID_ARG;
    *base = p->host;
    *bytes = p->cfg.num_host_blocks * p->blk;
    return KV_OK;
}

int32_t kv_get_stats(kv_pool_t *p, kv_stats_t *st)
{
    if (!p || !st) return KV_ERR_INVALID_ARG;
    harvest_call_timing(p);
    p->stats.device_status = *(volatile unsigned int *)p->status_host;
    *st = p->stats;
    return KV_OK;
}

int32_t kv_probe_link_ex(int32_t device_id, const kv_probe_spec_t *spec, kv_link_probe_t *out)
{
    if (!out || !spec || spec->copy_bytes <= 0 || spec->total_bytes < spec->copy_bytes || spec->rounds <= 0 || spec->rows < 0)
        return fail(nullptr, KV_ERR_INVALID_ARG, "bad probe arguments");
    const int64_t rows = spec->rows > 1 ? spec->rows : 1;
    const int64_t slices = spec->slices > 1 ? spec->slices : 1;
    if (spec->copy_bytes % (rows * slices)) return fail(nullptr, KV_ERR_INVALID_ARG, "copy_bytes must be a multiple of rows x slices");
    const size_t width = (size_t)(spec->copy_bytes / (rows * slices));
    const size_t hpitch = spec->host_pitch > 0 ? (size_t)spec->host_pitch : width;
    const size_t dpitch = spec->dev_pitch > 0 ? (size_t)spec->dev_pitch : width;
    if (hpitch < width || dpitch < width) return fail(nullptr, KV_ERR_INVALID_ARG, "pitch smaller than a row");
    // 3-D transfers: slices of `rows` rows; on the host a slice starts host_slice_rows row pitches after the
    // one before (at least `rows`), on the device the slices are packed
    const size_t hslice_rows = slices > 1 ? (size_t)std::max<int64_t>(spec->host_slice_rows, rows) : (size_t)rows;
    // bytes from the first byte of a transfer to its last, on each side
    const size_t foot_h = ((size_t)(slices - 1) * hslice_rows + (size_t)(rows - 1)) * hpitch + width;
    const size_t foot_d = ((size_t)(slices * rows) - 1) * dpitch + width;
    if ((size_t)spec->span_bytes < foot_h || (size_t)spec->span_bytes < foot_d)
        return fail(nullptr, KV_ERR_INVALID_ARG, "span_bytes smaller than one transfer's footprint");
    memset(out, 0, sizeof(*out));
    KV_CUDA(nullptr, cudaSetDevice(device_id));
    const size_t span = (size_t)spec->span_bytes;
    const size_t slots_h = (span - foot_h) / width + 1, slots_d = (span - foot_d) / width + 1;
    const int64_t n = spec->total_bytes / spec->copy_bytes;
    // where each transfer starts: consecutive (wrapping) or seeded pseudo-random row-aligned offsets
    std::vector<size_t> off_h[2], off_d[2];
    try {
        for (int k = 0; k < 2; ++k) {
            off_h[k].resize((size_t)n);
            off_d[k].resize((size_t)n);
        }
    } catch (...) {
        return fail(nullptr, KV_ERR_NOMEM, "out of host memory");
    }
    uint64_t lcg = 0x9E3779B97F4A7C15ull;
    for (int k = 0; k < 2; ++k)
        for (int64_t i = 0; i < n; ++i) {
            lcg = lcg * 6364136223846793005ull + 1442695040888963407ull;
            const size_t r1 = (size_t)(lcg >> 33);
            lcg = lcg * 6364136223846793005ull + 1442695040888963407ull;
            const size_t r2 = (size_t)(lcg >> 33);
            // consecutive transfers tile the span when they are plain (one row, or rows packed back to back)
            const size_t step_h = (hpitch == width && slices == 1) ? (size_t)rows : 1;
            const size_t step_d = (dpitch == width) ? (size_t)(rows * slices) : 1;
            off_h[k][(size_t)i] = (spec->scattered ? r1 % slots_h : ((size_t)i * step_h) % slots_h) * width;
            off_d[k][(size_t)i] = (spec->scattered ? r2 % slots_d : ((size_t)i * step_d) % slots_d) * width;
        }
    uint8_t *h[2] = {nullptr, nullptr}, *dv[2] = {nullptr, nullptr};
    cudaStream_t st[2] = {nullptr, nullptr};
    cudaEvent_t ev[4] = {};
    int32_t rc = KV_OK;
    auto cleanup = [&]() {
        for (int k = 0; k < 2; ++k) {
            if (h[k]) (void)cudaFreeHost(h[k]);
            if (dv[k]) (void)cudaFree(dv[k]);
            if (st[k]) (void)cudaStreamDestroy(st[k]);
        }
        for (int k = 0; k < 4; ++k)
            if (ev[k]) (void)cudaEventDestroy(ev[k]);
    };
#define KV_PROBE(expr)                                  \
    do {                                                \
        cudaError_t e_ = (expr);                        \
        if (e_ != cudaSuccess) {                        \
            rc = fail_cuda(nullptr, e_, #expr);         \
            cleanup();                                  \
            return rc;                                  \
        }                                               \
    } while (0)
    for (int k = 0; k < 2; ++k) {
        KV_PROBE(cudaHostAlloc((void **)&h[k], span, cudaHostAllocDefault));
        memset(h[k], k + 1, span);
        KV_PROBE(cudaMalloc((void **)&dv[k], span));
        KV_PROBE(cudaMemset(dv[k], 0, span));
        KV_PROBE(cudaStreamCreateWithFlags(&st[k], cudaStreamNonBlocking));
    }
    for (int k = 0; k < 4; ++k) KV_PROBE(cudaEventCreate(&ev[k]));
    auto copy3d = [&](uint8_t *hp, uint8_t *dp, bool to_host, cudaStream_t stream) {
        cudaMemcpy3DParms p3 = {};
        const cudaPitchedPtr hpp = make_cudaPitchedPtr(hp, hpitch, width, hslice_rows);     // slice pitch = pitch x rows per slice
        const cudaPitchedPtr dpp = make_cudaPitchedPtr(dp, dpitch, width, (size_t)rows);
        p3.srcPtr = to_host ? dpp : hpp;
        p3.dstPtr = to_host ? hpp : dpp;
        p3.extent = make_cudaExtent(width, (size_t)rows, (size_t)slices);
        p3.kind = to_host ? cudaMemcpyDeviceToHost : cudaMemcpyHostToDevice;
        return cudaMemcpy3DAsync(&p3, stream);
    };
    auto d2h = [&](int64_t i) {
        uint8_t *hp = h[0] + off_h[0][(size_t)i], *dp = dv[0] + off_d[0][(size_t)i];
        if (slices > 1) return copy3d(hp, dp, true, st[0]);
        return rows == 1 ? cudaMemcpyAsync(hp, dp, width, cudaMemcpyDeviceToHost, st[0])
                         : cudaMemcpy2DAsync(hp, hpitch, dp, dpitch, width, (size_t)rows, cudaMemcpyDeviceToHost, st[0]);
    };
    auto h2d = [&](int64_t i) {
        uint8_t *hp = h[1] + off_h[1][(size_t)i], *dp = dv[1] + off_d[1][(size_t)i];
        if (slices > 1) return copy3d(hp, dp, false, st[1]);
        return rows == 1 ? cudaMemcpyAsync(dp, hp, width, cudaMemcpyHostToDevice, st[1])
                         : cudaMemcpy2DAsync(dp, dpitch, hp, hpitch, width, (size_t)rows, cudaMemcpyHostToDevice, st[1]);
    };
    const double gb = (double)spec->copy_bytes * (double)n / 1e9;
    double best_d2h = 0, best_h2d = 0, best_sum = 0, best_bd = 0, best_bh = 0;
    for (int round = 0; round <= spec->rounds; ++round) {       // round 0 warms up
        float ms = 0.f;
        KV_PROBE(cudaEventRecord(ev[0], st[0]));
        for (int64_t i = 0; i < n; ++i) KV_PROBE(d2h(i));
        KV_PROBE(cudaEventRecord(ev[1], st[0]));
        KV_PROBE(cudaStreamSynchronize(st[0]));
        KV_PROBE(cudaEventElapsedTime(&ms, ev[0], ev[1]));
        if (round) best_d2h = std::max(best_d2h, gb / (ms * 1e-3));
        KV_PROBE(cudaEventRecord(ev[0], st[1]));
        for (int64_t i = 0; i < n; ++i) KV_PROBE(h2d(i));
        KV_PROBE(cudaEventRecord(ev[1], st[1]));
        KV_PROBE(cudaStreamSynchronize(st[1]));
        KV_PROBE(cudaEventElapsedTime(&ms, ev[0], ev[1]));
        if (round) best_h2d = std::max(best_h2d, gb / (ms * 1e-3));
        // both at once; window = first start to last end
        KV_PROBE(cudaEventRecord(ev[0], st[0]));
        KV_PROBE(cudaEventRecord(ev[2], st[1]));
        for (int64_t i = 0; i < n; ++i) {
            KV_PROBE(d2h(i));
            KV_PROBE(h2d(i));
        }
        KV_PROBE(cudaEventRecord(ev[1], st[0]));
        KV_PROBE(cudaEventRecord(ev[3], st[1]));
        KV_PROBE(cudaStreamSynchronize(st[0]));
        KV_PROBE(cudaStreamSynchronize(st[1]));
        float t_out = 0.f, t_in = 0.f, a = 0.f, b = 0.f;
        KV_PROBE(cudaEventElapsedTime(&t_out, ev[0], ev[1]));
        KV_PROBE(cudaEventElapsedTime(&t_in, ev[2], ev[3]));
        const bool fwd = cudaEventElapsedTime(&a, ev[0], ev[2]) == cudaSuccess;
        const bool bwd = cudaEventElapsedTime(&b, ev[2], ev[0]) == cudaSuccess;
        const float offs = (fwd && a > 0.f) ? a : ((bwd && b > 0.f) ? -b : 0.f);
        const float win = std::max(t_out, offs + t_in) - std::min(0.f, offs);
        const double sum = 2 * gb / (win * 1e-3);
        if (round && sum > best_sum) {
            best_sum = sum;
            best_bd = gb / (t_out * 1e-3);
            best_bh = gb / (t_in * 1e-3);
        }
    }
#undef KV_PROBE
    out->d2h_gbs = best_d2h;
    out->h2d_gbs = best_h2d;
    out->bi_sum_gbs = best_sum;
    out->bi_d2h_gbs = best_bd;
    out->bi_h2d_gbs = best_bh;
    out->bytes = spec->copy_bytes;
    out->reps = (int32_t)std::min<int64_t>(n, INT32_MAX);
    cleanup();
    (void)cudaGetLastError();
    return KV_OK;
}

int32_t kv_probe_link(int32_t device_id, int64_t bytes, int32_t reps, kv_link_probe_t *out)
{
    if (bytes <= 0 || reps <= 0) return fail(nullptr, KV_ERR_INVALID_ARG, "bad probe arguments");
    kv_probe_spec_t spec;
    spec.copy_bytes = bytes;
    spec.total_bytes = bytes * reps;
    spec.span_bytes = bytes;
    spec.scattered = 0;
    spec.rounds = 3;
    spec.rows = 1;
    spec.host_pitch = spec.dev_pitch = 0;
    spec.slices = 1;
    spec.host_slice_rows = 0;
    return kv_probe_link_ex(device_id, &spec, out);
}

}  // extern "C"

// =================================================================================================
// Gather without any allocation.
//
// Some programs that want the gather cannot allocate CUDA memory at the point where they call it:
// a serving loop that must not hit the device-wide synchronisation cudaMalloc / cudaFree imply, a
// process whose device memory is entirely owned by another allocator (a framework's caching pool
// that was sized to the whole GPU), or a plug-in that is handed buffers and forbidden to make its
// own.  kv_pool_create allocates (descriptor rings, events, staging), so those callers cannot use
// a pool.  For them the id list that the copy kernel walks, and the status word its bounded waits
// report to, live in this fixed array, which every GPU that loads the library carries until exit.
#define KV_STATIC_STATUS_WORDS 64      // 256 bytes after the pairs; word 0 is the status word
static __device__ __align__(256) int2 kv_static_scratch[KV_STATIC_MAX_BLOCKS + KV_STATIC_STATUS_WORDS / 2];

namespace {
constexpr int KV_MAX_DEVICES = 64;
// device address of kv_static_scratch per device ordinal (in host code the array's name is only a
// host-side handle; kernels must be given the address cudaGetSymbolAddress returns)
void *g_static_scratch[KV_MAX_DEVICES] = {};
int2 g_static_pairs_host[KV_STATIC_MAX_BLOCKS];
}  // namespace

extern "C" int32_t kv_gather_blocks_static(const void *device_base, int32_t num_layers, int32_t block_size,
                                           int32_t kv_heads, int32_t head_dim, int64_t num_gpu_blocks,
                                           const int32_t *gpu_ids, int64_t n, void *dst_device, void *stream)
{
    const int64_t seg = kv_seg_bytes(block_size, kv_heads, head_dim);
    const int64_t blk = kv_blk_bytes(num_layers, block_size, kv_heads, head_dim);
    if (seg <= 0 || blk <= 0 || num_gpu_blocks <= 0 || num_gpu_blocks > INT32_MAX || seg > (1 << 30) ||
        2 * (int64_t)num_layers > (1 << 20))
        return fail(nullptr, KV_ERR_INVALID_ARG, "bad shape or pool size");
    if (seg % 16 != 0) return fail(nullptr, KV_ERR_UNSUPPORTED, "segment size must be a multiple of 16 bytes");
    if (n < 0) return fail(nullptr, KV_ERR_INVALID_ARG, "negative count");
    if (n == 0) return KV_OK;
    if (n > KV_STATIC_MAX_BLOCKS) {
        snprintf(g_err, 256, "n = %lld exceeds KV_STATIC_MAX_BLOCKS = %d, the capacity of the built-in id scratch",
                 (long long)n, KV_STATIC_MAX_BLOCKS);
        return KV_ERR_INVALID_ARG;
    }
    if (!device_base || !gpu_ids || !dst_device) return fail(nullptr, KV_ERR_INVALID_ARG, "null argument");
    if (((uintptr_t)device_base & 15) || ((uintptr_t)dst_device & 15))
        return fail(nullptr, KV_ERR_INVALID_ARG, "device_base and dst_device must be 16-byte aligned");
    for (int64_t i = 0; i < n; ++i) {
        if (gpu_ids[i] < 0 || (int64_t)gpu_ids[i] >= num_gpu_blocks) {
            snprintf(g_err, 256, "gpu_ids[%lld] = %d outside [0, %lld)", (long long)i, gpu_ids[i], (long long)num_gpu_blocks);
            return KV_ERR_RANGE;
        }
        g_static_pairs_host[i] = make_int2(gpu_ids[i], (int)i);
    }
    int dev = -1;
    KV_CUDA(nullptr, cudaGetDevice(&dev));
    if (dev < 0 || dev >= KV_MAX_DEVICES) return fail(nullptr, KV_ERR_UNSUPPORTED, "device ordinal beyond the table");
    if (!g_static_scratch[dev]) {
        // once per device, with that device current
        void *ptr = nullptr;
        KV_CUDA(nullptr, cudaGetSymbolAddress((void **)&ptr, kv_static_scratch));
        KV_CUDA(nullptr, prepare_bulk_kernels());
        g_static_scratch[dev] = ptr;
    }
    int2 *pairs = (int2 *)g_static_scratch[dev];
    unsigned int *status = (unsigned int *)(pairs + KV_STATIC_MAX_BLOCKS);
    cudaStream_t st = (cudaStream_t)stream;
    int sm_count = 0;
    KV_CUDA(nullptr, cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev));

    // the array keeps the previous call's contents: the pairs are overwritten, the status word is cleared
    KV_CUDA(nullptr, cudaMemcpyAsync(pairs, g_static_pairs_host, (size_t)n * sizeof(int2), cudaMemcpyHostToDevice, st));
    KV_CUDA(nullptr, cudaMemsetAsync(status, 0, sizeof(unsigned int), st));
    KvJob job;
    job.planes = 2 * num_layers;
    job.seg = (int)seg;
    job.chunk = (int)std::min<int64_t>(seg, BULK_STAGE);
    job.cps = (int)((seg + job.chunk - 1) / job.chunk);
    job.status = status;
    job.wait_polls = KV_WAIT_POLLS;
    job.wait_ns = KV_WAIT_NS;
    job.check_ids = 0;
    job.t_first = job.t_last = nullptr;
    job.dir[1] = KvDir{};
    KvDir &kd = job.dir[0];
    kd.src = KvSide{(unsigned long long)device_base, seg, num_gpu_blocks * seg};
    kd.dst = KvSide{(unsigned long long)dst_device, blk, seg};
    kd.pairs = pairs;
    kd.n = (int)n;
    kd.src_blocks = (int)num_gpu_blocks;
    kd.dst_blocks = (int)n;
    kd.ctas = clamp_ctas(job, kd, sm_count > 0 ? sm_count : 1);
    launch_bulk(nullptr, job, kd.ctas, st, false);
    KV_CUDA(nullptr, cudaGetLastError());
    unsigned int seen = 0;
    KV_CUDA(nullptr, cudaMemcpyAsync(&seen, status, sizeof(seen), cudaMemcpyDeviceToHost, st));
    KV_CUDA(nullptr, cudaStreamSynchronize(st));
    if (seen & KV_DEV_TIMEOUT) return fail(nullptr, KV_ERR_TIMEOUT, "a device-side wait ran out");
    return KV_OK;
}
