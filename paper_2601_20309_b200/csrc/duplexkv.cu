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
#include <cstring>
#include <new>
#include <vector>

namespace {

constexpr int KV_SLOTS = 8;            // descriptor / event ring depth per direction
constexpr int KV_MAX_CE_STREAMS = 4;
constexpr int BULK_STAGE = 16384;      // bytes per shared-memory stage of the bulk kernel
constexpr int BULK_NS = 8;             // stages
constexpr int BULK_AHEAD = 5;          // loads in flight ahead of the stores
constexpr int LDST_THREADS = 512;
constexpr int LDST_UNROLL = 4;         // 512 threads * 4 * 16 B = 32 KiB per item
constexpr int LDST_CHUNK = LDST_THREADS * LDST_UNROLL * 16;

thread_local char g_err[256] = "";

struct DirState {
    cudaStream_t stream = nullptr;
    bool owns_stream = false;
    int2 *ring_host = nullptr;         // pinned: KV_SLOTS slots of 2*cap pairs
    int2 *ring_dev = nullptr;          // device mirror
    cudaEvent_t ev_start[KV_SLOTS] = {};
    cudaEvent_t ev_end[KV_SLOTS] = {};
    uint64_t issued = 0;               // calls issued on this direction (sequence number of the latest)
    uint64_t done = 0;                 // latest call known to be complete
    uint8_t *stage = nullptr;          // HBM staging (STAGED path), allocated on first use
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
    int sm_count = 0;
    DirState dir[2];                   // 0 = out, 1 = in
    unsigned int *status_host = nullptr, *status_dev = nullptr;   // mapped pinned status word
    // per-block bookkeeping for validation and cross-direction ordering
    std::vector<uint32_t> g_mark, h_mark, g_mark2, h_mark2;
    uint32_t epoch = 0;
    std::vector<uint64_t> g_read_by_out, g_written_by_in, h_written_by_out, h_read_by_in;
    kv_stats_t stats;
    bool union_valid = false;
    int union_slot[2] = {-1, -1};      // slots of the latest call (per direction; -1 = not part of it)
    int32_t sticky = KV_OK;
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

KvSide device_side(const kv_pool *p)
{
    return KvSide{(unsigned long long)p->dev, p->seg, p->cfg.num_gpu_blocks * p->seg};
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

void fill_geometry(const kv_pool *p, KvJob &job)
{
    const int max_chunk = use_ldst(p) ? LDST_CHUNK : BULK_STAGE;
    job.planes = p->planes;
    job.seg = (int)p->seg;
    job.chunk = (int)std::min<int64_t>(p->seg, max_chunk);
    job.cps = (int)((p->seg + job.chunk - 1) / job.chunk);
    job.status = p->status_dev;
}

int clamp_ctas(const KvJob &job, const KvDir &d, int want)
{
    const long long items = (long long)d.n * job.planes * job.cps;
    return (int)std::max<long long>(1, std::min<long long>(want, items));
}

cudaError_t launch_job(kv_pool *p, const KvJob &job, cudaStream_t stream)
{
    const int grid = job.dir[0].ctas + job.dir[1].ctas;
    if (grid <= 0) return cudaSuccess;
    if (use_ldst(p)) {
        kv_copy_ldst<LDST_THREADS, LDST_UNROLL><<<grid, LDST_THREADS, 0, stream>>>(job);
    } else {
        kv_copy_bulk<BULK_STAGE, BULK_NS, BULK_AHEAD><<<grid, 32, BULK_STAGE * BULK_NS, stream>>>(job);
    }
    p->stats.kernel_launches++;
    return cudaGetLastError();
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
bool conflicts_with_other(kv_pool *p, int d, const int32_t *gpu_ids, const int32_t *host_ids, int64_t n)
{
    const DirState &o = p->dir[1 - d];
    if (o.done >= o.issued) return false;
    const std::vector<uint64_t> &gside = (d == 0) ? p->g_written_by_in : p->g_read_by_out;
    const std::vector<uint64_t> &hside = (d == 0) ? p->h_read_by_in : p->h_written_by_out;
    for (int64_t i = 0; i < n; ++i)
        if (gside[gpu_ids[i]] > o.done || hside[host_ids[i]] > o.done) return true;
    return false;
}

void note_use(kv_pool *p, int d, const int32_t *gpu_ids, const int32_t *host_ids, int64_t n, uint64_t seq)
{
    std::vector<uint64_t> &gside = (d == 0) ? p->g_read_by_out : p->g_written_by_in;
    std::vector<uint64_t> &hside = (d == 0) ? p->h_written_by_out : p->h_read_by_in;
    for (int64_t i = 0; i < n; ++i) {
        gside[gpu_ids[i]] = seq;
        hside[host_ids[i]] = seq;
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
    int64_t chunk_lo = 0;
    bool chunk_open = false;
    unsigned rr = 0;                   // round-robin cursor over the direction's CE streams
};

int resolve_path(const kv_pool *p, int d)
{
    int path = p->dir[d].path;
    if (path == KV_PATH_AUTO) path = kv_path_for(p->seg);
    return path;
}

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

int32_t begin_dir(kv_pool *p, DirCall &c, bool wait_other)
{
    DirState &s = p->dir[c.d];
    const uint64_t seq = s.issued + 1;
    c.slot = (int)(seq % KV_SLOTS);
    if (seq > KV_SLOTS) KV_CUDA(p, cudaEventSynchronize(s.ev_end[c.slot]));   // slot's previous user
    c.pairs_host = s.ring_host + (size_t)c.slot * 2 * p->cap;
    c.pairs_dev = s.ring_dev + (size_t)c.slot * 2 * p->cap;
    c.aux_host = c.pairs_host + p->cap;
    c.aux_dev = c.pairs_dev + p->cap;
    for (int64_t i = 0; i < c.n; ++i) {
        c.pairs_host[i] = (c.d == 0) ? make_int2(c.gpu_ids[i], c.host_ids[i]) : make_int2(c.host_ids[i], c.gpu_ids[i]);
        c.aux_host[i] = (c.d == 0) ? make_int2(c.gpu_ids[i], (int)i) : make_int2((int)i, c.gpu_ids[i]);
    }
    if (wait_other) {
        DirState &o = p->dir[1 - c.d];
        KV_CUDA(p, cudaStreamWaitEvent(s.stream, o.ev_end[o.issued % KV_SLOTS], 0));
    }
    KV_CUDA(p, cudaEventRecord(s.ev_start[c.slot], s.stream));
    if (c.path == KV_PATH_ZEROCOPY) {
        KV_CUDA(p, cudaMemcpyAsync(c.pairs_dev, c.pairs_host, (size_t)c.n * sizeof(int2), cudaMemcpyHostToDevice, s.stream));
    } else if (c.path == KV_PATH_STAGED) {
        KV_CUDA(p, cudaMemcpyAsync(c.aux_dev, c.aux_host, (size_t)c.n * sizeof(int2), cudaMemcpyHostToDevice, s.stream));
        if (!s.stage) {
            cudaError_t e = cudaMalloc((void **)&s.stage, (size_t)p->cfg.staging_bytes);
            if (e != cudaSuccess) {
                s.stage = nullptr;
                (void)cudaGetLastError();
                return fail(p, KV_ERR_NOMEM, "staging buffer allocation failed");
            }
        }
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

KvDir zerocopy_dir(kv_pool *p, const DirCall &c)
{
    KvDir d;
    d.src = (c.d == 0) ? device_side(p) : host_side(p);
    d.dst = (c.d == 0) ? host_side(p) : device_side(p);
    d.pairs = c.pairs_dev;
    d.n = (int)c.n;
    d.ctas = 0;
    return d;
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
            uint8_t *dv = p->dev + (pl * p->cfg.num_gpu_blocks + c.gpu_ids[i]) * p->seg;
            uint8_t *hv = host_block_ptr(p, c.host_ids[i]) + pl * (int64_t)host_pitch(p);
            KV_CUDA(p, cudaMemcpyAsync(c.d == 0 ? hv : dv, c.d == 0 ? dv : hv, (size_t)p->seg, kind, s.sub[i % s.nsub]));
            p->stats.ce_copies++;
            c.ce_next++;
        }
        finished = c.ce_next >= total;
        return KV_OK;
    }
    if (c.path == KV_PATH_CE2D) {
        // one strided transfer per block: `planes` rows of SEG bytes
        while (budget-- > 0 && c.ce_next < c.n) {
            const int64_t i = c.ce_next;
            uint8_t *dv = p->dev + (int64_t)c.gpu_ids[i] * p->seg;
            uint8_t *hv = host_block_ptr(p, c.host_ids[i]);
            const size_t dpitch = (size_t)(p->cfg.num_gpu_blocks * p->seg);
            cudaStream_t cs = s.sub[i % s.nsub];
            if (c.d == 0)
                KV_CUDA(p, cudaMemcpy2DAsync(hv, host_pitch(p), dv, dpitch, (size_t)p->seg, (size_t)p->planes, kind, cs));
            else
                KV_CUDA(p, cudaMemcpy2DAsync(dv, dpitch, hv, host_pitch(p), (size_t)p->seg, (size_t)p->planes, kind, cs));
            p->stats.ce_copies++;
            c.ce_next++;
        }
        finished = c.ce_next >= c.n;
        return KV_OK;
    }
    // STAGED: the list is cut into chunks of at most stage_blocks blocks.  Out: gather kernel into the
    // staging buffer, then one transfer per run of consecutive host ids.  In: the transfers, then the
    // scatter kernel.  Everything of one direction is on one stream, so reuse of the buffer is ordered.
    const int64_t stage_blocks = std::max<int64_t>(1, p->cfg.staging_bytes / p->blk);
    while (budget > 0 && c.chunk_lo < c.n) {
        const int64_t lo = c.chunk_lo, hi = std::min(c.n, lo + stage_blocks);
        KvJob job;
        fill_geometry(p, job);
        job.dir[1] = KvDir{};
        KvDir &kd = job.dir[0];
        // staging block of list position k is at stage + (k - lo)*BLK
        const KvSide st = packed_side(p, s.stage - lo * p->blk);
        kd.src = (c.d == 0) ? device_side(p) : st;
        kd.dst = (c.d == 0) ? st : device_side(p);
        kd.pairs = c.aux_dev + lo;
        kd.n = (int)(hi - lo);
        kd.ctas = clamp_ctas(job, kd, p->sm_count);
        if (c.ce_next == lo && !c.chunk_open) {
            // out: gather into the staging buffer first; both: the extra streams start after what
            // the main stream has done so far (the gather, or the previous chunk's scatter)
            if (c.d == 0) KV_CUDA(p, launch_job(p, job, s.stream));
            int32_t rc = ce_fork(p, s);
            if (rc != KV_OK) return rc;
            c.chunk_open = true;
        }
        while (budget > 0 && c.ce_next < hi) {
            int64_t k = c.ce_next, run = 1;
            if (p->cfg.host_layout == KV_HOST_BLOCK_FIRST) {
                while (k + run < hi && c.host_ids[k + run] == c.host_ids[k] + run) ++run;
                uint8_t *hv = host_block_ptr(p, c.host_ids[k]);
                uint8_t *sv = s.stage + (k - lo) * p->blk;
                KV_CUDA(p, cudaMemcpyAsync(c.d == 0 ? hv : sv, c.d == 0 ? sv : hv, (size_t)(run * p->blk), kind, s.sub[c.rr++ % s.nsub]));
            } else {
                uint8_t *hv = host_block_ptr(p, c.host_ids[k]);
                uint8_t *sv = s.stage + (k - lo) * p->blk;
                cudaStream_t cs = s.sub[c.rr++ % s.nsub];
                if (c.d == 0)
                    KV_CUDA(p, cudaMemcpy2DAsync(hv, host_pitch(p), sv, (size_t)p->seg, (size_t)p->seg, (size_t)p->planes, kind, cs));
                else
                    KV_CUDA(p, cudaMemcpy2DAsync(sv, (size_t)p->seg, hv, host_pitch(p), (size_t)p->seg, (size_t)p->planes, kind, cs));
            }
            p->stats.ce_copies++;
            c.ce_next += run;
            --budget;
        }
        if (c.ce_next >= hi) {
            int32_t rc = ce_join(p, s);
            if (rc != KV_OK) return rc;
            if (c.d == 1) KV_CUDA(p, launch_job(p, job, s.stream));
            c.chunk_lo = hi;
            c.chunk_open = false;
        }
    }
    finished = c.chunk_lo >= c.n;
    return KV_OK;
}

// Issue the payload movement of up to two prepared directions.
int32_t issue_calls(kv_pool *p, DirCall *calls, int ncalls, bool fused)
{
    // kernel (zero-copy) directions
    if (fused && ncalls == 2 && calls[0].path == KV_PATH_ZEROCOPY && calls[1].path == KV_PATH_ZEROCOPY) {
        KvJob job;
        fill_geometry(p, job);
        job.dir[0] = zerocopy_dir(p, calls[0]);
        job.dir[1] = zerocopy_dir(p, calls[1]);
        job.dir[0].ctas = clamp_ctas(job, job.dir[0], p->dir[0].ctas);
        job.dir[1].ctas = clamp_ctas(job, job.dir[1], p->dir[1].ctas);
        KV_CUDA(p, launch_job(p, job, p->dir[0].stream));
        return KV_OK;
    }
    for (int k = 0; k < ncalls; ++k) {
        DirCall &c = calls[k];
        if (c.path != KV_PATH_ZEROCOPY) continue;
        KvJob job;
        fill_geometry(p, job);
        job.dir[0] = zerocopy_dir(p, c);
        job.dir[1] = KvDir{};
        job.dir[0].ctas = clamp_ctas(job, job.dir[0], p->dir[c.d].ctas);
        KV_CUDA(p, launch_job(p, job, p->dir[c.d].stream));
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

int32_t run_calls(kv_pool *p, DirCall *calls, int ncalls, const bool *wait_other, bool fused)
{
    p->union_slot[0] = p->union_slot[1] = -1;
    for (int k = 0; k < ncalls; ++k) {
        calls[k].path = resolve_path(p, calls[k].d);
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
        for (int k = 0; k < ncalls && rc == KV_OK; ++k) rc = begin_dir(p, calls[k], wait_other[k]);
        if (rc == KV_OK) rc = issue_calls(p, calls, ncalls, true);
        for (int k = 0; k < ncalls && rc == KV_OK; ++k) rc = end_dir(p, calls[k]);
        p->dir[1].stream = keep;
        if (rc != KV_OK) return rc;
        KV_CUDA(p, cudaStreamWaitEvent(keep, p->dir[1].ev_end[calls[1].slot], 0));
    } else {
        for (int k = 0; k < ncalls; ++k) {
            int32_t rc = begin_dir(p, calls[k], wait_other[k]);
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

int32_t kv_path_for(int64_t seg_bytes)
{
    (void)seg_bytes;
    return KV_PATH_ZEROCOPY;
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
    if (cfg->path < KV_PATH_AUTO || cfg->path > KV_PATH_NAIVE || cfg->path_in < KV_PATH_AUTO || cfg->path_in > KV_PATH_NAIVE)
        return fail(nullptr, KV_ERR_INVALID_ARG, "unknown path");
    if (cfg->ctas_out < 0 || cfg->ctas_in < 0 || cfg->staging_bytes < 0 || cfg->ce_streams < 0 ||
        cfg->ce_streams > KV_MAX_CE_STREAMS)
        return fail(nullptr, KV_ERR_INVALID_ARG, "tuning value out of range");

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
    if (p->cfg.staging_bytes == 0) p->cfg.staging_bytes = 64ll << 20;
    if (p->cfg.staging_bytes < blk) p->cfg.staging_bytes = blk;

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

    const size_t host_bytes = (size_t)cfg->num_host_blocks * (size_t)blk;
    if (cfg->host_base) {
        p->host = (uint8_t *)cfg->host_base;
        cudaError_t e = cudaHostRegister(p->host, host_bytes, cudaHostRegisterMapped | cudaHostRegisterPortable);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            int32_t rc = fail(nullptr, KV_ERR_NOMEM, "cudaHostRegister of host_base failed");
            kv_pool_destroy(p);
            return rc;
        }
        p->registered_host = true;
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
        s.ctas = want_ctas[d] > 0 ? want_ctas[d] : 32;
        s.path = (d == 1 && cfg->path_in != KV_PATH_AUTO) ? cfg->path_in : cfg->path;
        s.nsub = cfg->ce_streams > 0 ? cfg->ce_streams : 1;
        s.sub[0] = s.stream;
        KV_CREATE_CUDA(cudaEventCreateWithFlags(&s.fork_ev, cudaEventDisableTiming));
        for (int k = 1; k < s.nsub; ++k) {
            KV_CREATE_CUDA(cudaStreamCreateWithFlags(&s.sub[k], cudaStreamNonBlocking));
            KV_CREATE_CUDA(cudaEventCreateWithFlags(&s.join_ev[k], cudaEventDisableTiming));
        }
    }
    KV_CREATE_CUDA(cudaFuncSetAttribute(kv_copy_bulk<BULK_STAGE, BULK_NS, BULK_AHEAD>,
                                        cudaFuncAttributeMaxDynamicSharedMemorySize, BULK_STAGE * BULK_NS));
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
        if (s.ring_host) (void)cudaFreeHost(s.ring_host);
        if (s.ring_dev) (void)cudaFree(s.ring_dev);
        if (s.stage) (void)cudaFree(s.stage);
        if (s.owns_stream && s.stream) (void)cudaStreamDestroy(s.stream);
    }
    if (p->status_host) (void)cudaFreeHost(p->status_host);
    if (p->owns_host && p->host) (void)cudaFreeHost(p->host);
    if (p->registered_host) (void)cudaHostUnregister(p->host);
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
        const bool fused = (p->cfg.flags & KV_FLAG_FUSED_ROTATE) && resolve_path(p, 0) == KV_PATH_ZEROCOPY &&
                           resolve_path(p, 1) == KV_PATH_ZEROCOPY && !wait[0] && !wait[1];
        return run_calls(p, calls, 2, wait, fused);
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

int32_t kv_sync(kv_pool_t *p)
{
    if (!p) return KV_ERR_INVALID_ARG;
    for (int d = 0; d < 2; ++d) {
        cudaError_t e = cudaStreamSynchronize(p->dir[d].stream);
        if (e != cudaSuccess) return fail_cuda(p, e, "cudaStreamSynchronize");
        p->dir[d].done = p->dir[d].issued;
    }
    if (p->union_valid) {
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
        } else {
            p->stats.last_union_ms = so >= 0 ? t_out : t_in;
        }
        (void)cudaGetLastError();
        p->union_valid = false;
    }
    const unsigned int st = *(volatile unsigned int *)p->status_host;
    p->stats.device_status = st;
    if (st & KV_DEV_TIMEOUT) {
        if (p->sticky == KV_OK) p->sticky = KV_ERR_TIMEOUT;
        snprintf(p->err, 256, "a device-side wait ran out (status 0x%x)", st);
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
    const uint64_t seq = s.issued + 1;
    const int slot = (int)(seq % KV_SLOTS);
    if (seq > KV_SLOTS) KV_CUDA(p, cudaEventSynchronize(s.ev_end[slot]));
    int2 *ph = s.ring_host + (size_t)slot * 2 * p->cap;
    int2 *pd = s.ring_dev + (size_t)slot * 2 * p->cap;
    for (int64_t i = 0; i < n; ++i) ph[i] = (d == 0) ? make_int2(gpu_ids[i], (int)i) : make_int2((int)i, gpu_ids[i]);
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
    const int want = (d == 0 ? p->cfg.ctas_out : p->cfg.ctas_in);
    kd.ctas = clamp_ctas(job, kd, want > 0 ? want : p->sm_count);
    KV_CUDA(p, launch_job(p, job, s.stream));
    KV_CUDA(p, cudaEventRecord(s.ev_end[slot], s.stream));
    s.issued = seq;
    p->union_slot[d] = slot;
    p->union_slot[1 - d] = -1;
    p->union_valid = true;
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
    p->stats.device_status = *(volatile unsigned int *)p->status_host;
    *st = p->stats;
    return KV_OK;
}

int32_t kv_probe_link(int32_t device_id, int64_t bytes, int32_t reps, kv_link_probe_t *out)
{
    if (!out || bytes <= 0 || reps <= 0) return fail(nullptr, KV_ERR_INVALID_ARG, "bad probe arguments");
    memset(out, 0, sizeof(*out));
    KV_CUDA(nullptr, cudaSetDevice(device_id));
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
        KV_PROBE(cudaHostAlloc((void **)&h[k], (size_t)bytes, cudaHostAllocDefault));
        memset(h[k], k + 1, (size_t)bytes);
        KV_PROBE(cudaMalloc((void **)&dv[k], (size_t)bytes));
        KV_PROBE(cudaMemset(dv[k], 0, (size_t)bytes));
        KV_PROBE(cudaStreamCreateWithFlags(&st[k], cudaStreamNonBlocking));
    }
    for (int k = 0; k < 4; ++k) KV_PROBE(cudaEventCreate(&ev[k]));
    const double gb = (double)bytes * reps / 1e9;
    double best_d2h = 0, best_h2d = 0, best_sum = 0, best_bd = 0, best_bh = 0;
    for (int round = 0; round < 4; ++round) {
        float ms = 0.f;
        KV_PROBE(cudaEventRecord(ev[0], st[0]));
        for (int r = 0; r < reps; ++r) KV_PROBE(cudaMemcpyAsync(h[0], dv[0], (size_t)bytes, cudaMemcpyDeviceToHost, st[0]));
        KV_PROBE(cudaEventRecord(ev[1], st[0]));
        KV_PROBE(cudaStreamSynchronize(st[0]));
        KV_PROBE(cudaEventElapsedTime(&ms, ev[0], ev[1]));
        if (round) best_d2h = std::max(best_d2h, gb / (ms * 1e-3));
        KV_PROBE(cudaEventRecord(ev[0], st[1]));
        for (int r = 0; r < reps; ++r) KV_PROBE(cudaMemcpyAsync(dv[1], h[1], (size_t)bytes, cudaMemcpyHostToDevice, st[1]));
        KV_PROBE(cudaEventRecord(ev[1], st[1]));
        KV_PROBE(cudaStreamSynchronize(st[1]));
        KV_PROBE(cudaEventElapsedTime(&ms, ev[0], ev[1]));
        if (round) best_h2d = std::max(best_h2d, gb / (ms * 1e-3));
        // both at once; window = first start to last end
        KV_PROBE(cudaEventRecord(ev[0], st[0]));
        KV_PROBE(cudaEventRecord(ev[2], st[1]));
        for (int r = 0; r < reps; ++r) {
            KV_PROBE(cudaMemcpyAsync(h[0], dv[0], (size_t)bytes, cudaMemcpyDeviceToHost, st[0]));
            KV_PROBE(cudaMemcpyAsync(dv[1], h[1], (size_t)bytes, cudaMemcpyHostToDevice, st[1]));
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
        const float off = (fwd && a > 0.f) ? a : ((bwd && b > 0.f) ? -b : 0.f);
        const float win = std::max(t_out, off + t_in) - std::min(0.f, off);
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
    out->bytes = bytes;
    out->reps = reps;
    cleanup();
    (void)cudaGetLastError();
    return KV_OK;
}

}  // extern "C"
