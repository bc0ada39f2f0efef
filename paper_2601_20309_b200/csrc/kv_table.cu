// Block table with eager block rotation: request-level bookkeeping on top of a pool.
//
// Follows the paper's section 4.3.2 ("Eager block rotation for data race free overlapping"): KV
// generation is incremental, so a block that is completely filled never changes again until its
// request finishes ("synced" once it has a copy in host memory), while the last, partly filled block
// is "dirty".  Full blocks are copied to host memory in the background before any preemption; when a
// request is preempted only what has no valid host copy is moved (normally the one dirty block) and
// the device blocks that do have one are simply released.  Because those blocks are released without
// waiting for any transfer, the requests that resume in the same rotation can take them at once, and
// the swap-in of a rotation never depends on its swap-out.  The host copies are kept while a request
// runs on the GPU (host-side duplication; no extra HBM).
//
// This file is host code only.  It decides WHICH blocks move and calls kv_swap_out / kv_rotate of the
// pool to move them; with no pool (kv_table_create_dry) it does the bookkeeping alone, which is how
// the allocator and the state machine are tested without a GPU.
//
// Host blocks are handed out in runs (first fit over the free extents, largest extents when nothing
// fits), so the blocks a request sends out together are neighbours in host memory and travel as few,
// long copy-engine transfers.  Device blocks come from a plain LIFO free list: the pack kernel makes
// the device side of a transfer contiguous whatever the ids are.
#include "../../include/duplexkv.h"

#include <algorithm>
#include <deque>
#include <cstdio>
#include <cstring>
#include <map>
#include <new>
#include <unordered_map>
#include <vector>

namespace {

struct TBlock {
    int32_t g = -1;             // device block id, -1 = none
    int32_t h = -1;             // host block id, -1 = none
    bool host_valid = false;    // the host copy holds the block's current content
};

struct TReq {
    int64_t tokens = 0;
    bool on_gpu = true;
    std::vector<TBlock> blocks;
};

struct TPending {
    int32_t g;
    int64_t out_seq, in_seq;
};

// free host blocks as disjoint extents start -> length
class ExtentAllocator {
  public:
    void reset(int64_t n)
    {
        free_.clear();
        if (n > 0) free_[0] = n;
        nfree_ = n;
    }
    int64_t free_blocks() const { return nfree_; }
    // take n blocks, as one run when some extent holds n, else from the largest extents downwards
    bool take(int64_t n, std::vector<int32_t> &out)
    {
        if (n > nfree_) return false;
        while (n > 0) {
            auto pick = free_.end();
            for (auto it = free_.begin(); it != free_.end(); ++it)        // first fit
                if (it->second >= n) {
                    pick = it;
                    break;
                }
            if (pick == free_.end())                                      // nothing fits: largest extent
                for (auto it = free_.begin(); it != free_.end(); ++it)
                    if (pick == free_.end() || it->second > pick->second) pick = it;
            const int64_t start = pick->first, len = pick->second, use = std::min(len, n);
            for (int64_t k = 0; k < use; ++k) out.push_back((int32_t)(start + k));
            free_.erase(pick);
            if (use < len) free_[start + use] = len - use;
            n -= use;
            nfree_ -= use;
        }
        return true;
    }
    void give(int32_t id)
    {
        int64_t start = id, len = 1;
        auto nxt = free_.lower_bound(start);
        if (nxt != free_.end() && nxt->first == start + 1) {              // merge with the extent after
            len += nxt->second;
            nxt = free_.erase(nxt);
        }
        if (nxt != free_.begin()) {                                       // merge with the extent before
            auto prv = std::prev(nxt);
            if (prv->first + prv->second == start) {
                start = prv->first;
                len += prv->second;
                free_.erase(prv);
            }
        }
        free_[start] = len;
        nfree_++;
    }
    int64_t extents() const { return (int64_t)free_.size(); }

  private:
    std::map<int64_t, int64_t> free_;
    int64_t nfree_ = 0;
};

}  // namespace

struct kv_table {
    kv_pool_t *pool = nullptr;      // nullptr = bookkeeping only
    int64_t nb_gpu = 0, nb_host = 0;
    int32_t block_size = 0;
    std::vector<int32_t> gpu_free;  // LIFO; safe for anyone to write
    // device blocks released while a transfer that may still touch them was in flight, with the numbers
    // of the latest swap-out and swap-in calls at release time.  The pool orders its own swap-ins behind
    // those calls, so a resume may take such blocks at once; a caller who writes tokens may not, so
    // kv_req_add / kv_req_append only hand out blocks from gpu_free and wait for the pool when that
    // runs short.
    std::deque<TPending> gpu_pending;
    ExtentAllocator host_free;
    std::unordered_map<int64_t, TReq> reqs;
    std::vector<int64_t> order;     // request ids in arrival order (eager rotation walks it round-robin)
    size_t eager_cursor = 0;
    kv_table_stats_t stats;
    // test hook (kv_table_fail_pool_call): the pool call that is `fail_after` calls away returns
    // `fail_code` instead of being made; -1 = not armed
    int64_t fail_after = -1;
    int32_t fail_code = KV_OK;
    char err[256];
};

namespace {

int32_t tfail(kv_table *t, int32_t code, const char *msg)
{
    snprintf(t->err, 256, "%s", msg);
    return code;
}

inline int64_t blocks_for(const kv_table *t, int64_t tokens) { return (tokens + t->block_size - 1) / t->block_size; }
inline bool is_full(const kv_table *t, const TReq &r, size_t i) { return (int64_t)(i + 1) * t->block_size <= r.tokens; }

TReq *find(kv_table *t, int64_t req)
{
    auto it = t->reqs.find(req);
    return it == t->reqs.end() ? nullptr : &it->second;
}

// host ids for the blocks of `r` listed in `idx` that have none yet, as one run where possible
bool give_host_ids(kv_table *t, TReq &r, const std::vector<size_t> &idx)
{
    int64_t need = 0;
    for (size_t i : idx)
        if (r.blocks[i].h < 0) ++need;
    if (need == 0) return true;
    std::vector<int32_t> ids;
    if (!t->host_free.take(need, ids)) return false;
    size_t k = 0;
    for (size_t i : idx)
        if (r.blocks[i].h < 0) r.blocks[i].h = ids[k++];
    return true;
}

// numbers of the latest swap-out and swap-in calls issued on the pool
TPending now(kv_table *t)
{
    TPending p{-1, 0, 0};
    if (t->pool) (void)kv_pool_progress(t->pool, &p.out_seq, nullptr, &p.in_seq, nullptr);
    return p;
}

void release_gpu(kv_table *t, int32_t g, const TPending &at)
{
    if (t->pool && (at.out_seq > 0 || at.in_seq > 0)) t->gpu_pending.push_back(TPending{g, at.out_seq, at.in_seq});
    else t->gpu_free.push_back(g);
}

// move released blocks that no transfer can touch any more to the free list; with `wait`, finish the transfers first
int32_t reclaim(kv_table *t, bool wait)
{
    if (t->gpu_pending.empty() || !t->pool) return KV_OK;
    if (wait) {
        int32_t rc = kv_sync(t->pool);
        if (rc != KV_OK) return rc;
    }
    int64_t out_done = 0, in_done = 0;
    (void)kv_pool_progress(t->pool, nullptr, &out_done, nullptr, &in_done);
    while (!t->gpu_pending.empty() && t->gpu_pending.front().out_seq <= out_done && t->gpu_pending.front().in_seq <= in_done) {
        t->gpu_free.push_back(t->gpu_pending.front().g);
        t->gpu_pending.pop_front();
    }
    return KV_OK;
}

// n device blocks that nobody is reading any more (for tokens the caller is about to write)
int32_t take_quiet_gpu(kv_table *t, int64_t n, std::vector<int32_t> &out)
{
    (void)reclaim(t, false);
    if ((int64_t)t->gpu_free.size() < n) {
        int32_t rc = reclaim(t, true);
        if (rc != KV_OK) return rc;
    }
    if ((int64_t)t->gpu_free.size() < n) return KV_ERR_NOMEM;
    for (int64_t k = 0; k < n; ++k) {
        out.push_back(t->gpu_free.back());
        t->gpu_free.pop_back();
    }
    return KV_OK;
}

// a device block for a swap-in destination: any released block will do
int32_t take_any_gpu(kv_table *t)
{
    int32_t g;
    if (!t->gpu_free.empty()) {
        g = t->gpu_free.back();
        t->gpu_free.pop_back();
    } else {
        g = t->gpu_pending.front().g;
        t->gpu_pending.pop_front();
    }
    return g;
}

inline int64_t gpu_available(const kv_table *t) { return (int64_t)(t->gpu_free.size() + t->gpu_pending.size()); }

// Is the pool call about to be made the one a test asked to fail?  (Host-side fault injection: the call
// is then not made at all, so nothing reaches the device.)
int32_t injected_failure(kv_table *t)
{
    if (t->fail_after < 0) return KV_OK;
    if (t->fail_after-- > 0) return KV_OK;
    snprintf(t->err, 256, "pool call failed (%d): injected by kv_table_fail_pool_call", t->fail_code);
    return t->fail_code;
}

int32_t pool_swap_out(kv_table *t, const std::vector<int32_t> &og, const std::vector<int32_t> &oh)
{
    int32_t rc = injected_failure(t);
    if (rc != KV_OK || !t->pool) return rc;
    rc = kv_swap_out(t->pool, og.data(), oh.data(), (int64_t)og.size());
    if (rc != KV_OK) snprintf(t->err, 256, "pool call failed (%d): %s", rc, kv_last_error(t->pool));
    return rc;
}

int32_t pool_rotate(kv_table *t, const std::vector<int32_t> &og, const std::vector<int32_t> &oh,
                    const std::vector<int32_t> &ih, const std::vector<int32_t> &ig)
{
    int32_t rc = injected_failure(t);
    if (rc != KV_OK || !t->pool) return rc;
    rc = kv_rotate(t->pool, og.data(), oh.data(), (int64_t)og.size(), ih.data(), ig.data(), (int64_t)ig.size());
    if (rc != KV_OK) snprintf(t->err, 256, "pool call failed (%d): %s", rc, kv_last_error(t->pool));
    return rc;
}

}  // namespace

extern "C" {

static int32_t table_new(kv_pool_t *pool, int64_t nb_gpu, int64_t nb_host, int32_t block_size, kv_table_t **out)
{
    if (!out) return KV_ERR_INVALID_ARG;
    *out = nullptr;
    if (nb_gpu <= 0 || nb_host <= 0 || nb_gpu > INT32_MAX || nb_host > INT32_MAX || block_size <= 0) return KV_ERR_INVALID_ARG;
    kv_table *t = new (std::nothrow) kv_table();
    if (!t) return KV_ERR_NOMEM;
    t->pool = pool;
    t->nb_gpu = nb_gpu;
    t->nb_host = nb_host;
    t->block_size = block_size;
    t->err[0] = 0;
    memset(&t->stats, 0, sizeof(t->stats));
    try {
        t->gpu_free.resize((size_t)nb_gpu);
        for (int64_t i = 0; i < nb_gpu; ++i) t->gpu_free[(size_t)i] = (int32_t)(nb_gpu - 1 - i);   // pops 0, 1, 2, ...
    } catch (...) {
        delete t;
        return KV_ERR_NOMEM;
    }
    t->host_free.reset(nb_host);
    *out = t;
    return KV_OK;
}

int32_t kv_table_create(kv_pool_t *pool, kv_table_t **out)
{
    if (!pool) return KV_ERR_INVALID_ARG;
    kv_pool_shape_t sh;
    int32_t rc = kv_pool_shape(pool, &sh);
    if (rc != KV_OK) return rc;
    return table_new(pool, sh.num_gpu_blocks, sh.num_host_blocks, sh.block_size, out);
}

int32_t kv_table_create_dry(int64_t num_gpu_blocks, int64_t num_host_blocks, int32_t block_size, kv_table_t **out)
{
    return table_new(nullptr, num_gpu_blocks, num_host_blocks, block_size, out);
}

int32_t kv_table_destroy(kv_table_t *t)
{
    if (!t) return KV_ERR_INVALID_ARG;
    delete t;
    return KV_OK;
}

const char *kv_table_last_error(kv_table_t *t) { return t ? t->err : "null table"; }

int32_t kv_req_add(kv_table_t *t, int64_t req, int64_t tokens)
{
    if (!t) return KV_ERR_INVALID_ARG;
    if (tokens <= 0) return tfail(t, KV_ERR_INVALID_ARG, "a request needs at least one token");
    if (find(t, req)) return tfail(t, KV_ERR_INVALID_ARG, "request id already present");
    const int64_t nb = blocks_for(t, tokens);
    if (nb > gpu_available(t)) return tfail(t, KV_ERR_NOMEM, "not enough free device blocks");
    try {
        std::vector<int32_t> ids;
        int32_t rc = take_quiet_gpu(t, nb, ids);
        if (rc != KV_OK) return tfail(t, rc, "could not obtain device blocks");
        TReq r;
        r.tokens = tokens;
        r.on_gpu = true;
        r.blocks.resize((size_t)nb);
        for (size_t i = 0; i < r.blocks.size(); ++i) r.blocks[i].g = ids[i];
        t->reqs.emplace(req, std::move(r));
        t->order.push_back(req);
    } catch (...) {
        return tfail(t, KV_ERR_NOMEM, "out of host memory");
    }
    return KV_OK;
}

int32_t kv_req_append(kv_table_t *t, int64_t req, int64_t new_tokens)
{
    if (!t) return KV_ERR_INVALID_ARG;
    TReq *r = find(t, req);
    if (!r) return tfail(t, KV_ERR_INVALID_ARG, "unknown request");
    if (!r->on_gpu) return tfail(t, KV_ERR_INVALID_ARG, "only a request that is on the GPU generates tokens");
    if (new_tokens <= 0) return tfail(t, KV_ERR_INVALID_ARG, "non-positive token count");
    const int64_t have = (int64_t)r->blocks.size(), want = blocks_for(t, r->tokens + new_tokens);
    if (want - have > gpu_available(t)) return tfail(t, KV_ERR_NOMEM, "not enough free device blocks");
    std::vector<int32_t> ids;
    try {
        int32_t rc = take_quiet_gpu(t, want - have, ids);
        if (rc != KV_OK) return tfail(t, rc, "could not obtain device blocks");
        r->blocks.resize((size_t)want);
    } catch (...) {
        return tfail(t, KV_ERR_NOMEM, "out of host memory");
    }
    // new tokens land in the partly filled last block first: a host copy of it goes stale
    if (r->tokens % t->block_size != 0) r->blocks[(size_t)have - 1].host_valid = false;
    for (int64_t i = have; i < want; ++i) r->blocks[(size_t)i].g = ids[(size_t)(i - have)];
    r->tokens += new_tokens;
    return KV_OK;
}

int32_t kv_eager_rotate(kv_table_t *t, int64_t max_blocks, int64_t *n_issued)
{
    if (n_issued) *n_issued = 0;
    if (!t || max_blocks < 0) return KV_ERR_INVALID_ARG;
    std::vector<int32_t> og, oh;
    std::vector<std::pair<int64_t, size_t>> picked;    // (request, block index)
    std::vector<bool> fresh_host;                      // per picked block: its host id was handed out by this call
    const size_t nreq = t->order.size();
    size_t visited = 0;
    // all or nothing: if the pool refuses the copy, the host ids handed out here go back and the walk stays put
    auto undo = [&]() {
        for (size_t k = picked.size(); k-- > 0;)
            if (k < fresh_host.size() && fresh_host[k]) {
                TBlock &b = t->reqs[picked[k].first].blocks[picked[k].second];
                t->host_free.give(b.h);
                b.h = -1;
            }
    };
    try {
        for (; visited < nreq && (int64_t)picked.size() < max_blocks; ++visited) {
            const int64_t id = t->order[(t->eager_cursor + visited) % nreq];
            TReq &r = t->reqs[id];
            if (!r.on_gpu) continue;
            std::vector<size_t> idx;
            for (size_t i = 0; i < r.blocks.size() && (int64_t)(picked.size() + idx.size()) < max_blocks; ++i)
                if (is_full(t, r, i) && !r.blocks[i].host_valid) idx.push_back(i);
            if (idx.empty()) continue;
            std::vector<bool> had;
            for (size_t i : idx) had.push_back(r.blocks[i].h >= 0);
            if (!give_host_ids(t, r, idx)) break;      // host pool exhausted: send what was gathered so far
            for (size_t q = 0; q < idx.size(); ++q) {
                picked.emplace_back(id, idx[q]);
                fresh_host.push_back(!had[q]);
            }
        }
        for (auto &pi : picked) {
            TBlock &b = t->reqs[pi.first].blocks[pi.second];
            og.push_back(b.g);
            oh.push_back(b.h);
        }
    } catch (...) {
        undo();
        return tfail(t, KV_ERR_NOMEM, "out of host memory");
    }
    if (!picked.empty()) {
        int32_t rc = pool_swap_out(t, og, oh);
        if (rc != KV_OK) {
            undo();
            return rc;
        }
    }
    if (nreq) t->eager_cursor = (t->eager_cursor + visited) % nreq;
    if (picked.empty()) return KV_OK;
    for (auto &pi : picked) t->reqs[pi.first].blocks[pi.second].host_valid = true;
    t->stats.eager_blocks += (int64_t)picked.size();
    t->stats.eager_calls++;
    if (n_issued) *n_issued = (int64_t)picked.size();
    return KV_OK;
}

int32_t kv_req_rotate(kv_table_t *t, const int64_t *preempt, int64_t n_preempt, const int64_t *resume, int64_t n_resume)
{
    if (!t || n_preempt < 0 || n_resume < 0 || (n_preempt && !preempt) || (n_resume && !resume)) return KV_ERR_INVALID_ARG;
    // ---- validation and capacity, before anything changes
    int64_t discard = 0, need_gpu = 0, need_host = 0;
    for (int64_t k = 0; k < n_preempt; ++k) {
        TReq *r = find(t, preempt[k]);
        if (!r || !r->on_gpu) return tfail(t, KV_ERR_INVALID_ARG, "a request to preempt is unknown or not on the GPU");
        for (int64_t j = 0; j < k; ++j)
            if (preempt[j] == preempt[k]) return tfail(t, KV_ERR_INVALID_ARG, "request listed twice");
        for (auto &b : r->blocks) {
            if (b.host_valid) ++discard;
            else if (b.h < 0) ++need_host;
        }
    }
    for (int64_t k = 0; k < n_resume; ++k) {
        TReq *r = find(t, resume[k]);
        if (!r || r->on_gpu) return tfail(t, KV_ERR_INVALID_ARG, "a request to resume is unknown or already on the GPU");
        for (int64_t j = 0; j < k; ++j)
            if (resume[j] == resume[k]) return tfail(t, KV_ERR_INVALID_ARG, "request listed twice");
        need_gpu += (int64_t)r->blocks.size();
    }
    if (need_gpu > gpu_available(t) + discard) return tfail(t, KV_ERR_NOMEM, "not enough free device blocks to resume");
    if (need_host > t->host_free.free_blocks()) return tfail(t, KV_ERR_NOMEM, "not enough free host blocks to preempt");

    std::vector<int32_t> og, oh, ih, ig;
    const TPending seq_before = now(t);             // transfers issued so far may still touch what is released now
    // All or nothing: steps 1 to 3 work on the table itself (the resuming requests take the very blocks the
    // preempted ones release), so what they touch is saved first and put back if the pool refuses the rotation.
    struct Saved {
        std::vector<int32_t> gpu_free;
        std::deque<TPending> gpu_pending;
        ExtentAllocator host_free;
        std::vector<std::pair<int64_t, std::vector<TBlock>>> blocks;
        int64_t discarded;
    } saved;
    try {
        saved.gpu_free = t->gpu_free;
        saved.gpu_pending = t->gpu_pending;
        saved.host_free = t->host_free;
        saved.discarded = t->stats.discarded_blocks;
        for (int64_t k = 0; k < n_preempt; ++k) saved.blocks.emplace_back(preempt[k], t->reqs[preempt[k]].blocks);
        for (int64_t k = 0; k < n_resume; ++k) saved.blocks.emplace_back(resume[k], t->reqs[resume[k]].blocks);
    } catch (...) {
        return tfail(t, KV_ERR_NOMEM, "out of host memory");
    }
    auto restore = [&]() {
        t->gpu_free.swap(saved.gpu_free);
        t->gpu_pending.swap(saved.gpu_pending);
        t->host_free = saved.host_free;
        t->stats.discarded_blocks = saved.discarded;
        for (auto &sb : saved.blocks) t->reqs[sb.first].blocks.swap(sb.second);
    };
    try {
        // ---- 1. device blocks that have a valid host copy are released at once, nothing is copied
        for (int64_t k = 0; k < n_preempt; ++k)
            for (auto &b : t->reqs[preempt[k]].blocks)
                if (b.host_valid) {
                    release_gpu(t, b.g, seq_before);
                    b.g = -1;
                    t->stats.discarded_blocks++;
                }
        // ---- 2. the resuming requests take device blocks (possibly the ones just released)
        for (int64_t k = 0; k < n_resume; ++k)
            for (auto &b : t->reqs[resume[k]].blocks) {
                b.g = take_any_gpu(t);
                ih.push_back(b.h);
                ig.push_back(b.g);
            }
        // ---- 3. what the preempted requests still have to send: blocks without a valid host copy
        for (int64_t k = 0; k < n_preempt; ++k) {
            TReq &r = t->reqs[preempt[k]];
            std::vector<size_t> idx;
            for (size_t i = 0; i < r.blocks.size(); ++i)
                if (!r.blocks[i].host_valid) idx.push_back(i);
            if (!give_host_ids(t, r, idx)) {          // excluded by the check above
                restore();
                return tfail(t, KV_ERR_NOMEM, "host pool exhausted");
            }
            for (size_t i : idx) {
                og.push_back(r.blocks[i].g);
                oh.push_back(r.blocks[i].h);
            }
        }
    } catch (...) {
        restore();
        return tfail(t, KV_ERR_NOMEM, "out of host memory");
    }
    // ---- 4. one rotation: its swap-in destinations are never its swap-out sources (those are still held)
    if (!og.empty() || !ig.empty()) {
        int32_t rc = pool_rotate(t, og, oh, ih, ig);
        if (rc != KV_OK) {
            restore();
            return rc;
        }
    }
    // ---- 5. the sent blocks' device ids are released; this call's swap-out is the one that reads them
    const TPending seq_after = now(t);
    for (int64_t k = 0; k < n_preempt; ++k) {
        TReq &r = t->reqs[preempt[k]];
        for (auto &b : r.blocks) {
            if (b.g >= 0) {
                release_gpu(t, b.g, seq_after);
                b.g = -1;
            }
            b.host_valid = true;
        }
        r.on_gpu = false;
    }
    for (int64_t k = 0; k < n_resume; ++k) t->reqs[resume[k]].on_gpu = true;
    t->stats.preempt_blocks_moved += (int64_t)og.size();
    t->stats.resume_blocks_moved += (int64_t)ig.size();
    t->stats.preempted_requests += n_preempt;
    t->stats.resumed_requests += n_resume;
    if (!og.empty() || !ig.empty()) t->stats.rotate_calls++;
    return KV_OK;
}

int32_t kv_req_preempt(kv_table_t *t, int64_t req) { return kv_req_rotate(t, &req, 1, nullptr, 0); }

int32_t kv_req_resume(kv_table_t *t, int64_t req) { return kv_req_rotate(t, nullptr, 0, &req, 1); }

int32_t kv_req_finish(kv_table_t *t, int64_t req)
{
    if (!t) return KV_ERR_INVALID_ARG;
    TReq *r = find(t, req);
    if (!r) return tfail(t, KV_ERR_INVALID_ARG, "unknown request");
    const TPending seq = now(t);                    // an eager copy or a swap-in of its blocks may still be in flight
    for (auto &b : r->blocks) {
        if (b.g >= 0) release_gpu(t, b.g, seq);
        if (b.h >= 0) t->host_free.give(b.h);
    }
    t->reqs.erase(req);
    auto it = std::find(t->order.begin(), t->order.end(), req);
    const size_t pos = (size_t)(it - t->order.begin());
    t->order.erase(it);
    if (t->eager_cursor > pos) t->eager_cursor--;
    if (!t->order.empty()) t->eager_cursor %= t->order.size();
    else t->eager_cursor = 0;
    return KV_OK;
}

int32_t kv_req_info(kv_table_t *t, int64_t req, kv_req_info_t *out)
{
    if (!t || !out) return KV_ERR_INVALID_ARG;
    TReq *r = find(t, req);
    if (!r) return tfail(t, KV_ERR_INVALID_ARG, "unknown request");
    memset(out, 0, sizeof(*out));
    out->tokens = r->tokens;
    out->num_blocks = (int64_t)r->blocks.size();
    out->on_gpu = r->on_gpu ? 1 : 0;
    for (size_t i = 0; i < r->blocks.size(); ++i) {
        if (r->blocks[i].host_valid) out->synced_blocks++;
        if (r->blocks[i].h >= 0) out->host_blocks++;
        if (!is_full(t, *r, i)) out->dirty_blocks++;
    }
    return KV_OK;
}

int32_t kv_req_blocks(kv_table_t *t, int64_t req, int32_t *gpu_ids, int32_t *host_ids, uint8_t *host_valid, int64_t cap)
{
    if (!t) return KV_ERR_INVALID_ARG;
    TReq *r = find(t, req);
    if (!r) return tfail(t, KV_ERR_INVALID_ARG, "unknown request");
    if (cap < (int64_t)r->blocks.size()) return tfail(t, KV_ERR_INVALID_ARG, "output arrays too short");
    for (size_t i = 0; i < r->blocks.size(); ++i) {
        if (gpu_ids) gpu_ids[i] = r->blocks[i].g;
        if (host_ids) host_ids[i] = r->blocks[i].h;
        if (host_valid) host_valid[i] = r->blocks[i].host_valid ? 1 : 0;
    }
    return KV_OK;
}

int32_t kv_table_fail_pool_call(kv_table_t *t, int64_t after_calls, int32_t code)
{
    if (!t || code >= 0) return KV_ERR_INVALID_ARG;
    t->fail_after = after_calls < 0 ? -1 : after_calls;
    t->fail_code = code;
    return KV_OK;
}

int32_t kv_table_get_stats(kv_table_t *t, kv_table_stats_t *out)
{
    if (!t || !out) return KV_ERR_INVALID_ARG;
    (void)reclaim(t, false);
    t->stats.free_gpu_blocks = gpu_available(t);
    t->stats.free_host_blocks = t->host_free.free_blocks();
    t->stats.free_host_extents = t->host_free.extents();
    t->stats.requests = (int64_t)t->reqs.size();
    *out = t->stats;
    return KV_OK;
}

}  // extern "C"
