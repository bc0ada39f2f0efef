/*
 * duplexkv.h -- C ABI of the B200 KV-block rotation engine.
 *
 * The operations are the data movement that the paper's DuplexKV rotation engine performs
 * (section 4.3, "Efficient Offloading and Memory Management"): a request's paged KV cache is
 * a set of fixed-size blocks scattered over a pool; rotating requests means copying the blocks
 * of some requests from GPU HBM to host DRAM (swap-out) and the blocks of others from host
 * DRAM into newly allocated HBM blocks (swap-in), with both directions in flight at once so
 * that the host link is used full-duplex.
 *
 * Layouts (elements are 16-bit words, never interpreted):
 *   device pool   [layer][K|V][block][block_size][kv_heads][head_dim]      ("layer-first", default), or
 *                 block-first like the host pool (KV_DEV_BLOCK_FIRST)
 *   host pool     [block][layer][K|V][block_size][kv_heads][head_dim]      ("block-first", default;
 *                 the paper's merged layout: all layers of one block contiguous), or layer-first
 *                 like the device pool.
 * SEG  = block_size*kv_heads*head_dim*2 bytes: one K or V plane of one block in one layer, the
 *        largest contiguous unit of the device layout.  SEG must be a multiple of 16.
 * BLK  = 2*num_layers*SEG bytes: one block over all layers.
 * Device byte offset of plane (l,kv) of block b: ((l*2+kv)*num_gpu_blocks + b)*SEG.
 * Host byte offset (block-first) of plane (l,kv) of block h: h*BLK + (l*2+kv)*SEG.
 *
 * Conventions
 *   - Every function returns a status (0 = KV_OK, negative = error); none throws, aborts or prints.
 *   - Id arrays are HOST pointers to int32 block ids; they are copied during the call.
 *   - Data-moving calls are asynchronous with respect to the device.  Swap-outs run in issue order on
 *     the pool's "out" stream, swap-ins on its "in" stream; a call is ordered after an earlier call of
 *     the other direction only when their lists touch the same block.  kv_sync waits for everything.
 *   - On any validation error nothing is launched and no byte moves.
 *   - One caller thread per pool.  There is no CPU fallback: every call needs the CUDA device.
 */
#ifndef DUPLEXKV_H_
#define DUPLEXKV_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* status codes */
#define KV_OK                 0
#define KV_ERR_INVALID_ARG   (-1)   /* null pointer, negative count, bad shape, count beyond pool size   */
#define KV_ERR_RANGE         (-2)   /* a block id outside [0, num_blocks) of its pool                    */
#define KV_ERR_DUP_DST       (-3)   /* the same destination block twice in one direction of one call     */
#define KV_ERR_HAZARD        (-4)   /* rotate lists overlap across directions and overlap is not allowed */
#define KV_ERR_CUDA          (-5)   /* a CUDA call failed; kv_last_error has the text                    */
#define KV_ERR_TIMEOUT       (-6)   /* a bounded device-side wait ran out (reported by kv_sync)          */
#define KV_ERR_NOMEM         (-7)   /* host or device allocation failed                                  */
#define KV_ERR_UNSUPPORTED   (-8)   /* combination not provided (e.g. SEG not a multiple of 16)          */

/* host pool layout */
#define KV_HOST_BLOCK_FIRST   0
#define KV_HOST_LAYER_FIRST   1

/* device pool layout */
#define KV_DEV_LAYER_FIRST    0     /* [layer][K|V][block]...: the layout the engine is built for        */
#define KV_DEV_BLOCK_FIRST    1     /* [block][layer][K|V]...: the paper's redesigned storage order      */

/* transfer paths (how the host link is driven) */
#define KV_PATH_AUTO          0     /* per call.  8 MiB or less per direction (blocks under 2 MiB: two blocks at most):
                                       CE2D, the lowest fixed cost.  Larger calls: STAGED when the
                                       copy-engine transfers the call needs would average 2.5 MiB or more,
                                       else ZEROCOPY (see kv_path_for)                                   */
#define KV_PATH_ZEROCOPY      1     /* SM kernels read/write mapped pinned host memory directly          */
#define KV_PATH_STAGED        2     /* pack kernel -> contiguous HBM staging -> copy engine (and reverse)*/
#define KV_PATH_CE2D          3     /* one strided 2-D copy-engine transfer per block, no kernel         */
#define KV_PATH_NAIVE         4     /* one copy-engine transfer per segment (the paper's "Naive" row)    */

/* flags */
#define KV_FLAG_ALLOW_OVERLAP   1   /* kv_rotate accepts lists that overlap across directions and orders
                                       the conflicting swap-ins after the swap-out                       */
#define KV_FLAG_LDST_KERNEL     2   /* ZEROCOPY/STAGED kernels use plain 16-byte loads/stores instead of
                                       bulk asynchronous copies through shared memory                    */
#define KV_FLAG_FUSED_ROTATE    4   /* ZEROCOPY kv_rotate with disjoint lists: one launch, CTAs split
                                       between the directions, on the out stream.  Without the flag this
                                       is done only for short lists (64 blocks or fewer each way) on an
                                       idle pool, where it saves a launch; longer ones use two streams   */
#define KV_FLAG_DEBUG_BOUNDS    16  /* the kernels compare every block id with its pool's size before they form an
                                       address from it; an id out of bounds is skipped (none of its bytes is
                                       touched), recorded in the status word, and kv_sync returns KV_ERR_RANGE.
                                       The host-side checks already refuse such ids before any launch; this
                                       guards the path from the id ring to the kernel (a debugging aid)   */
#define KV_FLAG_TIME_KERNELS    8   /* bracket every HBM-to-HBM gather / scatter kernel (STAGED pack / unpack,
                                       kv_gather_blocks, kv_scatter_blocks) with events on its own stream;
                                       kv_sync adds their durations to the timed_* statistics            */

typedef struct kv_pool kv_pool_t;   /* opaque; owned by the library */

typedef struct {
    int32_t num_layers, block_size, kv_heads, head_dim;   /* element = 2 bytes, fixed                     */
    int64_t num_gpu_blocks, num_host_blocks;
    void   *device_base;    /* DEVICE pointer, required: >= num_gpu_blocks*BLK bytes, 256-byte aligned;
                               borrowed (typically a torch tensor's storage)                              */
    void   *host_base;      /* HOST pointer or NULL.  NULL: the library allocates num_host_blocks*BLK
                               bytes of mapped pinned memory and owns it (an anonymous mapping that asks for
                               transparent huge pages, touched by several threads and then registered with
                               CUDA, which page-locks several times faster than cudaHostAlloc; cudaHostAlloc
                               when that fails, when the box has less than that much memory available, or
                               when the environment says DUPLEXKV_HOST_ALLOC=cuda).  Non-NULL: caller memory of that
                               size, 4096-byte aligned; the library page-locks it for the pool's lifetime.
                               Memory that is page-locked already (all of it: by cudaHostAlloc or
                               cudaHostRegister, or because it is the host memory of another pool) is
                               used as it is, which spares the seconds page-locking takes per 10 GB
                               when several pools of different shapes share one host buffer in turn     */
    int32_t host_layout;    /* KV_HOST_BLOCK_FIRST or KV_HOST_LAYER_FIRST                                 */
    int32_t device_id;
    void   *stream_out;     /* cudaStream_t or NULL (library creates a non-blocking stream)               */
    void   *stream_in;      /* likewise; must differ from stream_out for the directions to overlap        */
    int32_t path;           /* KV_PATH_* of the swap-out direction, and of swap-in unless path_in is set.
                               The environment overrides it: DUPLEXKV_PATH = auto | zerocopy | staged |
                               ce2d | naive (both directions); likewise DUPLEXKV_SMS_OUT / DUPLEXKV_SMS_IN
                               for ctas_out / ctas_in.  A value that does not parse fails the create       */
    int32_t flags;          /* KV_FLAG_*                                                                  */
    int32_t ctas_out;       /* CTAs of the zero-copy swap-out kernel, 0 = 64                              */
    int32_t ctas_in;        /* CTAs of the swap-in kernel, 0 = default                                    */
    int64_t staging_bytes;  /* per-direction HBM staging of the STAGED path (two halves used as a double
                               buffer, allocated at the first staged call); 0 = a sixteenth of the device
                               pool, but at most 2 GiB and at least 128 MiB (or the pool's own size if that
                               is smaller); never less than 2*BLK.  Larger halves mean fewer and longer
                               pack / unpack launches                                                     */
    int32_t path_in;        /* KV_PATH_* of the swap-in direction; KV_PATH_AUTO (0) = same as `path`      */
    int32_t ce_streams;     /* streams per direction that the copy-engine paths spread their transfers
                               over (1..4), 0 = 1                                                         */
    int32_t device_layout;  /* KV_DEV_LAYER_FIRST (default) or KV_DEV_BLOCK_FIRST: the variant of section
                               4.3.2 in which all layers of a device block are contiguous (a consumer of
                               the pool then strides by BLK between blocks).  kv_gather_blocks_static
                               reads layer-first pools only                                               */
    int32_t link_variant;   /* shape of the zero-copy kernels' transfers (a measurement knob; 0 is the default and
                               the quickest found): bulk kernel: 0 = 8 KiB copies, 8-stage ring; 1 = 32 KiB
                               copies, 4 stages; 2 = 64 KiB copies, 3 stages (segments of 4 KiB and less take
                               rings of their own size on several warps whatever the variant, see
                               kv_debug_ring_shape).  With KV_FLAG_LDST_KERNEL: 1 = 32-byte instead of
                               16-byte vectors per thread                                                 */
} kv_pool_config_t;

typedef struct {
    int64_t bytes_out, bytes_in;       /* payload bytes moved since the pool was created                  */
    int64_t calls_out, calls_in;       /* data-moving calls per direction                                 */
    int64_t kernel_launches;           /* kernels this library launched                                   */
    int64_t ce_copies;                 /* copy-engine transfers this library issued                       */
    double  last_out_ms, last_in_ms;   /* device time of the latest completed call per direction, from
                                          events on the launching streams.  Computed by kv_get_stats for
                                          the latest call a kv_sync has waited for: read the statistics
                                          after that kv_sync and before the next data-moving call          */
    double  last_union_ms;             /* first start to last end of the latest call (both directions
                                          for kv_rotate)                                                  */
    int32_t last_path_out, last_path_in;
    uint32_t device_status;            /* sticky bits written by kernels (0 = clean)                      */
    int32_t pad_;
    double  timed_kernel_ms;           /* KV_FLAG_TIME_KERNELS: summed device time of the timed kernels   */
    int64_t timed_kernel_bytes;        /* payload bytes those kernels moved (each read once, written once)*/
    int64_t timed_kernels;             /* how many launches the two sums cover                            */
    double  timed_kernel_exec_ms;      /* the same launches timed from inside: earliest CTA start to latest
                                          CTA end (%globaltimer), i.e. without the wait for the launch     */
    double  last_in_offset_ms;         /* latest kv_rotate: start of its swap-in window minus start of its
                                          swap-out window (with last_out_ms and last_in_ms: the timeline)  */
    int64_t requests_out, requests_in; /* requests that kv_rotate_req calls carried, per direction          */
} kv_stats_t;

typedef struct {
    double d2h_gbs, h2d_gbs;           /* each direction alone, GB/s (1e9 bytes per second)               */
    double bi_d2h_gbs, bi_h2d_gbs;     /* both at once: per-direction rates over the common window        */
    double bi_sum_gbs;                 /* both at once: total bytes / window                              */
    int64_t bytes; int32_t reps, pad_;
} kv_link_probe_t;

/*
 * Create a pool descriptor over caller device memory and (owned or borrowed) pinned host memory.
 * Sets the current device to cfg->device_id.  *out is NULL on failure.
 * Follows the paper's two-pool picture (HBM pool and DRAM swap space, section 5.1 set-up).
 */
int32_t kv_pool_create(const kv_pool_config_t *cfg, kv_pool_t **out);

/* Waits for all outstanding work, then frees what the library owns (never device_base, never a
 * caller-supplied host_base, never caller streams). */
int32_t kv_pool_destroy(kv_pool_t *pool);

/*
 * Swap-out (section 4.3: copy every segment of each listed HBM block to its DRAM block).
 * For i < n, every layer l and plane kv: host block host_ids[i] plane (l,kv) <- device block
 * gpu_ids[i] plane (l,kv).  The device pool is not modified.  host_ids must be unique
 * (KV_ERR_DUP_DST); gpu_ids may repeat.  n == 0 is a no-op.  Asynchronous.
 */
int32_t kv_swap_out(kv_pool_t *pool, const int32_t *gpu_ids, const int32_t *host_ids, int64_t n);

/*
 * Swap-in (section 4.3: copy every segment of each listed DRAM block into a newly allocated HBM
 * block).  For j < n: device block gpu_ids[j] <- host block host_ids[j], all planes.  The host pool
 * is not modified.  gpu_ids must be unique; host_ids may repeat.  Asynchronous.
 */
int32_t kv_swap_in(kv_pool_t *pool, const int32_t *host_ids, const int32_t *gpu_ids, int64_t n);

/*
 * Rotation: swap-out of (out_gpu -> out_host) and swap-in of (in_host -> in_gpu) in one call, both
 * directions in flight together.  The result is defined as swap-out THEN swap-in.  When a swap-in
 * destination is a swap-out source, or a swap-in source is a swap-out destination (the data race of
 * the paper's eager-block-rotation discussion), the call fails with KV_ERR_HAZARD and moves nothing,
 * unless the pool was created with KV_FLAG_ALLOW_OVERLAP: then the conflicting swap-in pairs are
 * issued after the swap-out completes and the rest still overlap.  Asynchronous.
 */
int32_t kv_rotate(kv_pool_t *pool,
                  const int32_t *out_gpu, const int32_t *out_host, int64_t n_out,
                  const int32_t *in_host, const int32_t *in_gpu, int64_t n_in);

/*
 * kv_rotate with the request boundaries of its lists, for per-request statistics only: request r of the
 * swap-out owns list entries out_req_offsets[r] .. out_req_offsets[r+1]-1 (HOST arrays of n_out_req + 1
 * and n_in_req + 1 non-decreasing offsets, first 0, last n_out / n_in; a direction without blocks takes
 * NULL and 0).  Moves exactly what kv_rotate would and adds the request counts to the statistics, so that
 * time and bytes per request can be had from kv_get_stats.  Bad offsets: KV_ERR_INVALID_ARG, nothing
 * moves.  (The paper rotates whole requests, section 4.2; a request is a contiguous run of the lists.)
 */
int32_t kv_rotate_req(kv_pool_t *pool,
                      const int32_t *out_gpu, const int32_t *out_host, int64_t n_out,
                      const int64_t *out_req_offsets, int64_t n_out_req,
                      const int32_t *in_host, const int32_t *in_gpu, int64_t n_in,
                      const int64_t *in_req_offsets, int64_t n_in_req);

/*
 * What copy-engine transfers the STAGED path would make for one direction of a call (no pool, no GPU).
 * Where the host ids form long runs (8 blocks and more on average) the list is taken in ascending order
 * of host id, each run is one transfer and equal runs at a constant spacing share one strided transfer.
 * Otherwise every block counts as a single: four blocks (of less than 4 MiB) whose ids form a 2 x 2
 * lattice (a, a+g, a+kg, a+kg+g) share one 3-D transfer, the blocks left over travel two per transfer
 * (neighbours in ascending order, any distance apart in host memory), lattices first; blocks of 4 MiB and
 * more travel two per transfer throughout -- transfers of few sizes keep the two copy
 * engines of a rotation in step (section 4.3.2's "merge small segments into large transfers", bounded
 * here by what the ids allow).  The sequence is cut into chunks of at most half_blocks blocks (one
 * staging half each; about four chunks for a call that would fit one half, a single chunk for a call of
 * 128 MiB or less).
 *   host_ids   HOST array of n host block ids (direction 0: swap-out destinations, 1: swap-in sources)
 *   ops        HOST array of ops_cap entries, filled in issue order; *n_ops = transfers needed
 *              (with ops_cap == 0 only the count is returned)
 *   order      HOST array of n entries or NULL: order[k] = index in host_ids of the block that takes
 *              staging position k (the staging order: the blocks of each transfer side by side, transfers
 *              in issue order)
 * A transfer moves slices x rows x blocks_per_row blocks: row r of slice s covers host blocks
 * host_block + s*slice_pitch_blocks + r*pitch_blocks .. + blocks_per_row - 1, and the transfer's blocks
 * take staging positions first_position .. in (slice, row, block) order.
 */
typedef struct {
    int64_t host_block, first_position, pitch_blocks;
    int32_t rows, blocks_per_row, chunk, slices;
    int64_t slice_pitch_blocks;
} kv_plan_op_t;
int32_t kv_plan_staged(int64_t blk_bytes, int64_t half_blocks, int32_t direction, const int32_t *host_ids, int64_t n,
                       kv_plan_op_t *ops, int64_t ops_cap, int64_t *n_ops, int32_t *order);

/* Wait for outstanding work, then change the transfer path of each direction (KV_PATH_*; AUTO
 * re-applies the rule of kv_path_for).  Pool contents are unaffected. */
int32_t kv_pool_set_path(kv_pool_t *pool, int32_t path_out, int32_t path_in);

/* Waits for outstanding work, then switches the per-call timing on (default) or off.  Off: calls record no
 * start events and the last_* statistics stay as they are, which takes a few microseconds off every call;
 * for callers that rotate single requests and time them with their own clock.  (Tuning of this library.) */
int32_t kv_pool_set_call_timing(kv_pool_t *pool, int32_t on);

/*
 * Bound of the waits inside the copy kernels (each wait of a kernel's main loop for a load it has
 * issued): `polls` immediate polls, then polls 200 ns apart for at most `ns` nanoseconds (default 16 and
 * 2 s; ns <= 60 s).  A wait that runs out makes its CTA record KV_DEV_TIMEOUT in the pool's status word,
 * wait (with the default bound) for the loads it still has in flight, drain its stores and return; the
 * bytes it had left are not moved, kv_sync reports KV_ERR_TIMEOUT and the pool stays in that state.
 * polls == 0 and ns == 0 make every such wait give up without looking, which is how the failure path is
 * exercised on a healthy GPU without a fault or a hang.  Applies to calls issued afterwards.  (Failure
 * handling of this library; the paper describes none.)
 */
int32_t kv_pool_set_wait_limit(kv_pool_t *pool, uint32_t polls, uint64_t ns);

/* Wait for both directions.  Returns KV_OK, or the first sticky asynchronous error
 * (KV_ERR_CUDA, KV_ERR_TIMEOUT).  The last_* timing fields describe the call it waited for once
 * kv_get_stats is called. */
int32_t kv_sync(kv_pool_t *pool);

/*
 * Device-side gather / scatter (the kernel half of the STAGED path, also usable on its own):
 * gather copies the listed device blocks, in list order, into a contiguous DEVICE buffer laid out
 * block-first (block i at i*BLK, planes in (layer, K|V) order); scatter is the inverse.  dst/src must
 * hold n*BLK bytes and be 16-byte aligned.  Runs on the out (gather) / in (scatter) stream and is
 * ordered like a call of that direction: a gather waits for an unfinished swap-in (or scatter) that
 * writes one of its blocks, a scatter for an unfinished swap-out (or gather) that reads one of its
 * blocks, and later calls of the other direction wait for it in the same way.  The buffer itself is
 * the caller's: nothing orders other work on dst_device / src_device.
 * This is the "merge small segments into large contiguous regions" step of section 4.3, done by
 * a kernel instead of a layout change.
 */
int32_t kv_gather_blocks(kv_pool_t *pool, const int32_t *gpu_ids, int64_t n, void *dst_device);
int32_t kv_scatter_blocks(kv_pool_t *pool, const void *src_device, const int32_t *gpu_ids, int64_t n);

/*
 * kv_gather_blocks for callers that cannot allocate.  (The paper has no counterpart: its engine
 * allocates freely.  This exists for users of this library.)
 *
 * Who that is: code that runs where a cudaMalloc is off limits -- inside a serving loop that must
 * not take the device-wide synchronisation an allocation or a free implies, in a process whose
 * whole GPU memory already belongs to another allocator, or in a component that is handed its
 * buffers and may not create any.  A pool (kv_pool_create) allocates descriptor rings, events and
 * staging, so such callers cannot hold one; this entry point needs none.
 *
 * Same result as kv_gather_blocks: the listed blocks of the layer-first pool at device_base
 * (num_gpu_blocks blocks of the given shape) are written, in list order, to dst_device block-first
 * (block i at i*BLK, planes in (layer, K|V) order).  device_base, dst_device: DEVICE pointers on the
 * CURRENT device, 16-byte aligned, dst_device holding n*BLK bytes.  gpu_ids: HOST pointer, ids may
 * repeat.  stream: a cudaStream_t of the current device, or NULL for the default stream.
 *
 * The id list the kernel walks and the kernel's status word sit in an array built into the library
 * (KV_STATIC_MAX_BLOCKS ids, 64.25 KiB of device memory on every GPU that loads the library, held
 * until the process exits).  n > KV_STATIC_MAX_BLOCKS is refused with KV_ERR_INVALID_ARG and a
 * message in kv_last_error(NULL); split longer lists.  The call makes no cudaMalloc, cudaFree,
 * cudaHostAlloc or stream / event creation.  It is SYNCHRONOUS: it returns when the gather has
 * finished (KV_OK), or with KV_ERR_RANGE / KV_ERR_INVALID_ARG / KV_ERR_UNSUPPORTED before anything
 * ran, or KV_ERR_CUDA / KV_ERR_TIMEOUT.
 *
 * The first call on each device looks up the array's device address and sets the kernel's
 * shared-memory limit for that device; make that first call before starting any stream capture.
 * All calls share the one array, which still holds the previous call's ids (they are overwritten,
 * and the status word is cleared, at the start of each call): two calls that overlap in time -- from
 * two threads, or on two streams -- race on it, also across different pools or shapes.  One call at
 * a time per device.
 */
#define KV_STATIC_MAX_BLOCKS 8192
int32_t kv_gather_blocks_static(const void *device_base, int32_t num_layers, int32_t block_size,
                                int32_t kv_heads, int32_t head_dim, int64_t num_gpu_blocks,
                                const int32_t *gpu_ids, int64_t n, void *dst_device, void *stream);

/* Host pool base (HOST pointer) and size, for filling and verification. */
int32_t kv_host_ptr(kv_pool_t *pool, void **base, int64_t *bytes);

int32_t kv_get_stats(kv_pool_t *pool, kv_stats_t *stats);

/* Text of the latest error on this pool (never NULL; static storage inside the pool).
 * With pool == NULL: the text of the latest kv_pool_create / kv_probe_link failure. */
const char *kv_last_error(kv_pool_t *pool);

/* SEG and BLK for a shape (bytes); 0 if the shape is invalid. */
int64_t kv_seg_bytes(int32_t block_size, int32_t kv_heads, int32_t head_dim);
int64_t kv_blk_bytes(int32_t num_layers, int32_t block_size, int32_t kv_heads, int32_t head_dim);

/* The path KV_PATH_AUTO resolves to for a large call of blocks of blk_bytes (= kv_blk_bytes of the shape) in
 * the worst case for the copy engines: host ids with no neighbours and no lattices in the list, so that
 * the blocks travel two per transfer.  Lists whose ids form runs or lattices make larger transfers and
 * go STAGED at smaller block sizes too; AUTO decides that per call from the transfers it plans. */
int32_t kv_path_for(int64_t blk_bytes);

/*
 * Host-link roofline probe (the analogue of the paper's appendix B bandwidth measurement, done
 * with plain pinned copy-engine transfers): times `reps` copies of `bytes` device->host, host->device,
 * and both at once on two streams; best of three rounds after one warm-up.  Allocates and frees
 * its own pinned and device buffers.
 */
int32_t kv_probe_link(int32_t device_id, int64_t bytes, int32_t reps, kv_link_probe_t *out);

/*
 * The same probe with the shape of the transfers as parameters: the bandwidth-versus-transfer-size
 * curve of the paper's motivation study (the figure of section 3.3 on full-duplex bandwidth against
 * segment size, and the launch-versus-transfer-time figure of section 4.3.1).  Each round issues
 * total_bytes/copy_bytes copy-engine transfers of copy_bytes back to back on one stream per direction.
 * rows <= 1: plain transfers.  rows > 1: strided 2-D transfers of `rows` rows of copy_bytes/rows bytes,
 * row r at start + r*host_pitch on the host and start + r*dev_pitch on the device (0 = rows packed).
 * slices > 1 (with rows > 1): 3-D transfers of `slices` x `rows` rows; on the host slice s starts
 * s*host_slice_rows*host_pitch after the first (host_slice_rows >= rows), on the device rows and slices are
 * packed at dev_pitch.  That is how four blocks on a 2 x 2 lattice of host addresses travel in one transfer.
 * The transfers start at consecutive places of span_bytes-sized buffers (wrapping), or at seeded
 * pseudo-random row-aligned offsets when scattered != 0.  One warm-up round, then `rounds` timed
 * ones; the best is kept.  out->bytes = copy_bytes, out->reps = transfers per round.
 */
typedef struct {
    int64_t copy_bytes, total_bytes, span_bytes;
    int32_t scattered, rounds;
    int64_t rows, host_pitch, dev_pitch;
    int64_t slices, host_slice_rows;
} kv_probe_spec_t;
int32_t kv_probe_link_ex(int32_t device_id, const kv_probe_spec_t *spec, kv_link_probe_t *out);

/* Shape of a pool (what kv_pool_create was given). */
typedef struct {
    int32_t num_layers, block_size, kv_heads, head_dim;
    int64_t num_gpu_blocks, num_host_blocks, seg_bytes, blk_bytes;
} kv_pool_shape_t;
int32_t kv_pool_shape(kv_pool_t *pool, kv_pool_shape_t *out);

/*
 * Make `stream` (a cudaStream_t of the pool's device; NULL = the default stream) wait, on the device and
 * without blocking the host, for everything issued so far in the given directions (bit 0 = swap-outs,
 * bit 1 = swap-ins; 3 = both).  This is how a compute stream picks up swapped-in blocks, or holds back
 * writes to blocks a swap-out still reads, in the paper's cross-iteration pipeline (section 4.3.2), where
 * rotation runs beside model execution and nobody wants a host-side kv_sync.
 */
int32_t kv_stream_wait(kv_pool_t *pool, void *stream, int32_t directions);

/*
 * The event that completes with the latest call issued so far in `direction` (0 = swap-outs, 1 = swap-ins):
 * *event receives a cudaEvent_t owned by the pool, or NULL when the direction has seen no call yet.  It
 * stays that call's event until eight further calls of the direction have been issued, and dies with the
 * pool.  For cudaStreamWaitEvent / cudaEventQuery / cudaEventSynchronize by whoever schedules the model's
 * kernels: the completion signal of the paper's cross-iteration pipeline (section 4.3.2), where iteration
 * t computes while the transfers of t+1 are in flight.  kv_stream_wait is the same thing done in one call.
 */
int32_t kv_completion_event(kv_pool_t *pool, int32_t direction, void **event);

/* Waits for outstanding work, then sets the CTAs of the zero-copy kernels per direction (0 = the default,
 * 64).  How many SMs a rotation may occupy beside model execution is a sizing decision of the caller. */
int32_t kv_pool_set_ctas(kv_pool_t *pool, int32_t ctas_out, int32_t ctas_in);

/* Which shape of the bulk-copy kernel a launch takes for segments of segment_bytes (host logic, no device
 * needed): the bytes of one work item, and the ring each issuing warp runs -- stage size, stages, loads
 * ahead of the stores -- and the issuing warps per CTA.  over_link = 0: HBM to HBM (pack, unpack, gather,
 * scatter); 1: the zero-copy kernels, with the pool's link_variant.  An item never exceeds a stage, and a
 * CTA uses stage_bytes * stages * warps bytes of dynamic shared memory (at most 227 KiB).  Any out pointer
 * may be NULL.  KV_ERR_INVALID_ARG for a segment size that is not a positive multiple of 16 or an unknown
 * variant. */
int32_t kv_debug_ring_shape(int64_t segment_bytes, int32_t over_link, int32_t link_variant, int32_t *item_bytes,
                            int32_t *stage_bytes, int32_t *stages, int32_t *ahead, int32_t *warps);

/* The predicate behind KV_FLAG_DEBUG_BOUNDS as a host function: 1 when both ids lie inside their pools. */
int32_t kv_debug_pair_in_bounds(int32_t src_id, int32_t dst_id, int32_t src_blocks, int32_t dst_blocks);

/* Calls issued and calls known to have completed, per direction (a non-blocking look at the pool's
 * end events).  Any pointer may be NULL.  kv_gather_blocks / kv_scatter_blocks count as calls of the
 * out / in direction. */
int32_t kv_pool_progress(kv_pool_t *pool, int64_t *out_issued, int64_t *out_done, int64_t *in_issued, int64_t *in_done);

/* ------------------------------------------------------------------------------------------------
 * Block table with eager block rotation (section 4.3.2, "Eager block rotation for data race free
 * overlapping", and the block table of the architecture figure in section 4.1).
 *
 * The table owns the free lists of both pools and, per request, the device block, host block and
 * state of every block.  A block that is completely filled never changes again; once it has a copy
 * in host memory it is "synced".  kv_eager_rotate copies full blocks to host memory in the
 * background; kv_req_rotate preempts and resumes whole requests with ONE kv_rotate on the pool,
 * moving out only the blocks that have no valid host copy (normally the single, partly filled
 * "dirty" block) and releasing the others' device blocks without any transfer, so that the requests
 * resuming in the same call can take them: the swap-in never depends on the swap-out.  Host copies
 * are kept while a request runs on the GPU.  Host blocks are handed out in runs, so blocks sent
 * together are neighbours in host memory and travel as few, long transfers.
 *
 * All calls return a status like the pool's; data movement is asynchronous (kv_sync on the pool
 * waits for it).  One caller thread.  The table does not write KV data: whoever runs the model
 * writes tokens into the device blocks kv_req_blocks reports.  Device blocks handed out by kv_req_add
 * and kv_req_append are never still being read by a swap-out (blocks released at a preemption are
 * held back until the copies that may read them have finished; the call waits for the pool if it
 * must), so the caller may write into them at once.  A host block released by kv_req_finish, and the
 * host pool in general, is only ever written by the pool's own swap-outs, which the pool orders.
 * Request ids are arbitrary int64 values chosen by the caller.
 */
typedef struct kv_table kv_table_t;

typedef struct {
    int64_t tokens, num_blocks;
    int64_t synced_blocks;      /* blocks whose host copy is valid                                   */
    int64_t host_blocks;        /* blocks that own a host block (valid or stale)                     */
    int64_t dirty_blocks;       /* partly filled blocks: 0 or 1 (the last one)                        */
    int32_t on_gpu, pad_;       /* 1 = runs on the GPU, 0 = preempted (lives in host memory)          */
} kv_req_info_t;

typedef struct {
    int64_t eager_blocks, eager_calls;          /* blocks copied out in the background, calls that did */
    int64_t preempt_blocks_moved;               /* blocks copied out at preemption time                */
    int64_t discarded_blocks;                   /* device blocks released at preemption without a copy */
    int64_t resume_blocks_moved;                /* blocks copied in at resume time                     */
    int64_t preempted_requests, resumed_requests, rotate_calls;
    int64_t free_gpu_blocks, free_host_blocks, free_host_extents, requests;
} kv_table_stats_t;

/* A table over `pool` (borrowed; destroy the table first).  Every block of both pools starts free. */
int32_t kv_table_create(kv_pool_t *pool, kv_table_t **out);
/* The same bookkeeping with no pool behind it: nothing is moved.  For planning and for testing the
 * allocator and the state machine on a machine without a GPU. */
int32_t kv_table_create_dry(int64_t num_gpu_blocks, int64_t num_host_blocks, int32_t block_size, kv_table_t **out);
int32_t kv_table_destroy(kv_table_t *table);
const char *kv_table_last_error(kv_table_t *table);

/* New request on the GPU whose first `tokens` tokens are about to be written (prefill): takes
 * ceil(tokens/block_size) device blocks.  KV_ERR_NOMEM (nothing changed) when they are not free. */
int32_t kv_req_add(kv_table_t *table, int64_t req, int64_t tokens);
/* `new_tokens` more tokens for a request on the GPU (decode): they go into the partly filled last
 * block first (its host copy, if any, becomes stale), then into newly taken device blocks. */
int32_t kv_req_append(kv_table_t *table, int64_t req, int64_t new_tokens);
/* Background step: copy up to max_blocks full blocks that have no valid host copy to host memory
 * (requests in arrival order, round robin across calls) with one kv_swap_out, and mark them synced.
 * *n_issued (may be NULL) = blocks sent.  Sends fewer when the host pool runs out.  If the pool refuses
 * the copy, the pool's status is returned and the table is as it was before the call. */
int32_t kv_eager_rotate(kv_table_t *table, int64_t max_blocks, int64_t *n_issued);
/* Preempt the listed requests (HOST array of ids; must be on the GPU) and resume the listed ones
 * (must be preempted) in one full-duplex kv_rotate.  All or nothing: KV_ERR_NOMEM / KV_ERR_INVALID_ARG,
 * and any status with which the pool refuses the rotation, leave the table unchanged. */
int32_t kv_req_rotate(kv_table_t *table, const int64_t *preempt, int64_t n_preempt,
                      const int64_t *resume, int64_t n_resume);
int32_t kv_req_preempt(kv_table_t *table, int64_t req);
int32_t kv_req_resume(kv_table_t *table, int64_t req);
/* The request is done: all its device and host blocks become free. */
int32_t kv_req_finish(kv_table_t *table, int64_t req);

int32_t kv_req_info(kv_table_t *table, int64_t req, kv_req_info_t *out);
/* Per block, in logical order: device id (-1 = none), host id (-1 = none), whether the host copy is
 * valid.  Output arrays are HOST memory of at least `cap` >= num_blocks entries; any may be NULL. */
int32_t kv_req_blocks(kv_table_t *table, int64_t req, int32_t *gpu_ids, int32_t *host_ids,
                      uint8_t *host_valid, int64_t cap);
int32_t kv_table_get_stats(kv_table_t *table, kv_table_stats_t *out);
/* Fault injection for tests, on the host only: the pool call the table makes after `after_calls` further
 * ones (0 = the very next kv_swap_out / kv_rotate it would issue) is not made and counts as having
 * returned `code` (a negative KV_ERR_*); later calls go through again.  after_calls < 0 disarms.  Works on
 * a dry table too.  Nothing is sent to the device, so no transfer is ever half done.  (The paper has no
 * counterpart; this is how the all-or-nothing promise of kv_req_rotate and kv_eager_rotate is tested.) */
int32_t kv_table_fail_pool_call(kv_table_t *table, int64_t after_calls, int32_t code);

#ifdef __cplusplus
}
#endif
#endif /* DUPLEXKV_H_ */
