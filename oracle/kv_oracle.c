/*
 * kv_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * Plain, slow, single-purpose CPU model of what the DuplexKV rotation engine
 * moves (paper section 4.3: "Efficient Offloading and Memory Management",
 * the segment / virtual-tensor model, the layer-first and block-first stride
 * formulas, and the swap-in / swap-out dependency discussion).
 *
 * Only tests, the smoke check and the bench's cpu_baseline / reference arm may
 * build or call this file.  It shares no code with the CUDA library: the
 * address formulas below are written out here on their own.
 *
 * State = two byte arrays:
 *   G   device-pool model, layer-first   [layer][K|V][block][bs][kv_heads][head_dim] 16-bit words
 *   Hs  host-pool model,   block-first   [block][layer][K|V][bs][kv_heads][head_dim]
 *       (or layer-first like G when host_layout == 1)
 *
 * A "segment" here is the largest contiguous run under the layer-first layout:
 * one K or V plane of one block in one layer, SEG = bs * kv_heads * head_dim * 2 bytes.
 * (The paper's S_seg = P x C counts K and V together; with K|V outside the block
 * index the contiguous unit is half of that.)
 *
 * Semantics (exact; the method is a permutation copy, no approximation):
 *   swap_out : for every pair (g_i, h_i), layer l, plane kv:  seg(Hs,l,kv,h_i) <- seg(G,l,kv,g_i);  G unchanged
 *   swap_in  : for every pair (h_j, g_j), layer l, plane kv:  seg(G,l,kv,g_j)  <- seg(Hs,l,kv,h_j); Hs unchanged
 *   rotate   : swap_out(out lists) THEN swap_in(in lists)   (sequential definition)
 * A call whose lists fail validation changes nothing.
 */
#define _POSIX_C_SOURCE 200809L
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#include <pthread.h>

typedef struct {
    int32_t num_layers;
    int32_t block_size;
    int32_t kv_heads;
    int32_t head_dim;
    int64_t num_gpu_blocks;
    int64_t num_host_blocks;
    int32_t host_layout; /* 0 = block-first, 1 = layer-first */
    int32_t dev_layout;  /* 0 = layer-first, 1 = block-first (the paper's redesigned storage order) */
} kvo_shape_t;

enum {
    KVO_OK = 0,
    KVO_ERR_INVALID_ARG = -1,
    KVO_ERR_RANGE = -2,
    KVO_ERR_DUP_DST = -3,
    KVO_ERR_HAZARD = -4
};

/* bytes of one K-or-V plane of one block in one layer */
int64_t kvo_seg_bytes(const kvo_shape_t *s)
{
    return (int64_t)s->block_size * s->kv_heads * s->head_dim * 2;
}

/* bytes of one block over all layers and both planes */
int64_t kvo_blk_bytes(const kvo_shape_t *s)
{
    return 2 * (int64_t)s->num_layers * kvo_seg_bytes(s);
}

/* layer-first: inside one (layer, plane) consecutive blocks are SEG apart;
 * block-first: all planes of a block are contiguous and consecutive blocks are one whole block apart
 * (section 4.3.2: the stride between block i and block j grows from (j-i)*S_seg to (j-i)*N_L*S_seg) */
int64_t kvo_dev_off(const kvo_shape_t *s, int64_t l, int64_t kv, int64_t b)
{
    int64_t plane = l * 2 + kv;
    if (s->dev_layout == 1)
        return b * kvo_blk_bytes(s) + plane * kvo_seg_bytes(s);
    return (plane * s->num_gpu_blocks + b) * kvo_seg_bytes(s);
}

/* block-first: consecutive blocks are N_L * S_seg apart, i.e. one whole block */
int64_t kvo_host_off(const kvo_shape_t *s, int64_t h, int64_t l, int64_t kv)
{
    int64_t plane = l * 2 + kv;
    if (s->host_layout == 1)
        return (plane * s->num_host_blocks + h) * kvo_seg_bytes(s);
    return h * kvo_blk_bytes(s) + plane * kvo_seg_bytes(s);
}

static int ids_in_range(const int32_t *ids, int64_t n, int64_t nb)
{
    for (int64_t i = 0; i < n; i++)
        if (ids[i] < 0 || (int64_t)ids[i] >= nb)
            return 0;
    return 1;
}

/* quadratic on purpose: obviously right, lists are short in the tests that use it */
static int has_dup(const int32_t *ids, int64_t n)
{
    for (int64_t i = 0; i < n; i++)
        for (int64_t j = i + 1; j < n; j++)
            if (ids[i] == ids[j])
                return 1;
    return 0;
}

static int intersects(const int32_t *a, int64_t na, const int32_t *b, int64_t nb)
{
    for (int64_t i = 0; i < na; i++)
        for (int64_t j = 0; j < nb; j++)
            if (a[i] == b[j])
                return 1;
    return 0;
}

/* validation of one direction: ranges, then duplicate destinations */
int32_t kvo_check_out(const kvo_shape_t *s, const int32_t *gpu_ids, const int32_t *host_ids, int64_t n)
{
    if (n < 0 || (n > 0 && (!gpu_ids || !host_ids)))
        return KVO_ERR_INVALID_ARG;
    if (!ids_in_range(gpu_ids, n, s->num_gpu_blocks) || !ids_in_range(host_ids, n, s->num_host_blocks))
        return KVO_ERR_RANGE;
    if (has_dup(host_ids, n))
        return KVO_ERR_DUP_DST;
    return KVO_OK;
}

int32_t kvo_check_in(const kvo_shape_t *s, const int32_t *host_ids, const int32_t *gpu_ids, int64_t n)
{
    if (n < 0 || (n > 0 && (!gpu_ids || !host_ids)))
        return KVO_ERR_INVALID_ARG;
    if (!ids_in_range(gpu_ids, n, s->num_gpu_blocks) || !ids_in_range(host_ids, n, s->num_host_blocks))
        return KVO_ERR_RANGE;
    if (has_dup(gpu_ids, n))
        return KVO_ERR_DUP_DST;
    return KVO_OK;
}

/*
 * The race of the paper's data-race figure: a swap-in destination that is a
 * swap-out source (device side), or a swap-in source that is a swap-out
 * destination (host side), makes the two directions order-dependent.
 */
int32_t kvo_check_rotate(const kvo_shape_t *s,
                         const int32_t *out_gpu, const int32_t *out_host, int64_t n_out,
                         const int32_t *in_host, const int32_t *in_gpu, int64_t n_in,
                         int32_t allow_overlap)
{
    int32_t rc = kvo_check_out(s, out_gpu, out_host, n_out);
    if (rc != KVO_OK)
        return rc;
    rc = kvo_check_in(s, in_host, in_gpu, n_in);
    if (rc != KVO_OK)
        return rc;
    if (!allow_overlap) {
        if (intersects(in_gpu, n_in, out_gpu, n_out) || intersects(in_host, n_in, out_host, n_out))
            return KVO_ERR_HAZARD;
    }
    return KVO_OK;
}

static void out_pairs(const kvo_shape_t *s, const uint8_t *G, uint8_t *Hs,
                      const int32_t *gpu_ids, const int32_t *host_ids, int64_t lo, int64_t hi)
{
    int64_t seg = kvo_seg_bytes(s);
    for (int64_t i = lo; i < hi; i++)
        for (int64_t l = 0; l < s->num_layers; l++)
            for (int64_t kv = 0; kv < 2; kv++)
                memcpy(Hs + kvo_host_off(s, host_ids[i], l, kv),
                       G + kvo_dev_off(s, l, kv, gpu_ids[i]), (size_t)seg);
}

static void in_pairs(const kvo_shape_t *s, uint8_t *G, const uint8_t *Hs,
                     const int32_t *host_ids, const int32_t *gpu_ids, int64_t lo, int64_t hi)
{
    int64_t seg = kvo_seg_bytes(s);
    for (int64_t j = lo; j < hi; j++)
        for (int64_t l = 0; l < s->num_layers; l++)
            for (int64_t kv = 0; kv < 2; kv++)
                memcpy(G + kvo_dev_off(s, l, kv, gpu_ids[j]),
                       Hs + kvo_host_off(s, host_ids[j], l, kv), (size_t)seg);
}

int32_t kvo_swap_out(const kvo_shape_t *s, const uint8_t *G, uint8_t *Hs,
                     const int32_t *gpu_ids, const int32_t *host_ids, int64_t n)
{
    int32_t rc = kvo_check_out(s, gpu_ids, host_ids, n);
    if (rc != KVO_OK)
        return rc;
    out_pairs(s, G, Hs, gpu_ids, host_ids, 0, n);
    return KVO_OK;
}

int32_t kvo_swap_in(const kvo_shape_t *s, uint8_t *G, const uint8_t *Hs,
                    const int32_t *host_ids, const int32_t *gpu_ids, int64_t n)
{
    int32_t rc = kvo_check_in(s, host_ids, gpu_ids, n);
    if (rc != KVO_OK)
        return rc;
    in_pairs(s, G, Hs, host_ids, gpu_ids, 0, n);
    return KVO_OK;
}

int32_t kvo_rotate(const kvo_shape_t *s, uint8_t *G, uint8_t *Hs,
                   const int32_t *out_gpu, const int32_t *out_host, int64_t n_out,
                   const int32_t *in_host, const int32_t *in_gpu, int64_t n_in,
                   int32_t allow_overlap)
{
    int32_t rc = kvo_check_rotate(s, out_gpu, out_host, n_out, in_host, in_gpu, n_in, allow_overlap);
    if (rc != KVO_OK)
        return rc;
    out_pairs(s, G, Hs, out_gpu, out_host, 0, n_out);
    in_pairs(s, G, Hs, in_host, in_gpu, 0, n_in);
    return KVO_OK;
}

/*
 * Same rotate, pairs split over host threads in disjoint contiguous ranges:
 * every thread finishes its share of the swap-out, all threads meet at a
 * barrier, then every thread does its share of the swap-in.  With unique
 * destinations inside each direction the ranges never write the same bytes,
 * so the result equals kvo_rotate.  Used only to time the oracle on all cores.
 */
typedef struct {
    const kvo_shape_t *s;
    uint8_t *G, *Hs;
    const int32_t *out_gpu, *out_host, *in_host, *in_gpu;
    int64_t out_lo, out_hi, in_lo, in_hi;
    pthread_barrier_t *bar;
} kvo_job_t;

static void *rotate_worker(void *p)
{
    kvo_job_t *j = (kvo_job_t *)p;
    out_pairs(j->s, j->G, j->Hs, j->out_gpu, j->out_host, j->out_lo, j->out_hi);
    pthread_barrier_wait(j->bar);
    in_pairs(j->s, j->G, j->Hs, j->in_host, j->in_gpu, j->in_lo, j->in_hi);
    return NULL;
}

int32_t kvo_rotate_mt(const kvo_shape_t *s, uint8_t *G, uint8_t *Hs,
                      const int32_t *out_gpu, const int32_t *out_host, int64_t n_out,
                      const int32_t *in_host, const int32_t *in_gpu, int64_t n_in,
                      int32_t allow_overlap, int32_t threads)
{
    int32_t rc = kvo_check_rotate(s, out_gpu, out_host, n_out, in_host, in_gpu, n_in, allow_overlap);
    if (rc != KVO_OK)
        return rc;
    if (threads < 1)
        return KVO_ERR_INVALID_ARG;
    pthread_t *tid = (pthread_t *)malloc(sizeof(pthread_t) * (size_t)threads);
    kvo_job_t *job = (kvo_job_t *)malloc(sizeof(kvo_job_t) * (size_t)threads);
    pthread_barrier_t bar;
    if (!tid || !job) {
        free(tid);
        free(job);
        return KVO_ERR_INVALID_ARG;
    }
    pthread_barrier_init(&bar, NULL, (unsigned)threads);
    for (int32_t t = 0; t < threads; t++) {
        job[t].s = s;
        job[t].G = G;
        job[t].Hs = Hs;
        job[t].out_gpu = out_gpu;
        job[t].out_host = out_host;
        job[t].in_host = in_host;
        job[t].in_gpu = in_gpu;
        job[t].out_lo = n_out * t / threads;
        job[t].out_hi = n_out * (t + 1) / threads;
        job[t].in_lo = n_in * t / threads;
        job[t].in_hi = n_in * (t + 1) / threads;
        job[t].bar = &bar;
        pthread_create(&tid[t], NULL, rotate_worker, &job[t]);
    }
    for (int32_t t = 0; t < threads; t++)
        pthread_join(tid[t], NULL);
    pthread_barrier_destroy(&bar);
    free(tid);
    free(job);
    return KVO_OK;
}
