/*
 * enl.h -- C ABI of the selective-KV attention library for navigation-map memory (B200, sm_100a).
 *
 * The paper (EfficientNav, arXiv 2510.18546) states the problem this boundary follows:
 *   - Sec. 3.2 "Discrete Memory Caching": the navigation map is clustered into groups, each
 *     group's KV cache is computed on its own and kept; any subset, in any order, is re-used
 *     without recomputation; new objects are concatenated at the END of their group.
 *   - App. C "Detailed Planning Example": the planner's prompt is the selected groups followed
 *     by the new tokens (instruction + trajectory).
 *   - App. A "LLM inference and KV Cache": Attn = softmax(Q K^T / sqrt(D)) V; decoding
 *     concatenates the new token's K/V to what is already there.
 *   - Sec. 3.3 "Attention-based Memory Clustering": the attention between new tokens and an
 *     existing group decides clustering; this library returns the un-averaged primitive, the
 *     post-softmax probability mass that each query row puts on each selected group.
 *
 * All K/V/Q/O tensors are bf16, row-major, DEVICE memory owned by the caller and kept alive
 * until the stream reaches the call.  Index arrays (select list, prefix counts) are HOST
 * memory and are consumed before the call returns.  The library owns the page pool, the
 * group tables, the gather-plan buffers and the split-KV scratch, all allocated in
 * enl_cache_create; enl_attend and enl_group_store allocate no device memory.
 *
 * Every device operation is enqueued on the stream the caller passes (a cudaStream_t cast to
 * void*; NULL = the legacy default stream).  No call synchronises the device except
 * enl_cache_create, enl_cache_free, enl_cache_status and enl_cache_selfcheck.  Validation
 * happens on the host before anything is enqueued: a call that returns a validation error
 * (ENL_E_INVAL, ENL_E_NOGROUP, ENL_E_NOMEM, ENL_E_LIMIT, ENL_E_EVICTED) has enqueued nothing
 * and has left the cache unchanged.  ENL_E_CUDA (a launch or copy that the runtime refused)
 * can come after the tables were updated and after earlier launches of the same call were
 * enqueued: treat the cache as unusable then.
 *
 * No position encoding is applied here: cached K is stored as the caller produced it (already
 * rotated at whatever positions the caller assigned to the group), so results do not depend
 * on the order of the select list except for the order of the mass slots.
 */
#ifndef ENL_H
#define ENL_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct enl_cache enl_cache_t;            /* opaque */

enum { ENL_BF16 = 1 };
enum { ENL_DEVICE_NONE = -1 };                   /* bookkeeping-only cache: tables, no GPU   */
enum { ENL_REPLACE = 0, ENL_APPEND = 1 };        /* enl_group_store modes                    */

enum {                                            /* enl_attend_args_t.flags                  */
    ENL_PLAN_ONLY = 1u,                           /* validate + build the gather plan + fill  */
                                                  /* sel_off_out, enqueue nothing             */
    ENL_MASS_ONLY = 2u                            /* only group_mass / group_mass_sum are     */
                                                  /* wanted: `out` is not written (may be     */
                                                  /* NULL); needs group_mass                  */
};

enum {                                            /* return codes                             */
    ENL_OK         =  0,
    ENL_E_INVAL    = -1,   /* null pointer, bad shape, n_q > n_new, duplicate id in a list ...  */
    ENL_E_NOGROUP  = -2,   /* group id out of range, or never stored for that layer            */
    ENL_E_NOMEM    = -3,   /* page pool, plan buffers or a create-time allocation exhausted    */
    ENL_E_CUDA     = -4,   /* a CUDA call failed, or a GPU operation on a bookkeeping cache    */
    ENL_E_TIMEOUT  = -5,   /* a bounded wait inside a kernel expired (see enl_cache_status)    */
    ENL_E_LIMIT    = -6,   /* a size beyond the fixed maxima of enl_attend_static              */
                           /* -7 is not used                                                    */
    ENL_E_EVICTED  = -8,   /* the group's K/V is in the slow tier only (see enl_step_prepare)   */
    ENL_E_CORRUPT  = -9    /* enl_cache_selfcheck: a guard page of the pool has been written    */
};

typedef struct {
    int32_t n_layers, n_q_heads, n_kv_heads;     /* n_q_heads = n_kv_heads * {1,2,4,8,16}    */
    int32_t head_dim;                            /* 64 or 128                                */
    int32_t page_tokens;                         /* 0 = library default (16); only 16 today  */
    int32_t max_groups;                          /* group ids are 0 .. max_groups-1          */
    int64_t max_tokens;                          /* pool capacity, tokens summed over groups */
    int32_t dtype;                               /* ENL_BF16                                 */
    int32_t device;                              /* CUDA ordinal, or ENL_DEVICE_NONE         */
    int32_t max_batch;                           /* episodes per enl_attend; 0 = 64          */
    int32_t max_q_tokens;                        /* query rows per enl_attend; 0 = 16384     */
    int64_t scratch_bytes;                       /* split-KV scratch; 0 = 64 MiB             */
} enl_cache_desc_t;

/*
 * Sec. 3.2: create the store that keeps every group's K/V.  Allocates, on desc->device, the
 * K and V page pools for all layers ([layer][page][kv head][page_tokens][head_dim] bf16,
 * zero-filled), the plan buffers and the scratch.  Synchronises the device.
 * Errors: ENL_E_INVAL (bad shape), ENL_E_NOMEM (allocation failed), ENL_E_CUDA.
 */
int enl_cache_create(const enl_cache_desc_t *desc, enl_cache_t **out);

/*
 * Sec. 3.2: write one group's K/V for one layer (every group's KV cache is computed on its
 * own and kept), or append rows after the group's current end (newly detected objects join
 * the end of their group; the rows already there are not touched).
 *   k_dev, v_dev : [n_tokens][n_kv_heads][head_dim] bf16, device; may be NULL only on a
 *                  bookkeeping-only cache.
 *   mode         : ENL_REPLACE sets the group's length for this layer to n_tokens;
 *                  ENL_APPEND adds n_tokens rows after the current length.
 * Pages are shared by all layers of a group, so a group's length must agree across the layers
 * that are attended: enl_attend uses the length stored for the layer it is given.
 * n_tokens = 0 is legal (an empty group).
 * Errors: ENL_E_INVAL, ENL_E_NOGROUP (id out of range), ENL_E_NOMEM (pool exhausted; state
 * unchanged), ENL_E_CUDA.
 */
int enl_group_store(enl_cache_t *c, int32_t group_id, int32_t layer, int32_t n_tokens,
                    const void *k_dev, const void *v_dev, int32_t mode, void *cuda_stream);

/*
 * Sec. 3.2, the same operation for every layer at once: a group's description (or the new
 * objects appended to it) passes through all layers of the planner in one prefill, so the K/V
 * of all layers arrive together.  One kernel launch per 64 pages instead of one per layer.
 *   k_dev, v_dev : HOST arrays of n_layers device pointers, k_dev[l] = layer l's
 *                  [n_tokens][n_kv_heads][head_dim] bf16 rows; consumed before the call
 *                  returns.  May be NULL only on a bookkeeping-only cache.
 *   mode         : as in enl_group_store, applied to every layer.
 * Before the call every layer must hold the same length of the group (or none): ENL_E_INVAL
 * otherwise.  All or nothing: a call that returns an error has changed no layer.
 * Errors: as enl_group_store.
 */
int enl_group_store_all_layers(enl_cache_t *c, int32_t group_id, int32_t n_tokens,
                               const void *const *k_dev, const void *const *v_dev, int32_t mode,
                               void *cuda_stream);

typedef struct {
    int32_t layer;
    int32_t batch;                     /* independent episodes in this call, >= 1              */
    const int32_t *sel_ids;            /* HOST [n_sel]: selected group ids, episode by episode */
    const int32_t *cu_sel;             /* HOST [batch+1] prefix counts into sel_ids            */
    const int32_t *cu_q;               /* HOST [batch+1] prefix counts of query rows           */
    const int32_t *cu_new;             /* HOST [batch+1] prefix counts of new-token keys       */
                                       /*   all three may be NULL when batch == 1              */
    int32_t n_sel, n_q, n_new;         /* totals over the batch                                */
    const void *q;                     /* device bf16 [n_q][n_q_heads][head_dim]               */
    const void *k_new, *v_new;         /* device bf16 [n_new][n_kv_heads][head_dim]            */
    void *out;                         /* device bf16 [n_q][n_q_heads][head_dim]               */
    float *group_mass;                 /* device fp32 or NULL.  Row r (global over the batch), */
                                       /*   q head h, slot s of its episode at                 */
                                       /*   (r*n_q_heads + h)*mass_stride + s; slot s < G_b is */
                                       /*   the s-th id of the episode's list, slot G_b the    */
                                       /*   new tokens; entries past G_b are not written       */
    int32_t mass_stride;               /* >= max_b(G_b) + 1                                    */
    int32_t *sel_off_out;              /* HOST or NULL, [n_sel + batch]: per episode the       */
                                       /*   exclusive prefix sum (G_b + 1 entries, in tokens)  */
                                       /*   of its selected groups' lengths                    */
    int32_t split_hint;                /* 0 = library chooses the number of KV splits,         */
                                       /*   k >= 1 = use k splits (clamped to what fits)       */
    uint32_t flags;                    /* ENL_PLAN_ONLY, ENL_MASS_ONLY                         */
    /* Sec. 3.3 consumes only an average of the mass over an object's tokens, the q heads and  */
    /* the scored layers.  With group_mass_sum the call ADDS, for every object o and slot s,   */
    /* the sum over the object's query rows and all q heads of the row's mass on s to          */
    /* group_mass_sum[o * sum_stride + s] (one reduction inside the attention kernel, one      */
    /* atomic add per warp, object and slot), so that the caller zeroes the array once, lets   */
    /* the scored layers accumulate and never reads the per-row masses back:                   */
    /* enl_cluster_assign_sums turns the sums into averages and decisions.                     */
    float *group_mass_sum;             /* device fp32 [n_obj][sum_stride] or NULL; needs       */
                                       /*   group_mass (which the kernel still fills)          */
    int32_t sum_stride;                /* >= max_b(G_b) + 1                                    */
    int32_t n_obj;                     /* objects; 0 when group_mass_sum is NULL               */
    const int32_t *obj_off;            /* HOST [n_obj+1], ascending: object o owns query rows  */
                                       /*   obj_off[o] .. obj_off[o+1]-1 (global over the      */
                                       /*   batch); rows outside every span are not summed     */
} enl_attend_args_t;

/*
 * App. A + App. C + Sec. 3.3: for every episode b, query row r and q head h (reading kv head
 * h / (n_q_heads / n_kv_heads)):
 *   keys   = the stored rows of the episode's selected groups, in list order, then the new
 *            keys 0 .. c with c = (n_new_b - n_q_b) + r  (prefill: n_q_b = n_new_b; a decode
 *            step passes n_q_b = 1 and the grown new-token buffer);
 *   out    = softmax(q . keys / sqrt(head_dim)) . values           (fp32 accumulate, bf16 out)
 *   mass   = the same probabilities summed per slot (fp32); every row sums to 1.
 * A group appears at most once in an episode's list (the retrieval's x_i is 0 or 1, Sec. 3.4);
 * an empty list is legal (plain causal attention), so is a zero-length group (mass 0).
 * Errors: ENL_E_INVAL, ENL_E_NOGROUP, ENL_E_NOMEM (plan larger than the plan buffers),
 * ENL_E_CUDA.  Kernel-side bounded waits report through enl_cache_status.
 */
int enl_attend(enl_cache_t *c, const enl_attend_args_t *args, void *cuda_stream);

/* Releases everything enl_cache_create allocated.  Synchronises the device.  NULL is a no-op. */
int enl_cache_free(enl_cache_t *c);

/* ---- helpers (not part of the four calls above) ---------------------------------------- */

/* Static text for a return code. */
const char *enl_strerror(int code);

/* Current length in tokens of a group for a layer, -1 if never stored, ENL_E_* on a bad id. */
int32_t enl_group_len(const enl_cache_t *c, int32_t group_id, int32_t layer);

/* Synchronises the device and returns ENL_OK, or ENL_E_TIMEOUT if any kernel of this cache
 * gave up on a bounded wait since the last call (the flag is then cleared). */
int enl_cache_status(enl_cache_t *c);

/* Synchronises the device and checks the two pages of every layer's K and V pool that no group ever owns
 * (the all-zero page that stands for "no page" at the low end, a guard page at the high end): a kernel that
 * wrote outside the pages it was given shows up as ENL_E_CORRUPT.  A debugging aid; ENL_OK otherwise. */
int enl_cache_selfcheck(enl_cache_t *c);

/*
 * Read-back of the gather plan built by the last enl_attend (host copy), for tests of the
 * integer book-keeping.  Each array pointer may be NULL; counts are always written.
 *   stream_pages[i], stream_meta[i] : page id and (slot << 8 | valid tokens) of KV-stream entry i
 *   ep_stream_off[b], ep_cached_tiles[b] : first entry and number of 128-key tiles of episode b
 *   n_splits : KV splits chosen;  n_items : CTAs of the attention launch
 *   merge_kind : how the splits are merged: 0 no splits, 1 partial results in the scratch buffer and a
 *                second (merge) kernel, 2 inside the attention kernel by pairs of CTAs (two splits,
 *                head_dim 128), 3 inside the one-token decode kernel
 */
int enl_plan_inspect(const enl_cache_t *c, int32_t cap_entries, int32_t *stream_pages,
                     int32_t *stream_meta, int32_t *n_entries, int32_t cap_batch,
                     int32_t *ep_stream_off, int32_t *ep_cached_tiles, int32_t *n_splits,
                     int32_t *n_items, int32_t *merge_kind);

/* ---- slow tier: all groups live in host memory, the selected ones are loaded once per step ------ */

typedef struct {
    int32_t n_hit;                     /* selected groups that were already in device memory          */
    int32_t n_miss;                    /* selected groups loaded from the slow tier by this call      */
    int32_t n_evicted;                 /* groups pushed out of device memory to make room             */
    int64_t bytes_h2d, bytes_d2h;      /* page bytes moved, all layers, K and V                       */
} enl_prepare_stats_t;

/*
 * Sec. 3.2: the KV cache of every group lives in slow memory and only the selected groups are brought
 * into device memory, once per planning step rather than once per decoded token.
 * enl_tier_enable gives the cache a slow tier: a pinned host pool (same page format) for
 * host_tokens tokens summed over groups (plus one page of slack per group).  From then on a group is in
 * device memory, in the slow tier, or in both.
 * enl_group_evict copies a group's pages to the slow tier (all layers; skipped when the copy there is
 * current) and releases its device pages.
 * enl_step_prepare makes every group of the select list device-resident before the step's attends:
 * a resident group is a hit, any other is loaded from the slow tier once, for all layers; when the
 * device pool is short, the least recently selected groups outside the list are evicted first.  The
 * cache hit rate of the step (Sec. 3.4, last paragraph) is n_hit / n_sel.
 * All copies are enqueued on the stream (kernels that read or write the pinned pool directly).
 * enl_attend / enl_group_store on a group that is only in the slow tier return ENL_E_EVICTED.
 * Errors: ENL_E_INVAL, ENL_E_NOGROUP, ENL_E_NOMEM (host pool or device pool too small for the
 * request; residency is unchanged then), ENL_E_CUDA.
 */
int enl_tier_enable(enl_cache_t *c, int64_t host_tokens);
int enl_group_evict(enl_cache_t *c, int32_t group_id, void *cuda_stream);
int enl_step_prepare(enl_cache_t *c, const int32_t *sel_ids, int32_t n_sel, void *cuda_stream,
                     enl_prepare_stats_t *stats);
/* 1 if the group's pages are in device memory, 0 if only in the slow tier, ENL_E_* on a bad id. */
int enl_group_resident(const enl_cache_t *c, int32_t group_id);

/* ---- clustering reduce: what consumes the group mass ------------------------------------------ */

#define ENL_CLUSTER_MAX_LAYERS   16
#define ENL_CLUSTER_MAX_OBJECTS  480

typedef struct {
    int32_t n_layers;                  /* scored layers (the paper: about 1/10 of the model)          */
    const float *const *mass;          /* HOST array of n_layers DEVICE pointers: the group_mass of   */
                                       /*   the scoring enl_attend of each layer,                     */
                                       /*   [n_q][n_q_heads][mass_stride] fp32                        */
    int32_t n_q, n_q_heads, mass_stride;
    int32_t n_groups;                  /* slots 0 .. n_groups-1 are the existing groups (the slot of  */
                                       /*   the new tokens, if present, lies beyond and is ignored)   */
    int32_t n_obj;                     /* newly detected objects                                      */
    const int32_t *obj_off;            /* HOST [n_obj+1]: object o owns query rows obj_off[o] ..      */
                                       /*   obj_off[o+1]-1 (its tokens in the new-token prompt)       */
    float threshold;
    float *avg;                        /* device fp32 [n_obj][n_groups]: mean mass over the object's  */
                                       /*   rows, all q heads and all scored layers                   */
    int32_t *assign;                   /* device int32 [n_obj]: the group with the largest average if */
                                       /*   it exceeds threshold (lowest index on ties), else -1 =    */
                                       /*   "open a new group"                                        */
} enl_cluster_args_t;

/*
 * Sec. 3.3 "Attention-based Memory Clustering": a newly detected object joins an existing group when
 * the average attention between the two exceeds a threshold, else it opens a new group;
 * the paper leaves open over what the average runs and which group wins when several exceed it: here
 * the mean over the object's token rows, q heads and scored layers of the probability mass on the
 * group, and the group with the largest mean.  An object with an empty span gets average 0.
 * Everything is enqueued on the stream; allocates nothing.  Errors: ENL_E_INVAL (null pointer, spans
 * not ascending or beyond n_q, mass_stride < n_groups), ENL_E_LIMIT (more than ENL_CLUSTER_MAX_LAYERS
 * layers or ENL_CLUSTER_MAX_OBJECTS objects per call), ENL_E_CUDA.
 */
int enl_cluster_assign(const enl_cluster_args_t *args, void *cuda_stream);

/*
 * The same decision from the sums that enl_attend accumulated in group_mass_sum over the scored
 * layers: avg[o][g] = mass_sum[o * sum_stride + g] / (rows of object o * n_q_heads * n_layers),
 * assign as above.  mass_sum, avg [n_obj][n_groups] and assign [n_obj] are device memory, obj_off
 * is HOST [n_obj+1] (the spans given to enl_attend).  Enqueued on the stream; allocates nothing.
 * Errors: ENL_E_INVAL, ENL_E_LIMIT (more than ENL_CLUSTER_MAX_OBJECTS objects), ENL_E_CUDA.
 */
int enl_cluster_assign_sums(const float *mass_sum, int32_t sum_stride, int32_t n_groups, int32_t n_obj,
                            const int32_t *obj_off, int32_t n_q_heads, int32_t n_layers, float threshold,
                            float *avg, int32_t *assign, void *cuda_stream);

/* ---- retrieval knapsack: what produces the select list ----------------------------------------- */

/*
 * Sec. 3.4, Eq. 1-2: choose x_i in {0,1} maximising sum (P_i - threshold) x_i subject to
 * sum M_i x_i <= M.  Host-only integer dynamic programme: M_i are rounded UP and M rounded DOWN to
 * multiples of `quantum` bytes (so the budget is never exceeded), groups with P_i <= threshold are
 * never taken; of two choices with the same value the one found first (fewer late groups) is kept.  Writes the chosen group indices in ascending
 * order to sel_out (capacity n) and returns their count, or ENL_E_INVAL / ENL_E_NOMEM (the table
 * needs n * (M / quantum + 1) bytes).
 */
int enl_select_knapsack(int32_t n, const float *prob, float threshold, const int64_t *mem_bytes,
                        int64_t budget_bytes, int64_t quantum, int32_t *sel_out);

/* ---- optional: rotary position encoding of rows before they are stored ------------------------ */

#define ENL_ROPE_MAX_HEAD_DIM 256

/*
 * Sec. 3.2 mentions position encoding by citation only: every group keeps the positions it was
 * computed with, and appended tokens continue them.  The attention and the store take K (and Q)
 * as given; no call of the path rotates anything.  A caller that holds un-rotated rows can rotate
 * them here, in place, before enl_group_store / enl_attend: rotary position embedding as published
 * (Su et al., "RoFormer"), channel pair j of every head turned by the angle pos * base^(-2j/D):
 *   (x1, x2) -> (x1 cos - x2 sin, x2 cos + x1 sin),
 * the pair being channels (2j, 2j+1) if interleaved != 0, else (j, j + D/2).  The paper fixes
 * neither the base nor the pairing; both are the caller's.
 *   rows      : device bf16 [n][n_heads][head_dim], 4-byte aligned, rotated in place
 *   positions : device int32 [n], or NULL: row i then has position first_pos + i
 * Angles are formed in double precision and reduced before sine and cosine are taken in fp32;
 * results are rounded to bf16.  Enqueued on the stream; allocates nothing.
 * Errors: ENL_E_INVAL (null rows, n < 0, n_heads < 1, odd head_dim, base <= 0), ENL_E_LIMIT
 * (head_dim > ENL_ROPE_MAX_HEAD_DIM), ENL_E_CUDA.
 */
int enl_rope_rotate(void *rows, int32_t n, int32_t n_heads, int32_t head_dim, const int32_t *positions,
                    int32_t first_pos, double base, int32_t interleaved, void *cuda_stream);

/* ---- an entry point that allocates nothing ------------------------------------------------ */

#define ENL_STATIC_MAX_SEGMENTS  255                 /* cached segments per call                      */
#define ENL_STATIC_MAX_KEYS      65536               /* cached keys + new keys per call               */
#define ENL_STATIC_SCRATCH_BYTES (4u << 20)          /* size of the library's built-in scratch array  */

typedef struct {
    int32_t n_q_heads, n_kv_heads;     /* n_q_heads = n_kv_heads * {1,2,4,8}                        */
    int32_t head_dim;                  /* 64 or 128                                                 */
    int32_t n_seg;                     /* cached segments (groups) in the key stream, may be 0      */
    const int32_t *seg_len;            /* HOST [n_seg]: tokens per segment, in stream order         */
    int32_t n_new;                     /* new-token keys the query sees (its own included), >= 1    */
    const void *q;                     /* device bf16 [n_q_heads][head_dim]: the one query token    */
    const void *k, *v;                 /* device bf16 [sum(seg_len) + n_new][n_kv_heads][head_dim]: */
                                       /*   the segments back to back, then the new keys            */
    void *out;                         /* device bf16 [n_q_heads][head_dim]                         */
    float *group_mass;                 /* device fp32 [n_q_heads][n_seg + 1] or NULL; slot n_seg =  */
                                       /*   the new tokens                                          */
} enl_static_args_t;

/*
 * (The paper has no counterpart: this entry point exists for deployment reasons only.)
 * One decode-style query token attends over segments of cached keys plus the new keys, exactly as an
 * enl_attend call with n_q = 1 would, but WITHOUT touching any allocator: no cache object, no
 * cudaMalloc / cudaFree, no allocating library routine, no host heap.  It is meant for callers
 * that are not allowed to allocate once they are running -- a planner tick inside a real-time
 * control loop with memory fixed at start-up, code hosted by another runtime that owns the whole
 * device heap, a process whose allocator is sealed after initialisation.  Such callers cannot create
 * a cache (the paged pool is an allocation), so they pass the key/value stream as ONE contiguous
 * buffer they own, and the split-KV partial results go to a fixed array of ENL_STATIC_SCRATCH_BYTES
 * that is part of the library image: every GPU that loads the library carries that array until the
 * process exits, whether or not this function is ever called.
 *
 * The work is split over up to 64 key ranges whose partial outputs, log-sum-exps and per-segment
 * sums are written to the built-in array and merged by a second kernel into out / group_mass.
 * Limits: at most ENL_STATIC_MAX_SEGMENTS segments, ENL_STATIC_MAX_KEYS keys in all, 8 q heads per
 * kv head, and partials that fit the array (n_q_heads * (head_dim + n_seg + 2) * 4 bytes per
 * 1024 keys); anything larger returns ENL_E_LIMIT and enqueues nothing.
 *
 * The first call on a device looks up the array's device address (cudaGetSymbolAddress, with that
 * device current) and keeps it; make that first call outside any stream capture.  All calls share the
 * one array and it keeps the previous call's partials: a call overwrites everything it later reads,
 * so back-to-back calls on one stream are fine, but two calls whose kernels overlap on the GPU
 * (different streams, no dependency) race on it and give wrong results.  Use one stream, or order the
 * calls with events.
 * Errors: ENL_E_INVAL (null pointer, bad shape, negative length), ENL_E_LIMIT, ENL_E_CUDA.
 */
int enl_attend_static(const enl_static_args_t *args, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* ENL_H */
