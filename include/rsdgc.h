/*
 * rsdgc.h -- C ABI of the B200 (sm_100a) RS-DGC gradient-compression library.
 *
 * The library implements the per-iteration compression step of RS-DGC (arxiv 2312.17530):
 * local gradient accumulation (Eq. 12), the Neighborhood Statistical Indicator of every
 * gradient neighborhood (Eq. 8-10), the per-layer keep count (Eq. 11), the choice of the
 * top neighborhoods of each layer (Algorithm 1, second half), the payload of kept values
 * plus neighborhood indices (Sec. III-C), the same-device aggregation of several workers'
 * payloads (Eq. 12 third line / Eq. 2 "Sync"), and the layer-wise dynamic compression
 * ratio from the weights (Eq. 3-5, Algorithm 1 first half).
 *
 * Conventions
 *  - Every function returns an int: RSDGC_OK (0) or a negative rsdgc_error.  Nothing
 *    throws, aborts or prints.  Argument errors are reported synchronously; conditions that
 *    are only known on the device (non-finite indicator, payload capacity exceeded) are
 *    recorded in a device status word read by rsdgc_get_status().
 *  - "dev" pointers are device memory of the plan's device, owned by the caller; "host"
 *    pointers are host memory.  The library allocates only the plan (a host struct plus
 *    small device tables).  No call reads device memory on the host except
 *    rsdgc_get_status() and rsdgc_compress_host(), which synchronise the stream.
 *  - `stream` is a CUDA stream handle (cudaStream_t passed as void*; NULL = default
 *    stream).  All device work is enqueued on it and is asynchronous.  A plan holds
 *    per-layer scratch tables, so at most one call per plan may be in flight at a time:
 *    issue all calls that share a plan on one stream (or order them yourself).
 *  - Layout: a layer l is a row-major rows x cols matrix partitioned into nh x nw
 *    neighborhoods ("tiles"; edge tiles are clipped).  TC = ceil(cols/nw), TR =
 *    ceil(rows/nh), K_l = TR*TC, tile index k = tile_row*TC + tile_col (layer-local,
 *    int32).  All layers of one quantity (gradients, accumulator/"residual", weights,
 *    dense output) live in one flat arena; layer l starts at element elem_offset_l
 *    (a multiple of 64 elements) given by rsdgc_plan_layer_info().  Padding elements
 *    between layers are never read or written.  Indicator keys live in a flat array of
 *    total_tiles_padded entries, layer l starting at tile_offset_l.
 *  - Payload: idx_dev[idx_offset_l + s] is the s-th kept tile of layer l (ascending),
 *    val_dev[val_offset_l + s*nh*nw + a*nw + b] its element (a, b) (+0 where the tile is
 *    clipped), with idx_offset_l = sum_{l'<l} k_l' and val_offset_l = sum_{l'<l}
 *    k_l' * nh_l' * nw_l'; counts_dev[l] = k_l.  The values are binary32.  A plan created
 *    with RSDGC_PAYLOAD_BF16 uses bfloat16 values instead (an option of this library; the
 *    paper sends binary32): val_dev is then an array of 16-bit words, the value sent is
 *    q = v rounded to the nearest bfloat16 (ties to even), and the accumulator keeps v - q
 *    (exact in binary32) instead of +0, so the rounding error is sent later like everything
 *    else that was not sent (Eq. 12).  Capacities and offsets count values, not bytes.
 */
#ifndef RSDGC_H_
#define RSDGC_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct rsdgc_plan rsdgc_plan; /* opaque, library-owned */

typedef enum { RSDGC_F32 = 0, RSDGC_BF16 = 1 } rsdgc_dtype;

typedef enum {
    RSDGC_OK = 0,
    RSDGC_ERR_INVALID = -1,   /* null pointer, non-positive size, value out of range      */
    RSDGC_ERR_ALIGNMENT = -2, /* a device pointer is not 16-byte aligned                  */
    RSDGC_ERR_CAPACITY = -3,  /* a size exceeds what the library supports                 */
    RSDGC_ERR_CUDA = -4,      /* a CUDA runtime call failed (see rsdgc_last_cuda_error)   */
    RSDGC_ERR_NOMEM = -5      /* host or device allocation of the plan failed             */
} rsdgc_error;

/* plan flags */
#define RSDGC_KEEP_AT_LEAST_ONE 1u /* k_l = max(1, ceil(K_l * ratio_l)): every layer sends >= 1 tile */
#define RSDGC_NO_BULK_COPY 2u      /* first pass: register-staged kernel for every item           */
#define RSDGC_MOMENTUM 4u          /* the plan is used with rsdgc_compress_momentum() (Eq. 12 l.1) */
#define RSDGC_PAYLOAD_BF16 8u      /* payload values are bfloat16 instead of binary32 (see below)  */
#define RSDGC_NO_FUSED_TAIL 16u    /* always the chained selection kernels, also on plans of small  */
                                   /* layers (which otherwise select and pack in one kernel)        */

/* bits of rsdgc_status.flags */
#define RSDGC_STATUS_NONFINITE 1u         /* some indicator was NaN/Inf (ranked first as +Inf)  */
#define RSDGC_STATUS_PAYLOAD_OVERFLOW 2u  /* idx/val capacity too small; excess tiles not sent   */
#define RSDGC_STATUS_TIMEOUT 4u           /* a bounded on-chip wait gave up; results are invalid  */
#define RSDGC_STATUS_BOUNDS 8u            /* bounds-checked builds (RSDGC_DEBUG) only: a kernel    */
                                          /* formed an index outside its buffers; access skipped  */

typedef struct {
    int64_t rows, cols; /* row-major 2-D view of the layer (Sec. III-C)            */
    int32_t nh, nw;     /* neighborhood shape (the paper's p x p patch, Eq. 7)     */
} rsdgc_layer_desc;

typedef struct {
    int32_t n_layers;
    int32_t grad_dtype;          /* rsdgc_dtype of the gradient arena                       */
    int64_t arena_elems;         /* length of every element arena, padding included         */
    int64_t total_elems;         /* sum of rows*cols                                        */
    int64_t total_tiles;         /* sum of K_l                                              */
    int64_t total_tiles_padded;  /* length of the key / indicator array                     */
    int64_t workspace_bytes;     /* size of the workspace rsdgc_compress() needs            */
    int32_t max_slot;            /* max over layers of nh*nw                                */
    int32_t reserved;
} rsdgc_info;

typedef struct {
    int64_t elem_offset; /* start of the layer in the element arenas              */
    int64_t tile_offset; /* start of the layer in the key / indicator array       */
    int64_t rows, cols;
    int32_t nh, nw;
    int64_t n_tiles;     /* K_l                                                   */
} rsdgc_layer_info;

typedef struct {
    uint32_t flags;        /* RSDGC_STATUS_* bits since the last rsdgc_get_status()            */
    uint32_t reserved;
    int64_t nonfinite;     /* number of non-finite indicators seen                             */
    int64_t idx_needed;    /* payload size the last rsdgc_compress() wanted (tiles)            */
    int64_t val_needed;    /* payload size the last rsdgc_compress() wanted (values)           */
} rsdgc_status;

/*
 * Builds the plan for a set of layers (Algorithm 1's loop over l = 1..L with the
 * neighborhoods of Eq. 7): arena offsets, tile counts, the work lists the kernels walk and
 * the per-layer device tables.  `alpha` is the hyper-parameter of Eq. 8 (0 <= alpha <= 1).
 * `flags`: an OR of RSDGC_KEEP_AT_LEAST_ONE, RSDGC_NO_BULK_COPY, RSDGC_MOMENTUM,
 * RSDGC_PAYLOAD_BF16 and RSDGC_NO_FUSED_TAIL, or 0.  `device` is the CUDA device ordinal.  On success
 * *out owns host memory and a few MB of device memory until rsdgc_plan_destroy().
 * Errors: INVALID (null, n_layers < 1, rows/cols/nh/nw < 1, alpha outside [0,1] or NaN,
 * unknown dtype), CAPACITY (a layer with more than 2^31-1 elements, nh*nw > 4096, or more
 * than 2048 layers), CUDA / NOMEM.
 */
int rsdgc_plan_create(const rsdgc_layer_desc *layers_host, int32_t n_layers, int32_t grad_dtype,
                      float alpha, uint32_t flags, int32_t device, rsdgc_plan **out);

/* Frees the plan; the caller must make sure no work that uses it is still in flight. */
int rsdgc_plan_destroy(rsdgc_plan *plan);

/* Sizes derived from the plan (host only). */
int rsdgc_plan_info(const rsdgc_plan *plan, rsdgc_info *out_host);
int rsdgc_plan_layer_info(const rsdgc_plan *plan, int32_t layer, rsdgc_layer_info *out_host);

/* Upper bound of the payload sizes (in tiles and in values) when every layer's ratio is at
 * most max_ratio: sum_l min(K_l, ceil(K_l*max_ratio) + 1) and the same weighted by nh*nw. */
int rsdgc_plan_payload_bound(const rsdgc_plan *plan, float max_ratio, int64_t *idx_capacity_host,
                             int64_t *val_capacity_host);

/*
 * Layer-wise dynamic compression ratio (Eq. 3-5; Algorithm 1, per-epoch part): importance
 * |w| (Eq. 3), one ranking over all layers of the plan, the ceil(global_keep * G) largest
 * survive (Eq. 4; equal magnitudes: lower arena position first), ratios_dev[l] =
 * survivors_l / G_l in binary32 (Eq. 5).  Implemented as a three-level radix selection on
 * the magnitude bits: no sort, three reads of the weights.
 * weights_dev: binary32 arena with the plan's layer offsets (read only).
 * ratios_dev: out, n_layers floats.  global_keep in [0, 1].
 * The call takes no workspace: its per-layer histograms and counters are among the small device
 * tables the plan owns.
 * Errors: INVALID, ALIGNMENT, CUDA.
 */
int rsdgc_update_ratios(rsdgc_plan *plan, const float *weights_dev, float global_keep,
                        float *ratios_dev, void *stream);

/*
 * The ratio rule of rsdgc_update_ratios() for callers that must not allocate device memory.
 * (The paper has no counterpart: it describes the rule, Eq. 3-5, not how memory is managed.)
 *
 * Who cannot allocate: code that runs while a stream capture is open on its thread (cudaMalloc
 * is not allowed there), runtimes that hand all device memory to their own pool at start-up
 * and forbid driver allocations afterwards, and loops that cannot afford the device-wide
 * synchronisation an allocation or a free may imply.  rsdgc_plan_create() allocates, so such
 * callers cannot use a plan; this entry point needs none.  The caller passes the weights and
 * the output; every byte of scratch (per-layer histograms, counters) lives in one fixed array
 * inside the library: about 513 KB of device memory on every GPU that loads the library, kept
 * until the process exits.
 *
 * weights_dev: binary32 weights; layer l occupies layer_sizes_host[l] elements starting at
 *   element layer_offsets_host[l] (a multiple of 4).  ratios_dev: out, n_layers floats.  The
 *   result equals rsdgc_update_ratios() on a plan with the same layers and offsets.
 * Limits: 1 <= n_layers <= RSDGC_NOALLOC_MAX_LAYERS, each layer below 2^31 elements; beyond
 *   them the call returns RSDGC_ERR_CAPACITY and does nothing.  Other errors: INVALID,
 *   ALIGNMENT, CUDA.
 * The first call on a device looks up the device address of the scratch array (one runtime
 * query, with that device current; later calls reuse it): make that first call before any
 * stream capture begins.  No call allocates or frees memory.
 * All calls on a device share the scratch array, and it keeps what the previous call left in
 * it, so each call starts by clearing it on `stream`.  Two calls whose work overlaps on the
 * GPU (different streams, or different threads) race on it and give wrong ratios: order them.
 */
#define RSDGC_NOALLOC_MAX_LAYERS 64
int rsdgc_update_ratios_noalloc(const float *weights_dev, const int64_t *layer_offsets_host,
                                const int64_t *layer_sizes_host, int32_t n_layers, float global_keep,
                                float *ratios_dev, void *stream);

/*
 * One worker's per-iteration compression (Algorithm 1, per-iteration part; Eq. 8-12):
 *   v = g + r, written in place over the residual arena           (Eq. 12, second line)
 *   NSI of every tile of v in binary32                            (Eq. 8-10)
 *   k_l = ceil(K_l * ratios_dev[l]) clipped to [0 or 1, K_l]      (Eq. 11)
 *   the k_l tiles of largest NSI per layer, ties to the lower tile index, found by a
 *   three-level radix selection on the NSI bit patterns           (Algorithm 1 ranking)
 *   payload idx/val/counts as described at the top of this file   (Sec. III-C)
 *   residual entries of sent tiles set to +0                      (Eq. 12)
 * grads_dev: gradient arena, binary32 or bfloat16 as the plan says (read only).
 * residual_dev: binary32 arena, in: accumulator r, out: r' (what was not sent).
 * ratios_dev: n_layers floats; values <= 0 give k_l = 0 (or 1 with KEEP_AT_LEAST_ONE),
 *   values >= 1 keep every tile.
 * idx_dev/val_dev: payload buffers of idx_capacity tiles / val_capacity values; if the
 *   payload does not fit, the tiles that do not fit are neither written nor removed from
 *   the residual and RSDGC_STATUS_PAYLOAD_OVERFLOW is raised.  counts_dev: out, n_layers.
 * nsi_dev: optional (may be NULL) out array of total_tiles_padded floats receiving the
 *   indicator of every tile (layer l at tile_offset_l).
 * workspace_dev: workspace_bytes bytes, 16-byte aligned; may be NULL when nsi_dev is given.
 * Errors: INVALID, ALIGNMENT, CUDA.
 */
int rsdgc_compress(rsdgc_plan *plan, const void *grads_dev, float *residual_dev,
                   const float *ratios_dev, int32_t *idx_dev, int64_t idx_capacity,
                   void *val_dev, int64_t val_capacity, int32_t *counts_dev, float *nsi_dev,
                   void *workspace_dev, void *stream);

/*
 * The same step with momentum correction ahead of the accumulation (Eq. 12, first and second
 * line): u = momentum * u + g (product then sum, each rounded to binary32), v = r + u; the
 * rest is rsdgc_compress().  velocity_dev: binary32 arena with the plan's layout, in: u of the
 * previous iteration (zeros at the start), out: the new u; it is not masked where tiles are
 * sent (Eq. 12 does not say so).  The plan must have been created with RSDGC_MOMENTUM, which
 * sizes the first pass for the third stream (20 instead of 12 bytes per element); such a plan
 * is not accepted by rsdgc_compress().  momentum in [0, 1]; 0 reproduces rsdgc_compress().
 * Errors: INVALID, ALIGNMENT, CUDA.
 */
int rsdgc_compress_momentum(rsdgc_plan *plan, const void *grads_dev, float *velocity_dev, float momentum,
                            float *residual_dev, const float *ratios_dev, int32_t *idx_dev,
                            int64_t idx_capacity, void *val_dev, int64_t val_capacity, int32_t *counts_dev,
                            float *nsi_dev, void *workspace_dev, void *stream);

/*
 * The same step for the n_workers data-parallel workers that share this GPU (Sec. III-A: every
 * node k compresses its own gradient with the same per-layer ratios; Eq. 12 per worker k), in
 * one call: one accumulate+NSI pass per worker, then the selection, index and gather kernels
 * run once each over all workers.  Results per worker are exactly those of n_workers calls of
 * rsdgc_compress().
 * rsdgc_plan_reserve_workers() gives the plan the selection tables of n_workers workers (a few
 * MB of device memory each; allocates, so call it once outside any stream capture);
 * rsdgc_compress_workers() returns CAPACITY if fewer workers were reserved.
 * grads_dev_host / residual_dev_host / idx_dev_host / val_dev_host / counts_dev_host: HOST
 * arrays of n_workers DEVICE pointers, one arena / payload per worker (no two workers may share
 * an accumulator or a payload buffer); idx_capacity / val_capacity hold for every worker.
 * workspace_dev: n_workers * workspace_bytes bytes, 16-byte aligned.  Not for plans created
 * with RSDGC_MOMENTUM.  With rsdgc_profile_enable() a call records one set of events per group
 * of up to 16 workers: stage 0 spans the accumulate+NSI passes of all the workers of the group,
 * the later stages the single launches that serve them all.
 * Errors: INVALID, ALIGNMENT, CAPACITY, CUDA / NOMEM.
 */
int rsdgc_plan_reserve_workers(rsdgc_plan *plan, int32_t n_workers);
int rsdgc_compress_workers(rsdgc_plan *plan, int32_t n_workers, const void *const *grads_dev_host,
                           float *const *residual_dev_host, const float *ratios_dev,
                           int32_t *const *idx_dev_host, int64_t idx_capacity,
                           void *const *val_dev_host, int64_t val_capacity,
                           int32_t *const *counts_dev_host, void *workspace_dev, void *stream);

/*
 * Same step with the gradient and the payload in HOST memory: copies grads_host into
 * grads_dev (a caller-owned staging arena), runs rsdgc_compress(), waits, and copies
 * counts and exactly the used part of idx/val back to the host buffers (which must hold
 * idx_capacity / val_capacity entries).  Pinned host memory makes the copies asynchronous
 * to the CPU but is not required.  *idx_used_host / *val_used_host receive the payload
 * sizes.  The accumulator stays on the device.  Synchronises the stream.
 */
int rsdgc_compress_host(rsdgc_plan *plan, const void *grads_host, void *grads_dev,
                        float *residual_dev, const float *ratios_dev, int32_t *idx_dev,
                        int64_t idx_capacity, void *val_dev, int64_t val_capacity,
                        int32_t *counts_dev, void *workspace_dev, int32_t *idx_host,
                        void *val_host, int32_t *counts_host, int64_t *idx_used_host,
                        int64_t *val_used_host, void *stream);

/*
 * rsdgc_compress_host() for the n_workers workers of a GPU (Sec. III-A: every node compresses its
 * own gradient), pipelined: staging_dev_host holds TWO caller-owned device arenas of the
 * gradient's type; worker w + 1's gradient is copied into one (on a stream the plan owns) while
 * worker w is compressed out of the other on `stream`, and worker w's counts and payload buffers
 * are copied back right behind its compress.  The payload sizes are not known on the host before
 * the end, so idx_host[w] / val_host[w] must hold idx_capacity / val_capacity entries and receive
 * the whole buffers; idx_used_host[w] / val_used_host[w] say how much of them is payload.
 * grads_host / residual_dev_host / idx_dev_host / val_dev_host / counts_dev_host / idx_host /
 * val_host / counts_host: HOST arrays of n_workers pointers; workspace_dev: workspace_bytes bytes
 * (the workers take turns).  Pinned host memory lets the copies overlap the compression.  Waits
 * for both streams once, at the end; not for use during stream capture.  The first call on a plan
 * creates the copy stream and events.  Not for plans created with RSDGC_MOMENTUM.
 * Errors: INVALID, ALIGNMENT, CUDA.
 */
int rsdgc_compress_workers_host(rsdgc_plan *plan, int32_t n_workers, const void *const *grads_host,
                                void *const *staging_dev_host, float *const *residual_dev_host,
                                const float *ratios_dev, int32_t *const *idx_dev_host, int64_t idx_capacity,
                                void *const *val_dev_host, int64_t val_capacity,
                                int32_t *const *counts_dev_host, void *workspace_dev,
                                int32_t *const *idx_host, void *const *val_host, int32_t *const *counts_host,
                                int64_t *idx_used_host, int64_t *val_used_host, void *stream);

/*
 * Aggregation of n_workers payloads into a dense gradient on the same device (Eq. 12,
 * third line: sum over workers of sparse(v); Eq. 2 "Sync"):
 *   dense[i] = dense[i] + scale * sent_w[i]   for w = 0 .. n_workers-1 in that order,
 * product then sum, each rounded to binary32 (scale = 1 gives the paper's plain sum).
 * idx_dev_host / val_dev_host / counts_dev_host: HOST arrays of n_workers DEVICE pointers
 * to payloads produced by rsdgc_compress() with this plan (or an identical one): the tile
 * indices of a layer must be ascending.  idx_capacity / val_capacity: the number of entries
 * every worker's idx / val buffer holds (the capacities given to rsdgc_compress()); a payload
 * that did not fit them (RSDGC_STATUS_PAYLOAD_OVERFLOW: counts say more than was written) is
 * aggregated as far as it was written, nothing is read past the buffers.  dense_dev: binary32
 * arena, in/out.  Entries whose tile index breaks the order or lies outside the layer are skipped.
 * Errors: INVALID, ALIGNMENT, CUDA.
 */
int rsdgc_decompress_accumulate(rsdgc_plan *plan, int32_t n_workers,
                                const int32_t *const *idx_dev_host,
                                const void *const *val_dev_host,
                                const int32_t *const *counts_dev_host, int64_t idx_capacity,
                                int64_t val_capacity, float scale, float *dense_dev, void *stream);

/*
 * The same aggregation into a dense arena that holds nothing yet (Eq. 12, third line, as an
 * assignment: g_t = scale * sum over workers of sparse(v)):
 *   dense[i] = +0, then dense[i] = dense[i] + scale * sent_w[i] for w = 0 .. n_workers-1,
 * i.e. exactly a zero fill of every layer's elements followed by rsdgc_decompress_accumulate(),
 * in the same launch (no separate pass over the arena).  Padding elements between layers are
 * not written.  n_workers = 0 gives all +0.  Arguments and errors as above.
 */
int rsdgc_decompress_assign(rsdgc_plan *plan, int32_t n_workers, const int32_t *const *idx_dev_host,
                            const void *const *val_dev_host, const int32_t *const *counts_dev_host,
                            int64_t idx_capacity, int64_t val_capacity, float scale, float *dense_dev,
                            void *stream);

/*
 * Per-element (coordinate) view of a payload.  The payload of Sec. III-C names neighborhoods;
 * this expands the indices to one arena position per payload value, for receivers that scatter
 * element by element:
 *   coo_index_dev[j] = elem_offset_l + i * cols_l + jj   for payload value j = val_offset_l +
 *   s * nh * nw + a * nw + b of tile idx[idx_offset_l + s] = (tr, tc), i = tr * nh + a,
 *   jj = tc * nw + b, and -1 where (i, jj) lies outside the layer (the +0 padding of clipped
 *   tiles) or the tile index is not one of the layer's.
 * The values are not touched: (coo_index_dev[j], val_dev[j]) are the pairs.  At most
 * coo_capacity entries are written (payload order).  idx_dev / counts_dev as produced by
 * rsdgc_compress().  Errors: INVALID, ALIGNMENT, CUDA.
 */
int rsdgc_payload_to_coo(rsdgc_plan *plan, const int32_t *idx_dev, const int32_t *counts_dev,
                         int64_t *coo_index_dev, int64_t coo_capacity, void *stream);

/* Waits for the stream, copies the device status word to *out_host and clears it. */
int rsdgc_get_status(rsdgc_plan *plan, void *stream, rsdgc_status *out_host);

/* Text for an rsdgc_error; the cudaError_t of the last RSDGC_ERR_CUDA of this thread. */
const char *rsdgc_strerror(int code);
int rsdgc_last_cuda_error(void);

/* =========================================================================================
 * Diagnostics.  Nothing below is needed to run the method; these calls exist for tests, timing
 * breakdowns and the host-logic checks.
 * ========================================================================================= */

/* Diagnostic: copies the work list of the accumulate+NSI pass, 9 int32 per item: layer,
 * first tile row, tile rows, first tile col, tile cols (the items of a layer partition its
 * tile grid), the kernel that takes the item (0 = bulk-copy kernel, 1 = register-staged
 * kernel), the CTA of that kernel that owns it, the row pitch (elements) of the item's block in
 * shared memory, and the item's flags (1 = one contiguous run, 2 = 128-bit accesses, 4 = bulk
 * copies, 8 = no clipped tile); grids_host[0..1] receive the two kernels'
 * grid sizes and n_flush_host[l] how many (kernel, CTA) pairs touch layer l.  Any pointer
 * may be NULL.  Returns the number of items (or a negative rsdgc_error).  Host only. */
int64_t rsdgc_plan_worklist(const rsdgc_plan *plan, int32_t *items_host, int64_t items_capacity,
                            int32_t *grids_host, int32_t *n_flush_host);

/* Diagnostic: plans whose layers all have at most 262144 tiles select and pack in one kernel per
 * layer-size class instead of the chained selection kernels (unless RSDGC_NO_FUSED_TAIL is set or the
 * layers need more thread-block clusters than the device holds at a time).  Copies that kernel's
 * work list, 6 int32 per CTA: layer, first tile, tiles (0: a cluster rank without work), CTAs that
 * share the layer, this CTA's rank among them, cluster rank of the first of them; the cluster
 * variant's CTAs first (8 per cluster), then the one-CTA layers.  info_host[0..2] receive the two
 * counts and the number of clusters.  Returns the number of CTAs (0: the plan takes the chained
 * kernels) or a negative rsdgc_error.  Host only. */
int64_t rsdgc_plan_tail_slices(const rsdgc_plan *plan, int32_t *slices_host, int64_t capacity,
                               int32_t *info_host);

/*
 * Optional per-kernel timing of rsdgc_compress().  While enabled, every rsdgc_compress() on
 * this plan records CUDA events on its stream: with level 1 only before and after the first
 * pass (accumulate+NSI, the kernel that moves all the bytes), with level 2 after each of the
 * RSDGC_N_COMPRESS_KERNELS stages as well (accumulate+NSI, refine level 2, refine level 3 with
 * the per-chunk counts, mark, gather; on plans that select and pack in one kernel per layer-size
 * class: accumulate+NSI, the cluster kernel, the one-CTA kernel, and two empty stages).  Events
 * between kernels cost about 3 us each, so level 2 is for
 * breakdowns, not for throughput numbers.  rsdgc_profile_read() waits for the recorded events,
 * adds the elapsed milliseconds of every timed stage over all recorded calls into
 * ms_per_kernel_host[RSDGC_N_COMPRESS_KERNELS] (untimed stages stay 0), stores the number of
 * calls and forgets them.  Level 0 (the default) records nothing; not for use during stream
 * capture.
 */
#define RSDGC_N_COMPRESS_KERNELS 5
int rsdgc_profile_enable(rsdgc_plan *plan, int32_t level);
int rsdgc_profile_read(rsdgc_plan *plan, double *ms_per_kernel_host, int64_t *n_calls_host);

/* Number of kernels this library has launched in this process (all plans). */
int64_t rsdgc_launch_count(void);

/*
 * Self-test of the bounded on-chip wait the first pass relies on (the paper has no counterpart):
 * launches one warp that arms a shared-memory barrier for bytes no copy will ever deliver (nothing
 * is in flight before or after), polls it `polls` times (1 .. 2^20) with the library's bounded
 * wait, gives up and raises RSDGC_STATUS_TIMEOUT in the plan's status word, which the next
 * rsdgc_get_status() returns and clears.  The context stays usable.  Errors: INVALID, CUDA.
 */
int rsdgc_selftest_bounded_wait(rsdgc_plan *plan, int32_t polls, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* RSDGC_H_ */
