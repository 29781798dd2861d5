/* mfet.h - C ABI of the multi-faceted embedding-table lookup library (sm_100a).
 *
 * The library computes the lookup path of a ranking model whose sparse ID
 * features are embedded through large hashed tables:
 *
 *   raw 64-bit ID --hash--> table row --gather--> pooled (sum / mean / weighted
 *   sum) over a ragged bag --> one dense fp32 row per sample, the outputs of all
 *   (feature, table) slots side by side.
 *
 * Terms. A FEATURE is one ragged list of IDs per sample. A SLOT is one
 * (feature, table) lookup that yields `dim` output columns; a multi-faceted
 * feature has several slots, one per facet table, in adjacent columns. B is the
 * batch size, F the number of features, L the number of slots, nnz the number
 * of IDs in the batch.
 *
 * Conventions shared by every entry point.
 *   - Return value: MFET_OK (0) or a negative MFET_ERR_* code. Nothing is
 *     printed, thrown or aborted. Argument errors are found on the host before
 *     anything is launched.
 *   - "dev" pointers are device memory of the handle's GPU, "host" pointers are
 *     ordinary host memory; the library never allocates device memory in any
 *     call that takes a stream, and never frees or keeps ownership of caller
 *     memory. Calls that take a stream are asynchronous on it and do not
 *     synchronise, unless stated.
 *   - `mfet_stream_t` is a cudaStream_t passed as void* (NULL = default stream).
 *   - No CPU fallback exists: every step runs in the library's own kernels.
 */
#ifndef MFET_H_
#define MFET_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define MFET_API __attribute__((visibility("default")))
#else
#define MFET_API
#endif

typedef struct mfet_tables mfet_tables_t; /* opaque, library-owned */
typedef void* mfet_stream_t;              /* a cudaStream_t */

enum { MFET_F32 = 0, MFET_F16 = 1, MFET_BF16 = 2, MFET_INT4 = 3 };
enum { MFET_POOL_SUM = 0, MFET_POOL_MEAN = 1, MFET_POOL_WSUM = 2 };
enum { MFET_LOC_DEVICE = 0, MFET_LOC_HOST = 1 };
enum { MFET_VAL_NORMAL = 0, MFET_VAL_GRID = 1 };
enum { MFET_BATCH_IDS_ARE_ROWS = 1, MFET_BATCH_PREFETCHED = 2 }; /* mfet_batch_shape_t.flags */
enum { MFET_OPT_GROUP_POLICY = 1, MFET_OPT_TILE = 2, MFET_OPT_PROFILE = 3, MFET_OPT_STAGE_IDS = 4,
       MFET_OPT_OVERLAP_LAUNCHES = 5 };

enum {
  MFET_OK = 0,
  MFET_ERR_INVALID_ARG = -1,    /* null pointer, bad enum, bad size, bad id   */
  MFET_ERR_NOT_REGISTERED = -2, /* host table used before its memory was given */
  MFET_ERR_ALIGNMENT = -3,      /* pointer or stride not 16-byte aligned       */
  MFET_ERR_UNSUPPORTED_DIM = -4,/* row bytes not a multiple of 16              */
  MFET_ERR_WORKSPACE = -5,      /* workspace missing or too small              */
  MFET_ERR_CUDA = -6,           /* a CUDA runtime call failed                  */
  MFET_ERR_TIMEOUT = -7         /* reserved for bounded device-side waits      */
};

/* Bits of the device error word (mfet_query_status). */
enum {
  MFET_DEV_ROW_RANGE = 1u,      /* a pre-hashed row index was >= rows: the lookup is skipped for a
                                   table in device memory, and counts as the table's last row for a
                                   table in host memory and in mfet_embedding_bag_backward        */
  MFET_DEV_OFFSETS = 2u,        /* offsets decreased inside a bag; bag skipped */
  MFET_DEV_CAPACITY = 4u,       /* a host-path batch exceeded the workspace    */
  MFET_DEV_BOUNDS = 8u,         /* only in the bounds-checked build of the library: a kernel formed an
                                   index outside its array; the access was skipped               */
  MFET_DEV_STALLED = 16u        /* a dedup tile waited two seconds for the counts of the tiles before
                                   it and gave up: the dedup result of that call is undefined     */
};

/* One embedding table. Rows are `dim` elements of `dtype`, row-major.
 * Paper, Section 2.2: categorical IDs reach their vectors through hashed
 * lookup tables; `rows` is that table's vocabulary size. */
typedef struct {
  void* data;           /* MFET_LOC_DEVICE: dev pointer, 16-byte aligned, caller-owned,
                           must outlive the handle. MFET_LOC_HOST: ignored (the memory
                           is supplied later by mfet_host_tables_register).            */
  uint64_t rows;        /* 1 .. 2^63-1                                                  */
  uint32_t dim;         /* elements per row; stored row bytes must be a multiple of 16  */
  uint32_t dtype;       /* MFET_F32 / MFET_F16 / MFET_BF16 / MFET_INT4 (dim % 8 == 0)          */
  uint32_t location;    /* MFET_LOC_DEVICE / MFET_LOC_HOST                              */
  uint32_t flags;       /* must be 0                                                    */
  uint64_t hash_seed;   /* XORed into the raw ID before hashing; 0 = plain hash         */
  uint64_t row_stride_bytes; /* 0 = dense rows; otherwise >= row bytes, multiple of 16  */
} mfet_table_desc_t;

/* Shape of one batch. */
typedef struct {
  int32_t batch;               /* B >= 0                                              */
  int32_t n_features;          /* F >= 1                                              */
  int32_t n_slots;             /* L >= 1                                              */
  int32_t flags;               /* MFET_BATCH_IDS_ARE_ROWS: `ids` already hold row indices (no
                                  hashing); MFET_BATCH_PREFETCHED: see mfet_host_prefetch */
  const int32_t* slot_feature; /* host int32[L]: feature read by each slot            */
  int64_t out_ld;              /* floats per row of `out`; 0 = sum of the slots' dims */
} mfet_batch_shape_t;

/* Stored bytes of one row: dim*4 (F32), dim*2 (F16/BF16); INT4: dim/2 nibble
 * bytes + fp16 scale + fp16 bias, rounded up to a multiple of 16 (dim even).
 * Returns 0 for a bad dtype. */
MFET_API uint64_t mfet_row_bytes(uint32_t dim, uint32_t dtype);

/* Create a table set on GPU `device` (a CUDA ordinal). Copies the descriptors;
 * allocates only small host-side bookkeeping, one pinned status word, one
 * internal stream and two events. Errors: INVALID_ARG (null, n_tables < 1, rows
 * == 0, rows >= 2^63, bad dtype/location, flags != 0, null data for a device
 * table), UNSUPPORTED_DIM, ALIGNMENT, CUDA. */
MFET_API int mfet_tables_create(const mfet_table_desc_t* descs /*host*/, int32_t n_tables, int32_t device,
                       mfet_tables_t** out /*host*/);

/* Destroy the handle; unpins only host memory that the library pinned itself.
 * Synchronises the internal stream. NULL is accepted. */
MFET_API int mfet_tables_destroy(mfet_tables_t* t);

/* Give a MFET_LOC_HOST table its memory (paper, Section 3.3: the largest tables
 * stay in CPU memory while scoring runs on the GPU; here the GPU reads them in
 * place through the unified address space instead of over an RPC).
 * host_ptr: 16-byte-aligned host memory holding at least rows*stride bytes,
 * caller-owned, valid until destroy. flags bit0 clear: the library pins and
 * maps it (cudaHostRegister) and unpins it at destroy; bit0 set: the memory is
 * already pinned and mapped. Errors: INVALID_ARG (bad id, not a host table,
 * already registered, too few bytes), ALIGNMENT, CUDA. */
MFET_API int mfet_host_tables_register(mfet_tables_t* t, int32_t table_id, void* host_ptr, uint64_t bytes,
                              uint32_t flags);

/* rows_out[i] = splitmix64(ids[i] XOR hash_seed) mod rows of table `table_id`,
 * as a non-negative int64 (paper, Section 2.2; the paper names no hash
 * function, this is the library's). ids: dev u64[n]; rows_out: dev i64[n];
 * n >= 0. In-place (rows_out aliasing ids) is allowed. */
MFET_API int mfet_hash_ids(const mfet_tables_t* t, int32_t table_id, const uint64_t* ids, int64_t n,
                  int64_t* rows_out, mfet_stream_t stream);

/* The lookup path for one batch (paper, Sections 1, 2.2, 3.3 and 4.1.1: hashed
 * tables, several facet tables per ID feature all feeding the ranker, largest
 * table in host memory). For slot s with feature f = slot_feature[s], table
 * t = table_ids[s], D = dim_t, and sample b:
 *   bag   = ids[offsets[f*B+b] .. offsets[f*B+b+1])
 *   value = sum over the bag of c_i * row_t(hash_t(id_i)),  c_i = 1 (SUM, MEAN)
 *           or weights[i] (WSUM); MEAN divides by the bag length; an empty bag
 *           gives zeros
 *   out[b*out_ld + col_s + d] = value[d],  col_s = sum of dims of slots before s.
 * Accumulation is fp32 in an order that depends only on the inputs, so repeated
 * calls give identical bits.
 *   ids      dev u64[nnz], bags stored feature-major (all samples of feature 0,
 *            then feature 1, ...); never NULL, even when nnz == 0
 *   offsets  dev i64[F*B + 1], nondecreasing
 *   weights  dev f32[nnz], read only by WSUM slots; may be NULL if there is none
 *   table_ids, pooling  host i32[L]
 *   out      dev f32[B, out_ld]; the columns of all slots are fully overwritten
 * Slots whose table is in host memory run on the library's internal stream
 * (dedup -> cache probe -> host fetch -> pool), overlapped with the others and
 * joined back into `stream`; they need a workspace (mfet_set_workspace). The
 * host never learns how many IDs such a slot has: the kernels read the count from
 * `offsets` and are sized by the workspace capacity; a slot with more IDs than
 * that sets MFET_DEV_CAPACITY and its columns are written as zeros.
 * Calls on one handle must not overlap on the GPU when they use the workspace.
 * Errors: INVALID_ARG, NOT_REGISTERED, WORKSPACE, CUDA. */
MFET_API int mfet_embedding_bag_forward(mfet_tables_t* t, const mfet_batch_shape_t* shape,
                               const uint64_t* ids, const int64_t* offsets, const float* weights,
                               const int32_t* table_ids, const int32_t* pooling, float* out,
                               mfet_stream_t stream);

/* Early fetch for the next batch (paper, Sections 1 and 3.4: the embedding fetch from the
 * CPU side is started as early as possible so that it runs in parallel with the rest of
 * serving and adds no latency). For a batch with exactly ONE host-table slot this runs that
 * slot's hash -> dedup -> cache probe -> fetch of the missed rows now, on the library's
 * internal streams (ordered after what `stream` holds at the call, not joined back to it;
 * the fetch has a stream of its own, so the dedup of one batch runs while the rows of the
 * batch before it still cross PCIe), into one of two result sets of the workspace. The matching mfet_embedding_bag_forward
 * call - same ids/offsets contents, shape.flags | MFET_BATCH_PREFETCHED - then only pools,
 * and gives the same bits as a call without prefetch. At most two prefetches may be
 * outstanding; they are consumed in order. ids/offsets must stay unchanged until the
 * matching forward call has been issued. A forward call without the flag for a batch that
 * has a host-table slot is refused (INVALID_ARG) while a prefetch is outstanding.
 * Errors: INVALID_ARG (not exactly one host-table slot, two prefetches outstanding, ...),
 * NOT_REGISTERED, WORKSPACE, ALIGNMENT, CUDA. */
MFET_API int mfet_host_prefetch(mfet_tables_t* t, const mfet_batch_shape_t* shape, const uint64_t* ids,
                       const int64_t* offsets, const int32_t* table_ids, mfet_stream_t stream);

/* Gradient of the pooled output with respect to the rows of ONE slot's table (paper,
 * Section 4.3: the pretrained tables are fine-tuned inside the ranking model, not frozen),
 * as a sparse list: grad_rows = ascending distinct rows that the slot looked up,
 * grad_vals[k, :] = sum over the lookups i of row grad_rows[k] of
 *     c_i * grad_out[b(i), col_slot : col_slot + dim],
 * c_i = 1 (SUM), 1/len(bag) (MEAN) or weights[i] (WSUM), accumulated in fp32 in an order that depends only
 * on the inputs and the workspace capacity (a row's lookups in input order, long runs in pieces of 64 to 256
 * lookups whose partial sums are added in order), so repeated calls give identical bits.
 *   shape, ids, offsets, weights, table_ids, pooling: as in the forward call
 *   grad_out   dev f32[B, out_ld]: gradient of `out`
 *   slot       which slot's table (0 <= slot < L); its table may live in HBM or host memory
 *   grad_rows  dev i64[n], grad_vals dev f32[n, dim], n_rows dev i64[1]; n = number of IDs
 *              of the slot's feature (at most the workspace capacity)
 * Uses the workspace (the sort of the dedup). Errors: INVALID_ARG, WORKSPACE, CUDA. */
MFET_API int mfet_embedding_bag_backward(mfet_tables_t* t, const mfet_batch_shape_t* shape, const uint64_t* ids,
                                const int64_t* offsets, const float* weights, const int32_t* table_ids,
                                const int32_t* pooling, const float* grad_out, int32_t slot,
                                int64_t* grad_rows, float* grad_vals, int64_t* n_rows, mfet_stream_t stream);

/* In-batch dedup of hashed rows, done before host reads so that each distinct
 * row crosses PCIe once (paper, Section 3.3 motivates keeping host traffic off
 * the latency path). uniq = ascending distinct values of rows[0..n);
 * inverse[i] = position of rows[i] in uniq; *n_unique = their number.
 *   rows dev i64[n] (values in [0, 2^63)); uniq dev i64[n]; inverse dev i32[n];
 *   n_unique dev i64[1]; 0 <= n <= workspace capacity (and n < 2^31).
 *   max_row: exclusive upper bound of the values if known (it shortens the
 *   sort), 0 if unknown. A value >= max_row gives an undefined order.
 * Uses the workspace. Errors: INVALID_ARG, WORKSPACE, CUDA. */
MFET_API int mfet_dedup_rows(mfet_tables_t* t, const int64_t* rows, int64_t n, int64_t* uniq,
                    int32_t* inverse, int64_t* n_unique, int64_t max_row, mfet_stream_t stream);

/* The same dedup for callers that have no device memory to lend and must not
 * ask the driver for any. (This entry point has no counterpart in the paper; it
 * exists for embedding the library in hosts with a closed memory budget.)
 * Typical cases: a plug-in running inside a serving process whose whole GPU
 * memory was handed to another allocator at start-up, so a later cudaMalloc
 * fails or evicts somebody else's pool; a latency-critical request thread, for
 * which cudaMalloc/cudaFree are off limits because they synchronise the whole
 * device; code that holds no table handle and therefore no workspace.
 * Nothing is allocated here, by the library or on its behalf: the sort's
 * scratch is a fixed array compiled into the library, about 6.1 MiB that every
 * GPU using the library holds until the process ends. Hence the limit:
 *   0 <= n <= MFET_STATIC_DEDUP_MAX_IDS, otherwise MFET_ERR_WORKSPACE (use
 *   mfet_dedup_rows with a workspace for larger batches).
 * device: CUDA ordinal of the GPU that owns rows/uniq/inverse/n_unique (0..63);
 * the other arguments and the result are those of mfet_dedup_rows, bit for bit.
 * The first call on each GPU looks up the device address of the built-in array
 * (a runtime query, once per GPU); make that first call outside any stream
 * capture. All calls on a GPU share the one array and it keeps whatever the
 * previous call left (each call overwrites what it reads, nothing needs
 * clearing): two calls whose kernels can overlap on the GPU - different
 * streams without an ordering, or several host threads - race on it and give
 * wrong results; order them on one stream or with events.
 * Errors: INVALID_ARG, WORKSPACE (n too large), CUDA. */
#define MFET_STATIC_DEDUP_MAX_IDS 262144
MFET_API int mfet_dedup_rows_static(int32_t device, const int64_t* rows, int64_t n, int64_t* uniq,
                           int32_t* inverse, int64_t* n_unique, int64_t max_row, mfet_stream_t stream);

/* Device bytes that the hot-row cache of `n` rows of table `table_id` needs. */
MFET_API int mfet_cache_bytes(const mfet_tables_t* t, int32_t table_id, int64_t n, uint64_t* bytes /*host*/);

/* Build the HBM cache of a host table (the paper leaves caching strategies as
 * future work, Section 5; this is the library's): copies the listed rows from
 * the registered host memory into `cache_mem` and builds the lookup index.
 * rows_sorted: host i64[n], strictly increasing, each < rows. cache_mem: dev,
 * 256-byte aligned, caller-owned, at least mfet_cache_bytes(); must stay valid
 * while the handle uses it. n == 0 removes the cache. The call returns after
 * the build has finished on `stream` (it synchronises that stream).
 * Errors: INVALID_ARG, NOT_REGISTERED, ALIGNMENT, WORKSPACE (cache_bytes too small), CUDA. */
MFET_API int mfet_cache_build(mfet_tables_t* t, int32_t table_id, const int64_t* rows_sorted, int64_t n,
                     void* cache_mem, uint64_t cache_bytes, mfet_stream_t stream);

/* Workspace for the host-table path and mfet_dedup_rows: device bytes needed to
 * handle up to `max_ids` IDs per host-table slot per call; max_ids < 2^30 - 1
 * (the dedup hands counts from tile to tile in 30 bits), else INVALID_ARG. */
MFET_API int mfet_workspace_bytes(const mfet_tables_t* t, int64_t max_ids, uint64_t* bytes /*host*/);

/* Attach a caller-owned, 256-byte-aligned device workspace sized by
 * mfet_workspace_bytes(max_ids). It must stay valid while the handle uses it;
 * calls that use it must not overlap on the GPU. */
MFET_API int mfet_set_workspace(mfet_tables_t* t, void* dev_ptr, uint64_t bytes, int64_t max_ids);

/* Same result as mfet_embedding_bag_forward with the batch in HOST memory: the
 * call copies ids/offsets/weights to the device, runs the path, copies `out`
 * back and waits for it. `dev_io` is caller-owned device scratch of at least
 * mfet_host_io_bytes(); host buffers should be pinned for full copy speed.
 * nnz = offsets[F*B]. */
MFET_API int mfet_host_io_bytes(const mfet_tables_t* t, const mfet_batch_shape_t* shape, const int32_t* table_ids,
                       int64_t nnz, uint64_t* bytes /*host*/);
MFET_API int mfet_embedding_bag_forward_host(mfet_tables_t* t, const mfet_batch_shape_t* shape,
                                    const uint64_t* ids_host, const int64_t* offsets_host,
                                    const float* weights_host, int64_t nnz, const int32_t* table_ids,
                                    const int32_t* pooling, float* out_host, void* dev_io,
                                    uint64_t dev_io_bytes, mfet_stream_t stream);

/* The same without the final wait: the copies and kernels are queued on `stream` and the call
 * returns. `out_host` is complete once `stream` has been synchronised (or an event recorded
 * after the call has fired); the host buffers must be pinned and must stay untouched until
 * then, and `dev_io` must not be shared with another call in flight. Two calls on two
 * streams with two `dev_io` buffers overlap one step's result copy with the next step's
 * input copy and kernels. */
MFET_API int mfet_embedding_bag_forward_host_async(mfet_tables_t* t, const mfet_batch_shape_t* shape,
                                    const uint64_t* ids_host, const int64_t* offsets_host,
                                    const float* weights_host, int64_t nnz, const int32_t* table_ids,
                                    const int32_t* pooling, float* out_host, void* dev_io,
                                    uint64_t dev_io_bytes, mfet_stream_t stream);

/* Synthetic table contents (the paper's tables are pretrained weights that are
 * not public; this counter-based generator stands in for them):
 *   k = r*dim + d;  u = splitmix64(value_key + k)
 *   MFET_VAL_NORMAL: s = sum of the four 16-bit fields of u;
 *                    v = float(s - 131070) * fp32(0.01 / 37837.227)
 *   MFET_VAL_GRID:   v = float((u & 255) - 128) * 2^-13
 * rounded to nearest-even into `dtype` (F32 / F16 / BF16). MFET_INT4 (paper, Section
 * 4.1.2: the tables are post-training quantised to INT4; the paper gives no format, this
 * is the library's): per row, scale = fp16((max-min)/15), bias = fp16(min), code =
 * clamp(rint((v - bias)/scale), 0, 15) with the quotient in double precision; stored as
 * dim/2 bytes of codes (element d in the low nibble of byte d/2 when d is even), the fp16
 * scale, the fp16 bias, zero padding to a multiple of 16 bytes. A looked-up element is
 * fma(code, scale, bias) in fp32.
 * data: dev memory, or pinned+mapped host memory (written through the unified
 * address space); rows [row0, row0+n_rows) are written. */
MFET_API int mfet_table_fill(void* data, uint64_t row0, uint64_t n_rows, uint32_t dim, uint32_t dtype,
                    uint64_t row_stride_bytes, uint64_t value_key, uint32_t value_mode,
                    mfet_stream_t stream);

/* Read the device error word (bits MFET_DEV_*) without synchronising: it lives
 * in pinned host memory that kernels write to. clear != 0 resets it. */
MFET_API int mfet_query_status(mfet_tables_t* t, uint32_t* device_error_bits /*host*/, int32_t clear);

/* Tuning knobs. MFET_OPT_GROUP_POLICY: how the pooling kernel maps lanes to
 * bags: 0 = a bag of 64 or more IDs gets a whole warp, a shorter one the lanes that
 * cover one row (default), 1 = one row's lanes for every bag, 2 = a warp for every
 * bag. The result is the same up to the order of fp32 additions. MFET_OPT_TILE:
 * samples per thread block of the pooling kernel: 0 = chosen per launch so that the
 * blocks fill the SMs evenly (default), or 8 .. 128. MFET_OPT_STAGE_IDS:
 * how many IDs of a tile the pooling kernel hashes into shared memory at a time:
 * 0 = default (4096), or 32 .. 8192; a tile with more
 * IDs is pooled in several passes and a bag cut by a pass boundary continues from
 * its partial sum (same result up to the order of fp32 additions).
 * MFET_OPT_OVERLAP_LAUNCHES: 1 = the pooling kernel of a forward call may begin while the
 * kernel launched before it on the same stream is still running (programmatic dependent
 * launch): it reads its offsets, IDs and weights and hashes them, and waits for that kernel
 * to complete before it writes `out` or reads it. Only for callers whose ids / offsets /
 * weights are NOT written by the kernel that precedes the call on the stream (copies that
 * precede it are waited for as usual); back-to-back forward calls then overlap by the
 * start-up phase of a launch. Default 0. MFET_OPT_PROFILE:
 * 1 = record CUDA events around the stages of the host-table path of every forward
 * call (read them with mfet_profile_read). */
MFET_API int mfet_set_option(mfet_tables_t* t, int32_t option, int64_t value);

/* Stage times of the host-table path of the most recent forward call that had a
 * host-table slot, in milliseconds: stage_ms[0] hash + dedup + cache probe,
 * [1] fetch of the missed rows from host memory, [2] pooling. Waits for that
 * call's host-table path to finish. Needs MFET_OPT_PROFILE = 1 (else INVALID_ARG). */
MFET_API int mfet_profile_read(mfet_tables_t* t, float* stage_ms /*host float[3]*/);

/* Distinct rows (n_unique) and distinct rows not found in the HBM cache (n_miss: what
 * crossed PCIe) of the most recent host-table slot that ran. Waits for the internal
 * stream and copies two counters out of the workspace. Errors: INVALID_ARG, WORKSPACE
 * (no workspace attached), CUDA. */
MFET_API int mfet_host_path_counts(mfet_tables_t* t, int64_t* n_unique /*host*/, int64_t* n_miss /*host*/);

/* The intermediate results of the most recent host-table slot that ran (paper, Section 3.3
 * motivates them: only distinct rows that the GPU does not already hold should leave host
 * memory): its distinct rows in ascending order, for each of them where the row is found
 * (src[j] >= 0: that slot of the HBM cache; src[j] < 0: entry -1 - src[j] of the list of rows
 * fetched from host memory), and that list, `miss_rows`, ascending. Counts as returned by
 * mfet_host_path_counts. uniq dev i64[capacity], src dev i32[capacity], miss_rows dev
 * i64[capacity]; any of them may be NULL. Waits for the internal streams and for the copies.
 * Errors: INVALID_ARG (capacity smaller than a count), WORKSPACE (none attached), CUDA. */
MFET_API int mfet_host_path_result(mfet_tables_t* t, int64_t* uniq, int32_t* src, int64_t* miss_rows,
                          int64_t capacity);

/* dst[m, :] = row rows[m] of host table `table_id`, m < n: the zero-copy read of listed rows
 * from the registered host memory (paper, Section 3.3: the largest tables stay in host
 * memory), as the lookup path issues it for the rows that miss the cache. rows dev i64[n],
 * each in [0, table rows); dst dev [n, row bytes], 16-byte aligned. Asynchronous on `stream`.
 * Errors: INVALID_ARG (not a host table, ...), NOT_REGISTERED, ALIGNMENT, CUDA. */
MFET_API int mfet_host_fetch_rows(mfet_tables_t* t, int32_t table_id, const int64_t* rows, int64_t n, void* dst,
                         mfet_stream_t stream);

/* Version tag of a table set (paper, Section 3.3 and Algorithm 2: embeddings travel with the
 * version id of the tables that produced them, so that they are scored by the matching
 * upper model). The library stores the tag and returns it unchanged; the caller sends it
 * along with `out`. Two table sets with different tags can be alive side by side during a
 * roll-out (Algorithm 1). Default tag: 0. */
MFET_API int mfet_tables_set_version(mfet_tables_t* t, uint64_t version);
MFET_API int mfet_tables_version(const mfet_tables_t* t, uint64_t* version /*host*/);

/* Number of kernels the library has launched on behalf of this handle. */
MFET_API int mfet_launch_count(const mfet_tables_t* t, uint64_t* launches /*host*/);

/* Static, human-readable name of a status code. */
MFET_API const char* mfet_status_string(int status);

#ifdef __cplusplus
}
#endif
#endif /* MFET_H_ */
