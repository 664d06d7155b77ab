/*
 * bsa.h -- C ABI of the B200 (sm_100a) forward of dynamic block-sparse attention.
 *
 * A request R = <A, M, B, x> (paper, Section 3 "Online request path" and Section 4.4) supplies a
 * logical block mask M with geometry B = (B_Q, B_KV) and the tensor properties x (here: bf16 or fp16,
 * head dim d in {64, 128, 256}, layout [heads, N, d] or [N, heads, d]; bsa_options_t carries the non-default
 * ones, and N_kv when keys and queries differ in number).  The library computes masked attention
 * (Section 2.1, Eq. 1)
 *
 *     O_M = softmax(Q K^T / sqrt(d) + B_M) V,   B_M = 0 on E(M), -inf elsewhere,
 *
 * plus the fp32 log-sum-exp of each row, touching only physical tiles that cover active blocks.
 *
 * Entry points: bsa_plan_create[_ex|_packed] -> bsa_forward (any number of times) -> bsa_plan_destroy;
 * bsa_request_device (create + forward in one call); bsa_request_host (the same from host buffers);
 * bsa_plan_cache_* (prepared plans reused when the mask repeats); bsa_plan_get_info / bsa_plan_export_* (what
 * was planned); bsa_lut_* / bsa_catalog_* (plan table and catalog); bsa_mask_stats_noalloc.
 *
 * All pointers named *_dev are DEVICE pointers on the current CUDA device; pointers named
 * *_host are HOST pointers.  No function throws; every call returns a status.  `stream` is a
 * cudaStream_t passed as void* (NULL = the legacy default stream).
 */
#ifndef BSA_H_
#define BSA_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define BSA_API __attribute__((visibility("default")))
#else
#define BSA_API
#endif

typedef struct bsa_plan bsa_plan_t; /* opaque; owned by the library */

typedef enum {
    BSA_OK = 0,
    BSA_ERR_INVALID_ARG = 1,      /* null pointer, N <= 0, heads <= 0, ... (GPU untouched)            */
    BSA_ERR_UNSUPPORTED = 2,      /* d not in {64,128,256}; B_Q/B_KV not a power of two in [16,256]  */
    BSA_ERR_NO_ELIGIBLE_PLAN = 3, /* Algorithm 2, last line: no plan of the ranking is eligible      */
    BSA_ERR_OOM = 4,              /* device or host allocation failed                               */
    BSA_ERR_CUDA = 5,             /* a CUDA call failed; see bsa_last_cuda_error()                   */
    BSA_ERR_DEVICE_TIMEOUT = 6,   /* a bounded device-side wait expired (kernel gave up, no hang)    */
    BSA_ERR_LUT = 7               /* plan-table file missing, malformed, or for another catalog      */
} bsa_status_t;

/* Mapping of one dimension of the logical geometry onto the physical tile (Section 4.2). */
enum { BSA_MAP_DIRECT = 0, BSA_MAP_COARSENED = 1, BSA_MAP_REFINED = 2 };
/* Traversal order of the work queue (Section 4.3). */
enum {
    BSA_ORDER_HEAD_MAJOR_LPT = 0,     /* longest first inside each head                                         */
    BSA_ORDER_GLOBAL_LPT = 1,         /* longest first over all heads                                           */
    BSA_ORDER_NATURAL = 2,            /* row-major, unsorted (baseline of the task-organisation ablation)       */
    BSA_ORDER_HEAD_MAJOR_BUCKETS = 3, /* by half-octave length bucket inside each head, row-major inside a bucket */
    BSA_ORDER_GLOBAL_BUCKETS = 4      /* the same over all heads                                                */
};

/* One catalog entry: a physical plan P = <g_Q, g_KV, sigma, e> (Section 4.1).  g_Q and g_KV follow
 * from (B_Q, B_KV) and the tile shape; sigma = {order, split_tau, split_pmax, stages}; e = kernel. */
typedef struct bsa_plan_desc {
    int32_t plan_id;
    int32_t T_Q, T_KV;       /* physical tile geometry                                               */
    int32_t stages;          /* K/V ring depth (pipeline depth); 0 = as many as shared memory holds  */
    int32_t split_tau;       /* a Q tile row with more than tau tiles is split ...                   */
    int32_t split_pmax;      /* ... into at most pmax KV ranges (1 = never split)                    */
    int32_t order;           /* BSA_ORDER_*                                                          */
    int32_t kernel;          /* kernel variant id                                                    */
    char name[48];
} bsa_plan_desc_t;

/* Element type of Q, K, V and O (a tensor property x of the request, Section 4.4).  Scores, softmax state and the
 * output accumulator are fp32 either way; P is rounded to the same 16-bit type for the second product.  Half inputs
 * are served by the single-tile, ping-pong and row-block kernels; the plans of the paired and of the column-split
 * kernel are not eligible for such a request. */
enum { BSA_DTYPE_BF16 = 0, BSA_DTYPE_FP16 = 1 };
/* Storage layout of Q, K, V and O (another tensor property of the request, Section 3 / Section 4.4):
 * [heads][N][d] (head-major, the default) or [N][heads][d] (token-major, what a fused QKV projection of a
 * [batch, sequence, heads, d] model leaves behind).  Only strides change (tensor maps and output addressing); every
 * catalog plan serves both.  LSE is [heads][N] either way. */
enum { BSA_LAYOUT_HND = 0, BSA_LAYOUT_NHD = 1 };

typedef struct bsa_options {
    int32_t force_plan_id;        /* >= 0: skip the lookup and use this catalog entry (still checked for
                                     eligibility); -1: Algorithm 2                                   */
    int32_t dtype;                /* BSA_DTYPE_*: element type of Q, K, V and O (tensor property x)   */
    int64_t max_workspace_bytes;  /* Split-K workspace the request may bind; <= 0: library default   */
    int64_t N_kv;                 /* key/value tokens per head (Section 2.1: K, V are N_kv x d); <= 0: N_kv = N.
                                     The mask then has ceil(N_kv / B_KV) block columns, K and V are
                                     [heads, N_kv, d]; Q, O and LSE keep N rows.                      */
    int32_t layout;               /* BSA_LAYOUT_*                                                     */
    int32_t batch;                /* explicit batch size (the paper's batch is a request dimension, Section 5.1); 0 or 1:
                                     none.  `heads` still counts all independent problems, batch x heads-per-element
                                     (mask [heads, nQb, nKb], LSE [heads, N]), and must be a multiple of it.  With
                                     BSA_LAYOUT_HND the tensors are [batch][heads/batch][N][d], which is [heads][N][d]:
                                     nothing changes.  With BSA_LAYOUT_NHD they are [batch][N][heads/batch][d]: the
                                     plan is then one token-major plan per batch element (each selects its own
                                     catalog plan) and bsa_forward runs them one after the other on the stream;
                                     bsa_plan_get_info sums them, bsa_plan_export_* and the plan cache answer
                                     BSA_ERR_UNSUPPORTED for such a plan.                              */
} bsa_options_t;

/* Scalar mask statistics s_A(M) (Section 5.1) and what launch preparation produced. */
typedef struct bsa_plan_info {
    bsa_plan_desc_t plan;         /* the selected plan                                               */
    int32_t map_q, map_kv;        /* BSA_MAP_* per dimension                                         */
    int32_t heads, d, B_Q, B_KV;
    int64_t N;
    int32_t nQb, nKb, nQt, nKt;   /* logical block grid and physical tile grid per head              */
    int32_t member_bits;          /* membership bits per 128-row slot (1 = no intra-tile mask needed) */
    int32_t lut_hit;              /* 1: regime found in the plan table; 0: base plan used            */
    int32_t regime_bucket[4];     /* N, density, skew, run-coverage bucket indices used for lookup   */
    int64_t nnz_blocks;           /* active logical blocks                                           */
    int64_t blocks_in_runs;       /* active blocks in runs of length >= 2                            */
    int32_t max_row_nnz;
    int32_t member_words;         /* 64-bit membership words per tile: one per 128-row slot (T_Q / 128) */
    double density, run_coverage, skew;
    int64_t ntiles;               /* physical tiles                                                  */
    int64_t nitems;               /* work items (Q tile rows x KV partitions)                        */
    int64_t nsplit_rows;          /* 128-row tile rows merged by the Split-K reduction kernel        */
    int64_t workspace_bytes;      /* Split-K workspace owned by the plan                             */
    int64_t covered_pairs;        /* token pairs the tiles compute, incl. masked-out ones            */
    /* host wall time of bsa_plan_create, microseconds */
    float us_mask_state;          /* launch of the mask-state kernels                                */
    float us_stats_sync;          /* waiting for + copying the scalar statistics                     */
    float us_lookup;              /* regime lookup + ranked fallback + eligibility                   */
    float us_launch_prep;         /* CSR fill, tile mapping, task organisation (launch + allocs)    */
    float us_total;
    int32_t device_status;        /* 0, or BSA_ERR_DEVICE_TIMEOUT if any forward hit a bounded wait  */
    int64_t N_kv;                 /* key/value tokens per head (= N unless the options said otherwise) */
    int32_t dtype;                /* BSA_DTYPE_* of the request                                        */
    int32_t layout;               /* BSA_LAYOUT_* of the request                                       */
} bsa_plan_info_t;

/* ---------------------------------------------------------------------------------------------
 * bsa_plan_create -- online plan selection and launch preparation (Section 5.2, Algorithm 2).
 *
 * Builds the shared mask state mu(M) on the GPU (block-CSR offsets, active KV column indices and
 * the scalar statistics), passes only the scalars to the host (the one synchronisation of the
 * call), looks up the regime in the loaded plan table, takes the first eligible plan of its
 * ranking (base plan on a miss), then derives that plan's metadata on the GPU: physical tile
 * lists with membership bits (Direct / Coarsened / Refined mapping, Section 4.2), work items per Q
 * tile row, Split-K partitions of heavy rows, longest-first order (Section 4.3).
 *
 *   mask_dev : uint8 [heads, ceil(N/B_Q), ceil(N_kv/B_KV)], row-major, nonzero = active block.
 *              Borrowed: read by kernels this call submits to `stream`; it may be freed or
 *              overwritten by work ordered after the call on that stream (or after a stream sync).
 *   B_Q,B_KV : logical block geometry, powers of two in [16, 256].
 *   N        : query tokens per head, N_q of Section 2.1; need not be a multiple of the block sizes.
 *              The key/value token count N_kv equals N unless options->N_kv says otherwise (_ex variants).
 *   heads    : independent (batch x head) problems.
 *   d        : head dimension, 64, 128 or 256 (256: served by the single-tile kernels with 64-key tiles, whose
 *              256-column output accumulator fills half of tensor memory).  Scale is 1/sqrt(d);
 *              attention is non-causal.
 *   out_plan : receives the plan; the plan owns its device buffers (CSR, tile lists, work items,
 *              Split-K workspace).  Reusable for any number of forwards with the same mask.
 *
 * Runs on the legacy default stream (the _ex variant takes a stream and options) and returns after
 * the statistics copy; the remaining preparation kernels are stream-ordered before any forward
 * submitted to the same stream.  A forward on ANOTHER stream must be ordered after the create by the caller.
 * Errors: INVALID_ARG / UNSUPPORTED (GPU untouched), NO_ELIGIBLE_PLAN, OOM, CUDA.
 */
BSA_API bsa_status_t bsa_plan_create(const uint8_t* mask_dev, int B_Q, int B_KV, int64_t N, int heads, int d,
                             bsa_plan_t** out_plan);
BSA_API bsa_status_t bsa_plan_create_ex(const uint8_t* mask_dev, int B_Q, int B_KV, int64_t N, int heads, int d,
                                const bsa_options_t* options /* may be NULL */, void* stream,
                                bsa_plan_t** out_plan);

/* The same for a bit-packed mask (the paper does not fix a mask format, Section 2.1 only defines M; this variant has
 * no counterpart there).  Row (h, qb) starts at mask_bits_dev + (h * nQb + qb) * row_stride_bytes; block column c of
 * the row is bit (c & 7) of its byte c >> 3 (1 = active; numpy.packbits(..., bitorder="little")).  Bits at or beyond
 * nKb and the padding bytes of a row are ignored.  mask_bits_dev must be 4-byte aligned and row_stride_bytes a
 * multiple of 4 that holds nKb bits, else INVALID_ARG (GPU untouched).  Device memory, borrowed for the call.  The
 * planner then reads one eighth of the byte format's mask traffic; everything downstream is identical, and so is
 * every output (the GPU tests compare the two plans' exported structures and outputs bit for bit). */
BSA_API bsa_status_t bsa_plan_create_packed(const uint8_t* mask_bits_dev, int64_t row_stride_bytes, int B_Q, int B_KV,
                                    int64_t N, int heads, int d, const bsa_options_t* options /* may be NULL */,
                                    void* stream, bsa_plan_t** out_plan);

/* ---------------------------------------------------------------------------------------------
 * bsa_forward -- execute the plan's native kernels (Section 4: main attention kernel, then the
 * Split-K reduction kernel when the plan has partitions).
 *
 *   Q     : bf16 (fp16 if the plan was created with options->dtype = BSA_DTYPE_FP16) [heads, N, d], d contiguous,
 *           16-byte aligned base, device memory, borrowed.
 *   K,V   : the same type, [heads, N_kv, d] (N_kv = N unless the plan was created with options->N_kv).
 *   O     : the same type, [heads, N, d], written for every row; rows with no active block get 0.
 *   LSE   : fp32 [heads, N], natural-log log-sum-exp of the scaled scores over E(M); -inf for rows
 *           with no active block.
 *
 * Asynchronous on `stream`; no host synchronisation.  Forwards that share a plan must be
 * stream-ordered (they share the Split-K workspace).  A bounded device wait that expires is
 * recorded in the plan (see bsa_plan_get_info().device_status) -- the kernel returns, it never hangs.
 * Errors: INVALID_ARG (null or misaligned pointers), CUDA.
 */
BSA_API bsa_status_t bsa_forward(const bsa_plan_t* plan, const void* Q_dev, const void* K_dev, const void* V_dev,
                         void* O_dev, float* LSE_dev, void* stream);

/* One cold request on device buffers in a single call: bsa_plan_create_ex (row_stride_bytes = 0) or
 * bsa_plan_create_packed (> 0) followed by bsa_forward on the same stream, arguments as there.  The forward is
 * queued before the call returns, which saves a caller in an interpreted language the second trip through its
 * foreign-function layer (on the 200-us Mid request that trip is hidden behind the preparation kernels and the
 * single call measures the same).  *out_plan receives the plan (reusable
 * for further forwards; give it back with bsa_plan_destroy); on any error nothing is returned and nothing is kept.
 * Errors: those of the two calls; the pointer checks of bsa_forward come first (GPU untouched). */
BSA_API bsa_status_t bsa_request_device(const uint8_t* mask_dev, int64_t row_stride_bytes, int B_Q, int B_KV, int64_t N,
                                int heads, int d, const void* Q_dev, const void* K_dev, const void* V_dev, void* O_dev,
                                float* LSE_dev, const bsa_options_t* options /* may be NULL */, void* stream,
                                bsa_plan_t** out_plan);

/* Lets go of the plan.  A plan from bsa_plan_create* is freed with every device buffer it owns, and the call
 * synchronises with the plan's create stream.  A plan from bsa_plan_cache_get is shared: the call only drops the
 * caller's hold (no synchronisation) unless it was the last one.
 * The buffers go back to the memory pool in the create stream's order.  Forwards submitted to OTHER streams are
 * covered: every such bsa_forward leaves an event behind it that the free waits for, so the plan may be destroyed
 * (or evicted from a cache) right after the call returns.  The one exception is a forward recorded into a CUDA
 * graph: keep the plan alive until the last replay of that graph has completed. */
BSA_API bsa_status_t bsa_plan_destroy(bsa_plan_t* plan);

/* ---------------------------------------------------------------------------------------------
 * Plan cache -- the warm path of Section 5.2 (measured in Section 7.4, Table 7): while the mask stays the same across
 * layers or denoising steps, the prepared plan is reused and only the attention kernels run.  The
 * paper leaves the reuse to the caller; this cache recognises a repeated mask by itself.
 *
 * bsa_plan_cache_get runs the mask-statistics kernel (as bsa_plan_create does), which here also sums
 * a 128-bit position-salted fingerprint of the activity pattern, and looks up
 * (fingerprint, B_Q, B_KV, N, heads, d, mask format and alignment, options, device, plan-table
 * generation).  Hit: the prepared plan is returned (*out_hit = 1), nothing else is launched; if the
 * plan was prepared on another stream, `stream` is first made to wait for that preparation.  Miss:
 * the plan is prepared exactly as by bsa_plan_create_ex / bsa_plan_create_packed, kept in the cache
 * and returned (*out_hit = 0); beyond `capacity` plans the least recently used one is dropped.
 * Two different masks collide only if both 64-bit sums agree (no comparison of the masks follows).
 * A collision would hand back the plan of the OTHER mask: the forward would then attend over that
 * mask's blocks and return a wrong O and LSE without any error.  For masks that differ by accident the
 * chance is about 2^-128 per pair; a caller that must rule it out (masks chosen by an adversary) uses
 * bsa_plan_create* and keeps the plans itself.
 *
 *   row_stride_bytes : 0 = one byte per logical block (as bsa_plan_create); > 0 = bit-packed rows
 *                      (as bsa_plan_create_packed).  mask_dev is device memory, borrowed for the call.
 *   out_plan         : shared with the cache and with every other caller that got the same plan;
 *                      give it back with bsa_plan_destroy.  Forwards on one plan must be
 *                      stream-ordered (they share the Split-K workspace).
 *   out_hit          : may be NULL.
 * bsa_lut_load, bsa_lut_clear and bsa_force_plan start a new generation: plans selected before are
 * not returned afterwards.  All four calls are thread-safe.  bsa_plan_cache_destroy drops the
 * cache's holds (plans still held by callers stay valid) and synchronises with the create streams
 * of the plans it frees.  Errors: as bsa_plan_create_ex; INVALID_ARG for a null cache, capacity < 1
 * or a negative stride.
 */
typedef struct bsa_plan_cache bsa_plan_cache_t;
BSA_API bsa_status_t bsa_plan_cache_create(int capacity, bsa_plan_cache_t** out_cache);
BSA_API bsa_status_t bsa_plan_cache_get(bsa_plan_cache_t* cache, const uint8_t* mask_dev, int64_t row_stride_bytes, int B_Q,
                                int B_KV, int64_t N, int heads, int d, const bsa_options_t* options /* may be NULL */,
                                void* stream, bsa_plan_t** out_plan, int* out_hit);
/* bsa_plan_cache_get followed by bsa_forward on the same stream, in one call (as bsa_request_device is for
 * bsa_plan_create_ex): on a hit nothing lies between the arrival of the mask fingerprint and the launch of the
 * attention kernel but the table lookup.  *out_plan as for bsa_plan_cache_get (give it back with bsa_plan_destroy). */
BSA_API bsa_status_t bsa_plan_cache_request(bsa_plan_cache_t* cache, const uint8_t* mask_dev, int64_t row_stride_bytes,
                                    int B_Q, int B_KV, int64_t N, int heads, int d, const void* Q_dev, const void* K_dev,
                                    const void* V_dev, void* O_dev, float* LSE_dev,
                                    const bsa_options_t* options /* may be NULL */, void* stream, bsa_plan_t** out_plan,
                                    int* out_hit);
BSA_API bsa_status_t bsa_plan_cache_stats(bsa_plan_cache_t* cache, int64_t* hits, int64_t* misses, int64_t* evictions,
                                  int32_t* entries);
BSA_API bsa_status_t bsa_plan_cache_destroy(bsa_plan_cache_t* cache);

/* ---------------------------------------------------------------------------------------------
 * bsa_request_host -- one complete request from HOST buffers: copies mask, Q, K, V to the device,
 * creates the plan, runs the forward, copies O and LSE back, frees everything.  Same results as
 * the three calls above; used to measure end-to-end request cost including transfers.  Heads are
 * independent, so with the head-major layout the request is cut into up to 8 groups of heads (of
 * more than 32 MB of Q, K and V; smaller towards the end of the request where a single head already
 * has that much, so that little is left to do after the last input byte) that are pipelined: a
 * group's inputs travel while the previous group is planned and computed and the one before travels
 * back (pinned host buffers are needed for the copies to overlap).  Each group selects its own plan
 * from its own part of the mask.
 *   info_out (optional) receives the request's info: counts and times summed over the groups,
 *   statistics of the whole mask, the first group's plan.
 */
BSA_API bsa_status_t bsa_request_host(const uint8_t* mask_host, int B_Q, int B_KV, int64_t N, int heads, int d,
                              const void* Q_host, const void* K_host, const void* V_host,
                              void* O_host, float* LSE_host, const bsa_options_t* options,
                              bsa_plan_info_t* info_out);

/* ---------------------------------------------------------------------------------------------
 * bsa_mask_stats_noalloc -- the scalar mask statistics s_A(M) for callers that cannot allocate.
 * (The paper has no counterpart: its runtime always builds the statistics as part of plan selection.)
 *
 * Meant for hosts where a call into the CUDA allocator is off limits: a serving process that gave
 * all device memory to its own pool at start-up, a plug-in that lives under another component's
 * allocation policy, a loop that cannot afford the device-wide synchronisation or the late failure
 * of a cudaMalloc.  This call performs no cudaMalloc / cudaMallocAsync / cudaFree and uses no
 * allocating library routine.  Its scratch memory (one int32 counter per mask row plus three
 * accumulators) is a fixed array inside the library's device image: 256 + 4 * BSA_NOALLOC_MAX_ROWS
 * bytes (about 4 MiB), resident on every GPU that loads the library until the process exits.
 *
 *   mask_dev      : uint8 [heads, nQb, nKb], nonzero = active block (device, borrowed).
 *   stats_out_dev : int64 [4] in DEVICE memory, written on `stream`:
 *                   {active blocks, active blocks in runs of length >= 2, largest row count,
 *                    rows with no active block}.
 *   heads * nQb must not exceed BSA_NOALLOC_MAX_ROWS; larger masks are rejected with
 *   BSA_ERR_UNSUPPORTED before anything is launched.
 *
 * The first call on a device resolves the array's device address (cudaGetSymbolAddress) with that
 * device current.  Under CUDA's default lazy module loading that first call is also when the driver
 * loads the library's module onto the device and reserves the array (and the module's code) there,
 * so it is the one call that can still fail for lack of device memory (BSA_ERR_CUDA).  Make it once
 * per device at start-up: before the host hands the device's memory to its own pool, and before any
 * stream capture.  Later calls on that device touch neither the allocator nor the module loader
 * (the GPU test checks that the driver's free-memory figure does not move across them).  Host
 * threads that make their first call on a device concurrently all resolve and store the same
 * address; that is harmless.
 * All calls on a device share the one array, which still holds the previous call's data: the
 * accumulators are cleared on `stream` at the start of every call.  Two calls whose GPU work
 * overlaps (different streams, or different host threads) race on the array and give wrong results:
 * keep them stream-ordered.
 * Errors: INVALID_ARG (null pointers, non-positive sizes), UNSUPPORTED (too many rows), CUDA.
 */
#define BSA_NOALLOC_MAX_ROWS (1 << 20)
BSA_API bsa_status_t bsa_mask_stats_noalloc(const uint8_t* mask_dev, int heads, int nQb, int nKb,
                                    int64_t* stats_out_dev, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Introspection (tests, benches, the offline profiler).  These synchronise with the plan's stream.
 */
BSA_API bsa_status_t bsa_plan_get_info(const bsa_plan_t* plan, bsa_plan_info_t* info_out);

/* Block-CSR of the shared mask state: row_ptr_host int32 [heads*nQb + 1], col_idx_host int32
 * [nnz_blocks] (pass NULL to skip either).  Rows are (head, query block) in row-major order. */
BSA_API bsa_status_t bsa_plan_export_csr(const bsa_plan_t* plan, int32_t* row_ptr_host, int32_t* col_idx_host);

/* Physical tiles of one head, for the coverage check (a plan must preserve E(M), Section 2.2):
 *   tile_row_ptr_host int32 [nQt + 1]  offsets into the two arrays below (relative to this head),
 *   tile_col_host     int32 [cap]      KV tile index, ascending and unique inside a row,
 *   tile_member_host  uint64 [cap * W] membership words, W = T_Q / 128 per tile (info.member_words), one
 *                                      per 128-row slot of the tile: bit (a * sK + b) of word s set iff
 *                                      logical sub-block (a, b) of slot s is active, sK = max(1, T_KV / B_KV),
 *                                      a < max(1, 128 / B_Q), b < sK.  A zero word: the slot skips the tile.
 * `cap` is the capacity of the two arrays in entries; *ntiles_out receives the number needed
 * (call with cap = 0 and NULL arrays to size them). */
BSA_API bsa_status_t bsa_plan_export_tiles(const bsa_plan_t* plan, int head, int32_t* tile_row_ptr_host,
                                   int32_t* tile_col_host, uint64_t* tile_member_host, int64_t cap,
                                   int64_t* ntiles_out);

/* Work items in queue order: 8 int32 per item {head, q_tile, tile_begin, tile_end, part, nparts,
 * ws_slot, ntiles}; tile_begin/end index the plan's global tile arrays.  Sizing as above. */
BSA_API bsa_status_t bsa_plan_export_items(const bsa_plan_t* plan, int32_t* items_host, int64_t cap, int64_t* nitems_out);

/* ---------------------------------------------------------------------------------------------
 * Catalog C_A and plan table Pi_A (Section 4.4, Section 5).
 */
BSA_API int bsa_catalog_size(void);
BSA_API bsa_status_t bsa_catalog_get(int index, bsa_plan_desc_t* out);
/* Eligible(P, R) (Section 4.4): geometry, head dim, membership format and workspace. */
BSA_API int bsa_plan_eligible(int plan_id, int B_Q, int B_KV, int64_t N, int heads, int d, int64_t max_workspace_bytes);
/* The same with every request property eligibility looks at: N_kv (<= 0: N_kv = N) and the element type
 * (BSA_DTYPE_*).  bsa_plan_eligible is this call with N_kv = N and bf16. */
BSA_API int bsa_plan_eligible_ex(int plan_id, int B_Q, int B_KV, int64_t N, int64_t N_kv, int heads, int d, int dtype,
                                 int64_t max_workspace_bytes);
/* Base plan of a request key (eligible for every request with that key). */
BSA_API int bsa_base_plan(int B_Q, int B_KV, int d);
/* Hash of the catalog contents; a plan table built for another catalog is rejected. */
BSA_API uint64_t bsa_catalog_hash(void);

/* Load the versioned plan table (text file written by the offline profiler).  Replaces any table
 * loaded before.  On error the previous table is dropped and base plans are used. */
BSA_API bsa_status_t bsa_lut_load(const char* path);
BSA_API void bsa_lut_clear(void);
BSA_API int bsa_lut_num_regimes(void);
/* Request keys for which the loaded table holds a learned second-stage partition (Section 5.1: thresholds learned by
 * a decision tree over log2 N, heads, density, skew and run coverage; its leaves are regimes too).  A request is
 * looked up in the regimes of the fixed bucket edges first; if the table has no such regime, in its key's tree; if the
 * key has no tree either, the base plan is used.  In bsa_plan_info_t a tree lookup shows as lut_hit = 1 with
 * (leaf index + 1) << 8 added to regime_bucket[3]. */
BSA_API int bsa_lut_num_trees(void);
/* Regime lookup + ranked fallback only (no GPU): returns the plan id Algorithm 2 selects for these
 * request scalars, or -1 for no-eligible-plan.  *hit_out (optional) = 1 if the regime was found. */
BSA_API int bsa_lut_select(int B_Q, int B_KV, int64_t N, int heads, int d, double density, double run_coverage,
                   double skew, int64_t max_workspace_bytes, int* hit_out);
/* Bucket edges of the feature schema F_A, so the offline profiler partitions cases exactly as the
 * runtime does: writes the bucket indices {N, density, skew, run coverage} for the given scalars. */
BSA_API void bsa_lut_buckets(int64_t N, double density, double skew, double run_coverage, int32_t out[4]);

/* Process-wide default used when options->force_plan_id is not given: >= 0 forces a plan,
 * -1 restores Algorithm 2. */
BSA_API void bsa_force_plan(int plan_id);

/* ---------------------------------------------------------------------------------------------
 * Test hooks for the give-up path of the kernels' bounded waits (no counterpart in the paper).
 * Every wait inside the attention kernels (on a copy, an MMA, another warp) has a limit in SM clock
 * cycles; when it runs out the CTA records BSA_ERR_DEVICE_TIMEOUT in the plan's device_status, lets
 * its copies in flight land, frees its tensor memory and returns.  Both settings are per device
 * (the current one), apply to forwards launched afterwards, and synchronise the device.
 *   bsa_debug_set_wait_limit(cycles)   : the limit; <= 0 restores the default (2e9 cycles, about 1 s).
 *   bsa_debug_withhold_arrival(on)     : while on, the ping-pong kernel's V producer leaves out the
 *                                        copy of each CTA's first tile and the arrival announcing it,
 *                                        so the waits behind it run out.  Nothing faults; O and LSE
 *                                        of such a forward are undefined.
 */
BSA_API bsa_status_t bsa_debug_set_wait_limit(long long cycles);
/* Measurement hook: launches the Split-K reduction kernel of a plan alone on `stream`, over the partial results the
 * plan's last forward left in its workspace (so it can be timed by itself; O_dev and LSE_dev are written as by that
 * forward).  UNSUPPORTED for a plan without Split-K partitions. */
BSA_API bsa_status_t bsa_debug_merge_only(const bsa_plan_t* plan, void* O_dev, float* LSE_dev, void* stream);
BSA_API bsa_status_t bsa_debug_withhold_arrival(int on);

BSA_API const char* bsa_status_string(bsa_status_t s);
BSA_API const char* bsa_last_cuda_error(void);
BSA_API const char* bsa_version(void);
/* Number of this library's kernels launched since load (all plans, all streams). */
BSA_API int64_t bsa_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* BSA_H_ */
