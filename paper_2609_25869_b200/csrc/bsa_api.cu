// C ABI: online request path (paper Section 3 "Online request path", Section 5.2, Algorithm 2).
#include <math.h>
#include <stdio.h>
#include <string.h>
#include <time.h>

#include <atomic>
#include <list>
#include <mutex>
#include <new>
#include <unordered_map>

#include "bsa_common.h"

namespace bsa {
// bsa_lut.cpp
const bsa_plan_desc_t* catalog_entry(int plan_id);
bool make_geom(const bsa_plan_desc_t& P, int B_Q, int B_KV, int64_t N, int64_t N_kv, int heads, MapGeom* g);
int64_t plan_workspace_bytes(const bsa_plan_desc_t& P, int64_t N, int heads, int d);
bool plan_eligible(int plan_id, int B_Q, int B_KV, int64_t N, int heads, int d, int64_t max_ws, int64_t N_kv = 0,
                   int dtype = BSA_DTYPE_BF16);
int base_plan(int B_Q, int B_KV, int d);
uint64_t catalog_hash();
void lut_buckets(int64_t N, double density, double skew, double run_cov, int32_t out[4]);
void lut_clear();
int lut_num_regimes();
int lut_num_trees();
bsa_status_t lut_load(const char* path);
void set_force_plan(int id);
int get_force_plan();
int lut_select(int B_Q, int B_KV, int64_t N, int heads, int d, double density, double run_cov, double skew,
               int64_t max_ws, int* hit_out, int32_t buckets_out[4], int64_t N_kv = 0, int dtype = BSA_DTYPE_BF16);
int catalog_size();

static std::atomic<long long> g_launches{0};
// bumped whenever the plan table or the forced plan changes: cached plans selected before that are not reused
static std::atomic<unsigned> g_select_generation{0};
void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

static thread_local char g_cuda_err[256] = "";
static void set_cuda_err(cudaError_t e, const char* where) {
    snprintf(g_cuda_err, sizeof g_cuda_err, "%s: %s", where, cudaGetErrorString(e));
}

static double now_us() {
    timespec ts;
    clock_gettime(CLOCK_MONOTONIC, &ts);
    return ts.tv_sec * 1e6 + ts.tv_nsec * 1e-3;
}

static size_t align_up(size_t v, size_t a = 256) { return (v + a - 1) / a * a; }
}  // namespace bsa

using namespace bsa;

struct bsa_plan {
    bsa_plan_desc_t desc;
    MapGeom g;
    int d;
    int dtype;  // BSA_DTYPE_*
    int layout;  // BSA_LAYOUT_*
    int stages;
    cudaStream_t stream;
    int device;
    int num_sms;
    // arena 1 (allocated before the statistics copy)
    uint8_t* arena1;
    int32_t* row_nnz;
    int32_t* row_ptr;
    MaskStatsDev* stats;
    PlanCountersDev* counters;
    int32_t* head_counts;
    // arena 2 (sized from the statistics)
    uint8_t* arena2;
    int32_t* col_idx;
    int32_t* tile_begin;
    int32_t* tile_cnt;
    int32_t* row_parts;
    int32_t* tile_col;
    uint64_t* tile_member;
    WorkItem* items_tmp;
    WorkItem* items;
    SplitRow* split_rows;
    int64_t tile_cap;
    int64_t max_items;
    // Split-K workspace
    float* ws_O;
    float* ws_LSE;
    int64_t ws_bytes;
    // host-side record
    MaskStatsDev hstats;
    int lut_hit;
    int32_t buckets[4];
    float us_mask_state, us_stats_sync, us_lookup, us_launch_prep, us_total;
    // sharing (plan cache): the plan is freed when the last holder lets go; `ready` (cached plans only) is recorded
    // behind the preparation kernels so that a later request on another stream can wait for them
    std::atomic<int> refs;
    cudaEvent_t ready;
    // Recorded behind every forward that was submitted to a stream other than the plan's own (created at the first
    // such forward): the plan's buffers go back to the pool in the create stream's order, so that stream waits for
    // this event first.  Forwards on one plan are stream-ordered among themselves, so the latest record covers all.
    std::atomic<cudaEvent_t> last_use;
    // Batched token-major request (options->batch > 1 with BSA_LAYOUT_NHD): the plan is a list of per-batch-element
    // plans (each an ordinary token-major request over heads / batch heads) and owns nothing else on the device.
    bsa_plan** kids;
    int nkids;
};

// ---- plan cache (warm path of Section 5.2: a prepared plan is reused while the mask stays the same) ----
namespace {
struct CacheKey {
    uint64_t hash[2];
    int64_t N, N_kv, packed_stride, max_ws;
    int32_t B_Q, B_KV, heads, d, align, force, device, dtype, layout, pad;
    uint32_t generation;
    bool operator==(const CacheKey& o) const { return memcmp(this, &o, sizeof *this) == 0; }
};
struct CacheKeyHash {
    size_t operator()(const CacheKey& k) const { return (size_t)(k.hash[0] ^ (k.hash[1] * 0x9E3779B97F4A7C15ull)); }
};
}  // namespace
struct bsa_plan_cache {
    std::mutex mu;
    int capacity;
    std::list<std::pair<CacheKey, bsa_plan*>> lru;  // most recently used first
    std::unordered_map<CacheKey, std::list<std::pair<CacheKey, bsa_plan*>>::iterator, CacheKeyHash> index;
    int64_t hits, misses, evictions;
};

static bsa_status_t validate(const void* mask, int B_Q, int B_KV, int64_t N, int heads, int d, void* out) {
    if (!mask || !out || N <= 0 || heads <= 0) return BSA_ERR_INVALID_ARG;
    auto p2 = [](int v) { return v >= 16 && v <= 256 && (v & (v - 1)) == 0; };
    if (!(d == 64 || d == 128 || d == 256) || !p2(B_Q) || !p2(B_KV)) return BSA_ERR_UNSUPPORTED;
    if (N > (1ll << 30)) return BSA_ERR_UNSUPPORTED;
    return BSA_OK;
}
// key/value tokens per head of a request: the options' N_kv, else N
static int64_t request_n_kv(const bsa_options_t* options, int64_t N) {
    return (options && options->N_kv > 0) ? options->N_kv : N;
}

static bool release_plan(bsa_plan* p);
static void free_plan(bsa_plan* p) {
    if (!p) return;
    if (p->kids) {
        for (int b = 0; b < p->nkids; ++b)
            if (p->kids[b]) release_plan(p->kids[b]);
        delete[] p->kids;
    }
    if (p->ready) cudaEventDestroy(p->ready);
    if (cudaEvent_t lu = p->last_use.load(std::memory_order_acquire)) {
        // a forward on another stream may still be reading the arenas and the workspace
        cudaStreamWaitEvent(p->stream, lu, 0);
        cudaEventDestroy(lu);
    }
    if (p->arena1) cudaFreeAsync(p->arena1, p->stream);
    if (p->arena2) cudaFreeAsync(p->arena2, p->stream);
    if (p->ws_O) cudaFreeAsync(p->ws_O, p->stream);
    delete p;
}

#define BSA_CUDA(call, where)            \
    do {                                 \
        cudaError_t e__ = (call);        \
        if (e__ != cudaSuccess) {        \
            set_cuda_err(e__, where);    \
            free_plan(p);                \
            return e__ == cudaErrorMemoryAllocation ? BSA_ERR_OOM : BSA_ERR_CUDA; \
        }                                \
    } while (0)

// one holder lets go of the plan; the last one frees it (stream-ordered on the plan's create stream, no wait)
static bool release_plan(bsa_plan* p) {
    if (p->refs.fetch_sub(1, std::memory_order_acq_rel) > 1) return false;
    free_plan(p);
    return true;
}

// `packed_stride` = 0: one byte per logical block; > 0: bit-packed rows of that many bytes (bsa_plan_create_packed).
// `cache` (may be null): look the mask up after the statistics have arrived and reuse the prepared plan on a hit.
static bsa_status_t create_impl(const uint8_t* mask_dev, int64_t packed_stride, int B_Q, int B_KV, int64_t N, int heads,
                                int d, const bsa_options_t* options, void* stream_v, bsa_plan_t** out_plan,
                                bsa_plan_cache* cache = nullptr, int* cache_hit = nullptr) {
    bsa_status_t vs = validate(mask_dev, B_Q, B_KV, N, heads, d, out_plan);
    if (vs != BSA_OK) return vs;
    const int64_t N_kv = request_n_kv(options, N);
    if (N_kv > (1ll << 30)) return BSA_ERR_UNSUPPORTED;
    const int dtype = options ? options->dtype : BSA_DTYPE_BF16;
    if (dtype != BSA_DTYPE_BF16 && dtype != BSA_DTYPE_FP16) return BSA_ERR_UNSUPPORTED;
    const int layout = options ? options->layout : BSA_LAYOUT_HND;
    if (layout != BSA_LAYOUT_HND && layout != BSA_LAYOUT_NHD) return BSA_ERR_UNSUPPORTED;
    const int batch = (options && options->batch > 1) ? options->batch : 1;
    if (options && options->batch < 0) return BSA_ERR_INVALID_ARG;
    if (batch > 1 && heads % batch != 0) return BSA_ERR_INVALID_ARG;
    if (batch > 1 && layout == BSA_LAYOUT_NHD) {
        // [batch][N][heads / batch][d] tensors: one ordinary token-major plan per batch element (in the head-major
        // layout the batch folds into `heads` exactly and nothing has to be done)
        if (cache) return BSA_ERR_UNSUPPORTED;
        *out_plan = nullptr;
        bsa_plan* parent = new (std::nothrow) bsa_plan();
        if (!parent) return BSA_ERR_OOM;
        memset(static_cast<void*>(parent), 0, sizeof *parent);
        parent->refs.store(1, std::memory_order_relaxed);
        parent->last_use.store(nullptr, std::memory_order_relaxed);
        parent->stream = reinterpret_cast<cudaStream_t>(stream_v);
        parent->d = d;
        parent->dtype = dtype;
        parent->layout = layout;
        parent->kids = new (std::nothrow) bsa_plan*[batch]();
        if (!parent->kids) { delete parent; return BSA_ERR_OOM; }
        parent->nkids = batch;
        const int hb = heads / batch;
        const int64_t nQb64 = (N + B_Q - 1) / B_Q, nKb64 = (N_kv + B_KV - 1) / B_KV;
        const int64_t mask_step = packed_stride > 0 ? (int64_t)hb * nQb64 * packed_stride : (int64_t)hb * nQb64 * nKb64;
        bsa_options_t kid_opt = *options;
        kid_opt.batch = 0;
        for (int b = 0; b < batch; ++b) {
            bsa_status_t st = create_impl(mask_dev + (size_t)b * mask_step, packed_stride, B_Q, B_KV, N, hb, d, &kid_opt, stream_v,
                                          &parent->kids[b]);
            if (st != BSA_OK) {
                free_plan(parent);
                return st;
            }
        }
        MapGeom& pg = parent->g;  // enough of the geometry for bsa_forward's pointer steps and bsa_plan_get_info
        pg = parent->kids[0]->g;
        pg.H = heads;
        parent->desc = parent->kids[0]->desc;
        *out_plan = parent;
        return BSA_OK;
    }
    if (packed_stride > 0) {
        const int64_t nKb64 = (N_kv + B_KV - 1) / B_KV;
        if (packed_stride % 4 != 0 || packed_stride * 8 < nKb64 || (reinterpret_cast<uintptr_t>(mask_dev) & 3u))
            return BSA_ERR_INVALID_ARG;
    }
    *out_plan = nullptr;
    const double t0 = now_us();
    cudaStream_t stream = reinterpret_cast<cudaStream_t>(stream_v);
    bsa_plan* p = new (std::nothrow) bsa_plan();
    if (!p) return BSA_ERR_OOM;
    memset(static_cast<void*>(p), 0, sizeof *p);
    p->refs.store(1, std::memory_order_relaxed);
    p->last_use.store(nullptr, std::memory_order_relaxed);
    p->stream = stream;
    p->d = d;
    p->dtype = dtype;
    p->layout = layout;
    BSA_CUDA(cudaGetDevice(&p->device), "cudaGetDevice");
    BSA_CUDA(cudaDeviceGetAttribute(&p->num_sms, cudaDevAttrMultiProcessorCount, p->device), "device attribute");
    {
        // Plans are created and destroyed per request: keep freed arena memory in this process's default
        // stream-ordered pool instead of handing it back to the driver at every synchronisation (the
        // default threshold of 0 makes each larger request pay a fresh driver allocation, 10-80 ms).
        static std::atomic<unsigned long long> pool_ready_mask{0};
        const unsigned long long bit = 1ull << (p->device & 63);
        if (!(pool_ready_mask.load(std::memory_order_relaxed) & bit)) {
            cudaMemPool_t pool;
            if (cudaDeviceGetDefaultMemPool(&pool, p->device) == cudaSuccess) {
                unsigned long long keep = ~0ull;
                cudaMemPoolSetAttribute(pool, cudaMemPoolAttrReleaseThreshold, &keep);
            }
            pool_ready_mask.fetch_or(bit, std::memory_order_relaxed);
        }
    }

    const int nQb = (int)((N + B_Q - 1) / B_Q), nKb = (int)((N_kv + B_KV - 1) / B_KV);
    const int64_t nrows64 = (int64_t)heads * nQb;
    if (nrows64 >= (1ll << 31) - 8) { delete p; return BSA_ERR_UNSUPPORTED; }
    const int nrows = (int)nrows64;

    // ---- Algorithm 2, line 1: shared mask state mu(M), part 1 (row counts + scalar statistics) ----
    // Small masks: the column indices get room for every block of the mask in this first arena, so that the CSR fill
    // does not have to wait for the host to learn nnz: it is queued right behind the row scan and runs while the host
    // waits for the statistics and looks the plan up.
    const int64_t all_blocks = (int64_t)nrows * nKb;
    const bool early_fill = !cache && all_blocks <= (1ll << 20);  // (a cache hit would throw the fill away)
    size_t o_nnz = 0, o_ptr = align_up(o_nnz + sizeof(int32_t) * (size_t)nrows);
    size_t o_col_early = align_up(o_ptr + sizeof(int32_t) * ((size_t)nrows + 1));
    size_t o_zero = early_fill ? align_up(o_col_early + sizeof(int32_t) * (size_t)(all_blocks + 1)) : o_col_early;
    size_t o_cnt = o_zero, o_hc = o_cnt + 256;
    size_t a1_bytes = align_up(o_hc + sizeof(int32_t) * 3 * (size_t)heads);
    BSA_CUDA(cudaMallocAsync(&p->arena1, a1_bytes, stream), "arena1");
    p->row_nnz = reinterpret_cast<int32_t*>(p->arena1 + o_nnz);
    p->row_ptr = reinterpret_cast<int32_t*>(p->arena1 + o_ptr);
    p->counters = reinterpret_cast<PlanCountersDev*>(p->arena1 + o_cnt);
    p->head_counts = reinterpret_cast<int32_t*>(p->arena1 + o_hc);
    // The statistics accumulators live in a small device buffer of this host thread (one per device) that the
    // statistics kernel itself leaves at zero, so nothing has to be cleared in front of that kernel.  A request that
    // ended in an error may have left them dirty: then, and at first use, they are cleared here.
    constexpr int kAccDevices = kMaxDevices;
    static thread_local MaskStatsDev* acc_dev[kAccDevices] = {};
    static thread_local bool acc_clean[kAccDevices] = {};
    if (p->device < 0 || p->device >= kAccDevices) { free_plan(p); return BSA_ERR_UNSUPPORTED; }
    if (!acc_dev[p->device]) BSA_CUDA(cudaMalloc(&acc_dev[p->device], 256), "statistics accumulators");
    p->stats = acc_dev[p->device];
    if (!acc_clean[p->device]) BSA_CUDA(cudaMemsetAsync(p->stats, 0, 256, stream), "accumulator memset");
    acc_clean[p->device] = false;  // until this request's totals have arrived
    // ---- lines 3-5: only the scalars cross to the host.  The statistics kernel's last CTA posts them into pinned
    // host memory and the host polls for the sequence number (a few microseconds less than a copy command and an
    // event); if nothing arrives within a millisecond the host waits for the stream instead.
    static thread_local MaskStatsHost* posted = nullptr;
    static thread_local unsigned post_seq = 0;
    if (!posted) {
        BSA_CUDA(cudaMallocHost(&posted, sizeof(MaskStatsHost)), "pinned stats");
        memset(posted, 0, sizeof *posted);
    }
    const unsigned seq = ++post_seq ? post_seq : ++post_seq;  // never 0
    const uint32_t* mask_words = reinterpret_cast<const uint32_t*>(mask_dev);
    if (packed_stride > 0)
        BSA_CUDA(launch_mask_row_stats_packed(mask_words, packed_stride / 4, nrows, nKb, p->row_nnz, p->stats, stream, posted,
                                              seq, cache != nullptr),
                 "mask_row_stats_packed");
    else
        BSA_CUDA(launch_mask_row_stats(mask_dev, nrows, nKb, p->row_nnz, p->stats, stream, posted, seq, cache != nullptr),
                 "mask_row_stats");
    const double t1 = now_us();
    // the counters the later kernels add to (not needed before the statistics have reached the host)
    BSA_CUDA(cudaMemsetAsync(p->arena1 + o_zero, 0, a1_bytes - o_zero, stream), "memset");
    // the row-pointer scan needs nothing from the host: it runs while the host waits for the scalars
    BSA_CUDA(launch_row_scan(p->row_nnz, nrows, p->row_ptr, stream), "row_scan");
    if (early_fill) {
        p->col_idx = reinterpret_cast<int32_t*>(p->arena1 + o_col_early);
        if (packed_stride > 0)
            BSA_CUDA(launch_csr_fill_packed(mask_words, packed_stride / 4, nrows, nKb, p->row_ptr, p->col_idx, stream),
                     "csr_fill_packed");
        else
            BSA_CUDA(launch_csr_fill(mask_dev, nrows, nKb, p->row_ptr, p->col_idx, stream), "csr_fill");
    }
    // While the host would only wait: take the second arena now, at the size the previous request of this shape
    // needed on this thread plus a quarter (masks of one shape have similar nnz); if this request turns out to need
    // more, it is freed and taken again at the exact size below.
    struct LastArena {
        int B_Q, B_KV, heads, d;
        int64_t N, N_kv;
        size_t bytes;
    };
    static thread_local LastArena last_arena = {};
    const bool same_shape = last_arena.bytes && last_arena.B_Q == B_Q && last_arena.B_KV == B_KV &&
                            last_arena.heads == heads && last_arena.d == d && last_arena.N == N && last_arena.N_kv == N_kv;
    size_t arena2_have = 0;
    if (early_fill && same_shape) {
        arena2_have = last_arena.bytes + last_arena.bytes / 4 + 4096;
        BSA_CUDA(cudaMallocAsync(&p->arena2, arena2_have, stream), "arena2 (predicted)");
    }
    {
        volatile unsigned* flag = &posted->seq;
        const double t_poll = now_us();
        bool arrived = true;
        while (*flag != seq) {
            if (now_us() - t_poll > 1000.0) {
                arrived = false;
                break;
            }
        }
        if (!arrived) {  // a long queue in front of the kernel: wait for the stream instead of spinning on
            BSA_CUDA(cudaStreamSynchronize(stream), "stats sync");
            if (*flag != seq) {
                set_cuda_err(cudaErrorUnknown, "statistics were not posted");
                free_plan(p);
                return BSA_ERR_CUDA;
            }
        }
        std::atomic_thread_fence(std::memory_order_acquire);
        p->hstats.nnz = posted->nnz;
        p->hstats.in_runs = posted->in_runs;
        p->hstats.max_row_nnz = posted->max_row_nnz;
        p->hstats.blocks_done = 0;
        p->hstats.hash[0] = posted->hash[0];
        p->hstats.hash[1] = posted->hash[1];
        acc_clean[p->device] = true;  // the kernel's last CTA left the accumulators at zero
    }
    const double t2 = now_us();

    const int64_t max_ws = options ? options->max_workspace_bytes : 0;
    int forced = (options && options->force_plan_id >= 0) ? options->force_plan_id : get_force_plan();
    CacheKey key;
    if (cache) {
        // ---- warm path: the same activity pattern, request key and selection inputs give the same plan ----
        memset(&key, 0, sizeof key);
        key.hash[0] = p->hstats.hash[0];
        key.hash[1] = p->hstats.hash[1];
        key.N = N; key.N_kv = N_kv; key.packed_stride = packed_stride; key.max_ws = max_ws;
        key.B_Q = B_Q; key.B_KV = B_KV; key.heads = heads; key.d = d;
        key.align = packed_stride > 0 ? 0 : (int32_t)(reinterpret_cast<uintptr_t>(mask_dev) & 15u);
        key.force = forced; key.device = p->device; key.dtype = dtype; key.layout = layout;
        key.generation = g_select_generation.load(std::memory_order_relaxed);
        bsa_plan* found = nullptr;
        {
            std::lock_guard<std::mutex> lock(cache->mu);
            auto it = cache->index.find(key);
            if (it != cache->index.end()) {
                cache->lru.splice(cache->lru.begin(), cache->lru, it->second);
                found = it->second->second;
                found->refs.fetch_add(1, std::memory_order_relaxed);
                ++cache->hits;
            } else {
                ++cache->misses;
            }
        }
        if (found) {
            free_plan(p);  // only the first arena exists; its kernels are stream-ordered before the free
            p = nullptr;
            if (found->stream != stream) {
                cudaError_t e = cudaStreamWaitEvent(stream, found->ready, 0);
                if (e != cudaSuccess) {
                    set_cuda_err(e, "cache wait");
                    release_plan(found);
                    return BSA_ERR_CUDA;
                }
            }
            if (cache_hit) *cache_hit = 1;
            *out_plan = found;
            return BSA_OK;
        }
    }

    // ---- lines 6-19: regime lookup, ranked fallback, eligibility ----
    const double total_blocks = (double)nrows * nKb;
    const double nnz = (double)p->hstats.nnz;
    const double density = total_blocks > 0 ? nnz / total_blocks : 0.0;
    const double run_cov = nnz > 0 ? (double)p->hstats.in_runs / nnz : 0.0;
    const double skew = nnz > 0 ? (double)p->hstats.max_row_nnz / (nnz / (double)nrows) : 0.0;
    int plan_id;
    if (forced >= 0) {
        plan_id = plan_eligible(forced, B_Q, B_KV, N, heads, d, max_ws, N_kv, dtype) ? forced : -1;
        lut_buckets(N, density, skew, run_cov, p->buckets);
        p->lut_hit = 0;
    } else {
        plan_id = lut_select(B_Q, B_KV, N, heads, d, density, run_cov, skew, max_ws, &p->lut_hit, p->buckets, N_kv, dtype);
    }
    if (plan_id < 0) { free_plan(p); return BSA_ERR_NO_ELIGIBLE_PLAN; }
    p->desc = *catalog_entry(plan_id);
    make_geom(p->desc, B_Q, B_KV, N, N_kv, heads, &p->g);
    p->stages = p->desc.stages > 0 ? p->desc.stages : attention_max_stages(d, p->desc.T_KV, p->desc.kernel);
    const double t3 = now_us();

    // ---- launch preparation: derive only the selected plan's metadata from the block-CSR ----
    const MapGeom& g = p->g;
    const int64_t nnz_i = (int64_t)p->hstats.nnz;
    p->tile_cap = nnz_i * g.rq * g.rk;
    if (p->tile_cap >= (1ll << 31) - 8) { free_plan(p); return BSA_ERR_UNSUPPORTED; }
    const int pmax = p->desc.split_pmax < 1 ? 1 : p->desc.split_pmax;
    const int64_t trows = (int64_t)heads * g.nQt;
    p->max_items = trows * pmax;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t r = o; o = align_up(o + bytes); return r; };
    const size_t o_col = early_fill ? 0 : take(sizeof(int32_t) * (size_t)(nnz_i + 1));
    const size_t o_tb = take(sizeof(int32_t) * (size_t)trows);
    const size_t o_tc = take(sizeof(int32_t) * (size_t)trows);
    const size_t o_rp = take(sizeof(int32_t) * (size_t)trows);
    const size_t o_tcol = take(sizeof(int32_t) * (size_t)(p->tile_cap + 1));
    const size_t o_tmem = take(sizeof(uint64_t) * (size_t)(p->tile_cap + 1) * g.slots);
    const size_t o_it0 = take(sizeof(WorkItem) * (size_t)p->max_items);
    const size_t o_it1 = take(sizeof(WorkItem) * (size_t)p->max_items);
    const size_t o_sr = take(sizeof(SplitRow) * (size_t)(pmax > 1 ? trows * g.slots : 1));
    const size_t org_bytes = organize_scratch_bytes(g, p->desc.order, pmax);
    const size_t o_org = take(org_bytes ? org_bytes : 4);
    if (p->arena2 && o > arena2_have) {  // the prediction was too small
        cudaFreeAsync(p->arena2, stream);
        p->arena2 = nullptr;
    }
    if (!p->arena2) BSA_CUDA(cudaMallocAsync(&p->arena2, o, stream), "arena2");
    last_arena = LastArena{B_Q, B_KV, heads, d, N, N_kv, o};
    if (!early_fill) p->col_idx = reinterpret_cast<int32_t*>(p->arena2 + o_col);
    p->tile_begin = reinterpret_cast<int32_t*>(p->arena2 + o_tb);
    p->tile_cnt = reinterpret_cast<int32_t*>(p->arena2 + o_tc);
    p->row_parts = reinterpret_cast<int32_t*>(p->arena2 + o_rp);
    p->tile_col = reinterpret_cast<int32_t*>(p->arena2 + o_tcol);
    p->tile_member = reinterpret_cast<uint64_t*>(p->arena2 + o_tmem);
    p->items_tmp = reinterpret_cast<WorkItem*>(p->arena2 + o_it0);
    p->items = reinterpret_cast<WorkItem*>(p->arena2 + o_it1);
    p->split_rows = reinterpret_cast<SplitRow*>(p->arena2 + o_sr);
    p->ws_bytes = plan_workspace_bytes(p->desc, N, heads, d);
    if (p->ws_bytes > 0) {
        BSA_CUDA(cudaMallocAsync(&p->ws_O, (size_t)p->ws_bytes, stream), "workspace");
        p->ws_LSE = p->ws_O + (size_t)p->max_items * g.T_Q * d;
    }
    if (early_fill) {
        // already queued before the statistics arrived
    } else if (packed_stride > 0) {
        BSA_CUDA(launch_csr_fill_packed(mask_words, packed_stride / 4, nrows, nKb, p->row_ptr, p->col_idx, stream),
                 "csr_fill_packed");
    } else {
        BSA_CUDA(launch_csr_fill(mask_dev, nrows, nKb, p->row_ptr, p->col_idx, stream), "csr_fill");
    }
    BSA_CUDA(launch_tile_map(g, p->row_ptr, p->col_idx, p->desc.split_tau, pmax, p->tile_begin, p->tile_cnt,
                             p->row_parts, p->tile_col, p->tile_member, p->head_counts, p->counters, stream, nnz_i),
             "tile_map");
    BSA_CUDA(launch_organize(g, p->desc.order, pmax, p->tile_begin, p->tile_cnt, p->row_parts, p->head_counts,
                             p->items_tmp, p->items, p->split_rows, p->counters, stream,
                             org_bytes ? reinterpret_cast<int32_t*>(p->arena2 + o_org) : nullptr),
             "organize");
    const double t4 = now_us();
    p->us_mask_state = (float)(t1 - t0);
    p->us_stats_sync = (float)(t2 - t1);
    p->us_lookup = (float)(t3 - t2);
    p->us_launch_prep = (float)(t4 - t3);
    p->us_total = (float)(t4 - t0);
    if (cache) {
        BSA_CUDA(cudaEventCreateWithFlags(&p->ready, cudaEventDisableTiming), "cache event");
        BSA_CUDA(cudaEventRecord(p->ready, stream), "cache event record");
        p->refs.store(2, std::memory_order_relaxed);  // the cache and the caller
        bsa_plan* dropped[2] = {nullptr, nullptr};
        {
            std::lock_guard<std::mutex> lock(cache->mu);
            auto it = cache->index.find(key);
            if (it != cache->index.end()) {  // another thread prepared the same mask meanwhile: the newer plan stays
                dropped[0] = it->second->second;
                cache->lru.erase(it->second);
                cache->index.erase(it);
            }
            cache->lru.emplace_front(key, p);
            cache->index[key] = cache->lru.begin();
            if ((int)cache->lru.size() > cache->capacity) {
                dropped[1] = cache->lru.back().second;
                cache->index.erase(cache->lru.back().first);
                cache->lru.pop_back();
                ++cache->evictions;
            }
        }
        for (bsa_plan* q : dropped)
            if (q) release_plan(q);
        if (cache_hit) *cache_hit = 0;
    }
    *out_plan = p;
    return BSA_OK;
}

extern "C" bsa_status_t bsa_plan_cache_create(int capacity, bsa_plan_cache_t** out_cache) {
    if (!out_cache || capacity < 1) return BSA_ERR_INVALID_ARG;
    bsa_plan_cache* c = new (std::nothrow) bsa_plan_cache();
    if (!c) return BSA_ERR_OOM;
    c->capacity = capacity;
    c->hits = c->misses = c->evictions = 0;
    *out_cache = c;
    return BSA_OK;
}

extern "C" bsa_status_t bsa_plan_cache_get(bsa_plan_cache_t* cache, const uint8_t* mask_dev, int64_t row_stride_bytes, int B_Q,
                                           int B_KV, int64_t N, int heads, int d, const bsa_options_t* options,
                                           void* stream_v, bsa_plan_t** out_plan, int* out_hit) {
    if (!cache || row_stride_bytes < 0) return BSA_ERR_INVALID_ARG;
    int hit = 0;
    bsa_status_t st = create_impl(mask_dev, row_stride_bytes, B_Q, B_KV, N, heads, d, options, stream_v, out_plan, cache, &hit);
    if (st == BSA_OK && out_hit) *out_hit = hit;
    return st;
}

extern "C" bsa_status_t bsa_plan_cache_request(bsa_plan_cache_t* cache, const uint8_t* mask_dev, int64_t row_stride_bytes,
                                               int B_Q, int B_KV, int64_t N, int heads, int d, const void* Q, const void* K,
                                               const void* V, void* O, float* LSE, const bsa_options_t* options,
                                               void* stream_v, bsa_plan_t** out_plan, int* out_hit) {
    if (!cache || !out_plan || row_stride_bytes < 0) return BSA_ERR_INVALID_ARG;
    *out_plan = nullptr;
    if (!Q || !K || !V || !O || !LSE) return BSA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(Q) | reinterpret_cast<uintptr_t>(K) | reinterpret_cast<uintptr_t>(V) |
         reinterpret_cast<uintptr_t>(O)) & 15)
        return BSA_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(LSE) & 3) return BSA_ERR_INVALID_ARG;
    bsa_plan_t* plan = nullptr;
    int hit = 0;
    bsa_status_t st = create_impl(mask_dev, row_stride_bytes, B_Q, B_KV, N, heads, d, options, stream_v, &plan, cache, &hit);
    if (st != BSA_OK) return st;
    st = bsa_forward(plan, Q, K, V, O, LSE, stream_v);
    if (st != BSA_OK) {
        bsa_plan_destroy(plan);
        return st;
    }
    if (out_hit) *out_hit = hit;
    *out_plan = plan;
    return BSA_OK;
}

extern "C" bsa_status_t bsa_plan_cache_stats(bsa_plan_cache_t* cache, int64_t* hits, int64_t* misses, int64_t* evictions,
                                             int32_t* entries) {
    if (!cache) return BSA_ERR_INVALID_ARG;
    std::lock_guard<std::mutex> lock(cache->mu);
    if (hits) *hits = cache->hits;
    if (misses) *misses = cache->misses;
    if (evictions) *evictions = cache->evictions;
    if (entries) *entries = (int32_t)cache->lru.size();
    return BSA_OK;
}

extern "C" bsa_status_t bsa_plan_cache_destroy(bsa_plan_cache_t* cache) {
    if (!cache) return BSA_ERR_INVALID_ARG;
    cudaError_t e = cudaSuccess;
    for (auto& kv : cache->lru) {
        cudaStream_t s = kv.second->stream;
        if (release_plan(kv.second)) {
            cudaError_t e1 = cudaStreamSynchronize(s);
            if (e == cudaSuccess) e = e1;
        }
    }
    delete cache;
    if (e != cudaSuccess) {
        set_cuda_err(e, "cache destroy sync");
        return BSA_ERR_CUDA;
    }
    return BSA_OK;
}

extern "C" bsa_status_t bsa_plan_create_ex(const uint8_t* mask_dev, int B_Q, int B_KV, int64_t N, int heads, int d,
                                           const bsa_options_t* options, void* stream_v, bsa_plan_t** out_plan) {
    return create_impl(mask_dev, 0, B_Q, B_KV, N, heads, d, options, stream_v, out_plan);
}

extern "C" bsa_status_t bsa_plan_create_packed(const uint8_t* mask_bits_dev, int64_t row_stride_bytes, int B_Q, int B_KV,
                                               int64_t N, int heads, int d, const bsa_options_t* options, void* stream_v,
                                               bsa_plan_t** out_plan) {
    if (row_stride_bytes <= 0) return BSA_ERR_INVALID_ARG;
    return create_impl(mask_bits_dev, row_stride_bytes, B_Q, B_KV, N, heads, d, options, stream_v, out_plan);
}

extern "C" bsa_status_t bsa_plan_create(const uint8_t* mask_dev, int B_Q, int B_KV, int64_t N, int heads, int d,
                                        bsa_plan_t** out_plan) {
    return bsa_plan_create_ex(mask_dev, B_Q, B_KV, N, heads, d, nullptr, nullptr, out_plan);
}

static void fill_forward_args(const bsa_plan_t* p, const void* Q, const void* K, const void* V, void* O, float* LSE,
                              ForwardArgs& a) {
    memset(&a, 0, sizeof a);
    a.Q = Q; a.K = K; a.V = V; a.O = O; a.LSE = LSE;
    a.items = p->items;
    a.split_rows = p->split_rows;
    a.tile_col = p->tile_col;
    a.tile_member = p->tile_member;
    a.counters = p->counters;
    a.ws_O = p->ws_O;
    a.ws_LSE = p->ws_LSE;
    a.g = p->g;
    a.d = p->d;
    a.stages = p->stages;
    a.kernel = p->desc.kernel;
    a.has_split = p->desc.split_pmax > 1;
    a.max_items = (int32_t)(p->max_items < (1 << 30) ? p->max_items : (1 << 30));
    a.max_split_rows = p->g.H * p->g.nQt * p->g.slots;
    a.num_sms = p->num_sms;
    a.device = p->device;
    a.f16 = p->dtype == BSA_DTYPE_FP16;
    a.nhd = p->layout == BSA_LAYOUT_NHD;
}

extern "C" bsa_status_t bsa_debug_merge_only(const bsa_plan_t* p, void* O, float* LSE, void* stream_v) {
    if (!p || !O || !LSE) return BSA_ERR_INVALID_ARG;
    if (p->kids || p->desc.split_pmax <= 1) return BSA_ERR_UNSUPPORTED;
    ForwardArgs a;
    fill_forward_args(p, nullptr, nullptr, nullptr, O, LSE, a);
    cudaError_t e = launch_merge(a, reinterpret_cast<cudaStream_t>(stream_v));
    if (e != cudaSuccess) {
        set_cuda_err(e, "merge launch");
        return BSA_ERR_CUDA;
    }
    return BSA_OK;
}

extern "C" bsa_status_t bsa_forward(const bsa_plan_t* p, const void* Q, const void* K, const void* V, void* O,
                                    float* LSE, void* stream_v) {
    if (!p || !Q || !K || !V || !O || !LSE) return BSA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(Q) | reinterpret_cast<uintptr_t>(K) | reinterpret_cast<uintptr_t>(V) |
         reinterpret_cast<uintptr_t>(O)) & 15)
        return BSA_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(LSE) & 3) return BSA_ERR_INVALID_ARG;
    if (p->kids) {  // batched token-major request: element b's tensors start b * N * (heads / batch) * d elements further
        const int hb = p->g.H / p->nkids;
        const size_t q_step = (size_t)p->g.N * hb * p->d * 2, kv_step = (size_t)p->g.N_kv * hb * p->d * 2;
        for (int b = 0; b < p->nkids; ++b) {
            bsa_status_t st = bsa_forward(p->kids[b], static_cast<const uint8_t*>(Q) + b * q_step,
                                          static_cast<const uint8_t*>(K) + b * kv_step, static_cast<const uint8_t*>(V) + b * kv_step,
                                          static_cast<uint8_t*>(O) + b * q_step, LSE + (size_t)b * hb * p->g.N, stream_v);
            if (st != BSA_OK) return st;
        }
        return BSA_OK;
    }
    ForwardArgs a;
    fill_forward_args(p, Q, K, V, O, LSE, a);
    const char* detail = "launch";
    cudaStream_t fstream = reinterpret_cast<cudaStream_t>(stream_v);
    cudaError_t e = launch_forward(a, fstream, &detail);
    if (e != cudaSuccess) {
        set_cuda_err(e, detail);
        return BSA_ERR_CUDA;
    }
    if (fstream != p->stream) {
        // The plan's memory is freed in the create stream's order: leave a marker behind this forward that the free
        // waits for.  Not while `stream` is being captured (an event recorded into a graph cannot be waited for from
        // outside it): whoever replays a captured forward keeps the plan alive until the replays are done.
        cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(fstream, &cs) == cudaSuccess && cs == cudaStreamCaptureStatusNone) {
            bsa_plan* mp = const_cast<bsa_plan*>(p);
            cudaEvent_t lu = mp->last_use.load(std::memory_order_acquire);
            if (!lu) {
                cudaEvent_t fresh = nullptr;
                e = cudaEventCreateWithFlags(&fresh, cudaEventDisableTiming);
                if (e != cudaSuccess) {
                    set_cuda_err(e, "last-use event");
                    return BSA_ERR_CUDA;
                }
                if (mp->last_use.compare_exchange_strong(lu, fresh, std::memory_order_acq_rel)) lu = fresh;
                else cudaEventDestroy(fresh);  // another thread was first; `lu` now holds its event
            }
            e = cudaEventRecord(lu, fstream);
            if (e != cudaSuccess) {
                set_cuda_err(e, "last-use record");
                return BSA_ERR_CUDA;
            }
        }
    }
    return BSA_OK;
}

extern "C" bsa_status_t bsa_request_device(const uint8_t* mask_dev, int64_t row_stride_bytes, int B_Q, int B_KV, int64_t N,
                                           int heads, int d, const void* Q, const void* K, const void* V, void* O,
                                           float* LSE, const bsa_options_t* options, void* stream_v,
                                           bsa_plan_t** out_plan) {
    if (!out_plan || row_stride_bytes < 0) return BSA_ERR_INVALID_ARG;
    *out_plan = nullptr;
    if (!Q || !K || !V || !O || !LSE) return BSA_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(Q) | reinterpret_cast<uintptr_t>(K) | reinterpret_cast<uintptr_t>(V) |
         reinterpret_cast<uintptr_t>(O)) & 15)
        return BSA_ERR_INVALID_ARG;
    if (reinterpret_cast<uintptr_t>(LSE) & 3) return BSA_ERR_INVALID_ARG;
    bsa_plan_t* plan = nullptr;
    bsa_status_t st = create_impl(mask_dev, row_stride_bytes, B_Q, B_KV, N, heads, d, options, stream_v, &plan);
    if (st != BSA_OK) return st;
    st = bsa_forward(plan, Q, K, V, O, LSE, stream_v);
    if (st != BSA_OK) {
        bsa_plan_destroy(plan);
        return st;
    }
    *out_plan = plan;
    return BSA_OK;
}

extern "C" bsa_status_t bsa_plan_destroy(bsa_plan_t* p) {
    if (!p) return BSA_ERR_INVALID_ARG;
    cudaStream_t s = p->stream;
    if (!release_plan(p)) return BSA_OK;  // a plan cache (or another request that got it from there) still holds it
    cudaError_t e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) {
        set_cuda_err(e, "destroy sync");
        return BSA_ERR_CUDA;
    }
    return BSA_OK;
}

// counts and times of `info` added to `tot` (the request's info over several sub-plans)
static void add_info(bsa_plan_info_t& tot, const bsa_plan_info_t& info) {
    tot.heads += info.heads;
    tot.nnz_blocks += info.nnz_blocks;
    tot.blocks_in_runs += info.blocks_in_runs;
    if (info.max_row_nnz > tot.max_row_nnz) tot.max_row_nnz = info.max_row_nnz;
    tot.ntiles += info.ntiles;
    tot.nitems += info.nitems;
    tot.nsplit_rows += info.nsplit_rows;
    tot.workspace_bytes += info.workspace_bytes;
    tot.covered_pairs += info.covered_pairs;
    tot.us_mask_state += info.us_mask_state;
    tot.us_stats_sync += info.us_stats_sync;
    tot.us_lookup += info.us_lookup;
    tot.us_launch_prep += info.us_launch_prep;
    tot.us_total += info.us_total;
    tot.device_status |= info.device_status;
}
static void finish_info(bsa_plan_info_t& tot) {
    const double rows = (double)tot.heads * (double)tot.nQb, nnz = (double)tot.nnz_blocks;
    tot.density = rows > 0 ? nnz / (rows * (double)tot.nKb) : 0.0;
    tot.run_coverage = nnz > 0 ? (double)tot.blocks_in_runs / nnz : 0.0;
    tot.skew = nnz > 0 ? (double)tot.max_row_nnz / (nnz / rows) : 0.0;
}

extern "C" bsa_status_t bsa_plan_get_info(const bsa_plan_t* p, bsa_plan_info_t* info) {
    if (!p || !info) return BSA_ERR_INVALID_ARG;
    if (p->kids) {  // statistics of the whole mask, sums over the batch elements, the first element's plan
        for (int b = 0; b < p->nkids; ++b) {
            bsa_plan_info_t one;
            bsa_status_t st = bsa_plan_get_info(p->kids[b], &one);
            if (st != BSA_OK) return st;
            if (b == 0) *info = one;
            else add_info(*info, one);
        }
        finish_info(*info);
        return BSA_OK;
    }
    cudaError_t e = cudaDeviceSynchronize();
    PlanCountersDev c;
    if (e == cudaSuccess) e = cudaMemcpy(&c, p->counters, sizeof c, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) {
        set_cuda_err(e, "get_info");
        return BSA_ERR_CUDA;
    }
    memset(info, 0, sizeof *info);
    info->plan = p->desc;
    const MapGeom& g = p->g;
    info->map_q = g.sQ > 1 ? BSA_MAP_COARSENED : (g.rq > 1 ? BSA_MAP_REFINED : BSA_MAP_DIRECT);
    info->map_kv = g.sK > 1 ? BSA_MAP_COARSENED : (g.rk > 1 ? BSA_MAP_REFINED : BSA_MAP_DIRECT);
    info->heads = g.H; info->d = p->d; info->B_Q = g.B_Q; info->B_KV = g.B_KV; info->N = g.N; info->N_kv = g.N_kv; info->dtype = p->dtype; info->layout = p->layout;
    info->nQb = g.nQb; info->nKb = g.nKb; info->nQt = g.nQt; info->nKt = g.nKt;
    info->member_bits = g.sQ128 * g.sK;
    info->member_words = g.slots;
    info->lut_hit = p->lut_hit;
    memcpy(info->regime_bucket, p->buckets, sizeof p->buckets);
    info->nnz_blocks = (int64_t)p->hstats.nnz;
    info->blocks_in_runs = (int64_t)p->hstats.in_runs;
    info->max_row_nnz = (int32_t)p->hstats.max_row_nnz;
    const double nrows = (double)g.H * g.nQb;
    const double nnz = (double)p->hstats.nnz;
    info->density = nrows > 0 ? nnz / (nrows * g.nKb) : 0.0;
    info->run_coverage = nnz > 0 ? (double)p->hstats.in_runs / nnz : 0.0;
    info->skew = nnz > 0 ? (double)p->hstats.max_row_nnz / (nnz / nrows) : 0.0;
    info->ntiles = (int64_t)c.ntiles;
    info->nitems = c.nitems;
    info->nsplit_rows = c.nsplit_rows;  // physical tile rows with more than one partition
    info->workspace_bytes = p->ws_bytes;
    info->covered_pairs = (int64_t)c.nslot_tiles * (g.T_Q < kTQ ? g.T_Q : kTQ) * g.T_KV;
    info->us_mask_state = p->us_mask_state;
    info->us_stats_sync = p->us_stats_sync;
    info->us_lookup = p->us_lookup;
    info->us_launch_prep = p->us_launch_prep;
    info->us_total = p->us_total;
    info->device_status = c.status;
    return BSA_OK;
}

extern "C" bsa_status_t bsa_plan_export_csr(const bsa_plan_t* p, int32_t* row_ptr_host, int32_t* col_idx_host) {
    if (!p) return BSA_ERR_INVALID_ARG;
    if (p->kids) return BSA_ERR_UNSUPPORTED;  // ask the per-element plans of a batched token-major request
    cudaError_t e = cudaDeviceSynchronize();
    const size_t nrows = (size_t)p->g.H * p->g.nQb;
    if (e == cudaSuccess && row_ptr_host)
        e = cudaMemcpy(row_ptr_host, p->row_ptr, sizeof(int32_t) * (nrows + 1), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && col_idx_host && p->hstats.nnz)
        e = cudaMemcpy(col_idx_host, p->col_idx, sizeof(int32_t) * (size_t)p->hstats.nnz, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) {
        set_cuda_err(e, "export_csr");
        return BSA_ERR_CUDA;
    }
    return BSA_OK;
}

extern "C" bsa_status_t bsa_plan_export_tiles(const bsa_plan_t* p, int head, int32_t* tile_row_ptr_host,
                                              int32_t* tile_col_host, uint64_t* tile_member_host, int64_t cap,
                                              int64_t* ntiles_out) {
    if (!p || head < 0 || head >= p->g.H || !ntiles_out) return BSA_ERR_INVALID_ARG;
    if (p->kids) return BSA_ERR_UNSUPPORTED;
    cudaError_t e = cudaDeviceSynchronize();
    const int nQt = p->g.nQt;
    int32_t* tb = new (std::nothrow) int32_t[2 * (size_t)nQt];
    if (!tb) return BSA_ERR_OOM;
    int32_t* tc = tb + nQt;
    if (e == cudaSuccess)
        e = cudaMemcpy(tb, p->tile_begin + (size_t)head * nQt, sizeof(int32_t) * nQt, cudaMemcpyDeviceToHost);
    if (e == cudaSuccess)
        e = cudaMemcpy(tc, p->tile_cnt + (size_t)head * nQt, sizeof(int32_t) * nQt, cudaMemcpyDeviceToHost);
    int64_t total = 0;
    for (int t = 0; t < nQt && e == cudaSuccess; ++t) total += tc[t];
    *ntiles_out = total;
    bsa_status_t st = BSA_OK;
    if (e == cudaSuccess && tile_row_ptr_host && tile_col_host && tile_member_host) {
        if (cap < total) {
            st = BSA_ERR_INVALID_ARG;
        } else {
            int64_t off = 0;
            for (int t = 0; t < nQt && e == cudaSuccess; ++t) {
                tile_row_ptr_host[t] = (int32_t)off;
                if (tc[t]) {
                    e = cudaMemcpy(tile_col_host + off, p->tile_col + tb[t], sizeof(int32_t) * tc[t],
                                   cudaMemcpyDeviceToHost);
                    if (e == cudaSuccess)
                        e = cudaMemcpy(tile_member_host + off * p->g.slots, p->tile_member + (size_t)tb[t] * p->g.slots,
                                       sizeof(uint64_t) * tc[t] * p->g.slots, cudaMemcpyDeviceToHost);
                }
                off += tc[t];
            }
            tile_row_ptr_host[nQt] = (int32_t)off;
        }
    }
    delete[] tb;
    if (e != cudaSuccess) {
        set_cuda_err(e, "export_tiles");
        return BSA_ERR_CUDA;
    }
    return st;
}

extern "C" bsa_status_t bsa_plan_export_items(const bsa_plan_t* p, int32_t* items_host, int64_t cap,
                                              int64_t* nitems_out) {
    if (!p || !nitems_out) return BSA_ERR_INVALID_ARG;
    if (p->kids) return BSA_ERR_UNSUPPORTED;
    cudaError_t e = cudaDeviceSynchronize();
    PlanCountersDev c;
    if (e == cudaSuccess) e = cudaMemcpy(&c, p->counters, sizeof c, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) {
        set_cuda_err(e, "export_items");
        return BSA_ERR_CUDA;
    }
    *nitems_out = c.nitems;
    if (items_host) {
        if (cap < c.nitems) return BSA_ERR_INVALID_ARG;
        e = cudaMemcpy(items_host, p->items, sizeof(WorkItem) * (size_t)c.nitems, cudaMemcpyDeviceToHost);
        if (e != cudaSuccess) {
            set_cuda_err(e, "export_items copy");
            return BSA_ERR_CUDA;
        }
    }
    return BSA_OK;
}

extern "C" bsa_status_t bsa_request_host(const uint8_t* mask_host, int B_Q, int B_KV, int64_t N, int heads, int d,
                                         const void* Q_host, const void* K_host, const void* V_host, void* O_host,
                                         float* LSE_host, const bsa_options_t* options, bsa_plan_info_t* info_out) {
    if (!Q_host || !K_host || !V_host || !O_host || !LSE_host) return BSA_ERR_INVALID_ARG;
    bsa_plan_t* dummy = nullptr;
    bsa_status_t vs = validate(mask_host, B_Q, B_KV, N, heads, d, &dummy);
    if (vs != BSA_OK) return vs;
    const int64_t N_kv = request_n_kv(options, N);
    if (N_kv > (1ll << 30)) return BSA_ERR_UNSUPPORTED;
    const size_t nQb = (size_t)((N + B_Q - 1) / B_Q), nKb = (size_t)((N_kv + B_KV - 1) / B_KV);
    const size_t mbytes = (size_t)heads * nQb * nKb;
    const size_t tbytes = (size_t)heads * (size_t)N * d * 2;      // Q, O
    const size_t kbytes = (size_t)heads * (size_t)N_kv * d * 2;   // K, V
    const size_t lbytes = (size_t)heads * (size_t)N * 4;
    const size_t o_m = 0, o_q = align_up(mbytes), o_k = o_q + align_up(tbytes), o_v = o_k + align_up(kbytes),
                 o_o = o_v + align_up(kbytes), o_l = o_o + align_up(tbytes), total = o_l + align_up(lbytes);
    // Heads are independent, and with the head-major layout a range of heads is a contiguous slice of every tensor:
    // the request is cut into up to 8 groups of heads (more than 32 MB of Q, K, V each: with smaller groups the
    // copies themselves got slower, 43 instead of 53 GB/s) and pipelined over three streams kept per host thread --
    // inputs of group g+1 travel (s2) while group g is planned and computed (s) and the output of group g-1 travels
    // back (s3; the link is full duplex).  What is left after the last input byte is one group's forward and its
    // output copy.  The token-major layout is not cut.
    const size_t head_in = ((size_t)N + 2 * (size_t)N_kv) * d * 2;
    const int hmin = (int)(((size_t)32 << 20) / (head_in ? head_in : 1)) + 1;  // fewest heads a group may have
    int hc = hmin;                                                             // heads per group
    if (hc < (heads + 7) / 8) hc = (heads + 7) / 8;
    if (hc > heads || (options && options->layout == BSA_LAYOUT_NHD)) hc = heads;
    const int G = (heads + hc - 1) / hc;
    // Group boundaries.  Where the smallest allowed group is well below the even share, the last two groups are made
    // small (hmin and 2 hmin heads) and the others share the rest: the tail after the last input byte is then the
    // forward and the output copy of hmin heads instead of hc (24 heads of the Hunyuan-shaped request: 4 4 4 3 3 3 2 1).
    int hb[9];
    for (int g = 0; g <= G; ++g) hb[g] = g * hc < heads ? g * hc : heads;
    if (G >= 4 && 3 * hmin < hc + (heads - (G - 1) * hc)) {
        const int rest = heads - 3 * hmin, ng = G - 2;
        int at = 0;
        for (int g = 0; g < ng; ++g) {
            hb[g] = at;
            at += rest / ng + (g < rest % ng ? 1 : 0);
        }
        hb[G - 2] = at;
        hb[G - 1] = at + 2 * hmin;
        hb[G] = heads;
    }
    static thread_local cudaStream_t s = nullptr, s2 = nullptr, s3 = nullptr;
    static thread_local cudaEvent_t buf_ready = nullptr, in_ready[8] = {}, out_ready[8] = {};
    cudaError_t e = cudaSuccess;
    if (!s) e = cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking);
    if (e == cudaSuccess && !s2) e = cudaStreamCreateWithFlags(&s2, cudaStreamNonBlocking);
    if (e == cudaSuccess && !s3) e = cudaStreamCreateWithFlags(&s3, cudaStreamNonBlocking);
    if (e == cudaSuccess && !buf_ready) e = cudaEventCreateWithFlags(&buf_ready, cudaEventDisableTiming);
    for (int g = 0; g < 8 && e == cudaSuccess; ++g) {
        if (!in_ready[g]) e = cudaEventCreateWithFlags(&in_ready[g], cudaEventDisableTiming);
        if (e == cudaSuccess && !out_ready[g]) e = cudaEventCreateWithFlags(&out_ready[g], cudaEventDisableTiming);
    }
    if (e != cudaSuccess) { set_cuda_err(e, "request streams"); return BSA_ERR_CUDA; }
    uint8_t* buf = nullptr;
    bsa_status_t st = BSA_OK;
    bsa_plan_t* plans[8] = {};
    e = cudaMallocAsync(&buf, total, s);
    if (e != cudaSuccess) { set_cuda_err(e, "request buffers"); return BSA_ERR_OOM; }
    e = cudaMemcpyAsync(buf + o_m, mask_host, mbytes, cudaMemcpyHostToDevice, s);
    // the buffer exists once `s` reaches this point: order the other streams behind it
    if (e == cudaSuccess) e = cudaEventRecord(buf_ready, s);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(s2, buf_ready, 0);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(s3, buf_ready, 0);
    const size_t q_head = (size_t)N * d * 2, k_head = (size_t)N_kv * d * 2, l_head = (size_t)N * 4;
    for (int g = 0; g < G && e == cudaSuccess; ++g) {  // all input copies are queued first, in group order
        const size_t h0 = (size_t)hb[g], nh = (size_t)(hb[g + 1] - hb[g]);
        e = cudaMemcpyAsync(buf + o_q + h0 * q_head, static_cast<const uint8_t*>(Q_host) + h0 * q_head, nh * q_head,
                            cudaMemcpyHostToDevice, s2);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(buf + o_k + h0 * k_head, static_cast<const uint8_t*>(K_host) + h0 * k_head, nh * k_head,
                                cudaMemcpyHostToDevice, s2);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(buf + o_v + h0 * k_head, static_cast<const uint8_t*>(V_host) + h0 * k_head, nh * k_head,
                                cudaMemcpyHostToDevice, s2);
        if (e == cudaSuccess) e = cudaEventRecord(in_ready[g], s2);
    }
    for (int g = 0; g < G && e == cudaSuccess && st == BSA_OK; ++g) {
        const size_t h0 = (size_t)hb[g];
        const int nh = hb[g + 1] - hb[g];
        st = bsa_plan_create_ex(buf + o_m + h0 * nQb * nKb, B_Q, B_KV, N, nh, d, options, s, &plans[g]);
        if (st != BSA_OK) break;
        e = cudaStreamWaitEvent(s, in_ready[g], 0);
        if (e != cudaSuccess) break;
        st = bsa_forward(plans[g], buf + o_q + h0 * q_head, buf + o_k + h0 * k_head, buf + o_v + h0 * k_head,
                         buf + o_o + h0 * q_head, reinterpret_cast<float*>(buf + o_l + h0 * l_head), s);
        if (st != BSA_OK) break;
        e = cudaEventRecord(out_ready[g], s);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(s3, out_ready[g], 0);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(static_cast<uint8_t*>(O_host) + h0 * q_head, buf + o_o + h0 * q_head, (size_t)nh * q_head,
                                cudaMemcpyDeviceToHost, s3);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(reinterpret_cast<uint8_t*>(LSE_host) + h0 * l_head, buf + o_l + h0 * l_head,
                                (size_t)nh * l_head, cudaMemcpyDeviceToHost, s3);
    }
    // every stream is drained on every path: copies may still be in flight after an error
    cudaError_t e3 = cudaStreamSynchronize(s3), e2 = cudaStreamSynchronize(s2), e1 = cudaStreamSynchronize(s);
    if (e == cudaSuccess) e = e3 != cudaSuccess ? e3 : (e2 != cudaSuccess ? e2 : e1);
    if (st == BSA_OK && e == cudaSuccess) {
        // one info for the whole request: counts add up over the groups, the plan is the first group's
        bsa_plan_info_t tot;
        memset(&tot, 0, sizeof tot);
        for (int g = 0; g < G && st == BSA_OK; ++g) {
            bsa_plan_info_t info;
            st = bsa_plan_get_info(plans[g], &info);
            if (st != BSA_OK) break;
            if (info.device_status != 0) st = BSA_ERR_DEVICE_TIMEOUT;
            if (g == 0) {
                tot = info;
                continue;
            }
            add_info(tot, info);
        }
        if (G > 1) finish_info(tot);
        if (info_out) *info_out = tot;
    }
    for (int g = 0; g < G; ++g)
        if (plans[g]) bsa_plan_destroy(plans[g]);
    cudaFreeAsync(buf, s);
    cudaStreamSynchronize(s);
    if (e != cudaSuccess) { set_cuda_err(e, "request"); return BSA_ERR_CUDA; }
    return st;
}

extern "C" int bsa_catalog_size(void) { return catalog_size(); }
extern "C" bsa_status_t bsa_catalog_get(int index, bsa_plan_desc_t* out) {
    const bsa_plan_desc_t* e = catalog_entry(index);
    if (!e || !out) return BSA_ERR_INVALID_ARG;
    *out = *e;
    return BSA_OK;
}
extern "C" int bsa_plan_eligible(int plan_id, int B_Q, int B_KV, int64_t N, int heads, int d, int64_t max_ws) {
    return plan_eligible(plan_id, B_Q, B_KV, N, heads, d, max_ws) ? 1 : 0;
}
extern "C" int bsa_plan_eligible_ex(int plan_id, int B_Q, int B_KV, int64_t N, int64_t N_kv, int heads, int d, int dtype,
                                    int64_t max_ws) {
    return plan_eligible(plan_id, B_Q, B_KV, N, heads, d, max_ws, N_kv, dtype) ? 1 : 0;
}
extern "C" int bsa_base_plan(int B_Q, int B_KV, int d) { return base_plan(B_Q, B_KV, d); }
extern "C" uint64_t bsa_catalog_hash(void) { return catalog_hash(); }
extern "C" bsa_status_t bsa_lut_load(const char* path) {
    g_select_generation.fetch_add(1, std::memory_order_relaxed);
    return lut_load(path);
}
extern "C" void bsa_lut_clear(void) {
    g_select_generation.fetch_add(1, std::memory_order_relaxed);
    lut_clear();
}
extern "C" int bsa_lut_num_regimes(void) { return lut_num_regimes(); }
extern "C" int bsa_lut_num_trees(void) { return lut_num_trees(); }
extern "C" int bsa_lut_select(int B_Q, int B_KV, int64_t N, int heads, int d, double density, double run_coverage,
                              double skew, int64_t max_ws, int* hit_out) {
    return lut_select(B_Q, B_KV, N, heads, d, density, run_coverage, skew, max_ws, hit_out, nullptr);
}
extern "C" void bsa_lut_buckets(int64_t N, double density, double skew, double run_coverage, int32_t out[4]) {
    lut_buckets(N, density, skew, run_coverage, out);
}
extern "C" void bsa_force_plan(int plan_id) {
    g_select_generation.fetch_add(1, std::memory_order_relaxed);
    set_force_plan(plan_id);
}

extern "C" const char* bsa_status_string(bsa_status_t s) {
    switch (s) {
        case BSA_OK: return "ok";
        case BSA_ERR_INVALID_ARG: return "invalid argument";
        case BSA_ERR_UNSUPPORTED: return "unsupported geometry or head dimension";
        case BSA_ERR_NO_ELIGIBLE_PLAN: return "no eligible plan";
        case BSA_ERR_OOM: return "out of memory";
        case BSA_ERR_CUDA: return "CUDA error";
        case BSA_ERR_DEVICE_TIMEOUT: return "bounded device wait expired";
        case BSA_ERR_LUT: return "plan table rejected";
    }
    return "unknown status";
}
extern "C" const char* bsa_last_cuda_error(void) { return g_cuda_err; }
extern "C" const char* bsa_version(void) { return "bsa-b200 0.1 (sm_100a)"; }
extern "C" int64_t bsa_kernel_launch_count(void) { return g_launches.load(); }
