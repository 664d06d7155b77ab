// Internal declarations shared by the planner, the attention kernels and the C ABI.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/bsa.h"

namespace bsa {

constexpr int kMaxDevices = 64;  // per-device host state (accumulators, kernel attributes) is kept for this many GPUs
constexpr int kTQ = 128;  // rows of one tcgen05 MMA (one 128-row slot); the row-block kernel's tiles are smaller

// One unit of work for a persistent CTA: one Q tile row of one head, restricted to the KV tiles
// [tile_begin, tile_end) of the plan's tile arrays (a Split-K partition when nparts > 1).
struct WorkItem {
    int32_t head;
    int32_t q_tile;
    int32_t tile_begin;
    int32_t tile_end;
    int32_t part;
    int32_t nparts;
    int32_t ws_slot;  // workspace slot of this partition (valid when nparts > 1)
    int32_t ntiles;   // tile_end - tile_begin (sort key)
};
static_assert(sizeof(WorkItem) == 32, "WorkItem must be 32 bytes");

struct SplitRow {
    int32_t head;
    int32_t q_tile;   // 128-row tile index
    int32_t ws_slot;  // workspace slot (128 rows each) of partition 0
    int32_t nparts;   // low 16 bits: partitions; high 16 bits: slot stride between partitions
};

// Scalars produced on the device during plan creation.
struct MaskStatsDev {
    unsigned long long nnz;
    unsigned long long in_runs;
    unsigned int max_row_nnz;
    unsigned int blocks_done;  // CTAs of the statistics kernel that have added their share (starts at zero)
    unsigned long long hash[2];  // 128-bit fingerprint of the activity pattern (only when asked for, else 0)
};
// The statistics as the kernel's last CTA posts them into pinned host memory; `seq` is written last.
struct MaskStatsHost {
    unsigned long long nnz;
    unsigned long long in_runs;
    unsigned long long hash[2];
    unsigned int max_row_nnz;
    unsigned int seq;
};
struct PlanCountersDev {
    unsigned long long ntiles;       // physical tiles (a 256-row tile counts once)
    unsigned long long nslot_tiles;  // 128-row MMA tiles actually computed
    int32_t nitems;
    int32_t nsplit_rows;
    int32_t nslots;
    int32_t status;  // set by kernels when a bounded wait expires (0 = ok)
};

// Geometry of the logical -> physical mapping of one plan instance.
struct MapGeom {
    int32_t H, nQb, nKb, nQt, nKt;
    int32_t B_Q, B_KV, T_Q, T_KV;
    int32_t slots;   // 128-row MMA slots per physical tile row (T_Q / 128)
    int32_t sQ128;   // logical rows per 128-row slot (1 when B_Q >= 128)
    int32_t sQ, rq;  // logical rows per tile row (coarsened) / tile rows per logical row (refined)
    int32_t sK, rk;  // same for columns
    int32_t lgBQ, lgBKV, lgSK;
    int64_t N;     // query tokens per head (rows of Q, O, LSE)
    int64_t N_kv;  // key/value tokens per head (rows of K, V; columns of the score matrix)
};

// ---- planner entry points (bsa_planner.cu); all launch on `stream`, none synchronises -------
// `post` (may be null): pinned host memory the last CTA writes the totals to, tagged with `seq`.
// `with_hash`: also accumulate the 128-bit fingerprint of the activity pattern (the plan cache's key).
cudaError_t launch_mask_row_stats(const uint8_t* mask, int nrows, int nKb, int32_t* row_nnz, MaskStatsDev* stats,
                                  cudaStream_t stream, MaskStatsHost* post = nullptr, unsigned seq = 0,
                                  bool with_hash = false);
cudaError_t launch_row_scan(const int32_t* row_nnz, int nrows, int32_t* row_ptr, cudaStream_t stream);
cudaError_t launch_mask_row_stats_packed(const uint32_t* mask, long long stride_words, int nrows, int nKb,
                                         int32_t* row_nnz, MaskStatsDev* stats, cudaStream_t stream,
                                         MaskStatsHost* post = nullptr, unsigned seq = 0, bool with_hash = false);
cudaError_t launch_csr_fill_packed(const uint32_t* mask, long long stride_words, int nrows, int nKb,
                                   const int32_t* row_ptr, int32_t* col_idx, cudaStream_t stream);
cudaError_t launch_csr_fill(const uint8_t* mask, int nrows, int nKb, const int32_t* row_ptr, int32_t* col_idx,
                            cudaStream_t stream);
cudaError_t launch_tile_map(const MapGeom& g, const int32_t* row_ptr, const int32_t* col_idx, int split_tau,
                            int split_pmax, int32_t* tile_begin, int32_t* tile_cnt, int32_t* row_parts,
                            int32_t* tile_col, uint64_t* tile_member, int32_t* head_counts /* [3*H] */,
                            PlanCountersDev* counters, cudaStream_t stream, int64_t nnz = 0);
// `scratch` (may be null): organize_scratch_bytes() bytes in the plan's arena for the long-list path.
cudaError_t launch_organize(const MapGeom& g, int order, int split_pmax, const int32_t* tile_begin,
                            const int32_t* tile_cnt, const int32_t* row_parts, const int32_t* head_counts, WorkItem* items_tmp,
                            WorkItem* items, SplitRow* split_rows, PlanCountersDev* counters, cudaStream_t stream,
                            int32_t* scratch = nullptr);
size_t organize_smem_bytes(const MapGeom& g, int order, int split_pmax);
size_t organize_scratch_bytes(const MapGeom& g, int order, int split_pmax);

// ---- attention + merge (bsa_attention.cu) ----------------------------------------------------
struct ForwardArgs {
    const void* Q;
    const void* K;
    const void* V;
    void* O;
    float* LSE;
    const WorkItem* items;
    const SplitRow* split_rows;
    const int32_t* tile_col;
    const uint64_t* tile_member;
    PlanCountersDev* counters;
    float* ws_O;    // [nslots][128][d] fp32, normalised partial outputs
    float* ws_LSE;  // [nslots][128]    fp32, partial log-sum-exp
    MapGeom g;
    int32_t d;
    int32_t stages;
    int32_t kernel;
    int32_t has_split;
    int32_t max_items;       // host-side upper bound of the item count
    int32_t max_split_rows;  // host-side upper bound
    int32_t num_sms;
    int32_t device;          // CUDA device the plan lives on
    int32_t f16;             // 1: Q, K, V, O are IEEE half (ping-pong-kernel plans only); 0: bf16
    int32_t nhd;             // 1: Q, K, V, O are stored [N][heads][d] (token-major); 0: [heads][N][d]
};
cudaError_t launch_forward(const ForwardArgs& a, cudaStream_t stream, const char** err_detail);
cudaError_t launch_merge(const ForwardArgs& a, cudaStream_t stream);  // the Split-K reduction kernel alone
// Row-block kernel (bsa_attention_rb.cu): 16-row physical Q tiles on the register-level tensor instruction.
constexpr int kKernelRowBlock = 5;
cudaError_t launch_forward_rb(const ForwardArgs& a, cudaStream_t stream, const char** err_detail);
int rb_max_chunk(int d);  // largest T_KV (keys per staged chunk) for head dimension d
// `stages` counts K buffers plus V buffers for the paired kernel (kernel 1), K = V ring depth for kernel 0
int attention_max_stages(int d, int T_KV, int kernel);
int attention_smem_bytes(int d, int T_KV, int stages, int kernel);

void count_launch(int n = 1);

}  // namespace bsa
