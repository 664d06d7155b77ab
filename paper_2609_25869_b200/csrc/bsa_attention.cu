// Main attention kernel and Split-K reduction kernel for sm_100a (paper Section 4: "Native CUDA
// catalog"; Section 2.3 data-compute pipeline; Section 4.3 Split-K).
//
// One persistent CTA per SM walks the ordered work-item list.  Inside a CTA the roles are
// warp-specialised:
//   warps 0-3  softmax / correction / epilogue: one thread per query row (TMEM lane), reads the
//              score tile S from tensor memory, applies the intra-tile membership mask, keeps the
//              online-softmax state (m, l) in registers, writes bf16 P back into tensor memory;
//   warp 4     TMA producer: gathers K and V tiles by tile index into shared-memory rings
//              (128-byte swizzle), and the Q tile once per work item;
//   warp 5     MMA issuer: tcgen05.mma S = Q K^T (both operands in shared memory) and
//              O += P V (P from tensor memory, V from shared memory, MN-major), fp32 accumulators
//              in tensor memory; tcgen05.commit signals the mbarriers.
// S is double-buffered so Q K^T of tile j+1 overlaps the softmax of tile j.
#include <cuda.h>
#include <cuda_bf16.h>
#include <math.h>

#include <atomic>

#include "bsa_common.h"
#include "sm100_ptx.cuh"

namespace bsa {

using namespace ptx;


// Optional timeline tracing (compile with -DBSA_TRACE): CTA 0 records clock64() at barrier events of the
// single-tile kernel, per role, into a device buffer that bsa_debug_trace_copy() reads back.
#if defined(BSA_TRACE) || defined(BSA_PHASES)
__device__ long long g_trace[12][4096];  // producer, Q K^T (or single) issuer, softmax warps 0-7, P V issuer (role 6 in the 7-warp kernel)
__device__ long long g_trace_aux[12][4];  // last tile's stamps inside softmax_tile, per warp
__device__ long long g_cta_times[2][4096];  // %globaltimer at entry and exit of every CTA of the ping-pong kernel
#endif
#ifdef BSA_TRACE
#define BSA_TRACE_DECL(n) int n = 0
#define BSA_TRACE_POINT(role, n, tag)                                              \
    do {                                                                           \
        if (blockIdx.x == 0 && (n) < 4096) g_trace[role][(n)++] = (clock64() << 8) | (tag); \
    } while (0)
#else
#define BSA_TRACE_DECL(n)
#define BSA_TRACE_POINT(role, n, tag)
#endif

// Optional phase accounting (compile with -DBSA_PHASES): every softmax warp of the ping-pong kernel adds up the clocks it
// spends between fixed points of its tile loop; CTA 1 writes the sums out at its end (bsa_debug_trace_copy, roles 2-9).
#ifdef BSA_PHASES
#define BSA_PH_DECL uint32_t ph_acc[8] = {0, 0, 0, 0, 0, 0, 0, 0}, ph_n = 0, ph_t = (uint32_t)clock()
#define BSA_PH(k) do { const uint32_t now_ = (uint32_t)clock(); ph_acc[k] += now_ - ph_t; ph_t = now_; } while (0)
#define BSA_STAMP(role, tile, k) do { if (blockIdx.x == 1 && (tile) >= 40 && (tile) < 240) g_trace[role][16 + 4 * ((tile) - 40) + (k)] = clock64(); } while (0)
#else
#define BSA_PH_DECL
#define BSA_PH(k)
#define BSA_STAMP(role, tile, k)
#endif

// Test hook (bsa_debug_withhold_arrival): while non-zero, the V producer of the ping-pong kernel leaves out the copy
// of the first tile of its CTA together with the arrival that would announce it.  Nothing is in flight for that slot,
// so nothing can fault; the waits that depend on the tile simply run out, which is how the give-up path (status word,
// copies in flight allowed to land, TMEM freed, kernel returns) is exercised without a protocol error.
__device__ int g_withhold_arrival = 0;

namespace {

constexpr int kMaxStages = 6;
constexpr int kThreads = 192;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS0 = 0, kColS1 = 128, kColO = 256;
constexpr uint32_t kColP0 = 384, kColP1 = 448;  // separate bf16 P buffers of the column-split kernel
constexpr float kRescaleThreshold = 8.0f;  // log2 units: P stays below 2^8 between rescales

struct AttnParams {
    const WorkItem* items;
    const int32_t* tile_col;
    const uint64_t* tile_member;
    PlanCountersDev* counters;
    __nv_bfloat16* O;
    float* LSE;
    float* ws_O;
    float* ws_LSE;
    unsigned long long full_member;
    int64_t o_head, o_row;  // element strides of O (and of Q) between heads and between token rows
    int32_t N;    // query tokens per head
    int32_t Nkv;  // key/value tokens per head
    int32_t lgBQ;   // log2(B_Q) when B_Q < 128, else 31 (row >> 31 == 0)
    int32_t lgBKV;  // log2(B_KV) when B_KV < T_KV, else 31
    int32_t sK;     // logical KV sub-blocks per tile
    int32_t stages;    // K ring depth (and V ring depth for the single-tile kernel)
    int32_t stages_v;  // V ring depth of the paired kernel
    float scale_log2;  // log2(e) / sqrt(d)
};

struct __align__(8) Barriers {
    uint64_t q_full, q_empty, o_free;
    uint64_t k_full[kMaxStages], k_empty[kMaxStages], v_full[kMaxStages], v_empty[kMaxStages];
    uint64_t s_full[2], p_ready[2], pv_done[2];
};

// One score tile of one query row (thread = row = TMEM lane): mask, running reference maximum,
// P = exp2(s * c2 - m_ref) rounded to bf16 and written to t_p (over S in place when t_p == t_s), running sum.
// The reference maximum moves only when the tile maximum exceeds it by kRescaleThreshold (log2
// units), so P stays below 2^8 and the running output needs rescaling (by `alpha`) only then.
template <int TK, bool F16 = false>
__device__ __forceinline__ void softmax_tile(uint32_t t_s, uint32_t t_p, bool need_mask, uint32_t row_bits, int lgBKV, int n_valid,
                                             float c2, bool not_first, float& m_ref, float& l, float& alpha,
                                             bool& rescale) {
    uint32_t r[TK];
#pragma unroll
    for (int c = 0; c < TK / 32; ++c) tmem_ld32(t_s + c * 32, &r[c * 32]);
    tc_wait_ld();
#ifdef BSA_TRACE
    if ((threadIdx.x & 31) == 0 && blockIdx.x == 0) g_trace_aux[threadIdx.x >> 5][0] = clock64();
#endif
    if (need_mask) {
        // B_KV >= 16: a group of 16 key columns lies inside one logical block, so one activity bit serves the group
#pragma unroll
        for (int gq = 0; gq < TK / 16; ++gq) {
            const bool grp = (row_bits >> ((gq * 16) >> lgBKV)) & 1u;
#pragma unroll
            for (int i = gq * 16; i < gq * 16 + 16; ++i) r[i] = (grp && i < n_valid) ? r[i] : 0xff800000u;  // -inf
        }
    }
    float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
    for (int i = 0; i < TK; i += 8) {
        m0 = max3(m0, __uint_as_float(r[i]), __uint_as_float(r[i + 1]));
        m1 = max3(m1, __uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
        m2 = max3(m2, __uint_as_float(r[i + 4]), __uint_as_float(r[i + 5]));
        m3 = max3(m3, __uint_as_float(r[i + 6]), __uint_as_float(r[i + 7]));
    }
    const float mx2 = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3)) * c2;
    alpha = 1.f;
    rescale = false;
    if (mx2 > m_ref + kRescaleThreshold) {
        alpha = ex2_approx(m_ref - mx2);  // m_ref = -inf -> 0
        rescale = not_first && (m_ref != -INFINITY);
        m_ref = mx2;
    }
    const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
#ifdef BSA_TRACE
    if ((threadIdx.x & 31) == 0 && blockIdx.x == 0) g_trace_aux[threadIdx.x >> 5][1] = clock64();
#endif
    // scale-and-shift and the row sums run as packed two-lane fp32 operations
    const uint64_t c22 = pack_f32x2(c2, c2), nm2 = pack_f32x2(neg_m, neg_m);
    uint64_t sum01 = pack_f32x2(0.f, 0.f), sum23 = sum01;
#pragma unroll
    for (int i = 0; i < TK; i += 4) {
        float x0, x1, x2, x3;
        unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), c22, nm2), x0, x1);
        unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(r[i + 2]), __uint_as_float(r[i + 3])), c22, nm2), x2, x3);
        const float p0 = ex2_approx(x0), p1 = ex2_approx(x1), p2 = ex2_approx(x2), p3 = ex2_approx(x3);
        sum01 = add_f32x2(sum01, pack_f32x2(p0, p1));
        sum23 = add_f32x2(sum23, pack_f32x2(p2, p3));
        r[i / 2] = pack_16x2<F16>(p0, p1);
        r[i / 2 + 1] = pack_16x2<F16>(p2, p3);
    }
    float s0, s1, s2, s3;
    unpack_f32x2(sum01, s0, s1);
    unpack_f32x2(sum23, s2, s3);
#ifdef BSA_TRACE
    if ((threadIdx.x & 31) == 0 && blockIdx.x == 0) g_trace_aux[threadIdx.x >> 5][2] = clock64();
#endif
#pragma unroll
    for (int c = 0; c < TK / 32; ++c) tmem_st16(t_p + c * 16, &r[c * 16]);
    l = l * alpha + ((s0 + s1) + (s2 + s3));
}

// DUAL = true adds a seventh warp so that Q K^T and P V are issued by two different threads: the
// Q K^T issuer runs up to two tiles ahead (S is double-buffered) instead of stalling behind the wait
// for the softmax of the previous tile; ordering between the two issuers is carried by mbarriers only.
template <int D, int TK, bool DUAL, bool F16>
__global__ void __launch_bounds__(DUAL ? kThreads + 32 : kThreads, 1)
bsa_attention_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                     const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
    constexpr int NSUB = D / 64;              // 64-column (128-byte) sub-tiles per row
    constexpr int Q_SUB = kTQ * 128;          // bytes of one [128][64] bf16 sub-tile
    constexpr int KV_SUB = TK * 128;          // bytes of one [TK][64] bf16 sub-tile
    constexpr int KV_TILE = NSUB * KV_SUB;
    // dynamic shared memory starts on a 1024-byte boundary (the swizzled tiles need it); checked below
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t* sQ = smem;
    uint8_t* sK = sQ + NSUB * Q_SUB;
    uint8_t* sV = sK + p.stages * KV_TILE;
    __shared__ Barriers bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ uint32_t abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (smem_u32(smem) & 1023u) {  // never expected; fail with a status instead of corrupting tiles
        if (tid == 0) atomicExch(&p.counters->status, (int)BSA_ERR_CUDA);
        return;
    }
    const int NS = p.stages;

    if (tid == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bars.q_full), 1);
        mbar_init(smem_u32(&bars.q_empty), 1);
        mbar_init(smem_u32(&bars.o_free), 128);
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(smem_u32(&bars.k_full[s]), 1);
            mbar_init(smem_u32(&bars.k_empty[s]), 1);
            mbar_init(smem_u32(&bars.v_full[s]), 1);
            mbar_init(smem_u32(&bars.v_empty[s]), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&bars.s_full[s]), 1);
            mbar_init(smem_u32(&bars.p_ready[s]), 128);
            mbar_init(smem_u32(&bars.pv_done[s]), 1);
        }
        fence_mbar_init();
    }
    if (warp == 5) {
        tmem_alloc(smem_u32(&tmem_base_s), kTmemCols);
        tmem_relinquish();
    }
    if (warp == 4 && lane == 0) {
        prefetch_tensormap(&tmQ);
        prefetch_tensormap(&tmK);
        prefetch_tensormap(&tmV);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    volatile uint32_t* abortp = &abort_flag;
    const int n_items = p.counters->nitems;

    if (warp == 4) {
        // =========================== TMA producer ===========================
        if (lane == 0) {
            uint32_t itq = 0, g = 0;
            bool ok = true;
            BSA_TRACE_DECL(tn);
            for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
                const WorkItem it = p.items[idx];
                if (it.ntiles == 0) continue;
                ok = mbar_wait(smem_u32(&bars.q_empty), (itq & 1) ^ 1, abortp);
                if (!ok) break;
                mbar_arrive_expect_tx(smem_u32(&bars.q_full), NSUB * Q_SUB);
                for (int s = 0; s < NSUB; ++s)
                    tma_load_3d(smem_u32(sQ + s * Q_SUB), &tmQ, smem_u32(&bars.q_full), s * 64, it.q_tile * kTQ, it.head);
                int col_next = p.tile_col[it.tile_begin];  // tile metadata is fetched one tile ahead of its use
                for (int j = it.tile_begin; j < it.tile_end; ++j, ++g) {
                    const int col_cur = col_next;
                    if (j + 1 < it.tile_end) col_next = p.tile_col[j + 1];
                    const int stage = g % NS;
                    const uint32_t ph = (g / NS) & 1;
                    const int kv0 = col_cur * TK;
                    ok = mbar_wait(smem_u32(&bars.k_empty[stage]), ph ^ 1, abortp);
                    if (!ok) break;
                    BSA_TRACE_POINT(0, tn, 20);
                    mbar_arrive_expect_tx(smem_u32(&bars.k_full[stage]), KV_TILE);
                    for (int s = 0; s < NSUB; ++s)
                        tma_load_3d(smem_u32(sK + stage * KV_TILE + s * KV_SUB), &tmK, smem_u32(&bars.k_full[stage]),
                                    s * 64, kv0, it.head);
                    ok = mbar_wait(smem_u32(&bars.v_empty[stage]), ph ^ 1, abortp);
                    if (!ok) break;
                    BSA_TRACE_POINT(0, tn, 22);
                    mbar_arrive_expect_tx(smem_u32(&bars.v_full[stage]), KV_TILE);
                    for (int s = 0; s < NSUB; ++s)
                        tma_load_3d(smem_u32(sV + stage * KV_TILE + s * KV_SUB), &tmV, smem_u32(&bars.v_full[stage]),
                                    s * 64, kv0, it.head);
                }
                ++itq;
            }
            if (!ok) {
                // let copies in flight land before the CTA's shared memory goes away
                const uint64_t t0 = globaltimer_ns();
                while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
            }
        }
    } else if (warp == 5 && !DUAL) {
        // =========================== MMA issuer ===========================
        if (lane == 0) {
            constexpr uint32_t idesc_qk = make_idesc_f32(kTQ, TK, 0, 0, F16);
            constexpr uint32_t idesc_pv = make_idesc_f32(kTQ, D, 0, 1, F16);
            const uint64_t descQ = make_smem_desc_sw128(smem_u32(sQ), 16, 1024);
            const uint64_t descK = make_smem_desc_sw128(smem_u32(sK), 16, 1024);
            const uint64_t descV = make_smem_desc_sw128(smem_u32(sV), KV_SUB, 1024);
            uint32_t itq = 0, g = 0;
            bool ok = true;
            BSA_TRACE_DECL(tn);
            for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
                const int n = p.items[idx].ntiles;
                if (n == 0) continue;
                ok = mbar_wait(smem_u32(&bars.q_full), itq & 1, abortp);
                if (!ok) break;
                for (int j = 0; j <= n && ok; ++j) {
                    if (j < n) {
                        const uint32_t gs = g + j;
                        const int stage = gs % NS;
                        const uint32_t ph = (gs / NS) & 1, sb = gs & 1;
                        ok = mbar_wait(smem_u32(&bars.k_full[stage]), ph, abortp);
                        if (!ok) break;
                        BSA_TRACE_POINT(1, tn, 1);
                        tc_fence_after();
                        // S[sb] = Q K^T.  The previous user of S[sb] (P of tile gs-2, read by its PV MMA)
                        // precedes this MMA in issue order on the same pipe.
                        const uint32_t d_s = tmem + (sb ? kColS1 : kColS0);
#pragma unroll
                        for (int k = 0; k < D / 16; ++k) {
                            const uint64_t a = descQ + (uint64_t)(((k / 4) * Q_SUB + (k % 4) * 32) >> 4);
                            const uint64_t b = descK + (uint64_t)((stage * KV_TILE + (k / 4) * KV_SUB + (k % 4) * 32) >> 4);
                            mma_ss(d_s, a, b, idesc_qk, k > 0);
                        }
                        mma_commit(smem_u32(&bars.k_empty[stage]));
                        mma_commit(smem_u32(&bars.s_full[sb]));
                        BSA_TRACE_POINT(1, tn, 2);
                        if (j == n - 1) mma_commit(smem_u32(&bars.q_empty));
                    }
                    if (j >= 1) {
                        const uint32_t gp = g + j - 1;
                        const int stage = gp % NS;
                        const uint32_t ph = (gp / NS) & 1, sb = gp & 1;
                        ok = mbar_wait(smem_u32(&bars.p_ready[sb]), (gp >> 1) & 1, abortp);
                        if (!ok) break;
                        BSA_TRACE_POINT(1, tn, 3);
                        ok = mbar_wait(smem_u32(&bars.v_full[stage]), ph, abortp);
                        if (!ok) break;
                        BSA_TRACE_POINT(1, tn, 4);
                        if (j == 1) {
                            ok = mbar_wait(smem_u32(&bars.o_free), (itq & 1) ^ 1, abortp);
                            if (!ok) break;
                        }
                        tc_fence_after();
                        const uint32_t a_p = tmem + (sb ? kColS1 : kColS0);
#pragma unroll
                        for (int k = 0; k < TK / 16; ++k) {
                            const uint64_t b = descV + (uint64_t)((stage * KV_TILE + k * 2048) >> 4);
                            mma_ts(tmem + kColO, a_p + k * 8, b, idesc_pv, (j > 1 || k > 0) ? 1u : 0u);
                        }
                        mma_commit(smem_u32(&bars.v_empty[stage]));
                        mma_commit(smem_u32(&bars.pv_done[sb]));
                        BSA_TRACE_POINT(1, tn, 5);
                    }
                }
                g += n;
                ++itq;
            }
        }
    } else if (warp == 5) {
        // =========================== Q K^T issuer (DUAL) ===========================
        if (lane == 0) {
            constexpr uint32_t idesc_qk = make_idesc_f32(kTQ, TK, 0, 0, F16);
            const uint64_t descQ = make_smem_desc_sw128(smem_u32(sQ), 16, 1024);
            const uint64_t descK = make_smem_desc_sw128(smem_u32(sK), 16, 1024);
            uint32_t itq = 0, g = 0;
            bool ok = true;
            BSA_TRACE_DECL(tn);
            for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
                const int n = p.items[idx].ntiles;
                if (n == 0) continue;
                ok = mbar_wait(smem_u32(&bars.q_full), itq & 1, abortp);
                if (!ok) break;
                for (int j = 0; j < n; ++j) {
                    const uint32_t gs = g + j;
                    const int stage = gs % NS;
                    const uint32_t ph = (gs / NS) & 1, sb = gs & 1;
                    ok = mbar_wait(smem_u32(&bars.k_full[stage]), ph, abortp);
                    if (!ok) break;
                    BSA_TRACE_POINT(1, tn, 1);
                    // S[sb] still holds P of tile gs-2 (written in place) until that tile's P V has completed.
                    // (Measured: giving P its own columns so that Q K^T may start right after the softmax of
                    // tile gs-2 was slower -- the early Q K^T delays the P V the softmax chain is waiting for.)
                    if (gs >= 2) {
                        ok = mbar_wait(smem_u32(&bars.pv_done[sb]), ((gs >> 1) - 1) & 1, abortp);
                        if (!ok) break;
                    }
                    BSA_TRACE_POINT(1, tn, 6);
                    tc_fence_after();
                    const uint32_t d_s = tmem + (sb ? kColS1 : kColS0);
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint64_t a = descQ + (uint64_t)(((k / 4) * Q_SUB + (k % 4) * 32) >> 4);
                        const uint64_t b = descK + (uint64_t)((stage * KV_TILE + (k / 4) * KV_SUB + (k % 4) * 32) >> 4);
                        mma_ss(d_s, a, b, idesc_qk, k > 0);
                    }
                    mma_commit(smem_u32(&bars.k_empty[stage]));
                    mma_commit(smem_u32(&bars.s_full[sb]));
                    BSA_TRACE_POINT(1, tn, 2);
                    if (j == n - 1) mma_commit(smem_u32(&bars.q_empty));
                }
                g += n;
                ++itq;
            }
        }
    } else if (warp == 6) {
        // =========================== P V issuer (DUAL) ===========================
        if (lane == 0) {
            constexpr uint32_t idesc_pv = make_idesc_f32(kTQ, D, 0, 1, F16);
            const uint64_t descV = make_smem_desc_sw128(smem_u32(sV), KV_SUB, 1024);
            uint32_t itq = 0, g = 0;
            bool ok = true;
            BSA_TRACE_DECL(tn);
            for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
                const int n = p.items[idx].ntiles;
                if (n == 0) continue;
                for (int j = 0; j < n; ++j) {
                    const uint32_t gp = g + j;
                    const int stage = gp % NS;
                    const uint32_t ph = (gp / NS) & 1, sb = gp & 1;
                    ok = mbar_wait(smem_u32(&bars.p_ready[sb]), (gp >> 1) & 1, abortp);
                    if (!ok) break;
                    BSA_TRACE_POINT(6, tn, 3);
                    ok = mbar_wait(smem_u32(&bars.v_full[stage]), ph, abortp);
                    if (!ok) break;
                    if (j == 0) {
                        ok = mbar_wait(smem_u32(&bars.o_free), (itq & 1) ^ 1, abortp);
                        if (!ok) break;
                    }
                    tc_fence_after();
                    const uint32_t a_p = tmem + (sb ? kColS1 : kColS0);
#pragma unroll
                    for (int k = 0; k < TK / 16; ++k) {
                        const uint64_t b = descV + (uint64_t)((stage * KV_TILE + k * 2048) >> 4);
                        mma_ts(tmem + kColO, a_p + k * 8, b, idesc_pv, (j > 0 || k > 0) ? 1u : 0u);
                    }
                    mma_commit(smem_u32(&bars.v_empty[stage]));
                    mma_commit(smem_u32(&bars.pv_done[sb]));
                    BSA_TRACE_POINT(6, tn, 5);
                }
                g += n;
                ++itq;
            }
        }
    } else {
        // =========================== softmax / correction / epilogue ===========================
        const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
        uint32_t itq = 0, g = 0;
        bool ok = true;
        BSA_TRACE_DECL(tn);
        const float c2 = p.scale_log2;
        const unsigned long long sub_mask = (p.sK >= 64) ? ~0ull : ((1ull << p.sK) - 1ull);
        for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
            const WorkItem it = p.items[idx];
            const int row = it.q_tile * kTQ + tid;
            const bool row_ok = row < p.N;
            if (it.ntiles == 0) {
                // no physical tile touches this Q tile row: O = 0, LSE = -inf
                if (row_ok) {
                    uint4* o = reinterpret_cast<uint4*>(p.O + ((size_t)it.head * p.o_head + (size_t)row * p.o_row));
#pragma unroll
                    for (int c = 0; c < D / 8; ++c) o[c] = make_uint4(0, 0, 0, 0);
                    p.LSE[(size_t)it.head * p.N + row] = -INFINITY;
                }
                continue;
            }
            float m_ref = -INFINITY, l = 0.f;
            int col_next = p.tile_col[it.tile_begin];  // tile metadata is fetched one tile ahead of its use
            unsigned long long member_next = p.tile_member[it.tile_begin];
            for (int j = 0; j < it.ntiles; ++j) {
                const uint32_t gs = g + j, sb = gs & 1;
                const int kv0 = col_next * TK;
                const unsigned long long member = member_next;
                if (j + 1 < it.ntiles) {
                    col_next = p.tile_col[it.tile_begin + j + 1];
                    member_next = p.tile_member[it.tile_begin + j + 1];
                }
                const bool need_mask = (member != p.full_member) || (kv0 + TK > p.Nkv);
                const uint32_t row_bits = (uint32_t)((member >> ((tid >> p.lgBQ) * p.sK)) & sub_mask);
                const int n_valid = p.Nkv - kv0;  // columns >= n_valid do not exist
                ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.s_full[sb]), (gs >> 1) & 1, abortp));
                if (!ok) break;
                if (lane == 0) BSA_TRACE_POINT(2 + warp, tn, 10);
                tc_fence_after();
                const uint32_t t_s = tmem + lane_base + (sb ? kColS1 : kColS0);
                float alpha;
                bool rescale;
                softmax_tile<TK, F16>(t_s, t_s, need_mask, row_bits, p.lgBKV, n_valid, c2, j > 0, m_ref, l, alpha, rescale);
#ifdef BSA_TRACE
                if (lane == 0 && blockIdx.x == 0 && tn + 3 < 4096) {
                    g_trace[2 + warp][tn++] = (g_trace_aux[warp][0] << 8) | 11;
                    g_trace[2 + warp][tn++] = (g_trace_aux[warp][1] << 8) | 12;
                    g_trace[2 + warp][tn++] = (g_trace_aux[warp][2] << 8) | 14;
                }
#endif
                if (lane == 0) BSA_TRACE_POINT(2 + warp, tn, 13);
                // ---- correction: rescale the running output when the reference moved ----
                if (j > 0 && __any_sync(0xffffffffu, rescale)) {
                    const uint32_t gp = gs - 1;
                    ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.pv_done[gp & 1]), (gp >> 1) & 1, abortp));
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t t_o = tmem + lane_base + kColO;
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t r[32];
                        tmem_ld32(t_o + c * 32, r);
                        tc_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                        tmem_st32(t_o + c * 32, r);
                    }
                }
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(smem_u32(&bars.p_ready[sb]));
                if (lane == 0) BSA_TRACE_POINT(2 + warp, tn, 16);
            }
            if (!ok) break;
            // ---- epilogue ----
            {
                const uint32_t gl = g + it.ntiles - 1;
                ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.pv_done[gl & 1]), (gl >> 1) & 1, abortp));
                if (!ok) break;
                tc_fence_after();
                const float inv_l = (l > 0.f) ? 1.f / l : 0.f;
                const float lse = (l > 0.f) ? fmaf(m_ref, 0.6931471805599453f, logf(l)) : -INFINITY;
                const uint32_t t_o = tmem + lane_base + kColO;
                if (it.nparts == 1) {
                    __nv_bfloat16* orow = p.O + ((size_t)it.head * p.o_head + (size_t)row * p.o_row);
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t r[32];
                        tmem_ld32(t_o + c * 32, r);
                        tc_wait_ld();
                        if (row_ok) {
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                uint4 v;
                                v.x = pack_16x2<F16>(__uint_as_float(r[q * 8 + 0]) * inv_l, __uint_as_float(r[q * 8 + 1]) * inv_l);
                                v.y = pack_16x2<F16>(__uint_as_float(r[q * 8 + 2]) * inv_l, __uint_as_float(r[q * 8 + 3]) * inv_l);
                                v.z = pack_16x2<F16>(__uint_as_float(r[q * 8 + 4]) * inv_l, __uint_as_float(r[q * 8 + 5]) * inv_l);
                                v.w = pack_16x2<F16>(__uint_as_float(r[q * 8 + 6]) * inv_l, __uint_as_float(r[q * 8 + 7]) * inv_l);
                                *reinterpret_cast<uint4*>(orow + c * 32 + q * 8) = v;
                            }
                        }
                    }
                    if (row_ok) p.LSE[(size_t)it.head * p.N + row] = lse;
                } else {
                    float* orow = p.ws_O + ((size_t)it.ws_slot * kTQ + tid) * D;
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t r[32];
                        tmem_ld32(t_o + c * 32, r);
                        tc_wait_ld();
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            float4 v = make_float4(__uint_as_float(r[q * 4 + 0]) * inv_l, __uint_as_float(r[q * 4 + 1]) * inv_l,
                                                   __uint_as_float(r[q * 4 + 2]) * inv_l, __uint_as_float(r[q * 4 + 3]) * inv_l);
                            *reinterpret_cast<float4*>(orow + c * 32 + q * 4) = v;
                        }
                    }
                    p.ws_LSE[(size_t)it.ws_slot * kTQ + tid] = lse;
                }
                tc_fence_before();
                mbar_arrive(smem_u32(&bars.o_free));
            }
            g += it.ntiles;
            ++itq;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (tid == 0 && abort_flag) atomicExch(&p.counters->status, (int)BSA_ERR_DEVICE_TIMEOUT);
    if (warp == 5) tmem_dealloc(tmem, kTmemCols);
}

// ==========================================================================================
// Paired kernel: one CTA owns a 256-row physical Q tile as two 128-row MMA slots.  Both slots
// walk the same (merged) KV tile list, so every K/V tile is fetched into shared memory once and
// feeds up to two Q tiles; a slot whose membership word for a tile is zero skips it.  Each slot
// has its own softmax warpgroup, S/P columns and O accumulator in tensor memory; the single MMA
// warp alternates between the slots (PV of the previous tile, then Q K^T of the next), so one
// slot's softmax runs under the other slot's MMAs.
//   warps 0-3 / 4-7 : softmax + correction + epilogue of slot 0 / slot 1 (more registers)
//   warp 8          : TMA producer    warp 9 : Q K^T issuer    warp 10 : P V issuer (this warpgroup gives registers back)
// Register budget: 384 threads launch with 168 registers each (504 per lane across the three
// warpgroups); setmaxnreg moves them to 216 + 216 + 72 = 504.  The sum must not exceed the launch
// allocation, otherwise the second setmaxnreg.inc never gets its registers and the CTA stalls.
// ==========================================================================================
constexpr int kPairThreads = 384;

struct __align__(8) PairBarriers {
    uint64_t q_full, q_empty;
    uint64_t k_full[kMaxStages], k_empty[kMaxStages], v_full[kMaxStages], v_empty[kMaxStages];
    uint64_t s_full[2], p_ready[2], pv_done[2], o_free[2];
};

template <int R>
__device__ __forceinline__ void reg_inc() {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(R));
}
template <int R>
__device__ __forceinline__ void reg_dec() {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(R));
}

template <int D, int TK>
__global__ void __launch_bounds__(kPairThreads, 1)
bsa_attention_pair_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                          const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
    constexpr int NSUB = D / 64;
    constexpr int Q_SUB = kTQ * 128;
    constexpr int Q_TILE = NSUB * Q_SUB;
    constexpr int KV_SUB = TK * 128;
    constexpr int KV_TILE = NSUB * KV_SUB;
    // dynamic shared memory starts on a 1024-byte boundary (the swizzled tiles need it); checked below
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t* sQ = smem;                       // [2 slots][NSUB][128][64]
    uint8_t* sK = sQ + 2 * Q_TILE;            // [stages][NSUB][TK][64]
    uint8_t* sV = sK + p.stages * KV_TILE;    // [stages_v][NSUB][TK][64]
    __shared__ PairBarriers bars;
    __shared__ uint32_t tmem_base_s;
    __shared__ uint32_t abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (smem_u32(smem) & 1023u) {  // never expected; fail with a status instead of corrupting tiles
        if (tid == 0) atomicExch(&p.counters->status, (int)BSA_ERR_CUDA);
        return;
    }
    const int NSK = p.stages, NSV = p.stages_v;

    if (tid == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bars.q_full), 1);
        mbar_init(smem_u32(&bars.q_empty), 1);
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(smem_u32(&bars.k_full[s]), 1);
            mbar_init(smem_u32(&bars.k_empty[s]), 1);
            mbar_init(smem_u32(&bars.v_full[s]), 1);
            mbar_init(smem_u32(&bars.v_empty[s]), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&bars.s_full[s]), 1);
            mbar_init(smem_u32(&bars.p_ready[s]), 128);
            mbar_init(smem_u32(&bars.pv_done[s]), 1);
            mbar_init(smem_u32(&bars.o_free[s]), 128);
        }
        fence_mbar_init();
    }
    if (warp == 9) {
        tmem_alloc(smem_u32(&tmem_base_s), kTmemCols);
        tmem_relinquish();
    }
    if (warp == 8 && lane == 0) {
        prefetch_tensormap(&tmQ);
        prefetch_tensormap(&tmK);
        prefetch_tensormap(&tmV);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    volatile uint32_t* abortp = &abort_flag;
    const int n_items = p.counters->nitems;

    if (warp >= 8) {
        reg_dec<72>();
        if (warp == 8 && lane == 0) {
            // =========================== TMA producer ===========================
            uint32_t itq = 0, g = 0;
            bool ok = true;
            for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
                const WorkItem it = p.items[idx];
                if (it.ntiles == 0) continue;
                ok = mbar_wait(smem_u32(&bars.q_empty), (itq & 1) ^ 1, abortp);
                if (!ok) break;
                mbar_arrive_expect_tx(smem_u32(&bars.q_full), 2 * Q_TILE);
                for (int x = 0; x < 2; ++x)
                    for (int s = 0; s < NSUB; ++s)
                        tma_load_3d(smem_u32(sQ + x * Q_TILE + s * Q_SUB), &tmQ, smem_u32(&bars.q_full), s * 64,
                                    it.q_tile * (2 * kTQ) + x * kTQ, it.head);
                int col_next = p.tile_col[it.tile_begin];  // tile metadata is fetched one tile ahead of its use
                for (int j = it.tile_begin; j < it.tile_end; ++j, ++g) {
                    const int col_cur = col_next;
                    if (j + 1 < it.tile_end) col_next = p.tile_col[j + 1];
                    const int sk = g % NSK, sv = g % NSV;
                    const uint32_t phk = (g / NSK) & 1, phv = (g / NSV) & 1;
                    const int kv0 = col_cur * TK;
                    ok = mbar_wait(smem_u32(&bars.k_empty[sk]), phk ^ 1, abortp);
                    if (!ok) break;
                    mbar_arrive_expect_tx(smem_u32(&bars.k_full[sk]), KV_TILE);
                    for (int s = 0; s < NSUB; ++s)
                        tma_load_3d(smem_u32(sK + sk * KV_TILE + s * KV_SUB), &tmK, smem_u32(&bars.k_full[sk]), s * 64,
                                    kv0, it.head);
                    ok = mbar_wait(smem_u32(&bars.v_empty[sv]), phv ^ 1, abortp);
                    if (!ok) break;
                    mbar_arrive_expect_tx(smem_u32(&bars.v_full[sv]), KV_TILE);
                    for (int s = 0; s < NSUB; ++s)
                        tma_load_3d(smem_u32(sV + sv * KV_TILE + s * KV_SUB), &tmV, smem_u32(&bars.v_full[sv]), s * 64,
                                    kv0, it.head);
                }
                ++itq;
            }
            if (!ok) {
                const uint64_t t0 = globaltimer_ns();
                while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
            }
        } else if (warp == 9 && lane == 0) {
            // =========================== Q K^T issuer (both slots) ===========================
            constexpr uint32_t idesc_qk = make_idesc_bf16_f32(kTQ, TK, 0, 0);
            const uint64_t descQ = make_smem_desc_sw128(smem_u32(sQ), 16, 1024);
            const uint64_t descK = make_smem_desc_sw128(smem_u32(sK), 16, 1024);
            uint32_t itq = 0, g = 0;
            uint32_t nqk[2] = {0, 0};  // Q K^T tiles issued per slot
            bool ok = true;
            for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
                const WorkItem it = p.items[idx];
                const int n = it.ntiles;
                if (n == 0) continue;
                ok = mbar_wait(smem_u32(&bars.q_full), itq & 1, abortp);
                if (!ok) break;
                ulonglong2 mem_next = *reinterpret_cast<const ulonglong2*>(p.tile_member + (size_t)it.tile_begin * 2);
                for (int j = 0; j < n && ok; ++j) {
                    const uint32_t gj = g + j;
                    const int sk = gj % NSK;
                    const ulonglong2 mem = mem_next;
                    if (j + 1 < n)
                        mem_next = *reinterpret_cast<const ulonglong2*>(p.tile_member + (size_t)(it.tile_begin + j + 1) * 2);
                    ok = mbar_wait(smem_u32(&bars.k_full[sk]), (gj / NSK) & 1, abortp);
                    if (!ok) break;
#pragma unroll
                    for (int x = 0; x < 2; ++x) {
                        if ((x == 0 ? mem.x : mem.y) == 0ull) continue;
                        // S_x holds the bf16 P of the slot's previous tile until that tile's P V has completed
                        if (nqk[x] >= 1) {
                            ok = mbar_wait(smem_u32(&bars.pv_done[x]), (nqk[x] - 1) & 1, abortp);
                            if (!ok) break;
                        }
                        tc_fence_after();
                        const uint32_t d_s = tmem + x * 128;
#pragma unroll
                        for (int k = 0; k < D / 16; ++k) {
                            const uint64_t a = descQ + (uint64_t)((x * Q_TILE + (k / 4) * Q_SUB + (k % 4) * 32) >> 4);
                            const uint64_t b = descK + (uint64_t)((sk * KV_TILE + (k / 4) * KV_SUB + (k % 4) * 32) >> 4);
                            mma_ss(d_s, a, b, idesc_qk, k > 0);
                        }
                        mma_commit(smem_u32(&bars.s_full[x]));
                        ++nqk[x];
                    }
                    if (!ok) break;
                    mma_commit(smem_u32(&bars.k_empty[sk]));
                }
                if (!ok) break;
                mma_commit(smem_u32(&bars.q_empty));
                g += n;
                ++itq;
            }
        } else if (warp == 10 && lane == 0) {
            // =========================== P V issuer (both slots) ===========================
            constexpr uint32_t idesc_pv = make_idesc_bf16_f32(kTQ, D, 0, 1);
            const uint64_t descV = make_smem_desc_sw128(smem_u32(sV), KV_SUB, 1024);
            uint32_t g = 0;
            uint32_t npv[2] = {0, 0};  // P V tiles issued per slot: phase of p_ready / pv_done
            uint32_t oit[2] = {0, 0};  // items in which the slot had tiles: phase of o_free
            bool ok = true;
            for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
                const WorkItem it = p.items[idx];
                const int n = it.ntiles;
                if (n == 0) continue;
                bool started[2] = {false, false};
                ulonglong2 mem_next = *reinterpret_cast<const ulonglong2*>(p.tile_member + (size_t)it.tile_begin * 2);
                for (int j = 0; j < n && ok; ++j) {
                    const uint32_t gj = g + j;
                    const int sv = gj % NSV;
                    const ulonglong2 mem = mem_next;
                    if (j + 1 < n)
                        mem_next = *reinterpret_cast<const ulonglong2*>(p.tile_member + (size_t)(it.tile_begin + j + 1) * 2);
                    ok = mbar_wait(smem_u32(&bars.v_full[sv]), (gj / NSV) & 1, abortp);
                    if (!ok) break;
#pragma unroll
                    for (int x = 0; x < 2; ++x) {
                        if ((x == 0 ? mem.x : mem.y) == 0ull) continue;
                        ok = mbar_wait(smem_u32(&bars.p_ready[x]), npv[x] & 1, abortp);
                        if (!ok) break;
                        if (!started[x]) {
                            ok = mbar_wait(smem_u32(&bars.o_free[x]), (oit[x] & 1) ^ 1, abortp);
                            if (!ok) break;
                        }
                        tc_fence_after();
                        const uint32_t d_o = tmem + kColO + x * 128, a_p = tmem + x * 128;
#pragma unroll
                        for (int k = 0; k < TK / 16; ++k) {
                            const uint64_t b = descV + (uint64_t)((sv * KV_TILE + k * 2048) >> 4);
                            mma_ts(d_o, a_p + k * 8, b, idesc_pv, (started[x] || k > 0) ? 1u : 0u);
                        }
                        mma_commit(smem_u32(&bars.pv_done[x]));
                        ++npv[x];
                        started[x] = true;
                    }
                    if (!ok) break;
                    mma_commit(smem_u32(&bars.v_empty[sv]));
                }
                if (!ok) break;
                for (int x = 0; x < 2; ++x)
                    if (started[x]) ++oit[x];
                g += n;
            }
        }
    } else {
        // =========================== softmax / correction / epilogue of slot x ===========================
        reg_inc<216>();
        const int x = warp >> 2;
        const int tw = tid & 127;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t t_s = tmem + lane_base + x * 128;
        const uint32_t t_o = tmem + lane_base + kColO + x * 128;
        uint32_t cnt = 0;  // tiles this slot has processed: phase of s_full / p_ready / pv_done
        bool ok = true;
        const float c2 = p.scale_log2;
        const unsigned long long sub_mask = (p.sK >= 64) ? ~0ull : ((1ull << p.sK) - 1ull);
        for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
            const WorkItem it = p.items[idx];
            const int row = it.q_tile * (2 * kTQ) + x * kTQ + tw;
            const bool row_ok = row < p.N;
            float m_ref = -INFINITY, l = 0.f;
            int nmine = 0;
            int col_next = 0;
            unsigned long long member_next = 0ull;
            if (it.ntiles > 0) {  // tile metadata is fetched one tile ahead of its use
                col_next = p.tile_col[it.tile_begin];
                member_next = p.tile_member[(size_t)it.tile_begin * 2 + x];
            }
            for (int j = 0; j < it.ntiles; ++j) {
                const unsigned long long member = member_next;
                const int kv0 = col_next * TK;
                if (j + 1 < it.ntiles) {
                    col_next = p.tile_col[it.tile_begin + j + 1];
                    member_next = p.tile_member[(size_t)(it.tile_begin + j + 1) * 2 + x];
                }
                if (member == 0ull) continue;
                const bool need_mask = (member != p.full_member) || (kv0 + TK > p.Nkv);
                const uint32_t row_bits = (uint32_t)((member >> ((tw >> p.lgBQ) * p.sK)) & sub_mask);
                const int n_valid = p.Nkv - kv0;
                ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.s_full[x]), cnt & 1, abortp));
                if (!ok) break;
                tc_fence_after();
                float alpha;
                bool rescale;
                softmax_tile<TK>(t_s, t_s, need_mask, row_bits, p.lgBKV, n_valid, c2, nmine > 0, m_ref, l, alpha, rescale);
                if (nmine > 0 && __any_sync(0xffffffffu, rescale)) {
                    ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.pv_done[x]), (cnt - 1) & 1, abortp));
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t r[32];
                        tmem_ld32(t_o + c * 32, r);
                        tc_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                        tmem_st32(t_o + c * 32, r);
                    }
                }
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(smem_u32(&bars.p_ready[x]));
                ++cnt;
                ++nmine;
            }
            if (!ok) break;
            if (nmine == 0) {
                // no tile of this item reaches this slot's rows: O = 0, LSE = -inf (or an empty partial state)
                if (it.nparts == 1) {
                    if (row_ok) {
                        uint4* o = reinterpret_cast<uint4*>(p.O + ((size_t)it.head * p.o_head + (size_t)row * p.o_row));
#pragma unroll
                        for (int c = 0; c < D / 8; ++c) o[c] = make_uint4(0, 0, 0, 0);
                        p.LSE[(size_t)it.head * p.N + row] = -INFINITY;
                    }
                } else {
                    float4* o = reinterpret_cast<float4*>(p.ws_O + ((size_t)(it.ws_slot + x) * kTQ + tw) * D);
#pragma unroll
                    for (int c = 0; c < D / 4; ++c) o[c] = make_float4(0.f, 0.f, 0.f, 0.f);
                    p.ws_LSE[(size_t)(it.ws_slot + x) * kTQ + tw] = -INFINITY;
                }
                continue;
            }
            ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.pv_done[x]), (cnt - 1) & 1, abortp));
            if (!ok) break;
            tc_fence_after();
            const float inv_l = (l > 0.f) ? 1.f / l : 0.f;
            const float lse = (l > 0.f) ? fmaf(m_ref, 0.6931471805599453f, logf(l)) : -INFINITY;
            if (it.nparts == 1) {
                __nv_bfloat16* orow = p.O + ((size_t)it.head * p.o_head + (size_t)row * p.o_row);
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t r[32];
                    tmem_ld32(t_o + c * 32, r);
                    tc_wait_ld();
                    if (row_ok) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            uint4 v;
                            v.x = pack_bf16x2(__uint_as_float(r[q * 8 + 0]) * inv_l, __uint_as_float(r[q * 8 + 1]) * inv_l);
                            v.y = pack_bf16x2(__uint_as_float(r[q * 8 + 2]) * inv_l, __uint_as_float(r[q * 8 + 3]) * inv_l);
                            v.z = pack_bf16x2(__uint_as_float(r[q * 8 + 4]) * inv_l, __uint_as_float(r[q * 8 + 5]) * inv_l);
                            v.w = pack_bf16x2(__uint_as_float(r[q * 8 + 6]) * inv_l, __uint_as_float(r[q * 8 + 7]) * inv_l);
                            *reinterpret_cast<uint4*>(orow + c * 32 + q * 8) = v;
                        }
                    }
                }
                if (row_ok) p.LSE[(size_t)it.head * p.N + row] = lse;
            } else {
                float* orow = p.ws_O + ((size_t)(it.ws_slot + x) * kTQ + tw) * D;
#pragma unroll
                for (int c = 0; c < D / 32; ++c) {
                    uint32_t r[32];
                    tmem_ld32(t_o + c * 32, r);
                    tc_wait_ld();
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        float4 v = make_float4(__uint_as_float(r[q * 4 + 0]) * inv_l, __uint_as_float(r[q * 4 + 1]) * inv_l,
                                               __uint_as_float(r[q * 4 + 2]) * inv_l, __uint_as_float(r[q * 4 + 3]) * inv_l);
                        *reinterpret_cast<float4*>(orow + c * 32 + q * 4) = v;
                    }
                }
                p.ws_LSE[(size_t)(it.ws_slot + x) * kTQ + tw] = lse;
            }
            tc_fence_before();
            mbar_arrive(smem_u32(&bars.o_free[x]));
        }
    }

    tc_fence_before();
    __syncthreads();
    if (tid == 0 && abort_flag) atomicExch(&p.counters->status, (int)BSA_ERR_DEVICE_TIMEOUT);
    if (warp == 9) tmem_dealloc(tmem, kTmemCols);
}

// ==========================================================================================
// Column-split kernel: same work decomposition as bsa_attention_kernel (one 128-row Q tile per
// CTA, S double-buffered), but TWO threads per query row: softmax warps 0-3 take the left half of
// the score tile's columns, warps 4-7 the right half (both may read the same TMEM lanes).  The two
// threads of a row exchange their half-row maxima through shared memory so they take identical
// reference-maximum decisions; each keeps a partial sum, added up once in the epilogue.  P goes to
// its own TMEM columns (the halves of S being read by the partner must not be overwritten).
//   warps 0-7 : softmax / correction / epilogue    warp 8 : TMA producer
//   warp 9 : Q K^T issuer    warp 10 : P V issuer (separate threads, ordered through mbarriers only)
// ==========================================================================================
constexpr int kCsThreads = 352;

struct __align__(8) CsBarriers {
    uint64_t q_full, q_empty, o_free, xchg;
    uint64_t k_full[kMaxStages], k_empty[kMaxStages], v_full[kMaxStages], v_empty[kMaxStages];
    uint64_t s_full[2], p_ready[2], pv_done[2];
};

template <int D, int TK>
__global__ void __launch_bounds__(kCsThreads, 1)
bsa_attention_cs_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                        const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
    constexpr int NSUB = D / 64;
    constexpr int Q_SUB = kTQ * 128;
    constexpr int KV_SUB = TK * 128;
    constexpr int KV_TILE = NSUB * KV_SUB;
    constexpr int NC = TK / 2;  // score columns per softmax thread
    constexpr int DC = D / 2;   // output columns per softmax thread
    // dynamic shared memory starts on a 1024-byte boundary (the swizzled tiles need it); checked below
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t* sQ = smem;
    uint8_t* sK = sQ + NSUB * Q_SUB;
    uint8_t* sV = sK + p.stages * KV_TILE;
    __shared__ CsBarriers bars;
    __shared__ float xbuf[2][2][kTQ];  // [use parity][column half][row]: half-row maxima / partial sums
    __shared__ uint32_t tmem_base_s;
    __shared__ uint32_t abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (smem_u32(smem) & 1023u) {  // never expected; fail with a status instead of corrupting tiles
        if (tid == 0) atomicExch(&p.counters->status, (int)BSA_ERR_CUDA);
        return;
    }
    const int NS = p.stages;

    if (tid == 0) {
        abort_flag = 0;
        mbar_init(smem_u32(&bars.q_full), 1);
        mbar_init(smem_u32(&bars.q_empty), 1);
        mbar_init(smem_u32(&bars.o_free), 256);
        mbar_init(smem_u32(&bars.xchg), 256);
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(smem_u32(&bars.k_full[s]), 1);
            mbar_init(smem_u32(&bars.k_empty[s]), 1);
            mbar_init(smem_u32(&bars.v_full[s]), 1);
            mbar_init(smem_u32(&bars.v_empty[s]), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&bars.s_full[s]), 1);
            mbar_init(smem_u32(&bars.p_ready[s]), 256);
            mbar_init(smem_u32(&bars.pv_done[s]), 1);
        }
        fence_mbar_init();
    }
    if (warp == 9) {
        tmem_alloc(smem_u32(&tmem_base_s), kTmemCols);
        tmem_relinquish();
    }
    if (warp == 8 && lane == 0) {
        prefetch_tensormap(&tmQ);
        prefetch_tensormap(&tmK);
        prefetch_tensormap(&tmV);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    volatile uint32_t* abortp = &abort_flag;
    const int n_items = p.counters->nitems;

    if (warp == 8) {
        // =========================== TMA producer ===========================
        if (lane == 0) {
            uint32_t itq = 0, g = 0;
            bool ok = true;
            for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
                const WorkItem it = p.items[idx];
                if (it.ntiles == 0) continue;
                ok = mbar_wait(smem_u32(&bars.q_empty), (itq & 1) ^ 1, abortp);
                if (!ok) break;
                mbar_arrive_expect_tx(smem_u32(&bars.q_full), NSUB * Q_SUB);
                for (int s = 0; s < NSUB; ++s)
                    tma_load_3d(smem_u32(sQ + s * Q_SUB), &tmQ, smem_u32(&bars.q_full), s * 64, it.q_tile * kTQ, it.head);
                int col_next = p.tile_col[it.tile_begin];  // tile metadata is fetched one tile ahead of its use
                for (int j = it.tile_begin; j < it.tile_end; ++j, ++g) {
                    const int col_cur = col_next;
                    if (j + 1 < it.tile_end) col_next = p.tile_col[j + 1];
                    const int stage = g % NS;
                    const uint32_t ph = (g / NS) & 1;
                    const int kv0 = col_cur * TK;
                    ok = mbar_wait(smem_u32(&bars.k_empty[stage]), ph ^ 1, abortp);
                    if (!ok) break;
                    mbar_arrive_expect_tx(smem_u32(&bars.k_full[stage]), KV_TILE);
                    for (int s = 0; s < NSUB; ++s)
                        tma_load_3d(smem_u32(sK + stage * KV_TILE + s * KV_SUB), &tmK, smem_u32(&bars.k_full[stage]),
                                    s * 64, kv0, it.head);
                    ok = mbar_wait(smem_u32(&bars.v_empty[stage]), ph ^ 1, abortp);
                    if (!ok) break;
                    mbar_arrive_expect_tx(smem_u32(&bars.v_full[stage]), KV_TILE);
                    for (int s = 0; s < NSUB; ++s)
                        tma_load_3d(smem_u32(sV + stage * KV_TILE + s * KV_SUB), &tmV, smem_u32(&bars.v_full[stage]),
                                    s * 64, kv0, it.head);
                }
                ++itq;
            }
            if (!ok) {
                const uint64_t t0 = globaltimer_ns();
                while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
            }
        }
    } else if (warp == 9) {
        // =========================== Q K^T issuer ===========================
        if (lane == 0) {
            constexpr uint32_t idesc_qk = make_idesc_bf16_f32(kTQ, TK, 0, 0);
            const uint64_t descQ = make_smem_desc_sw128(smem_u32(sQ), 16, 1024);
            const uint64_t descK = make_smem_desc_sw128(smem_u32(sK), 16, 1024);
            uint32_t itq = 0, g = 0;
            bool ok = true;
            for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
                const int n = p.items[idx].ntiles;
                if (n == 0) continue;
                ok = mbar_wait(smem_u32(&bars.q_full), itq & 1, abortp);
                if (!ok) break;
                for (int j = 0; j < n; ++j) {
                    const uint32_t gs = g + j;
                    const int stage = gs % NS;
                    const uint32_t ph = (gs / NS) & 1, sb = gs & 1;
                    ok = mbar_wait(smem_u32(&bars.k_full[stage]), ph, abortp);
                    if (!ok) break;
                    // S[sb] was last read by the softmax of tile gs-2.  P lives in its own columns, so Q K^T could
                    // start as soon as that softmax has arrived on p_ready, but issuing it ahead of the P V of
                    // tile gs-2 delays the P V the softmax chain waits for (measured slower): keep the order
                    // P V (gs-2) -> Q K^T (gs)
                    if (gs >= 2) {
                        ok = mbar_wait(smem_u32(&bars.pv_done[sb]), ((gs >> 1) - 1) & 1, abortp);
                        if (!ok) break;
                    }
                    tc_fence_after();
                    const uint32_t d_s = tmem + (sb ? kColS1 : kColS0);
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint64_t a = descQ + (uint64_t)(((k / 4) * Q_SUB + (k % 4) * 32) >> 4);
                        const uint64_t b = descK + (uint64_t)((stage * KV_TILE + (k / 4) * KV_SUB + (k % 4) * 32) >> 4);
                        mma_ss(d_s, a, b, idesc_qk, k > 0);
                    }
                    mma_commit(smem_u32(&bars.k_empty[stage]));
                    mma_commit(smem_u32(&bars.s_full[sb]));
                    if (j == n - 1) mma_commit(smem_u32(&bars.q_empty));
                }
                g += n;
                ++itq;
            }
        }
    } else if (warp == 10) {
        // =========================== P V issuer ===========================
        if (lane == 0) {
            constexpr uint32_t idesc_pv = make_idesc_bf16_f32(kTQ, D, 0, 1);
            const uint64_t descV = make_smem_desc_sw128(smem_u32(sV), KV_SUB, 1024);
            uint32_t itq = 0, g = 0;
            bool ok = true;
            for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
                const int n = p.items[idx].ntiles;
                if (n == 0) continue;
                for (int j = 0; j < n; ++j) {
                    const uint32_t gp = g + j;
                    const int stage = gp % NS;
                    const uint32_t ph = (gp / NS) & 1, sb = gp & 1;
                    ok = mbar_wait(smem_u32(&bars.p_ready[sb]), (gp >> 1) & 1, abortp);
                    if (!ok) break;
                    ok = mbar_wait(smem_u32(&bars.v_full[stage]), ph, abortp);
                    if (!ok) break;
                    if (j == 0) {
                        ok = mbar_wait(smem_u32(&bars.o_free), (itq & 1) ^ 1, abortp);
                        if (!ok) break;
                    }
                    tc_fence_after();
                    const uint32_t a_p = tmem + (sb ? kColP1 : kColP0);
#pragma unroll
                    for (int k = 0; k < TK / 16; ++k) {
                        const uint64_t b = descV + (uint64_t)((stage * KV_TILE + k * 2048) >> 4);
                        mma_ts(tmem + kColO, a_p + k * 8, b, idesc_pv, (j > 0 || k > 0) ? 1u : 0u);
                    }
                    mma_commit(smem_u32(&bars.v_empty[stage]));
                    mma_commit(smem_u32(&bars.pv_done[sb]));
                }
                g += n;
                ++itq;
            }
        }
    } else {
        // =========================== softmax / correction / epilogue ===========================
        const int half = warp >> 2;   // which half of the columns this thread owns
        const int tw = tid & 127;     // query row inside the tile = TMEM lane
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        uint32_t itq = 0, g = 0, xuse = 0;
        bool ok = true;
        const float c2 = p.scale_log2;
        const unsigned long long sub_mask = (p.sK >= 64) ? ~0ull : ((1ull << p.sK) - 1ull);
        // exchange one float with the partner thread of this row (bounded wait, no hardware barrier)
        auto exchange = [&](float mine, float& other) -> bool {
            const uint32_t par = xuse & 1;
            xbuf[par][half][tw] = mine;
            mbar_arrive(smem_u32(&bars.xchg));
            const bool got = mbar_wait(smem_u32(&bars.xchg), par, abortp);
            other = xbuf[par][half ^ 1][tw];
            ++xuse;
            return got;
        };
        for (int idx = blockIdx.x; idx < n_items && ok; idx += gridDim.x) {
            const WorkItem it = p.items[idx];
            const int row = it.q_tile * kTQ + tw;
            const bool row_ok = row < p.N;
            if (it.ntiles == 0) {
                if (row_ok) {
                    uint4* o = reinterpret_cast<uint4*>(p.O + ((size_t)it.head * p.o_head + (size_t)row * p.o_row) + half * DC);
#pragma unroll
                    for (int c = 0; c < DC / 8; ++c) o[c] = make_uint4(0, 0, 0, 0);
                    if (half == 0) p.LSE[(size_t)it.head * p.N + row] = -INFINITY;
                }
                continue;
            }
            float m_ref = -INFINITY, l = 0.f;
            int col_next = p.tile_col[it.tile_begin];  // tile metadata is fetched one tile ahead of its use
            unsigned long long member_next = p.tile_member[it.tile_begin];
            for (int j = 0; j < it.ntiles; ++j) {
                const uint32_t gs = g + j, sb = gs & 1;
                const int kv0 = col_next * TK;
                const unsigned long long member = member_next;
                if (j + 1 < it.ntiles) {
                    col_next = p.tile_col[it.tile_begin + j + 1];
                    member_next = p.tile_member[it.tile_begin + j + 1];
                }
                const bool need_mask = (member != p.full_member) || (kv0 + TK > p.Nkv);
                const uint32_t row_bits = (uint32_t)((member >> ((tw >> p.lgBQ) * p.sK)) & sub_mask);
                const int n_valid = p.Nkv - kv0;
                ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.s_full[sb]), (gs >> 1) & 1, abortp));
                if (!ok) break;
                tc_fence_after();
                const uint32_t t_s = tmem + lane_base + (sb ? kColS1 : kColS0) + half * NC;
                const uint32_t t_p = tmem + lane_base + (sb ? kColP1 : kColP0) + half * (NC / 2);
                uint32_t r[NC];
#pragma unroll
                for (int c = 0; c < NC / 32; ++c) tmem_ld32(t_s + c * 32, &r[c * 32]);
                tc_wait_ld();
                if (need_mask) {
#pragma unroll
                    for (int i = 0; i < NC; ++i) {
                        const int col = half * NC + i;
                        const bool act = ((row_bits >> (col >> p.lgBKV)) & 1u) && (col < n_valid);
                        r[i] = act ? r[i] : 0xff800000u;
                    }
                }
                float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
                for (int i = 0; i < NC; i += 4) {
                    m0 = fmaxf(m0, __uint_as_float(r[i]));
                    m1 = fmaxf(m1, __uint_as_float(r[i + 1]));
                    m2 = fmaxf(m2, __uint_as_float(r[i + 2]));
                    m3 = fmaxf(m3, __uint_as_float(r[i + 3]));
                }
                float mx = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3)), mx_other;
                ok = __all_sync(0xffffffffu, exchange(mx, mx_other));
                if (!ok) break;
                const float mx2 = fmaxf(mx, mx_other) * c2;
                float alpha = 1.f;
                bool rescale = false;
                if (mx2 > m_ref + kRescaleThreshold) {
                    alpha = ex2_approx(m_ref - mx2);
                    rescale = (j > 0) && (m_ref != -INFINITY);
                    m_ref = mx2;
                }
                const float neg_m = (m_ref == -INFINITY) ? 0.f : -m_ref;
                float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
                for (int i = 0; i < NC; i += 8) {
                    float t[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) t[k] = fmaf(__uint_as_float(r[i + k]), c2, neg_m);
#pragma unroll
                    for (int k = 0; k < 8; ++k) t[k] = ex2_approx(t[k]);
                    s0 += t[0] + t[4];
                    s1 += t[1] + t[5];
                    s2 += t[2] + t[6];
                    s3 += t[3] + t[7];
#pragma unroll
                    for (int k = 0; k < 4; ++k) r[i / 2 + k] = pack_bf16x2(t[2 * k], t[2 * k + 1]);
                }
                // P[sb] was last read by the P V of tile gs-2, issued by another thread than Q K^T: make sure it is done
                if (gs >= 2) {
                    ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.pv_done[sb]), ((gs >> 1) - 1) & 1, abortp));
                    if (!ok) break;
                }
#pragma unroll
                for (int c = 0; c < NC / 32; ++c) tmem_st16(t_p + c * 16, &r[c * 16]);
                l = l * alpha + ((s0 + s1) + (s2 + s3));
                if (j > 0 && __any_sync(0xffffffffu, rescale)) {
                    const uint32_t gp = gs - 1;
                    ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.pv_done[gp & 1]), (gp >> 1) & 1, abortp));
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t t_o = tmem + lane_base + kColO + half * DC;
#pragma unroll
                    for (int c = 0; c < DC / 32; ++c) {
                        uint32_t o[32];
                        tmem_ld32(t_o + c * 32, o);
                        tc_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                        tmem_st32(t_o + c * 32, o);
                    }
                }
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(smem_u32(&bars.p_ready[sb]));
            }
            if (!ok) break;
            // ---- epilogue: add the two partial sums, normalise, store this thread's half of the row ----
            {
                float l_other;
                ok = __all_sync(0xffffffffu, exchange(l, l_other));
                if (!ok) break;
                const float l_tot = (half == 0) ? (l + l_other) : (l_other + l);
                const uint32_t gl = g + it.ntiles - 1;
                ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.pv_done[gl & 1]), (gl >> 1) & 1, abortp));
                if (!ok) break;
                tc_fence_after();
                const float inv_l = (l_tot > 0.f) ? 1.f / l_tot : 0.f;
                const float lse = (l_tot > 0.f) ? fmaf(m_ref, 0.6931471805599453f, logf(l_tot)) : -INFINITY;
                const uint32_t t_o = tmem + lane_base + kColO + half * DC;
                if (it.nparts == 1) {
                    __nv_bfloat16* orow = p.O + ((size_t)it.head * p.o_head + (size_t)row * p.o_row) + half * DC;
#pragma unroll
                    for (int c = 0; c < DC / 32; ++c) {
                        uint32_t o[32];
                        tmem_ld32(t_o + c * 32, o);
                        tc_wait_ld();
                        if (row_ok) {
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                uint4 v;
                                v.x = pack_bf16x2(__uint_as_float(o[q * 8 + 0]) * inv_l, __uint_as_float(o[q * 8 + 1]) * inv_l);
                                v.y = pack_bf16x2(__uint_as_float(o[q * 8 + 2]) * inv_l, __uint_as_float(o[q * 8 + 3]) * inv_l);
                                v.z = pack_bf16x2(__uint_as_float(o[q * 8 + 4]) * inv_l, __uint_as_float(o[q * 8 + 5]) * inv_l);
                                v.w = pack_bf16x2(__uint_as_float(o[q * 8 + 6]) * inv_l, __uint_as_float(o[q * 8 + 7]) * inv_l);
                                *reinterpret_cast<uint4*>(orow + c * 32 + q * 8) = v;
                            }
                        }
                    }
                    if (row_ok && half == 0) p.LSE[(size_t)it.head * p.N + row] = lse;
                } else {
                    float* orow = p.ws_O + ((size_t)it.ws_slot * kTQ + tw) * D + half * DC;
#pragma unroll
                    for (int c = 0; c < DC / 32; ++c) {
                        uint32_t o[32];
                        tmem_ld32(t_o + c * 32, o);
                        tc_wait_ld();
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            float4 v = make_float4(__uint_as_float(o[q * 4 + 0]) * inv_l, __uint_as_float(o[q * 4 + 1]) * inv_l,
                                                   __uint_as_float(o[q * 4 + 2]) * inv_l, __uint_as_float(o[q * 4 + 3]) * inv_l);
                            *reinterpret_cast<float4*>(orow + c * 32 + q * 4) = v;
                        }
                    }
                    if (half == 0) p.ws_LSE[(size_t)it.ws_slot * kTQ + tw] = lse;
                }
                tc_fence_before();
                mbar_arrive(smem_u32(&bars.o_free));
            }
            g += it.ntiles;
            ++itq;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (tid == 0 && abort_flag) atomicExch(&p.counters->status, (int)BSA_ERR_DEVICE_TIMEOUT);
    if (warp == 9) tmem_dealloc(tmem, kTmemCols);
}

// ==========================================================================================
// Ping-pong kernel: one 128-row Q tile per CTA, TWO softmax warpgroups that take alternate KV
// tiles (warpgroup x owns the tiles whose running index has parity x, and with them S buffer x
// and P buffer x).  While one warpgroup is in its exponential phase the other loads its scores,
// finds its row maxima and waits for nothing but the previous tile's reference maximum, so the
// XU pipe and the tensor pipe both stay fed.  One O accumulator is shared: both warpgroups
// follow the SAME reference maximum per row, handed from tile to tile through shared memory
// (`mref`, one float per row, published right after a tile's max phase).  Each warpgroup keeps a
// partial row sum, converted whenever the reference it last saw has moved.  P has its own TMEM
// columns, so S[x] is free again as soon as warpgroup x has read it into registers (`s_free`).
// A third warpgroup owns the epilogue: at the end of a work item the softmax warpgroups only hand
// over their row sums (expressed in the item's final reference) and move straight on to the next
// item's tiles; the epilogue warpgroup waits for the item's last P V, drains the accumulator,
// normalises and stores, and releases the accumulator for the next item's first P V, which cannot
// be issued before that item's first softmax tile is done anyway.
//   warps 0-3 / 4-7 : softmax warpgroups 0 / 1      warp 8 : K and Q TMA producer   warp 11 : V TMA producer
//   warp 9 : Q K^T issuer      warp 10 : P V issuer    warps 12-15 : epilogue warpgroup
// Registers (setmaxnreg): softmax 192, epilogue 80, producers and issuers 48 per thread; the sum over the CTA,
// 256*192 + 128*80 + 128*48 = 65536, is exactly the launch allocation of 512 threads x 128.
// TMEM columns: S0 0, S1 128, O 256, P0 384, P1 448.
// ==========================================================================================
constexpr int kPpThreads = 512;

// The k-th work item of CTA b out of G: rounds of G consecutive items, alternately dealt forwards and backwards.
// Items arrive longest first, so dealing every round in the same direction would hand CTA 0 the longest item of
// every round and the last CTA the shortest; reversing every other round evens the per-CTA sums out.
__device__ __forceinline__ int cta_item_index(int k, int b, int G) { return k * G + ((k & 1) ? (G - 1 - b) : b); }

// Work item `idx` through the read-only path (items are written by the planner before the launch); past the end
// of the list the item has ntiles = -1 (an item with ntiles = 0 is a real row without active columns).
__device__ __forceinline__ WorkItem load_item(const WorkItem* items, int idx, int n_items) {
    WorkItem it;
    if (idx < n_items) {
        const int4* src = reinterpret_cast<const int4*>(items + idx);
        const int4 a = __ldg(src), b = __ldg(src + 1);
        it.head = a.x; it.q_tile = a.y; it.tile_begin = a.z; it.tile_end = a.w;
        it.part = b.x; it.nparts = b.y; it.ws_slot = b.z; it.ntiles = b.w;
    } else {
        it.head = it.q_tile = it.tile_begin = it.tile_end = it.part = it.ws_slot = 0;
        it.nparts = 1;
        it.ntiles = -1;
    }
    return it;
}

// The two fields of a work item the softmax warpgroups need, prefetched into registers with loads that stay put.
struct ItemSpan {
    int tile_begin, ntiles;  // ntiles = -1 past the end of the list
};
__device__ __forceinline__ ItemSpan load_item_span(const WorkItem* items, int idx, int n_items) {
    ItemSpan r;
    r.tile_begin = 0;
    r.ntiles = -1;
    if (idx < n_items) {
        const int* w = reinterpret_cast<const int*>(items + idx);
        r.tile_begin = ldg_pinned_s32(w + 2);
        r.ntiles = ldg_pinned_s32(w + 7);
    }
    return r;
}

// Slot and phase of a shared-memory ring, advanced once per tile (the single-thread roles sit on the path of every
// tile: no division by the ring depth there).
struct RingPos {
    int stage = 0;
    uint32_t phase = 0;
    __device__ __forceinline__ void advance(int depth) {
        if (++stage == depth) {
            stage = 0;
            phase ^= 1u;
        }
    }
};

struct __align__(8) PpBarriers {
    uint64_t q_full[2], q_empty[2], o_free, o_full, e_ready, e_taken;
    uint64_t k_full[kMaxStages], k_empty[kMaxStages], v_full[kMaxStages], v_empty[kMaxStages];
    uint64_t s_full[2], s_free[2], p_ready[2], pv_done[2];
};

template <int D, int TK, bool F16>
__global__ void __launch_bounds__(kPpThreads, 1)
bsa_attention_pp_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                        const __grid_constant__ CUtensorMap tmV, const AttnParams p) {
    constexpr int NSUB = D / 64;
    constexpr int Q_SUB = kTQ * 128;
    constexpr int KV_SUB = TK * 128;
    constexpr int KV_TILE = NSUB * KV_SUB;
    // dynamic shared memory starts on a 1024-byte boundary (the swizzled tiles need it); checked below
    extern __shared__ __align__(1024) uint8_t smem[];
    uint8_t* sQ = smem;                      // two Q tiles: the next item's is loaded while this one's is in use
    uint8_t* sK = sQ + 2 * NSUB * Q_SUB;     // NSK K tiles (a K tile lives from its load to the end of its Q K^T)
    uint8_t* sV = sK + p.stages * KV_TILE;   // NSV V tiles (a V tile lives about two tiles longer, until its P V)
    __shared__ PpBarriers bars;
    // [publishing warpgroup][row]: the reference maximum after that warpgroup's latest tile.  One 32-bit word per
    // row carries value and sequence together: reference values keep their two lowest mantissa bits clear, and
    // the word's two low bits hold (publish index + 1) mod 4, so the reader of the next tile (always the same
    // row's thread of the other warpgroup, which consumes every publish in order) needs one shared-memory
    // read, with no barrier in front of it, to know whether the value it got is the one it waits for.
    __shared__ uint32_t mref[2][kTQ];
    __shared__ float lfin[2][kTQ];   // [warpgroup][row]: an item's partial row sums in its final reference
    __shared__ float mfin[kTQ];      // the item's final reference maximum (log2 domain) per row
    __shared__ uint32_t tmem_base_s;
    __shared__ uint32_t abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
#ifdef BSA_TRACE
    if (tid == 0 && blockIdx.x < 4096) g_cta_times[0][blockIdx.x] = (long long)globaltimer_ns();
#endif
    if (smem_u32(smem) & 1023u) {  // never expected; fail with a status instead of corrupting tiles
        if (tid == 0) atomicExch(&p.counters->status, (int)BSA_ERR_CUDA);
        return;
    }
    const int NSK = p.stages, NSV = p.stages_v;

    if (tid == 0) {
        abort_flag = 0;
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bars.q_full[b]), 1);
            mbar_init(smem_u32(&bars.q_empty[b]), 1);
        }
        mbar_init(smem_u32(&bars.o_free), 128);   // epilogue threads: accumulator drained
        mbar_init(smem_u32(&bars.o_full), 1);     // P V issuer: the item's last P V has completed
        mbar_init(smem_u32(&bars.e_ready), 256);  // softmax threads: row sums of the item are in shared memory
        mbar_init(smem_u32(&bars.e_taken), 128);  // epilogue threads: row sums read
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(smem_u32(&bars.k_full[s]), 1);
            mbar_init(smem_u32(&bars.k_empty[s]), 1);
            mbar_init(smem_u32(&bars.v_full[s]), 1);
            mbar_init(smem_u32(&bars.v_empty[s]), 1);
        }
        for (int s = 0; s < 2; ++s) {
            mbar_init(smem_u32(&bars.s_full[s]), 1);
            mbar_init(smem_u32(&bars.s_free[s]), 128);
            mbar_init(smem_u32(&bars.p_ready[s]), 128);
            mbar_init(smem_u32(&bars.pv_done[s]), 1);
        }
        fence_mbar_init();
    }
    if (tid < 2 * kTQ) (&mref[0][0])[tid] = 0u;  // tag 0: matches no first publish
    if (warp == 9) {
        tmem_alloc(smem_u32(&tmem_base_s), kTmemCols);
        tmem_relinquish();
    }
    if (warp == 8 && lane == 0) {
        prefetch_tensormap(&tmQ);
        prefetch_tensormap(&tmK);
        prefetch_tensormap(&tmV);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_s;
    volatile uint32_t* abortp = &abort_flag;
    // Launched with programmatic stream serialisation, this grid may start while the kernel in front of it (the task
    // organisation) is still running: everything above touches only this CTA's shared memory, TMEM and the kernel
    // parameters; nothing below runs before that kernel has completed and its writes are visible.
    grid_dependency_wait();
    const int n_items = p.counters->nitems;
    const int n_rounds = (n_items + (int)gridDim.x - 1) / (int)gridDim.x;

    if (warp >= 12) {
        // =========================== epilogue warpgroup ===========================
        reg_dec<80>();
        const int tw = tid & 127;
        const uint32_t t_o = tmem + ((uint32_t)((warp & 3) * 32) << 16) + kColO;
        uint32_t itn = 0;  // non-empty items seen
        bool ok = true;
        BSA_TRACE_DECL(tn);
        WorkItem it_next = load_item(p.items, cta_item_index(0, blockIdx.x, gridDim.x), n_items);
        for (int kr = 0; kr < n_rounds && ok; ++kr) {
            const WorkItem it = it_next;
            it_next = load_item(p.items, cta_item_index(kr + 1, blockIdx.x, gridDim.x), n_items);
            const int row = it.q_tile * kTQ + tw;
            const bool row_ok = row < p.N;
            if (it.ntiles < 0) continue;  // past the end of the list
            if (it.ntiles == 0) {  // no active column: zero output, LSE = -inf
                if (row_ok) {
                    uint4* o = reinterpret_cast<uint4*>(p.O + ((size_t)it.head * p.o_head + (size_t)row * p.o_row));
#pragma unroll
                    for (int c = 0; c < D / 8; ++c) o[c] = make_uint4(0, 0, 0, 0);
                    p.LSE[(size_t)it.head * p.N + row] = -INFINITY;
                }
                continue;
            }
            ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.e_ready), itn & 1, abortp));
            if (!ok) break;
            const float l_tot = lfin[0][tw] + lfin[1][tw];
            const float m_final = mfin[tw];
            mbar_arrive(smem_u32(&bars.e_taken));
            const float inv_l = (l_tot > 0.f) ? 1.f / l_tot : 0.f;
            const float lse = (l_tot > 0.f) ? fmaf(m_final, 0.6931471805599453f, logf(l_tot)) : -INFINITY;
            if (lane == 0) BSA_TRACE_POINT(11, tn, 32);
            ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.o_full), itn & 1, abortp));
            if (!ok) break;
            tc_fence_after();
            if (lane == 0) BSA_TRACE_POINT(11, tn, 31);
            ++itn;
            __nv_bfloat16* orow = p.O + ((size_t)it.head * p.o_head + (size_t)row * p.o_row);
            float* wrow = p.ws_O + ((size_t)it.ws_slot * kTQ + tw) * D;
#pragma unroll 1  // once per item: a rolled loop keeps the kernel's code small
            for (int c = 0; c < D / 32; ++c) {
                uint32_t o[32];
                tmem_ld32(t_o + c * 32, o);
                tc_wait_ld();
                if (c == D / 32 - 1) {  // the accumulator is in registers: the next item's first P V may overwrite it
                    tc_fence_before();
                    mbar_arrive(smem_u32(&bars.o_free));
                    if (lane == 0) BSA_TRACE_POINT(11, tn, 33);
                }
                if (it.nparts == 1) {
                    if (row_ok) {  // 32-byte stores: every thread fills whole 32-byte sectors of its own row
#pragma unroll
                        for (int q = 0; q < 2; ++q) {
                            uint32_t v[8];
#pragma unroll
                            for (int e = 0; e < 8; ++e)
                                v[e] = pack_16x2<F16>(__uint_as_float(o[q * 16 + 2 * e]) * inv_l,
                                                   __uint_as_float(o[q * 16 + 2 * e + 1]) * inv_l);
                            st_global_v8(orow + c * 32 + q * 16, v);
                        }
                    }
                } else {  // Split-K partial: normalised fp32 rows in the workspace
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        uint32_t v[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e) v[e] = __float_as_uint(__uint_as_float(o[q * 8 + e]) * inv_l);
                        st_global_v8(wrow + c * 32 + q * 8, v);
                    }
                }
            }
            if (it.nparts == 1) {
                if (row_ok) p.LSE[(size_t)it.head * p.N + row] = lse;
            } else {
                p.ws_LSE[(size_t)it.ws_slot * kTQ + tw] = lse;
            }
            if (lane == 0) BSA_TRACE_POINT(11, tn, 34);
        }
    } else if (warp >= 8) {
        reg_dec<48>();
        if (warp == 8 && lane == 0) {
            // =========================== K and Q producer ===========================
            // K tiles run up to NSK tiles ahead of the Q K^T issuer and never wait for V slots (the V tiles have a
            // thread of their own in warp 11).  Q tiles alternate between two buffers: an item's Q tile may be
            // loaded once the last Q K^T of the item two before it has completed, so it is queued when this thread
            // enters the item BEFORE it and issued as soon as that condition is implied by a K slot this thread has
            // already waited for (Q K^T of tile g-NSK done) or is found true: this thread never blocks on a Q buffer
            // while K slots are free, and a new item's first Q K^T does not wait for its Q tile.
            uint32_t g = 0, itq = 0;  // itq: Q tiles issued (buffer itq & 1)
            uint32_t seq = 0;          // non-empty items entered
            RingPos ring;              // K ring position of tile g
            bool ok = true;
            BSA_TRACE_DECL(tn);
            int pq_row0 = 0, pq_row1 = 0, pq_row2 = 0, pq_head0 = 0, pq_head1 = 0, pq_head2 = 0;
            int pq_need0 = 0, pq_need1 = 0, pq_need2 = 0, npend = 0;
            uint32_t queued = 0;             // Q tiles queued so far (= sequence number of the next item to queue)
            int buf_last0 = -1000000, buf_last1 = -1000000;  // last global tile of the item that last used each buffer
            auto issue_q = [&]() -> bool {  // loads the oldest pending Q tile
                const uint32_t b = itq & 1;
                if (!mbar_wait(smem_u32(&bars.q_empty[b]), ((itq >> 1) & 1) ^ 1, abortp)) return false;
                mbar_arrive_expect_tx(smem_u32(&bars.q_full[b]), NSUB * Q_SUB);
                tma_load_4d(smem_u32(sQ + b * NSUB * Q_SUB), &tmQ, smem_u32(&bars.q_full[b]), 0, pq_row0, 0, pq_head0);
                ++itq;
                pq_row0 = pq_row1; pq_head0 = pq_head1; pq_need0 = pq_need1;
                pq_row1 = pq_row2; pq_head1 = pq_head2; pq_need1 = pq_need2;
                --npend;
                return true;
            };
            // queue the Q tile of an item whose tiles are [first, first + n): it needs its buffer's previous user done
            auto queue_q = [&](const WorkItem& w, int first, int n) -> bool {
                while (npend >= 3)  // queue full (many short items ahead of the Q K^T issuer): wait for a buffer
                    if (!issue_q()) return false;
                const uint32_t b = queued & 1;
                const int qrow = w.q_tile * kTQ, need = b ? buf_last1 : buf_last0;
                if (npend == 0) { pq_row0 = qrow; pq_head0 = w.head; pq_need0 = need; }
                else if (npend == 1) { pq_row1 = qrow; pq_head1 = w.head; pq_need1 = need; }
                else { pq_row2 = qrow; pq_head2 = w.head; pq_need2 = need; }
                ++npend;
                if (b) buf_last1 = first + n - 1; else buf_last0 = first + n - 1;
                ++queued;
                return true;
            };
            WorkItem it_next = load_item(p.items, cta_item_index(0, blockIdx.x, gridDim.x), n_items);
            for (int kr = 0; kr < n_rounds && ok; ++kr) {
                const WorkItem it = it_next;
                it_next = load_item(p.items, cta_item_index(kr + 1, blockIdx.x, gridDim.x), n_items);
                if (it.ntiles <= 0) continue;
                if (queued == seq) ok = queue_q(it, (int)g, it.ntiles);  // not queued ahead (first item, or after an empty one)
                if (ok && it_next.ntiles > 0 && queued == seq + 1) ok = queue_q(it_next, (int)g + it.ntiles, it_next.ntiles);
                if (!ok) break;
                ++seq;
                int col_next = p.tile_col[it.tile_begin];
                for (int j = it.tile_begin; j < it.tile_end && ok; ++j, ++g, ring.advance(NSK)) {
                    const int col_cur = col_next;
                    if (j + 1 < it.tile_end) col_next = p.tile_col[j + 1];
                    const int stage = ring.stage;
                    const uint32_t ph = ring.phase;
                    while (ok && npend > 0 &&
                           (pq_need0 <= (int)g - NSK ||
                            mbar_test_wait(smem_u32(&bars.q_empty[itq & 1]), ((itq >> 1) & 1) ^ 1)))
                        ok = issue_q();
                    if (!ok) break;
                    BSA_TRACE_POINT(0, tn, 19);
                    ok = mbar_wait(smem_u32(&bars.k_empty[stage]), ph ^ 1, abortp);
                    if (!ok) break;
                    BSA_TRACE_POINT(0, tn, 20);
                    mbar_arrive_expect_tx(smem_u32(&bars.k_full[stage]), KV_TILE);
                    tma_load_4d(smem_u32(sK + stage * KV_TILE), &tmK, smem_u32(&bars.k_full[stage]), 0, col_cur * TK, 0, it.head);
                    BSA_TRACE_POINT(0, tn, 21);
                }
            }
            while (ok && npend > 0) ok = issue_q();
            if (!ok) {
                const uint64_t t0 = globaltimer_ns();
                while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
            }
        } else if (warp == 11 && lane == 0) {
            // =========================== V producer ===========================
            uint32_t g = 0;
            RingPos ring;  // V ring position of tile g
            bool ok = true;
            const bool withhold = *reinterpret_cast<volatile int*>(&g_withhold_arrival) != 0;  // test hook, see above
            WorkItem it_next = load_item(p.items, cta_item_index(0, blockIdx.x, gridDim.x), n_items);
            for (int kr = 0; kr < n_rounds && ok; ++kr) {
                const WorkItem it = it_next;
                it_next = load_item(p.items, cta_item_index(kr + 1, blockIdx.x, gridDim.x), n_items);
                if (it.ntiles <= 0) continue;
                int col_next = p.tile_col[it.tile_begin];
                for (int j = it.tile_begin; j < it.tile_end; ++j, ++g, ring.advance(NSV)) {
                    const int col_cur = col_next;
                    if (j + 1 < it.tile_end) col_next = p.tile_col[j + 1];
                    const int stage = ring.stage;
                    const uint32_t ph = ring.phase;
                    if (withhold && g == 0) continue;  // this tile never arrives
                    ok = mbar_wait(smem_u32(&bars.v_empty[stage]), ph ^ 1, abortp);
                    if (!ok) break;
                    mbar_arrive_expect_tx(smem_u32(&bars.v_full[stage]), KV_TILE);
                    tma_load_4d(smem_u32(sV + stage * KV_TILE), &tmV, smem_u32(&bars.v_full[stage]), 0, col_cur * TK, 0, it.head);
                }
            }
            if (!ok) {
                const uint64_t t0 = globaltimer_ns();
                while (globaltimer_ns() - t0 < 200000ull) __nanosleep(1000);
            }
        } else if (warp == 9 && lane == 0) {
            // =========================== Q K^T issuer ===========================
            constexpr uint32_t idesc_qk = make_idesc_f32(kTQ, TK, 0, 0, F16);
            const uint64_t descQ0 = make_smem_desc_sw128(smem_u32(sQ), 16, 1024);
            const uint64_t descK = make_smem_desc_sw128(smem_u32(sK), 16, 1024);
            RingPos ring;  // K ring position of the tile being issued
            uint32_t itq = 0, g = 0;
            bool ok = true;
            BSA_TRACE_DECL(tn);
            BSA_PH_DECL;
            int n_next = load_item(p.items, cta_item_index(0, blockIdx.x, gridDim.x), n_items).ntiles;
            for (int kr = 0; kr < n_rounds && ok; ++kr) {
                const int n = n_next;
                n_next = load_item(p.items, cta_item_index(kr + 1, blockIdx.x, gridDim.x), n_items).ntiles;
                if (n <= 0) continue;
                const uint32_t qb = itq & 1;  // this item's Q buffer
                ok = mbar_wait(smem_u32(&bars.q_full[qb]), (itq >> 1) & 1, abortp);
                if (!ok) break;
                const uint64_t descQ = descQ0 + (uint64_t)((qb * NSUB * Q_SUB) >> 4);
                for (int j = 0; j < n; ++j, ring.advance(NSK)) {
                    const uint32_t gs = g + j;
                    const int stage = ring.stage;
                    const uint32_t ph = ring.phase, sb = gs & 1;
                    // K tile present, and S[sb] read into registers by the softmax of tile gs-2
                    if (gs >= 2)
                        ok = mbar_wait2(smem_u32(&bars.s_free[sb]), ((gs >> 1) - 1) & 1, smem_u32(&bars.k_full[stage]), ph, abortp);
                    else
                        ok = mbar_wait(smem_u32(&bars.k_full[stage]), ph, abortp);
                    if (!ok) break;
                    BSA_PH(0);
                    BSA_STAMP(0, gs, 0);
                    BSA_TRACE_POINT(1, tn, 6);
                    tc_fence_after();
                    const uint32_t d_s = tmem + (sb ? kColS1 : kColS0);
#pragma unroll
                    for (int k = 0; k < D / 16; ++k) {
                        const uint64_t a = descQ + (uint64_t)(((k / 4) * Q_SUB + (k % 4) * 32) >> 4);
                        const uint64_t b = descK + (uint64_t)((stage * KV_TILE + (k / 4) * KV_SUB + (k % 4) * 32) >> 4);
                        mma_ss(d_s, a, b, idesc_qk, k > 0);
                    }
                    mma_commit(smem_u32(&bars.k_empty[stage]));
                    mma_commit(smem_u32(&bars.s_full[sb]));
                    BSA_PH(1);
                    BSA_STAMP(0, gs, 1);
#ifdef BSA_PHASES
                    ++ph_n;
#endif
                    BSA_TRACE_POINT(1, tn, 2);
                    if (j == n - 1) mma_commit(smem_u32(&bars.q_empty[qb]));
                }
                g += n;
                ++itq;
            }
#ifdef BSA_PHASES
            if (blockIdx.x == 1) { g_trace[0][0] = ph_acc[0]; g_trace[0][1] = ph_acc[1]; g_trace[0][8] = ph_n; }
#endif
        } else if (warp == 10 && lane == 0) {
            // =========================== P V issuer ===========================
            constexpr uint32_t idesc_pv = make_idesc_f32(kTQ, D, 0, 1, F16);
            const uint64_t descV = make_smem_desc_sw128(smem_u32(sV), KV_SUB, 1024);
            RingPos ring;  // V ring position of the tile being issued
            uint32_t itq = 0, g = 0;
            bool ok = true;
            BSA_TRACE_DECL(tn);
            BSA_PH_DECL;
            int n_next = load_item(p.items, cta_item_index(0, blockIdx.x, gridDim.x), n_items).ntiles;
            for (int kr = 0; kr < n_rounds && ok; ++kr) {
                const int n = n_next;
                n_next = load_item(p.items, cta_item_index(kr + 1, blockIdx.x, gridDim.x), n_items).ntiles;
                if (n <= 0) continue;
                for (int j = 0; j < n; ++j, ring.advance(NSV)) {
                    const uint32_t gp = g + j;
                    const int stage = ring.stage;
                    const uint32_t ph = ring.phase, sb = gp & 1;
                    // V tile present (normally long before), accumulator drained by the epilogue (first tile of an
                    // item), and last the P tile, which is the one this thread normally waits for
                    if (j == 0) {
                        ok = mbar_wait(smem_u32(&bars.o_free), (itq & 1) ^ 1, abortp);
                        if (!ok) break;
                    }
                    ok = mbar_wait2(smem_u32(&bars.v_full[stage]), ph, smem_u32(&bars.p_ready[sb]), (gp >> 1) & 1, abortp);
                    if (!ok) break;
                    BSA_PH(0);
                    BSA_STAMP(1, gp, 0);
                    BSA_TRACE_POINT(10, tn, 3);

                    tc_fence_after();
                    const uint32_t a_p = tmem + (sb ? kColP1 : kColP0);
#pragma unroll
                    for (int k = 0; k < TK / 16; ++k) {
                        const uint64_t b = descV + (uint64_t)((stage * KV_TILE + k * 2048) >> 4);
                        mma_ts(tmem + kColO, a_p + k * 8, b, idesc_pv, (j > 0 || k > 0) ? 1u : 0u);
                    }
                    mma_commit(smem_u32(&bars.v_empty[stage]));
                    mma_commit(smem_u32(&bars.pv_done[sb]));
                    if (j == n - 1) mma_commit(smem_u32(&bars.o_full));
                    BSA_PH(1);
                    BSA_STAMP(1, gp, 1);
#ifdef BSA_PHASES
                    ++ph_n;
#endif
                    BSA_TRACE_POINT(10, tn, 5);
                }
                g += n;
                ++itq;
            }
#ifdef BSA_PHASES
            if (blockIdx.x == 1) { g_trace[1][0] = ph_acc[0]; g_trace[1][1] = ph_acc[1]; g_trace[1][8] = ph_n; }
#endif
        }
    } else {
        // =========================== softmax warpgroup x ===========================
        reg_inc<192>();
        const int x = warp >> 2;
        const int tw = tid & 127;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t t_s = tmem + lane_base + (x ? kColS1 : kColS0);
        const uint32_t t_p = tmem + lane_base + (x ? kColP1 : kColP0);
        const uint32_t t_o = tmem + lane_base + kColO;
        uint32_t g = 0;          // running tile index at the start of the current item (all warpgroups agree)
        uint32_t itn = 0;        // non-empty items finished
        bool ok = true;
        BSA_TRACE_DECL(tn);
        const float c2 = p.scale_log2;
        const unsigned long long sub_mask = (p.sK >= 64) ? ~0ull : ((1ull << p.sK) - 1ull);
        BSA_PH_DECL;
        // The reference after global tile t (taken by the other warpgroup), given a word read earlier from its slot:
        // if that word already carries the publish's tag it is used, else the slot is polled (bounded).
        auto take_reference = [&](uint32_t t, uint32_t word, float& m_out) -> bool {
            const uint32_t tag = ((t >> 1) + 1) & 3u;
            if ((word & 3u) != tag) {
                volatile uint32_t* slot = &mref[x ^ 1][tw];
                long long t0 = 0;
                uint32_t spins = 0;
                while (true) {
                    word = *slot;
                    if ((word & 3u) == tag) break;
                    if ((++spins & 63u) == 0) {
                        if (*abortp) return false;
                        const long long now = clock64();
                        if (t0 == 0) t0 = now;
                        if (now - t0 > *reinterpret_cast<volatile long long*>(&g_wait_limit_cycles)) {
                            *abortp = 1;
                            return false;
                        }
                    }
                }
            }
            m_out = __uint_as_float(word & ~3u);
            return true;
        };
        // work items are fetched two items ahead and the first tile's metadata one item ahead, so that neither the
        // item nor the metadata that depends on it is waited for at an item boundary
        ItemSpan it_next = load_item_span(p.items, cta_item_index(0, blockIdx.x, gridDim.x), n_items);
        ItemSpan it_next2 = load_item_span(p.items, cta_item_index(1, blockIdx.x, gridDim.x), n_items);
        int first_col = 0;
        unsigned long long first_member = 0ull;
        {
            const int j0n = ((g & 1) == (uint32_t)x) ? 0 : 1;
            if (j0n < it_next.ntiles) {
                first_col = ldg_pinned_s32(p.tile_col + it_next.tile_begin + j0n);
                first_member = ldg_pinned_u64(p.tile_member + it_next.tile_begin + j0n);
            }
        }
        for (int kr = 0; kr < n_rounds && ok; ++kr) {
            const ItemSpan it = it_next;
            it_next = it_next2;
            it_next2 = load_item_span(p.items, cta_item_index(kr + 2, blockIdx.x, gridDim.x), n_items);
            const int n = it.ntiles;
            int col_next = first_col;
            unsigned long long member_next = first_member;
            {   // the next item's first tile of this warpgroup: its parity follows from g + n
                const int j0n = (((g + n) & 1) == (uint32_t)x) ? 0 : 1;
                if (j0n < it_next.ntiles) {
                    first_col = ldg_pinned_s32(p.tile_col + it_next.tile_begin + j0n);
                    first_member = ldg_pinned_u64(p.tile_member + it_next.tile_begin + j0n);
                }
            }
            if (n <= 0) continue;  // the epilogue warpgroup writes the empty rows
            float m_know = -INFINITY;  // reference maximum this thread's partial sum l is expressed in
            float l = 0.f;
            // first local tile index of this warpgroup inside the item
            const int j0 = ((g & 1) == (uint32_t)x) ? 0 : 1;
            for (int j = j0; j < n; j += 2) {
                const uint32_t gs = g + j;
                const int kv0 = col_next * TK;
                const unsigned long long member = member_next;
                if (j + 2 < n) {
                    col_next = ldg_pinned_s32(p.tile_col + it.tile_begin + j + 2);
                    member_next = ldg_pinned_u64(p.tile_member + it.tile_begin + j + 2);
                }
                const bool need_mask = (member != p.full_member) || (kv0 + TK > p.Nkv);
                const uint32_t row_bits = (uint32_t)((member >> ((tw >> p.lgBQ) * p.sK)) & sub_mask);
                const int n_valid = p.Nkv - kv0;
                if (lane == 0 && j == j0) BSA_TRACE_POINT(2 + warp, tn, 35);
                BSA_PH(7);
                ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.s_full[x]), (gs >> 1) & 1, abortp));
                if (!ok) break;
                BSA_PH(0);
                if (lane == 0) BSA_STAMP(2 + warp, gs, 0);
                if (lane == 0) BSA_TRACE_POINT(2 + warp, tn, 10);
                tc_fence_after();
                uint32_t r[TK];
#pragma unroll
                for (int c = 0; c < TK / 32; ++c) tmem_ld32(t_s + c * 32, &r[c * 32]);
                tc_wait_ld();
                BSA_PH(1);
                tc_fence_before();
                mbar_arrive(smem_u32(&bars.s_free[x]));  // S[x] is in registers: the next Q K^T into it may start
                if (lane == 0) BSA_TRACE_POINT(2 + warp, tn, 11);
                // The previous tile's reference has normally been published by now: its slot is read here and the
                // word checked after the max phase, so that the shared-memory round trip overlaps that phase.
                const uint32_t ref_word = *reinterpret_cast<volatile uint32_t*>(&mref[x ^ 1][tw]);
                if (need_mask) {
                    // B_KV >= 16, so a group of 16 key columns lies inside one logical block: one activity bit per
                    // group, two instructions per element.  (Skipping, per warp, the groups none of its 32 rows needs
                    // was tried and lost: a warpgroup still waits for its slowest warp, and the branches cost more
                    // than the exponentials they save.)
#pragma unroll
                    for (int gq = 0; gq < TK / 16; ++gq) {
                        const bool grp = (row_bits >> ((gq * 16) >> p.lgBKV)) & 1u;
#pragma unroll
                        for (int i = gq * 16; i < gq * 16 + 16; ++i) r[i] = (grp && i < n_valid) ? r[i] : 0xff800000u;
                    }
                }
                float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
                for (int i = 0; i < TK; i += 8) {
                    m0 = max3(m0, __uint_as_float(r[i]), __uint_as_float(r[i + 1]));
                    m1 = max3(m1, __uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
                    m2 = max3(m2, __uint_as_float(r[i + 4]), __uint_as_float(r[i + 5]));
                    m3 = max3(m3, __uint_as_float(r[i + 6]), __uint_as_float(r[i + 7]));
                }
                const float mx2 = fmaxf(fmaxf(m0, m1), fmaxf(m2, m3)) * c2;
#ifdef BSA_TRACE
                if (lane == 0 && mx2 != 12345.f) BSA_TRACE_POINT(2 + warp, tn, 17);
#endif
                // ---- reference maximum handed over from the previous tile (other warpgroup) ----
                float m_prev = -INFINITY;
                if (gs > 0) {  // every publish is consumed, in order, also across item boundaries (the tags rely on it)
                    float m_taken;
                    ok = __all_sync(0xffffffffu, take_reference(gs - 1, ref_word, m_taken));
                    if (!ok) break;
                    if (j > 0) m_prev = m_taken;  // the previous tile belongs to this item
                }
#ifdef BSA_PHASES
                {
                    float f0_ = mx2, f1_ = m_prev;  // real instructions that read the values: the clock is read after them
                    asm volatile("mov.b32 %0, %0;\n\tmov.b32 %1, %1;" : "+f"(f0_), "+f"(f1_));
                }
#endif
                BSA_PH(2);
#ifdef BSA_TRACE
                if (lane == 0 && m_prev != 12345.f) BSA_TRACE_POINT(2 + warp, tn, 18);
#endif
                if (lane == 0) BSA_TRACE_POINT(2 + warp, tn, 12);
                if (m_prev != m_know) {  // the other warpgroup moved the reference since this thread last looked
                    l *= ex2_approx(m_know - m_prev);  // m_know = -inf only while l = 0
                    m_know = m_prev;
                }
                float alpha = 1.f;
                bool rescale = false;
                if (mx2 > m_know + kRescaleThreshold) {
                    const float m_new = __uint_as_float(__float_as_uint(mx2) & ~3u);  // two low bits clear (see mref)
                    alpha = ex2_approx(m_know - m_new);
                    rescale = (j > 0) && (m_know != -INFINITY);
                    l *= alpha;
                    m_know = m_new;
                }
                // publish: the next tile's warpgroup may take its decision
                *reinterpret_cast<volatile uint32_t*>(&mref[x][tw]) = __float_as_uint(m_know) | (((gs >> 1) + 1) & 3u);
                BSA_PH(3);
                const float neg_m = (m_know == -INFINITY) ? 0.f : -m_know;
                const uint64_t c22 = pack_f32x2(c2, c2), nm2 = pack_f32x2(neg_m, neg_m);
                uint64_t sum01 = pack_f32x2(0.f, 0.f), sum23 = sum01;
                // P[x] was last read by the P V of tile gs-2 (normally long complete).  With d = 64 it is waited for
                // here and the P tile stored 32 columns at a time while the next columns are still being exponentiated
                // (+4 % on Stress-B); with d = 128 the stores follow the loop (the split loop was 1-2 % slower there).
                constexpr bool kStoreInLoop = (D == 64);
                if (kStoreInLoop && gs >= 2) {
                    ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.pv_done[x]), ((gs >> 1) - 1) & 1, abortp));
                    if (!ok) break;
                    tc_fence_after();
                }
#pragma unroll
                for (int i = 0; i < TK; i += 4) {
                    float x0, x1, x2, x3;
                    unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), c22, nm2), x0, x1);
                    unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(r[i + 2]), __uint_as_float(r[i + 3])), c22, nm2), x2, x3);
                    const float p0 = ex2_approx(x0), p1 = ex2_approx(x1), p2 = ex2_approx(x2), p3 = ex2_approx(x3);
                    sum01 = add_f32x2(sum01, pack_f32x2(p0, p1));
                    sum23 = add_f32x2(sum23, pack_f32x2(p2, p3));
                    r[i / 2] = pack_16x2<F16>(p0, p1);
                    r[i / 2 + 1] = pack_16x2<F16>(p2, p3);
                    if (kStoreInLoop && (i & 31) == 28) tmem_st16(t_p + (i >> 5) * 16, &r[(i >> 5) * 16]);
                }
                float s0, s1, s2, s3;
                unpack_f32x2(sum01, s0, s1);
                unpack_f32x2(sum23, s2, s3);
                l += (s0 + s1) + (s2 + s3);
#ifdef BSA_PHASES
                {
                    float f0_ = l;
                    uint32_t u0_ = r[TK / 2 - 1];
                    asm volatile("mov.b32 %0, %0;\n\tmov.b32 %1, %1;" : "+f"(f0_), "+r"(u0_));
                }
#endif
                BSA_PH(4);
                if (lane == 0) BSA_STAMP(2 + warp, gs, 1);
                if (lane == 0) BSA_TRACE_POINT(2 + warp, tn, 14);
                if (!kStoreInLoop) {
                    if (gs >= 2) {
                        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.pv_done[x]), ((gs >> 1) - 1) & 1, abortp));
                        if (!ok) break;
                    }
                    BSA_PH(5);
                    if (lane == 0) BSA_STAMP(2 + warp, gs, 2);
#pragma unroll
                    for (int c = 0; c < TK / 32; ++c) tmem_st16(t_p + c * 16, &r[c * 16]);
                }
                // ---- the reference moved at this tile: rescale the running output (after the P V of tile gs-1) ----
                if (j > 0 && __any_sync(0xffffffffu, rescale)) {
                    const uint32_t gp = gs - 1;
                    ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.pv_done[x ^ 1]), (gp >> 1) & 1, abortp));
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll 1  // rare path: kept small
                    for (int c = 0; c < D / 32; ++c) {
                        uint32_t o[32];
                        tmem_ld32(t_o + c * 32, o);
                        tc_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                        tmem_st32(t_o + c * 32, o);
                    }
                }
                tc_wait_st();
                tc_fence_before();
                mbar_arrive(smem_u32(&bars.p_ready[x]));
                BSA_PH(6);
                if (lane == 0) BSA_STAMP(2 + warp, gs, 3);
#ifdef BSA_PHASES
                ++ph_n;
#endif
                if (lane == 0) BSA_TRACE_POINT(2 + warp, tn, 16);
            }
            if (!ok) break;
            // ---- hand this warpgroup's row sums, expressed in the item's final reference, to the epilogue warpgroup ----
            {
                const uint32_t gl = g + n - 1;  // last tile of the item
                const bool owner = (gl & 1) == (uint32_t)x;
                float m_final = m_know;
                if (!owner) {  // the other warpgroup took the last tile: its publish holds the final reference
                    ok = __all_sync(0xffffffffu,
                                    take_reference(gl, *reinterpret_cast<volatile uint32_t*>(&mref[x ^ 1][tw]), m_final));
                    if (!ok) break;
                }
                if (m_final != m_know) l *= ex2_approx(m_know - m_final);  // l = 0 whenever m_know = -inf
                // the previous item's sums must have been read
                ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars.e_taken), (itn & 1) ^ 1, abortp));
                if (!ok) break;
                lfin[x][tw] = l;
                if (owner) mfin[tw] = m_final;
                mbar_arrive(smem_u32(&bars.e_ready));
                ++itn;
                if (lane == 0) BSA_TRACE_POINT(2 + warp, tn, 30);
            }
            g += n;
            BSA_PH(7);  // item boundary: sums handed over, next item's first tile not yet waited for
        }
#ifdef BSA_PHASES
        if (blockIdx.x == 1 && lane == 0) {
            for (int k = 0; k < 8; ++k) g_trace[2 + warp][k] = ph_acc[k];
            g_trace[2 + warp][8] = ph_n;
        }
#endif
    }

    tc_fence_before();
    __syncthreads();
    if (tid == 0 && abort_flag) atomicExch(&p.counters->status, (int)BSA_ERR_DEVICE_TIMEOUT);
    if (warp == 9) tmem_dealloc(tmem, kTmemCols);
#ifdef BSA_TRACE
    if (tid == 0 && blockIdx.x < 4096) g_cta_times[1][blockIdx.x] = (long long)globaltimer_ns();
#endif
}

// ------------------------------------------------------------------------------------------
// Split-K reduction (Section 4.3): partial states were stored as (normalised O_p, LSE_p), so
// rescaling to the common maximum, merging and normalising is
//     LSE = log sum_p exp(LSE_p),  O = sum_p exp(LSE_p - LSE) O_p,
// taken in fixed partition order (bitwise reproducible).  One CTA per split Q tile row.
// ------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(256) bsa_merge_kernel(const SplitRow* __restrict__ split_rows,
                                                         const PlanCountersDev* __restrict__ counters,
                                                         const float* __restrict__ ws_O, const float* __restrict__ ws_LSE,
                                                         __nv_bfloat16* __restrict__ O, float* __restrict__ LSE, int N,
                                                         int f16, long long o_head, long long o_row) {
    constexpr int GROUPS = D / 8;                   // 8 output columns (16 bytes of bf16 or fp16) per thread
    constexpr int CHUNKS = kTQ * GROUPS / 256;      // CTAs' worth of work per merged 128-row tile
    const int n_units = counters->nsplit_rows * CHUNKS;
    for (int cu = blockIdx.x; cu < n_units; cu += gridDim.x) {
        const SplitRow s = split_rows[cu / CHUNKS];
        const int nparts = s.nparts & 0xffff, stride = s.nparts >> 16;
        const int u = (cu % CHUNKS) * 256 + threadIdx.x;
        const int r = u / GROUPS, gcol = (u % GROUPS) * 8;
        const int row = s.q_tile * kTQ + r;
        if (row >= N) continue;
        // all partial LSEs of the row first (independent loads), then the weights, then the weighted sum
        float lse_p[32];
        float m = -INFINITY;
#pragma unroll 4
        for (int q = 0; q < nparts; ++q) {
            lse_p[q & 31] = ws_LSE[(size_t)(s.ws_slot + q * stride) * kTQ + r];
            m = fmaxf(m, lse_p[q & 31]);
        }
        const float m_use = (m == -INFINITY) ? 0.f : m;
        float tot = 0.f;
        float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        for (int q = 0; q < nparts; ++q) {
            const size_t slot = (size_t)(s.ws_slot + q * stride);
            const float w = __expf(lse_p[q & 31] - m_use);
            tot += w;
            const float4* src = reinterpret_cast<const float4*>(ws_O + (slot * kTQ + r) * D + gcol);
            const float4 a = src[0], b = src[1];
            acc[0] = fmaf(w, a.x, acc[0]); acc[1] = fmaf(w, a.y, acc[1]);
            acc[2] = fmaf(w, a.z, acc[2]); acc[3] = fmaf(w, a.w, acc[3]);
            acc[4] = fmaf(w, b.x, acc[4]); acc[5] = fmaf(w, b.y, acc[5]);
            acc[6] = fmaf(w, b.z, acc[6]); acc[7] = fmaf(w, b.w, acc[7]);
        }
        const float inv = (tot > 0.f) ? 1.f / tot : 0.f;
        uint4 v;
        if (f16) {
            v.x = pack_f16x2(acc[0] * inv, acc[1] * inv);
            v.y = pack_f16x2(acc[2] * inv, acc[3] * inv);
            v.z = pack_f16x2(acc[4] * inv, acc[5] * inv);
            v.w = pack_f16x2(acc[6] * inv, acc[7] * inv);
        } else {
            v.x = pack_bf16x2(acc[0] * inv, acc[1] * inv);
            v.y = pack_bf16x2(acc[2] * inv, acc[3] * inv);
            v.z = pack_bf16x2(acc[4] * inv, acc[5] * inv);
            v.w = pack_bf16x2(acc[6] * inv, acc[7] * inv);
        }
        *reinterpret_cast<uint4*>(O + ((size_t)s.head * o_head + (size_t)row * o_row) + gcol) = v;
        if (gcol == 0) LSE[(size_t)s.head * N + row] = (tot > 0.f) ? m_use + logf(tot) : -INFINITY;
    }
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// bf16 [heads][N][d] viewed as a 3-D tensor {d, N, heads}; box = {64, rows, 1}; rows beyond N read as zero.
// `nhd`: the tensor is stored [N][heads][d] instead (token-major); only the two byte strides change.
bool encode_map(CUtensorMap* m, const void* base, int64_t N, int heads, int d, int box_rows, bool f16, bool nhd) {
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return false;
    cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)N, (cuuint64_t)heads};
    cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)N * (cuuint64_t)d * 2};
    if (nhd) {
        strides[0] = (cuuint64_t)heads * (cuuint64_t)d * 2;
        strides[1] = (cuuint64_t)d * 2;
    }
    cuuint32_t box[3] = {64, (cuuint32_t)box_rows, 1};
    cuuint32_t es[3] = {1, 1, 1};
    return enc(m, f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims,
               strides, box, es,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same tensor as {64 columns, N rows, d/64 column groups, heads}; box = {64, rows, d/64, 1}: one copy lands all
// 64-column sub-tiles of a row block back to back (the [sub-tile][row][64] layout the MMA descriptors address).
bool encode_map4(CUtensorMap* m, const void* base, int64_t N, int heads, int d, int box_rows, bool f16, bool nhd) {
    EncodeTiledFn enc = get_encode_fn();
    if (!enc) return false;
    cuuint64_t dims[4] = {64, (cuuint64_t)N, (cuuint64_t)(d / 64), (cuuint64_t)heads};
    cuuint64_t strides[3] = {(cuuint64_t)d * 2, 128, (cuuint64_t)N * (cuuint64_t)d * 2};
    if (nhd) {
        strides[0] = (cuuint64_t)heads * (cuuint64_t)d * 2;
        strides[2] = (cuuint64_t)d * 2;
    }
    cuuint32_t box[4] = {64, (cuuint32_t)box_rows, (cuuint32_t)(d / 64), 1};
    cuuint32_t es[4] = {1, 1, 1, 1};
    return enc(m, f16 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT16 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims,
               strides, box, es,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D, int TK, int KERNEL>
cudaError_t launch_attn(const ForwardArgs& a, const AttnParams& p, cudaStream_t stream, const char** err) {
    CUtensorMap tq, tk, tv;
    const bool ok_maps = (KERNEL == 4)
                             ? (encode_map4(&tq, a.Q, a.g.N, a.g.H, D, kTQ, a.f16, a.nhd) &&
                                encode_map4(&tk, a.K, a.g.N_kv, a.g.H, D, TK, a.f16, a.nhd) &&
                                encode_map4(&tv, a.V, a.g.N_kv, a.g.H, D, TK, a.f16, a.nhd))
                             : (encode_map(&tq, a.Q, a.g.N, a.g.H, D, kTQ, a.f16, a.nhd) &&
                                encode_map(&tk, a.K, a.g.N_kv, a.g.H, D, TK, a.f16, a.nhd) &&
                                encode_map(&tv, a.V, a.g.N_kv, a.g.H, D, TK, a.f16, a.nhd));
    if (!ok_maps) {
        *err = "cuTensorMapEncodeTiled failed";
        return cudaErrorInvalidValue;
    }
    const int smem = attention_smem_bytes(D, TK, a.stages, KERNEL);
    if (a.f16 && (KERNEL == 1 || KERNEL == 2)) {  // not instantiated for half inputs (eligibility says so too)
        *err = "fp16 inputs need a single-tile, ping-pong or row-block plan";
        return cudaErrorInvalidValue;
    }
    // largest size already allowed, per instantiation and per device (the attribute belongs to the device's copy of
    // the kernel); concurrent first calls may both set it, which is harmless
    static std::atomic<int> attr_bytes_dev[kMaxDevices];
    const int dev = (a.device >= 0 && a.device < kMaxDevices) ? a.device : 0;
    if (smem > attr_bytes_dev[dev].load(std::memory_order_relaxed)) {
        cudaError_t e;
        if constexpr (KERNEL == 0 || KERNEL == 3) {
            e = cudaFuncSetAttribute(bsa_attention_kernel<D, TK, KERNEL == 3, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e == cudaSuccess)
                e = cudaFuncSetAttribute(bsa_attention_kernel<D, TK, KERNEL == 3, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        }
        else if constexpr (KERNEL == 1)
            e = cudaFuncSetAttribute(bsa_attention_pair_kernel<D, TK>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        else if constexpr (KERNEL == 2)
            e = cudaFuncSetAttribute(bsa_attention_cs_kernel<D, TK>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        else {
            e = cudaFuncSetAttribute(bsa_attention_pp_kernel<D, TK, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
            if (e == cudaSuccess)
                e = cudaFuncSetAttribute(bsa_attention_pp_kernel<D, TK, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        }
        if (e != cudaSuccess) {
            *err = "cudaFuncSetAttribute(max dynamic shared memory)";
            return e;
        }
        attr_bytes_dev[dev].store(smem, std::memory_order_relaxed);
    }
    int grid = a.num_sms < a.max_items ? a.num_sms : a.max_items;
    if (grid < 1) grid = 1;
    if constexpr (KERNEL == 0 || KERNEL == 3) {
        constexpr int threads = KERNEL == 3 ? kThreads + 32 : kThreads;
        if (a.f16)
            bsa_attention_kernel<D, TK, KERNEL == 3, true><<<grid, threads, smem, stream>>>(tq, tk, tv, p);
        else
            bsa_attention_kernel<D, TK, KERNEL == 3, false><<<grid, threads, smem, stream>>>(tq, tk, tv, p);
    }
    else if constexpr (KERNEL == 1)
        bsa_attention_pair_kernel<D, TK><<<grid, kPairThreads, smem, stream>>>(tq, tk, tv, p);
    else if constexpr (KERNEL == 2)
        bsa_attention_cs_kernel<D, TK><<<grid, kCsThreads, smem, stream>>>(tq, tk, tv, p);
    else {
        // The ping-pong kernel waits for its predecessor itself (grid_dependency_wait), so it may be scheduled while
        // the task-organisation kernel is still sorting: its launch latency and prologue overlap that kernel.
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)grid);
        cfg.blockDim = dim3((unsigned)kPpThreads);
        cfg.dynamicSmemBytes = (size_t)smem;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaError_t le = a.f16 ? cudaLaunchKernelEx(&cfg, bsa_attention_pp_kernel<D, TK, true>, tq, tk, tv, p)
                               : cudaLaunchKernelEx(&cfg, bsa_attention_pp_kernel<D, TK, false>, tq, tk, tv, p);
        count_launch();
        return le;
    }
    count_launch();
    return cudaGetLastError();
}

}  // namespace

// Shared-memory budget: 227 KB per CTA minus each kernel's static shared memory (barriers, exchange
// buffer), which the compiler rounds up to the 1024-byte alignment of the dynamic part.
static int static_smem_bytes(int kernel) { return (kernel == 2 || kernel == 4) ? 3072 : 1024; }

static int kv_buffers_that_fit(int d, int T_KV, int kernel) {
    const int q = ((kernel == 1 || kernel == 4) ? 2 : 1) * kTQ * d * 2;  // kernel 1: two Q slots; kernel 4: two Q buffers
    const int kv = T_KV * d * 2;
    return (232448 - static_smem_bytes(kernel) - q) / kv;
}

static void split_stages(int total, int kernel, int* nk, int* nv) {
    if (kernel == 4) {
        // a K tile lives for one tile period (load -> its Q K^T), a V tile for about three (load -> its P V): two K
        // buffers measured as fast as three, so V gets three fifths
        *nk = total * 2 / 5;
        if (*nk < 2) *nk = 2;
    } else {
        *nk = total / 2;  // V is held one step longer than K, it gets the odd buffer
    }
    *nv = total - *nk;
    if (*nk > kMaxStages) *nk = kMaxStages;
    if (*nv > kMaxStages) *nv = kMaxStages;
}

int attention_max_stages(int d, int T_KV, int kernel) {
    if (kernel == kKernelRowBlock) return (d <= 128 && T_KV <= rb_max_chunk(d)) ? 2 : 0;  // one K and one V buffer per warp
    if (d == 256 && !((kernel == 0 || kernel == 3) && T_KV == 64)) return 0;  // see launch_forward
    const int nb = kv_buffers_that_fit(d, T_KV, kernel);
    if (kernel == 1 || kernel == 4) return nb > 2 * kMaxStages ? 2 * kMaxStages : nb;  // total K + V buffers
    const int s = nb / 2;
    return s > kMaxStages ? kMaxStages : s;
}

int attention_smem_bytes(int d, int T_KV, int stages, int kernel) {
    const int q = ((kernel == 1 || kernel == 4) ? 2 : 1) * kTQ * d * 2;
    const int kv = T_KV * d * 2;
    int need = q + ((kernel == 1 || kernel == 4) ? stages : 2 * stages) * kv;
    // more than half of the SM's shared memory, so exactly one CTA (and one 512-column TMEM allocation) per SM
    if (need < 120 * 1024) need = 120 * 1024;
    return need;
}

#if defined(BSA_TRACE) || defined(BSA_PHASES)
extern "C" __attribute__((visibility("default"))) int bsa_debug_trace_copy(long long* host, int role) {
    if (role >= 100)  // 100 / 101: CTA entry / exit times
        return (int)cudaMemcpyFromSymbol(host, g_cta_times, sizeof(long long) * 4096, sizeof(long long) * 4096 * (role - 100));
    return (int)cudaMemcpyFromSymbol(host, g_trace, sizeof(long long) * 4096, sizeof(long long) * 4096 * role);
}
#endif

// Test hooks: the limit of the bounded device waits, and the withheld arrival described at g_withhold_arrival.
extern "C" __attribute__((visibility("default"))) bsa_status_t bsa_debug_set_wait_limit(long long cycles) {
    const long long v = cycles > 0 ? cycles : 2000000000ll;
    return cudaMemcpyToSymbol(ptx::g_wait_limit_cycles, &v, sizeof v) == cudaSuccess ? BSA_OK : BSA_ERR_CUDA;
}
extern "C" __attribute__((visibility("default"))) bsa_status_t bsa_debug_withhold_arrival(int on) {
    const int v = on ? 1 : 0;
    return cudaMemcpyToSymbol(g_withhold_arrival, &v, sizeof v) == cudaSuccess ? BSA_OK : BSA_ERR_CUDA;
}

cudaError_t launch_forward(const ForwardArgs& a, cudaStream_t stream, const char** err_detail) {
    AttnParams p;
    p.items = a.items;
    p.tile_col = a.tile_col;
    p.tile_member = a.tile_member;
    p.counters = a.counters;
    p.O = reinterpret_cast<__nv_bfloat16*>(a.O);
    p.LSE = a.LSE;
    p.ws_O = a.ws_O;
    p.ws_LSE = a.ws_LSE;
    const int bits = a.g.sQ128 * a.g.sK;
    p.full_member = (bits >= 64) ? ~0ull : ((1ull << bits) - 1ull);
    p.N = (int32_t)a.g.N;
    p.Nkv = (int32_t)a.g.N_kv;
    p.o_head = a.nhd ? (int64_t)a.d : (int64_t)a.g.N * a.d;
    p.o_row = a.nhd ? (int64_t)a.g.H * a.d : (int64_t)a.d;
    p.lgBQ = (a.g.sQ128 > 1) ? a.g.lgBQ : 31;
    p.lgBKV = (a.g.sK > 1) ? a.g.lgBKV : 31;
    p.sK = a.g.sK;
    p.stages = a.stages;
    p.stages_v = a.stages;
    if (a.kernel == 1 || a.kernel == 4) split_stages(a.stages, a.kernel, &p.stages, &p.stages_v);
    p.scale_log2 = (float)(1.4426950408889634 / sqrt((double)a.d));
    cudaError_t e;
    if (a.kernel == kKernelRowBlock) return launch_forward_rb(a, stream, err_detail);
    const int key = a.kernel * 1000 + a.d + a.g.T_KV / 64;  // kernel, d, T_KV
    if (key == 128 + 2) e = launch_attn<128, 128, 0>(a, p, stream, err_detail);
    else if (key == 128 + 1) e = launch_attn<128, 64, 0>(a, p, stream, err_detail);
    else if (key == 64 + 2) e = launch_attn<64, 128, 0>(a, p, stream, err_detail);
    else if (key == 64 + 1) e = launch_attn<64, 64, 0>(a, p, stream, err_detail);
    else if (key == 1000 + 128 + 2) e = launch_attn<128, 128, 1>(a, p, stream, err_detail);
    else if (key == 1000 + 128 + 1) e = launch_attn<128, 64, 1>(a, p, stream, err_detail);
    else if (key == 1000 + 64 + 2) e = launch_attn<64, 128, 1>(a, p, stream, err_detail);
    else if (key == 1000 + 64 + 1) e = launch_attn<64, 64, 1>(a, p, stream, err_detail);
    else if (key == 2000 + 128 + 2) e = launch_attn<128, 128, 2>(a, p, stream, err_detail);
    else if (key == 2000 + 128 + 1) e = launch_attn<128, 64, 2>(a, p, stream, err_detail);
    else if (key == 2000 + 64 + 2) e = launch_attn<64, 128, 2>(a, p, stream, err_detail);
    else if (key == 2000 + 64 + 1) e = launch_attn<64, 64, 2>(a, p, stream, err_detail);
    else if (key == 3000 + 128 + 2) e = launch_attn<128, 128, 3>(a, p, stream, err_detail);
    else if (key == 3000 + 128 + 1) e = launch_attn<128, 64, 3>(a, p, stream, err_detail);
    else if (key == 3000 + 64 + 2) e = launch_attn<64, 128, 3>(a, p, stream, err_detail);
    else if (key == 3000 + 64 + 1) e = launch_attn<64, 64, 3>(a, p, stream, err_detail);
    // d = 256: the output accumulator takes 256 of the 512 tensor-memory columns, which leaves room for the two score
    // buffers only where P is written in place over S (the single-tile kernels), with 64-key tiles
    else if (key == 256 + 1) e = launch_attn<256, 64, 0>(a, p, stream, err_detail);
    else if (key == 3000 + 256 + 1) e = launch_attn<256, 64, 3>(a, p, stream, err_detail);
    else if (key == 4000 + 128 + 2) e = launch_attn<128, 128, 4>(a, p, stream, err_detail);
    else if (key == 4000 + 128 + 1) e = launch_attn<128, 64, 4>(a, p, stream, err_detail);
    else if (key == 4000 + 64 + 2) e = launch_attn<64, 128, 4>(a, p, stream, err_detail);
    else if (key == 4000 + 64 + 1) e = launch_attn<64, 64, 4>(a, p, stream, err_detail);
    else {
        *err_detail = "no kernel for this (d, T_KV)";
        return cudaErrorInvalidValue;
    }
    if (e != cudaSuccess) return e;
    if (a.has_split) e = launch_merge(a, stream);
    return e;
}

// Split-K reduction alone (also the merge-only test hook: the workspace then holds an earlier forward's partials).
cudaError_t launch_merge(const ForwardArgs& a, cudaStream_t stream) {
    const long long o_head = a.nhd ? (long long)a.d : (long long)a.g.N * a.d;
    const long long o_row = a.nhd ? (long long)a.g.H * a.d : (long long)a.d;
    // one CTA per 256 (row, 8-column) units of a merged tile, grid-strided beyond 8 waves
    const long long want = (long long)a.max_split_rows * (kTQ * (a.d / 8) / 256);
    int grid = want < 8ll * a.num_sms ? (int)want : 8 * a.num_sms;
    if (grid < 1) grid = 1;
    if (a.d == 256)
        bsa_merge_kernel<256><<<grid, 256, 0, stream>>>(a.split_rows, a.counters, a.ws_O, a.ws_LSE,
                                                        reinterpret_cast<__nv_bfloat16*>(a.O), a.LSE, (int)a.g.N, a.f16, o_head, o_row);
    else if (a.d == 128)
        bsa_merge_kernel<128><<<grid, 256, 0, stream>>>(a.split_rows, a.counters, a.ws_O, a.ws_LSE,
                                                        reinterpret_cast<__nv_bfloat16*>(a.O), a.LSE, (int)a.g.N, a.f16, o_head, o_row);
    else
        bsa_merge_kernel<64><<<grid, 256, 0, stream>>>(a.split_rows, a.counters, a.ws_O, a.ws_LSE,
                                                       reinterpret_cast<__nv_bfloat16*>(a.O), a.LSE, (int)a.g.N, a.f16, o_head, o_row);
    count_launch();
    return cudaGetLastError();
}

}  // namespace bsa
