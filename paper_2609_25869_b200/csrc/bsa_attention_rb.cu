// Row-block attention kernel: physical Q tiles of 16 rows (paper Section 4.2: the physical tile need not be the
// logical block; Section 4.4: a catalog holds several tile shapes per architecture).
//
// The tensor-memory kernels of bsa_attention.cu compute 128 query rows per MMA, so logical blocks of 16 to 64 rows
// are Coarsened onto them and every physical tile also computes the pairs of its inactive sub-blocks (4-5 times the
// active pairs on masks whose neighbouring row blocks select different columns).  This kernel keeps such masks at
// their own granularity instead: one WARP owns a 16-row fragment of a logical row block (a 16-row physical tile,
// Refined along Q for B_Q > 16) and walks that block's own KV tile list with the register-level tensor instruction
// mma.sync.m16n8k16 (bf16 or fp16 in, fp32 accumulate), FlashAttention-2 style:
//   * K and V chunks of T_KV keys (8 KB each at most) are gathered with cp.async into a 16 KB staging area private to
//     the warp (128-byte-row XOR swizzle), K read back with ldmatrix, V with ldmatrix.trans; the next K chunk is in
//     flight during the softmax and P V of the current one, the next V chunk during the next Q K^T;
//   * S = Q K^T, online softmax with the running row maximum in the exp2 domain, P rounded to bf16 in registers
//     (the accumulator layout of two 8-key tiles is the A-operand layout of one 16-key step), O += P V;
//   * no block-level synchronisation at all: warps are independent, twelve per SM.
// The register-level instruction peaks at about a third of the tcgen05 rate on this GPU, so the kernel pays off only
// where Coarsening wastes more than that; the plan table decides per regime.
#include <cuda_bf16.h>
#include <math.h>

#include <atomic>

#include "bsa_common.h"

namespace bsa {
namespace {

constexpr int kRbWarps = 12;        // warps per CTA (one CTA per SM)
constexpr int kRbStageBytes = 8192; // one K or V chunk
constexpr unsigned kFullMask = 0xffffffffu;

struct RbParams {
    const __nv_bfloat16* Q;
    const __nv_bfloat16* K;
    const __nv_bfloat16* V;
    __nv_bfloat16* O;
    float* LSE;
    const WorkItem* items;
    const int32_t* tile_col;
    const PlanCountersDev* counters;
    long long q_head, q_row;    // element strides of Q and O between heads / token rows
    long long kv_head, kv_row;  // the same for K and V
    int32_t N, Nkv;
    float scale_log2;           // log2(e) / sqrt(d)
};

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

// 16-byte asynchronous copy global -> shared; src_bytes = 0 writes zeros (rows beyond the last key).
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
                 : "r"(addr));
}
// D (16x8, fp32) += A (16x16, row-major) * B (16x8, column-major); A and B bf16, or IEEE half with F16
template <bool F16>
__device__ __forceinline__ void mma_16816(float* c, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    if (F16)
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
    else
        asm volatile(
            "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
            : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
            : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
template <bool F16>
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {  // two fp32 -> the kernel's 16-bit element type
    uint32_t r;
    if (F16)
        asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    else
        asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
    return r;
}

// Byte offset of 16-byte chunk `chunk` of row `row` in a staged tile whose rows are ROWB bytes: the chunk index is
// XORed with the row's low three bits, so the eight row addresses of an ldmatrix fall into eight different bank groups.
template <int ROWB>
__device__ __forceinline__ uint32_t swz(int row, int chunk) {
    return (uint32_t)(row * ROWB + ((chunk ^ (row & 7)) << 4));
}

// Gathers keys [key0, key0 + CK) of one head (rows of D bf16) into a staging buffer; rows at or beyond n_rows are
// written as zeros.  512 bytes per warp instruction, consecutive lanes on consecutive 16-byte chunks of a row.
template <int D, int CK>
__device__ __forceinline__ void stage_chunk(uint32_t dst, const __nv_bfloat16* __restrict__ base, long long row_stride,
                                            int key0, int n_rows, int lane) {
    constexpr int CPR = D / 8;                 // 16-byte chunks per row
    constexpr int ITERS = CK * CPR / 32;
#pragma unroll
    for (int i = 0; i < ITERS; ++i) {
        const int idx = i * 32 + lane;
        const int row = idx / CPR, chunk = idx % CPR;
        const int key = key0 + row;
        const bool ok = key < n_rows;
        const __nv_bfloat16* src = base + (long long)(ok ? key : n_rows - 1) * row_stride + chunk * 8;
        cp_async16(dst + swz<D * 2>(row, chunk), src, ok ? 16 : 0);
    }
}

template <int D, int CK, bool F16>
__global__ void __launch_bounds__(kRbWarps * 32, 1) bsa_attention_rb_kernel(const RbParams p) {
    static_assert(CK * D * 2 <= kRbStageBytes, "a chunk must fit its staging buffer");
    static_assert(CK % 16 == 0 && D % 16 == 0, "whole MMA steps");
    constexpr int NT_S = CK / 8;   // 8-key accumulator tiles of S
    constexpr int KS_QK = D / 16;  // 16-wide steps over the head dimension
    constexpr int KS_PV = CK / 16; // 16-key steps of P V
    constexpr int NT_O = D / 8;    // 8-column accumulator tiles of O
    extern __shared__ __align__(128) uint8_t smem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    uint8_t* stage = smem + warp * 2 * kRbStageBytes;
    const uint32_t sK = smem_addr(stage), sV = sK + kRbStageBytes;

    const int n_items = p.counters->nitems;
    const int total_warps = (int)gridDim.x * kRbWarps;
    const int gw = (int)blockIdx.x * kRbWarps + warp;
    const int n_rounds = (n_items + total_warps - 1) / total_warps;
    const float c2 = p.scale_log2;

    for (int k = 0; k < n_rounds; ++k) {
        // items arrive longest first: rounds are dealt alternately forwards and backwards to even out the warps' sums
        const int idx = k * total_warps + ((k & 1) ? (total_warps - 1 - gw) : gw);
        if (idx >= n_items) continue;
        const int4 ia = __ldg(reinterpret_cast<const int4*>(p.items + idx));
        const int head = ia.x, q_tile = ia.y, tile_begin = ia.z, tile_end = ia.w;
        const int row0 = q_tile * 16;
        const int r_lo = row0 + g, r_hi = row0 + g + 8;
        __nv_bfloat16* o_lo = p.O + (long long)head * p.q_head + (long long)r_lo * p.q_row;
        __nv_bfloat16* o_hi = p.O + (long long)head * p.q_head + (long long)r_hi * p.q_row;
        if (tile_end <= tile_begin) {  // no active column: zero output, LSE = -inf
#pragma unroll
            for (int n = 0; n < NT_O; ++n) {
                if (r_lo < p.N) *reinterpret_cast<uint32_t*>(o_lo + n * 8 + 2 * t) = 0u;
                if (r_hi < p.N) *reinterpret_cast<uint32_t*>(o_hi + n * 8 + 2 * t) = 0u;
            }
            if (t == 0) {
                if (r_lo < p.N) p.LSE[(long long)head * p.N + r_lo] = -INFINITY;
                if (r_hi < p.N) p.LSE[(long long)head * p.N + r_hi] = -INFINITY;
            }
            continue;
        }
        const __nv_bfloat16* Kh = p.K + (long long)head * p.kv_head;
        const __nv_bfloat16* Vh = p.V + (long long)head * p.kv_head;
        // first K and V chunks on their way while the Q fragment is loaded
        int col = __ldg(p.tile_col + tile_begin);
        stage_chunk<D, CK>(sK, Kh, p.kv_row, col * CK, p.Nkv, lane);
        cp_async_commit();
        stage_chunk<D, CK>(sV, Vh, p.kv_row, col * CK, p.Nkv, lane);
        cp_async_commit();
        // Q fragment (A operand, row-major 16 x 16 per step): rows g and g+8, columns 2t, 2t+1 and 8 further
        uint32_t qa[KS_QK][4];
        {
            const __nv_bfloat16* q_lo = p.Q + (long long)head * p.q_head + (long long)r_lo * p.q_row;
            const __nv_bfloat16* q_hi = p.Q + (long long)head * p.q_head + (long long)r_hi * p.q_row;
#pragma unroll
            for (int ks = 0; ks < KS_QK; ++ks) {
                const int c = ks * 16 + 2 * t;
                qa[ks][0] = (r_lo < p.N) ? __ldg(reinterpret_cast<const uint32_t*>(q_lo + c)) : 0u;
                qa[ks][1] = (r_hi < p.N) ? __ldg(reinterpret_cast<const uint32_t*>(q_hi + c)) : 0u;
                qa[ks][2] = (r_lo < p.N) ? __ldg(reinterpret_cast<const uint32_t*>(q_lo + c + 8)) : 0u;
                qa[ks][3] = (r_hi < p.N) ? __ldg(reinterpret_cast<const uint32_t*>(q_hi + c + 8)) : 0u;
            }
        }
        float o[NT_O][4];
#pragma unroll
        for (int n = 0; n < NT_O; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
        float m_lo = -INFINITY, m_hi = -INFINITY;  // running row maxima, exp2 domain (score * c2)
        float l_lo = 0.f, l_hi = 0.f;              // this thread's share of the row sums

        for (int j = tile_begin; j < tile_end; ++j) {
            const int key0 = col * CK;
            const bool more = j + 1 < tile_end;
            const int col_next = more ? __ldg(p.tile_col + j + 1) : 0;
            // ---- S = Q K^T ----
            cp_async_wait<1>();  // K chunk j has landed (V chunk j may still be in flight)
            __syncwarp();
            float s[NT_S][4];
#pragma unroll
            for (int n = 0; n < NT_S; ++n) s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.f;
#pragma unroll
            for (int np = 0; np < NT_S / 2; ++np) {
#pragma unroll
                for (int ks = 0; ks < KS_QK; ++ks) {
                    // four 8x8 matrices: keys np*16 + {0..7, 8..15} x head-dim columns ks*16 + {0..7, 8..15}
                    const int key = np * 16 + ((lane >> 4) << 3) + (lane & 7);
                    const int chunk = ks * 2 + ((lane >> 3) & 1);
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4(sK + swz<D * 2>(key, chunk), b0, b1, b2, b3);
                    mma_16816<F16>(s[2 * np], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b0, b1);
                    mma_16816<F16>(s[2 * np + 1], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b2, b3);
                }
            }
            __syncwarp();  // every lane has read the K buffer
            if (more) stage_chunk<D, CK>(sK, Kh, p.kv_row, col_next * CK, p.Nkv, lane);
            cp_async_commit();
            // ---- online softmax ----
            if (key0 + CK > p.Nkv) {  // ragged last chunk: keys at or beyond N_kv do not exist
#pragma unroll
                for (int n = 0; n < NT_S; ++n) {
                    const int kc = key0 + n * 8 + 2 * t;
                    if (kc >= p.Nkv) s[n][0] = s[n][2] = -INFINITY;
                    if (kc + 1 >= p.Nkv) s[n][1] = s[n][3] = -INFINITY;
                }
            }
            float mx_lo = -INFINITY, mx_hi = -INFINITY;
#pragma unroll
            for (int n = 0; n < NT_S; ++n) {
                mx_lo = fmaxf(mx_lo, fmaxf(s[n][0], s[n][1]));
                mx_hi = fmaxf(mx_hi, fmaxf(s[n][2], s[n][3]));
            }
            mx_lo = fmaxf(mx_lo, __shfl_xor_sync(kFullMask, mx_lo, 1));
            mx_hi = fmaxf(mx_hi, __shfl_xor_sync(kFullMask, mx_hi, 1));
            mx_lo = fmaxf(mx_lo, __shfl_xor_sync(kFullMask, mx_lo, 2));
            mx_hi = fmaxf(mx_hi, __shfl_xor_sync(kFullMask, mx_hi, 2));
            const float mn_lo = fmaxf(m_lo, mx_lo * c2), mn_hi = fmaxf(m_hi, mx_hi * c2);
            const float a_lo = (m_lo == -INFINITY) ? 0.f : ex2(m_lo - mn_lo);
            const float a_hi = (m_hi == -INFINITY) ? 0.f : ex2(m_hi - mn_hi);
            m_lo = mn_lo;
            m_hi = mn_hi;
            const float nm_lo = (mn_lo == -INFINITY) ? 0.f : -mn_lo, nm_hi = (mn_hi == -INFINITY) ? 0.f : -mn_hi;
            float sum_lo = 0.f, sum_hi = 0.f;
            uint32_t pa[KS_PV][4];  // P as the A operand of P V
#pragma unroll
            for (int n = 0; n < NT_S; ++n) {
                const float p0 = ex2(fmaf(s[n][0], c2, nm_lo)), p1 = ex2(fmaf(s[n][1], c2, nm_lo));
                const float p2 = ex2(fmaf(s[n][2], c2, nm_hi)), p3 = ex2(fmaf(s[n][3], c2, nm_hi));
                sum_lo += p0 + p1;
                sum_hi += p2 + p3;
                pa[n >> 1][(n & 1) * 2 + 0] = pack_bf16<F16>(p0, p1);
                pa[n >> 1][(n & 1) * 2 + 1] = pack_bf16<F16>(p2, p3);
            }
            l_lo = fmaf(l_lo, a_lo, sum_lo);
            l_hi = fmaf(l_hi, a_hi, sum_hi);
            if (__any_sync(kFullMask, a_lo != 1.f || a_hi != 1.f)) {  // a maximum moved: rescale the running output
#pragma unroll
                for (int n = 0; n < NT_O; ++n) {
                    o[n][0] *= a_lo;
                    o[n][1] *= a_lo;
                    o[n][2] *= a_hi;
                    o[n][3] *= a_hi;
                }
            }
            // ---- O += P V ----
            cp_async_wait<1>();  // V chunk j has landed (K chunk j+1 may still be in flight)
            __syncwarp();
#pragma unroll
            for (int ks = 0; ks < KS_PV; ++ks) {
#pragma unroll
                for (int nd = 0; nd < NT_O / 2; ++nd) {
                    // four 8x8 matrices, transposed on the way: keys ks*16 + {0..7, 8..15} x columns nd*16 + {0..7, 8..15}
                    const int key = ks * 16 + (((lane >> 3) & 1) << 3) + (lane & 7);
                    const int chunk = nd * 2 + (lane >> 4);
                    uint32_t b0, b1, b2, b3;
                    ldmatrix_x4_trans(sV + swz<D * 2>(key, chunk), b0, b1, b2, b3);
                    mma_16816<F16>(o[2 * nd], pa[ks][0], pa[ks][1], pa[ks][2], pa[ks][3], b0, b1);
                    mma_16816<F16>(o[2 * nd + 1], pa[ks][0], pa[ks][1], pa[ks][2], pa[ks][3], b2, b3);
                }
            }
            __syncwarp();  // every lane has read the V buffer
            if (more) stage_chunk<D, CK>(sV, Vh, p.kv_row, col_next * CK, p.Nkv, lane);
            cp_async_commit();
            col = col_next;
        }
        cp_async_wait<0>();
        // ---- epilogue: row sums over the four lanes of a row, normalise, store ----
        l_lo += __shfl_xor_sync(kFullMask, l_lo, 1);
        l_hi += __shfl_xor_sync(kFullMask, l_hi, 1);
        l_lo += __shfl_xor_sync(kFullMask, l_lo, 2);
        l_hi += __shfl_xor_sync(kFullMask, l_hi, 2);
        const float inv_lo = (l_lo > 0.f) ? 1.f / l_lo : 0.f, inv_hi = (l_hi > 0.f) ? 1.f / l_hi : 0.f;
#pragma unroll
        for (int n = 0; n < NT_O; ++n) {
            if (r_lo < p.N) *reinterpret_cast<uint32_t*>(o_lo + n * 8 + 2 * t) = pack_bf16<F16>(o[n][0] * inv_lo, o[n][1] * inv_lo);
            if (r_hi < p.N) *reinterpret_cast<uint32_t*>(o_hi + n * 8 + 2 * t) = pack_bf16<F16>(o[n][2] * inv_hi, o[n][3] * inv_hi);
        }
        if (t == 0) {
            if (r_lo < p.N)
                p.LSE[(long long)head * p.N + r_lo] = (l_lo > 0.f) ? fmaf(m_lo, 0.6931471805599453f, logf(l_lo)) : -INFINITY;
            if (r_hi < p.N)
                p.LSE[(long long)head * p.N + r_hi] = (l_hi > 0.f) ? fmaf(m_hi, 0.6931471805599453f, logf(l_hi)) : -INFINITY;
        }
    }
}

template <int D, int CK, bool F16>
cudaError_t launch_rb_t(const ForwardArgs& a, const RbParams& p, cudaStream_t stream, const char** err) {
    constexpr int smem = kRbWarps * 2 * kRbStageBytes;
    static std::atomic<int> attr_set_dev[kMaxDevices];
    const int dev = (a.device >= 0 && a.device < kMaxDevices) ? a.device : 0;
    if (!attr_set_dev[dev].load(std::memory_order_relaxed)) {
        cudaError_t e = cudaFuncSetAttribute(bsa_attention_rb_kernel<D, CK, F16>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
        if (e != cudaSuccess) {
            *err = "cudaFuncSetAttribute(max dynamic shared memory)";
            return e;
        }
        attr_set_dev[dev].store(1, std::memory_order_relaxed);
    }
    long long want = ((long long)a.max_items + kRbWarps - 1) / kRbWarps;
    int grid = want < a.num_sms ? (int)want : a.num_sms;
    if (grid < 1) grid = 1;
    bsa_attention_rb_kernel<D, CK, F16><<<grid, kRbWarps * 32, smem, stream>>>(p);
    count_launch();
    return cudaGetLastError();
}
template <int D, int CK>
cudaError_t launch_rb(const ForwardArgs& a, const RbParams& p, cudaStream_t stream, const char** err) {
    return a.f16 ? launch_rb_t<D, CK, true>(a, p, stream, err) : launch_rb_t<D, CK, false>(a, p, stream, err);
}

}  // namespace

// Largest KV chunk (keys) the row-block kernel can stage for head dimension d.
int rb_max_chunk(int d) { return kRbStageBytes / (d * 2); }

cudaError_t launch_forward_rb(const ForwardArgs& a, cudaStream_t stream, const char** err_detail) {
    RbParams p;
    p.Q = reinterpret_cast<const __nv_bfloat16*>(a.Q);
    p.K = reinterpret_cast<const __nv_bfloat16*>(a.K);
    p.V = reinterpret_cast<const __nv_bfloat16*>(a.V);
    p.O = reinterpret_cast<__nv_bfloat16*>(a.O);
    p.LSE = a.LSE;
    p.items = a.items;
    p.tile_col = a.tile_col;
    p.counters = a.counters;
    p.q_head = a.nhd ? (long long)a.d : (long long)a.g.N * a.d;
    p.q_row = a.nhd ? (long long)a.g.H * a.d : (long long)a.d;
    p.kv_head = a.nhd ? (long long)a.d : (long long)a.g.N_kv * a.d;
    p.kv_row = a.nhd ? (long long)a.g.H * a.d : (long long)a.d;
    p.N = (int32_t)a.g.N;
    p.Nkv = (int32_t)a.g.N_kv;
    p.scale_log2 = (float)(1.4426950408889634 / sqrt((double)a.d));
    const int key = a.d * 1000 + a.g.T_KV;
    if (key == 64 * 1000 + 64) return launch_rb<64, 64>(a, p, stream, err_detail);
    if (key == 64 * 1000 + 32) return launch_rb<64, 32>(a, p, stream, err_detail);
    if (key == 64 * 1000 + 16) return launch_rb<64, 16>(a, p, stream, err_detail);
    if (key == 128 * 1000 + 32) return launch_rb<128, 32>(a, p, stream, err_detail);
    if (key == 128 * 1000 + 16) return launch_rb<128, 16>(a, p, stream, err_detail);
    *err_detail = "no row-block kernel for this (d, T_KV)";
    return cudaErrorInvalidValue;
}

}  // namespace bsa
