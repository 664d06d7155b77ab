// Plan construction on the GPU (paper Section 5.2 "Regime lookup" / "Launch preparation",
// Section 4.2 physical mapping, Section 4.3 task organisation).
//
//   mask_row_stats : M -> active blocks per row + scalar statistics s_A(M) (density inputs,
//                    active-block-run coverage, max row nnz)
//   row_scan       : exclusive scan -> block-CSR offsets
//   csr_fill       : sorted active KV column indices (block-CSR of the shared mask state mu(M))
//   tile_map       : block-CSR -> physical tiles with membership bits (Direct / Coarsened / Refined)
//                    + Split-K partition count of every Q tile row
//   organize       : work items (Q tile row x KV partition), ordered longest-first
//
// All kernels are integer-only and bandwidth-bound; none needs the host between them.
#include "bsa_common.h"

namespace bsa {

namespace {

constexpr unsigned kFull = 0xffffffffu;

// ------------------------------------------------------------------------------------------
// Both mask passes read a row as aligned 16-byte words, one word per lane and step (512 bytes per
// warp step); bytes of a word that fall outside the row are masked off.  `row_word_bits` returns,
// for the word at index `w` (in 16-byte units of the flat mask array), a 16-bit mask of the bytes
// that belong to [row_begin, row_end) and are non-zero.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned row_word_bits(const uint4* __restrict__ words, long long w, long long row_begin,
                                                  long long row_end) {
    const long long byte0 = w * 16;
    if (byte0 >= row_end || byte0 + 16 <= row_begin) return 0u;
    const uint4 v = __ldg(words + w);
    unsigned bits = 0;
    const unsigned parts[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const unsigned ne = __vcmpne4(parts[q], 0u);  // 0xff per non-zero byte
        bits |= ((ne & 1u) | ((ne >> 7) & 2u) | ((ne >> 14) & 4u) | ((ne >> 21) & 8u)) << (4 * q);
    }
    // keep only the bytes inside the row
    const int lo = row_begin > byte0 ? (int)(row_begin - byte0) : 0;
    const int hi = row_end < byte0 + 16 ? (int)(row_end - byte0) : 16;
    const unsigned keep = (hi >= 16 ? 0xffffu : ((1u << hi) - 1u)) & ~((1u << lo) - 1u);
    return bits & keep;
}

// Called by thread 0 of every CTA of a statistics kernel after it has added its share: the CTA that finds itself last
// moves the totals into pinned host memory, so the host can read them without a copy command or an event.
__device__ __forceinline__ void post_stats_if_last(MaskStatsDev* stats, MaskStatsHost* post, unsigned seq) {
    if (!post) return;
    __threadfence();
    if (atomicAdd(&stats->blocks_done, 1u) != gridDim.x - 1) return;
    __threadfence();
    // the totals are taken out and the accumulators left at zero for the next request that uses them (no memset
    // in front of the next statistics kernel)
    post->nnz = atomicExch(&stats->nnz, 0ull);
    post->in_runs = atomicExch(&stats->in_runs, 0ull);
    post->hash[0] = atomicExch(&stats->hash[0], 0ull);
    post->hash[1] = atomicExch(&stats->hash[1], 0ull);
    post->max_row_nnz = atomicExch(&stats->max_row_nnz, 0u);
    atomicExch(&stats->blocks_done, 0u);
    __threadfence_system();
    *reinterpret_cast<volatile unsigned*>(&post->seq) = seq;
}

// Fingerprint of the activity pattern, for the plan cache: every non-empty word of a row (its activity bits `m`, at
// word position `pos` of row `row`) is mixed with its position by two different 64-bit finalisers, and the two
// results are summed over the mask modulo 2^64 (a sum, so that warps and CTAs can add their shares in any order).
__device__ __forceinline__ unsigned long long mix64(unsigned long long x, unsigned long long c1, unsigned long long c2) {
    x ^= x >> 33;
    x *= c1;
    x ^= x >> 29;
    x *= c2;
    x ^= x >> 32;
    return x;
}
struct MaskHash {
    unsigned long long a = 0, b = 0;
    __device__ __forceinline__ void add(unsigned m, int row, long long pos) {
        if (!m) return;
        const unsigned long long where = ((unsigned long long)(unsigned)row << 32) | (unsigned long long)(unsigned)pos;
        const unsigned long long x = where * 0x9E3779B97F4A7C15ull + (unsigned long long)m * 0xC2B2AE3D27D4EB4Full + 1ull;
        a += mix64(x, 0xFF51AFD7ED558CCDull, 0xC4CEB9FE1A85EC53ull);
        b += mix64(x ^ 0x5851F42D4C957F2Dull, 0xBF58476D1CE4E5B9ull, 0x94D049BB133111EBull);
    }
    // adds the warp's total to the two global sums
    __device__ __forceinline__ void flush(MaskStatsDev* stats, int lane) {
        for (int o = 16; o > 0; o >>= 1) {
            a += __shfl_down_sync(kFull, a, o);
            b += __shfl_down_sync(kFull, b, o);
        }
        if (lane == 0 && (a | b)) {
            atomicAdd(&stats->hash[0], a);
            atomicAdd(&stats->hash[1], b);
        }
    }
};

// ------------------------------------------------------------------------------------------
// mask_row_stats: one warp per (head, query-block) row.
// A block counts towards run coverage iff its left or right neighbour in the same row is active.
// ------------------------------------------------------------------------------------------
template <bool HASH>
__global__ void __launch_bounds__(256) mask_row_stats_kernel(const uint8_t* __restrict__ mask, int nrows, int nKb,
                                                              int32_t* __restrict__ row_nnz, MaskStatsDev* stats,
                                                              MaskStatsHost* post, unsigned seq, int rows_per_warp) {
    __shared__ unsigned s_nnz[8], s_runs[8], s_max[8];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // A warp takes `rows_per_warp` consecutive rows (1 in every launch today).
    unsigned w_nnz = 0, w_runs = 0, w_max = 0;
    MaskHash hash;
    for (int rr = 0; rr < rows_per_warp; ++rr) {
        const int row = (blockIdx.x * 8 + warp) * rows_per_warp + rr;
        if (row >= nrows) break;
        unsigned nnz = 0, runs = 0;
        // the mask base may be unaligned: address words relative to the enclosing 16-byte grid
        const unsigned long long base = reinterpret_cast<unsigned long long>(mask);
        const uint4* words = reinterpret_cast<const uint4*>(base & ~15ull);
        const long long rb = (long long)(base & 15ull) + (long long)row * nKb, re = rb + nKb;
        const long long w0 = rb >> 4, w1 = (re + 15) >> 4;
        // The last byte of a step does not know its right neighbour yet: if its left neighbour is inactive it is
        // counted one step later, by lane 0, once that neighbour (bit 0 of the next step) is known.
        unsigned carry = 0;  // bits 1:0 = the previous step's last two bytes (bit 1 = the last one)
        // three steps' words are in flight ahead of the one being counted (a row of a few KB is then read almost at once)
        unsigned m_q0 = row_word_bits(words, w0 + lane, rb, re);
        unsigned m_q1 = (w0 + 32 < w1) ? row_word_bits(words, w0 + 32 + lane, rb, re) : 0u;
        unsigned m_q2 = (w0 + 64 < w1) ? row_word_bits(words, w0 + 64 + lane, rb, re) : 0u;
        for (long long w = w0; w < w1; w += 32) {
            const unsigned m = m_q0;
            if (HASH) hash.add(m, row, w - w0 + lane);
            m_q0 = m_q1;
            m_q1 = m_q2;
            m_q2 = (w + 96 < w1) ? row_word_bits(words, w + 96 + lane, rb, re) : 0u;
            // neighbours across lanes: previous lane's bit 15, next lane's bit 0
            unsigned prev15 = __shfl_up_sync(kFull, m >> 15, 1);
            unsigned next0 = __shfl_down_sync(kFull, m & 1u, 1);
            if (lane == 0) prev15 = carry >> 1;
            if (lane == 31) next0 = 0u;
            const unsigned left = ((m << 1) | prev15) & 0xffffu, right = (m >> 1) | (next0 << 15);
            nnz += __popc(m);
            runs += __popc(m & (left | right));
            if (lane == 0 && carry == 2u && (m & 1u)) ++runs;  // previous step's last byte: active, left inactive, right active
            carry = __shfl_sync(kFull, (m >> 14) & 3u, 31);
        }
        for (int o = 16; o > 0; o >>= 1) {
            nnz += __shfl_down_sync(kFull, nnz, o);
            runs += __shfl_down_sync(kFull, runs, o);
        }
        if (lane == 0) {
            row_nnz[row] = (int32_t)nnz;
            w_nnz += nnz;
            w_runs += runs;
            w_max = max(w_max, nnz);
        }
    }
    if (HASH) hash.flush(stats, lane);
    if (lane == 0) {
        s_nnz[warp] = w_nnz;
        s_runs[warp] = w_runs;
        s_max[warp] = w_max;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long tn = 0, tr = 0;
        unsigned mx = 0;
        for (int w = 0; w < 8; ++w) {
            tn += s_nnz[w];
            tr += s_runs[w];
            mx = max(mx, s_max[w]);
        }
        if (tn) {
            atomicAdd(&stats->nnz, tn);
            atomicAdd(&stats->in_runs, tr);
            atomicMax(&stats->max_row_nnz, mx);
        }
        post_stats_if_last(stats, post, seq);
    }
}

// ------------------------------------------------------------------------------------------
// The same two mask passes for a bit-packed mask: bit (c & 7) of byte c >> 3 of a row is block column c; rows start
// every `stride_words` 32-bit words (4-byte aligned).  One 32-bit word (32 blocks) per lane and step; bits at or
// beyond nKb are ignored.  The mask traffic is one eighth of the byte format's.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ unsigned packed_row_word(const uint32_t* __restrict__ row, int w, int nwords, int nKb) {
    if (w >= nwords) return 0u;
    unsigned m = __ldg(row + w);
    const int valid = nKb - w * 32;
    if (valid < 32) m &= (1u << valid) - 1u;
    return m;
}

template <bool HASH>
__global__ void __launch_bounds__(256) mask_row_stats_packed_kernel(const uint32_t* __restrict__ mask, long long stride_words,
                                                                     int nrows, int nKb, int32_t* __restrict__ row_nnz,
                                                                     MaskStatsDev* stats, MaskStatsHost* post, unsigned seq) {
    __shared__ unsigned s_nnz[8], s_runs[8];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row = blockIdx.x * 8 + warp;
    unsigned nnz = 0, runs = 0;
    if (row < nrows) {
        const uint32_t* r = mask + (long long)row * stride_words;
        const int nwords = (nKb + 31) >> 5;
        unsigned carry = 0;  // bits 1:0 = the previous step's last two blocks (bit 1 = the last one)
        unsigned m_next = packed_row_word(r, lane, nwords, nKb);
        MaskHash hash;
        for (int w = 0; w < nwords; w += 32) {
            const unsigned m = m_next;
            if (HASH) hash.add(m, row, w + lane);
            m_next = (w + 32 < nwords) ? packed_row_word(r, w + 32 + lane, nwords, nKb) : 0u;
            unsigned prev31 = __shfl_up_sync(kFull, m >> 31, 1);
            unsigned next0 = __shfl_down_sync(kFull, m & 1u, 1);
            if (lane == 0) prev31 = carry >> 1;
            if (lane == 31) next0 = 0u;
            const unsigned left = (m << 1) | prev31, right = (m >> 1) | (next0 << 31);
            nnz += __popc(m);
            runs += __popc(m & (left | right));
            if (lane == 0 && carry == 2u && (m & 1u)) ++runs;  // see mask_row_stats_kernel
            carry = __shfl_sync(kFull, m >> 30, 31);
        }
        for (int o = 16; o > 0; o >>= 1) {
            nnz += __shfl_down_sync(kFull, nnz, o);
            runs += __shfl_down_sync(kFull, runs, o);
        }
        if (lane == 0) row_nnz[row] = (int32_t)nnz;
        if (HASH) hash.flush(stats, lane);
    }
    if (lane == 0) {
        s_nnz[warp] = nnz;
        s_runs[warp] = runs;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long tn = 0, tr = 0;
        unsigned mx = 0;
        for (int w = 0; w < 8; ++w) {
            tn += s_nnz[w];
            tr += s_runs[w];
            mx = max(mx, s_nnz[w]);
        }
        if (tn) {
            atomicAdd(&stats->nnz, tn);
            atomicAdd(&stats->in_runs, tr);
            atomicMax(&stats->max_row_nnz, mx);
        }
        post_stats_if_last(stats, post, seq);
    }
}

__global__ void __launch_bounds__(256) csr_fill_packed_kernel(const uint32_t* __restrict__ mask, long long stride_words,
                                                               int nrows, int nKb, const int32_t* __restrict__ row_ptr,
                                                               int32_t* __restrict__ col_idx) {
    __shared__ int32_t stage[8][1024];  // a step of the packed format covers 32 x 32 block columns
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row = blockIdx.x * 8 + warp;
    if (row >= nrows) return;
    int32_t* buf = stage[warp];
    const uint32_t* r = mask + (long long)row * stride_words;
    const int nwords = (nKb + 31) >> 5;
    int32_t out = row_ptr[row];
    unsigned m_next = packed_row_word(r, lane, nwords, nKb);
    for (int w = 0; w < nwords; w += 32) {
        unsigned m = m_next;
        m_next = (w + 32 < nwords) ? packed_row_word(r, w + 32 + lane, nwords, nKb) : 0u;
        const int cnt = __popc(m);
        int incl = cnt;
        for (int o = 1; o < 32; o <<= 1) {
            const int x = __shfl_up_sync(kFull, incl, o);
            if (lane >= o) incl += x;
        }
        const int total = __shfl_sync(kFull, incl, 31);
        if (total == 0) continue;
        int pos = incl - cnt;
        const int col0 = (w + lane) * 32;
        while (m) {
            const int b = __ffs(m) - 1;
            buf[pos++] = col0 + b;
            m &= m - 1;
        }
        __syncwarp();
        for (int j = lane; j < total; j += 32) col_idx[out + j] = buf[j];  // consecutive lanes, coalesced
        __syncwarp();
        out += total;
    }
}

// ------------------------------------------------------------------------------------------
// row_scan: exclusive scan of row_nnz by one CTA (rows are few: heads * query blocks).
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(1024) row_scan_kernel(const int32_t* __restrict__ row_nnz, int nrows,
                                                        int32_t* __restrict__ row_ptr) {
    __shared__ int32_t warp_excl[32];
    __shared__ int32_t step_total;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    int32_t carry = 0;  // sum of all rows before this step (same value in every thread)
    for (int i0 = 0; i0 < nrows; i0 += 4096) {
        const int i = i0 + tid * 4;  // four consecutive rows per thread, 16-byte accesses
        int4 v = make_int4(0, 0, 0, 0);
        if (i + 3 < nrows) {
            v = *reinterpret_cast<const int4*>(row_nnz + i);
        } else {
            if (i < nrows) v.x = row_nnz[i];
            if (i + 1 < nrows) v.y = row_nnz[i + 1];
            if (i + 2 < nrows) v.z = row_nnz[i + 2];
        }
        const int32_t t = v.x + v.y + v.z + v.w;
        int32_t incl = t;
        for (int o = 1; o < 32; o <<= 1) {
            const int32_t x = __shfl_up_sync(kFull, incl, o);
            if (lane >= o) incl += x;
        }
        __syncthreads();  // the previous step's warp_excl / step_total have been consumed
        if (lane == 31) warp_excl[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            const int32_t w = warp_excl[lane];
            int32_t wi = w;
            for (int o = 1; o < 32; o <<= 1) {
                const int32_t x = __shfl_up_sync(kFull, wi, o);
                if (lane >= o) wi += x;
            }
            warp_excl[lane] = wi - w;
            if (lane == 31) step_total = wi;
        }
        __syncthreads();
        const int32_t base = carry + warp_excl[warp] + incl - t;
        const int4 o4 = make_int4(base, base + v.x, base + v.x + v.y, base + v.x + v.y + v.z);
        if (i + 3 < nrows) {
            *reinterpret_cast<int4*>(row_ptr + i) = o4;
        } else {
            if (i < nrows) row_ptr[i] = o4.x;
            if (i + 1 < nrows) row_ptr[i + 1] = o4.y;
            if (i + 2 < nrows) row_ptr[i + 2] = o4.z;
        }
        carry += step_total;
    }
    if (tid == 0) row_ptr[nrows] = carry;
}

// ------------------------------------------------------------------------------------------
// csr_fill: one warp per row; a warp scan over the lanes' popcounts keeps columns ascending.
// The indices of a step (up to 512) are first put in order into a shared-memory buffer of the
// warp and then written out by consecutive lanes, so the global stores are coalesced 128-byte
// runs instead of one 4-byte store per active block scattered over the lanes.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void flush_step_indices(const int32_t* buf, int32_t* __restrict__ dst, int n, int lane) {
    for (int j = lane; j < n; j += 32) dst[j] = buf[j];
}

__global__ void __launch_bounds__(256) csr_fill_kernel(const uint8_t* __restrict__ mask, int nrows, int nKb,
                                                        const int32_t* __restrict__ row_ptr,
                                                        int32_t* __restrict__ col_idx) {
    __shared__ int32_t stage[8][512];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int row = blockIdx.x * 8 + warp;
    if (row >= nrows) return;
    int32_t* buf = stage[warp];
    const unsigned long long base = reinterpret_cast<unsigned long long>(mask);
    const uint4* words = reinterpret_cast<const uint4*>(base & ~15ull);
    const long long rb = (long long)(base & 15ull) + (long long)row * nKb, re = rb + nKb;
    const long long w0 = rb >> 4, w1 = (re + 15) >> 4;
    int32_t out = row_ptr[row];
    // three steps' words are in flight ahead of the one being written out
    unsigned m_next = row_word_bits(words, w0 + lane, rb, re);
    unsigned m_next2 = (w0 + 32 < w1) ? row_word_bits(words, w0 + 32 + lane, rb, re) : 0u;
    unsigned m_next3 = (w0 + 64 < w1) ? row_word_bits(words, w0 + 64 + lane, rb, re) : 0u;
    for (long long w = w0; w < w1; w += 32) {
        unsigned m = m_next;
        m_next = m_next2;
        m_next2 = m_next3;
        m_next3 = (w + 96 < w1) ? row_word_bits(words, w + 96 + lane, rb, re) : 0u;
        const int cnt = __popc(m);
        int incl = cnt;
        for (int o = 1; o < 32; o <<= 1) {
            const int x = __shfl_up_sync(kFull, incl, o);
            if (lane >= o) incl += x;
        }
        const int total = __shfl_sync(kFull, incl, 31);
        if (total == 0) continue;
        int pos = incl - cnt;
        const int col0 = (int)((w + lane) * 16 - rb);  // column of this word's byte 0
        while (m) {
            const int b = __ffs(m) - 1;
            buf[pos++] = col0 + b;
            m &= m - 1;
        }
        __syncwarp();
        flush_step_indices(buf, col_idx + out, total, lane);
        __syncwarp();
        out += total;
    }
}

// ------------------------------------------------------------------------------------------
// tile_map.  Output position of tile row t is a capacity offset computed from the block-CSR alone
// (row_ptr of its first logical row times the refinement factors), so no second scan is needed.
//
// Two kernels.  Where no dimension is Coarsened (B_Q >= T_Q and B_KV >= T_KV: Direct or Refined),
// the tile list of a tile row is the column list of its logical row, each column c expanded to
// c*rk .. c*rk+rk-1: already sorted and unique, every membership word all-ones.  One WARP per
// tile row streams it out (tile_map_expand_kernel).  Where a dimension is Coarsened, one CTA per
// tile row ORs the activity bits of its logical rows into a shared-memory array with one
// membership word per KV tile column and compacts the non-zero words in column order
// (tile_map_bitmap_kernel).
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ int32_t split_parts(int32_t cnt, int split_tau, int split_pmax) {
    if (split_pmax > 1 && cnt > split_tau) return min(split_pmax, (cnt + split_tau - 1) / split_tau);
    return 1;
}

__global__ void __launch_bounds__(256) tile_map_expand_kernel(MapGeom g, const int32_t* __restrict__ row_ptr,
                                                               const int32_t* __restrict__ col_idx, int split_tau,
                                                               int split_pmax, int32_t* __restrict__ tile_begin,
                                                               int32_t* __restrict__ tile_cnt, int32_t* __restrict__ row_parts,
                                                               int32_t* __restrict__ tile_col,
                                                               uint64_t* __restrict__ tile_member,
                                                               int32_t* __restrict__ head_counts, PlanCountersDev* counters) {
    __shared__ int32_t w_head[8], w_parts[8], w_cnt[8];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // see organize_kernel
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int trow = blockIdx.x * 8 + warp;
    const int nrows = g.H * g.nQt;
    int32_t cnt = 0, P = 0, h = -1;
    if (trow < nrows) {
        h = trow / g.nQt;
        const int t = trow % g.nQt;
        const int r = t / g.rq, sub = t % g.rq;
        const int32_t b = row_ptr[h * g.nQb + r], e = row_ptr[h * g.nQb + r + 1];
        const int32_t len = e - b;
        const int32_t cap_begin = (b * g.rq + sub * len) * g.rk;
        // Only the row's last column can lose part of its rk tile columns (ragged N_kv), so positions have no holes.
        for (int32_t i0 = 0; i0 < len; i0 += 128) {
            int32_t c[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) c[u] = (i0 + u * 32 + lane < len) ? col_idx[b + i0 + u * 32 + lane] : -1;
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                if (c[u] < 0) continue;
                const int32_t pos = cap_begin + (i0 + u * 32 + lane) * g.rk;
                for (int k = 0; k < g.rk; ++k) {
                    const int tc = c[u] * g.rk + k;
                    if (tc >= g.nKt) break;
                    tile_col[pos + k] = tc;
                    tile_member[(size_t)(pos + k) * g.slots] = 1ull;
                    if (g.slots == 2) tile_member[(size_t)(pos + k) * 2 + 1] = 1ull;
                }
            }
        }
        if (lane == 0) {
            cnt = len * g.rk;
            if (len > 0) {
                const int last = col_idx[e - 1];
                const int lost = (last + 1) * g.rk - g.nKt;
                if (lost > 0) cnt -= lost;
            }
            P = split_parts(cnt, split_tau, split_pmax);
            tile_begin[trow] = cap_begin;
            tile_cnt[trow] = cnt;
            row_parts[trow] = P;
        }
    }
    if (lane == 0) {
        w_head[warp] = h;
        w_parts[warp] = P;
        w_cnt[warp] = cnt;
    }
    __syncthreads();
    if (threadIdx.x == 0) {  // one set of atomics per head that this CTA's eight tile rows touch (one or two heads)
        unsigned long long tot = 0;
        int w = 0;
        while (w < 8 && w_head[w] >= 0) {
            const int hh = w_head[w];
            int32_t items = 0, nsplit = 0, slots = 0;
            for (; w < 8 && w_head[w] == hh; ++w) {
                items += w_parts[w];
                if (w_parts[w] > 1) {
                    ++nsplit;
                    slots += w_parts[w];
                }
                tot += (unsigned long long)w_cnt[w];
            }
            atomicAdd(&head_counts[3 * hh + 0], items);
            if (nsplit) {
                atomicAdd(&head_counts[3 * hh + 1], nsplit);
                atomicAdd(&head_counts[3 * hh + 2], slots);
            }
        }
        if (tot) {
            atomicAdd(&counters->ntiles, tot);
            atomicAdd(&counters->nslot_tiles, tot * (unsigned long long)g.slots);
        }
    }
}

constexpr int kTmThreads = 128;  // small CTAs: more tile rows in flight per SM
__global__ void __launch_bounds__(kTmThreads) tile_map_bitmap_kernel(MapGeom g, const int32_t* __restrict__ row_ptr,
                                                               const int32_t* __restrict__ col_idx, int split_tau,
                                                               int split_pmax, int32_t* __restrict__ tile_begin,
                                                               int32_t* __restrict__ tile_cnt, int32_t* __restrict__ row_parts,
                                                               int32_t* __restrict__ tile_col,
                                                               uint64_t* __restrict__ tile_member,
                                                               int32_t* __restrict__ head_counts, PlanCountersDev* counters,
                                                               int rows_per_cta) {
    extern __shared__ unsigned long long bm[];  // [slots][nKt]: one membership word per 128-row slot
    __shared__ int32_t warp_cnt[kTmThreads / 32];
    __shared__ int32_t warp_slot_cnt[kTmThreads / 32];
    __shared__ int32_t rp[20];  // CSR offsets of the tile row's logical rows (at most 16 of them, plus the end)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // see organize_kernel
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // A CTA takes `rows_per_cta` consecutive tile rows (1 in every launch today); thread 0 adds the rows' totals up per
    // head before it touches the global counters.
    int acc_head = -1;
    int32_t acc_items = 0, acc_nsplit = 0, acc_slots = 0;
    unsigned long long acc_tiles = 0, acc_slot_tiles = 0;
    auto flush_head = [&]() {
        if (acc_head < 0) return;
        atomicAdd(&head_counts[3 * acc_head + 0], acc_items);
        if (acc_nsplit) {
            atomicAdd(&head_counts[3 * acc_head + 1], acc_nsplit);
            atomicAdd(&head_counts[3 * acc_head + 2], acc_slots);
        }
        acc_items = acc_nsplit = acc_slots = 0;
    };
    for (int q = 0; q < rows_per_cta; ++q) {
    const int trow = blockIdx.x * rows_per_cta + q;
    if (trow >= g.H * g.nQt) break;
    const int h = trow / g.nQt, t = trow % g.nQt;
    // the logical rows this tile row reads: sQ of them (Coarsened or Direct along Q), or one (Refined along Q)
    const int r0 = (g.rq == 1) ? t * g.sQ : t / g.rq;
    const int nr = (g.rq == 1) ? min(g.sQ, g.nQb - r0) : 1;
    if (tid <= nr) rp[tid] = row_ptr[h * g.nQb + r0 + tid];
    for (int i = tid; i < g.nKt * g.slots; i += blockDim.x) bm[i] = 0ull;
    __syncthreads();

    // All entries of the tile row are one contiguous range of the column-index array (its logical rows are adjacent
    // in the block-CSR): one flat loop with four independent loads per thread in flight; the logical row of an entry
    // is the number of row boundaries at or below its index.
    const int32_t e0 = rp[0], e1 = rp[nr];
    int32_t cap_begin;
    if (g.rq == 1) {
        cap_begin = e0 * g.rk;
    } else {
        cap_begin = (e0 * g.rq + (t % g.rq) * (e1 - e0)) * g.rk;
    }
    // Every ratio of the geometry is a power of two: shifts and masks, no integer division in the loop.  A membership
    // bit is set with a 32-bit shared-memory atomic on the half of the 64-bit word it lies in (the 64-bit form is a
    // compare-and-swap loop).
    const int lgSQ128 = 31 - __clz(g.sQ128), lgRK = 31 - __clz(g.rk);
    const bool whole_tile_rows = g.B_Q >= g.T_Q;  // one logical row feeds every slot of the tile row
    unsigned* bm32 = reinterpret_cast<unsigned*>(bm);
    if (g.rq == 1 && g.rk == 1 && nr >= kTmThreads / 32) {
        // At least one logical row per warp: a warp walks whole rows, so the row of an entry (and with it the slot and the
        // sub-row bits) is known without the search below; two loads per lane in flight.
        for (int a = warp; a < nr; a += kTmThreads / 32) {
            const int slot_lo = whole_tile_rows ? 0 : a >> lgSQ128;
            const int slot_hi = whole_tile_rows ? g.slots - 1 : slot_lo;
            const int bit0 = (a & (g.sQ128 - 1)) << g.lgSK;
            const int32_t r1 = rp[a + 1];
            for (int32_t i = rp[a] + lane; i < r1; i += 64) {
                const int32_t ca = col_idx[i];
                const int32_t cb = (i + 32 < r1) ? col_idx[i + 32] : -1;
                for (int sl = slot_lo; sl <= slot_hi; ++sl) {
                    const int wbase = sl * g.nKt;
                    const int ba = bit0 + (ca & (g.sK - 1));
                    atomicOr(&bm32[2 * (wbase + (ca >> g.lgSK)) + (ba >> 5)], 1u << (ba & 31));
                    if (cb >= 0) {
                        const int bb = bit0 + (cb & (g.sK - 1));
                        atomicOr(&bm32[2 * (wbase + (cb >> g.lgSK)) + (bb >> 5)], 1u << (bb & 31));
                    }
                }
            }
        }
    } else
    for (int32_t i0 = e0 + tid; i0 < e1; i0 += 4 * kTmThreads) {
        int32_t c[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) c[u] = (i0 + u * kTmThreads < e1) ? col_idx[i0 + u * kTmThreads] : -1;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            if (c[u] < 0) continue;
            const int32_t i = i0 + u * kTmThreads;
            int a = 0;
            for (int k = 1; k < nr; ++k) a += (i >= rp[k]) ? 1 : 0;
            // which 128-row slot(s) the logical row feeds, and its sub-row inside the slot
            const int slot_lo = whole_tile_rows ? 0 : a >> lgSQ128;
            const int slot_hi = whole_tile_rows ? g.slots - 1 : slot_lo;
            const int arow = (g.rq == 1) ? (a & (g.sQ128 - 1)) : 0;
            for (int sl = slot_lo; sl <= slot_hi; ++sl) {
                const int wbase = sl * g.nKt;
                if (g.rk == 1) {
                    const int bit = (arow << g.lgSK) + (c[u] & (g.sK - 1));
                    atomicOr(&bm32[2 * (wbase + (c[u] >> g.lgSK)) + (bit >> 5)], 1u << (bit & 31));
                } else {
                    for (int k = 0; k < g.rk; ++k) {
                        const int tc = (c[u] << lgRK) + k;
                        if (tc < g.nKt) atomicOr(&bm32[2 * (wbase + tc) + (arow >> 5)], 1u << (arow & 31));
                    }
                }
            }
        }
    }
    __syncthreads();

    // Compaction in column order.  Each warp owns a contiguous range of tile columns: it counts its non-zero words,
    // the warps' counts are exchanged once, and the warp walks its range again to write them out (two block
    // barriers in all, whatever the number of tile columns).
    const int chunk = ((g.nKt + kTmThreads - 1) / kTmThreads) * 32;
    const int c0 = warp * chunk, c1 = min(g.nKt, c0 + chunk);
    int32_t my_cnt = 0, my_slots = 0;
    for (int i0 = c0; i0 < c1; i0 += 32) {
        const int i = i0 + lane;
        const unsigned long long w0 = (i < c1) ? bm[i] : 0ull;
        const unsigned long long w1 = (i < c1 && g.slots == 2) ? bm[g.nKt + i] : 0ull;
        my_cnt += __popc(__ballot_sync(kFull, (w0 | w1) != 0ull));
        my_slots += __popc(__ballot_sync(kFull, w0 != 0ull)) + __popc(__ballot_sync(kFull, w1 != 0ull));
    }
    if (lane == 0) {
        warp_cnt[warp] = my_cnt;
        warp_slot_cnt[warp] = my_slots;
    }
    __syncthreads();
    int32_t before = 0, total = 0, total_slots = 0;
    for (int k = 0; k < kTmThreads / 32; ++k) {
        if (k < warp) before += warp_cnt[k];
        total += warp_cnt[k];
        total_slots += warp_slot_cnt[k];
    }
    int32_t pos0 = cap_begin + before;
    for (int i0 = c0; i0 < c1; i0 += 32) {
        const int i = i0 + lane;
        const unsigned long long w0 = (i < c1) ? bm[i] : 0ull;
        const unsigned long long w1 = (i < c1 && g.slots == 2) ? bm[g.nKt + i] : 0ull;
        const bool any = (w0 | w1) != 0ull;
        const unsigned bits = __ballot_sync(kFull, any);
        if (any) {
            const int32_t pos = pos0 + __popc(bits & ((1u << lane) - 1u));
            tile_col[pos] = i;
            tile_member[(size_t)pos * g.slots] = w0;
            if (g.slots == 2) tile_member[(size_t)pos * 2 + 1] = w1;
        }
        pos0 += __popc(bits);
    }
    if (tid == 0) {
        const int32_t cnt = total;
        tile_begin[trow] = cap_begin;
        tile_cnt[trow] = cnt;
        const int32_t P = split_parts(cnt, split_tau, split_pmax);
        row_parts[trow] = P;
        if (h != acc_head) {
            flush_head();
            acc_head = h;
        }
        acc_items += P;
        if (P > 1) {
            ++acc_nsplit;
            acc_slots += P;
        }
        acc_tiles += (unsigned long long)cnt;
        acc_slot_tiles += (unsigned long long)total_slots;
    }
    __syncthreads();  // the next tile row reuses the shared-memory words and counts
    }  // tile rows of this CTA
    if (tid == 0) {
        flush_head();
        if (acc_tiles) {
            atomicAdd(&counters->ntiles, acc_tiles);
            atomicAdd(&counters->nslot_tiles, acc_slot_tiles);
        }
    }
}

// ------------------------------------------------------------------------------------------
// Tile map for Coarsened tiles with few membership bits (slots * sQ128 * sK <= 16, no Refined dimension) and dense rows: instead of
// one 64-bit word per KV tile column, shared memory holds one BIT PLANE per membership bit (a bitmap over the tile
// columns).  Zeroing and scanning then cost nKt/32 words per plane instead of nKt words, each warp walks whole logical
// rows (so the row of an entry is known without a search), and the output pass assembles a tile's membership word
// from the planes only for the columns that are present.  Same outputs, bit for bit, as tile_map_bitmap_kernel.
// ------------------------------------------------------------------------------------------
constexpr int kTpThreads = 128;
constexpr int kTpMaxWords = 128;  // bitmap words per plane: up to 4096 tile columns
constexpr int kTpMaxPlanes = 16;

__global__ void __launch_bounds__(kTpThreads) tile_map_planes_kernel(MapGeom g, const int32_t* __restrict__ row_ptr,
                                                               const int32_t* __restrict__ col_idx, int split_tau,
                                                               int split_pmax, int32_t* __restrict__ tile_begin,
                                                               int32_t* __restrict__ tile_cnt, int32_t* __restrict__ row_parts,
                                                               int32_t* __restrict__ tile_col,
                                                               uint64_t* __restrict__ tile_member,
                                                               int32_t* __restrict__ head_counts, PlanCountersDev* counters) {
    extern __shared__ uint32_t planes[];  // [nplanes][W], then pres[W], pref[W]
    __shared__ int32_t rp[20];
    __shared__ int32_t wsum[kTpThreads / 32], wslots[kTpThreads / 32];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");  // see organize_kernel
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int W = (g.nKt + 31) >> 5;
    const int bps = g.sQ128 * g.sK;        // membership bits per 128-row slot
    const int nplanes = g.slots * bps;
    uint32_t* pres = planes + nplanes * W;
    uint32_t* pref = pres + W;
    const int trow = blockIdx.x;
    const int h = trow / g.nQt, t = trow % g.nQt;
    const int r0 = t * g.sQ;
    const int nr = min(g.sQ, g.nQb - r0);
    if (tid <= nr) rp[tid] = row_ptr[h * g.nQb + r0 + tid];
    for (int i = tid; i < nplanes * W; i += kTpThreads) planes[i] = 0u;
    __syncthreads();
    const int lgSQ128 = 31 - __clz(g.sQ128);
    // entries: a warp takes whole logical rows, two loads per lane in flight
    for (int a = warp; a < nr; a += kTpThreads / 32) {
        const int plane0 = (a >> lgSQ128) * bps + ((a & (g.sQ128 - 1)) << g.lgSK);
        const int32_t e1 = rp[a + 1];
        for (int32_t i = rp[a] + lane; i < e1; i += 64) {
            const int32_t ca = col_idx[i];
            const int32_t cb = (i + 32 < e1) ? col_idx[i + 32] : -1;
            {
                const int tc = ca >> g.lgSK;
                atomicOr(&planes[(plane0 + (ca & (g.sK - 1))) * W + (tc >> 5)], 1u << (tc & 31));
            }
            if (cb >= 0) {
                const int tc = cb >> g.lgSK;
                atomicOr(&planes[(plane0 + (cb & (g.sK - 1))) * W + (tc >> 5)], 1u << (tc & 31));
            }
        }
    }
    __syncthreads();
    // presence per bitmap word, tile count and non-empty slot count, exclusive prefix of the counts over the words
    uint32_t pw = 0;
    int32_t nslot = 0;
    if (tid < W) {
        for (int sl = 0; sl < g.slots; ++sl) {
            uint32_t ps = 0;
            for (int b = 0; b < bps; ++b) ps |= planes[(sl * bps + b) * W + tid];
            pw |= ps;
            nslot += __popc(ps);
        }
    }
    const int32_t cnt = __popc(pw);
    int32_t incl = cnt, sincl = nslot;
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t x = __shfl_up_sync(kFull, incl, o);
        if (lane >= o) incl += x;
    }
    for (int o = 16; o > 0; o >>= 1) sincl += __shfl_xor_sync(kFull, sincl, o);
    if (lane == 31) wsum[warp] = incl;
    if (lane == 0) wslots[warp] = sincl;
    __syncthreads();
    int32_t before = 0, total = 0, total_slots = 0;
    for (int k = 0; k < kTpThreads / 32; ++k) {
        if (k < warp) before += wsum[k];
        total += wsum[k];
        total_slots += wslots[k];
    }
    if (tid < W) {
        pres[tid] = pw;
        pref[tid] = (uint32_t)(before + incl - cnt);
    }
    __syncthreads();
    // output in column order: a tile column's position is the count of present columns before it
    const int32_t cap_begin = rp[0];  // capacity offset of the tile row (rk == 1: one slot per CSR entry suffices)
    for (int tc = tid; tc < g.nKt; tc += kTpThreads) {
        const int w = tc >> 5, sh = tc & 31;
        const uint32_t pwd = pres[w];
        if (!((pwd >> sh) & 1u)) continue;
        const int32_t pos = cap_begin + (int32_t)pref[w] + __popc(pwd & ((1u << sh) - 1u));
        tile_col[pos] = tc;
        for (int sl = 0; sl < g.slots; ++sl) {
            unsigned long long word = 0ull;
            for (int b = 0; b < bps; ++b) word |= (unsigned long long)((planes[(sl * bps + b) * W + w] >> sh) & 1u) << b;
            tile_member[(size_t)pos * g.slots + sl] = word;
        }
    }
    if (tid == 0) {
        tile_begin[trow] = cap_begin;
        tile_cnt[trow] = total;
        const int32_t P = split_parts(total, split_tau, split_pmax);
        row_parts[trow] = P;
        atomicAdd(&head_counts[3 * h + 0], P);
        if (P > 1) {
            atomicAdd(&head_counts[3 * h + 1], 1);
            atomicAdd(&head_counts[3 * h + 2], P);
        }
        if (total) {
            atomicAdd(&counters->ntiles, (unsigned long long)total);
            atomicAdd(&counters->nslot_tiles, (unsigned long long)total_slots);
        }
    }
}

// ------------------------------------------------------------------------------------------
// organize: one CTA per group of Q tile rows (a head, or all heads for the global order).
//   A. scan the rows' partition counts -> unsorted items (row-major, partition-minor), Split-K
//      row list and workspace slots;
//   B. histogram of item lengths, suffix-summed so longer items come first;
//   C. one warp walks the items in order and assigns each its rank inside its length bucket
//      (stable: ties keep (head, q_tile, part) order), then all threads scatter.
// Shared memory: bins [nKt + 2] then one int per item of the group.
// ------------------------------------------------------------------------------------------
// Histogram size of the sort: one bin per item length, and at least the 64 half-octave buckets.
__host__ __device__ __forceinline__ int organize_bins(const MapGeom& g) { return g.nKt + 2 > 64 ? g.nKt + 2 : 64; }

// Half-octave bucket of an item length (0, 1, 2, 3, 4-5, 6-7, 8-11, 12-15, ...): the bucketed orders sort by it, so
// items of similar length keep their row-major order, and with it the K/V tiles neighbouring Q tiles share.
__host__ __device__ __forceinline__ int32_t length_bucket(int32_t n) {
    if (n <= 1) return n < 0 ? 0 : n;
    int lz = 0;
    while ((n >> (lz + 1)) != 0) ++lz;  // floor(log2 n), n >= 2
    return 2 * lz + ((n >> (lz - 1)) & 1);
}

// Lanes of the warp that hold the same key as this lane (32 shuffles: constant time, unlike match.any).
__device__ __forceinline__ unsigned warp_peers(int32_t k) {
    unsigned m = 0;
#pragma unroll
    for (int l = 0; l < 32; ++l) m |= (__shfl_sync(kFull, k, l) == k ? 1u : 0u) << l;
    return m;
}

__device__ __forceinline__ int32_t block_excl_scan(int32_t v, int32_t* warp_buf, int32_t* total_out) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    int32_t incl = v;
    for (int o = 1; o < 32; o <<= 1) {
        int32_t x = __shfl_up_sync(kFull, incl, o);
        if (lane >= o) incl += x;
    }
    __syncthreads();
    if (lane == 31) warp_buf[warp] = incl;
    __syncthreads();
    int32_t before = 0, total = 0;
    for (int k = 0; k < nw; ++k) {
        const int32_t s = warp_buf[k];
        if (k < warp) before += s;
        total += s;
    }
    *total_out = total;
    return before + incl - v;
}

__global__ void __launch_bounds__(1024) organize_kernel(MapGeom g, int order, int rank_warps_max, int key_cap, int no_split,
                                                         const int32_t* __restrict__ tile_begin,
                                                         const int32_t* __restrict__ tile_cnt,
                                                         const int32_t* __restrict__ row_parts,
                                                         const int32_t* __restrict__ head_counts,
                                                         WorkItem* __restrict__ items_tmp, WorkItem* __restrict__ items,
                                                         SplitRow* __restrict__ split_rows, PlanCountersDev* counters) {
    extern __shared__ int32_t sm[];
    __shared__ int32_t warp_buf[32];
    // Programmatic dependent launch along tile map -> organisation -> attention: a grid lets its successor be
    // scheduled as soon as all of its own CTAs have started, and waits for its predecessor's completion itself before
    // it reads anything (no-ops in ordinary launches).  The successor's launch latency and prologue then overlap.
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int nbins = organize_bins(g);
    const bool bucketed = (order == BSA_ORDER_HEAD_MAJOR_BUCKETS || order == BSA_ORDER_GLOBAL_BUCKETS);
    const bool global_group = (order == BSA_ORDER_GLOBAL_LPT || order == BSA_ORDER_GLOBAL_BUCKETS);
    int32_t* bins = sm;            // [nbins]
    int32_t* key = sm + nbins;     // [items of the group]: length, then rank
    const int tid = threadIdx.x;
    const int grp = blockIdx.x;
    int row0, row1, item_base = 0, split_base = 0, slot_base = 0;
    if (global_group) {
        row0 = 0;
        row1 = g.H * g.nQt;
    } else {
        row0 = grp * g.nQt;
        row1 = row0 + g.nQt;
        for (int hh = 0; hh < grp; ++hh) {
            item_base += head_counts[3 * hh + 0];
            split_base += head_counts[3 * hh + 1];
            slot_base += head_counts[3 * hh + 2];
        }
    }
    for (int i = tid; i < nbins; i += blockDim.x) bins[i] = 0;
    __syncthreads();

    // ---- A: unsorted items ----
    // One pass and one item per row (the common case of a short list under a plan that never splits): the item stays in
    // this thread's registers until it is written to its final place, instead of going through `items_tmp`.
    const bool resident = no_split && (row1 - row0) <= (int)blockDim.x;
    WorkItem mine;
    mine.head = mine.q_tile = mine.tile_begin = mine.tile_end = mine.part = mine.nparts = mine.ws_slot = mine.ntiles = 0;
    int32_t run_items = 0, run_split = 0, run_slots = 0;
    for (int r0 = row0; r0 < row1; r0 += blockDim.x) {
        const int r = r0 + tid;
        int32_t P, tot_i, tot_s = 0, tot_w = 0, off_i, off_s = 0, off_w = 0;
        if (no_split) {  // the plan never splits a row: one item per row, no scans needed
            P = (r < row1) ? 1 : 0;
            off_i = tid;
            tot_i = min((int)blockDim.x, row1 - r0);
        } else {
            P = (r < row1) ? row_parts[r] : 0;
            off_i = block_excl_scan(P, warp_buf, &tot_i);
            off_s = block_excl_scan(P > 1 ? 1 : 0, warp_buf, &tot_s);
            off_w = block_excl_scan(P > 1 ? P : 0, warp_buf, &tot_w);
        }
        if (r < row1) {
            const int32_t tb = tile_begin[r], cnt = tile_cnt[r];
            const int32_t slot = slot_base + run_slots + off_w;
            for (int p = 0; p < P; ++p) {
                WorkItem it;
                it.head = r / g.nQt;
                it.q_tile = r % g.nQt;
                // equal contiguous ranges (the 64-bit division only where a row is split)
                it.tile_begin = (P == 1) ? tb : tb + (int32_t)(((int64_t)cnt * p) / P);
                it.tile_end = (P == 1) ? tb + cnt : tb + (int32_t)(((int64_t)cnt * (p + 1)) / P);
                it.part = p;
                it.nparts = P;
                it.ws_slot = (P > 1) ? (slot + p) * g.slots : -1;  // 128-row workspace slots
                it.ntiles = it.tile_end - it.tile_begin;
                const int32_t li = run_items + off_i + p;
                if (resident)
                    mine = it;  // li == tid
                else
                    items_tmp[item_base + li] = it;
                key[li] = bucketed ? length_bucket(it.ntiles) : it.ntiles;
            }
            if (P > 1) {
                for (int sl = 0; sl < g.slots; ++sl) {
                    SplitRow s;
                    s.head = r / g.nQt;
                    s.q_tile = (r % g.nQt) * g.slots + sl;
                    s.ws_slot = slot * g.slots + sl;
                    s.nparts = P | (g.slots << 16);
                    split_rows[(size_t)(split_base + run_split + off_s) * g.slots + sl] = s;
                }
            }
        }
        run_items += tot_i;
        run_split += tot_s;
        run_slots += tot_w;
    }
    __syncthreads();
    const int32_t n_items = run_items;
    if (order == BSA_ORDER_NATURAL) {  // unsorted: the items stay in (head, q_tile, part) order
        if (resident) {
            if (tid < n_items) items[item_base + tid] = mine;
        } else {
            for (int i = tid; i < n_items; i += blockDim.x) items[item_base + i] = items_tmp[item_base + i];
        }
        if (tid == 0 && grp == gridDim.x - 1) {
            counters->nitems = item_base + n_items;
            counters->nsplit_rows = (split_base + run_split) * g.slots;
            counters->nslots = slot_base + run_slots;
        }
        return;
    }
    // ---- B + C1: stable counting sort by length (longest first; ties keep (head, q_tile, part) order) ----
    // The items are cut into contiguous chunks, one per ranking warp.  Every warp histograms its chunk into a private
    // row; the column sums give the bucket sizes, their suffix sums the bucket starts (longest first), and within a
    // bucket the warps' shares follow in chunk order; every warp then ranks its own chunk in order.  Lanes with equal
    // keys are found with 32 shuffles (warp_peers): `match.any` takes time in proportion to the number of distinct
    // keys in the warp and made this kernel 16 us long on 1024 items.
    int rank_warps = min(rank_warps_max, (n_items + 63) / 64);
    if (rank_warps < 1) rank_warps = 1;
    const int warp = tid >> 5, lane = tid & 31;
    int32_t* whist = key + key_cap;  // [rank_warps][nbins]; one warp alone uses `bins` itself
    int32_t* wb = (rank_warps >= 2) ? whist + warp * nbins : bins;
    const int chunk = (((n_items + rank_warps - 1) / rank_warps) + 31) & ~31;
    const int c0 = warp * chunk, c1 = min(n_items, c0 + chunk);
    if (rank_warps >= 2) {
        for (int i = tid; i < rank_warps * nbins; i += blockDim.x) whist[i] = 0;
        __syncthreads();
    }
    if (warp < rank_warps)
        for (int i = c0 + lane; i < c1; i += 32) atomicAdd(&wb[key[i]], 1);  // this warp's own row
    __syncthreads();
    if (rank_warps >= 2) {
        for (int b = tid; b < nbins; b += blockDim.x) {
            int32_t tot = 0;
            for (int w = 0; w < rank_warps; ++w) tot += whist[w * nbins + b];
            bins[b] = tot;
        }
        __syncthreads();
    }
    // bucket starts, longest first
    if (tid < 32) {
        int32_t carry = 0;
        for (int hi = nbins - 1; hi >= 0; hi -= 32) {
            const int b = hi - tid;
            const int32_t c = (b >= 0) ? bins[b] : 0;
            int32_t incl = c;
            for (int o = 1; o < 32; o <<= 1) {
                int32_t x = __shfl_up_sync(kFull, incl, o);
                if (tid >= o) incl += x;
            }
            if (b >= 0) bins[b] = carry + incl - c;
            carry += __shfl_sync(kFull, incl, 31);
        }
    }
    __syncthreads();
    if (rank_warps >= 2) {
        for (int b = tid; b < nbins; b += blockDim.x) {
            int32_t run = bins[b];
            for (int w = 0; w < rank_warps; ++w) {
                const int32_t c = whist[w * nbins + b];
                whist[w * nbins + b] = run;
                run += c;
            }
        }
        __syncthreads();
    }
    if (warp < rank_warps) {
        for (int i0 = c0; i0 < c1; i0 += 32) {
            const int i = i0 + lane;
            const bool valid = i < c1;
            const int32_t k = valid ? key[i] : -1 - lane;  // invalid lanes get unique keys
            const unsigned peers = warp_peers(k);
            int32_t rank = 0;
            if (valid) rank = wb[k] + __popc(peers & ((1u << lane) - 1u));
            __syncwarp();
            if (valid && (peers >> lane) <= 1u) wb[k] += __popc(peers);  // highest lane of the peer set
            __syncwarp();
            if (valid) key[i] = rank;
        }
    }
    __syncthreads();

    // ---- C2: scatter ----
    if (resident) {
        if (tid < n_items) items[item_base + key[tid]] = mine;
    } else {
        for (int i = tid; i < n_items; i += blockDim.x) items[item_base + key[i]] = items_tmp[item_base + i];
    }

    if (tid == 0) {
        if (global_group) {
            counters->nitems = n_items;
            counters->nsplit_rows = run_split * g.slots;
            counters->nslots = run_slots;
        } else if (grp == gridDim.x - 1) {
            counters->nitems = item_base + n_items;
            counters->nsplit_rows = (split_base + run_split) * g.slots;
            counters->nslots = slot_base + run_slots;
        }
    }
}

// ------------------------------------------------------------------------------------------
// organize, long lists: the global orders over many thousands of Q tile rows (one item per row:
// plans that never split) as a stable counting sort spread over many CTAs, three launches:
//   1. every CTA histograms the sort keys of its 256 consecutive rows;
//   2. one CTA turns the histograms into start positions: bins longest first, and inside a bin
//      the CTAs' shares in row order (so equal keys keep (head, q_tile) order);
//   3. every CTA ranks its rows in order (one warp, 32 rows per step, equal keys found with
//      shuffles) and writes each item straight to its final place.
// ------------------------------------------------------------------------------------------
constexpr int kOrgChunk = 256;  // rows per CTA

__device__ __forceinline__ int32_t organize_key(int32_t ntiles, bool bucketed) {
    return bucketed ? length_bucket(ntiles) : ntiles;
}

__global__ void __launch_bounds__(256) organize_hist_kernel(int nrows, int nbins, int bucketed,
                                                             const int32_t* __restrict__ tile_cnt,
                                                             int32_t* __restrict__ hist /* [chunks][nbins] */) {
    extern __shared__ int32_t sh[];
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");  // launched behind the tile map with programmatic serialisation
    for (int b = threadIdx.x; b < nbins; b += blockDim.x) sh[b] = 0;
    __syncthreads();
    const int r0 = blockIdx.x * kOrgChunk;
    for (int i = threadIdx.x; i < kOrgChunk && r0 + i < nrows; i += blockDim.x)
        atomicAdd(&sh[organize_key(tile_cnt[r0 + i], bucketed != 0)], 1);
    __syncthreads();
    for (int b = threadIdx.x; b < nbins; b += blockDim.x) hist[(size_t)blockIdx.x * nbins + b] = sh[b];
}

__global__ void __launch_bounds__(1024) organize_scan_kernel(int nrows, int nbins, int nchunks, int32_t* __restrict__ hist,
                                                              int32_t* __restrict__ bin_start /* [nbins] scratch */,
                                                              PlanCountersDev* counters) {
    __shared__ int32_t carry_s;
    // per bin: exclusive prefix over the chunks (in place), total into bin_start
    for (int b = threadIdx.x; b < nbins; b += blockDim.x) {
        int32_t run = 0;
        for (int c0 = 0; c0 < nchunks; c0 += 8) {  // eight independent loads in flight, then their running sums
            int32_t v[8];
#pragma unroll
            for (int u = 0; u < 8; ++u) v[u] = (c0 + u < nchunks) ? hist[(size_t)(c0 + u) * nbins + b] : 0;
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                if (c0 + u < nchunks) hist[(size_t)(c0 + u) * nbins + b] = run;
                run += v[u];
            }
        }
        bin_start[b] = run;
    }
    __syncthreads();
    // bin starts, longest first (warp 0 walks the bins from the top, 32 at a time)
    if (threadIdx.x < 32) {
        int32_t carry = 0;
        for (int hi = nbins - 1; hi >= 0; hi -= 32) {
            const int b = hi - (int)threadIdx.x;
            const int32_t c = (b >= 0) ? bin_start[b] : 0;
            int32_t incl = c;
            for (int o = 1; o < 32; o <<= 1) {
                const int32_t x = __shfl_up_sync(kFull, incl, o);
                if ((int)threadIdx.x >= o) incl += x;
            }
            if (b >= 0) bin_start[b] = carry + incl - c;
            carry += __shfl_sync(kFull, incl, 31);
        }
        if (threadIdx.x == 0) carry_s = carry;
    }
    // (the scatter kernel adds a bin's start to its chunk's prefix itself)
    if (threadIdx.x == 0) {
        counters->nitems = nrows;  // one item per row
        counters->nsplit_rows = 0;
        counters->nslots = 0;
        (void)carry_s;
    }
}

__global__ void __launch_bounds__(256) organize_scatter_kernel(MapGeom g, int nrows, int nbins, int bucketed,
                                                                const int32_t* __restrict__ tile_begin,
                                                                const int32_t* __restrict__ tile_cnt,
                                                                const int32_t* __restrict__ hist,
                                                                const int32_t* __restrict__ bin_start,
                                                                WorkItem* __restrict__ items) {
    extern __shared__ int32_t sh[];   // [nbins] next free position per key for this CTA's rows, then [kOrgChunk] ranks
    int32_t* next = sh;
    int32_t* rank = sh + nbins;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    for (int b = threadIdx.x; b < nbins; b += blockDim.x) next[b] = bin_start[b] + hist[(size_t)blockIdx.x * nbins + b];
    __syncthreads();
    const int r0 = blockIdx.x * kOrgChunk;
    const int n = min(kOrgChunk, nrows - r0);
    for (int i = threadIdx.x; i < n; i += blockDim.x) rank[i] = organize_key(tile_cnt[r0 + i], bucketed != 0);  // keys first
    __syncthreads();
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        for (int i0 = 0; i0 < n; i0 += 32) {
            const int i = i0 + lane;
            const bool valid = i < n;
            const int32_t k = valid ? rank[i] : -1 - lane;  // invalid lanes: unique keys
            const unsigned peers = warp_peers(k);
            if (valid) rank[i] = next[k] + __popc(peers & ((1u << lane) - 1u));
            __syncwarp();
            if (valid && (peers >> lane) <= 1u) next[k] += __popc(peers);  // highest lane of the peer set
            __syncwarp();
        }
    }
    __syncthreads();
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
        const int r = r0 + i;
        const int32_t tb = tile_begin[r], cnt = tile_cnt[r];
        int4* dst = reinterpret_cast<int4*>(items + rank[i]);
        dst[0] = make_int4(r / g.nQt, r % g.nQt, tb, tb + cnt);   // head, q_tile, tile_begin, tile_end
        dst[1] = make_int4(0, 1, -1, cnt);                         // part, nparts, ws_slot, ntiles
    }
}

}  // namespace

// Scratch (bytes) the long-list organisation needs in the plan's arena; 0 when the single-kernel path serves.
size_t organize_scratch_bytes(const MapGeom& g, int order, int split_pmax) {
    const bool global_group = (order == BSA_ORDER_GLOBAL_LPT || order == BSA_ORDER_GLOBAL_BUCKETS);
    const long long rows = (long long)g.H * g.nQt;
    if (!global_group || split_pmax > 1 || rows < 4096) return 0;
    const size_t chunks = (size_t)((rows + kOrgChunk - 1) / kOrgChunk);
    return (chunks + 1) * (size_t)organize_bins(g) * sizeof(int32_t);
}

cudaError_t launch_mask_row_stats(const uint8_t* mask, int nrows, int nKb, int32_t* row_nnz, MaskStatsDev* stats,
                                  cudaStream_t stream, MaskStatsHost* post, unsigned seq, bool with_hash) {
    const int rpw = 1;  // rows per warp (4 on large masks was measured slower: fewer, fatter CTAs hide less latency)
    const int grid = (nrows + 8 * rpw - 1) / (8 * rpw);
    if (with_hash)
        mask_row_stats_kernel<true><<<grid, 256, 0, stream>>>(mask, nrows, nKb, row_nnz, stats, post, seq, rpw);
    else
        mask_row_stats_kernel<false><<<grid, 256, 0, stream>>>(mask, nrows, nKb, row_nnz, stats, post, seq, rpw);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_mask_row_stats_packed(const uint32_t* mask, long long stride_words, int nrows, int nKb,
                                         int32_t* row_nnz, MaskStatsDev* stats, cudaStream_t stream, MaskStatsHost* post,
                                         unsigned seq, bool with_hash) {
    if (with_hash)
        mask_row_stats_packed_kernel<true>
            <<<(nrows + 7) / 8, 256, 0, stream>>>(mask, stride_words, nrows, nKb, row_nnz, stats, post, seq);
    else
        mask_row_stats_packed_kernel<false>
            <<<(nrows + 7) / 8, 256, 0, stream>>>(mask, stride_words, nrows, nKb, row_nnz, stats, post, seq);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_csr_fill_packed(const uint32_t* mask, long long stride_words, int nrows, int nKb,
                                   const int32_t* row_ptr, int32_t* col_idx, cudaStream_t stream) {
    csr_fill_packed_kernel<<<(nrows + 7) / 8, 256, 0, stream>>>(mask, stride_words, nrows, nKb, row_ptr, col_idx);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_row_scan(const int32_t* row_nnz, int nrows, int32_t* row_ptr, cudaStream_t stream) {
    row_scan_kernel<<<1, 1024, 0, stream>>>(row_nnz, nrows, row_ptr);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_csr_fill(const uint8_t* mask, int nrows, int nKb, const int32_t* row_ptr, int32_t* col_idx,
                            cudaStream_t stream) {
    csr_fill_kernel<<<(nrows + 7) / 8, 256, 0, stream>>>(mask, nrows, nKb, row_ptr, col_idx);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_tile_map(const MapGeom& g, const int32_t* row_ptr, const int32_t* col_idx, int split_tau,
                            int split_pmax, int32_t* tile_begin, int32_t* tile_cnt, int32_t* row_parts,
                            int32_t* tile_col, uint64_t* tile_member, int32_t* head_counts, PlanCountersDev* counters,
                            cudaStream_t stream, int64_t nnz) {
    if (g.sQ == 1 && g.sK == 1) {  // Direct or Refined in both dimensions: no membership bitmap needed
        tile_map_expand_kernel<<<(g.H * g.nQt + 7) / 8, 256, 0, stream>>>(g, row_ptr, col_idx, split_tau, split_pmax,
                                                                          tile_begin, tile_cnt, row_parts, tile_col,
                                                                          tile_member, head_counts, counters);
        count_launch();
        return cudaGetLastError();
    }
    const int nplanes = g.slots * g.sQ128 * g.sK, words = (g.nKt + 31) / 32;
    // Bit planes pay on dense rows (measured on (32,32) blocks, N = 75600: 3 % density 40 against 41 us, 10 % 71 against
    // 68, 30 % 90 against 109, 60 % 113 against 159): taken from 1536 active blocks per tile row on.
    const bool dense_rows = nnz >= (int64_t)1536 * g.H * g.nQt;
    if (dense_rows && g.rq == 1 && g.rk == 1 && nplanes <= kTpMaxPlanes && words <= kTpMaxWords &&
        !(g.B_Q >= g.T_Q && g.slots > 1)) {
        const size_t psmem = (size_t)(nplanes + 2) * words * sizeof(uint32_t);
        tile_map_planes_kernel<<<g.H * g.nQt, kTpThreads, psmem, stream>>>(g, row_ptr, col_idx, split_tau, split_pmax,
                                                                          tile_begin, tile_cnt, row_parts, tile_col,
                                                                          tile_member, head_counts, counters);
        count_launch();
        return cudaGetLastError();
    }
    const size_t smem = (size_t)g.nKt * g.slots * sizeof(unsigned long long);
    if (smem > 40 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(tile_map_bitmap_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    const int trows = g.H * g.nQt;
    const int rpc = 1;  // tile rows per CTA (4 on long lists was measured slower)
    tile_map_bitmap_kernel<<<(trows + rpc - 1) / rpc, kTmThreads, smem, stream>>>(g, row_ptr, col_idx, split_tau, split_pmax,
                                                                          tile_begin, tile_cnt, row_parts, tile_col,
                                                                          tile_member, head_counts, counters, rpc);
    count_launch();
    return cudaGetLastError();
}

static size_t organize_key_cap(const MapGeom& g, int order, int split_pmax) {
    const bool global_group = (order == BSA_ORDER_GLOBAL_LPT || order == BSA_ORDER_GLOBAL_BUCKETS);
    const size_t rows = global_group ? (size_t)g.H * g.nQt : (size_t)g.nQt;
    return rows * (size_t)(split_pmax < 1 ? 1 : split_pmax);
}

// Minimum (one ranking warp): length histogram + one key per item of a group.
size_t organize_smem_bytes(const MapGeom& g, int order, int split_pmax) {
    return ((size_t)organize_bins(g) + organize_key_cap(g, order, split_pmax)) * sizeof(int32_t);
}

cudaError_t launch_organize(const MapGeom& g, int order, int split_pmax, const int32_t* tile_begin,
                            const int32_t* tile_cnt, const int32_t* row_parts, const int32_t* head_counts,
                            WorkItem* items_tmp, WorkItem* items, SplitRow* split_rows, PlanCountersDev* counters,
                            cudaStream_t stream, int32_t* scratch) {
    if (scratch && organize_scratch_bytes(g, order, split_pmax) > 0) {
        const int nrows = g.H * g.nQt, nbins = organize_bins(g);
        const int nchunks = (nrows + kOrgChunk - 1) / kOrgChunk;
        const int bucketed = (order == BSA_ORDER_GLOBAL_BUCKETS) ? 1 : 0;
        int32_t* hist = scratch;
        int32_t* bin_start = scratch + (size_t)nchunks * nbins;
        const size_t sm1 = (size_t)nbins * sizeof(int32_t), sm3 = (size_t)(nbins + kOrgChunk) * sizeof(int32_t);
        if (sm3 > 40 * 1024) {
            cudaError_t e = cudaFuncSetAttribute(organize_scatter_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm3);
            if (e == cudaSuccess) e = cudaFuncSetAttribute(organize_hist_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sm3);
            if (e != cudaSuccess) return e;
        }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)nchunks);
        cfg.blockDim = dim3(256);
        cfg.dynamicSmemBytes = sm1;
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaError_t e = cudaLaunchKernelEx(&cfg, organize_hist_kernel, nrows, nbins, bucketed, tile_cnt, hist);
        count_launch();
        if (e != cudaSuccess) return e;
        organize_scan_kernel<<<1, 1024, 0, stream>>>(nrows, nbins, nchunks, hist, bin_start, counters);
        count_launch();
        organize_scatter_kernel<<<nchunks, 256, sm3, stream>>>(g, nrows, nbins, bucketed, tile_begin, tile_cnt, hist, bin_start,
                                                               items);
        count_launch();
        return cudaGetLastError();
    }
    // the caller checked organize_smem_bytes() against the device limit when it chose `order`; whatever shared
    // memory is left up to 200 KB holds per-warp histograms for the parallel ranking (up to one per warp)
    const size_t base = organize_smem_bytes(g, order, split_pmax);
    const size_t per_warp = (size_t)organize_bins(g) * sizeof(int32_t);
    const size_t budget = 200 * 1024;
    int rank_warps = base < budget ? (int)((budget - base) / per_warp) : 0;
    if (rank_warps > 32) rank_warps = 32;
    if (rank_warps < 2) rank_warps = 0;
    const size_t smem = base + (size_t)rank_warps * per_warp;
    if (smem > 48 * 1024) {  // the attribute is per device: set it whenever the default limit does not do
        cudaError_t e = cudaFuncSetAttribute(organize_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    const int grid = (order == BSA_ORDER_GLOBAL_LPT || order == BSA_ORDER_GLOBAL_BUCKETS) ? 1 : g.H;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(1024);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const cudaError_t e = cudaLaunchKernelEx(&cfg, organize_kernel, g, order, rank_warps,
                                             (int)organize_key_cap(g, order, split_pmax), split_pmax <= 1 ? 1 : 0, tile_begin,
                                             tile_cnt, row_parts, head_counts, items_tmp, items, split_rows, counters);
    count_launch();
    return e;
}

}  // namespace bsa
