// Token selection for segments too large for one thread block (long videos): the same result as
// select_kernel, computed by many blocks per segment over five launches that meet at global
// scratch memory.  No block ever waits for another block: every grid-wide dependency is a
// kernel boundary.
//
//   chunks     a block owns a chunk = some consecutive "region rows" (all tiles of region_h
//              consecutive token rows of one temporal slice), a contiguous token range that
//              contains only whole tiles, so the retention floor is decided inside the block;
//   K1 floor   keys of the chunk in shared memory -> reserved flags (one byte per token, global)
//              and the histogram of the top 11 key bits of the non-reserved tokens;
//   K2, K3     radix select, 11 + 11 + 10 bits from the top: every block scans the finished
//              global histogram of the previous digit (2048 bins, one block-wide suffix scan),
//              then histograms the next digit of the tokens still matching the prefix;
//   K4 count   the last scan gives the threshold key T and the number `need_eq` of tokens equal
//              to T still wanted; every block counts its sure and its equal tokens;
//   K5 place   a block sums the counts of the chunks before it and writes its kept tokens in
//              index order, splitting the equal-keyed ones by index.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "pdl.cuh"
#include "select.cuh"

namespace civic {

constexpr int kLargeThreads = 1024;
constexpr int kLargeMaxChunk = 16384;  // tokens per block: 64 KB of keys in shared memory
constexpr int kLargeBins = 2048;       // bins of the widest digit (11 bits)
constexpr int kLargeSelWords = 16;     // per-segment scalars kept between the launches

struct LargeParams {
    const float* scores;  // [n_seg, n]
    int32_t* keep_idx;    // [n_seg, k]
    int32_t n, t, h, w;
    int32_t region_h, region_w;
    int32_t m, k, k_fill;
    int32_t n_rh;            // region rows per temporal slice
    int32_t rows_per_chunk;  // region rows per block
    int32_t n_chunks;        // blocks per segment
    // scratch, all per segment
    uint32_t* hist;    // [n_seg][3][kLargeBins]
    uint32_t* sel;     // [n_seg][kLargeSelWords]: {digit0, rank1, digit1, rank2, T, need_eq}
    uint32_t* counts;  // [n_seg][n_chunks][2]: sure, equal
    uint8_t* flags;    // [n_seg][n]: 1 = reserved by the floor
};

// Token range [tok0, tok1) of a chunk: region rows [chunk * rows_per_chunk, ...) laid end to end.
__device__ __forceinline__ int region_row_start(const LargeParams& p, int g)
{
    const int tt = g / p.n_rh, ry = g - tt * p.n_rh;
    return tt * p.h * p.w + ry * p.region_h * p.w;  // g == t * n_rh gives n
}

__device__ __forceinline__ void chunk_range(const LargeParams& p, int chunk, int& g0, int& g1, int& tok0,
                                            int& tok1)
{
    g0 = min(chunk * p.rows_per_chunk, p.t * p.n_rh);  // a block past the last region row gets nothing
    g1 = min(g0 + p.rows_per_chunk, p.t * p.n_rh);
    tok0 = region_row_start(p, g0);
    tok1 = region_row_start(p, g1);
}

// Block-wide search of a finished histogram: the bin (counted from the top) that holds the
// rank-th candidate, and the rank inside that bin.  Every thread returns the same pair.
// `tmp` is 34 words of shared memory.
// Thread `tid` brings the counts of bins 2*tid and 2*tid+1 (0 beyond the histogram).
__device__ __forceinline__ void find_digit_counts(uint32_t c_lo, uint32_t c_hi, uint32_t rank, uint32_t* tmp,
                                                  uint32_t& digit, uint32_t& rank_in_bin)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const uint32_t local = c_lo + c_hi;
    uint32_t incl = local;  // sum over the threads >= mine of my warp
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t v = __shfl_down_sync(0xFFFFFFFFu, incl, d);
        if (lane + d < 32) incl += v;
    }
    if (lane == 0) tmp[warp] = incl;
    __syncthreads();
    uint32_t higher = 0;  // candidates in the warps above mine
    for (int wv = warp + 1; wv < kLargeThreads / 32; ++wv) higher += tmp[wv];
    const uint32_t above_hi = higher + incl - local;  // candidates in bins above 2*tid+1
    const uint32_t above_lo = above_hi + c_hi;
    if (above_hi < rank && rank <= above_hi + c_hi) { tmp[32] = 2 * tid + 1; tmp[33] = rank - above_hi; }
    if (above_lo < rank && rank <= above_lo + c_lo) { tmp[32] = 2 * tid; tmp[33] = rank - above_lo; }
    __syncthreads();
    digit = tmp[32];
    rank_in_bin = tmp[33];
    __syncthreads();
}

__device__ __forceinline__ void find_digit(const uint32_t* __restrict__ ghist, int bins, uint32_t rank,
                                           uint32_t* tmp, uint32_t& digit, uint32_t& rank_in_bin)
{
    const int tid = threadIdx.x;
    find_digit_counts(2 * tid < bins ? ghist[2 * tid] : 0u, 2 * tid + 1 < bins ? ghist[2 * tid + 1] : 0u, rank, tmp,
                      digit, rank_in_bin);
}

// Adds a block's shared-memory histogram to the segment's global one.
__device__ __forceinline__ void flush_hist(uint32_t* shist, uint32_t* ghist, int bins)
{
    for (int b = threadIdx.x; b < bins; b += blockDim.x) {
        const uint32_t c = shist[b];
        if (c) atomicAdd(&ghist[b], c);
    }
}

// The retention floor inside one chunk: bit i of `resv` (zeroed by the caller) is set for the
// reserved tokens; `keys` holds the chunk's keys.  Whole tiles only, by the choice of the chunks.
__device__ __forceinline__ void chunk_floor(const LargeParams& p, const uint32_t* keys, uint32_t* resv, int g0, int g1,
                                            int tok0, int cn, int cn_pad)
{
    const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31;
    const int n_rw = (p.w + p.region_w - 1) / p.region_w;
    if (p.m == 1) {
        // one thread per tile walks it in index order and keeps the first maximum
        const int n_reg = (g1 - g0) * n_rw;
        for (int r = tid; r < n_reg; r += nt) {
            const int g = g0 + r / n_rw, rx = r - (r / n_rw) * n_rw;
            const int ry = g % p.n_rh;
            const int rows = min(p.region_h, p.h - ry * p.region_h);
            const int base = region_row_start(p, g) - tok0;  // chunk-local index of the tile row
            const int w0 = rx * p.region_w, w1 = min(w0 + p.region_w, p.w);
            int best = base + w0;
            uint32_t best_key = keys[best];
            for (int y = 0; y < rows; ++y)
                for (int x = w0; x < w1; ++x) {
                    const uint32_t key = keys[base + y * p.w + x];
                    if (key > best_key) { best_key = key; best = base + y * p.w + x; }
                }
            atomicOr(&resv[best >> 5], 1u << (best & 31));
        }
    } else if (p.m > 1) {
        // a token is reserved iff fewer than m tokens of its tile beat it
        for (int i = tid; i < cn_pad; i += nt) {
            bool r = false;
            if (i < cn) {
                // region row of token i: region rows have region_h * w tokens except the last of a slice
                const int tok = tok0 + i;
                const int tt = tok / (p.h * p.w), in_slice = tok - tt * p.h * p.w;
                const int hh = in_slice / p.w, ww = in_slice - hh * p.w;
                const int h0 = (hh / p.region_h) * p.region_h, h1 = min(h0 + p.region_h, p.h);
                const int w0 = (ww / p.region_w) * p.region_w, w1 = min(w0 + p.region_w, p.w);
                const uint32_t mine = keys[i];
                int better = 0;
                for (int y = h0; y < h1; ++y) {
                    const int row = (tt * p.h + y) * p.w - tok0;
                    for (int x = w0; x < w1; ++x) {
                        const int j = row + x;
                        const uint32_t other = keys[j];
                        better += (other > mine) || (other == mine && j < i);
                    }
                }
                r = better < p.m;
            }
            const uint32_t word = __ballot_sync(0xFFFFFFFFu, r);
            if (lane == 0) resv[i >> 5] = word;
        }
    }
}

// K1: floor + histogram of key bits 31..21.
__global__ void __launch_bounds__(kLargeThreads) large_floor_kernel(const __grid_constant__ LargeParams p)
{
    extern __shared__ __align__(16) uint32_t smem[];
    uint32_t* shist = smem;                       // [kLargeBins]
    uint32_t* resv = shist + kLargeBins;          // [kLargeMaxChunk / 32] bit per chunk-local token
    uint32_t* keys = resv + kLargeMaxChunk / 32;  // [chunk tokens]
    const int tid = threadIdx.x, nt = blockDim.x;
    const int seg = blockIdx.x / p.n_chunks, chunk = blockIdx.x - seg * p.n_chunks;
    int g0, g1, tok0, tok1;
    chunk_range(p, chunk, g0, g1, tok0, tok1);
    const int cn = tok1 - tok0, cn_pad = (cn + 31) & ~31;
    const float* scores = p.scores + (size_t)seg * p.n + tok0;
    release_next_kernel();
    wait_for_prior_kernels();

    for (int i = tid; i < cn_pad; i += nt) keys[i] = i < cn ? score_key(__ldg(scores + i)) : 0u;
    for (int b = tid; b < kLargeBins; b += nt) shist[b] = 0u;
    for (int i = tid; i < kLargeMaxChunk / 32; i += nt) resv[i] = 0u;
    __syncthreads();

    chunk_floor(p, keys, resv, g0, g1, tok0, cn, cn_pad);
    __syncthreads();

    uint8_t* flags = p.flags + (size_t)seg * p.n + tok0;
    for (int i = tid; i < cn; i += nt) {
        const bool r = (resv[i >> 5] >> (i & 31)) & 1u;
        flags[i] = r ? 1 : 0;
        if (!r && p.k_fill > 0) atomicAdd(&shist[keys[i] >> 21], 1u);
    }
    __syncthreads();
    if (p.k_fill > 0) flush_hist(shist, p.hist + (size_t)seg * 3 * kLargeBins, kLargeBins);
}

// K2 (PASS 1) and K3 (PASS 2): finish the previous digit, histogram the next one.
template <int PASS>
__global__ void __launch_bounds__(kLargeThreads) large_hist_kernel(const __grid_constant__ LargeParams p)
{
    __shared__ uint32_t shist[kLargeBins];
    __shared__ uint32_t tmp[34];
    const int tid = threadIdx.x, nt = blockDim.x;
    const int seg = blockIdx.x / p.n_chunks, chunk = blockIdx.x - seg * p.n_chunks;
    int g0, g1, tok0, tok1;
    chunk_range(p, chunk, g0, g1, tok0, tok1);
    release_next_kernel();
    wait_for_prior_kernels();
    if (p.k_fill <= 0) return;
    uint32_t* sel = p.sel + (size_t)seg * kLargeSelWords;
    const uint32_t* ghist = p.hist + ((size_t)seg * 3 + (PASS - 1)) * kLargeBins;
    for (int b = tid; b < kLargeBins; b += nt) shist[b] = 0u;
    uint32_t digit, rank;
    const uint32_t rank_in = PASS == 1 ? (uint32_t)p.k_fill : sel[1];
    find_digit(ghist, kLargeBins, rank_in, tmp, digit, rank);  // its barriers also cover shist
    if (chunk == 0 && tid == 0) { sel[2 * (PASS - 1)] = digit; sel[2 * (PASS - 1) + 1] = rank; }
    // key bits that must match so far, and the digit to count
    const uint32_t prefix = PASS == 1 ? digit : ((sel[0] << 11) | digit);
    constexpr int kPrefixShift = PASS == 1 ? 21 : 10;
    const float* scores = p.scores + (size_t)seg * p.n;
    const uint8_t* flags = p.flags + (size_t)seg * p.n;
    for (int i = tok0 + tid; i < tok1; i += nt) {
        const uint32_t key = score_key(__ldg(scores + i));
        if (!flags[i] && (key >> kPrefixShift) == prefix)
            atomicAdd(&shist[PASS == 1 ? (key >> 10) & 0x7FFu : key & 0x3FFu], 1u);
    }
    __syncthreads();
    flush_hist(shist, p.hist + ((size_t)seg * 3 + PASS) * kLargeBins, PASS == 1 ? 2048 : 1024);
}

// Keep decision of one token once T and need_eq are known.
__device__ __forceinline__ void classify(const LargeParams& p, uint32_t key, bool reserved, uint32_t T,
                                         bool& sure, bool& eq)
{
    sure = reserved || (p.k_fill > 0 && key > T);
    eq = !reserved && p.k_fill > 0 && key == T;
}

// K4: threshold from the last histogram; per-chunk counts of sure and equal tokens.
__global__ void __launch_bounds__(kLargeThreads) large_count_kernel(const __grid_constant__ LargeParams p)
{
    __shared__ uint32_t tmp[34];
    __shared__ uint32_t tot[2];
    const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31;
    const int seg = blockIdx.x / p.n_chunks, chunk = blockIdx.x - seg * p.n_chunks;
    int g0, g1, tok0, tok1;
    chunk_range(p, chunk, g0, g1, tok0, tok1);
    release_next_kernel();
    wait_for_prior_kernels();
    uint32_t* sel = p.sel + (size_t)seg * kLargeSelWords;
    uint32_t T = 0xFFFFFFFFu, need_eq = 0;
    if (p.k_fill > 0) {
        uint32_t digit, rank;
        find_digit(p.hist + ((size_t)seg * 3 + 2) * kLargeBins, 1024, sel[3], tmp, digit, rank);
        T = (sel[0] << 21) | (sel[2] << 10) | digit;
        need_eq = rank;
    }
    if (tid < 2) tot[tid] = 0u;
    __syncthreads();
    if (chunk == 0 && tid == 0) { sel[4] = T; sel[5] = need_eq; }
    const float* scores = p.scores + (size_t)seg * p.n;
    const uint8_t* flags = p.flags + (size_t)seg * p.n;
    uint32_t sure_cnt = 0, eq_cnt = 0;
    for (int i0 = tok0 + (tid & ~31); i0 < tok1; i0 += nt) {
        const int i = i0 + lane;
        bool sure = false, eq = false;
        if (i < tok1) classify(p, score_key(__ldg(scores + i)), flags[i] != 0, T, sure, eq);
        sure_cnt += __popc(__ballot_sync(0xFFFFFFFFu, sure));
        eq_cnt += __popc(__ballot_sync(0xFFFFFFFFu, eq));
    }
    if (lane == 0) { atomicAdd(&tot[0], sure_cnt); atomicAdd(&tot[1], eq_cnt); }
    __syncthreads();
    if (tid < 2) p.counts[((size_t)seg * p.n_chunks + chunk) * 2 + tid] = tot[tid];
}

// K5: destinations in index order.
__global__ void __launch_bounds__(kLargeThreads) large_place_kernel(const __grid_constant__ LargeParams p)
{
    __shared__ uint32_t warp_sure[kLargeThreads / 32], warp_eq[kLargeThreads / 32];
    __shared__ uint32_t base[2];
    const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, n_warps = nt >> 5;
    const int seg = blockIdx.x / p.n_chunks, chunk = blockIdx.x - seg * p.n_chunks;
    int g0, g1, tok0, tok1;
    chunk_range(p, chunk, g0, g1, tok0, tok1);
    release_next_kernel();
    wait_for_prior_kernels();
    const uint32_t* sel = p.sel + (size_t)seg * kLargeSelWords;
    const uint32_t T = sel[4], need_eq = sel[5];
    if (tid < 2) base[tid] = 0u;
    __syncthreads();
    {   // kept / equal tokens in the chunks before this one
        const uint32_t* counts = p.counts + (size_t)seg * p.n_chunks * 2;
        uint32_t s = 0, e = 0;
        for (int c = tid; c < chunk; c += nt) { s += counts[2 * c]; e += counts[2 * c + 1]; }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            s += __shfl_xor_sync(0xFFFFFFFFu, s, d);
            e += __shfl_xor_sync(0xFFFFFFFFu, e, d);
        }
        if (lane == 0 && (s | e)) { atomicAdd(&base[0], s); atomicAdd(&base[1], e); }
    }
    const float* scores = p.scores + (size_t)seg * p.n;
    const uint8_t* flags = p.flags + (size_t)seg * p.n;
    int32_t* out = p.keep_idx + (size_t)seg * p.k;
    // each warp owns a contiguous run of 32-token words of the chunk: count, scan, place
    const int n_words = (tok1 - tok0 + 31) >> 5;
    const int words_per_warp = (n_words + n_warps - 1) / n_warps;
    const int w_begin = min(warp * words_per_warp, n_words), w_end = min(w_begin + words_per_warp, n_words);
    uint32_t sure_cnt = 0, eq_cnt = 0;
    for (int wd = w_begin; wd < w_end; ++wd) {
        const int i = tok0 + (wd << 5) + lane;
        bool sure = false, eq = false;
        if (i < tok1) classify(p, score_key(__ldg(scores + i)), flags[i] != 0, T, sure, eq);
        sure_cnt += __popc(__ballot_sync(0xFFFFFFFFu, sure));
        eq_cnt += __popc(__ballot_sync(0xFFFFFFFFu, eq));
    }
    if (lane == 0) { warp_sure[warp] = sure_cnt; warp_eq[warp] = eq_cnt; }
    __syncthreads();
    uint32_t sure_before = (lane < warp) ? warp_sure[lane] : 0u;  // n_warps <= 32
    uint32_t eq_before = (lane < warp) ? warp_eq[lane] : 0u;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        sure_before += __shfl_xor_sync(0xFFFFFFFFu, sure_before, d);
        eq_before += __shfl_xor_sync(0xFFFFFFFFu, eq_before, d);
    }
    sure_before += base[0];
    eq_before += base[1];
    const uint32_t lt = (1u << lane) - 1u;
    for (int wd = w_begin; wd < w_end; ++wd) {
        const int i = tok0 + (wd << 5) + lane;
        bool sure = false, eq = false;
        if (i < tok1) classify(p, score_key(__ldg(scores + i)), flags[i] != 0, T, sure, eq);
        const uint32_t sb = __ballot_sync(0xFFFFFFFFu, sure), eb = __ballot_sync(0xFFFFFFFFu, eq);
        const uint32_t my_eq_before = eq_before + __popc(eb & lt);
        const uint32_t my_sure_before = sure_before + __popc(sb & lt);
        if (sure || (eq && my_eq_before < need_eq)) {
            const uint32_t j = my_sure_before + min(my_eq_before, need_eq);
            if (j < (uint32_t)p.k) out[j] = i;  // always true when the counts are consistent
        }
        sure_before += __popc(sb);
        eq_before += __popc(eb);
    }
}

}  // namespace civic
