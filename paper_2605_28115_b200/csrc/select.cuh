// Token selection: top-K by fp32 score under a per-region retention floor.
// One thread block per segment; the segment's keys live in shared memory.
//
// Steps (all integer work on the fp32 bit patterns):
//   1. key transform   monotone map fp32 -> uint32, so that unsigned key order equals
//                      IEEE-754 totalOrder on the scores;
//                      the same sweep counts every token's leading digit and, for m = 1, raises
//                      its region's maximum (key, lowest index) with one shared-memory atomic;
//   2. floor           a token is reserved iff fewer than m tokens of its region beat it
//                      (higher key, or equal key and lower index); a reserved token leaves the
//                      digit count again;
//   3. radix select    over the non-reserved tokens, up to 4 passes of 8 bits from the top (the
//                      first pass only scans the counts of step 1):
//                      the key T of the k'-th best (as many leading bits as are needed to tell
//                      it apart) and how many tokens equal to T in those bits are still
//                      needed (k' = k - number reserved);
//   4. mask + scan     keep = reserved | key > T | (key == T and fewer than `need_eq`
//                      equal-keyed non-reserved tokens precede it); destinations come from
//                      a ballot/popc scan in index order, so the output is ascending.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "pdl.cuh"

namespace civic {

// Shape of one segment's selection problem.
struct SegShape {
    int32_t n, t, h, w;
    int32_t region_h, region_w;
    int32_t m;       // floor per region
    int32_t k;       // kept per segment
    int32_t k_fill;  // k - reserved count (>= 0), shape-only
    int32_t floor_slots;  // m == 1 only: number of regions if their maxima get shared-memory slots, else 0
};

// Regions whose maxima may get a shared-memory slot each (8 bytes): beyond that, and where the
// segment leaves no room, the floor walks every region's tile with one thread.
constexpr int kMaxFloorSlots = 8192;

struct SelectParams {
    const float* scores;  // [n_seg, n]
    int32_t* keep_idx;    // [n_seg, k]
    SegShape shape;       // shared by all segments
    // optional fused epilogue: kept positions of the full sequence, see seq_indices_kernel
    int32_t* seq_idx;   // [n_seg, seq_len - n + k] or NULL
    int32_t seq_len, vis_start;
};

// A ragged batch: every block reads its own segment's shape and offsets from the parameters.
constexpr int kMaxRaggedSegs = 64;
struct RaggedParams {
    const float* scores;  // concatenated, segment s starts at score_off[s]
    int32_t* keep_idx;    // concatenated, segment s starts at out_off[s]; segment-local indices
    int32_t* flat_idx;    // same layout, indices over the concatenated scores; or NULL
    SegShape shape[kMaxRaggedSegs];
    int32_t score_off[kMaxRaggedSegs];
    int32_t out_off[kMaxRaggedSegs];
};

__host__ __device__ inline size_t select_smem_bytes(int n, int floor_slots = 0)
{
    const size_t words = (size_t)(n + 31) / 32;
    // one 256-bin histogram per radix pass | per-warp totals (32) | 4 scalars | reserved bit
    // words | keys | (8-byte aligned) one 64-bit slot per region
    const size_t base = (4 * 256 + 32 + 4 + words + words * 32 + 1) / 2 * 2;
    return (base + 2 * (size_t)floor_slots) * sizeof(uint32_t);
}

// floor(a / d) for a, d < 2^16 by one multiplication: with M = floor(2^32 / d) + 1 the product a M
// exceeds a 2^32 / d by less than a / 2^32 < 2^-16 <= 1 / d, which cannot reach the next integer.
struct SmallDivisor {
    uint32_t m;  // 0: divisor 1
    __device__ explicit SmallDivisor(uint32_t d) : m(d <= 1 ? 0u : 0xFFFFFFFFu / d + 1u) {}
    __device__ __forceinline__ uint32_t div(uint32_t a) const { return m ? __umulhi(a, m) : a; }
};

__device__ __forceinline__ uint32_t score_key(float s)
{
    const uint32_t b = __float_as_uint(s);
    return b ^ ((b & 0x80000000u) ? 0xFFFFFFFFu : 0x80000000u);
}

// Cost model: the whole block lives on ONE SM, so the kernel is bound by instruction issue
// (32 warps share 4 schedulers), not by latency.  Everything that need not be done per token
// is done by few threads: the floor with m = 1 by one thread per region, the 256-bin digit
// scan by one warp.
__device__ __forceinline__ void select_block(const SegShape& d, const float* __restrict__ scores,
                                             int32_t* __restrict__ out, int32_t* __restrict__ seq,
                                             int seq_len, int vis_start, int32_t* __restrict__ flat,
                                             int flat_base)
{
    extern __shared__ __align__(16) uint32_t smem[];
    const int n = d.n;
    const int n_words = (n + 31) >> 5;
    const int n_pad = n_words << 5;
    uint32_t* hist = smem;                 // [4][256], one histogram per radix pass
    uint32_t* warp_tot = hist + 4 * 256;   // [32]
    uint32_t* scal = warp_tot + 32;        // [0] chosen digit, [1] rank inside its bin, [2] whole bin wanted
    uint32_t* resv = scal + 4;             // [n_words] bit i%32 of word i/32
    uint32_t* keys = resv + n_words;       // [n_pad]

    const int tid = threadIdx.x, nt = blockDim.x;
    const int lane = tid & 31, warp = tid >> 5, n_warps = nt >> 5;
    release_next_kernel();
    wait_for_prior_kernels();

    const bool fast_floor = d.floor_slots > 0;  // m == 1 and a slot per region
    const bool fill = d.k_fill > 0;
    unsigned long long* slots = reinterpret_cast<unsigned long long*>(smem + ((4 * 256 + 32 + 4 + n_words + n_pad + 1) & ~1));
    const int n_rh = (d.h + d.region_h - 1) / d.region_h, n_rw = (d.w + d.region_w - 1) / d.region_w;
    const int n_reg = d.t * n_rh * n_rw;

    // 0. the first scores are requested before anything else; clear the histograms, the reserved
    // bits and the regions' slots meanwhile
    constexpr int kPre = 4;
    float pre[kPre];
#pragma unroll
    for (int u = 0; u < kPre; ++u) pre[u] = tid + u * nt < n ? __ldg(scores + tid + u * nt) : 0.f;
    for (int b = tid; b < 4 * 256; b += nt) hist[b] = 0u;
    if (tid == 0) warp_tot[0] = 0u;  // OR of (key XOR the first key): the bits in which keys differ (step 1)
    for (int i = tid; i < n_words; i += nt) resv[i] = 0u;
    if (fast_floor)
        for (int r = tid; r < n_reg; r += nt) slots[r] = 0ull;
    __syncthreads();

    // 1. keys; every token is counted under its leading digit (the reserved ones leave again in
    // step 2); with a slot per region the token also raises its region's maximum: key in the upper
    // half, the complement of the index in the lower, so that equal keys go to the lowest index
    const SmallDivisor by_hw((uint32_t)(d.h * d.w)), by_w((uint32_t)d.w);
    const SmallDivisor by_rh((uint32_t)min(d.region_h, d.h)), by_rw((uint32_t)min(d.region_w, d.w));
    const uint32_t key0 = score_key(__ldg(scores));  // n >= 1
    uint32_t differ = 0u;
    auto take = [&](int i, float score) {
        const uint32_t key = i < n ? score_key(score) : 0u;
        keys[i] = key;
        if (i < n) {
            differ |= key ^ key0;
            if (fill) atomicAdd(&hist[key >> 24], 1u);
            if (fast_floor) {
                const uint32_t tt = by_hw.div((uint32_t)i), rem = (uint32_t)i - tt * (uint32_t)(d.h * d.w);
                const uint32_t hh = by_w.div(rem), ww = rem - hh * (uint32_t)d.w;
                const uint32_t r = (tt * (uint32_t)n_rh + by_rh.div(hh)) * (uint32_t)n_rw + by_rw.div(ww);
                atomicMax(&slots[r], ((unsigned long long)key << 32) | (0xFFFFFFFFu - (uint32_t)i));
            }
        }
    };
#pragma unroll
    for (int u = 0; u < kPre; ++u)
        if (tid + u * nt < n_pad) take(tid + u * nt, pre[u]);
    for (int i = tid + kPre * nt; i < n_pad; i += nt) take(i, i < n ? __ldg(scores + i) : 0.f);
    if (fill) {
        differ = __reduce_or_sync(0xFFFFFFFFu, differ);
        if (lane == 0 && differ) atomicOr(&warp_tot[0], differ);
    }
    __syncthreads();

    // 2. floor
    if (fast_floor) {
        for (int r = tid; r < n_reg; r += nt) {
            const unsigned long long top = slots[r];
            const uint32_t best = 0xFFFFFFFFu - (uint32_t)top;
            atomicOr(&resv[best >> 5], 1u << (best & 31));
            if (fill) atomicSub(&hist[(uint32_t)(top >> 56)], 1u);
        }
    } else if (d.m == 1) {
        // one thread per region walks its tile in index order and keeps the first maximum
        for (int r = tid; r < n_reg; r += nt) {
            const int tt = r / (n_rh * n_rw), rem = r - tt * (n_rh * n_rw);
            const int ry = rem / n_rw, rx = rem - ry * n_rw;
            const int h0 = ry * d.region_h, w0 = rx * d.region_w;
            const int h1 = min(h0 + d.region_h, d.h), w1 = min(w0 + d.region_w, d.w);
            int best = (tt * d.h + h0) * d.w + w0;
            uint32_t best_key = keys[best];
            for (int y = h0; y < h1; ++y) {
                const int row = (tt * d.h + y) * d.w;
                for (int x = w0; x < w1; ++x) {
                    const uint32_t key = keys[row + x];
                    if (key > best_key) { best_key = key; best = row + x; }
                }
            }
            atomicOr(&resv[best >> 5], 1u << (best & 31));
            if (fill) atomicSub(&hist[best_key >> 24], 1u);
        }
    } else if (d.m > 1) {
        // general m: a token is reserved iff fewer than m tokens of its tile beat it
        const int hw = d.h * d.w;
        for (int i = tid; i < n_pad; i += nt) {
            bool r = false;
            if (i < n) {
                const int tt = i / hw, rem = i - tt * hw;
                const int hh = rem / d.w, ww = rem - hh * d.w;
                const int h0 = (hh / d.region_h) * d.region_h, w0 = (ww / d.region_w) * d.region_w;
                const int h1 = min(h0 + d.region_h, d.h), w1 = min(w0 + d.region_w, d.w);
                const uint32_t mine = keys[i];
                int better = 0;
                for (int y = h0; y < h1; ++y) {
                    const int row = (tt * d.h + y) * d.w;
                    for (int x = w0; x < w1; ++x) {
                        const int j = row + x;
                        const uint32_t other = keys[j];
                        better += (other > mine) || (other == mine && j < i);
                    }
                }
                r = better < d.m;
                if (r && fill) atomicSub(&hist[mine >> 24], 1u);
            }
            const uint32_t word = __ballot_sync(0xFFFFFFFFu, r);
            if (lane == 0) resv[i >> 5] = word;
        }
    }
    __syncthreads();

    // 3. radix select of the k_fill-th best non-reserved key, 8 bits per pass from the top, down to
    // the lowest bit in which the segment's keys differ at all: the bits below it are the same in
    // every key and decide nothing (scores quantised to a few levels have constant low mantissa
    // bits, whose passes would count every candidate into one bin and sweep the tokens for nothing).
    uint32_t prefix = 0xFFFFFFFFu, mask = 0xFFFFFFFFu, need_eq = 0;
    if (d.k_fill > 0) {
        mask = 0;
        uint32_t rank = (uint32_t)d.k_fill;  // 1-based rank among the candidates still matching
        prefix = 0;
        const uint32_t any_differ = warp_tot[0];
        const int win_lo = any_differ ? __ffs(any_differ) - 1 : 32;  // all keys equal: the leading digit alone
#pragma unroll 1
        for (int pass = 0; pass == 0 || 32 - 8 * pass > win_lo; ++pass) {
            const int shift = pass == 0 ? 24 : max(24 - 8 * pass, win_lo);
            const uint32_t digit_mask = (1u << (32 - 8 * pass - shift)) - 1u;
            uint32_t* h = hist + 256 * pass;
            if (pass > 0) {  // the leading digit was counted in steps 1 and 2
                for (int i = tid; i < n_pad; i += nt) {
                    const uint32_t key = keys[i];
                    const bool cand = i < n && !((resv[i >> 5] >> (i & 31)) & 1u) && (key & mask) == prefix;
                    const uint32_t digit = (key >> shift) & digit_mask;
                    // plain shared-memory atomics: on B200 they measured faster than aggregating
                    // equal digits per warp first (8 ballots + popc, or match.any), even when every
                    // candidate of the block falls into one bin
                    if (cand) atomicAdd(&h[digit], 1u);
                }
                __syncthreads();
            }
            if (warp == 0) {
                // lane l owns bins 8l .. 8l+7; lanes are scanned from the top bin downwards
                const uint4 lo = reinterpret_cast<const uint4*>(h)[2 * lane];
                const uint4 hi = reinterpret_cast<const uint4*>(h)[2 * lane + 1];
                const uint32_t c[8] = {hi.w, hi.z, hi.y, hi.x, lo.w, lo.z, lo.y, lo.x};  // descending bins
                const uint32_t local = c[0] + c[1] + c[2] + c[3] + c[4] + c[5] + c[6] + c[7];
                uint32_t incl = local;  // inclusive sum over lanes >= mine
#pragma unroll
                for (int dist = 1; dist < 32; dist <<= 1) {
                    const uint32_t v = __shfl_down_sync(0xFFFFFFFFu, incl, dist);
                    if (lane + dist < 32) incl += v;
                }
                uint32_t above = incl - local;  // candidates in bins above this lane's
                if (above < rank && rank <= incl) {
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        if (above < rank && rank <= above + c[q]) {
                            scal[0] = 8 * lane + 7 - q;
                            scal[1] = rank - above;
                            scal[2] = rank - above == c[q];  // the whole bin is wanted
                        }
                        above += c[q];
                    }
                }
            }
            __syncthreads();
            prefix |= scal[0] << shift;
            mask |= digit_mask << shift;
            rank = scal[1];
            // Every candidate that still matches the prefix is wanted: the lower bits cannot change
            // the outcome, so the remaining passes are skipped (with continuous scores the bin of
            // the threshold usually holds a single token after two passes).
            if (scal[2]) break;
        }
        need_eq = rank;
    }
    const uint32_t T = prefix;  // compared under `mask`: the key bits decided so far

    // 4. keep mask and ascending destinations.  Each warp owns a contiguous run of 32-token
    // words; pass A counts, pass B places.
    const int words_per_warp = (n_words + n_warps - 1) / n_warps;
    const int w_begin = min(warp * words_per_warp, n_words);
    const int w_end = min(w_begin + words_per_warp, n_words);
    uint32_t sure_cnt = 0, eq_cnt = 0;
    for (int wd = w_begin; wd < w_end; ++wd) {
        const int i = (wd << 5) + lane;
        const uint32_t key = keys[i];
        const bool r = (resv[wd] >> lane) & 1u;
        const bool sure = i < n && (r || (d.k_fill > 0 && (key & mask) > T));
        const bool eq = i < n && !r && d.k_fill > 0 && (key & mask) == T;
        sure_cnt += __popc(__ballot_sync(0xFFFFFFFFu, sure));
        eq_cnt += __popc(__ballot_sync(0xFFFFFFFFu, eq));
    }
    if (lane == 0) warp_tot[warp] = (eq_cnt << 16) | sure_cnt;  // n <= 65535 per field
    __syncthreads();
    uint32_t base = (lane < warp) ? warp_tot[lane] : 0u;  // n_warps <= 32
#pragma unroll
    for (int dist = 16; dist > 0; dist >>= 1) base += __shfl_xor_sync(0xFFFFFFFFu, base, dist);
    uint32_t sure_before = base & 0xFFFFu, eq_before = base >> 16;
    const uint32_t lt = (1u << lane) - 1u;
    for (int wd = w_begin; wd < w_end; ++wd) {
        const int i = (wd << 5) + lane;
        const uint32_t key = keys[i];
        const bool r = (resv[wd] >> lane) & 1u;
        const bool sure = i < n && (r || (d.k_fill > 0 && (key & mask) > T));
        const bool eq = i < n && !r && d.k_fill > 0 && (key & mask) == T;
        const uint32_t sb = __ballot_sync(0xFFFFFFFFu, sure), eb = __ballot_sync(0xFFFFFFFFu, eq);
        const uint32_t my_eq_before = eq_before + __popc(eb & lt);
        const uint32_t my_sure_before = sure_before + __popc(sb & lt);
        if (sure || (eq && my_eq_before < need_eq)) {
            const uint32_t j = my_sure_before + min(my_eq_before, need_eq);
            out[j] = i;
            if (seq) seq[vis_start + j] = vis_start + i;
            if (flat) flat[j] = flat_base + i;
        }
        sure_before += __popc(sb);
        eq_before += __popc(eb);
    }
    // fused sequence indices: text in front of the visual span keeps its positions, text
    // behind it moves up by the n - k dropped visual tokens
    if (seq) {
        for (int j = tid; j < vis_start; j += nt) seq[j] = j;
        const int s_out = seq_len - n + d.k;
        for (int j = vis_start + d.k + tid; j < s_out; j += nt) seq[j] = j - d.k + n;
    }
}

__global__ void __launch_bounds__(1024) select_kernel(const __grid_constant__ SelectParams p)
{
    const SegShape& d = p.shape;
    int32_t* seq = p.seq_idx ? p.seq_idx + (size_t)blockIdx.x * (p.seq_len - d.n + d.k) : nullptr;
    select_block(d, p.scores + (size_t)blockIdx.x * d.n, p.keep_idx + (size_t)blockIdx.x * d.k, seq,
                 p.seq_len, p.vis_start, nullptr, 0);
}

__global__ void __launch_bounds__(1024) select_ragged_kernel(const __grid_constant__ RaggedParams p)
{
    const SegShape& d = p.shape[blockIdx.x];
    const int32_t out_off = p.out_off[blockIdx.x], score_off = p.score_off[blockIdx.x];
    select_block(d, p.scores + score_off, p.keep_idx + out_off, nullptr, 0, 0,
                 p.flat_idx ? p.flat_idx + out_off : nullptr, score_off);
}

// seq_idx[s, :] = text positions before the visual span, vis_start + kept visual indices,
// text positions behind the span.
__global__ void seq_indices_kernel(const int32_t* __restrict__ keep_idx, int32_t* __restrict__ seq_idx,
                                   int n_seq, int k, int vis_start, int n_vis, int s_out)
{
    release_next_kernel();
    wait_for_prior_kernels();
    const long long total = (long long)n_seq * s_out;
    for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < total;
         e += (long long)gridDim.x * blockDim.x) {
        const int s = (int)(e / s_out), j = (int)(e - (long long)s * s_out);
        int32_t v;
        if (j < vis_start) v = j;
        else if (j < vis_start + k) v = vis_start + keep_idx[(size_t)s * k + (j - vis_start)];
        else v = j - k + n_vis;
        seq_idx[e] = v;
    }
}

}  // namespace civic
