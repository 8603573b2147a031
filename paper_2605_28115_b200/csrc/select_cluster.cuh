// Token selection for a segment beyond one thread block, in ONE launch: a thread-block cluster
// per segment.  Same result as select_kernel and as the five launches of select_large.cuh.
//
// The blocks of a cluster split the segment into chunks of whole region rows (as in
// select_large.cuh), each keeps the keys of its chunk in its own shared memory for the whole
// kernel, and the blocks meet at the hardware cluster barrier:
//   floor      decided inside the block; histogram of key bits 31..21 of the non-reserved tokens
//   ---- barrier; every block adds up the cluster's histograms over distributed shared memory
//        and finds the digit itself (all blocks get the same answer, nothing is broadcast)
//   bits 20..10, then bits 9..0 the same way: two more barriers
//   count      the threshold key T and the number of tokens equal to T still wanted are known;
//              every block counts its sure and its equal tokens
//   ---- barrier; a block reads the counts of the blocks before it
//   place      kept tokens written in index order, the equal-keyed ones split by index
//   ---- barrier: no block leaves while another may still read its shared memory
// Every block of a cluster runs every barrier, whatever its chunk holds (it may be empty).
#pragma once
#include "select_large.cuh"

namespace civic {

constexpr int kClusterThreads = 1024;
constexpr int kClusterBlocks = 4;        // blocks per cluster (clusters of 8 measured 8 us slower per call:
                                         // twice the remote histogram reads and a wider barrier)
constexpr int kClusterMaxChunk = 16384;  // tokens per block: 64 KB of keys in shared memory

__host__ __device__ constexpr size_t select_cluster_smem_bytes(int chunk_tokens)
{
    return (size_t)(3 * kLargeBins + kClusterMaxChunk / 32 + ((chunk_tokens + 31) & ~31)) * 4;
}

__device__ __forceinline__ void cluster_barrier()  // all threads of all blocks of the cluster
{
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// word at the same shared-memory offset in block `rank` of the cluster
__device__ __forceinline__ uint32_t peer_shared_u32(const uint32_t* mine, uint32_t rank)
{
    uint32_t remote, v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;"
                 : "=r"(remote) : "r"((uint32_t)__cvta_generic_to_shared(mine)), "r"(rank));
    asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(remote) : "memory");
    return v;
}

// p.n_chunks = blocks per cluster (grid = n_seg clusters); p.hist, p.sel, p.counts, p.flags unused.
__global__ void __launch_bounds__(kClusterThreads) select_cluster_kernel(const __grid_constant__ LargeParams p)
{
    extern __shared__ __align__(16) uint32_t smem[];
    uint32_t* hist = smem;                          // [3][kLargeBins]: digits of 11, 11 and 10 bits
    uint32_t* resv = hist + 3 * kLargeBins;         // [kClusterMaxChunk / 32] bit per chunk-local token
    uint32_t* keys = resv + kClusterMaxChunk / 32;  // [chunk tokens]
    __shared__ uint32_t tmp[34];
    __shared__ uint32_t tot[2];  // sure and equal tokens of this chunk; read by the later blocks
    __shared__ uint32_t warp_sure[kClusterThreads / 32], warp_eq[kClusterThreads / 32];
    const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5, n_warps = nt >> 5;
    const int n_blocks = p.n_chunks;
    const int seg = blockIdx.x / n_blocks, chunk = blockIdx.x - seg * n_blocks;  // chunk = rank in the cluster
    int g0, g1, tok0, tok1;
    chunk_range(p, chunk, g0, g1, tok0, tok1);
    const int cn = tok1 - tok0, cn_pad = (cn + 31) & ~31;
    const float* scores = p.scores + (size_t)seg * p.n + tok0;
    release_next_kernel();
    wait_for_prior_kernels();

    for (int i = tid; i < cn_pad; i += nt) keys[i] = i < cn ? score_key(__ldg(scores + i)) : 0u;
    for (int b = tid; b < 3 * kLargeBins; b += nt) hist[b] = 0u;
    for (int i = tid; i < kClusterMaxChunk / 32; i += nt) resv[i] = 0u;
    if (tid < 2) tot[tid] = 0u;
    __syncthreads();
    chunk_floor(p, keys, resv, g0, g1, tok0, cn, cn_pad);
    __syncthreads();
    auto reserved = [&](int i) { return ((resv[i >> 5] >> (i & 31)) & 1u) != 0; };
    // counts of bins 2 * tid and 2 * tid + 1 of digit `which`, over the whole cluster
    auto cluster_bins = [&](int which, int bins, uint32_t& c_lo, uint32_t& c_hi) {
        c_lo = c_hi = 0u;
        if (2 * tid < bins)
            for (int r = 0; r < n_blocks; ++r) {
                c_lo += peer_shared_u32(hist + which * kLargeBins + 2 * tid, (uint32_t)r);
                c_hi += peer_shared_u32(hist + which * kLargeBins + 2 * tid + 1, (uint32_t)r);
            }
    };

    const bool fill = p.k_fill > 0;
    if (fill)
        for (int i = tid; i < cn; i += nt)
            if (!reserved(i)) atomicAdd(&hist[keys[i] >> 21], 1u);
    cluster_barrier();
    uint32_t d0 = 0, d1 = 0, rank = 0, c_lo, c_hi;
    if (fill) {
        cluster_bins(0, kLargeBins, c_lo, c_hi);
        find_digit_counts(c_lo, c_hi, (uint32_t)p.k_fill, tmp, d0, rank);
        for (int i = tid; i < cn; i += nt)
            if (!reserved(i) && (keys[i] >> 21) == d0) atomicAdd(&hist[kLargeBins + ((keys[i] >> 10) & 0x7FFu)], 1u);
    }
    cluster_barrier();
    if (fill) {
        cluster_bins(1, kLargeBins, c_lo, c_hi);
        find_digit_counts(c_lo, c_hi, rank, tmp, d1, rank);
        const uint32_t prefix = (d0 << 11) | d1;
        for (int i = tid; i < cn; i += nt)
            if (!reserved(i) && (keys[i] >> 10) == prefix) atomicAdd(&hist[2 * kLargeBins + (keys[i] & 0x3FFu)], 1u);
    }
    cluster_barrier();
    uint32_t T = 0xFFFFFFFFu, need_eq = 0;
    if (fill) {
        uint32_t d2;
        cluster_bins(2, 1024, c_lo, c_hi);
        find_digit_counts(c_lo, c_hi, rank, tmp, d2, need_eq);
        T = (d0 << 21) | (d1 << 10) | d2;
    }

    // each warp owns a contiguous run of 32-token words of the chunk: count, scan, place
    const int n_words = cn_pad >> 5;
    const int words_per_warp = (n_words + n_warps - 1) / n_warps;
    const int w_begin = min(warp * words_per_warp, n_words), w_end = min(w_begin + words_per_warp, n_words);
    uint32_t sure_cnt = 0, eq_cnt = 0;
    for (int wd = w_begin; wd < w_end; ++wd) {
        const int i = (wd << 5) + lane;
        bool sure = false, eq = false;
        if (i < cn) classify(p, keys[i], reserved(i), T, sure, eq);
        sure_cnt += __popc(__ballot_sync(0xFFFFFFFFu, sure));
        eq_cnt += __popc(__ballot_sync(0xFFFFFFFFu, eq));
    }
    if (lane == 0) {
        warp_sure[warp] = sure_cnt;
        warp_eq[warp] = eq_cnt;
        if (sure_cnt | eq_cnt) { atomicAdd(&tot[0], sure_cnt); atomicAdd(&tot[1], eq_cnt); }
    }
    cluster_barrier();
    uint32_t sure_before = (lane < warp) ? warp_sure[lane] : 0u;  // n_warps <= 32
    uint32_t eq_before = (lane < warp) ? warp_eq[lane] : 0u;
    if (lane < chunk) {  // the few blocks before this one
        sure_before += peer_shared_u32(&tot[0], (uint32_t)lane);
        eq_before += peer_shared_u32(&tot[1], (uint32_t)lane);
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        sure_before += __shfl_xor_sync(0xFFFFFFFFu, sure_before, d);
        eq_before += __shfl_xor_sync(0xFFFFFFFFu, eq_before, d);
    }
    int32_t* out = p.keep_idx + (size_t)seg * p.k;
    const uint32_t lt = (1u << lane) - 1u;
    for (int wd = w_begin; wd < w_end; ++wd) {
        const int i = (wd << 5) + lane;
        bool sure = false, eq = false;
        if (i < cn) classify(p, keys[i], reserved(i), T, sure, eq);
        const uint32_t sb = __ballot_sync(0xFFFFFFFFu, sure), eb = __ballot_sync(0xFFFFFFFFu, eq);
        const uint32_t my_eq_before = eq_before + __popc(eb & lt);
        const uint32_t my_sure_before = sure_before + __popc(sb & lt);
        if (sure || (eq && my_eq_before < need_eq)) {
            const uint32_t j = my_sure_before + min(my_eq_before, need_eq);
            if (j < (uint32_t)p.k) out[j] = tok0 + i;  // always true when the counts are consistent
        }
        sure_before += __popc(sb);
        eq_before += __popc(eb);
    }
    cluster_barrier();
}

}  // namespace civic
