// Order-preserving row gather: dst[t][s, j, :] = src[t][s, idx[s, j], :] for a table of
// tensors that share one index array (all layers' K and V, or the hidden states).
// Pure data movement, HBM-bound: rows are opaque bytes.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "pdl.cuh"

namespace civic {

constexpr int kMaxGatherTensors = 160;  // K and V of 80 layers per launch
constexpr int kGatherThreads = 256;

struct GatherParams {
    const char* src[kMaxGatherTensors];  // each [n_seq, seq_len, row_bytes]
    char* dst[kMaxGatherTensors];        // each [n_seq, s_out, row_bytes]
    const int32_t* idx;                  // [n_seq, s_out]
    // optional 3 x int32 rows gathered by the same index (position ids); NULL = none
    const int32_t* pos_src;              // [n_seq, seq_len, 3]
    int32_t* pos_dst;                    // [n_seq, s_out, 3]
    int32_t n_tensors, n_seq, seq_len, s_out;
    uint32_t row_bytes;
    uint32_t main_blocks;  // blocks [0, main_blocks) move rows, the rest move pos ids
};

template <typename VecT>
__device__ __forceinline__ VecT load_stream(const VecT* p);
template <>
__device__ __forceinline__ uint4 load_stream<uint4>(const uint4* p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
template <>
__device__ __forceinline__ uint32_t load_stream<uint32_t>(const uint32_t* p)
{
    uint32_t v;
    asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
}
__device__ __forceinline__ void store_stream(uint4* p, uint4 v) { __stcs(p, v); }
__device__ __forceinline__ void store_stream(uint32_t* p, uint32_t v) { __stcs(p, v); }

__device__ __forceinline__ void gather_pos(const GatherParams& p, int block, int n_blocks)
{
    const long long total = (long long)p.n_seq * p.s_out * 3;
    for (long long e = (long long)block * blockDim.x + threadIdx.x; e < total;
         e += (long long)n_blocks * blockDim.x) {
        const long long row = e / 3;
        const int c = (int)(e - row * 3);
        const int s = (int)(row / p.s_out);
        const int32_t i = p.idx[row];
        p.pos_dst[e] = p.pos_src[((size_t)s * p.seq_len + i) * 3 + c];
    }
}

// One warp per row segment, no grid-stride loop.  A segment is up to 32 * UNROLL vectors
// (2 KB for 16-byte vectors) of one destination row; segments are numbered row-major, so
// the hardware block scheduler sweeps source and destination in address order, which
// measured faster on B200 than a persistent grid-stride loop.  Every lane has its UNROLL
// loads in flight before its first store.
template <typename VecT, int UNROLL>
__global__ void __launch_bounds__(kGatherThreads) gather_rows_kernel(const __grid_constant__ GatherParams p)
{
    wait_for_prior_kernels();
    if (blockIdx.x >= p.main_blocks) {
        gather_pos(p, blockIdx.x - p.main_blocks, gridDim.x - p.main_blocks);
        return;
    }
    constexpr int kSegVecs = 32 * UNROLL;
    const int lane = threadIdx.x & 31;
    const int vecs = p.row_bytes / sizeof(VecT);
    const int segs_per_row = (vecs + kSegVecs - 1) / kSegVecs;
    const long long rows_per_tensor = (long long)p.n_seq * p.s_out;
    const long long total_segs = rows_per_tensor * p.n_tensors * segs_per_row;
    const long long item = (long long)blockIdx.x * (kGatherThreads / 32) + (threadIdx.x >> 5);
    if (item >= total_segs) return;

    const long long row = item / segs_per_row;
    const int seg = (int)(item - row * segs_per_row);
    const int tensor = (int)(row / rows_per_tensor);
    const long long rem = row - (long long)tensor * rows_per_tensor;  // s * s_out + j
    const int s = (int)(rem / p.s_out);
    const int32_t i = __ldg(p.idx + rem);
    const VecT* src = reinterpret_cast<const VecT*>(p.src[tensor] + ((size_t)s * p.seq_len + i) * p.row_bytes);
    VecT* dst = reinterpret_cast<VecT*>(p.dst[tensor] + (size_t)rem * p.row_bytes);

    const int v0 = seg * kSegVecs + lane;
    VecT buf[UNROLL];
#pragma unroll
    for (int u = 0; u < UNROLL; ++u)
        if (v0 + 32 * u < vecs) buf[u] = load_stream(src + v0 + 32 * u);
#pragma unroll
    for (int u = 0; u < UNROLL; ++u)
        if (v0 + 32 * u < vecs) store_stream(dst + v0 + 32 * u, buf[u]);
}

}  // namespace civic
