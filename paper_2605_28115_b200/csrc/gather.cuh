// Order-preserving row gather: dst[t][q, j, :] = src[t][q, idx[q, j], :] for a table of
// tensors that share one index array (all layers' K and V, or the hidden states).
// Pure data movement, HBM-bound: rows are opaque bytes.
//
// One kernel template covers the layouts of the library:
//   kPlain  token-major rows, contiguous destination                (civic_compact, civic_compact_kv)
//   kHeads  head-major tensors [n_seq, n_heads, seq_len, head_bytes]: a "plane" q is one
//           (sequence, head) pair and uses index row q / idx_div    (civic_compact_kv_heads)
//   kPaged  token-major source, destination rows placed through a block table
//                                                                   (civic_compact_kv_paged)
//   kMerge  two sources: text rows outside the visual span, kept visual rows inside it
//                                                                   (civic_merge_embeddings)
// and two work decompositions: rows of at least one warp tile are cut into tiles (LARGE), shorter
// rows are packed several to a tile (SMALL) so that every lane still moves full 16-byte vectors.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

#include "pdl.cuh"

namespace civic {

constexpr int kMaxGatherTensors = 160;  // K and V of 80 layers per launch
constexpr int kGatherThreads = 256;

enum GatherMode { kPlain = 0, kHeads = 1, kPaged = 2, kMerge = 3 };

struct GatherParams {
    const char* src[kMaxGatherTensors];  // each [n_planes, seq_len, row_bytes]
    char* dst[kMaxGatherTensors];        // each [n_planes, s_out, row_bytes] (kPaged: the cache)
    const int32_t* idx;                  // [n_planes / idx_div, s_out]; kMerge: keep_idx [n_planes, k_vis]
    // optional 3 x int32 rows gathered by the same index (position ids); NULL = none
    const int32_t* pos_src;              // [n_planes, seq_len, 3]
    int32_t* pos_dst;                    // [n_planes, s_out, 3]
    int32_t n_tensors, n_planes, seq_len, s_out;
    uint32_t row_bytes;
    uint32_t main_blocks;  // blocks [0, main_blocks) move rows, the rest move pos ids
    int32_t idx_div;       // kHeads: planes (heads) per index row
    // kPaged: row j of plane q lives in page block_table[q, j / page_size], slot j % page_size
    const int32_t* block_table;  // [n_planes, max_pages]
    int32_t max_pages, page_size;
    // kMerge: src[0] is the text [n_planes, seq_len, row], visual the dense visual rows
    const char* visual;  // [n_planes, n_vis, row]
    int32_t vis_start, n_vis, k_vis;
    // index validation (kernels instantiated with CHECK only): int32[4] fault record, see
    // report_bad_index; n_pages bounds the block table's entries
    int32_t* check;
    int32_t n_pages;
};

// Fault record of the checked kernels: {code, plane, position, offending value}.  The first
// thread to find a fault claims word 0 (0 -> code) and fills in the rest; later faults leave the
// record alone, so it names ONE offending entry.  The record is sticky: only the caller clears it.
enum IndexFault { kIndexOk = 0, kIndexOutOfRange = 1, kIndexNotAscending = 2, kIndexBadPage = 3 };
__device__ __forceinline__ void report_bad_index(int32_t* record, int code, int plane, int pos, int value)
{
    if (atomicCAS(record, 0, code) == 0) {
        record[1] = plane;
        record[2] = pos;
        record[3] = value;
    }
}

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

template <bool CHECK>
__device__ __forceinline__ void gather_pos(const GatherParams& p, int block, int n_blocks)
{
    const long long total = (long long)p.n_planes * p.s_out * 3;
    for (long long e = (long long)block * blockDim.x + threadIdx.x; e < total;
         e += (long long)n_blocks * blockDim.x) {
        const long long row = e / 3;
        const int c = (int)(e - row * 3);
        const int s = (int)(row / p.s_out);
        const int32_t i = p.idx[row];
        if (CHECK && (uint32_t)i >= (uint32_t)p.seq_len) {  // neither read nor written
            report_bad_index(p.check, kIndexOutOfRange, s, (int)(row - (long long)s * p.s_out), i);
            continue;
        }
        p.pos_dst[e] = p.pos_src[((size_t)s * p.seq_len + i) * 3 + c];
    }
}

// Source row of output row j of plane q; idx_row is the plane's row of the index array.
// With CHECK an index outside its range is recorded and the function returns false: the caller
// then neither reads nor writes that row.
template <int MODE, bool CHECK>
__device__ __forceinline__ bool source_row(const GatherParams& p, int tensor, int q, int idx_row, int j,
                                           const char*& src)
{
    if constexpr (MODE == kMerge) {
        if (j < p.vis_start) {
            src = p.src[0] + ((size_t)q * p.seq_len + j) * p.row_bytes;
        } else if (j < p.vis_start + p.k_vis) {
            const int32_t i = __ldg(p.idx + (size_t)q * p.k_vis + (j - p.vis_start));
            if (CHECK && (uint32_t)i >= (uint32_t)p.n_vis) {
                report_bad_index(p.check, kIndexOutOfRange, q, j - p.vis_start, i);
                return false;
            }
            src = p.visual + ((size_t)q * p.n_vis + i) * p.row_bytes;
        } else {
            src = p.src[0] + ((size_t)q * p.seq_len + (j - p.k_vis + p.n_vis)) * p.row_bytes;
        }
    } else {
        const int32_t i = __ldg(p.idx + (size_t)idx_row * p.s_out + j);
        if (CHECK && (uint32_t)i >= (uint32_t)p.seq_len) {
            report_bad_index(p.check, kIndexOutOfRange, idx_row, j, i);
            return false;
        }
        src = p.src[tensor] + ((size_t)q * p.seq_len + i) * p.row_bytes;
    }
    return true;
}

template <int MODE, bool CHECK>
__device__ __forceinline__ bool destination_row(const GatherParams& p, int tensor, int q, int j, char*& dst)
{
    if constexpr (MODE == kPaged) {
        const int32_t page = __ldg(p.block_table + (size_t)q * p.max_pages + j / p.page_size);
        if (CHECK && (uint32_t)page >= (uint32_t)p.n_pages) {
            report_bad_index(p.check, kIndexBadPage, q, j / p.page_size, page);
            return false;
        }
        dst = p.dst[tensor] + ((size_t)page * p.page_size + j % p.page_size) * p.row_bytes;
    } else {
        dst = p.dst[tensor] + ((size_t)q * p.s_out + j) * p.row_bytes;
    }
    return true;
}

// One warp per tile of 32 * UNROLL vectors (2 KB for 16-byte vectors), no grid-stride loop.
// Tiles are numbered row-major over [tensor][plane][row], so the hardware block scheduler sweeps
// source and destination in address order, which measured faster on B200 than a persistent
// grid-stride loop.  Every lane has its UNROLL loads in flight before its first store.
// LARGE: a row is ceil(vecs / tile) tiles.  SMALL: a tile is floor(tile / vecs) whole rows.
template <typename VecT, int UNROLL, int MODE, bool SMALL, bool CHECK>
__global__ void __launch_bounds__(kGatherThreads) gather_rows_kernel(const __grid_constant__ GatherParams p)
{
    wait_for_prior_kernels();
    if (blockIdx.x >= p.main_blocks) {
        gather_pos<CHECK>(p, blockIdx.x - p.main_blocks, gridDim.x - p.main_blocks);
        return;
    }
    constexpr int kTileVecs = 32 * UNROLL;
    const int lane = threadIdx.x & 31;
    const int vecs = p.row_bytes / sizeof(VecT);
    const long long rows_per_tensor = (long long)p.n_planes * p.s_out;
    const long long total_rows = rows_per_tensor * p.n_tensors;
    const long long item = (long long)blockIdx.x * (kGatherThreads / 32) + (threadIdx.x >> 5);

    if constexpr (!SMALL) {
        const int tiles_per_row = (vecs + kTileVecs - 1) / kTileVecs;
        if (item >= total_rows * tiles_per_row) return;
        const long long row = item / tiles_per_row;
        const int tile = (int)(item - row * tiles_per_row);
        const int tensor = (int)(row / rows_per_tensor);
        const long long rem = row - (long long)tensor * rows_per_tensor;  // q * s_out + j
        const int q = (int)(rem / p.s_out);
        const int j = (int)(rem - (long long)q * p.s_out);
        const int idx_row = MODE == kHeads ? q / p.idx_div : q;
        const char* src_row = nullptr;
        char* dst_row = nullptr;
        const bool ok = source_row<MODE, CHECK>(p, tensor, q, idx_row, j, src_row) &&
                        destination_row<MODE, CHECK>(p, tensor, q, j, dst_row);
        if (CHECK && !ok) return;  // the whole warp: a tile lies inside one row
        const VecT* src = reinterpret_cast<const VecT*>(src_row);
        VecT* dst = reinterpret_cast<VecT*>(dst_row);
        const int v0 = tile * kTileVecs + lane;
        VecT buf[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u)
            if (v0 + 32 * u < vecs) buf[u] = load_stream(src + v0 + 32 * u);
#pragma unroll
        for (int u = 0; u < UNROLL; ++u)
            if (v0 + 32 * u < vecs) store_stream(dst + v0 + 32 * u, buf[u]);
    } else {
        // The host takes this path only when all rows of the launch number below 2^31, so the
        // tile's first row is decomposed with 32-bit divisions, once; the lanes then step from
        // it by additions (a tile rarely crosses a plane, almost never a tensor).
        const uint32_t uvecs = (uint32_t)vecs;
        const uint32_t rows_per_tile = kTileVecs / uvecs;  // >= 2 by the host's choice
        const uint32_t row0 = (uint32_t)item * rows_per_tile;
        if (row0 >= (uint32_t)total_rows) return;
        const uint32_t s_out = (uint32_t)p.s_out, n_planes = (uint32_t)p.n_planes;
        const uint32_t tensor0 = row0 / (uint32_t)rows_per_tensor;
        const uint32_t rem0 = row0 - tensor0 * (uint32_t)rows_per_tensor;
        const uint32_t q0 = rem0 / s_out, j0 = rem0 - q0 * s_out;
        const uint32_t heads = MODE == kHeads ? (uint32_t)p.idx_div : 1u;
        const uint32_t s0 = q0 / heads, h0 = q0 - s0 * heads;
        const uint32_t step_r = 32u / uvecs, step_c = 32u - step_r * uvecs;
        uint32_t r = (uint32_t)lane / uvecs, c = (uint32_t)lane - r * uvecs;
        VecT buf[UNROLL];
        VecT* dst[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            dst[u] = nullptr;
            uint32_t tensor = tensor0, q = q0, idx_row = s0, h = h0, j = j0 + r;
            while (j >= s_out) {  // next plane; next index row after the last head; next tensor
                j -= s_out;
                ++q;
                if (++h == heads) { h = 0; ++idx_row; }
                if (q == n_planes) { q = 0; idx_row = 0; ++tensor; }
            }
            if (r < rows_per_tile && tensor < (uint32_t)p.n_tensors) {
                const char* src_row = nullptr;
                char* dst_row = nullptr;
                const bool ok = source_row<MODE, CHECK>(p, (int)tensor, (int)q, (int)idx_row, (int)j, src_row) &&
                                destination_row<MODE, CHECK>(p, (int)tensor, (int)q, (int)j, dst_row);
                if (!CHECK || ok) {
                    buf[u] = load_stream(reinterpret_cast<const VecT*>(src_row) + c);
                    dst[u] = reinterpret_cast<VecT*>(dst_row) + c;
                }
            }
            r += step_r;
            c += step_c;
            if (c >= uvecs) { c -= uvecs; ++r; }
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u)
            if (dst[u]) store_stream(dst[u], buf[u]);
    }
}

// out[c, s, j] = pos[c, s, idx[s, j]] for plane-major position ids.  `check` (a fault record as
// in report_bad_index, or NULL) switches the range test of the indices on.
__global__ void gather_pos_planes_kernel(const int32_t* __restrict__ pos, const int32_t* __restrict__ idx,
                                         int32_t* __restrict__ out, int n_planes, int n_seq, int seq_len,
                                         int s_out, int32_t* check)
{
    release_next_kernel();
    wait_for_prior_kernels();
    const long long per_plane = (long long)n_seq * s_out, total = per_plane * n_planes;
    for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < total;
         e += (long long)gridDim.x * blockDim.x) {
        const int c = (int)(e / per_plane);
        const long long rem = e - (long long)c * per_plane;  // s * s_out + j
        const int s = (int)(rem / s_out);
        const int32_t i = idx[rem];
        if (check && (uint32_t)i >= (uint32_t)seq_len) {
            report_bad_index(check, kIndexOutOfRange, s, (int)(rem - (long long)s * s_out), i);
            continue;
        }
        out[e] = pos[((size_t)c * n_seq + s) * seq_len + i];
    }
}

// Stand-alone validation of an index array [n_rows, row_len]: every value in [0, limit) and, if
// asked, every row strictly ascending.  Thread per entry; faults go to the record.
__global__ void validate_indices_kernel(const int32_t* __restrict__ idx, int n_rows, int row_len, int limit,
                                        int ascending, int32_t* record)
{
    wait_for_prior_kernels();
    const long long total = (long long)n_rows * row_len;
    for (long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x; e < total;
         e += (long long)gridDim.x * blockDim.x) {
        const int row = (int)(e / row_len), j = (int)(e - (long long)row * row_len);
        const int32_t i = idx[e];
        if ((uint32_t)i >= (uint32_t)limit) report_bad_index(record, kIndexOutOfRange, row, j, i);
        else if (ascending && j > 0 && idx[e - 1] >= i) report_bad_index(record, kIndexNotAscending, row, j, i);
    }
}

}  // namespace civic
