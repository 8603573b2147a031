// C ABI of the library: host-side validation and kernel launches.  See include/civic.h
// for the contract of every entry point.
#include "../../include/civic.h"

#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstring>

#include "aggregate.cuh"
#include "gather.cuh"
#include "kv_attention.cuh"
#include "select.cuh"
#include "select_cluster.cuh"
#include "select_large.cuh"

namespace {

constexpr size_t kMaxDynamicSmem = 227 * 1024;

std::atomic<uint64_t> g_launches{0};
std::atomic<int> g_programmatic{1};

bool programmatic() { return g_programmatic.load(std::memory_order_relaxed) != 0; }
thread_local char g_cuda_error[512] = "";

// Fault record the calling thread's compaction calls validate their index arrays into (device
// int32[4]); NULL = the unchecked kernels.
thread_local int32_t* g_index_check = nullptr;

civic_status_t cuda_fail(cudaError_t e, const char* what)
{
    snprintf(g_cuda_error, sizeof g_cuda_error, "%s: %s", what, cudaGetErrorString(e));
    (void)cudaGetLastError();  // the runtime's own "last error" is not left behind for the caller's next call
    return CIVIC_ERR_CUDA;
}

#define CIVIC_CUDA_TRY(expr)                                        \
    do {                                                            \
        cudaError_t e_ = (expr);                                    \
        if (e_ != cudaSuccess) return cuda_fail(e_, #expr);         \
    } while (0)

bool overlaps(const void* a, size_t a_bytes, const void* b, size_t b_bytes)
{
    if (!a || !b || a_bytes == 0 || b_bytes == 0) return false;
    const uintptr_t a0 = (uintptr_t)a, b0 = (uintptr_t)b;
    return a0 < b0 + b_bytes && b0 < a0 + a_bytes;
}

bool aligned(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }

int64_t reserved_count(const civic_select_desc_t& d)
{
    if (d.t < 1 || d.h < 1 || d.w < 1 || d.region_h < 1 || d.region_w < 1 || d.floor_per_region < 0)
        return -1;
    const int64_t m = d.floor_per_region;
    const int64_t fh = d.h / d.region_h, eh = d.h % d.region_h;  // full tiles, edge extent
    const int64_t fw = d.w / d.region_w, ew = d.w % d.region_w;
    auto take = [m](int64_t size) { return size < m ? size : m; };
    int64_t per_slice = fh * fw * take((int64_t)d.region_h * d.region_w);
    if (ew) per_slice += fh * take((int64_t)d.region_h * ew);
    if (eh) per_slice += fw * take(eh * (int64_t)d.region_w);
    if (eh && ew) per_slice += take(eh * ew);
    return per_slice * d.t;
}

int sm_count()
{
    static std::atomic<int> cached[64];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    int v = cached[dev].load(std::memory_order_relaxed);
    if (v == 0) {
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || v <= 0)
            v = 148;
        cached[dev].store(v, std::memory_order_relaxed);
    }
    return v;
}

// Index of the current device in the per-device caches below, or -1 (then nothing is cached).
int device_slot()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return -1;
    return dev;
}

// The largest dynamic shared memory a kernel may ask for is a per-device function attribute.
// It is raised ONCE per device to the most the kernel can ever need, not per call to that
// call's size: two host threads launching different shapes would otherwise undo each other's
// setting between cudaFuncSetAttribute and the launch.
template <class Kernel>
civic_status_t allow_dynamic_smem(Kernel kernel, size_t max_bytes, std::atomic<int>* done /*[64]*/)
{
    const int dev = device_slot();
    if (dev >= 0 && done[dev].load(std::memory_order_acquire)) return CIVIC_OK;
    CIVIC_CUDA_TRY(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)max_bytes));
    if (dev >= 0) done[dev].store(1, std::memory_order_release);
    return CIVIC_OK;
}

// Launch the row gather for up to kMaxGatherTensors tensors sharing one index array.
template <int MODE, bool CHECK>
civic_status_t launch_gather_checked(civic::GatherParams& p, cudaStream_t stream);

template <int MODE>
civic_status_t launch_gather(civic::GatherParams& p, cudaStream_t stream)
{
    p.check = g_index_check;
    return p.check ? launch_gather_checked<MODE, true>(p, stream) : launch_gather_checked<MODE, false>(p, stream);
}

template <int MODE, bool CHECK>
civic_status_t launch_gather_checked(civic::GatherParams& p, cudaStream_t stream)
{
    const long long total_rows = (long long)p.n_tensors * p.n_planes * p.s_out;
    const bool has_pos = p.pos_src != nullptr;
    const long long pos_elems = has_pos ? (long long)p.n_planes * p.s_out * 3 : 0;
    if (total_rows == 0 && pos_elems == 0) return CIVIC_OK;

    bool vec16 = p.row_bytes % 16 == 0 && aligned(p.visual, 16);
    for (int i = 0; i < p.n_tensors && vec16; ++i)
        vec16 = aligned(p.src[i], 16) && aligned(p.dst[i], 16);
    // one warp per tile of 32 * UNROLL vectors: a slice of a long row, or several short rows
    const int threads = civic::kGatherThreads, warps = threads / 32;
    const long long tile_vecs = vec16 ? 32 * 4 : 32 * 8;
    const long long vecs = p.row_bytes / (vec16 ? 16 : 4);
    const bool small = 2 * vecs <= tile_vecs && total_rows < 0x7FFFFFFFLL;
    const long long items = small ? (total_rows + tile_vecs / vecs - 1) / (tile_vecs / vecs)
                                  : total_rows * ((vecs + tile_vecs - 1) / tile_vecs);
    const long long main_blocks = (items + warps - 1) / warps;
    long long pos_blocks = (pos_elems + threads - 1) / threads;
    if (pos_blocks > sm_count()) pos_blocks = sm_count();
    if (main_blocks + pos_blocks > 0x7FFFFFFFLL) return CIVIC_ERR_UNSUPPORTED;
    p.main_blocks = (uint32_t)main_blocks;
    const unsigned grid = (unsigned)(main_blocks + pos_blocks);
    const bool pdl = programmatic();
    cudaError_t e;
    if (vec16)
        e = small ? civic::launch(pdl, civic::gather_rows_kernel<uint4, 4, MODE, true, CHECK>, grid, threads, 0, stream, p)
                  : civic::launch(pdl, civic::gather_rows_kernel<uint4, 4, MODE, false, CHECK>, grid, threads, 0, stream, p);
    else
        e = small ? civic::launch(pdl, civic::gather_rows_kernel<uint32_t, 8, MODE, true, CHECK>, grid, threads, 0, stream, p)
                  : civic::launch(pdl, civic::gather_rows_kernel<uint32_t, 8, MODE, false, CHECK>, grid, threads, 0, stream, p);
    CIVIC_CUDA_TRY(e);
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return CIVIC_OK;
}

// Validation shared by the three K/V calls: pointer tables, alignment, no destination
// overlapping a source, another destination or the index array.
civic_status_t check_kv_tables(const void* const* k_src, const void* const* v_src, void* const* k_dst,
                               void* const* v_dst, int32_t n_layers, size_t src_bytes, size_t dst_bytes,
                               const void* idx, size_t idx_bytes)
{
    if (!k_src || !v_src || !k_dst || !v_dst) return CIVIC_ERR_INVALID_ARG;
    for (int l = 0; l < n_layers; ++l) {
        if (!k_src[l] || !v_src[l] || !k_dst[l] || !v_dst[l]) return CIVIC_ERR_INVALID_ARG;
        if (!aligned(k_src[l], 4) || !aligned(v_src[l], 4) || !aligned(k_dst[l], 4) ||
            !aligned(v_dst[l], 4))
            return CIVIC_ERR_ALIGNMENT;
    }
    for (int a = 0; a < 2 * n_layers; ++a) {
        const void* da = (a & 1) ? v_dst[a >> 1] : k_dst[a >> 1];
        if (overlaps(da, dst_bytes, idx, idx_bytes)) return CIVIC_ERR_INVALID_ARG;
        for (int b = 0; b < 2 * n_layers; ++b) {
            const void* sb = (b & 1) ? v_src[b >> 1] : k_src[b >> 1];
            const void* db = (b & 1) ? v_dst[b >> 1] : k_dst[b >> 1];
            if (overlaps(da, dst_bytes, sb, src_bytes)) return CIVIC_ERR_INVALID_ARG;
            if (a != b && overlaps(da, dst_bytes, db, dst_bytes)) return CIVIC_ERR_INVALID_ARG;
        }
    }
    return CIVIC_OK;
}

// Fills the pointer tables of `p` chunk by chunk and launches MODE once per chunk of layers.
template <int MODE>
civic_status_t launch_kv(civic::GatherParams base, const void* const* k_src, const void* const* v_src,
                         void* const* k_dst, void* const* v_dst, int32_t n_layers, cudaStream_t stream)
{
    const int layers_per_launch = civic::kMaxGatherTensors / 2;
    for (int l0 = 0; l0 < n_layers; l0 += layers_per_launch) {
        const int nl = n_layers - l0 < layers_per_launch ? n_layers - l0 : layers_per_launch;
        civic::GatherParams p = base;
        for (int l = 0; l < nl; ++l) {
            p.src[2 * l] = (const char*)k_src[l0 + l];
            p.dst[2 * l] = (char*)k_dst[l0 + l];
            p.src[2 * l + 1] = (const char*)v_src[l0 + l];
            p.dst[2 * l + 1] = (char*)v_dst[l0 + l];
        }
        p.n_tensors = 2 * nl;
        const civic_status_t st = launch_gather<MODE>(p, stream);
        if (st != CIVIC_OK) return st;
    }
    return CIVIC_OK;
}

// Work split and scratch layout of the many-block selection.
struct LargePlan {
    int32_t n, n_rh, rows_per_chunk, n_chunks, chunk_tokens;
    size_t hist_off, counts_off, flags_off, total;  // byte offsets into the workspace
};

// The default chunk size depends on shapes only (not on the device), so that the workspace size
// is a pure function of the arguments: 148 = one block for each SM of a B200.
constexpr int64_t kLargeBlocksTarget = 148;

size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// CIVIC_OK and a filled plan, or the reason the shape cannot be handled.
civic_status_t plan_large(const civic_select_desc_t& d, int32_t n_seg, int32_t chunk_tokens, LargePlan& pl)
{
    if (reserved_count(d) < 0 || n_seg < 0 || chunk_tokens < 0) return CIVIC_ERR_INVALID_ARG;
    const int64_t n = (int64_t)d.t * d.h * d.w;
    if (n > INT32_MAX) return CIVIC_ERR_UNSUPPORTED;
    const int64_t rh = d.region_h < d.h ? d.region_h : d.h;  // tokens of the tallest region row
    const int64_t row_tokens = rh * d.w;
    if (chunk_tokens > civic::kLargeMaxChunk) chunk_tokens = civic::kLargeMaxChunk;
    if (chunk_tokens == 0) {
        // default: about one block per SM over the whole launch, between 2048 tokens and the
        // capacity (measured on B200: fewer, larger blocks leave SMs idle; many more blocks pay
        // for their atomic flushes into the shared global histograms)
        int64_t c = ((int64_t)n_seg * n + kLargeBlocksTarget - 1) / kLargeBlocksTarget;
        c = c < 2048 ? 2048 : (c > civic::kLargeMaxChunk ? civic::kLargeMaxChunk : c);
        if (c < row_tokens && row_tokens <= civic::kLargeMaxChunk) c = row_tokens;
        chunk_tokens = (int32_t)c;
    }
    if (row_tokens > chunk_tokens) return CIVIC_ERR_UNSUPPORTED;
    pl.n = (int32_t)n;
    pl.n_rh = (d.h + d.region_h - 1) / d.region_h;
    pl.rows_per_chunk = (int32_t)(chunk_tokens / row_tokens);
    const int64_t region_rows = (int64_t)d.t * pl.n_rh;
    pl.n_chunks = (int32_t)((region_rows + pl.rows_per_chunk - 1) / pl.rows_per_chunk);
    pl.chunk_tokens = (int32_t)(pl.rows_per_chunk * row_tokens);
    if ((int64_t)pl.n_chunks * n_seg > INT32_MAX) return CIVIC_ERR_UNSUPPORTED;
    pl.hist_off = 0;
    pl.counts_off = round_up((size_t)n_seg * (3 * civic::kLargeBins + civic::kLargeSelWords) * 4, 256);
    pl.flags_off = pl.counts_off + round_up((size_t)n_seg * pl.n_chunks * 2 * 4, 256);
    pl.total = pl.flags_off + round_up((size_t)n_seg * (size_t)n, 256);
    return CIVIC_OK;
}

// One cluster of four thread blocks per segment, one launch (select_cluster.cuh).  Returns
// CIVIC_ERR_UNSUPPORTED without launching when the segment does not fit a cluster, the five
// launches are expected to be faster, or the device cannot place a cluster; the caller then
// takes the five launches.  Measured on B200 (us per call): the cluster takes 18.5 (3 K tokens
// per block) to 26.6 (12.5 K per block) whatever the number of segments up to 16; the five
// launches take 22.6 while their blocks of 2048 tokens fit one wave of 148 and 34 .. 41 beyond.
civic_status_t launch_cluster_select(const float* scores, int32_t n_seg, const civic_select_desc_t& d,
                                     int32_t* keep_idx, const LargePlan& pl, int32_t k_fill, cudaStream_t stream)
{
    const int64_t rh = d.region_h < d.h ? d.region_h : d.h;
    const int64_t row_tokens = rh * d.w, region_rows = (int64_t)d.t * pl.n_rh;
    const int blocks = civic::kClusterBlocks;
    const int64_t rows_per_chunk = (region_rows + blocks - 1) / blocks;
    const int64_t chunk_tokens = rows_per_chunk * row_tokens;
    const bool one_wave_of_small_blocks = (int64_t)n_seg * pl.n <= kLargeBlocksTarget * 2048;
    if (chunk_tokens > civic::kClusterMaxChunk || (int64_t)n_seg * blocks > INT32_MAX ||
        (pl.n > 16384 && one_wave_of_small_blocks))
        return CIVIC_ERR_UNSUPPORTED;
    civic::LargeParams p;
    memset(&p, 0, sizeof p);
    p.scores = scores;
    p.keep_idx = keep_idx;
    p.n = pl.n; p.t = d.t; p.h = d.h; p.w = d.w;
    p.region_h = d.region_h; p.region_w = d.region_w;
    p.m = d.floor_per_region; p.k = d.k; p.k_fill = k_fill;
    p.n_rh = pl.n_rh; p.rows_per_chunk = (int32_t)rows_per_chunk; p.n_chunks = blocks;
    const size_t smem = civic::select_cluster_smem_bytes((int)chunk_tokens);
    static std::atomic<int> smem_allowed[64];
    const civic_status_t as = allow_dynamic_smem(civic::select_cluster_kernel,
                                                 civic::select_cluster_smem_bytes(civic::kClusterMaxChunk), smem_allowed);
    if (as != CIVIC_OK) return as;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(n_seg * blocks));
    cfg.blockDim = dim3(civic::kClusterThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)blocks;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    int n_attr = 1;
    if (programmatic()) {
        attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
        ++n_attr;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n_attr;
    // Can the device hold a cluster of this kernel at all?  Asked once per device, for the largest
    // block the kernel is ever launched with (a smaller one then fits too): 1 = yes, 2 = no.
    static std::atomic<int> placeable[64];
    const int dev = device_slot();
    int fits = dev >= 0 ? placeable[dev].load(std::memory_order_relaxed) : 0;
    if (fits == 0) {
        cudaLaunchConfig_t probe = cfg;
        probe.gridDim = dim3((unsigned)blocks);
        probe.dynamicSmemBytes = civic::select_cluster_smem_bytes(civic::kClusterMaxChunk);
        int resident = 0;
        CIVIC_CUDA_TRY(cudaOccupancyMaxActiveClusters(&resident, civic::select_cluster_kernel, &probe));
        fits = resident >= 1 ? 1 : 2;
        if (dev >= 0) placeable[dev].store(fits, std::memory_order_relaxed);
    }
    if (fits != 1) return CIVIC_ERR_UNSUPPORTED;
    CIVIC_CUDA_TRY(cudaLaunchKernelEx(&cfg, civic::select_cluster_kernel, p));
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return CIVIC_OK;
}

// The many-block selection; `ws` holds pl.total bytes of scratch.  With the library's own
// chunking (`own_chunks`) a segment that fits a cluster of blocks takes the one-launch path.
civic_status_t launch_large(const float* scores, int32_t n_seg, const civic_select_desc_t& d,
                            int32_t* keep_idx, char* ws, const LargePlan& pl, int32_t k_fill,
                            cudaStream_t stream, bool own_chunks)
{
    if (own_chunks) {
        const civic_status_t cs = launch_cluster_select(scores, n_seg, d, keep_idx, pl, k_fill, stream);
        if (cs != CIVIC_ERR_UNSUPPORTED) return cs;
    }
    civic::LargeParams p;
    p.scores = scores;
    p.keep_idx = keep_idx;
    p.n = pl.n; p.t = d.t; p.h = d.h; p.w = d.w;
    p.region_h = d.region_h; p.region_w = d.region_w;
    p.m = d.floor_per_region; p.k = d.k; p.k_fill = k_fill;
    p.n_rh = pl.n_rh; p.rows_per_chunk = pl.rows_per_chunk; p.n_chunks = pl.n_chunks;
    p.hist = (uint32_t*)(ws + pl.hist_off);
    p.sel = p.hist + (size_t)n_seg * 3 * civic::kLargeBins;
    p.counts = (uint32_t*)(ws + pl.counts_off);
    p.flags = (uint8_t*)(ws + pl.flags_off);
    // histograms and scalars start at zero
    CIVIC_CUDA_TRY(cudaMemsetAsync(ws + pl.hist_off, 0,
                                   (size_t)n_seg * (3 * civic::kLargeBins + civic::kLargeSelWords) * 4, stream));
    const size_t smem = (size_t)(civic::kLargeBins + civic::kLargeMaxChunk / 32 + ((pl.chunk_tokens + 31) & ~31)) * 4;
    {
        static std::atomic<int> smem_allowed[64];
        const size_t most = (size_t)(civic::kLargeBins + civic::kLargeMaxChunk / 32 + civic::kLargeMaxChunk) * 4;
        const civic_status_t as = allow_dynamic_smem(civic::large_floor_kernel, most, smem_allowed);
        if (as != CIVIC_OK) return as;
    }
    const unsigned grid = (unsigned)(n_seg * pl.n_chunks), threads = civic::kLargeThreads;
    const bool pdl = programmatic();
    CIVIC_CUDA_TRY(civic::launch(pdl, civic::large_floor_kernel, grid, threads, smem, stream, p));
    CIVIC_CUDA_TRY(civic::launch(pdl, civic::large_hist_kernel<1>, grid, threads, 0, stream, p));
    CIVIC_CUDA_TRY(civic::launch(pdl, civic::large_hist_kernel<2>, grid, threads, 0, stream, p));
    CIVIC_CUDA_TRY(civic::launch(pdl, civic::large_count_kernel, grid, threads, 0, stream, p));
    CIVIC_CUDA_TRY(civic::launch(pdl, civic::large_place_kernel, grid, threads, 0, stream, p));
    g_launches.fetch_add(5, std::memory_order_relaxed);
    return CIVIC_OK;
}

// Regions that get a shared-memory slot for their maximum (floor of one token per region): all of
// them if they are few enough and the segment leaves the room, else none (the floor then walks
// the tiles, one thread per region).  The slots cost one 64-bit shared-memory atomic per token, and
// the SM serves about one such atomic per clock whatever the addresses: beyond one token per thread
// the walk is faster as long as the tiles are small (n = 3136, tiles of 2 x 2 or 4 x 4: 8.9 and 9.8 us
// per call against 9.9 and 10.5 us with slots; n = 1024: 6.9 against 6.8 us).
int32_t select_floor_slots(const civic_select_desc_t& d, int64_t n)
{
    if (d.floor_per_region != 1) return 0;
    if (n > 1024 && (int64_t)d.region_h * d.region_w <= 64) return 0;
    const int64_t n_reg = (int64_t)d.t * ((d.h + d.region_h - 1) / d.region_h) * ((d.w + d.region_w - 1) / d.region_w);
    if (n_reg > civic::kMaxFloorSlots || civic::select_smem_bytes((int)n, (int)n_reg) > kMaxDynamicSmem) return 0;
    return (int32_t)n_reg;
}

int select_threads(int64_t n)
{
    const int64_t threads = (n + 31) / 32 * 32;
    return (int)(threads < 128 ? 128 : (threads > 1024 ? 1024 : threads));
}

civic_status_t select_impl(const float* scores, int32_t n_seg, const civic_select_desc_t* desc,
                           int32_t* keep_idx, int32_t* seq_idx, int32_t seq_len, int32_t vis_start,
                           void* stream)
{
    if (!desc || n_seg < 0) return CIVIC_ERR_INVALID_ARG;
    const int64_t n_res = reserved_count(*desc);
    if (n_res < 0) return CIVIC_ERR_INVALID_ARG;
    const int64_t n = (int64_t)desc->t * desc->h * desc->w;
    if (n > INT32_MAX) return CIVIC_ERR_UNSUPPORTED;
    if (desc->k < 0 || desc->k > n) return CIVIC_ERR_K_RANGE;
    if (n_res > desc->k) return CIVIC_ERR_FLOOR_EXCEEDS_K;
    if (n_seg == 0 || desc->k == 0) return CIVIC_OK;
    if (!scores || !keep_idx) return CIVIC_ERR_INVALID_ARG;
    if (!aligned(scores, 4) || !aligned(keep_idx, 4)) return CIVIC_ERR_ALIGNMENT;
    if (n > civic_select_max_tokens()) return CIVIC_ERR_UNSUPPORTED;
    if (overlaps(scores, (size_t)n_seg * n * 4, keep_idx, (size_t)n_seg * desc->k * 4))
        return CIVIC_ERR_INVALID_ARG;

    civic::SelectParams p;
    p.scores = scores;
    p.keep_idx = keep_idx;
    p.shape = civic::SegShape{(int32_t)n, desc->t, desc->h, desc->w, desc->region_h, desc->region_w,
                              desc->floor_per_region, desc->k, (int32_t)(desc->k - n_res),
                              select_floor_slots(*desc, n)};
    p.seq_idx = seq_idx;
    p.seq_len = seq_len;
    p.vis_start = vis_start;

    const size_t smem = civic::select_smem_bytes(p.shape.n, p.shape.floor_slots);
    {
        static std::atomic<int> smem_allowed[64];
        const civic_status_t as = allow_dynamic_smem(civic::select_kernel, kMaxDynamicSmem, smem_allowed);
        if (as != CIVIC_OK) return as;
    }
    const int threads = select_threads(p.shape.n);
    CIVIC_CUDA_TRY(civic::launch(programmatic(), civic::select_kernel, (unsigned)n_seg, (unsigned)threads,
                                 smem, (cudaStream_t)stream, p));
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return CIVIC_OK;
}

// ---- civic_select_large without any caller-provided or allocated scratch -------------------
//
// The scratch of the many-block selection lives in this fixed array inside the library's device
// image: every GPU that loads the library holds it until the process exits.  In host code the
// name g_static_scratch is only a handle for the runtime, not an address a kernel may use;
// its device address is looked up with cudaGetSymbolAddress, once per device.
constexpr size_t kStaticScratchBytes = (size_t)2 << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// Device address of the static scratch on the CURRENT device.
civic_status_t static_scratch_address(char** out)
{
    static std::atomic<char*> cached[64];
    int dev = -1;
    CIVIC_CUDA_TRY(cudaGetDevice(&dev));
    const bool cacheable = dev >= 0 && dev < 64;
    char* ptr = cacheable ? cached[dev].load(std::memory_order_acquire) : nullptr;
    if (!ptr) {
        void* sym = nullptr;
        CIVIC_CUDA_TRY(cudaGetSymbolAddress(&sym, g_static_scratch));
        ptr = (char*)sym;
        if (cacheable) cached[dev].store(ptr, std::memory_order_release);
    }
    *out = ptr;
    return CIVIC_OK;
}

// ---- compact visual aggregation (Eq. 8) ----------------------------------------------------

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime (no link against libcuda).
civic_status_t tensor_map_encoder(EncodeTiledFn* out)
{
    static std::atomic<void*> cached{nullptr};
    void* fn = cached.load(std::memory_order_acquire);
    if (!fn) {
        cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
        CIVIC_CUDA_TRY(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q));
        if (q != cudaDriverEntryPointSuccess || !fn) return cuda_fail(cudaErrorNotSupported, "cuTensorMapEncodeTiled");
        cached.store(fn, std::memory_order_release);
    }
    *out = (EncodeTiledFn)fn;
    return CIVIC_OK;
}

// bf16 tensor of rank 2 or 3, innermost dimension first; boxes of 64 elements (128 B, swizzled).
// box_cols = 64 gives the swizzled 128-byte rows the MMA descriptors expect, 32 rows of 64 bytes with
// the 64-byte swizzle (output staging); any other width (a multiple of 8 columns) a plain box.
civic_status_t make_map(EncodeTiledFn enc, CUtensorMap* map, const void* base, int rank, const uint64_t* dims,
                        const uint64_t* strides_bytes, uint32_t box_rows, uint32_t box_cols = 64)
{
    cuuint64_t gdim[3] = {dims[0], dims[1], rank == 3 ? dims[2] : 1};
    cuuint64_t gstr[2] = {strides_bytes[0], rank == 3 ? strides_bytes[1] : 0};
    cuuint32_t box[3] = {box_cols, box_rows, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gdim, gstr,
                           box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           box_cols == 64 ? CU_TENSOR_MAP_SWIZZLE_128B
                                          : (box_cols == 32 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_NONE),
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        snprintf(g_cuda_error, sizeof g_cuda_error, "cuTensorMapEncodeTiled failed with CUresult %d", (int)r);
        return CIVIC_ERR_CUDA;
    }
    return CIVIC_OK;
}

struct AggPlan {
    int32_t t_ld, n_tiles_t, values_bn;
    int32_t n_panels;
    size_t q_off, qsum_off, stats_off, p_off, lpart_off, invl_off, mass_off, total;
    size_t prepared_total;  // Q_A in bf16 | its row sums: what civic_anchor_prepare writes
};

civic_status_t plan_aggregate(int32_t n_img, int32_t t_e, int32_t m_e, int32_t d_v, AggPlan& pl)
{
    if (n_img < 0 || t_e < 1 || m_e < 1 || d_v < 1) return CIVIC_ERR_INVALID_ARG;
    if (d_v % 64) return CIVIC_ERR_UNSUPPORTED;
    pl.t_ld = (t_e + 7) / 8 * 8;
    pl.n_tiles_t = (t_e + civic::kScoresBN - 1) / civic::kScoresBN;
    pl.values_bn = d_v % 256 == 0 ? 256 : (d_v % 192 == 0 ? 192 : (d_v % 128 == 0 ? 128 : 256));
    const int64_t m_tiles = (m_e + civic::kAggBM - 1) / civic::kAggBM;
    if (n_img > 65535 || m_tiles * pl.n_tiles_t * n_img > INT32_MAX || m_tiles * ((d_v + 127) / 128) * n_img > INT32_MAX)
        return CIVIC_ERR_UNSUPPORTED;
    size_t off = 0;
    auto take = [&off](size_t bytes) { const size_t at = off; off += round_up(bytes, 256); return at; };
    pl.q_off = take((size_t)m_e * d_v * 2);
    pl.qsum_off = take((size_t)m_e * 4);
    pl.prepared_total = off;
    pl.stats_off = take((size_t)n_img * t_e * 8);
    pl.p_off = take((size_t)n_img * m_e * pl.t_ld * 2);
    pl.lpart_off = take((size_t)n_img * m_e * 2 * pl.n_tiles_t * 4);  // two column halves per token tile
    pl.invl_off = take((size_t)n_img * m_e * 4);
    pl.n_panels = 4 * ((m_e + civic::kAggBM - 1) / civic::kAggBM);  // panels of 32 anchors
    pl.mass_off = take((size_t)n_img * pl.n_panels * pl.t_ld * 4);  // per-panel column sums of the token mass
    pl.total = off;
    return CIVIC_OK;
}

// map_a, map_b, map_c: operands (what each Op loads through them); map_d, map_e: results stored by bulk
// tensor copies (maps an Op does not use may repeat another one)
template <class Op>
civic_status_t launch_gemm(const CUtensorMap& map_a, const CUtensorMap& map_b, const CUtensorMap& map_c,
                           const CUtensorMap& map_d, const CUtensorMap& map_e, const typename Op::Params& params,
                           int32_t total_tiles, cudaStream_t stream)
{
    const size_t smem = sizeof(typename Op::Smem) + 1024;
    {
        static std::atomic<int> smem_allowed[64];
        const civic_status_t as = allow_dynamic_smem(civic::aggregate_gemm_kernel<Op>, smem, smem_allowed);
        if (as != CIVIC_OK) return as;
    }
    // persistent: one block per SM, or one pair of blocks (a cluster of two) per two SMs
    const int workers_max = sm_count() / Op::kCtas;
    const int workers = total_tiles < workers_max ? total_tiles : workers_max;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(workers * Op::kCtas));
    cfg.blockDim = dim3((unsigned)(civic::kAggThreads + 32 * Op::kSideWarps));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    int n_attr = 0;
    if (Op::kCtas == 2) {
        attr[n_attr].id = cudaLaunchAttributeClusterDimension;
        attr[n_attr].val.clusterDim.x = 2;
        attr[n_attr].val.clusterDim.y = 1;
        attr[n_attr].val.clusterDim.z = 1;
        ++n_attr;
    }
    if (programmatic()) {
        attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
        ++n_attr;
    }
    cfg.attrs = attr;
    cfg.numAttrs = n_attr;
    if (Op::kCtas == 2) {
        // not every SM need have a partner free: size the persistent grid to the clusters that
        // can really be resident together (asked once per device)
        static std::atomic<int> resident[64];
        int dev = 0;
        CIVIC_CUDA_TRY(cudaGetDevice(&dev));
        int n = dev >= 0 && dev < 64 ? resident[dev].load(std::memory_order_relaxed) : 0;
        if (n == 0) {
            CIVIC_CUDA_TRY(cudaOccupancyMaxActiveClusters(&n, civic::aggregate_gemm_kernel<Op>, &cfg));
            if (n < 1) return CIVIC_ERR_UNSUPPORTED;
            if (dev >= 0 && dev < 64) resident[dev].store(n, std::memory_order_relaxed);
        }
        if (workers > n) cfg.gridDim = dim3((unsigned)(n * 2));
    }
    CIVIC_CUDA_TRY(cudaLaunchKernelEx(&cfg, civic::aggregate_gemm_kernel<Op>, map_a, map_b, map_c, map_d, map_e, params));
    return CIVIC_OK;
}

}  // namespace

extern "C" {

const char* civic_status_string(civic_status_t s)
{
    switch (s) {
        case CIVIC_OK: return "CIVIC_OK";
        case CIVIC_ERR_INVALID_ARG: return "CIVIC_ERR_INVALID_ARG";
        case CIVIC_ERR_K_RANGE: return "CIVIC_ERR_K_RANGE";
        case CIVIC_ERR_FLOOR_EXCEEDS_K: return "CIVIC_ERR_FLOOR_EXCEEDS_K";
        case CIVIC_ERR_ALIGNMENT: return "CIVIC_ERR_ALIGNMENT";
        case CIVIC_ERR_UNSUPPORTED: return "CIVIC_ERR_UNSUPPORTED";
        case CIVIC_ERR_CUDA: return "CIVIC_ERR_CUDA";
        case CIVIC_ERR_WORKSPACE: return "CIVIC_ERR_WORKSPACE";
    }
    return "CIVIC_ERR_UNKNOWN";
}

const char* civic_last_cuda_error(void) { return g_cuda_error; }

uint64_t civic_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int32_t civic_set_programmatic_launch(int32_t enable)
{
    return g_programmatic.exchange(enable ? 1 : 0, std::memory_order_relaxed);
}

int32_t civic_select_max_tokens(void)
{
    // largest n whose keys, reserved bits and histogram fit into one block's shared memory;
    // the scan also packs two counts of at most n into 16 bits each
    int32_t words = (int32_t)((kMaxDynamicSmem / sizeof(uint32_t) - (4 * 256 + 32 + 4)) / 33);
    int32_t n = words * 32;
    return n < 65535 ? n : 65535;
}

int64_t civic_reserved_count(const civic_select_desc_t* desc)
{
    return desc ? reserved_count(*desc) : -1;
}

civic_status_t civic_select(const float* scores, int32_t n_seg, const civic_select_desc_t* desc,
                            int32_t* keep_idx, void* stream)
{
    return select_impl(scores, n_seg, desc, keep_idx, nullptr, 0, 0, stream);
}

civic_status_t civic_select_seq(const float* scores, int32_t n_seq, const civic_select_desc_t* desc,
                                int32_t seq_len, int32_t vis_start, int32_t* keep_idx,
                                int32_t* seq_idx, void* stream)
{
    if (!desc || seq_len < 0 || vis_start < 0) return CIVIC_ERR_INVALID_ARG;
    const int64_t n = (int64_t)desc->t * desc->h * desc->w;
    if (desc->t < 1 || desc->h < 1 || desc->w < 1 || n > INT32_MAX) return CIVIC_ERR_INVALID_ARG;
    if ((int64_t)vis_start + n > seq_len) return CIVIC_ERR_INVALID_ARG;
    if (desc->k < 0 || desc->k > n) return CIVIC_ERR_K_RANGE;
    const int64_t s_out = (int64_t)seq_len - n + desc->k;
    if (n_seq > 0 && s_out > 0) {
        if (!seq_idx) return CIVIC_ERR_INVALID_ARG;
        if (!aligned(seq_idx, 4)) return CIVIC_ERR_ALIGNMENT;
        if (overlaps(seq_idx, (size_t)n_seq * s_out * 4, keep_idx, (size_t)n_seq * desc->k * 4) ||
            overlaps(seq_idx, (size_t)n_seq * s_out * 4, scores, (size_t)n_seq * n * 4))
            return CIVIC_ERR_INVALID_ARG;
    }
    if (desc->k == 0) {
        // nothing to select: the sequence indices are the text positions alone
        const civic_status_t st = select_impl(scores, n_seq, desc, keep_idx, nullptr, 0, 0, stream);
        if (st != CIVIC_OK) return st;
        return civic_seq_indices(keep_idx, n_seq, 0, seq_len, vis_start, (int32_t)n, seq_idx, stream);
    }
    return select_impl(scores, n_seq, desc, keep_idx, seq_idx, seq_len, vis_start, stream);
}

size_t civic_select_static_scratch_bytes(void) { return kStaticScratchBytes; }

civic_status_t civic_select_large_static(const float* scores, int32_t n_seg, const civic_select_desc_t* desc,
                                         int32_t* keep_idx, int32_t chunk_tokens, void* stream)
{
    if (!desc || n_seg < 0) return CIVIC_ERR_INVALID_ARG;
    const int64_t n_res = reserved_count(*desc);
    if (n_res < 0) return CIVIC_ERR_INVALID_ARG;
    const int64_t n = (int64_t)desc->t * desc->h * desc->w;
    if (n > INT32_MAX) return CIVIC_ERR_UNSUPPORTED;
    if (desc->k < 0 || desc->k > n) return CIVIC_ERR_K_RANGE;
    if (n_res > desc->k) return CIVIC_ERR_FLOOR_EXCEEDS_K;
    LargePlan pl;
    const civic_status_t st = plan_large(*desc, n_seg, chunk_tokens, pl);
    if (st != CIVIC_OK) return st;
    if (pl.total > kStaticScratchBytes) return CIVIC_ERR_WORKSPACE;  // beyond the built-in scratch
    if (n_seg == 0 || desc->k == 0) return CIVIC_OK;
    if (!scores || !keep_idx) return CIVIC_ERR_INVALID_ARG;
    if (!aligned(scores, 4) || !aligned(keep_idx, 4)) return CIVIC_ERR_ALIGNMENT;
    if (overlaps(scores, (size_t)n_seg * n * 4, keep_idx, (size_t)n_seg * desc->k * 4))
        return CIVIC_ERR_INVALID_ARG;
    char* scratch = nullptr;
    const civic_status_t st2 = static_scratch_address(&scratch);
    if (st2 != CIVIC_OK) return st2;
    // the histograms and scalars inside the scratch are cleared by launch_large on every call
    return launch_large(scores, n_seg, *desc, keep_idx, scratch, pl, (int32_t)(desc->k - n_res),
                        (cudaStream_t)stream, chunk_tokens == 0);
}

size_t civic_anchor_aggregate_workspace_bytes(int32_t n_img, int32_t t_e, int32_t m_e, int32_t d_v)
{
    AggPlan pl;
    return plan_aggregate(n_img, t_e, m_e, d_v, pl) == CIVIC_OK ? pl.total : 0;
}

size_t civic_anchor_prepared_bytes(int32_t m_e, int32_t d_v)
{
    AggPlan pl;
    return plan_aggregate(1, 1, m_e, d_v, pl) == CIVIC_OK ? pl.prepared_total : 0;
}

civic_status_t civic_anchor_prepare(const float* anchors, int32_t m_e, int32_t d_v, void* prepared,
                                    size_t prepared_bytes, void* stream)
{
    AggPlan pl;
    const civic_status_t st = plan_aggregate(1, 1, m_e, d_v, pl);
    if (st != CIVIC_OK) return st;
    if (!anchors || !prepared) return CIVIC_ERR_INVALID_ARG;
    if (!aligned(anchors, 4) || !aligned(prepared, 256)) return CIVIC_ERR_ALIGNMENT;
    if (prepared_bytes < pl.prepared_total) return CIVIC_ERR_WORKSPACE;
    if (overlaps(anchors, (size_t)m_e * d_v * 4, prepared, pl.prepared_total)) return CIVIC_ERR_INVALID_ARG;
    char* prep = (char*)prepared;
    CIVIC_CUDA_TRY(civic::launch(programmatic(), civic::aggregate_prep_kernel, (unsigned)((m_e + 7) / 8), 256u, 0,
                                 (cudaStream_t)stream, anchors, m_e, (const __nv_bfloat16*)nullptr, 0LL, d_v, 1e-5f,
                                 1e-12f, (__nv_bfloat16*)(prep + pl.q_off), (float*)(prep + pl.qsum_off),
                                 (float2*)nullptr, (int*)nullptr));
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return CIVIC_OK;
}

// Eq. 8 with the anchors either raw (`anchors`, normalised here on every call) or prepared once
// (`prepared`, written by civic_anchor_prepare).
static civic_status_t aggregate_impl(const void* x0, const float* anchors, const void* prepared, int32_t n_img,
                                     int32_t t_e, int32_t m_e, int32_t d_v, float tau, void* z0, float* token_mass,
                                     void* workspace, size_t workspace_bytes, int32_t* device_status, void* stream_)
{
    AggPlan pl;
    const civic_status_t st = plan_aggregate(n_img, t_e, m_e, d_v, pl);
    if (st != CIVIC_OK) return st;
    if (!(tau >= 0.025f) || !(tau <= 1e30f)) return CIVIC_ERR_UNSUPPORTED;  // also rejects NaN
    if (n_img == 0) return CIVIC_OK;
    if (!x0 || (!anchors && !prepared) || !z0 || !device_status) return CIVIC_ERR_INVALID_ARG;
    if (!aligned(x0, 16) || !aligned(z0, 16) || !aligned(anchors, 4) || !aligned(prepared, 256) ||
        !aligned(token_mass, 4) || !aligned(device_status, 4))
        return CIVIC_ERR_ALIGNMENT;
    if (!workspace || workspace_bytes < pl.total) return CIVIC_ERR_WORKSPACE;
    if (!aligned(workspace, 256)) return CIVIC_ERR_ALIGNMENT;
    const size_t x_bytes = (size_t)n_img * t_e * d_v * 2, z_bytes = (size_t)n_img * m_e * d_v * 2;
    const void* a_any = anchors ? (const void*)anchors : prepared;
    const size_t a_bytes = anchors ? (size_t)m_e * d_v * 4 : pl.prepared_total;
    if (overlaps(z0, z_bytes, x0, x_bytes) || overlaps(z0, z_bytes, a_any, a_bytes) ||
        overlaps(workspace, pl.total, x0, x_bytes) || overlaps(workspace, pl.total, z0, z_bytes) ||
        overlaps(workspace, pl.total, a_any, a_bytes) ||
        overlaps(token_mass, (size_t)n_img * t_e * 4, z0, z_bytes) ||
        overlaps(token_mass, (size_t)n_img * t_e * 4, workspace, pl.total) ||
        overlaps(device_status, 4, workspace, pl.total) || overlaps(device_status, 4, z0, z_bytes))
        return CIVIC_ERR_INVALID_ARG;

    cudaStream_t stream = (cudaStream_t)stream_;
    char* ws = (char*)workspace;
    char* prep = prepared ? (char*)const_cast<void*>(prepared) : ws;
    __nv_bfloat16* q = (__nv_bfloat16*)(prep + pl.q_off);
    float* qsum = (float*)(prep + pl.qsum_off);
    float2* stats = (float2*)(ws + pl.stats_off);
    __nv_bfloat16* p = (__nv_bfloat16*)(ws + pl.p_off);
    float* lpart = (float*)(ws + pl.lpart_off);
    float* inv_l = (float*)(ws + pl.invl_off);

    EncodeTiledFn enc = nullptr;
    const civic_status_t est = tensor_map_encoder(&enc);
    if (est != CIVIC_OK) return est;
    CUtensorMap map_q, map_x_scores, map_p, map_p_store, map_x_values;
    civic_status_t ms;
    {
        const uint64_t dims[2] = {(uint64_t)d_v, (uint64_t)m_e}, str[1] = {(uint64_t)d_v * 2};
        if ((ms = make_map(enc, &map_q, q, 2, dims, str, civic::kAggBM)) != CIVIC_OK) return ms;
    }
    {
        const uint64_t dims[3] = {(uint64_t)d_v, (uint64_t)t_e, (uint64_t)n_img};
        const uint64_t str[2] = {(uint64_t)d_v * 2, (uint64_t)t_e * d_v * 2};
        if ((ms = make_map(enc, &map_x_scores, x0, 3, dims, str, 128)) != CIVIC_OK) return ms;  // two boxes per stage
        if ((ms = make_map(enc, &map_x_values, x0, 3, dims, str, civic::kAggBK)) != CIVIC_OK) return ms;
    }
    {
        const uint64_t dims[3] = {(uint64_t)t_e, (uint64_t)m_e, (uint64_t)n_img};
        const uint64_t str[2] = {(uint64_t)pl.t_ld * 2, (uint64_t)m_e * pl.t_ld * 2};
        if ((ms = make_map(enc, &map_p, p, 3, dims, str, civic::kAggBM)) != CIVIC_OK) return ms;
        if ((ms = make_map(enc, &map_p_store, p, 3, dims, str, 32)) != CIVIC_OK) return ms;  // 32-row boxes written by a warp
    }

    const bool pdl = programmatic();
    const long long n_tokens = (long long)n_img * t_e;
    const int32_t prep_anchors = prepared ? 0 : m_e;  // prepared anchors: the launch takes the tokens only
    const int rows_per_warp = 32 / civic::kPrepLanes;
    const long long prep_warps = prep_anchors + (n_tokens + rows_per_warp - 1) / rows_per_warp;  // an anchor per warp
    CIVIC_CUDA_TRY(civic::launch(pdl, civic::aggregate_prep_kernel, (unsigned)((prep_warps + 7) / 8), 256u, 0,
                                 stream, anchors, prep_anchors, (const __nv_bfloat16*)x0, n_tokens, d_v, 1e-5f, 1e-12f, q,
                                 qsum, stats, (int*)device_status));  // also clears the status word

    const int32_t m_tiles = (m_e + civic::kAggBM - 1) / civic::kAggBM;
    civic::ScoresParams sp;
    sp.stats = stats; sp.qsum = qsum; sp.p = p; sp.lpart = lpart; sp.error = device_status;
    sp.m_e = m_e; sp.t_e = t_e; sp.d_v = d_v; sp.t_ld = pl.t_ld;
    sp.inv_tau_log2e = 1.4426950408889634f / tau;
    civic_status_t gs;
    if (m_tiles >= 2) {  // pairs of blocks share tiles of 256 anchors
        const int32_t m_pairs = (m_tiles + 1) / 2;
        sp.grid = civic::TileGrid{m_pairs, pl.n_tiles_t, n_img, m_pairs * pl.n_tiles_t * n_img};
        gs = launch_gemm<civic::ScoresPairOp>(map_q, map_x_scores, map_p_store, map_p_store, map_p_store, sp, sp.grid.total, stream);
    } else {
        sp.grid = civic::TileGrid{m_tiles, pl.n_tiles_t, n_img, m_tiles * pl.n_tiles_t * n_img};
        gs = launch_gemm<civic::ScoresOp>(map_q, map_x_scores, map_p_store, map_p_store, map_p_store, sp, sp.grid.total, stream);
    }
    if (gs != CIVIC_OK) return gs;
    civic::ValuesParams vp;
    vp.lpart = lpart; vp.z = (__nv_bfloat16*)z0; vp.inv_l = inv_l; vp.error = device_status;
    vp.m_e = m_e; vp.t_e = t_e; vp.d_v = d_v; vp.n_parts = 2 * pl.n_tiles_t; vp.t_ld = pl.t_ld;
    vp.mass_partial = token_mass ? (float*)(ws + pl.mass_off) : nullptr;
    vp.pw = (const __nv_bfloat16*)p;
    const int32_t f_tiles = (d_v + pl.values_bn - 1) / pl.values_bn;
    vp.grid = civic::TileGrid{m_tiles, f_tiles, n_img, m_tiles * f_tiles * n_img};
    if (pl.values_bn == 256) gs = launch_gemm<civic::ValuesOp<256>>(map_p, map_x_values, map_p, map_p, map_p, vp, vp.grid.total, stream);
    else if (pl.values_bn == 192) gs = launch_gemm<civic::ValuesOp<192>>(map_p, map_x_values, map_p, map_p, map_p, vp, vp.grid.total, stream);
    else gs = launch_gemm<civic::ValuesOp<128>>(map_p, map_x_values, map_p, map_p, map_p, vp, vp.grid.total, stream);
    if (gs != CIVIC_OK) return gs;
    int n_launched = 3;
    if (token_mass) {
        float* partial = (float*)(ws + pl.mass_off);
        CIVIC_CUDA_TRY(civic::launch(pdl, civic::token_mass_reduce_kernel, dim3((unsigned)((t_e + 63) / 64), (unsigned)n_img),
                                     64u, 0, stream, (const float*)partial, t_e, pl.t_ld, pl.n_panels, token_mass));
        n_launched += 1;
    }
    g_launches.fetch_add(n_launched, std::memory_order_relaxed);
    return CIVIC_OK;
}

civic_status_t civic_anchor_aggregate(const void* x0, const float* anchors, int32_t n_img, int32_t t_e,
                                      int32_t m_e, int32_t d_v, float tau, void* z0, float* token_mass,
                                      void* workspace, size_t workspace_bytes, int32_t* device_status,
                                      void* stream)
{
    if (!anchors && n_img > 0) return CIVIC_ERR_INVALID_ARG;
    return aggregate_impl(x0, anchors, nullptr, n_img, t_e, m_e, d_v, tau, z0, token_mass, workspace, workspace_bytes,
                          device_status, stream);
}

civic_status_t civic_anchor_aggregate_prepared(const void* x0, const void* prepared, int32_t n_img, int32_t t_e,
                                               int32_t m_e, int32_t d_v, float tau, void* z0, float* token_mass,
                                               void* workspace, size_t workspace_bytes, int32_t* device_status,
                                               void* stream)
{
    if (!prepared && n_img > 0) return CIVIC_ERR_INVALID_ARG;
    return aggregate_impl(x0, nullptr, prepared, n_img, t_e, m_e, d_v, tau, z0, token_mass, workspace, workspace_bytes,
                          device_status, stream);
}

// ---- KV-compressed visual attention (Eq. 9) -------------------------------------------------

struct KvAttnPlan {
    int32_t dim, compress_bn;
    int32_t d_pad, dim_ld;      // a head's columns in K_c / V_c (zero padded to a multiple of 16), all heads'
    int32_t kv_slots, q_slots, v_stream, n_buf;  // shared- and tensor-memory plan of the attention kernel
    int32_t n_parts;
    size_t r16_off, colsum_off, partial_off, kc_off, vc_off, total, attn_smem;
    size_t prepared_total;      // R in bf16 | column sums | panel sums: what civic_kv_attention_prepare writes
};

static civic_status_t plan_kv_attention(int32_t n_img, int32_t m_e, int32_t n_heads, int32_t head_dim, int32_t s,
                                        KvAttnPlan& pl)
{
    if (n_img < 0 || m_e < 1 || n_heads < 1 || head_dim < 1 || s < 1) return CIVIC_ERR_INVALID_ARG;
    if (head_dim % 8 || head_dim > 128 || s % 64 || s > 512 || n_img > 65535 || n_heads > 65535)
        return CIVIC_ERR_UNSUPPORTED;
    const int64_t dim = (int64_t)n_heads * head_dim;
    if (dim > (1 << 20)) return CIVIC_ERR_UNSUPPORTED;
    pl.dim = (int32_t)dim;
    pl.d_pad = (head_dim + 15) / 16 * 16;
    pl.dim_ld = n_heads * pl.d_pad;
    // shared memory, in order of preference: K_c and V_c of two pairs (the next pair loads while
    // this one runs) and three Q tiles in flight; fewer Q tiles; one pair; V_c streamed
    const int tries[7][3] = {{2, 3, 0}, {2, 2, 0}, {1, 3, 0}, {1, 2, 0}, {1, 1, 0}, {1, 2, 1}, {1, 1, 1}};
    pl.attn_smem = 0;
    for (const auto& t : tries) {
        const size_t bytes = civic::attn_smem_bytes(head_dim, pl.d_pad, s, t[0], t[1], t[2]);
        if (bytes <= kMaxDynamicSmem) {
            pl.kv_slots = t[0];
            pl.q_slots = t[1];
            pl.v_stream = t[2];
            pl.attn_smem = bytes;
            break;
        }
    }
    pl.n_buf = civic::attn_buffers(pl.d_pad, s);
    if (pl.attn_smem == 0) return CIVIC_ERR_UNSUPPORTED;
    // widest tile that divides the features; 128 before 192: only tiles whose halves are whole 64-column
    // boxes take the staged store (1152 features: 52.8 us per call with 192-wide tiles, 50.5 us with 128)
    pl.compress_bn = dim % 256 == 0 ? 256 : (dim % 128 == 0 ? 128 : (dim % 192 == 0 ? 192 : 128));
    size_t off = 0;
    auto take = [&off](size_t bytes) { const size_t at = off; off += round_up(bytes, 256); return at; };
    pl.r16_off = take((size_t)m_e * s * 2);
    pl.colsum_off = take((size_t)s * 4);
    pl.n_parts = (m_e + civic::kAssignRows - 1) / civic::kAssignRows;
    pl.partial_off = take((size_t)pl.n_parts * s * 4);
    pl.prepared_total = off;
    pl.kc_off = take((size_t)n_img * s * pl.dim_ld * 2);
    pl.vc_off = take((size_t)n_img * s * pl.dim_ld * 2);
    pl.total = off;
    return CIVIC_OK;
}

// R -> bf16 and its column sums into `prep` (laid out as the head of the plan's workspace).
// `reduce`: also add the panels' sums up (one more small launch), for a result that is kept.
static civic_status_t launch_assign_prepare(const float* r, int32_t m_e, int32_t s, const KvAttnPlan& pl, char* prep,
                                            bool reduce, int32_t* status_to_clear, cudaStream_t stream)
{
    const bool pdl = programmatic();
    CIVIC_CUDA_TRY(civic::launch(pdl, civic::assign_convert_kernel, (unsigned)pl.n_parts, (unsigned)s, 0, stream, r, m_e,
                                 s, (__nv_bfloat16*)(prep + pl.r16_off), (float*)(prep + pl.partial_off),
                                 (int*)status_to_clear));
    g_launches.fetch_add(1, std::memory_order_relaxed);
    if (reduce) {
        CIVIC_CUDA_TRY(civic::launch(pdl, civic::assign_colsum_kernel, (unsigned)((s + 127) / 128), 128u, 0, stream,
                                     (const float*)(prep + pl.partial_off), pl.n_parts, s, (float*)(prep + pl.colsum_off)));
        g_launches.fetch_add(1, std::memory_order_relaxed);
    }
    return CIVIC_OK;
}

// The compression GEMM and the attention kernel; r16 / colsum come from the caller's prepared
// buffer or were just written into the workspace (then colsum_parts holds n_parts panel sums).
static civic_status_t kv_attention_impl(const void* q, const void* k, const void* v, const float* r, const void* prepared,
                                        int32_t n_img, int32_t m_e, int32_t n_heads, int32_t head_dim, int32_t s,
                                        void* out, void* workspace, size_t workspace_bytes, int32_t* device_status,
                                        void* stream_)
{
    KvAttnPlan pl;
    const civic_status_t st = plan_kv_attention(n_img, m_e, n_heads, head_dim, s, pl);
    if (st != CIVIC_OK) return st;
    if (n_img == 0) return CIVIC_OK;
    if (!q || !k || !v || (!r && !prepared) || !out || !device_status) return CIVIC_ERR_INVALID_ARG;
    if (!aligned(q, 16) || !aligned(k, 16) || !aligned(v, 16) || !aligned(out, 16) || !aligned(r, 4) ||
        !aligned(prepared, 256) || !aligned(device_status, 4))
        return CIVIC_ERR_ALIGNMENT;
    if (!workspace || workspace_bytes < pl.total) return CIVIC_ERR_WORKSPACE;
    if (!aligned(workspace, 256)) return CIVIC_ERR_ALIGNMENT;
    const size_t x_bytes = (size_t)n_img * m_e * pl.dim * 2;
    const size_t r_bytes = r ? (size_t)m_e * s * 4 : pl.prepared_total;
    const void* r_any = r ? (const void*)r : prepared;
    if (overlaps(out, x_bytes, q, x_bytes) || overlaps(out, x_bytes, k, x_bytes) || overlaps(out, x_bytes, v, x_bytes) ||
        overlaps(out, x_bytes, r_any, r_bytes) || overlaps(workspace, pl.total, out, x_bytes) ||
        overlaps(workspace, pl.total, q, x_bytes) || overlaps(workspace, pl.total, k, x_bytes) ||
        overlaps(workspace, pl.total, v, x_bytes) || overlaps(workspace, pl.total, r_any, r_bytes) ||
        overlaps(device_status, 4, workspace, pl.total) || overlaps(device_status, 4, out, x_bytes))
        return CIVIC_ERR_INVALID_ARG;

    cudaStream_t stream = (cudaStream_t)stream_;
    char* ws = (char*)workspace;
    const char* prep = prepared ? (const char*)prepared : ws;
    const __nv_bfloat16* r16 = (const __nv_bfloat16*)(prep + pl.r16_off);
    __nv_bfloat16* kc = (__nv_bfloat16*)(ws + pl.kc_off);
    __nv_bfloat16* vc = (__nv_bfloat16*)(ws + pl.vc_off);

    EncodeTiledFn enc = nullptr;
    civic_status_t ms = tensor_map_encoder(&enc);
    if (ms != CIVIC_OK) return ms;
    CUtensorMap map_r, map_k_in, map_v_in, map_q, map_kc, map_vc, map_kc_out, map_vc_out, map_o, map_o_tail;
    {
        const uint64_t dims[2] = {(uint64_t)s, (uint64_t)m_e}, str[1] = {(uint64_t)s * 2};
        if ((ms = make_map(enc, &map_r, r16, 2, dims, str, 64)) != CIVIC_OK) return ms;
    }
    const int32_t tail = head_dim % 32;
    {
        const uint64_t dims[3] = {(uint64_t)pl.dim, (uint64_t)m_e, (uint64_t)n_img};
        const uint64_t str[2] = {(uint64_t)pl.dim * 2, (uint64_t)m_e * pl.dim * 2};
        if ((ms = make_map(enc, &map_k_in, k, 3, dims, str, 64)) != CIVIC_OK) return ms;
        if ((ms = make_map(enc, &map_v_in, v, 3, dims, str, 64)) != CIVIC_OK) return ms;
        if ((ms = make_map(enc, &map_q, q, 3, dims, str, civic::kAggBM)) != CIVIC_OK) return ms;
        // output boxes of 32 rows x 32 columns (what one softmax warp stages at a time), and the
        // head's last columns where its width is not a multiple of 32
        if ((ms = make_map(enc, &map_o, out, 3, dims, str, 32, 32)) != CIVIC_OK) return ms;
        if ((ms = make_map(enc, &map_o_tail, out, 3, dims, str, 32, tail ? (uint32_t)tail : 32u)) != CIVIC_OK) return ms;
    }
    {
        const uint64_t dims[3] = {(uint64_t)pl.dim_ld, (uint64_t)s, (uint64_t)n_img};
        const uint64_t str[2] = {(uint64_t)pl.dim_ld * 2, (uint64_t)s * pl.dim_ld * 2};
        if ((ms = make_map(enc, &map_kc, kc, 3, dims, str, 64)) != CIVIC_OK) return ms;
        if ((ms = make_map(enc, &map_vc, vc, 3, dims, str, 64)) != CIVIC_OK) return ms;
        // the compression's staged stores: 32 rows (one epilogue warp's anchors) x 64 columns
        if ((ms = make_map(enc, &map_kc_out, kc, 3, dims, str, 32)) != CIVIC_OK) return ms;
        if ((ms = make_map(enc, &map_vc_out, vc, 3, dims, str, 32)) != CIVIC_OK) return ms;
    }

    const int32_t q_tiles = (m_e + civic::kAggBM - 1) / civic::kAggBM;
    const int64_t total_tiles = (int64_t)q_tiles * n_heads * n_img;
    if (total_tiles > INT32_MAX) return CIVIC_ERR_UNSUPPORTED;
    civic::AttnParams ap;
    ap.error = device_status; ap.m_e = m_e; ap.s = s;
    ap.d = head_dim; ap.d_pad = pl.d_pad; ap.d_ld = pl.d_pad;
    ap.n_heads = n_heads; ap.q_tiles = q_tiles; ap.total_tiles = (int32_t)total_tiles;
    ap.n_buf = pl.n_buf; ap.kv_slots = pl.kv_slots; ap.q_slots = pl.q_slots; ap.v_stream = pl.v_stream;
    ap.scale_log2e = 1.4426950408889634f / sqrtf((float)head_dim);
    {
        static std::atomic<int> smem_allowed[64];
        const civic_status_t as = allow_dynamic_smem(civic::kv_attention_kernel, kMaxDynamicSmem, smem_allowed);
        if (as != CIVIC_OK) return as;
    }
    // persistent: one block per SM (a block holds up to all of an SM's tensor memory)
    const unsigned attn_blocks = (unsigned)std::min<int64_t>(total_tiles, sm_count());

    // everything that can fail on the host has happened: from here on work is enqueued
    const bool pdl = programmatic();
    civic::CompressParams cp;
    if (prepared) {  // no small kernel in front: a one-thread kernel clears the status word
        CIVIC_CUDA_TRY(civic::launch(pdl, civic::clear_status_kernel, 1u, 32u, 0, stream, (int*)device_status));
        g_launches.fetch_add(1, std::memory_order_relaxed);
        cp.colsum_parts = (const float*)(prep + pl.colsum_off);
        cp.n_parts = 1;
    } else {
        const civic_status_t as = launch_assign_prepare(r, m_e, s, pl, ws, false, device_status, stream);
        if (as != CIVIC_OK) return as;
        cp.colsum_parts = (const float*)(ws + pl.partial_off);
        cp.n_parts = pl.n_parts;
    }
    cp.error = device_status; cp.s = s; cp.m_e = m_e; cp.d_v = pl.dim;
    cp.head_dim = head_dim; cp.head_ld = pl.d_pad; cp.out_ld = pl.dim_ld;
    const int32_t s_tiles = (s + civic::kAggBM - 1) / civic::kAggBM;
    const int32_t f_tiles = (pl.dim + pl.compress_bn - 1) / pl.compress_bn;
    // K and V in one launch: the tile grid runs over 2 n_img "images"
    cp.grid = civic::TileGrid{s_tiles, f_tiles, 2 * n_img, s_tiles * f_tiles * 2 * n_img};
    cp.out = kc; cp.out_v = vc; cp.n_img = n_img;
    {
        civic_status_t gs;
        if (pl.compress_bn == 256) gs = launch_gemm<civic::CompressOp<256>>(map_r, map_k_in, map_v_in, map_kc_out, map_vc_out, cp, cp.grid.total, stream);
        else if (pl.compress_bn == 192) gs = launch_gemm<civic::CompressOp<192>>(map_r, map_k_in, map_v_in, map_kc_out, map_vc_out, cp, cp.grid.total, stream);
        else gs = launch_gemm<civic::CompressOp<128>>(map_r, map_k_in, map_v_in, map_kc_out, map_vc_out, cp, cp.grid.total, stream);
        if (gs != CIVIC_OK) return gs;
    }
    CIVIC_CUDA_TRY(civic::launch(pdl, civic::kv_attention_kernel, dim3(attn_blocks), (unsigned)civic::kAttnThreads,
                                 pl.attn_smem, stream, map_q, map_kc, map_vc, map_o, map_o_tail, ap));
    g_launches.fetch_add(2, std::memory_order_relaxed);
    return CIVIC_OK;
}

size_t civic_kv_compressed_attention_workspace_bytes(int32_t n_img, int32_t m_e, int32_t n_heads, int32_t head_dim,
                                                     int32_t s)
{
    KvAttnPlan pl;
    return plan_kv_attention(n_img, m_e, n_heads, head_dim, s, pl) == CIVIC_OK ? pl.total : 0;
}

civic_status_t civic_kv_compressed_attention(const void* q, const void* k, const void* v, const float* r,
                                             int32_t n_img, int32_t m_e, int32_t n_heads, int32_t head_dim,
                                             int32_t s, void* out, void* workspace, size_t workspace_bytes,
                                             int32_t* device_status, void* stream)
{
    if (!r && n_img > 0) return CIVIC_ERR_INVALID_ARG;
    return kv_attention_impl(q, k, v, r, nullptr, n_img, m_e, n_heads, head_dim, s, out, workspace, workspace_bytes,
                             device_status, stream);
}

size_t civic_kv_attention_prepared_bytes(int32_t m_e, int32_t s)
{
    KvAttnPlan pl;
    return plan_kv_attention(1, m_e, 1, 64, s, pl) == CIVIC_OK ? pl.prepared_total : 0;
}

civic_status_t civic_kv_attention_prepare(const float* r, int32_t m_e, int32_t s, void* prepared, size_t prepared_bytes,
                                          void* stream)
{
    KvAttnPlan pl;
    const civic_status_t st = plan_kv_attention(1, m_e, 1, 64, s, pl);
    if (st != CIVIC_OK) return st;
    if (!r || !prepared) return CIVIC_ERR_INVALID_ARG;
    if (!aligned(r, 4) || !aligned(prepared, 256)) return CIVIC_ERR_ALIGNMENT;
    if (prepared_bytes < pl.prepared_total) return CIVIC_ERR_WORKSPACE;
    if (overlaps(r, (size_t)m_e * s * 4, prepared, pl.prepared_total)) return CIVIC_ERR_INVALID_ARG;
    return launch_assign_prepare(r, m_e, s, pl, (char*)prepared, true, nullptr, (cudaStream_t)stream);
}

civic_status_t civic_kv_compressed_attention_prepared(const void* q, const void* k, const void* v, const void* prepared,
                                                      int32_t n_img, int32_t m_e, int32_t n_heads, int32_t head_dim,
                                                      int32_t s, void* out, void* workspace, size_t workspace_bytes,
                                                      int32_t* device_status, void* stream)
{
    if (!prepared && n_img > 0) return CIVIC_ERR_INVALID_ARG;
    return kv_attention_impl(q, k, v, nullptr, prepared, n_img, m_e, n_heads, head_dim, s, out, workspace,
                             workspace_bytes, device_status, stream);
}

civic_status_t civic_select_ragged(const float* scores, int32_t n_seg, const civic_select_desc_t* descs,
                                   int32_t* keep_idx, int32_t* flat_idx, void* stream)
{
    if (n_seg < 0 || (n_seg > 0 && !descs)) return CIVIC_ERR_INVALID_ARG;
    // validate every segment before anything is launched
    int64_t total_n = 0, total_k = 0;
    for (int s = 0; s < n_seg; ++s) {
        const civic_select_desc_t& d = descs[s];
        const int64_t n_res = reserved_count(d);
        if (n_res < 0) return CIVIC_ERR_INVALID_ARG;
        const int64_t n = (int64_t)d.t * d.h * d.w;
        if (n > civic_select_max_tokens()) return CIVIC_ERR_UNSUPPORTED;
        if (d.k < 0 || d.k > n) return CIVIC_ERR_K_RANGE;
        if (n_res > d.k) return CIVIC_ERR_FLOOR_EXCEEDS_K;
        total_n += n;
        total_k += d.k;
        if (total_n > INT32_MAX) return CIVIC_ERR_UNSUPPORTED;
    }
    if (total_k == 0) return CIVIC_OK;
    if (!scores || !keep_idx) return CIVIC_ERR_INVALID_ARG;
    if (!aligned(scores, 4) || !aligned(keep_idx, 4) || !aligned(flat_idx, 4)) return CIVIC_ERR_ALIGNMENT;
    if (overlaps(scores, (size_t)total_n * 4, keep_idx, (size_t)total_k * 4) ||
        overlaps(scores, (size_t)total_n * 4, flat_idx, (size_t)total_k * 4) ||
        overlaps(keep_idx, (size_t)total_k * 4, flat_idx, (size_t)total_k * 4))
        return CIVIC_ERR_INVALID_ARG;

    int32_t score_off = 0, out_off = 0;
    for (int s0 = 0; s0 < n_seg; s0 += civic::kMaxRaggedSegs) {
        const int ns = n_seg - s0 < civic::kMaxRaggedSegs ? n_seg - s0 : civic::kMaxRaggedSegs;
        civic::RaggedParams p;
        memset(&p, 0, sizeof p);
        p.scores = scores;
        p.keep_idx = keep_idx;
        p.flat_idx = flat_idx;
        int32_t n_max = 1;
        size_t smem_max = 0;
        for (int s = 0; s < ns; ++s) {
            const civic_select_desc_t& d = descs[s0 + s];
            const int32_t n = d.t * d.h * d.w;
            p.shape[s] = civic::SegShape{n, d.t, d.h, d.w, d.region_h, d.region_w, d.floor_per_region, d.k,
                                         (int32_t)(d.k - reserved_count(d)), select_floor_slots(d, n)};
            smem_max = std::max(smem_max, civic::select_smem_bytes(n, p.shape[s].floor_slots));
            p.score_off[s] = score_off;
            p.out_off[s] = out_off;
            score_off += n;
            out_off += d.k;
            n_max = n > n_max ? n : n_max;
        }
        const size_t smem = smem_max;
        {
            static std::atomic<int> smem_allowed[64];
            const civic_status_t as = allow_dynamic_smem(civic::select_ragged_kernel, kMaxDynamicSmem, smem_allowed);
            if (as != CIVIC_OK) return as;
        }
        CIVIC_CUDA_TRY(civic::launch(programmatic(), civic::select_ragged_kernel, (unsigned)ns,
                                     (unsigned)select_threads(n_max), smem, (cudaStream_t)stream, p));
        g_launches.fetch_add(1, std::memory_order_relaxed);
    }
    return CIVIC_OK;
}

int32_t civic_floor_from_ratio(int32_t region_h, int32_t region_w, int32_t num, int32_t den)
{
    if (region_h < 1 || region_w < 1 || num < 0 || den < 1 || num > den) return -1;
    const int64_t size = (int64_t)region_h * region_w;
    if (size > INT32_MAX) return -1;
    return (int32_t)((size * num + den - 1) / den);
}

size_t civic_select_workspace_bytes(const civic_select_desc_t* desc, int32_t n_seg, int32_t chunk_tokens)
{
    LargePlan pl;
    if (!desc || plan_large(*desc, n_seg, chunk_tokens, pl) != CIVIC_OK) return 0;
    return pl.total;
}

civic_status_t civic_select_large(const float* scores, int32_t n_seg, const civic_select_desc_t* desc,
                                  int32_t* keep_idx, void* workspace, size_t workspace_bytes,
                                  int32_t chunk_tokens, void* stream)
{
    if (!desc || n_seg < 0) return CIVIC_ERR_INVALID_ARG;
    const int64_t n_res = reserved_count(*desc);
    if (n_res < 0) return CIVIC_ERR_INVALID_ARG;
    const int64_t n = (int64_t)desc->t * desc->h * desc->w;
    if (n > INT32_MAX) return CIVIC_ERR_UNSUPPORTED;
    if (desc->k < 0 || desc->k > n) return CIVIC_ERR_K_RANGE;
    if (n_res > desc->k) return CIVIC_ERR_FLOOR_EXCEEDS_K;
    LargePlan pl;
    const civic_status_t st = plan_large(*desc, n_seg, chunk_tokens, pl);
    if (st != CIVIC_OK) return st;
    if (n_seg == 0 || desc->k == 0) return CIVIC_OK;
    if (!scores || !keep_idx) return CIVIC_ERR_INVALID_ARG;
    if (!aligned(scores, 4) || !aligned(keep_idx, 4)) return CIVIC_ERR_ALIGNMENT;
    if (!workspace || workspace_bytes < pl.total) return CIVIC_ERR_WORKSPACE;
    if (!aligned(workspace, 256)) return CIVIC_ERR_ALIGNMENT;
    if (overlaps(scores, (size_t)n_seg * n * 4, keep_idx, (size_t)n_seg * desc->k * 4) ||
        overlaps(workspace, pl.total, keep_idx, (size_t)n_seg * desc->k * 4) ||
        overlaps(workspace, pl.total, scores, (size_t)n_seg * n * 4))
        return CIVIC_ERR_INVALID_ARG;
    return launch_large(scores, n_seg, *desc, keep_idx, (char*)workspace, pl, (int32_t)(desc->k - n_res),
                        (cudaStream_t)stream, chunk_tokens == 0);
}

civic_status_t civic_compact(const void* hidden, size_t row_bytes, const int32_t* pos_ids,
                             const int32_t* keep_idx, int32_t n_seg, int32_t n, int32_t k,
                             void* hidden_out, int32_t* pos_out, void* stream)
{
    if (n_seg < 0 || n < 0 || k < 0) return CIVIC_ERR_INVALID_ARG;
    if (k > n) return CIVIC_ERR_K_RANGE;
    if ((hidden == nullptr) != (hidden_out == nullptr)) return CIVIC_ERR_INVALID_ARG;
    if ((pos_ids == nullptr) != (pos_out == nullptr)) return CIVIC_ERR_INVALID_ARG;
    if (hidden && (row_bytes == 0 || row_bytes > UINT32_MAX)) return CIVIC_ERR_INVALID_ARG;
    if (hidden && (row_bytes % 4 || !aligned(hidden, 4) || !aligned(hidden_out, 4)))
        return CIVIC_ERR_ALIGNMENT;
    if (!aligned(pos_ids, 4) || !aligned(pos_out, 4) || !aligned(keep_idx, 4)) return CIVIC_ERR_ALIGNMENT;
    if (n_seg == 0 || k == 0 || (!hidden && !pos_ids)) return CIVIC_OK;
    if (!keep_idx) return CIVIC_ERR_INVALID_ARG;
    const size_t in_rows = (size_t)n_seg * n, out_rows = (size_t)n_seg * k;
    if (overlaps(hidden, in_rows * row_bytes, hidden_out, out_rows * row_bytes) ||
        overlaps(pos_ids, in_rows * 12, pos_out, out_rows * 12) ||
        overlaps(keep_idx, out_rows * 4, hidden_out, out_rows * row_bytes) ||
        overlaps(keep_idx, out_rows * 4, pos_out, out_rows * 12))
        return CIVIC_ERR_INVALID_ARG;

    civic::GatherParams p;
    memset(&p, 0, sizeof p);
    p.n_tensors = hidden ? 1 : 0;
    p.src[0] = (const char*)hidden;
    p.dst[0] = (char*)hidden_out;
    p.idx = keep_idx;
    p.pos_src = pos_ids;
    p.pos_dst = pos_out;
    p.n_planes = n_seg; p.seq_len = n; p.s_out = k;
    p.idx_div = 1;
    p.row_bytes = hidden ? (uint32_t)row_bytes : 4;
    return launch_gather<civic::kPlain>(p, (cudaStream_t)stream);
}

civic_status_t civic_seq_indices(const int32_t* keep_idx, int32_t n_seq, int32_t k, int32_t seq_len,
                                 int32_t vis_start, int32_t n_vis, int32_t* seq_idx, void* stream)
{
    if (n_seq < 0 || k < 0 || seq_len < 0 || vis_start < 0 || n_vis < 0) return CIVIC_ERR_INVALID_ARG;
    if ((int64_t)vis_start + n_vis > seq_len) return CIVIC_ERR_INVALID_ARG;
    if (k > n_vis) return CIVIC_ERR_K_RANGE;
    const int64_t s_out = (int64_t)seq_len - n_vis + k;
    if (n_seq == 0 || s_out == 0) return CIVIC_OK;
    if (!seq_idx || (k > 0 && !keep_idx)) return CIVIC_ERR_INVALID_ARG;
    if (!aligned(seq_idx, 4) || !aligned(keep_idx, 4)) return CIVIC_ERR_ALIGNMENT;
    if (overlaps(keep_idx, (size_t)n_seq * k * 4, seq_idx, (size_t)n_seq * s_out * 4))
        return CIVIC_ERR_INVALID_ARG;
    const long long total = (long long)n_seq * s_out;
    const int threads = 256;
    long long blocks = (total + threads - 1) / threads;
    if (blocks > 4LL * sm_count()) blocks = 4LL * sm_count();
    CIVIC_CUDA_TRY(civic::launch(programmatic(), civic::seq_indices_kernel, (unsigned)blocks, threads, 0,
                                 (cudaStream_t)stream, keep_idx, seq_idx, n_seq, k, vis_start, n_vis,
                                 (int)s_out));
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return CIVIC_OK;
}

civic_status_t civic_compact_kv(const void* const* k_src, const void* const* v_src,
                                void* const* k_dst, void* const* v_dst, int32_t n_layers,
                                int32_t n_seq, int32_t seq_len, int32_t s_out, size_t row_bytes,
                                const int32_t* seq_idx, void* stream)
{
    if (n_layers < 0 || n_seq < 0 || seq_len < 0 || s_out < 0) return CIVIC_ERR_INVALID_ARG;
    if (s_out > seq_len) return CIVIC_ERR_K_RANGE;
    if (row_bytes == 0 || row_bytes > UINT32_MAX) return CIVIC_ERR_INVALID_ARG;
    if (row_bytes % 4) return CIVIC_ERR_ALIGNMENT;
    if (n_layers == 0 || n_seq == 0 || s_out == 0) return CIVIC_OK;
    if (!seq_idx) return CIVIC_ERR_INVALID_ARG;
    if (!aligned(seq_idx, 4)) return CIVIC_ERR_ALIGNMENT;
    const civic_status_t st =
        check_kv_tables(k_src, v_src, k_dst, v_dst, n_layers, (size_t)n_seq * seq_len * row_bytes,
                        (size_t)n_seq * s_out * row_bytes, seq_idx, (size_t)n_seq * s_out * 4);
    if (st != CIVIC_OK) return st;
    civic::GatherParams p;
    memset(&p, 0, sizeof p);
    p.idx = seq_idx;
    p.n_planes = n_seq; p.seq_len = seq_len; p.s_out = s_out;
    p.idx_div = 1;
    p.row_bytes = (uint32_t)row_bytes;
    return launch_kv<civic::kPlain>(p, k_src, v_src, k_dst, v_dst, n_layers, (cudaStream_t)stream);
}

civic_status_t civic_compact_kv_heads(const void* const* k_src, const void* const* v_src,
                                      void* const* k_dst, void* const* v_dst, int32_t n_layers,
                                      int32_t n_seq, int32_t n_heads, int32_t seq_len, int32_t s_out,
                                      size_t head_bytes, const int32_t* seq_idx, void* stream)
{
    if (n_layers < 0 || n_seq < 0 || n_heads < 0 || seq_len < 0 || s_out < 0) return CIVIC_ERR_INVALID_ARG;
    if (s_out > seq_len) return CIVIC_ERR_K_RANGE;
    if (head_bytes == 0 || head_bytes > UINT32_MAX) return CIVIC_ERR_INVALID_ARG;
    if (head_bytes % 4) return CIVIC_ERR_ALIGNMENT;
    if ((int64_t)n_seq * n_heads > INT32_MAX) return CIVIC_ERR_UNSUPPORTED;
    if (n_layers == 0 || n_seq == 0 || n_heads == 0 || s_out == 0) return CIVIC_OK;
    if (!seq_idx) return CIVIC_ERR_INVALID_ARG;
    if (!aligned(seq_idx, 4)) return CIVIC_ERR_ALIGNMENT;
    const size_t planes = (size_t)n_seq * n_heads;
    const civic_status_t st =
        check_kv_tables(k_src, v_src, k_dst, v_dst, n_layers, planes * seq_len * head_bytes,
                        planes * s_out * head_bytes, seq_idx, (size_t)n_seq * s_out * 4);
    if (st != CIVIC_OK) return st;
    civic::GatherParams p;
    memset(&p, 0, sizeof p);
    p.idx = seq_idx;
    p.n_planes = (int32_t)planes; p.seq_len = seq_len; p.s_out = s_out;
    p.idx_div = n_heads;
    p.row_bytes = (uint32_t)head_bytes;
    return launch_kv<civic::kHeads>(p, k_src, v_src, k_dst, v_dst, n_layers, (cudaStream_t)stream);
}

civic_status_t civic_compact_kv_paged(const void* const* k_src, const void* const* v_src,
                                      void* const* k_cache, void* const* v_cache, int32_t n_layers,
                                      int32_t n_seq, int32_t seq_len, int32_t s_out, size_t row_bytes,
                                      const int32_t* seq_idx, const int32_t* block_table,
                                      int32_t max_pages_per_seq, int32_t page_size, int32_t n_pages,
                                      void* stream)
{
    if (n_layers < 0 || n_seq < 0 || seq_len < 0 || s_out < 0 || max_pages_per_seq < 0 ||
        page_size < 1 || n_pages < 0)
        return CIVIC_ERR_INVALID_ARG;
    if (s_out > seq_len) return CIVIC_ERR_K_RANGE;
    if ((int64_t)max_pages_per_seq * page_size < s_out) return CIVIC_ERR_INVALID_ARG;
    if (row_bytes == 0 || row_bytes > UINT32_MAX) return CIVIC_ERR_INVALID_ARG;
    if (row_bytes % 4) return CIVIC_ERR_ALIGNMENT;
    if (n_layers == 0 || n_seq == 0 || s_out == 0) return CIVIC_OK;
    if (!seq_idx || !block_table) return CIVIC_ERR_INVALID_ARG;
    if (!aligned(seq_idx, 4) || !aligned(block_table, 4)) return CIVIC_ERR_ALIGNMENT;
    const size_t cache_bytes = (size_t)n_pages * page_size * row_bytes;
    civic_status_t st =
        check_kv_tables(k_src, v_src, k_cache, v_cache, n_layers, (size_t)n_seq * seq_len * row_bytes,
                        cache_bytes, seq_idx, (size_t)n_seq * s_out * 4);
    if (st != CIVIC_OK) return st;
    for (int l = 0; l < n_layers; ++l)
        if (overlaps(k_cache[l], cache_bytes, block_table, (size_t)n_seq * max_pages_per_seq * 4) ||
            overlaps(v_cache[l], cache_bytes, block_table, (size_t)n_seq * max_pages_per_seq * 4))
            return CIVIC_ERR_INVALID_ARG;
    civic::GatherParams p;
    memset(&p, 0, sizeof p);
    p.idx = seq_idx;
    p.n_planes = n_seq; p.seq_len = seq_len; p.s_out = s_out;
    p.idx_div = 1;
    p.row_bytes = (uint32_t)row_bytes;
    p.block_table = block_table;
    p.max_pages = max_pages_per_seq;
    p.page_size = page_size;
    p.n_pages = n_pages;
    return launch_kv<civic::kPaged>(p, k_src, v_src, k_cache, v_cache, n_layers, (cudaStream_t)stream);
}

civic_status_t civic_merge_embeddings(const void* text, const void* visual, size_t row_bytes,
                                      const int32_t* keep_idx, int32_t n_seq, int32_t seq_len,
                                      int32_t vis_start, int32_t n_vis, int32_t k, void* merged,
                                      void* stream)
{
    if (n_seq < 0 || seq_len < 0 || vis_start < 0 || n_vis < 0 || k < 0) return CIVIC_ERR_INVALID_ARG;
    if ((int64_t)vis_start + n_vis > seq_len) return CIVIC_ERR_INVALID_ARG;
    if (k > n_vis) return CIVIC_ERR_K_RANGE;
    if (row_bytes == 0 || row_bytes > UINT32_MAX) return CIVIC_ERR_INVALID_ARG;
    const int64_t s_out = (int64_t)seq_len - n_vis + k;
    if (n_seq == 0 || s_out == 0) return CIVIC_OK;
    if (!text || !merged || (k > 0 && (!visual || !keep_idx))) return CIVIC_ERR_INVALID_ARG;
    if (row_bytes % 4 || !aligned(text, 4) || !aligned(visual, 4) || !aligned(merged, 4) ||
        !aligned(keep_idx, 4))
        return CIVIC_ERR_ALIGNMENT;
    const size_t out_bytes = (size_t)n_seq * s_out * row_bytes;
    if (overlaps(merged, out_bytes, text, (size_t)n_seq * seq_len * row_bytes) ||
        overlaps(merged, out_bytes, visual, (size_t)n_seq * n_vis * row_bytes) ||
        overlaps(merged, out_bytes, keep_idx, (size_t)n_seq * k * 4))
        return CIVIC_ERR_INVALID_ARG;
    civic::GatherParams p;
    memset(&p, 0, sizeof p);
    p.n_tensors = 1;
    p.src[0] = (const char*)text;
    p.dst[0] = (char*)merged;
    p.idx = keep_idx;
    p.n_planes = n_seq; p.seq_len = seq_len; p.s_out = (int32_t)s_out;
    p.idx_div = 1;
    p.row_bytes = (uint32_t)row_bytes;
    p.visual = (const char*)visual;
    p.vis_start = vis_start; p.n_vis = n_vis; p.k_vis = k;
    return launch_gather<civic::kMerge>(p, (cudaStream_t)stream);
}

civic_status_t civic_compact_pos_planes(const int32_t* pos, int32_t n_planes, int32_t n_seq,
                                        int32_t seq_len, const int32_t* seq_idx, int32_t s_out,
                                        int32_t* pos_out, void* stream)
{
    if (n_planes < 0 || n_seq < 0 || seq_len < 0 || s_out < 0) return CIVIC_ERR_INVALID_ARG;
    if (s_out > seq_len) return CIVIC_ERR_K_RANGE;
    const long long total = (long long)n_planes * n_seq * s_out;
    if (total == 0) return CIVIC_OK;
    if (!pos || !seq_idx || !pos_out) return CIVIC_ERR_INVALID_ARG;
    if (!aligned(pos, 4) || !aligned(seq_idx, 4) || !aligned(pos_out, 4)) return CIVIC_ERR_ALIGNMENT;
    if (overlaps(pos_out, (size_t)total * 4, pos, (size_t)n_planes * n_seq * seq_len * 4) ||
        overlaps(pos_out, (size_t)total * 4, seq_idx, (size_t)n_seq * s_out * 4))
        return CIVIC_ERR_INVALID_ARG;
    const int threads = 256;
    long long blocks = (total + threads - 1) / threads;
    if (blocks > 8LL * sm_count()) blocks = 8LL * sm_count();
    CIVIC_CUDA_TRY(civic::launch(programmatic(), civic::gather_pos_planes_kernel, (unsigned)blocks, threads, 0,
                                 (cudaStream_t)stream, pos, seq_idx, pos_out, n_planes, n_seq, seq_len,
                                 s_out, g_index_check));
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return CIVIC_OK;
}

civic_status_t civic_set_index_check(int32_t* fault_record)
{
    if (!aligned(fault_record, 4)) return CIVIC_ERR_ALIGNMENT;
    g_index_check = fault_record;
    return CIVIC_OK;
}

civic_status_t civic_validate_indices(const int32_t* idx, int32_t n_rows, int32_t row_len, int32_t limit,
                                      int32_t require_ascending, int32_t* fault_record, void* stream)
{
    if (n_rows < 0 || row_len < 0 || limit < 0) return CIVIC_ERR_INVALID_ARG;
    const long long total = (long long)n_rows * row_len;
    if (total == 0) return CIVIC_OK;
    if (!idx || !fault_record) return CIVIC_ERR_INVALID_ARG;
    if (!aligned(idx, 4) || !aligned(fault_record, 4)) return CIVIC_ERR_ALIGNMENT;
    if (overlaps(idx, (size_t)total * 4, fault_record, 16)) return CIVIC_ERR_INVALID_ARG;
    const int threads = 256;
    long long blocks = (total + threads - 1) / threads;
    if (blocks > 8LL * sm_count()) blocks = 8LL * sm_count();
    CIVIC_CUDA_TRY(civic::launch(programmatic(), civic::validate_indices_kernel, (unsigned)blocks, threads, 0,
                                 (cudaStream_t)stream, idx, n_rows, row_len, limit, require_ascending, fault_record));
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return CIVIC_OK;
}

civic_status_t civic_selftest_bounded_wait(uint64_t limit_cycles, int32_t* record, void* stream)
{
    if (!record || limit_cycles == 0 || limit_cycles > ((uint64_t)1 << 24)) return CIVIC_ERR_INVALID_ARG;
    if (!aligned(record, 4)) return CIVIC_ERR_ALIGNMENT;
    CIVIC_CUDA_TRY(cudaMemsetAsync(record, 0, 8, (cudaStream_t)stream));
    CIVIC_CUDA_TRY(civic::launch(programmatic(), civic::bounded_wait_selftest_kernel, 1u, 64u, 0, (cudaStream_t)stream,
                                 (unsigned long long)limit_cycles, (int*)record));
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return CIVIC_OK;
}

}  // extern "C"
