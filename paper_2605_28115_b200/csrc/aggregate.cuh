// Compact visual aggregation (Eq. 8 of the paper) on the 5th-generation tensor cores:
//
//     K_0 = Norm(LN(X_0)),  Q_A = Norm(LN(A)),  W_A = softmax(Q_A K_0^T / tau),  Z_0 = W_A X_0
//
// Algebra used (exact in real arithmetic): LN's 1/sqrt(var + eps) cancels under the l2
// normalisation, so K_0[i] = r_i (x_i - mu_i 1) with r_i = 1 / ||x_i - mu_i 1||, and
//     Q_A[m] . K_0[i] = r_i (Q_A[m] . x_i  -  mu_i * sum_j Q_A[m, j]).
// The first contraction therefore runs on the RAW tokens; normalising them costs two scalars per
// token (mu_i, r_i) that the epilogue applies, and one scalar per anchor (the exact sum of its
// bf16-rounded row).  Cosines are bounded by 1, so the softmax needs no running maximum:
// P = exp((s - 1) / tau) cannot overflow and, for tau >= 0.025, cannot underflow bf16.
//
// Kernels
//   aggregate_prep_kernel   A (fp32) -> Q_A (bf16) and the row sums of the rounded values, a warp per
//                           anchor; X_0 (bf16) -> (mu_i, r_i), eight lanes per token; HBM-bound
//   aggregate_gemm_kernel<ScoresOp>   tcgen05 GEMM  S = Q_A X_0^T  (both operands K-major), epilogue
//                           P = exp((r (S - mu qsum) - 1) / tau) as bf16 + partial row sums
//   aggregate_gemm_kernel<ValuesOp>   tcgen05 GEMM  Z_0 = (P X_0) / l  (A = P K-major, B = X_0 MN-major);
//                           four side warps add up the columns of W_A = P / l by panels of 32 anchors
//   token_mass_reduce_kernel   adds those panels: the per-token importance
//
// GEMM skeleton (both): persistent blocks of 320 threads (448 with side warps), one per SM.  Warp 0 =
// TMA producer (one elected lane), warp 1 = TMEM allocation + MMA issue (one elected lane), warps
// 2..9 = epilogue (each reads its own quarter of the 128 TMEM lanes), warps 10..13 = side warps of
// an Op that has them.  Operand tiles arrive by
// cp.async.bulk.tensor with 128-byte swizzle into a ring of stages guarded by full/empty
// mbarriers; two accumulators alternate in TMEM so the epilogue overlaps the next tile's MMAs.
// The score GEMM runs on pairs of blocks (cta_group::2): with both operands in shared memory a
// single block has to take in and hand out 187 bytes per clock for a 128 x 256 tile, more than
// shared memory delivers; the pair halves the B traffic.
// Every wait is bounded: on a time-out the thread raises the kernel's error word, the block
// stops issuing work, waits (bounded) for its copies in flight, frees its TMEM and returns.
#pragma once
#include <cstdint>
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "pdl.cuh"

namespace civic {

constexpr int kAggThreads = 320;      // producer warp, MMA warp, eight epilogue warps (an Op's side warps come on top)
constexpr int kAggBM = 128;           // anchors per tile (TMEM lanes)
constexpr int kAggBK = 64;            // 64 bf16 = one 128-byte swizzle row
constexpr int kScoresBN = 256;        // tokens per tile of the first GEMM
constexpr unsigned long long kWaitLimitCycles = 1ull << 31;  // about a second

enum AggError { kAggOk = 0, kAggTimeoutFull = 1, kAggTimeoutEmpty = 2, kAggTimeoutAcc = 3, kAggMisaligned = 4 };

// ----------------------------------------------------------------------------- PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when the block has been told to stop (*abort != 0) or the limit
// (SM cycles) ran out, in which case it also raises *abort and records `code` in the kernel's
// error word.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort, int* error, int code,
                                          unsigned long long limit = kWaitLimitCycles)
{
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort) return false;
        if ((unsigned long long)(clock64() - t0) > limit) {
            *abort = 1;
            atomicCAS(error, 0, code);
            return false;
        }
    }
}
__device__ __forceinline__ void fence_barrier_init()
{
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, int x, int y, int z, uint64_t* bar)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t cols)  // whole warp
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t cols)  // whole warp
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] B[smem], bf16 operands, fp32 accumulator, one CTA.
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.u32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n"
        ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// One lane of a converged warp (the same one every time).
__device__ __forceinline__ bool elect_one()
{
    uint32_t chosen;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "elect.sync _|p, 0xFFFFFFFF;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(chosen));
    return chosen != 0;
}
// The mbarrier gets one arrival once every MMA issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// ---- bulk tensor store of a shared-memory box (one thread issues; OOB parts of the box are clipped)
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tma_store_3d(const CUtensorMap* map, const void* src, int x, int y, int z)
{
    asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.bulk_group [%0, {%1, %2, %3}], [%4];"
                 ::"l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(src)) : "memory");
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
}
// the issuing thread's earlier stores have finished READING shared memory (it may be overwritten)
__device__ __forceinline__ void tma_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// the issuing thread's earlier stores are complete (written)
__device__ __forceinline__ void tma_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// ---- two blocks of a cluster working as one MMA unit (cta_group::2).  Block rank 0 (the leader)
// issues the MMAs; every block loads its half of the operands into its own shared memory, but all
// transaction bytes are counted on the LEADER's "full" barrier; the leader's commits arrive on
// the barriers of both blocks (multicast of the commit signal only, never of a load).
__device__ __forceinline__ uint32_t cluster_ctarank()
{
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_sync()  // all threads of both blocks
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// shared::cluster address of `p` (a shared-memory object of this block) in the block of rank `rank`
__device__ __forceinline__ uint32_t cluster_address(const void* p, uint32_t rank)
{
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_u32(p)), "r"(rank));
    return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr)
{
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ void tma_load_2d_pair(void* dst, const CUtensorMap* map, int x, int y, uint32_t bar_cluster_addr)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(void* dst, const CUtensorMap* map, int x, int y, int z, uint32_t bar_cluster_addr)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(smem_u32(dst)), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t* slot, uint32_t cols)  // the same warp of both blocks
{
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t cols)
{
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// D (256 rows: 128 in each block's TMEM) (+)= A (128 rows from each block) B (N / 2 columns from each block)
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate)
{
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.u32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n"
        ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// one arrival on the barrier at this shared-memory offset in BOTH blocks, once the MMAs issued so far are done
__device__ __forceinline__ void umma_commit_pair(uint64_t* bar)
{
    const uint16_t both = 3;
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(smem_u32(bar)), "h"(both) : "memory");
}

// Shared-memory operand descriptor, 128-byte swizzle, tile base 1024-byte aligned.
//   K-major  (rows of 64 bf16 = 128 B): 8-row groups 1024 B apart (stride offset); the leading
//             offset is unused with swizzling (set to one 16-byte unit).
//   MN-major (the 64 contiguous elements run along M or N): 8 K-rows of 128 B form a group,
//             groups 1024 B apart (stride offset); the next 64 elements along M/N start
//             `leading_bytes` further on.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr, uint32_t leading_bytes, uint32_t stride_bytes)
{
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr >> 4) & 0x3FFFu);
    d |= (uint64_t)((leading_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((stride_bytes >> 4) & 0x3FFFu) << 32;
    d |= 1ull << 46;  // descriptor version of this architecture
    d |= 2ull << 61;  // 128-byte swizzle
    return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = m (128, or 256 for a pair of blocks), N = n;
// a_mn_major / b_mn_major = 1 when the operand's contiguous dimension is M / N rather than K.
__host__ __device__ constexpr uint32_t umma_idesc(int n, int b_mn_major, int m = kAggBM, int a_mn_major = 0)
{
    return (1u << 4)                      // accumulator fp32
           | (1u << 7) | (1u << 10)       // A, B bf16
           | ((uint32_t)a_mn_major << 15) // A major
           | ((uint32_t)b_mn_major << 16) // B major
           | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// ----------------------------------------------------------------------------- small kernels

// Both preparations in one launch.  Warps [0, m_e) take an anchor each: Q_A = Norm(LN(A)) rounded
// to bf16, and qsum[m] = sum of the ROUNDED row (what the tensor core will really multiply the token
// mean with).  The other warps take 32 / kPrepLanes tokens each: (mu_i, r_i) with
// K_0[i] = r_i (x_i - mu_i), r_i = 0 for a token whose features are all equal.  Few registers on
// purpose: the token part is HBM-bound and lives on occupancy (a version that held the whole row in
// registers measured slower).
__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, d);
    return v;
}

// scale such that Norm(LN(row)) = (row - mean) * scale; 0 when the row has no direction
__device__ __forceinline__ float normalise_scale(float ss, int d_v, float ln_eps, float norm_eps)
{
    const float inv_std = rsqrtf(ss / d_v + ln_eps);
    const float norm = sqrtf(ss) * inv_std;  // l2 norm of the layer-normalised row
    return ss > 0.f ? inv_std / fmaxf(norm, norm_eps) : 0.f;
}

// Token part: lanes per row and 16-byte loads in flight per lane.  Measured on 32768 rows of 1152 bf16
// (75 MB), us: 32 lanes x 5 loads 17.8 - 25.8, 16 x 5 17.1, 16 x 9 15.7, 8 x 6 13.0 (5.8 TB/s), 8 x 18 13.0,
// 4 x 9 16.0, 2 x 9 21.5.
constexpr int kPrepLanes = 8;
constexpr int kPrepUnroll = 6;
__global__ void __launch_bounds__(256) aggregate_prep_kernel(const float* __restrict__ anchors, int m_e,
                                                             const __nv_bfloat16* __restrict__ x, long long n_tokens,
                                                             int d_v, float ln_eps, float norm_eps,
                                                             __nv_bfloat16* __restrict__ q, float* __restrict__ qsum,
                                                             float2* __restrict__ stats, int* __restrict__ status)
{
    wait_for_prior_kernels();
    if (status && blockIdx.x == 0 && threadIdx.x == 0) *status = 0;  // the call's status word starts clean
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (warp < m_e) {
        // ---- anchor row (fp32): three passes, the row stays in L1
        const float* a = anchors + warp * d_v;
        float s = 0.f;
        for (int j = lane; j < d_v; j += 32) s += a[j];
        const float mean = warp_sum(s) / d_v;
        float ss = 0.f;
        for (int j = lane; j < d_v; j += 32) { const float c = a[j] - mean; ss += c * c; }
        const float scale = normalise_scale(warp_sum(ss), d_v, ln_eps, norm_eps);
        float rounded_sum = 0.f;
        for (int j = lane; j < d_v; j += 32) {
            const __nv_bfloat16 v = __float2bfloat16_rn((a[j] - mean) * scale);
            q[warp * d_v + j] = v;
            rounded_sum += __bfloat162float(v);
        }
        rounded_sum = warp_sum(rounded_sum);
        if (lane == 0) qsum[warp] = rounded_sum;
        return;
    }
    // ---- token rows (bf16, d_v a multiple of 8): kPrepLanes lanes per row, so that a warp's fixed work
    // (the two reductions, the normalisation, the addressing: 40 % of its instructions with a row per
    // warp, and the pass was bound by instruction issue at 45 % of the DRAM rate) serves four rows, and
    // no lane idles in a last partial iteration (1152 features are 4.5 loads of 16 bytes per lane of a
    // whole warp).  Sums are taken relative to the row's first element so that the variance keeps its
    // accuracy.
    const long long tok_first = (warp - m_e) * (32 / kPrepLanes);
    if (tok_first >= n_tokens) return;  // the whole warp: nothing below touches x without a token (x may be null)
    const long long tok = tok_first + lane / kPrepLanes;
    const bool tok_ok = tok < n_tokens;  // past the end: the warp's first row again, not stored
    const int l16 = lane % kPrepLanes;
    const int vecs = d_v >> 3;
    const uint4* row = reinterpret_cast<const uint4*>(x + (tok_ok ? tok : tok_first) * d_v);
    const float shift = __bfloat162float(x[(tok_ok ? tok : tok_first) * d_v]);
    float s = 0.f, s2 = 0.f;
#pragma unroll kPrepUnroll
    for (int v = l16; v < vecs; v += kPrepLanes) {
        const uint4 u = __ldg(row + v);
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const float2 f = __bfloat1622float2(h[e]);
            const float a = f.x - shift, b = f.y - shift;
            s += a + b;
            s2 += a * a + b * b;
        }
    }
#pragma unroll
    for (int d = kPrepLanes / 2; d > 0; d >>= 1) {  // within the row's lanes
        s += __shfl_xor_sync(0xFFFFFFFFu, s, d);
        s2 += __shfl_xor_sync(0xFFFFFFFFu, s2, d);
    }
    if (l16 == 0 && tok_ok) {
        const float mean_shifted = s / d_v;
        const float ss = fmaxf(s2 - s * mean_shifted, 0.f);  // sum (x - mu)^2
        stats[tok] = make_float2(mean_shifted + shift, normalise_scale(ss, d_v, ln_eps, norm_eps));
    }
}

// ----------------------------------------------------------------------------- the two GEMMs
//
// One persistent kernel template: a block walks tiles t = blockIdx.x, blockIdx.x + gridDim.x, ...
// with the anchor tile fastest, so blocks that run at the same time share their X_0 tile in L2.
// Two TMEM accumulators alternate between tiles: the epilogue warps drain one while the MMA thread
// already fills the other.  `Op` supplies the tile width, how a stage is loaded, B's descriptor
// and the epilogue.  Eight epilogue warps: two per TMEM lane quarter, each taking half of the
// tile's columns (one warp per scheduler cannot hide its own latencies; measured 14 us per
// 128 x 256 tile with four warps against 6.7 us of MMA time).

struct TileGrid {
    int32_t m_tiles, n_tiles, n_img, total;
};

__device__ __forceinline__ void tile_coords(const TileGrid& g, int t, int& m_tile, int& n_tile, int& img)
{
    m_tile = t % g.m_tiles;
    const int rest = t / g.m_tiles;
    n_tile = rest % g.n_tiles;
    img = rest / g.n_tiles;
}

// One unit of work of a worker (a block, or a pair of blocks).
struct Tile {
    int m_tile;  // anchor tile of the worker: 128 anchors per block
    int n0, n;   // first column and width of the tile (tokens for the scores, features for the values)
    int n_tile;  // column tile number
    int img;
};

// i-th tile of a worker, tiles of one width dealt out round-robin
__device__ __forceinline__ bool round_robin_tile(const TileGrid& g, int width, int worker, int n_workers, int i, Tile& tl)
{
    const int t = worker + i * n_workers;
    if (t >= g.total) return false;
    tile_coords(g, t, tl.m_tile, tl.n_tile, tl.img);
    tl.n0 = tl.n_tile * width;
    tl.n = width;
    return true;
}

__device__ __forceinline__ void mbar_arrive(uint64_t* bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// 32 consecutive fp32 columns of this warp's 32 TMEM lanes (thread t gets lane base + t), split
// into issue and wait, so that the next chunk's load runs under the current
// chunk's arithmetic.  The wait names the registers as in/out operands: nothing that uses them
// can be scheduled above it.
__device__ __forceinline__ void tmem_load_issue(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_load_wait(uint32_t (&r)[32])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                   "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]),
                   "+r"(r[16]), "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]),
                   "+r"(r[24]), "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
                 :: "memory");
}
__device__ __forceinline__ float exp2_fast(float x)
{
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Walks the `cols` (a multiple of 32) accumulator columns of one warp in chunks of 32 with two
// register buffers; `body(acc, c0)` consumes chunk c0.
template <class Body>
__device__ __forceinline__ void for_each_chunk(uint32_t taddr, int cols, Body&& body)
{
    uint32_t even[32], odd[32];
    tmem_load_issue(taddr, even);
#pragma unroll 1
    for (int c0 = 0; c0 < cols; c0 += 64) {
        tmem_load_wait(even);
        if (c0 + 32 < cols) tmem_load_issue(taddr + c0 + 32, odd);
        body(even, c0);
        if (c0 + 32 < cols) {
            tmem_load_wait(odd);
            if (c0 + 64 < cols) tmem_load_issue(taddr + c0 + 64, even);
            body(odd, c0 + 32);
        }
    }
}

struct ScoresParams {
    const float2* stats;    // [n_img, t_e]  (mu, r)
    const float* qsum;      // [m_e]
    __nv_bfloat16* p;       // [n_img, m_e, t_ld]
    float* lpart;           // [n_img, m_e, 2 * n_tiles_t] partial row sums of the rounded P
    int* error;             // kernel error word (0 = fine)
    TileGrid grid;
    int32_t m_e, t_e, d_v, t_ld;
    float inv_tau_log2e;    // log2(e) / tau
};

struct ValuesParams {
    const float* lpart;   // [n_img, m_e, n_parts]
    __nv_bfloat16* z;     // [n_img, m_e, d_v]
    float* inv_l;         // [n_img, m_e] written by the blocks of the first feature tile
    float* mass_partial;  // [n_img, 4 m_tiles, t_ld] column sums of W_A by panels of 32 anchors, or null
    const __nv_bfloat16* pw;  // [n_img, m_e, t_ld] P as global memory, for the side warps
    int* error;
    TileGrid grid;
    int32_t m_e, t_e, d_v, n_parts, t_ld;
};

constexpr int kEpilogueWarps = 8;

template <int BN_, int STAGES_, bool SCORES_, bool STAGING_ = SCORES_>
struct alignas(1024) GemmSmem {
    __nv_bfloat16 a[STAGES_][kAggBM * kAggBK];  // 128 rows x 128 B, K-major
    __nv_bfloat16 b[STAGES_][BN_ * kAggBK];
    uint8_t out[STAGING_ ? kEpilogueWarps : 1][STAGING_ ? 32 * 128 : 1024];  // per epilogue warp: 32 rows x 64 bf16, 128-byte swizzled,
                                                // for the bulk store of a result (scores, compression)
    float2 stats[SCORES_ ? kEpilogueWarps : 1][128];  // per epilogue warp: (mu, r log2e / tau) of its columns (scores only)
    float side_w[4][32];  // per side warp: 1 / l of its 32 anchor rows (values only)
    uint64_t full[STAGES_], empty[STAGES_], acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    int abort;
};

// S = Q_A X_0^T, K = features, both operands K-major.
//   PAIR = false: one block per tile of 128 anchors x 256 tokens.
//   PAIR = true:  two blocks of a cluster share a tile of 256 anchors x 256 tokens; each loads its
//                 own 128 anchors and HALF of the tokens, so a block moves 32 KB per K step
//                 instead of 48 KB for the same arithmetic (the one-block kernel is bound by the
//                 bytes it can keep in flight, not by the tensor pipe).
template <bool PAIR>
struct ScoresOpT {
    static constexpr int BN = 256, STAGES = PAIR ? 5 : 3, kCtas = PAIR ? 2 : 1, kSideWarps = 0;
    static constexpr bool kAMnMajor = false, kBMnMajor = false;
    using Params = ScoresParams;
    using Smem = GemmSmem<PAIR ? 128 : 256, STAGES, true>;
    static constexpr uint32_t kStageBytes = (kAggBM + (PAIR ? 128 : 256)) * kAggBK * 2;  // per block
    static __device__ __forceinline__ int k_steps(const Params& p) { return p.d_v / kAggBK; }
    static __device__ __forceinline__ bool tile(const Params& p, int worker, int n_workers, int i, Tile& tl)
    {
        return round_robin_tile(p.grid, BN, worker, n_workers, i, tl);
    }
    // m0: this block's first anchor; rank: block rank in the pair
    static __device__ __forceinline__ void load(const Params&, Smem& sm, int s, const CUtensorMap* map_a,
                                                const CUtensorMap* map_b, const CUtensorMap*, int k, int m0,
                                                const Tile& tl, uint32_t rank, uint32_t leader_full)
    {
        const int n0 = tl.n0, img = tl.img;
        if constexpr (PAIR) {
            if (rank == 0) mbar_expect_tx(&sm.full[s], 2 * kStageBytes);  // both blocks' bytes
            tma_load_2d_pair(sm.a[s], map_a, k * kAggBK, m0, leader_full);
            tma_load_3d_pair(sm.b[s], map_b, k * kAggBK, n0 + 128 * (int)rank, img, leader_full);
        } else {
            mbar_expect_tx(&sm.full[s], kStageBytes);
            tma_load_2d(sm.a[s], map_a, k * kAggBK, m0, &sm.full[s]);
            tma_load_3d(sm.b[s], map_b, k * kAggBK, n0, img, &sm.full[s]);                        // tokens n0 ..
            tma_load_3d(sm.b[s] + 128 * kAggBK, map_b, k * kAggBK, n0 + 128, img, &sm.full[s]);  // .. + 128
        }
    }
    static __device__ __forceinline__ uint64_t a_desc(uint32_t a0, int kk) { return umma_desc(a0 + kk * 32, 16, 1024); }
    static __device__ __forceinline__ uint64_t b_desc(uint32_t b0, int kk) { return umma_desc(b0 + kk * 32, 16, 1024); }

    // P = 2^(r' (acc - mu qsum) - c) for 32 columns of one anchor row, r' = r c, c = log2(e) / tau;
    // MASK: columns at or beyond n_valid are tokens past the end of the image and give 0.
    template <bool MASK>
    static __device__ __forceinline__ void chunk(const uint32_t (&acc)[32], const float2* st, float qs, float neg_c,
                                                 int n_valid, float& row_sum, uint32_t (&packed)[16])
    {
#pragma unroll
        for (int c = 0; c < 32; c += 2) {
            const float2 s0 = st[c], s1 = st[c + 1];
            float v0 = exp2_fast(fmaf(s0.y, fmaf(-s0.x, qs, __uint_as_float(acc[c])), neg_c));
            float v1 = exp2_fast(fmaf(s1.y, fmaf(-s1.x, qs, __uint_as_float(acc[c + 1])), neg_c));
            if (MASK) {
                v0 = c < n_valid ? v0 : 0.f;
                v1 = c + 1 < n_valid ? v1 : 0.f;
            }
            const __nv_bfloat162 h = __floats2bfloat162_rn(v0, v1);
            row_sum += __low2float(h) + __high2float(h);
            packed[c >> 1] = *reinterpret_cast<const uint32_t*>(&h);
        }
    }

    // Before the accumulator is waited for: the (mu, r log2e / tau) of this warp's 128 token
    // columns go to the warp's private shared-memory copy (no barrier between warps).
    static __device__ __forceinline__ void prefetch(const Params& p, Smem& sm, int ewarp, int lane, const Tile& tl)
    {
        const int img = tl.img;
        const int nh = tl.n0 + (ewarp >> 2) * 128;
        float2* stats = sm.stats[ewarp];
        __syncwarp();
#pragma unroll
        for (int c = lane; c < 128; c += 32) {
            const int tok = nh + c;
            float2 st = tok < p.t_e ? p.stats[(size_t)img * p.t_e + tok] : make_float2(0.f, 0.f);
            st.y *= p.inv_tau_log2e;
            stats[c] = st;
        }
        __syncwarp();
    }

    // thread = one anchor row of one half (128 token columns) of the tile.  The weights leave
    // through shared memory and a bulk tensor store, 32 rows x 64 columns at a time: whole
    // 128-byte lines reach L2 (16-byte stores from the registers, one row per lane, measured
    // 2.5 kcycles per 32 columns: every piece is a memory request of its own).
    static __device__ __forceinline__ void epilogue(const Params& p, Smem& sm, const CUtensorMap* map_c, const CUtensorMap*,
                                                    uint32_t tmem, int ewarp, int lane, int m0, const Tile& tl)
    {
        const int img = tl.img, n_tile = tl.n_tile;
        const int quarter = ewarp & 3, half = ewarp >> 2;
        const int nh = tl.n0 + half * 128;  // first token of this warp's columns
        const float2* stats = sm.stats[ewarp];
        uint8_t* out = sm.out[ewarp];
        const int m = m0 + quarter * 32 + lane;
        const bool row_ok = m < p.m_e;
        const float qs = row_ok ? p.qsum[m] : 0.f;
        const float neg_c = -p.inv_tau_log2e;
        float row_sum = 0.f;
        const bool full_tile = nh + 128 <= p.t_e;  // warp-uniform
        for_each_chunk(tmem + ((uint32_t)(quarter * 32) << 16) + half * 128, 128,
                       [&](const uint32_t (&acc)[32], int c0) {
            uint32_t packed[16];
            if (full_tile) chunk<false>(acc, stats + c0, qs, neg_c, 32, row_sum, packed);
            else chunk<true>(acc, stats + c0, qs, neg_c, p.t_e - nh - c0, row_sum, packed);
            if ((c0 & 32) == 0) {  // first half of a 64-column group: the buffer must be free again
                if (lane == 0) tma_store_wait_read();
                __syncwarp();
            }
            // row `lane` of the box, 16-byte pieces j = 0..3 (or 4..7) at the swizzled position j ^ (row % 8)
            const int j0 = (c0 & 32) >> 3;
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4)
                *reinterpret_cast<uint4*>(out + lane * 128 + (((j0 + q4) ^ (lane & 7)) << 4)) =
                    make_uint4(packed[4 * q4], packed[4 * q4 + 1], packed[4 * q4 + 2], packed[4 * q4 + 3]);
            if (c0 & 32) {  // the group is complete: hand it to the copy engine
                fence_async_smem();
                __syncwarp();
                if (lane == 0) tma_store_3d(map_c, out, nh + c0 - 32, m0 + quarter * 32, img);
            }
        });
        if (row_ok) p.lpart[((size_t)img * p.m_e + m) * (2 * p.grid.n_tiles) + 2 * n_tile + half] = row_sum;
    }
};
using ScoresOp = ScoresOpT<false>;
using ScoresPairOp = ScoresOpT<true>;

// Z_0 = (P X_0) / l, K = tokens; A = P K-major, B = X_0 MN-major (blocks of 64 tokens x 128 B, one
// per 64 features, 8 KB apart).  One block per tile of 128 anchors x BN features (BN = 128, 192 or
// 256).  A pair version (256 anchors x 256 features, a last tile of 128, tiles dealt out widest
// first in serpentine order) ran 15 % fewer cycles per tile but no faster in time on the
// power-capped GPU (184.4 vs 184.8 us per call), so the simpler kernel stayed.
__device__ __forceinline__ void values_epilogue(const ValuesParams& p, uint32_t tmem, int ewarp, int lane, int m0,
                                                const Tile& tl)
{
    const int half_cols = tl.n >> 1;  // 64, 96 or 128 feature columns per warp
    const int quarter = ewarp & 3, half = ewarp >> 2;
    const int m = m0 + quarter * 32 + lane;
    const bool row_ok = m < p.m_e;
    float l = 0.f;  // the row's partial sums from the first GEMM
    if (row_ok) {
        const float* lp = p.lpart + ((size_t)tl.img * p.m_e + m) * p.n_parts;
        for (int t = 0; t < p.n_parts; ++t) l += lp[t];
    }
    const float inv_l = l > 0.f ? 1.f / l : 0.f;
    if (row_ok && tl.n0 == 0 && half == 0) p.inv_l[(size_t)tl.img * p.m_e + m] = inv_l;
    const int nh = tl.n0 + half * half_cols;
    __nv_bfloat16* out = p.z + ((size_t)tl.img * p.m_e + (row_ok ? m : 0)) * p.d_v + nh;
    for_each_chunk(tmem + ((uint32_t)(quarter * 32) << 16) + half * half_cols, half_cols,
                   [&](const uint32_t (&acc)[32], int c0) {
        if (row_ok) {
#pragma unroll
            for (int q4 = 0; q4 < 4; ++q4) {
                if (nh + c0 + q4 * 8 < p.d_v) {  // d_v is a multiple of 8
                    uint32_t w[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const __nv_bfloat162 h =
                            __floats2bfloat162_rn(__uint_as_float(acc[q4 * 8 + 2 * e]) * inv_l,
                                                  __uint_as_float(acc[q4 * 8 + 2 * e + 1]) * inv_l);
                        w[e] = *reinterpret_cast<const uint32_t*>(&h);
                    }
                    *reinterpret_cast<uint4*>(out + c0 + q4 * 8) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
        }
    });
}

template <int BN_>
struct ValuesOp {
    static constexpr int BN = BN_, STAGES = BN_ == 256 ? 4 : 5, kCtas = 1, kSideWarps = 4;
    static constexpr bool kAMnMajor = false, kBMnMajor = true;
    using Params = ValuesParams;
    using Smem = GemmSmem<BN, STAGES, false>;
    static __device__ __forceinline__ int k_steps(const Params& p) { return (p.t_e + kAggBK - 1) / kAggBK; }
    static __device__ __forceinline__ bool tile(const Params& p, int worker, int n_workers, int i, Tile& tl)
    {
        return round_robin_tile(p.grid, BN, worker, n_workers, i, tl);
    }
    static __device__ __forceinline__ void load(const Params&, Smem& sm, int s, const CUtensorMap* map_a,
                                                const CUtensorMap* map_b, const CUtensorMap*, int k, int m0,
                                                const Tile& tl, uint32_t, uint32_t)
    {
        mbar_expect_tx(&sm.full[s], (kAggBM + BN) * kAggBK * 2);
        tma_load_3d(sm.a[s], map_a, k * kAggBK, m0, tl.img, &sm.full[s]);
#pragma unroll
        for (int j = 0; j < BN / 64; ++j)  // 64 features x 64 tokens per box
            tma_load_3d(sm.b[s] + j * (kAggBK * 64), map_b, tl.n0 + j * 64, k * kAggBK, tl.img, &sm.full[s]);
    }
    static __device__ __forceinline__ uint64_t a_desc(uint32_t a0, int kk) { return umma_desc(a0 + kk * 32, 16, 1024); }
    // 16 token rows of 128 B per K step; the next 64 features start one box (8 KB) further on
    static __device__ __forceinline__ uint64_t b_desc(uint32_t b0, int kk) { return umma_desc(b0 + kk * 2048, kAggBK * 128, 1024); }
    static __device__ __forceinline__ void prefetch(const Params&, Smem&, int, int, const Tile&) {}
    static __device__ __forceinline__ void epilogue(const Params& p, Smem&, const CUtensorMap*, const CUtensorMap*,
                                                    uint32_t tmem, int ewarp, int lane, int m0, const Tile& tl)
    {
        values_epilogue(p, tmem, ewarp, lane, m0, tl);
    }
    // Token mass (column sums of W_A = P / l) on the way: while a block works on a tile of the first
    // feature panel, four side warps add up the columns of that tile's 128 rows of P, read from global
    // memory (the rows the block's own tensor copies fetch at about the same time, so one of the two
    // finds them in L2) and not from the stages in shared memory, whose bandwidth is what bounds the
    // GEMM: side warps reading the stages made the tile three times slower.  Side warp sw takes the
    // anchors 32 sw .. 32 sw + 31; lane = 8 neighbouring tokens (16 bytes) of every fourth row.  The
    // sums of a panel of 32 anchors go to mass_partial; a small kernel adds the panels in order.
    static __device__ __forceinline__ bool side_active(const Params& p, const Tile& tl)
    {
        return p.mass_partial != nullptr;
    }
    static __device__ __forceinline__ void side_tile(const Params& p, Smem& sm, int sw, int lane, int m0, const Tile& tl)
    {
        {   // 1 / l of row m0 + 32 sw + lane: the same sum, in the same order, as the epilogue's
            const int m = m0 + sw * 32 + lane;
            float l = 0.f;
            if (m < p.m_e) {
                const float* lp = p.lpart + ((size_t)tl.img * p.m_e + m) * p.n_parts;
                int t = 0;
                for (; t + 8 <= p.n_parts; t += 8) {
                    float v[8];
#pragma unroll
                    for (int e = 0; e < 8; ++e) v[e] = __ldg(lp + t + e);
#pragma unroll
                    for (int e = 0; e < 8; ++e) l += v[e];
                }
                for (; t < p.n_parts; ++t) l += __ldg(lp + t);
            }
            __syncwarp();  // the previous tile's weights have been read
            sm.side_w[sw][lane] = l > 0.f ? 1.f / l : 0.f;
            __syncwarp();
        }
        const int group = lane >> 3, c8 = (lane & 7) * 8;  // rows group, group + 4, ...; tokens c8 .. c8 + 7 of a slab
        float w[8];
        bool row_ok[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            w[i] = sm.side_w[sw][4 * i + group];
            row_ok[i] = m0 + sw * 32 + 4 * i + group < p.m_e;
        }
        const __nv_bfloat16* rows = p.pw + ((size_t)tl.img * p.m_e + m0 + sw * 32 + group) * p.t_ld + c8;
        float* out = p.mass_partial + ((size_t)tl.img * (4 * p.grid.m_tiles) + (m0 / kAggBM) * 4 + sw) * p.t_ld + c8;
        // slabs of 64 tokens, dealt out over the feature tiles of this panel of anchors; t_ld is a multiple of 8
        for (int col = tl.n_tile * 64; col < p.t_ld; col += 64 * p.grid.n_tiles) {
            const bool col_ok = col + c8 < p.t_ld;
            uint4 u[8];
#pragma unroll
            for (int i = 0; i < 8; ++i)
                u[i] = col_ok && row_ok[i] ? __ldcs(reinterpret_cast<const uint4*>(rows + (size_t)(4 * i) * p.t_ld + col))
                                           : make_uint4(0u, 0u, 0u, 0u);
            float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint32_t x[4] = {u[i].x, u[i].y, u[i].z, u[i].w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    acc[2 * e] = fmaf(__uint_as_float(x[e] << 16), w[i], acc[2 * e]);
                    acc[2 * e + 1] = fmaf(__uint_as_float(x[e] & 0xFFFF0000u), w[i], acc[2 * e + 1]);
                }
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) {  // the four row groups, always in the same order
                acc[e] += __shfl_xor_sync(0xFFFFFFFFu, acc[e], 8);
                acc[e] += __shfl_xor_sync(0xFFFFFFFFu, acc[e], 16);
            }
            if (group == 0 && col_ok) {
                *reinterpret_cast<float4*>(out + col) = make_float4(acc[0], acc[1], acc[2], acc[3]);
                *reinterpret_cast<float4*>(out + col + 4) = make_float4(acc[4], acc[5], acc[6], acc[7]);
            }
        }
    }
};

// K_c = Rbar^T K (and V_c = Rbar^T V) of the KV-compressed attention: tile of 128 memory anchors x
// BN features, K = compact tokens.  A = R [m_e, s] read as R^T, i.e. MN-major (two blocks of 64
// tokens x 64 anchors); B = K or V [m_e, d] MN-major as above.  The epilogue divides row s by the
// column sum of R.
struct CompressParams {
    const float* colsum_parts;  // [n_parts, s] column sums of the bf16-rounded assignment matrix, by row panel
    int32_t n_parts;
    __nv_bfloat16* out;    // [n_img, s, out_ld]  K_c
    __nv_bfloat16* out_v;  // [n_img, s, out_ld]  V_c
    int* error;
    TileGrid grid;         // over 2 n_img "images": K of every image, then V
    int32_t s, m_e, d_v, n_img;
    // Output layout: the d_v features are heads of head_dim columns; every head is written as
    // head_ld >= head_dim columns, the extra ones zero (out_ld = d_v / head_dim * head_ld).  The
    // attention kernel reads whole 16-column K steps, so a 72-wide head is stored 80 wide.
    int32_t head_dim, head_ld, out_ld;
};

template <int BN_>
struct CompressOp {
    static constexpr int BN = BN_, STAGES = BN_ == 128 ? 5 : 4, kCtas = 1, kSideWarps = 0;
    static constexpr bool kAMnMajor = true, kBMnMajor = true;
    using Params = CompressParams;
    using Smem = GemmSmem<BN, STAGES, false, true>;
    static __device__ __forceinline__ int k_steps(const Params& p) { return (p.m_e + kAggBK - 1) / kAggBK; }
    static __device__ __forceinline__ bool tile(const Params& p, int worker, int n_workers, int i, Tile& tl)
    {
        return round_robin_tile(p.grid, BN, worker, n_workers, i, tl);
    }
    // "Images" [0, n_img) of the tile grid compress K (map_b), [n_img, 2 n_img) compress V (map_v).
    static __device__ __forceinline__ void load(const Params& p, Smem& sm, int s, const CUtensorMap* map_a,
                                                const CUtensorMap* map_b, const CUtensorMap* map_v, int k, int m0,
                                                const Tile& tl, uint32_t, uint32_t)
    {
        const bool second = tl.img >= p.n_img;
        const CUtensorMap* map_x = second ? map_v : map_b;
        const int img = second ? tl.img - p.n_img : tl.img;
        mbar_expect_tx(&sm.full[s], (kAggBM + BN) * kAggBK * 2);
        tma_load_2d(sm.a[s], map_a, m0, k * kAggBK, &sm.full[s]);                       // anchors m0 .. + 64
        tma_load_2d(sm.a[s] + kAggBK * 64, map_a, m0 + 64, k * kAggBK, &sm.full[s]);    // .. + 128
#pragma unroll
        for (int j = 0; j < BN / 64; ++j)
            tma_load_3d(sm.b[s] + j * (kAggBK * 64), map_x, tl.n0 + j * 64, k * kAggBK, img, &sm.full[s]);
    }
    static __device__ __forceinline__ uint64_t a_desc(uint32_t a0, int kk) { return umma_desc(a0 + kk * 2048, kAggBK * 128, 1024); }
    static __device__ __forceinline__ uint64_t b_desc(uint32_t b0, int kk) { return umma_desc(b0 + kk * 2048, kAggBK * 128, 1024); }
    // Before the accumulator is waited for: the divisor of this thread's row (memory anchor),
    // the panels' column sums added in a fixed order so that every tile gets the same value.
    // It waits in the thread's own shared-memory slot (the statistics array is unused here).
    static __device__ __forceinline__ void prefetch(const Params& p, Smem& sm, int ewarp, int lane, const Tile& tl)
    {
        const int row = tl.m_tile * kAggBM + (ewarp & 3) * 32 + lane;
        float sum = 0.f;
        if (row < p.s) {
#pragma unroll 8
            for (int q = 0; q < p.n_parts; ++q) sum += __ldg(p.colsum_parts + (size_t)q * p.s + row);
        }
        reinterpret_cast<float*>(sm.stats[0])[ewarp * 32 + lane] = sum > 0.f ? 1.f / sum : 0.f;
    }
    // map_k / map_v: K_c and V_c [n_img, s, d_v] with boxes of 32 rows x 64 columns, for the staged store
    static __device__ __forceinline__ void epilogue(const Params& p, Smem& sm, const CUtensorMap* map_k,
                                                    const CUtensorMap* map_v, uint32_t tmem, int ewarp, int lane, int m0,
                                                    const Tile& tl)
    {
        const int half_cols = tl.n >> 1;
        const int quarter = ewarp & 3, half = ewarp >> 2;
        const int row = m0 + quarter * 32 + lane;  // memory anchor
        const bool row_ok = row < p.s;
        const float inv = reinterpret_cast<const float*>(sm.stats[0])[ewarp * 32 + lane];
        const int nh = tl.n0 + half * half_cols;
        const bool second = tl.img >= p.n_img;
        if (p.head_ld == p.head_dim && (half_cols & 63) == 0) {
            // Plain layout: the rows leave through swizzled staging rows and one bulk tensor store per
            // 32 rows x 64 columns (whole 128-byte lines; 16-byte stores straight from the registers, one
            // row per lane, took 7000 cycles for a 128 x 256 tile, as long as half of its MMAs).
            uint8_t* out = sm.out[ewarp];
            const CUtensorMap* map = second ? map_v : map_k;
            const int img = second ? tl.img - p.n_img : tl.img;
            for_each_chunk(tmem + ((uint32_t)(quarter * 32) << 16) + half * half_cols, half_cols,
                           [&](const uint32_t (&acc)[32], int c0) {
                uint32_t w[16];
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                    const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(acc[2 * e]) * inv,
                                                                   __uint_as_float(acc[2 * e + 1]) * inv);
                    w[e] = *reinterpret_cast<const uint32_t*>(&h);
                }
                if ((c0 & 32) == 0) {  // first half of a 64-column group: the buffer must be free again
                    if (lane == 0) tma_store_wait_read();
                    __syncwarp();
                }
                const int j0 = (c0 & 32) >> 3;
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4)
                    *reinterpret_cast<uint4*>(out + lane * 128 + (((j0 + q4) ^ (lane & 7)) << 4)) =
                        make_uint4(w[4 * q4], w[4 * q4 + 1], w[4 * q4 + 2], w[4 * q4 + 3]);
                if (c0 & 32) {  // the group is complete: hand it to the copy engine (clipped at s rows, d_v columns)
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0 && nh + c0 - 32 < p.d_v && m0 + quarter * 32 < p.s)
                        tma_store_3d(map, out, nh + c0 - 32, m0 + quarter * 32, img);
                }
            });
            return;
        }
        __nv_bfloat16* out = (second ? p.out_v : p.out) +
                             ((size_t)(second ? tl.img - p.n_img : tl.img) * p.s + (row_ok ? row : 0)) * p.out_ld;
        const int pad = p.head_ld - p.head_dim;  // 0 or 8 columns (head_dim is a multiple of 8)
        for_each_chunk(tmem + ((uint32_t)(quarter * 32) << 16) + half * half_cols, half_cols,
                       [&](const uint32_t (&acc)[32], int c0) {
            if (row_ok) {
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    const int f = nh + c0 + q4 * 8;  // first of 8 features: a group never straddles two heads
                    if (f < p.d_v) {
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(acc[q4 * 8 + 2 * e]) * inv,
                                                                           __uint_as_float(acc[q4 * 8 + 2 * e + 1]) * inv);
                            w[e] = *reinterpret_cast<const uint32_t*>(&h);
                        }
                        const int head = pad ? f / p.head_dim : 0;
                        __nv_bfloat16* at = out + f + head * pad;
                        *reinterpret_cast<uint4*>(at) = make_uint4(w[0], w[1], w[2], w[3]);
                        if (pad && f - head * p.head_dim == p.head_dim - 8)  // the head's last group: zeros behind it
                            *reinterpret_cast<uint4*>(at + 8) = make_uint4(0u, 0u, 0u, 0u);
                    }
                }
            }
        });
    }
};

template <class Op>
__global__ void __launch_bounds__(kAggThreads + 32 * Op::kSideWarps) aggregate_gemm_kernel(const __grid_constant__ CUtensorMap map_a,
                                                                     const __grid_constant__ CUtensorMap map_b,
                                                                     const __grid_constant__ CUtensorMap map_c,
                                                                     const __grid_constant__ CUtensorMap map_d,
                                                                     const __grid_constant__ CUtensorMap map_e,
                                                                     const typename Op::Params p)
{
    constexpr int STAGES = Op::STAGES;
    constexpr bool kPair = Op::kCtas == 2;
    constexpr uint32_t kAccStride = 256;  // TMEM columns between the two accumulators
    extern __shared__ uint8_t smem_raw[];
    using Smem = typename Op::Smem;
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int k_steps = Op::k_steps(p);
    volatile int* abort = &sm.abort;
    // a "worker" is one block, or one pair of blocks; p.grid counts the workers' tiles
    const uint32_t rank = kPair ? cluster_ctarank() : 0u;
    const int worker = kPair ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    const int n_workers = kPair ? (int)(gridDim.x >> 1) : (int)gridDim.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(&sm.full[s], 1); mbar_init(&sm.empty[s], 1); }
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sm.acc_full[b], 1);
            mbar_init(&sm.acc_empty[b], kEpilogueWarps * Op::kCtas);  // the leader's collects both blocks' warps
        }
        sm.abort = 0;
        fence_barrier_init();
    }
    if (warp == 1) {
        if (kPair) tmem_alloc_pair(&sm.tmem_base, 512);
        else tmem_alloc(&sm.tmem_base, 512);
    }
    wait_for_prior_kernels();
    tc_fence_before_sync();
    __syncthreads();
    if (kPair) cluster_sync();  // the partner's barriers exist before anything is signalled on them
    tc_fence_after_sync();
    const uint32_t tmem_base = sm.tmem_base;
    const bool stop = *p.error != 0;  // an earlier block of this launch already failed

    // A wait on the "empty" side uses the opposite parity, so the first pass over a fresh
    // barrier falls through (nothing has to be drained yet).
    // Producer and MMA warp: the whole warp walks the loops and the waits in step and one elected lane
    // issues.  A lone lane (the rest of the warp parked) keeps every operand in its own registers and
    // moves them to the uniform registers the copy and MMA instructions read one value at a time:
    // measured 120 cycles per tensor copy, so that a stage of six copies took 735 cycles to request
    // and the whole K loop of the compression ran at the producer's pace, not the tensor core's.
    if (warp == 0 && !stop) {
        // ---- producer (in every block)
        uint32_t it = 0;  // stages issued so far, over all tiles
        bool ok = true;
        Tile tl;
        for (int i = 0; ok && Op::tile(p, worker, n_workers, i, tl); ++i) {
            const int m0 = (tl.m_tile * Op::kCtas + (int)rank) * kAggBM;
            for (int k = 0; k < k_steps; ++k, ++it) {
                const int s = it % STAGES;
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(&sm.empty[s], ((it / STAGES) & 1) ^ 1, abort, p.error, kAggTimeoutEmpty)) != 0;
                if (!ok) break;
                if (elect_one())
                    Op::load(p, sm, s, &map_a, &map_b, &map_c, k, m0, tl, rank, kPair ? cluster_address(&sm.full[s], 0) : 0u);
                __syncwarp();
            }
        }
        if (*abort && lane == 0) {  // let the copies already in flight land before the block goes away
            if (rank == 0) {
                for (uint32_t j = it > (uint32_t)STAGES ? it - STAGES : 0; j < it; ++j) {
                    const long long t0 = clock64();
                    while (!mbar_try_wait(&sm.full[j % STAGES], (j / STAGES) & 1) &&
                           (unsigned long long)(clock64() - t0) < kWaitLimitCycles) {}
                }
            } else {  // the partner cannot poll the leader's barrier: give its copies ample time
                const long long t0 = clock64();
                while ((unsigned long long)(clock64() - t0) < (1ull << 22)) {}
            }
        }
    } else if (warp == 1 && !stop && rank == 0) {
        // ---- MMA issue (leader only): 4 instructions of K = 16 per stage
        uint32_t it = 0;
        bool ok = true;
        Tile tl;
        for (int local = 0; ok && Op::tile(p, worker, n_workers, local, tl); ++local) {
            const uint32_t idesc = umma_idesc(tl.n, Op::kBMnMajor ? 1 : 0, kAggBM * Op::kCtas, Op::kAMnMajor ? 1 : 0);
            const int buf = local & 1;
            ok = __all_sync(0xFFFFFFFFu, mbar_wait(&sm.acc_empty[buf], ((local >> 1) & 1) ^ 1, abort, p.error, kAggTimeoutAcc)) != 0;
            if (!ok) break;
            tc_fence_after_sync();
            const uint32_t tmem_acc = tmem_base + buf * kAccStride;
            for (int k = 0; k < k_steps; ++k, ++it) {
                const int s = it % STAGES;
                ok = __all_sync(0xFFFFFFFFu, mbar_wait(&sm.full[s], (it / STAGES) & 1, abort, p.error, kAggTimeoutFull)) != 0;
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t a0 = smem_u32(sm.a[s]), b0 = smem_u32(sm.b[s]);
                if (elect_one()) {
#pragma unroll
                    for (int kk = 0; kk < kAggBK / 16; ++kk) {
                        if (kPair) umma_bf16_pair(tmem_acc, Op::a_desc(a0, kk), Op::b_desc(b0, kk), idesc, (k | kk) != 0);
                        else umma_bf16(tmem_acc, Op::a_desc(a0, kk), Op::b_desc(b0, kk), idesc, (k | kk) != 0);
                    }
                    // frees the stage (in both blocks) once these MMAs have read it
                    if (kPair) umma_commit_pair(&sm.empty[s]);
                    else umma_commit(&sm.empty[s]);
                }
                __syncwarp();
            }
            if (ok && elect_one()) {
                if (kPair) umma_commit_pair(&sm.acc_full[buf]);
                else umma_commit(&sm.acc_full[buf]);
            }
            __syncwarp();
        }
    } else if (warp >= 2 + kEpilogueWarps) {
        // ---- side warps (an Op that has them): work of their own beside the tiles, no part in the pipeline
        if constexpr (Op::kSideWarps > 0) {
            if (!stop) {
                Tile tl;
                for (int local = 0; Op::tile(p, worker, n_workers, local, tl); ++local)
                    if (Op::side_active(p, tl)) Op::side_tile(p, sm, warp - (2 + kEpilogueWarps), lane, tl.m_tile * kAggBM, tl);
            }
        }
    } else if (warp >= 2 && !stop) {
        // ---- epilogue: warps 2..9; a warp may read the TMEM lane quarter (warp index mod 4)
        const int ewarp = ((warp & 3) | ((warp - 2) & 4));  // quarter in bits 0-1, column half in bit 2
        Tile tl;
        for (int local = 0; Op::tile(p, worker, n_workers, local, tl); ++local) {
            const int m0 = (tl.m_tile * Op::kCtas + (int)rank) * kAggBM;
            const int buf = local & 1;
            Op::prefetch(p, sm, ewarp, lane, tl);
            // tcgen05.ld is warp-collective: the whole warp goes on, or none of it
            if (!__all_sync(0xFFFFFFFFu, mbar_wait(&sm.acc_full[buf], (local >> 1) & 1, abort, p.error, kAggTimeoutAcc)))
                break;
            tc_fence_after_sync();
            Op::epilogue(p, sm, &map_d, &map_e, tmem_base + buf * kAccStride, ewarp, lane, m0, tl);
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {  // this warp has drained its part of the accumulator
                if (kPair) mbar_arrive_cluster(cluster_address(&sm.acc_empty[buf], 0));
                else mbar_arrive(&sm.acc_empty[buf]);
            }
        }
        if (lane == 0) tma_store_wait_all();  // this warp's bulk stores have been written
    }
    tc_fence_before_sync();
    __syncthreads();
    if (kPair) cluster_sync();  // neither block leaves while the other may still signal it or read its tiles
    if (warp == 1) {
        tc_fence_after_sync();
        if (kPair) tmem_dealloc_pair(tmem_base, 512);
        else tmem_dealloc(tmem_base, 512);
    }
}

// Self-test of the bounded wait: one block, one mbarrier that nobody ever arrives on, no copy and
// no MMA in flight.  Thread 0 waits with the caller's (short) limit, runs into it and raises the
// block's stop flag; thread 32 waits on the same barrier with the library's ordinary limit and must
// leave through the stop flag.  record[0] = the time-out code, record[1] = 1 if the second waiter
// left because of the flag.
__global__ void __launch_bounds__(64) bounded_wait_selftest_kernel(unsigned long long limit, int* record)
{
    __shared__ uint64_t bar;
    __shared__ int stop;
    wait_for_prior_kernels();
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        stop = 0;
        fence_barrier_init();
    }
    __syncthreads();
    volatile int* abort = &stop;
    if (threadIdx.x == 0) {
        mbar_wait(&bar, 0, abort, record, kAggTimeoutFull, limit);
    } else if (threadIdx.x == 32) {
        const bool ok = mbar_wait(&bar, 0, abort, record, kAggTimeoutAcc);
        if (!ok && *abort) record[1] = 1;
    }
}

// Column sums of W_A: mass[img, i] = sum_m P[m, i] / l[m], in two deterministic steps: the side
// warps of the value GEMM leave the sums of panels of 32 anchors (ValuesOp::side_tile), and
// token_mass_reduce_kernel adds the panels in a fixed order.
// A kernel of its own for the first step (a block per panel of 128 rows over a slab of 256 token
// columns, its eight warps every eighth row) took 11.8 us on 8 x 1024 x 4096 weights, reading P from
// global memory once more after the GEMM; beside the GEMM the same reads cost it 4.5 us.
__global__ void __launch_bounds__(64) token_mass_reduce_kernel(const float* __restrict__ partial, int t_e, int t_ld,
                                                                int n_panels, float* __restrict__ mass)
{
    wait_for_prior_kernels();
    const int img = blockIdx.y;
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= t_e) return;
    const float* col = partial + (size_t)img * n_panels * t_ld + i;
    float acc = 0.f;
#pragma unroll 16
    for (int q = 0; q < n_panels; ++q) acc += col[(size_t)q * t_ld];
    mass[(size_t)img * t_e + i] = acc;
}

}  // namespace civic
