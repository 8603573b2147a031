// KV-compressed visual attention (Eq. 9 of the paper) for already projected Q, K, V:
//
//     K_c = Rbar^T K,  V_c = Rbar^T V,  Attn_c = softmax(Q K_c^T / sqrt(d)) V_c   per head
//
// R [m_e, s] assigns the m_e compact tokens to s memory anchors; Rbar is R with every column
// divided by its sum.  The compression is a GEMM of the persistent template (CompressOp in
// aggregate.cuh), one launch for K and V together.  This file holds the preparation of R and the
// attention itself: one block per (range of query tiles, head, image).  With at most 256 memory
// anchors a head's whole K_c and V_c fit in shared memory and stay there while the block walks
// its tiles of 128 queries; per tile there are two MMA chains and one softmax between them,
// with no running maximum to maintain:
//   TMA      K_c[:, head] [s, d] (K-major) and V_c[:, head] [s, d] (MN-major) once; Q tiles
//            [128, d] into a ring of two
//   MMA 1    S = Q K_c^T -> TMEM columns [0, s)
//   softmax  thread per query row: maximum, exp2, row sum; P cut to bf16 and packed straight back
//            into TMEM, columns [0, s / 2), behind the thread's own reads of S
//   MMA 2    O = P V_c with the A operand read from TMEM -> TMEM columns [s / 2, s / 2 + d).
//            (With P in shared memory this chain was bound by shared-memory reads: 4 KB of P
//            for every 2 KB of V_c and only 64 or 128 output columns to amortise them.)
//   store    O / row sum as bf16, staged in swizzled shared memory, one bulk tensor store of
//            32 rows per warp
// A block is a serial chain; two blocks share an SM (shared memory and tensor memory allow it
// for 64-wide heads) and fill each other's waits.  Every wait is bounded as in aggregate.cuh.
#pragma once
#include "aggregate.cuh"

namespace civic {

// R (fp32) -> bf16 copy and the column sums of the ROUNDED values (what the tensor core will
// multiply with): a block converts kAssignRows rows and writes their column sums; the compression
// GEMM's epilogue adds the panels' sums in a fixed order.
constexpr int kAssignRows = 16;
__global__ void assign_convert_kernel(const float* __restrict__ r, int m_e, int s, __nv_bfloat16* __restrict__ r16,
                                      float* __restrict__ partial, int* __restrict__ status)
{
    wait_for_prior_kernels();
    if (status && blockIdx.x == 0 && threadIdx.x == 0) *status = 0;  // the call's status word starts clean
    const int m_begin = blockIdx.x * kAssignRows, m_end = min(m_begin + kAssignRows, m_e);
    for (int c = threadIdx.x; c < s; c += blockDim.x) {
        float sum = 0.f;
#pragma unroll
        for (int m = m_begin; m < m_begin + kAssignRows; ++m) {
            if (m >= m_end) break;
            const __nv_bfloat16 v = __float2bfloat16_rn(r[(size_t)m * s + c]);
            r16[(size_t)m * s + c] = v;
            sum += __bfloat162float(v);
        }
        partial[(size_t)blockIdx.x * s + c] = sum;
    }
}
// Adds the panels' column sums in their fixed order: colsum[c] = sum_q partial[q, c].  Used when R is
// prepared once for many calls (the compression GEMM then reads one value per anchor).
__global__ void assign_colsum_kernel(const float* __restrict__ partial, int n_parts, int s, float* __restrict__ colsum)
{
    wait_for_prior_kernels();
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= s) return;
    float sum = 0.f;
    for (int q = 0; q < n_parts; ++q) sum += partial[(size_t)q * s + c];
    colsum[c] = sum;
}

// Clears a call's status word where the call has no small kernel in front of its tensor-core
// kernels to do it.  (A memset node would do, but the stream cannot overlap its launch with the
// kernels before and after it: measured 4 us per call.)
__global__ void clear_status_kernel(int* __restrict__ status)
{
    release_next_kernel();
    wait_for_prior_kernels();
    if (threadIdx.x == 0) *status = 0;
}

constexpr int kAttnThreads = 192;  // warp 0: TMA, warp 1: TMEM + MMA, warps 2..5: one query row per thread

struct AttnParams {
    int* error;
    int32_t m_e, s;
    int32_t d;                // head dimension (a multiple of 8)
    int32_t d_pad;            // d rounded up to a multiple of 16: the K of the first chain, the N of the second
    int32_t d_ld;             // columns per head of K_c and V_c (d_pad: zero columns behind the d real ones)
    int32_t tiles_per_block;  // query tiles of 128 rows walked by one block
    int32_t q_slots;          // Q tiles in flight: 2, or 1 where shared memory is short
    int32_t v_stream;         // 0: the head's V_c stays resident; 1: streamed per query tile in blocks of 64 anchors
    float scale_log2e;        // log2(e) / sqrt(d)
};

// D[tmem] (+)= A[tmem] B[smem]: A's row i on TMEM lane i, two bf16 of consecutive k per 32-bit column.
__device__ __forceinline__ void umma_bf16_a_tmem(uint32_t tmem_d, uint32_t tmem_a, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t accumulate)
{
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.u32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n"
        "}\n"
        ::"r"(tmem_d), "r"(tmem_a), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// 8 consecutive 32-bit columns of this warp's 32 TMEM lanes (thread t writes lane base + t)
__device__ __forceinline__ void tmem_store8(uint32_t taddr, const uint32_t (&r)[8])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
                 : "memory");
}
__device__ __forceinline__ void tmem_store_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// 16 fp32 columns at a time (the exponential pass keeps its register count down with these),
// issue and wait split as for the 32-column loads
__device__ __forceinline__ void tmem_load_issue16(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_load_wait16(uint32_t (&r)[16])
{
    asm volatile("tcgen05.wait::ld.sync.aligned;"
                 : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]),
                   "+r"(r[8]), "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
                 :: "memory");
}
// `cols` (a multiple of 32) columns in chunks of 16 with two register buffers
template <class Body>
__device__ __forceinline__ void for_each_chunk16(uint32_t taddr, int cols, Body&& body)
{
    uint32_t even[16], odd[16];
    tmem_load_issue16(taddr, even);
#pragma unroll 1
    for (int c0 = 0; c0 < cols; c0 += 32) {
        tmem_load_wait16(even);
        tmem_load_issue16(taddr + c0 + 16, odd);
        body(even, c0);
        tmem_load_wait16(odd);
        if (c0 + 32 < cols) tmem_load_issue16(taddr + c0 + 32, even);
        body(odd, c0 + 16);
    }
}

// max(a, b, c) in one instruction
__device__ __forceinline__ float fmax3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// 2^x for x <= 0 without the special-function unit: x = n + f with n = round(x), |f| <= 1/2;
// 2^f by a cubic (largest relative error 7.5e-5, far below the bf16 cut that follows) and n added
// into the exponent field.  Inputs below -125 give 2^-125 (any such weight is nothing beside the
// row's largest, which is 1).  Eight instructions on the FMA and integer pipes.
__device__ __forceinline__ float exp2_poly(float x)
{
    x = fmaxf(x, -125.f);
    const float t = x + 12582912.f;  // 1.5 * 2^23: the low mantissa bits now hold round(x)
    const float f = x - (t - 12582912.f);
    float p = fmaf(0.0551716685f, f, 0.2426111251f);
    p = fmaf(p, f, 0.6932609677f);
    p = fmaf(p, f, 0.9999280572f);
    return __uint_as_float(__float_as_uint(p) + (__float_as_uint(t) << 23));
}

__host__ __device__ constexpr int round_up_int(int x, int a) { return (x + a - 1) / a * a; }

// Shared memory: k [d_blocks][s x 128 B] | v [s/64 or 2][d_blocks][64 x 128 B] | q [q_slots][d_blocks][128 x 128 B]
// | o [4 warps][d_blocks][32 x 128 B] | barriers, d_blocks = ceil(d_pad / 64).  Every block of data is
// 1024-byte aligned; the kernel has no static shared memory, so the dynamic window itself starts on
// such a boundary (checked at run time) and no slack is set aside: 113 KB for 64-wide heads and 256
// anchors is exactly what lets two blocks share an SM.
__host__ __device__ constexpr size_t attn_smem_bytes(int d_pad, int s, int q_slots, int v_stream)
{
    const size_t db = (size_t)(d_pad + 63) / 64;
    return db * s * 128 + (size_t)(v_stream ? 2 : s / 64) * db * 8192 + (size_t)q_slots * db * 16384 + 4 * db * 4096 +
           1024 /* barriers */;
}
// TMEM columns of a block: S in [0, s), later P in [0, s / 2) and O in [s / 2, s / 2 + d_pad), read
// back in chunks of 32 columns
__host__ __device__ constexpr uint32_t attn_tmem_cols(int d_pad, int s)
{
    const int o_end = s / 2 + round_up_int(d_pad, 32);
    const int need = s > o_end ? s : o_end;
    return need <= 32 ? 32u : (need <= 64 ? 64u : (need <= 128 ? 128u : (need <= 256 ? 256u : 512u)));
}

// kPolyMask: which of the 16 columns of a chunk take their exponential on the FMA pipe
// (exp2_poly) instead of the special-function unit, which is the busiest unit of this kernel
// (16 results per clock and SM against 128 lanes of FMA).
constexpr uint32_t kPolyMask = 0x0000u;

// Registers are handed out per group of four warps, so a block of six warps is charged for eight:
// bounding the kernel as if it had 256 threads, two blocks per SM, keeps it at 128 registers.
__global__ void __launch_bounds__(256, 2) kv_attention_kernel(const __grid_constant__ CUtensorMap map_q,
                                                                    const __grid_constant__ CUtensorMap map_k,
                                                                    const __grid_constant__ CUtensorMap map_v,
                                                                    const __grid_constant__ CUtensorMap map_o,
                                                                    const __grid_constant__ CUtensorMap map_o_tail,
                                                                    const AttnParams p)
{
    extern __shared__ __align__(1024) uint8_t attn_smem[];
    uint8_t* base = attn_smem;
    // the swizzled tiles would be misplaced: the block then does no work (reported below, after
    // the wait for the previous kernels like every other access to global memory)
    const bool misplaced = (smem_u32(base) & 1023u) != 0;
    const int d = p.d, d_pad = p.d_pad, s = p.s, d_blocks = (d_pad + 63) >> 6, s_blocks = s >> 6;
    const int v_slots = p.v_stream ? 2 : s_blocks;
    uint8_t* k_sm = base;
    uint8_t* v_sm = k_sm + d_blocks * s * 128;
    uint8_t* q_sm = v_sm + v_slots * d_blocks * 8192;
    uint8_t* o_sm = q_sm + p.q_slots * d_blocks * 16384;
    struct Sync {
        uint64_t k_loaded, v_loaded, q_full[2], q_empty[2], v_full[2], v_empty[2], s_full, s_free, p_ready, o_done;
        uint32_t tmem_base;
        int abort;
    };
    Sync& sy = *reinterpret_cast<Sync*>(o_sm + 4 * d_blocks * 4096);
    // the warp index through a shuffle: the compiler then knows it is the same in all lanes and
    // keeps what depends only on it (the MMA warp's addresses and descriptors) in uniform registers
    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    const int head = blockIdx.y, img = blockIdx.z;
    const int tiles_total = (p.m_e + kAggBM - 1) / kAggBM;
    const int first = blockIdx.x * p.tiles_per_block;
    const int n_tiles = min(p.tiles_per_block, tiles_total - first);
    volatile int* abort = &sy.abort;
    const uint32_t tmem_cols = attn_tmem_cols(d_pad, s);
    const uint32_t o_col = (uint32_t)(s >> 1);
    const int q_slots = p.q_slots;

    if (threadIdx.x == 0) {
        mbar_init(&sy.k_loaded, 1);
        mbar_init(&sy.v_loaded, 1);
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sy.q_full[b], 1);
            mbar_init(&sy.q_empty[b], 1);
            mbar_init(&sy.v_full[b], 1);
            mbar_init(&sy.v_empty[b], 1);
        }
        mbar_init(&sy.s_full, 1);
        mbar_init(&sy.s_free, 4);   // one arrival per softmax warp
        mbar_init(&sy.p_ready, 4);
        mbar_init(&sy.o_done, 1);
        sy.abort = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(&sy.tmem_base, tmem_cols);
    wait_for_prior_kernels();
    if (misplaced && threadIdx.x == 0) atomicCAS(p.error, 0, kAggMisaligned);
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = sy.tmem_base;
    const bool stop = misplaced || *p.error != 0 || n_tiles <= 0;

    // A wait on a "free / empty" barrier uses the opposite parity, so the first pass over a
    // fresh barrier falls through.
    if (warp == 0 && lane == 0 && !stop) {
        // ---- producer.  Columns of this head: d real ones from head * d in Q, d_ld (zero padded)
        // from head * d_ld in K_c and V_c; a 64-column box that runs past the head brings the next
        // head's columns (or the zero fill past the tensor), which meet zeros of K_c in the first
        // chain and are never read by the second.
        const int qx = head * d, kx = head * p.d_ld;
        mbar_expect_tx(&sy.k_loaded, d_blocks * s * 128);
        for (int db = 0; db < d_blocks; ++db)
            for (int r0 = 0; r0 < s; r0 += 64)  // boxes of 64 anchors
                tma_load_3d(k_sm + db * s * 128 + r0 * 128, &map_k, kx + db * 64, r0, img, &sy.k_loaded);
        uint32_t v_it = 0;  // V_c blocks streamed so far
        bool ok = true;
        for (int t = 0; ok && t < n_tiles; ++t) {
            const int st = t % q_slots, round = t / q_slots;
            if (!mbar_wait(&sy.q_empty[st], (round & 1) ^ 1, abort, p.error, kAggTimeoutEmpty)) break;
            mbar_expect_tx(&sy.q_full[st], d_blocks * 16384);
            for (int db = 0; db < d_blocks; ++db)
                tma_load_3d(q_sm + (st * d_blocks + db) * 16384, &map_q, qx + db * 64, (first + t) * kAggBM, img,
                            &sy.q_full[st]);
            if (p.v_stream) {
                for (int sb = 0; sb < s_blocks; ++sb, ++v_it) {
                    const int slot = v_it & 1;
                    ok = mbar_wait(&sy.v_empty[slot], ((v_it >> 1) & 1) ^ 1, abort, p.error, kAggTimeoutEmpty);
                    if (!ok) break;
                    mbar_expect_tx(&sy.v_full[slot], d_blocks * 8192);
                    for (int db = 0; db < d_blocks; ++db)
                        tma_load_3d(v_sm + (slot * d_blocks + db) * 8192, &map_v, kx + db * 64, sb * 64, img,
                                    &sy.v_full[slot]);
                }
            } else if (t == 0) {  // V_c is not needed before the second chain of the first tile
                mbar_expect_tx(&sy.v_loaded, s_blocks * d_blocks * 8192);
                for (int sb = 0; sb < s_blocks; ++sb)
                    for (int db = 0; db < d_blocks; ++db)
                        tma_load_3d(v_sm + (sb * d_blocks + db) * 8192, &map_v, kx + db * 64, sb * 64, img,
                                    &sy.v_loaded);
            }
        }
        if (*abort) {  // copies still in flight after a time-out: give them ample time to land
            const long long t0 = clock64();
            while ((unsigned long long)(clock64() - t0) < (1ull << 22)) {}
        }
    } else if (warp == 1 && !stop) {
        // ---- MMA issue.  The whole warp walks the loop and the waits in step, one elected lane
        // issues: a lone lane would hold every operand in its own registers and pay for moving
        // them to the uniform registers the instruction reads, which made the 16 MMAs of the
        // second chain take longer to issue than to run.  One descriptor per shared-memory
        // operand, built once; a tile or K step further on only moves the start-address field
        // (16-byte units in the low bits; shared memory addresses never carry out of it).
        const int n_first = min(s, 256);  // an MMA is at most 256 columns wide: S takes one or two per K step
        const uint32_t idesc1a = umma_idesc(n_first, 0), idesc1b = umma_idesc(s - n_first > 0 ? s - n_first : 16, 0);
        const uint32_t idesc2 = umma_idesc(d_pad, 1);
        const uint64_t desc_q = umma_desc(smem_u32(q_sm), 16, 1024), desc_k = umma_desc(smem_u32(k_sm), 16, 1024);
        const uint64_t desc_v = umma_desc(smem_u32(v_sm), 8192, 1024);
        const int k_steps = d_pad >> 4;
        auto wait = [&](uint64_t* bar, uint32_t parity, int code) {
            return __all_sync(0xFFFFFFFFu, mbar_wait(bar, parity, abort, p.error, code)) != 0;
        };
        bool ok = wait(&sy.k_loaded, 0, kAggTimeoutFull);
        uint32_t v_it = 0;
        for (int t = 0; ok && t < n_tiles; ++t) {
            const int st = t % q_slots, round = t / q_slots;
            // S[128, s] = Q(t) K_c^T, K = d_pad; the previous tile's O has been read out of these columns
            if (!(ok = wait(&sy.q_full[st], round & 1, kAggTimeoutFull))) break;
            if (!(ok = wait(&sy.s_free, (t & 1) ^ 1, kAggTimeoutAcc))) break;
            tc_fence_after_sync();
            for (int kk = 0; kk < k_steps; ++kk) {
                const int db = kk >> 2, sub = kk & 3;
                const uint64_t a = desc_q + (uint64_t)(((st * d_blocks + db) * 16384) >> 4) + 2 * sub;
                const uint64_t b = desc_k + (uint64_t)((db * s * 128) >> 4) + 2 * sub;
                if (elect_one()) {
                    umma_bf16(tmem_base, a, b, idesc1a, kk != 0);
                    if (s > 256) umma_bf16(tmem_base + 256, a, b + (uint64_t)((256 * 128) >> 4), idesc1b, kk != 0);
                }
            }
            if (elect_one()) {
                umma_commit(&sy.q_empty[st]);
                umma_commit(&sy.s_full);
            }
            __syncwarp();
            if (!p.v_stream && t == 0 && !(ok = wait(&sy.v_loaded, 0, kAggTimeoutFull))) break;
            // O[128, d_pad] = P V_c, K = s: A from TMEM (8 columns per K step of 16), B blocks of 64
            // anchors are d_blocks x 8 KB apart, K steps inside a block 2 KB
            if (!(ok = wait(&sy.p_ready, t & 1, kAggTimeoutAcc))) break;
            tc_fence_after_sync();
            for (int sb = 0; sb < s_blocks; ++sb) {
                int v_block = sb;
                if (p.v_stream) {
                    v_block = v_it & 1;
                    if (!(ok = wait(&sy.v_full[v_block], (v_it >> 1) & 1, kAggTimeoutFull))) break;
                    tc_fence_after_sync();
                }
                const uint64_t b = desc_v + (uint64_t)((v_block * d_blocks * 8192) >> 4);
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
                    if (elect_one())
                        umma_bf16_a_tmem(tmem_base + o_col, tmem_base + (uint32_t)(sb * 32 + kk * 8), b + 128 * kk, idesc2,
                                         (sb | kk) != 0);
                if (p.v_stream) {
                    if (elect_one()) umma_commit(&sy.v_empty[v_block]);
                    ++v_it;
                }
            }
            if (!ok) break;
            if (elect_one()) umma_commit(&sy.o_done);
            __syncwarp();
        }
    } else if (warp >= 2 && !stop) {
        // ---- softmax and output: thread = query row (TMEM lane) 32 * (warp % 4) + lane
        const int quarter = warp & 3;
        const uint32_t tm = tmem_base + ((uint32_t)(quarter * 32) << 16);
        uint8_t* o_stage = o_sm + (warp - 2) * d_blocks * 4096;  // [d_blocks][32 rows x 128 B], swizzled
        const int full_blocks = d >> 6, tail = d & 63;           // 64-column blocks of the output, columns of the last
        const int o_cols = round_up_int(d_pad, 32);
        for (int t = 0; t < n_tiles; ++t) {
            if (!__all_sync(0xFFFFFFFFu, mbar_wait(&sy.s_full, t & 1, abort, p.error, kAggTimeoutAcc))) break;
            tc_fence_after_sync();
            float mx4[4] = {-3.0e38f, -3.0e38f, -3.0e38f, -3.0e38f};  // four chains instead of one
            for_each_chunk(tm, s, [&](const uint32_t (&acc)[32], int) {
#pragma unroll
                for (int c = 0; c < 32; c += 2)
                    mx4[(c >> 1) & 3] = fmax3(mx4[(c >> 1) & 3], __uint_as_float(acc[c]), __uint_as_float(acc[c + 1]));
            });
            const float shift = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * p.scale_log2e;
            // P(row, c) for the 16 columns of a chunk -> 8 packed columns at c / 2: always behind
            // the columns of S this thread has already taken into registers
            float row_sum = 0.f;
            for_each_chunk16(tm, s, [&](const uint32_t (&acc)[16], int c0) {
                uint32_t w[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    // The weights are cut to bf16 (upper halves of the fp32 words), not rounded: a
                    // rounding conversion shares its pipe with exp2, which already bounds this
                    // pass.  The row sum adds the cut values, so the common part of the error
                    // cancels in O / row sum.
                    const float a0 = fmaf(__uint_as_float(acc[2 * e]), p.scale_log2e, -shift);
                    const float a1 = fmaf(__uint_as_float(acc[2 * e + 1]), p.scale_log2e, -shift);
                    const uint32_t x0 = __float_as_uint(((kPolyMask >> (2 * e)) & 1u) ? exp2_poly(a0) : exp2_fast(a0));
                    const uint32_t x1 = __float_as_uint(((kPolyMask >> (2 * e + 1)) & 1u) ? exp2_poly(a1) : exp2_fast(a1));
                    row_sum += __uint_as_float(x0 & 0xFFFF0000u) + __uint_as_float(x1 & 0xFFFF0000u);
                    w[e] = __byte_perm(x0, x1, 0x7632);  // x0's upper half below x1's
                }
                tmem_store8(tm + (uint32_t)(c0 >> 1), w);
            });
            tmem_store_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sy.p_ready);
            if (!__all_sync(0xFFFFFFFFu, mbar_wait(&sy.o_done, t & 1, abort, p.error, kAggTimeoutAcc))) break;
            tc_fence_after_sync();
            const float inv = 1.f / row_sum;  // at least one term is exp2(0) = 1
            if (lane == 0) tma_store_wait_read();  // the previous tile's store has read the staging rows
            __syncwarp();
            for_each_chunk(tm + o_col, o_cols, [&](const uint32_t (&acc)[32], int c0) {
                if (c0 + 32 >= o_cols) {  // the last of O is in registers: the next tile's S may overwrite it
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sy.s_free);
                }
                const int blk = c0 >> 6;  // 64-column block of the output
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    const int col = c0 + q4 * 8;  // first of 8 output columns = one 16-byte piece
                    if (col >= d) continue;       // padding behind the head's last column
                    uint32_t w[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(acc[q4 * 8 + 2 * e]) * inv,
                                                                       __uint_as_float(acc[q4 * 8 + 2 * e + 1]) * inv);
                        w[e] = *reinterpret_cast<const uint32_t*>(&h);
                    }
                    const int piece = (col & 63) >> 3;
                    uint8_t* at = blk < full_blocks
                                      ? o_stage + blk * 4096 + lane * 128 + ((piece ^ (lane & 7)) << 4)  // swizzled box of 64 columns
                                      : o_stage + blk * 4096 + lane * (tail * 2) + (piece << 4);         // plain box of `tail` columns
                    *reinterpret_cast<uint4*>(at) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            });
            fence_async_smem();  // the bulk store reads the staging rows through the async proxy
            __syncwarp();
            if (lane == 0) {
                const int m_first = (first + t) * kAggBM + quarter * 32;
                if (m_first < p.m_e) {  // rows past m_e are clipped by the store
                    for (int db = 0; db < full_blocks; ++db)
                        tma_store_3d(&map_o, o_stage + db * 4096, head * d + db * 64, m_first, img);
                    if (tail) tma_store_3d(&map_o_tail, o_stage + full_blocks * 4096, head * d + full_blocks * 64, m_first, img);
                }
            }
        }
        if (lane == 0) tma_store_wait_read();
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, tmem_cols);
    }
}

}  // namespace civic
