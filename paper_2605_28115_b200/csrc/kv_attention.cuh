// KV-compressed visual attention (Eq. 9 of the paper) for already projected Q, K, V:
//
//     K_c = Rbar^T K,  V_c = Rbar^T V,  Attn_c = softmax(Q K_c^T / sqrt(d)) V_c   per head
//
// R [m_e, s] assigns the m_e compact tokens to s memory anchors; Rbar is R with every column
// divided by its sum.  The compression is a GEMM of the persistent template (CompressOp in
// aggregate.cuh), one launch for K and V together.  This file holds the preparation of R and the
// attention itself: ONE PERSISTENT BLOCK PER SM that walks a contiguous share of all (image, head,
// query tile) triples.  Per tile of 128 queries there are two MMA chains and one softmax between
// them, with no running maximum to maintain; the block's warps form a pipeline over the tiles:
//   TMA      K_c[:, head] [s, d] (K-major) and V_c[:, head] [s, d] (MN-major) whenever the (head,
//            image) pair changes, into the other shared-memory slot; Q tiles [128, d] into a ring
//   MMA 1    S = Q K_c^T into one of two tensor-memory buffers (the tile ahead of the softmax)
//   softmax  two warps per query row, each with half of the anchors: maximum, exp2, row sum; P cut
//            to bf16 and packed straight back into tensor memory behind the warp's own reads of S
//   MMA 2    O = P V_c with the A operand read from tensor memory, into the columns between the
//            two halves of P.  (With P in shared memory this chain was bound by shared-memory
//            reads: 4 KB of P for every 2 KB of V_c and only 64 or 128 output columns to amortise.)
//   output   O / row sum as bf16, staged in swizzled shared memory, one bulk tensor store per
//            32 rows x 32 columns; the buffer then takes the scores of the tile after next
// Every wait is bounded as in aggregate.cuh.
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

// warp 0: TMA, warp 1: TMEM + MMA, warps 2..9 and 10..17: two groups of softmax warps (one per tensor
// memory buffer, i.e. the even and the odd tiles), warps 18..21: output
constexpr int kAttnThreads = 704;

struct AttnParams {
    int* error;
    int32_t m_e, s;
    int32_t d;                // head dimension (a multiple of 8)
    int32_t d_pad;            // d rounded up to a multiple of 16: the K of the first chain, the N of the second
    int32_t d_ld;             // columns per head of K_c and V_c (d_pad: zero columns behind the d real ones)
    int32_t n_heads;
    int32_t q_tiles;          // query tiles of 128 rows per (head, image) pair
    int32_t total_tiles;      // over all pairs; blocks take contiguous, equal shares
    int32_t n_buf;            // S / P / O buffers in tensor memory: 2 (tiles overlap), or 1 where a tile needs more than 256 columns
    int32_t kv_slots;         // K_c / V_c copies in shared memory: 2 (the next pair loads while this one runs) or 1
    int32_t q_slots;          // Q tiles in flight: 1 .. 3
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
// 16 fp32 columns at a time (keeps the register count of the passes down), issue and wait split as
// for the 32-column loads
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
// `cols` (a multiple of 32) columns from `taddr` on in chunks of 16 with two register buffers, from
// the first column upwards or from the last chunk downwards; `body(acc, c0)` gets the chunk that
// starts at column taddr + c0.
template <class Body>
__device__ __forceinline__ void for_each_chunk16(uint32_t taddr, int cols, bool downwards, Body&& body)
{
    const int first = downwards ? cols - 16 : 0, step = downwards ? -16 : 16;
    uint32_t even[16], odd[16];
    tmem_load_issue16(taddr + first, even);
#pragma unroll 1
    for (int i = 0, c0 = first; i < cols; i += 32, c0 += 2 * step) {
        tmem_load_wait16(even);
        tmem_load_issue16(taddr + c0 + step, odd);
        body(even, c0);
        tmem_load_wait16(odd);
        if (i + 32 < cols) tmem_load_issue16(taddr + c0 + 2 * step, even);
        body(odd, c0 + step);
    }
}

// max(a, b, c) in one instruction
__device__ __forceinline__ float fmax3(float a, float b, float c)
{
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}

// x rounded up (towards +infinity) to a value with 16 zero low bits, as its upper half
__device__ __forceinline__ uint16_t upper_half_rounded_up(float x)
{
    const uint32_t b = __float_as_uint(x);
    return (uint16_t)(((b & 0x80000000u) ? b : b + 0xFFFFu) >> 16);
}

__host__ __device__ constexpr int round_up_int(int x, int a) { return (x + a - 1) / a * a; }

// Tensor memory of one tile, C columns.  The anchors are split between two sets of softmax warps:
//   S_a = scores of anchors [0, s/2)  in columns [0, s/2),      read upwards,   P_a packed into [0, s/4)
//   S_b = scores of anchors [s/2, s)  in columns [C - s/2, C),  read downwards, P_b packed into [C - s/4, C)
// so that each set writes its bf16 weights behind its own reads.  The columns in the middle are free
// by the time the second chain runs: O takes [o_col, o_col + d_pad) there and is read back in chunks
// of 32 columns.  o_col is a multiple of the next power of two at or above d_pad: with the accumulator
// of the second chain at column 96 (64 wide) its 16 MMAs ran for 3700 cycles instead of 600.  Where a
// tile fits 256 columns the block holds two such buffers and works on two tiles at once.
__host__ __device__ constexpr int attn_o_align(int d_pad) { return d_pad <= 32 ? 32 : (d_pad <= 64 ? 64 : 128); }
__host__ __device__ constexpr uint32_t attn_o_col(int d_pad, int s)
{
    return (uint32_t)round_up_int(s / 4, attn_o_align(d_pad));
}
__host__ __device__ constexpr uint32_t attn_tile_cols(int d_pad, int s)
{
    const int mid = (int)attn_o_col(d_pad, s) + round_up_int(d_pad, 32) + s / 4;
    const int need = s > mid ? s : mid;
    return need <= 32 ? 32u : (need <= 64 ? 64u : (need <= 128 ? 128u : (need <= 256 ? 256u : 512u)));
}
__host__ __device__ constexpr int attn_buffers(int d_pad, int s) { return attn_tile_cols(d_pad, s) <= 256 ? 2 : 1; }
__host__ __device__ constexpr uint32_t attn_tmem_cols(int d_pad, int s)
{
    return attn_buffers(d_pad, s) * attn_tile_cols(d_pad, s);
}
// 32-column chunks of the output; an output warp stages at most two of them at a time for its 32 rows
__host__ __device__ constexpr int attn_out_chunks(int d) { return (d + 31) / 32; }
__host__ __device__ constexpr int attn_stage_chunks(int d) { return attn_out_chunks(d) < 2 ? attn_out_chunks(d) : 2; }

// Shared memory: k [kv_slots][d_blocks][s x 128 B] | v [kv_slots][s/64][d_blocks][64 x 128 B] (streamed:
// [2][d_blocks][64 x 128 B]) | q [q_slots][d_blocks][128 x 128 B] | o [4 warps][chunks][32 rows x 64 B] |
// barriers and the row maxima the two sets of softmax warps show each other; d_blocks = ceil(d_pad / 64).
// Every block of data is 1024-byte aligned; the kernel has no static shared memory, so the dynamic
// window itself starts on such a boundary (checked at run time) and no slack is set aside.
__host__ __device__ constexpr size_t attn_smem_bytes(int d, int d_pad, int s, int kv_slots, int q_slots, int v_stream)
{
    const size_t db = (size_t)(d_pad + 63) / 64;
    return (size_t)kv_slots * db * s * 128 + (size_t)(v_stream ? 2 : kv_slots * (s / 64)) * db * 8192 +
           (size_t)q_slots * db * 16384 + 4 * (size_t)attn_stage_chunks(d) * 2048 + 4096 /* barriers, row maxima and sums */;
}

// One persistent block per SM.  Its warps form a pipeline over the block's query tiles:
//   producer   K_c / V_c of a (head, image) pair whenever the pair changes (into the other slot, while the
//              previous pair is still in use), Q tiles into a ring
//   MMA        S(j) = Q K_c^T for the tile one ahead, then O(i) = P(i) V_c as soon as P(i) is complete
//   softmax    maximum, exponentials, row sums of tile i; then straight on to tile i + 1, whose scores
//              are already waiting in the other buffer
//   output     O(i) / row sum -> bf16 -> staging -> bulk tensor store, which frees the buffer for S(i + 2)
// so that the special-function unit (16 exponentials per clock and SM, the scarcest unit here) is kept
// busy by the softmax warps while everything else runs beside it.
__global__ void __launch_bounds__(kAttnThreads, 1) kv_attention_kernel(const __grid_constant__ CUtensorMap map_q,
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
    const int kv_slots = p.kv_slots, q_slots = p.q_slots, n_buf = p.n_buf;
    const int out_chunks = attn_out_chunks(d), stage_chunks = attn_stage_chunks(d);
    const int k_slot_bytes = d_blocks * s * 128, v_slot_bytes = (p.v_stream ? 1 : s_blocks) * d_blocks * 8192;
    uint8_t* k_sm = base;
    uint8_t* v_sm = k_sm + kv_slots * k_slot_bytes;
    uint8_t* q_sm = v_sm + (p.v_stream ? 2 : kv_slots) * v_slot_bytes;
    uint8_t* o_sm = q_sm + q_slots * d_blocks * 16384;
    struct Sync {
        uint64_t kv_full[2], kv_empty[2], q_full[3], q_empty[3], v_full[2], v_empty[2];
        uint64_t s_full[2], s_free[2], p_ready[2], o_done[2];
        uint64_t pair[2][4];          // per group: the two softmax warps of a TMEM lane quarter meet here once per tile
        uint16_t row_max[2][2][128];  // per group and side of the anchor split: upper half of the row maximum, rounded up
        float row_sum[2][2][128];  // per buffer and side: sum of the row's cut weights, for the output warps
        uint32_t tmem_base;
        int abort;
    };
    static_assert(sizeof(Sync) <= 4096, "the barrier area is 4 KB");
    Sync& sy = *reinterpret_cast<Sync*>(o_sm + 4 * stage_chunks * 2048);
    // the warp index through a shuffle: the compiler then knows it is the same in all lanes and
    // keeps what depends only on it (the MMA warp's addresses and descriptors) in uniform registers
    const int warp = __shfl_sync(0xFFFFFFFFu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
    // this block's tiles: [g0, g0 + n_tiles) of the list ordered by (image, head, query tile)
    const int g0 = (int)((long long)p.total_tiles * blockIdx.x / gridDim.x);
    const int n_tiles = (int)((long long)p.total_tiles * (blockIdx.x + 1) / gridDim.x) - g0;
    volatile int* abort = &sy.abort;
    const uint32_t tile_cols = attn_tile_cols(d_pad, s);
    const uint32_t tmem_cols = attn_tmem_cols(d_pad, s);
    const uint32_t o_col = attn_o_col(d_pad, s);
    const int half_s = s >> 1;
    const uint32_t sb_col = tile_cols - (uint32_t)half_s;         // first column of S_b
    const uint32_t pb_col = tile_cols - (uint32_t)(half_s >> 1);  // first column of P_b

    if (threadIdx.x == 0) {
        for (int b = 0; b < 2; ++b) {
            mbar_init(&sy.kv_full[b], 1);
            mbar_init(&sy.kv_empty[b], 1);
            mbar_init(&sy.v_full[b], 1);
            mbar_init(&sy.v_empty[b], 1);
            mbar_init(&sy.s_full[b], 1);
            mbar_init(&sy.s_free[b], 4);   // one arrival per output warp
            mbar_init(&sy.p_ready[b], 8);  // one arrival per softmax warp
            mbar_init(&sy.o_done[b], 1);
        }
        for (int b = 0; b < 3; ++b) {
            mbar_init(&sy.q_full[b], 1);
            mbar_init(&sy.q_empty[b], 1);
        }
        for (int q = 0; q < 8; ++q) mbar_init(&sy.pair[q >> 2][q & 3], 2);  // one arrival per warp
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
    if (warp == 0 && !stop) {
        // ---- producer (the whole warp in step, an elected lane issues: see the MMA warp).  Columns of a
        // head: d real ones from head * d in Q, d_ld (zero padded) from head * d_ld in K_c and V_c; a
        // 64-column box that runs past the head brings the next head's columns (or the zero fill past
        // the tensor), which meet zeros of K_c in the first chain and are never read by the second.
        auto wait = [&](uint64_t* bar, uint32_t parity) {
            return __all_sync(0xFFFFFFFFu, mbar_wait(bar, parity, abort, p.error, kAggTimeoutEmpty)) != 0;
        };
        uint32_t v_it = 0;  // V_c blocks streamed so far
        int kv_seq = -1;
        int pair = g0 / p.q_tiles, tile = g0 - pair * p.q_tiles;
        bool ok = true, new_pair = true;
        for (int i = 0; ok && i < n_tiles; ++i) {
            const int img = pair / p.n_heads, head = pair - img * p.n_heads;
            const int qx = head * d, kx = head * p.d_ld;
            if (new_pair) {
                ++kv_seq;
                const int slot = kv_seq % kv_slots, round = kv_seq / kv_slots;
                if (!(ok = wait(&sy.kv_empty[slot], (round & 1) ^ 1))) break;
                if (elect_one()) {
                    mbar_expect_tx(&sy.kv_full[slot], k_slot_bytes + (p.v_stream ? 0 : v_slot_bytes));
                    for (int db = 0; db < d_blocks; ++db)
                        for (int r0 = 0; r0 < s; r0 += 64)  // boxes of 64 anchors
                            tma_load_3d(k_sm + slot * k_slot_bytes + db * s * 128 + r0 * 128, &map_k, kx + db * 64, r0, img,
                                        &sy.kv_full[slot]);
                    if (!p.v_stream)
                        for (int sb = 0; sb < s_blocks; ++sb)
                            for (int db = 0; db < d_blocks; ++db)
                                tma_load_3d(v_sm + slot * v_slot_bytes + (sb * d_blocks + db) * 8192, &map_v, kx + db * 64,
                                            sb * 64, img, &sy.kv_full[slot]);
                }
                __syncwarp();
            }
            const int st = i % q_slots;
            if (!(ok = wait(&sy.q_empty[st], ((i / q_slots) & 1) ^ 1))) break;
            if (elect_one()) {
                mbar_expect_tx(&sy.q_full[st], d_blocks * 16384);
                for (int db = 0; db < d_blocks; ++db)
                    tma_load_3d(q_sm + (st * d_blocks + db) * 16384, &map_q, qx + db * 64, tile * kAggBM, img, &sy.q_full[st]);
            }
            __syncwarp();
            if (p.v_stream) {
                for (int sb = 0; sb < s_blocks; ++sb, ++v_it) {
                    const int slot = v_it & 1;
                    if (!(ok = wait(&sy.v_empty[slot], ((v_it >> 1) & 1) ^ 1))) break;
                    if (elect_one()) {
                        mbar_expect_tx(&sy.v_full[slot], d_blocks * 8192);
                        for (int db = 0; db < d_blocks; ++db)
                            tma_load_3d(v_sm + (slot * d_blocks + db) * 8192, &map_v, kx + db * 64, sb * 64, img,
                                        &sy.v_full[slot]);
                    }
                    __syncwarp();
                }
            }
            new_pair = ++tile == p.q_tiles;
            if (new_pair) { tile = 0; ++pair; }
        }
        if (*abort && lane == 0) {  // copies still in flight after a time-out: give them ample time to land
            const long long t0 = clock64();
            while ((unsigned long long)(clock64() - t0) < (1ull << 22)) {}
        }
    } else if (warp == 1 && !stop) {
        // ---- MMA issue.  The whole warp walks the loops and the waits in step, one elected lane
        // issues.  The instruction reads its operands from uniform registers: whatever the compiler
        // cannot prove to be the same in all lanes it moves there one value at a time, which made an
        // MMA take 100 .. 200 cycles to issue instead of 40.  So everything that changes per tile is
        // computed once per tile and broadcast from lane 0 (after which it is provably uniform), and
        // the inner loops only add constants to it.  Descriptors: one per shared-memory operand,
        // built once; a slot, tile or K step further on only moves the start-address field (16-byte
        // units in the low 32 bits; shared memory addresses never carry out of it).
        auto uni = [](uint32_t v) { return __shfl_sync(0xFFFFFFFFu, v, 0); };
        const uint32_t idesc1 = umma_idesc(half_s, 0), idesc2 = umma_idesc(d_pad, 1);
        const bool one_wide = sb_col == (uint32_t)half_s && s <= 256;
        const uint32_t idesc1w = umma_idesc(one_wide ? s : 16, 0);
        const uint64_t desc_q = umma_desc(smem_u32(q_sm), 16, 1024), desc_k = umma_desc(smem_u32(k_sm), 16, 1024);
        const uint64_t desc_v = umma_desc(smem_u32(v_sm), 8192, 1024);
        const uint32_t hi_q = (uint32_t)(desc_q >> 32), hi_k = (uint32_t)(desc_k >> 32), hi_v = (uint32_t)(desc_v >> 32);
        auto desc = [](uint32_t hi, uint32_t lo) { return ((uint64_t)hi << 32) | lo; };
        const int k_steps = d_pad >> 4, half16 = half_s >> 4;
        const uint32_t k_db_step = (uint32_t)((s * 128) >> 4), k_half = (uint32_t)((half_s * 128) >> 4);
        const uint32_t v_blk_step = (uint32_t)((d_blocks * 8192) >> 4);
        auto wait = [&](uint64_t* bar, uint32_t parity, int code) {
            return __all_sync(0xFFFFFFFFu, mbar_wait(bar, parity, abort, p.error, code)) != 0;
        };
        bool ok = true;
        uint32_t v_it = 0;
        int next = 0;                                    // first tile whose scores have not been issued yet
        int pair1 = g0 / p.q_tiles, left1 = p.q_tiles - (g0 - pair1 * p.q_tiles);  // pair of tile `next`, its tiles left
        int pair2 = pair1, left2 = left1;                // the same for tile i of the output stream
        int seq1 = -1, last1 = -1;                       // pair sequence number of the scores stream
        int seq2 = -1, last2 = -1;                       // ... of the output stream, which lags behind
        for (int i = 0; ok && i < n_tiles; ++i) {
            // scores of the tiles ahead: as many as there are buffers, and never into a K_c slot
            // that a pair still waiting for its second chain occupies
            while (ok && next < n_tiles && next < i + n_buf) {
                if (pair1 != last1) {
                    if (seq1 + 1 - (pair2 == last2 ? seq2 : seq2 + 1) >= kv_slots) break;
                    last1 = pair1;
                    ++seq1;
                    if (!(ok = wait(&sy.kv_full[seq1 % kv_slots], (seq1 / kv_slots) & 1, kAggTimeoutFull))) break;
                }
                const int j = next, st = j % q_slots, buf = j % n_buf, k_slot = seq1 % kv_slots;
                // S_a, S_b [128, s/2] = Q(j) K_c^T, K = d_pad, once the buffer's last O has been read out
                if (!(ok = wait(&sy.q_full[st], (j / q_slots) & 1, kAggTimeoutFull))) break;
                if (!(ok = wait(&sy.s_free[buf], ((j / n_buf) & 1) ^ 1, kAggTimeoutAcc))) break;
                tc_fence_after_sync();
                const uint32_t tb = uni(tmem_base + (uint32_t)buf * tile_cols);
                const uint32_t a0 = uni((uint32_t)desc_q + (uint32_t)((st * d_blocks * 16384) >> 4));
                const uint32_t b0 = uni((uint32_t)desc_k + (uint32_t)((k_slot * k_slot_bytes) >> 4));
                if (one_wide) {  // S_a and S_b lie side by side: one MMA of s columns per K step
                    for (int kk = 0; kk < k_steps; ++kk) {
                        const uint32_t a = a0 + (uint32_t)(kk >> 2) * 1024u + 2u * (uint32_t)(kk & 3);
                        const uint32_t b = b0 + (uint32_t)(kk >> 2) * k_db_step + 2u * (uint32_t)(kk & 3);
                        if (elect_one()) umma_bf16(tb, desc(hi_q, a), desc(hi_k, b), idesc1w, kk != 0);
                    }
                } else {
                    for (int kk = 0; kk < k_steps; ++kk) {
                        const uint32_t a = a0 + (uint32_t)(kk >> 2) * 1024u + 2u * (uint32_t)(kk & 3);
                        const uint32_t b = b0 + (uint32_t)(kk >> 2) * k_db_step + 2u * (uint32_t)(kk & 3);
                        if (elect_one()) {
                            umma_bf16(tb, desc(hi_q, a), desc(hi_k, b), idesc1, kk != 0);
                            umma_bf16(tb + sb_col, desc(hi_q, a), desc(hi_k, b + k_half), idesc1, kk != 0);
                        }
                    }
                }
                if (elect_one()) {
                    umma_commit(&sy.q_empty[st]);
                    umma_commit(&sy.s_full[buf]);
                }
                __syncwarp();
                ++next;
                if (--left1 == 0) { ++pair1; left1 = p.q_tiles; }
            }
            if (!ok) break;
            // O(i)[128, d_pad] = P V_c, K = s in steps of 16 anchors: A from TMEM (8 columns per step;
            // P_a for the first half of the anchors, P_b for the second), B blocks of 64 anchors are
            // d_blocks x 8 KB apart, steps inside a block 2 KB
            if (pair2 != last2) { last2 = pair2; ++seq2; }
            const int buf = i % n_buf, v_slot = seq2 % kv_slots;
            if (!(ok = wait(&sy.p_ready[buf], (i / n_buf) & 1, kAggTimeoutAcc))) break;
            tc_fence_after_sync();
            const uint32_t tb = uni(tmem_base + (uint32_t)buf * tile_cols);
            const uint32_t to = tb + o_col, pa = tb, pb = tb + pb_col - (uint32_t)(half16 * 8);
            if (!p.v_stream) {
                const uint32_t v0 = uni((uint32_t)desc_v + (uint32_t)((v_slot * v_slot_bytes) >> 4));
                if ((half16 & 3) == 0) {  // both halves are whole blocks of 64 anchors: four K steps per block
                    for (int sb = 0; sb < s_blocks; ++sb) {
                        const uint32_t b = v0 + (uint32_t)sb * v_blk_step;
                        const uint32_t a = (sb * 4 < half16 ? pa : pb) + (uint32_t)(sb * 32);
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            if (elect_one())
                                umma_bf16_a_tmem(to, a + 8u * kk, desc(hi_v, b + 128u * kk), idesc2, (sb | kk) != 0);
                    }
                } else {
                    for (int k16 = 0; k16 < 2 * half16; ++k16) {
                        const uint32_t b = v0 + (uint32_t)(k16 >> 2) * v_blk_step + 128u * (uint32_t)(k16 & 3);
                        const uint32_t a = (k16 < half16 ? pa : pb) + (uint32_t)(k16 * 8);
                        if (elect_one()) umma_bf16_a_tmem(to, a, desc(hi_v, b), idesc2, k16 != 0);
                    }
                }
            } else {
                for (int sb = 0; sb < s_blocks; ++sb, ++v_it) {
                    const int slot = v_it & 1;
                    if (!(ok = wait(&sy.v_full[slot], (v_it >> 1) & 1, kAggTimeoutFull))) break;
                    tc_fence_after_sync();
                    const uint32_t v0 = uni((uint32_t)desc_v + (uint32_t)((slot * d_blocks * 8192) >> 4));
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk) {
                        const int k16 = sb * 4 + kk;
                        const uint32_t a = (k16 < half16 ? pa : pb) + (uint32_t)(k16 * 8);
                        if (elect_one()) umma_bf16_a_tmem(to, a, desc(hi_v, v0 + 128u * (uint32_t)kk), idesc2, k16 != 0);
                    }
                    if (elect_one()) umma_commit(&sy.v_empty[slot]);
                }
                if (!ok) break;
            }
            const bool pair_ends = left2 == 1 || i + 1 == n_tiles;  // its K_c / V_c slot may be loaded again
            if (elect_one()) {
                umma_commit(&sy.o_done[buf]);
                if (pair_ends) umma_commit(&sy.kv_empty[v_slot]);
            }
            __syncwarp();
            if (--left2 == 0) { ++pair2; left2 = p.q_tiles; }
        }
    } else if (warp >= 2 && warp < 18 && !stop) {
        // ---- softmax.  Two groups of eight warps: with two buffers group g takes the tiles i = g, g + 2,
        // ... (buffer g), so that two tiles are in different phases of their softmax at any time and
        // the special-function unit is not left idle while one tile looks for its maxima; with one
        // buffer group 0 takes every tile.  Within a group: thread = query row (TMEM lane)
        // 32 * (warp % 4) + lane and one side of the anchor split, S_a upwards or S_b downwards.  The two
        // threads of a row agree on the shift of the exponentials through shared memory (each side's
        // maximum, rounded up to 16 significant bits: any common shift at or above the true maximum
        // is as good as the maximum itself) and leave their row sums in shared memory for the output
        // warps.
        const int group = (warp - 2) >> 3, quarter = warp & 3, side = ((warp - 2) >> 2) & 1;
        const int row = quarter * 32 + lane;
        const uint32_t s_col = side ? sb_col : 0u, p_col = side ? pb_col : 0u;
        for (int i = group, turn = 0; i < n_tiles && group < n_buf; i += n_buf, ++turn) {
            const int buf = group;
            const uint32_t tm = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)buf * tile_cols;
            if (!__all_sync(0xFFFFFFFFu, mbar_wait(&sy.s_full[buf], (i / n_buf) & 1, abort, p.error, kAggTimeoutAcc))) break;
            tc_fence_after_sync();
            float mx4[4] = {-3.0e38f, -3.0e38f, -3.0e38f, -3.0e38f};  // four chains instead of one
            for_each_chunk16(tm + s_col, half_s, false, [&](const uint32_t (&acc)[16], int) {
#pragma unroll
                for (int c = 0; c < 16; c += 2)
                    mx4[(c >> 1) & 3] = fmax3(mx4[(c >> 1) & 3], __uint_as_float(acc[c]), __uint_as_float(acc[c + 1]));
            });
            sy.row_max[group][side][row] = upper_half_rounded_up(fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])));
            __syncwarp();
            if (lane == 0) mbar_arrive(&sy.pair[group][quarter]);
            if (!__all_sync(0xFFFFFFFFu, mbar_wait(&sy.pair[group][quarter], turn & 1, abort, p.error, kAggTimeoutAcc))) break;
            const float m_a = __uint_as_float((uint32_t)sy.row_max[group][0][row] << 16);
            const float m_b = __uint_as_float((uint32_t)sy.row_max[group][1][row] << 16);
            const float shift = fmaxf(m_a, m_b) * p.scale_log2e;
            // P(row, c) for the 16 columns of a chunk -> 8 packed columns at c / 2: always behind the
            // columns of S this thread has already taken into registers (side b: above them, going down)
            float sum4[4] = {0.f, 0.f, 0.f, 0.f};
            for_each_chunk16(tm + s_col, half_s, side != 0, [&](const uint32_t (&acc)[16], int c0) {
                uint32_t w[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    // The weights are cut to bf16 (upper halves of the fp32 words), not rounded: a
                    // rounding conversion shares its pipe with exp2.  The row sum adds the cut values,
                    // so the common part of the error cancels in O / row sum.
                    const uint32_t x0 = __float_as_uint(exp2_fast(fmaf(__uint_as_float(acc[2 * e]), p.scale_log2e, -shift)));
                    const uint32_t x1 = __float_as_uint(exp2_fast(fmaf(__uint_as_float(acc[2 * e + 1]), p.scale_log2e, -shift)));
                    sum4[e & 3] += __uint_as_float(x0 & 0xFFFF0000u) + __uint_as_float(x1 & 0xFFFF0000u);
                    w[e] = __byte_perm(x0, x1, 0x7632);  // x0's upper half below x1's
                }
                tmem_store8(tm + p_col + (uint32_t)(c0 >> 1), w);
            });
            sy.row_sum[buf][side][row] = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
            tmem_store_wait();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sy.p_ready[buf]);
        }
    } else if (warp >= 18 && !stop) {
        // ---- output: warp = TMEM lane quarter (warp % 4), thread = query row.  O / (sum_a + sum_b) as
        // bf16 through swizzled staging rows and one bulk tensor store per 32 columns.
        const int quarter = warp & 3;
        uint8_t* o_stage = o_sm + (warp - 18) * stage_chunks * 2048;  // [1 or 2 chunks][32 rows x 64 B]
        const int full_chunks = d >> 5, tail = d & 31;
        for (int i = 0; i < n_tiles; ++i) {
            const int buf = i % n_buf;
            const int pair = (g0 + i) / p.q_tiles, tile = (g0 + i) - pair * p.q_tiles;
            const int img = pair / p.n_heads, head = pair - img * p.n_heads;
            const int m_first = tile * kAggBM + quarter * 32;
            const uint32_t tm = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)buf * tile_cols;
            if (!__all_sync(0xFFFFFFFFu, mbar_wait(&sy.o_done[buf], (i / n_buf) & 1, abort, p.error, kAggTimeoutAcc))) break;
            tc_fence_after_sync();
            const int row = quarter * 32 + lane;
            const float inv = 1.f / (sy.row_sum[buf][0][row] + sy.row_sum[buf][1][row]);  // the largest term is about 1
            for (int c0 = 0; c0 < out_chunks; c0 += 2) {  // two chunks per round through the staging rows
                const int c_end = min(c0 + 2, out_chunks);
                // both chunks of the round are asked for at once; with the last one in registers the
                // buffer may take the scores of the tile after next
                uint32_t acc[2][32];
                tmem_load_issue(tm + o_col + 32 * c0, acc[0]);
                if (c0 + 1 < c_end) tmem_load_issue(tm + o_col + 32 * (c0 + 1), acc[1]);
                tmem_load_wait(acc[0]);
                if (c0 + 1 < c_end) tmem_load_wait(acc[1]);
                if (c_end == out_chunks) {
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sy.s_free[buf]);
                }
                if (lane == 0) tma_store_wait_read();  // the previous round's stores have read the staging rows
                __syncwarp();
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int c = c0 + u;
                    if (c >= c_end) break;
                    uint32_t w[16];
#pragma unroll
                    for (int e = 0; e < 16; ++e) {
                        const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(acc[u][2 * e]) * inv,
                                                                       __uint_as_float(acc[u][2 * e + 1]) * inv);
                        w[e] = *reinterpret_cast<const uint32_t*>(&h);
                    }
                    uint8_t* box = o_stage + u * 2048;
                    if (c < full_chunks) {  // 32 rows x 64 B, 64-byte swizzle: piece j of row r at j ^ ((r >> 1) & 3)
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            *reinterpret_cast<uint4*>(box + lane * 64 + ((j ^ ((lane >> 1) & 3)) << 4)) =
                                make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
                    } else {  // the head's last `tail` columns: a plain box, rows of tail * 2 bytes
#pragma unroll
                        for (int j = 0; j < 3; ++j)
                            if (j * 8 < tail)
                                *reinterpret_cast<uint4*>(box + lane * (tail * 2) + (j << 4)) =
                                    make_uint4(w[4 * j], w[4 * j + 1], w[4 * j + 2], w[4 * j + 3]);
                    }
                }
                fence_async_smem();  // the bulk stores read the staging rows through the async proxy
                __syncwarp();
                if (lane == 0 && m_first < p.m_e)  // rows past m_e are clipped by the store
                    for (int c = c0; c < c_end; ++c)
                        tma_store_3d(c < full_chunks ? &map_o : &map_o_tail, o_stage + (c - c0) * 2048, head * d + c * 32,
                                     m_first, img);
            }
        }
        if (lane == 0) tma_store_wait_all();
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, tmem_cols);
    }
}

}  // namespace civic
