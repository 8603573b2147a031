// KV-compressed visual attention (Eq. 9 of the paper) for already projected Q, K, V:
//
//     K_c = Rbar^T K,  V_c = Rbar^T V,  Attn_c = softmax(Q K_c^T / sqrt(d)) V_c   per head
//
// R [m_e, s] assigns the m_e compact tokens to s memory anchors; Rbar is R with every column
// divided by its sum.  The compression is a GEMM of the persistent template (CompressOp in
// aggregate.cuh), run once for K and once for V.  This file holds the preparation of R and the
// attention itself: one block per (128 queries, head, image).  With at most 256 memory anchors a
// head's whole K_c and V_c fit in shared memory, so the block issues two MMAs chains and one
// softmax between them, with no running maximum to maintain:
//   TMA      Q tile [128, d], K_c[:, head] [s, d] (K-major) and V_c[:, head] [s, d] (MN-major)
//   MMA 1    S = Q K_c^T -> TMEM columns [0, s)
//   softmax  thread per query row: maximum, exp2, row sum; P as bf16 into 128-byte-swizzled
//            shared memory (the A operand of the second chain)
//   MMA 2    O = P V_c -> TMEM columns [0, d) again
//   store    O / row sum as bf16
// Every wait is bounded as in aggregate.cuh.
#pragma once
#include "aggregate.cuh"

namespace civic {

// R (fp32) -> bf16 copy and the column sums of the ROUNDED values (what the tensor core will
// multiply with): a block converts kAssignRows rows and writes their column sums; the compression
// GEMM's epilogue adds the panels' sums in a fixed order.
constexpr int kAssignRows = 16;
__global__ void assign_convert_kernel(const float* __restrict__ r, int m_e, int s, __nv_bfloat16* __restrict__ r16,
                                      float* __restrict__ partial)
{
    wait_for_prior_kernels();
    const int m_begin = blockIdx.x * kAssignRows, m_end = min(m_begin + kAssignRows, m_e);
    for (int c = threadIdx.x; c < s; c += blockDim.x) {
        float sum = 0.f;
#pragma unroll 4
        for (int m = m_begin; m < m_end; ++m) {
            const __nv_bfloat16 v = __float2bfloat16_rn(r[(size_t)m * s + c]);
            r16[(size_t)m * s + c] = v;
            sum += __bfloat162float(v);
        }
        partial[(size_t)blockIdx.x * s + c] = sum;
    }
}
constexpr int kAttnThreads = 192;  // warp 0: TMA, warp 1: TMEM + MMA, warps 2..5: one query row per thread

struct AttnParams {
    __nv_bfloat16* out;  // [n_img, m_e, n_heads * d]
    int* error;
    int32_t m_e, n_heads, d, s;
    float scale_log2e;   // log2(e) / sqrt(d)
};

// Shared memory: region A = q [d/64][128 x 128 B] | k [d/64][s x 128 B], later overwritten by
// p [s/64][128 x 128 B] (Q and K_c are dead once the first MMA chain has completed); then
// v [s/64][d/64][64 x 128 B]; then the barriers.  Every block of data is 1024-byte aligned.
// 96 KB for 64-wide heads and 256 anchors: two blocks per SM.
__host__ __device__ constexpr size_t attn_region_a_bytes(int d, int s)
{
    const size_t qk = (size_t)(d / 64) * 16384 + (size_t)(d / 64) * s * 128, pr = (size_t)(s / 64) * 16384;
    return qk > pr ? qk : pr;
}
__host__ __device__ constexpr size_t attn_smem_bytes(int d, int s)
{
    return attn_region_a_bytes(d, s) + (size_t)(s / 64) * (d / 64) * 8192 + 1024 /* barriers */ + 1024 /* alignment slack */;
}

__global__ void __launch_bounds__(kAttnThreads) kv_attention_kernel(const __grid_constant__ CUtensorMap map_q,
                                                                    const __grid_constant__ CUtensorMap map_k,
                                                                    const __grid_constant__ CUtensorMap map_v,
                                                                    const AttnParams p)
{
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int d = p.d, s = p.s, d_blocks = d >> 6, s_blocks = s >> 6;
    uint8_t* q_sm = base;
    uint8_t* k_sm = q_sm + d_blocks * 16384;
    uint8_t* p_sm = base;  // takes over the Q / K_c region after the first MMA chain
    uint8_t* v_sm = base + attn_region_a_bytes(d, s);
    struct Sync {
        uint64_t loaded, scores_done, probs_ready, out_done;
        uint32_t tmem_base;
        int abort;
    };
    Sync& sy = *reinterpret_cast<Sync*>(v_sm + s_blocks * d_blocks * 8192);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * kAggBM, head = blockIdx.y, img = blockIdx.z;
    volatile int* abort = &sy.abort;
    // O takes over the first d columns of S (S is dead once every softmax warp has read it)
    const uint32_t tmem_cols = max(s, d) <= 64 ? 64u : (max(s, d) <= 128 ? 128u : 256u);

    if (threadIdx.x == 0) {
        mbar_init(&sy.loaded, 1);
        mbar_init(&sy.scores_done, 1);
        mbar_init(&sy.probs_ready, 4);  // one arrival per softmax warp
        mbar_init(&sy.out_done, 1);
        sy.abort = 0;
        fence_barrier_init();
    }
    if (warp == 1) tmem_alloc(&sy.tmem_base, tmem_cols);
    wait_for_prior_kernels();
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_s = sy.tmem_base, tmem_o = sy.tmem_base;
    const bool stop = *p.error != 0;

    if (warp == 0 && lane == 0 && !stop) {
        // ---- all operands of this block, one barrier
        const uint32_t bytes = d_blocks * 16384 + d_blocks * s * 128 + s_blocks * d_blocks * 8192;
        mbar_expect_tx(&sy.loaded, bytes);
        for (int db = 0; db < d_blocks; ++db) {
            tma_load_3d(q_sm + db * 16384, &map_q, head * d + db * 64, m0, img, &sy.loaded);
            for (int r0 = 0; r0 < s; r0 += 64)  // boxes of 64 anchors
                tma_load_3d(k_sm + db * s * 128 + r0 * 128, &map_k, head * d + db * 64, r0, img, &sy.loaded);
        }
        for (int sb = 0; sb < s_blocks; ++sb)
            for (int db = 0; db < d_blocks; ++db)
                tma_load_3d(v_sm + (sb * d_blocks + db) * 8192, &map_v, head * d + db * 64, sb * 64, img, &sy.loaded);
    } else if (warp == 1 && lane == 0 && !stop) {
        // ---- MMA 1: S[128, s] = Q K_c^T, K = d
        if (mbar_wait(&sy.loaded, 0, abort, p.error, kAggTimeoutFull)) {
            tc_fence_after_sync();
            const uint32_t idesc1 = umma_idesc(s, 0);
            for (int db = 0; db < d_blocks; ++db)
                for (int kk = 0; kk < 4; ++kk)
                    umma_bf16(tmem_s, umma_desc(smem_u32(q_sm + db * 16384) + kk * 32, 16, 1024),
                              umma_desc(smem_u32(k_sm + db * s * 128) + kk * 32, 16, 1024), idesc1, (db | kk) != 0);
            umma_commit(&sy.scores_done);
            // ---- MMA 2: O[128, d] = P V_c, K = s; B blocks of 64 features are 8 KB apart
            if (mbar_wait(&sy.probs_ready, 0, abort, p.error, kAggTimeoutAcc)) {
                tc_fence_after_sync();
                const uint32_t idesc2 = umma_idesc(d, 1);
                for (int sb = 0; sb < s_blocks; ++sb)
                    for (int kk = 0; kk < 4; ++kk)
                        umma_bf16(tmem_o, umma_desc(smem_u32(p_sm + sb * 16384) + kk * 32, 16, 1024),
                                  umma_desc(smem_u32(v_sm + sb * d_blocks * 8192) + kk * 2048, 8192, 1024), idesc2,
                                  (sb | kk) != 0);
                umma_commit(&sy.out_done);
            }
        }
    } else if (warp >= 2 && !stop) {
        // ---- softmax and output: thread = query row (TMEM lane) 32 * (warp % 4) + lane
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        const int m = m0 + row;
        const uint32_t lane_addr = (uint32_t)(quarter * 32) << 16;
        if (__all_sync(0xFFFFFFFFu, mbar_wait(&sy.scores_done, 0, abort, p.error, kAggTimeoutAcc))) {
            tc_fence_after_sync();
            float mx = -3.0e38f;
            for_each_chunk(tmem_s + lane_addr, s, [&](const uint32_t (&acc)[32], int) {
#pragma unroll
                for (int c = 0; c < 32; ++c) mx = fmaxf(mx, __uint_as_float(acc[c]));
            });
            const float shift = mx * p.scale_log2e;
            float row_sum = 0.f;
            for_each_chunk(tmem_s + lane_addr, s, [&](const uint32_t (&acc)[32], int c0) {
                uint8_t* blk = p_sm + (c0 >> 6) * 16384 + row * 128;  // this row in the 64-column block
                const int j0 = (c0 & 32) >> 3;                        // first 16-byte piece of the chunk
#pragma unroll
                for (int q4 = 0; q4 < 4; ++q4) {
                    uint32_t w[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const float a = exp2_fast(fmaf(__uint_as_float(acc[q4 * 8 + 2 * e]), p.scale_log2e, -shift));
                        const float b = exp2_fast(fmaf(__uint_as_float(acc[q4 * 8 + 2 * e + 1]), p.scale_log2e, -shift));
                        const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
                        row_sum += __low2float(h) + __high2float(h);
                        w[e] = *reinterpret_cast<const uint32_t*>(&h);
                    }
                    *reinterpret_cast<uint4*>(blk + (((j0 + q4) ^ (row & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            });
            fence_async_smem();      // the MMA reads P through the async proxy
            tc_fence_before_sync();  // and S has been read out of TMEM
            __syncwarp();
            if (lane == 0) mbar_arrive(&sy.probs_ready);
            if (__all_sync(0xFFFFFFFFu, mbar_wait(&sy.out_done, 0, abort, p.error, kAggTimeoutAcc))) {
                tc_fence_after_sync();
                const float inv = 1.f / row_sum;  // at least one term is exp2(0) = 1
                const bool row_ok = m < p.m_e;
                __nv_bfloat16* out = p.out + ((size_t)img * p.m_e + (row_ok ? m : 0)) * (p.n_heads * d) + head * d;
                for_each_chunk(tmem_o + lane_addr, d, [&](const uint32_t (&acc)[32], int c0) {
                    if (row_ok) {
#pragma unroll
                        for (int q4 = 0; q4 < 4; ++q4) {
                            uint32_t w[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const __nv_bfloat162 h = __floats2bfloat162_rn(__uint_as_float(acc[q4 * 8 + 2 * e]) * inv,
                                                                               __uint_as_float(acc[q4 * 8 + 2 * e + 1]) * inv);
                                w[e] = *reinterpret_cast<const uint32_t*>(&h);
                            }
                            *reinterpret_cast<uint4*>(out + c0 + q4 * 8) = make_uint4(w[0], w[1], w[2], w[3]);
                        }
                    }
                });
            }
        }
    }
    // copies still in flight after a time-out: give them ample time before the block goes away
    if (*abort && warp == 0 && lane == 0) {
        const long long t0 = clock64();
        while (!mbar_try_wait(&sy.loaded, 0) && (unsigned long long)(clock64() - t0) < kWaitLimitCycles) {}
    }
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(sy.tmem_base, tmem_cols);
    }
}

}  // namespace civic
