/*
 * civic.h -- C ABI of the CIVIC select + compact + KV-compaction library (CUDA, sm_100a).
 *
 * The library implements one hot path of CIVIC's compact inference pathway: deciding which
 * visual tokens survive, and packing the survivors' rows into contiguous, order-preserving
 * buffers so that no later stage reads non-contiguous memory.
 *
 * Conventions for every call
 *   - "dev" pointers are CUDA device pointers, "host" pointers ordinary host memory.
 *     A "dev" pointer may also be pinned, device-mapped host memory (cudaHostAlloc under
 *     unified addressing): the kernels then read only the rows they keep across PCIe and can
 *     write results straight to host memory, with no staging copy.
 *   - All buffers are owned by the caller.  Inputs are never written.  Outputs must not
 *     overlap inputs (checked where both extents are known; overlap -> CIVIC_ERR_INVALID_ARG).
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Work is
 *     enqueued on it and the call returns without synchronising.  The library allocates no
 *     device memory.  What it keeps between calls is named at the entry concerned: a launch
 *     counter, the programmatic-launch switch, the calling thread's index-check record
 *     (civic_set_index_check), per-device caches of device properties, and the contents of
 *     the scratch array built in for civic_select_large_static.
 *   - Arguments are validated on the host BEFORE anything is launched: every status other
 *     than CIVIC_OK and CIVIC_ERR_CUDA means that nothing was enqueued.  CIVIC_ERR_CUDA wraps
 *     a failed CUDA runtime call (its text is available from civic_last_cuda_error()); some
 *     entries enqueue several launches (civic_select_large, the two tensor-core calls, K/V
 *     calls over more than 80 layers, ragged batches over more than 64 segments), so after
 *     CIVIC_ERR_CUDA earlier launches of the same call may already be enqueued and its outputs
 *     and scratch are undefined.
 *   - Threads: every entry may be called from several host threads at once, on the same or
 *     different devices and streams, as long as concurrent calls do not share output or
 *     scratch buffers.  Process-wide switches (civic_set_programmatic_launch) are atomic;
 *     civic_set_index_check and civic_last_cuda_error are per calling thread.
 *   - No returned status depends on the data: whether the retention floor fits into the
 *     budget depends on shapes only.  What the kernels find on the device is reported through
 *     device words the caller reads after synchronising: the status word of the two
 *     tensor-core calls, and the fault record of civic_set_index_check /
 *     civic_validate_indices.  Without that check the validity of index arrays passed to the
 *     compaction calls (in range, one row per output row) is the caller's contract, as they
 *     normally come straight from civic_select / civic_seq_indices.
 *   - A token grid is (t, h, w), token index i = (tt*h + hh)*w + ww (row-major), n = t*h*w.
 */
#ifndef CIVIC_H_
#define CIVIC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    CIVIC_OK = 0,
    CIVIC_ERR_INVALID_ARG = 1,     /* null pointer, negative size, inconsistent shapes, overlap   */
    CIVIC_ERR_K_RANGE = 2,         /* k < 0 or k > n                                              */
    CIVIC_ERR_FLOOR_EXCEEDS_K = 3, /* sum over regions of min(m, |region|) > k                    */
    CIVIC_ERR_ALIGNMENT = 4,       /* row size or pointer not a multiple of 4 bytes               */
    CIVIC_ERR_UNSUPPORTED = 5,     /* segment too large for one thread block's shared memory      */
    CIVIC_ERR_CUDA = 6,            /* a CUDA runtime call failed                                  */
    CIVIC_ERR_WORKSPACE = 7        /* scratch memory missing or smaller than required             */
} civic_status_t;

/* Selection problem of ONE segment (an image or a video); every segment of a call shares it.
 * The retention floor tiles each temporal slice of the grid into region_h x region_w token
 * tiles (edge tiles are smaller when h or w is not a multiple) and keeps at least
 * floor_per_region tokens of every tile (all of a tile that has fewer).  Regions never span t. */
typedef struct {
    int32_t t, h, w;            /* token grid, all >= 1                                           */
    int32_t region_h, region_w; /* tile of the floor in tokens, both >= 1                         */
    int32_t floor_per_region;   /* m >= 0; 0 = plain top-K                                        */
    int32_t k;                  /* tokens kept per segment, 0 <= k <= n                           */
} civic_select_desc_t;

/*
 * civic_select -- which visual tokens survive.
 *
 * Paper: score-rank token dropping (Table 1 caption), selection as a routing overhead
 * (Eq. 3), kept under the "adaptive spatial retention floor" (Sections 1, 4.5; Table 2
 * "Min Keep Ratio").  The paper gives no algorithm for the floor; this call implements:
 *   order    token a beats token b iff score[a] > score[b], or the scores are equal and
 *            a < b.  Scores are compared in IEEE-754 totalOrder (-0 < +0, NaNs at the ends).
 *   reserve  in every region its min(m, |region|) best tokens;
 *   fill     the k - (number reserved) best of the remaining tokens of the segment;
 *   output   the union as ASCENDING segment-local token indices, exactly k per segment.
 *
 * scores    dev  [n_seg, n] fp32, contiguous
 * desc      host
 * keep_idx  dev  [n_seg, k] int32, written
 * One thread block handles one segment with its keys in shared memory:
 * n <= civic_select_max_tokens() or CIVIC_ERR_UNSUPPORTED.  n_seg == 0 or k == 0 enqueue
 * nothing and return CIVIC_OK.
 */
civic_status_t civic_select(const float* scores, int32_t n_seg, const civic_select_desc_t* desc,
                            int32_t* keep_idx, void* stream);

/*
 * civic_select_seq -- civic_select and civic_seq_indices in ONE launch.
 *
 * Paper: as civic_select, followed by the index form of Eq. 13 / Section 3.5 (see
 * civic_seq_indices).  Every sequence is `vis_start` text tokens, the n = t*h*w visual tokens of
 * one segment, then seq_len - vis_start - n text tokens; segment s belongs to sequence s.
 *
 * keep_idx  dev [n_seq, k] int32, written (as by civic_select)
 * seq_idx   dev [n_seq, seq_len - n + k] int32, written (as by civic_seq_indices with n_vis = n)
 * Same limits and errors as the two separate calls; vis_start + n > seq_len is
 * CIVIC_ERR_INVALID_ARG.
 */
civic_status_t civic_select_seq(const float* scores, int32_t n_seq, const civic_select_desc_t* desc,
                                int32_t seq_len, int32_t vis_start, int32_t* keep_idx,
                                int32_t* seq_idx, void* stream);

/*
 * civic_select_large -- civic_select for segments beyond one thread block (long videos).
 *
 * Paper: as civic_select; the paper's stated next step is long-form video (Section 5), where
 * one segment has far more tokens than a thread block can hold.  Same definition and the same
 * output as civic_select for any n up to 2^31 - 1, computed by many thread blocks per segment:
 * in five consecutive launches that communicate through `workspace`, or, with the library's own
 * chunking (chunk_tokens = 0) and where that is the faster of the two (segments up to 16 384
 * tokens, batches of segments up to 65 536), in ONE launch of a cluster of four thread blocks
 * per segment that communicate through distributed shared memory and leave `workspace` alone.
 *
 * workspace        dev, caller-owned scratch of at least civic_select_workspace_bytes(...)
 *                  bytes, 256-byte aligned; contents on entry are irrelevant, contents on return
 *                  are unspecified.  Two calls that may run concurrently need separate workspaces.
 * chunk_tokens     tokens handled by one thread block, at most 16384; 0 = the library default
 *                  (sized from the shapes for about one block per SM, 2048 .. 16384).  One
 *                  "region row" (region_h token rows of w tokens) must fit into a chunk,
 *                  otherwise CIVIC_ERR_UNSUPPORTED.  Pass the same value to
 *                  civic_select_workspace_bytes.
 * CIVIC_ERR_WORKSPACE if workspace is NULL or too small.  The only allocation-free requirement
 * on the caller is this scratch buffer; the call itself allocates nothing.
 */
civic_status_t civic_select_large(const float* scores, int32_t n_seg, const civic_select_desc_t* desc,
                                  int32_t* keep_idx, void* workspace, size_t workspace_bytes,
                                  int32_t chunk_tokens, void* stream);

/*
 * civic_select_large_static -- civic_select_large for callers that cannot allocate device memory.
 *
 * The paper has no counterpart to this call; it exists for the sake of its callers.  Code that
 * runs where cudaMalloc is off limits -- inside a serving engine that handed all device memory
 * to its own pool at start-up, in a plugin that owns no allocator, on a path that must not
 * touch the allocator because a latency budget or a memory cap forbids it -- has nowhere to get
 * the scratch buffer civic_select_large asks for.  This variant computes the same selection
 * with its scratch in a fixed array built into the library, so the caller passes inputs and
 * the output only.  The call allocates nothing, frees nothing and calls no allocating routine.
 *
 * Limits and sharing
 *   - The built-in scratch is civic_select_static_scratch_bytes() = 2 MiB, held by every GPU
 *     that loads the library until the process exits.  A shape whose
 *     civic_select_workspace_bytes(desc, n_seg, chunk_tokens) exceeds it is rejected with
 *     CIVIC_ERR_WORKSPACE and nothing is launched (2 MiB covers, for example, one video of about
 *     two million tokens or eight of 200 000).
 *   - All calls on one GPU share that one array, and it still holds the previous call's
 *     contents: the call clears the part that must start at zero itself.  Calls in ONE stream
 *     run one after the other and are safe; two calls of one process that can overlap on the
 *     GPU (different streams, whichever host threads issue them) race on the scratch and give
 *     wrong results.  Use civic_select_large with separate workspaces there.
 *   - The first call on each device looks up the array's device address (with that device
 *     current, as for every call).  Make that first call before starting any stream capture.
 *
 * Arguments, result and the other errors are those of civic_select_large.
 */
civic_status_t civic_select_large_static(const float* scores, int32_t n_seg, const civic_select_desc_t* desc,
                                         int32_t* keep_idx, int32_t chunk_tokens, void* stream);

/* Size in bytes of the scratch built into the library for civic_select_large_static. */
size_t civic_select_static_scratch_bytes(void);

/*
 * civic_select_ragged -- civic_select for a batch whose segments differ in shape and budget.
 *
 * Paper: as civic_select; instance-adaptive token budgets and mixed image/video batches are the
 * paper's stated next steps (Section 5).  Segment s has its own descriptor descs[s] (grid,
 * tiles, floor, k).  Scores are concatenated: segment s starts at the sum of the earlier
 * segments' n; keep_idx likewise at the sum of the earlier k.
 *
 * scores    dev  [sum n] fp32
 * descs     host [n_seg]
 * keep_idx  dev  [sum k] int32, written: ascending segment-local token indices per segment
 * flat_idx  dev  [sum k] int32 or NULL, written: the same tokens numbered over the concatenated
 *           scores (keep_idx + start of the segment).  With it a ragged batch is compacted by
 *           ONE civic_compact call: n_seg = 1, n = sum n, k = sum k, keep_idx = flat_idx.
 * Every segment must fit one thread block (n <= civic_select_max_tokens()); sum n < 2^31.
 * One launch per 64 segments.
 */
civic_status_t civic_select_ragged(const float* scores, int32_t n_seg, const civic_select_desc_t* descs,
                                   int32_t* keep_idx, int32_t* flat_idx, void* stream);

/*
 * civic_floor_from_ratio -- Table 2's "Min Keep Ratio" as a floor_per_region value.
 *
 * Paper: Section 4.5 / Table 2 vary the retention floor as a ratio (0.0, 0.2, 0.5) of the
 * tokens of a spatial region.  Returns the smallest m with m >= (num / den) * region_h *
 * region_w, in exact integer arithmetic (0/1 -> 0, i.e. plain top-K); -1 on invalid arguments
 * (num > den, den < 1, empty tile).  Host-only helper, nothing is launched.
 */
int32_t civic_floor_from_ratio(int32_t region_h, int32_t region_w, int32_t num, int32_t den);

/* Scratch bytes civic_select_large needs for this shape; 0 if the shape is invalid or unsupported. */
size_t civic_select_workspace_bytes(const civic_select_desc_t* desc, int32_t n_seg, int32_t chunk_tokens);

/* Largest n = t*h*w that civic_select accepts. */
int32_t civic_select_max_tokens(void);

/* Number of tokens the floor reserves per segment (shape-only); -1 on invalid arguments. */
int64_t civic_reserved_count(const civic_select_desc_t* desc);

/*
 * civic_compact -- pack the surviving tokens' hidden rows and 3-D position ids.
 *
 * Paper: Section 3.5 -- the compact visual sequence V_c (Eq. 12) is contiguous, and compact
 * visual positions are inherited from the dense span (copied, not renumbered).
 *   hidden_out[s, j, :] = hidden[s, keep_idx[s, j], :]      rows of row_bytes opaque bytes
 *   pos_out[s, j, :]    = pos_ids[s, keep_idx[s, j], :]     rows of 3 int32
 *
 * hidden      dev [n_seg, n, row_bytes] or NULL (then hidden_out must be NULL)
 * row_bytes   multiple of 4; multiples of 16 with 16-byte aligned buffers take the fast path
 * pos_ids     dev [n_seg, n, 3] int32 or NULL (then pos_out must be NULL)
 * keep_idx    dev [n_seg, k] int32, values in [0, n)
 * Both payloads are moved by ONE launch.
 */
civic_status_t civic_compact(const void* hidden, size_t row_bytes, const int32_t* pos_ids,
                             const int32_t* keep_idx, int32_t n_seg, int32_t n, int32_t k,
                             void* hidden_out, int32_t* pos_out, void* stream);

/*
 * civic_seq_indices -- kept rows of the full multimodal sequence.
 *
 * Paper: Eq. 13 (the compact prefill replaces the dense visual span by the compact one,
 * length L + M_p) and Section 3.5 (text positions are preserved).  The visual span of every
 * sequence is [vis_start, vis_start + n_vis); all positions outside it are text and always
 * kept.   seq_idx[s, :] = ascending( text positions  U  vis_start + keep_idx[s, :] ).
 *
 * keep_idx  dev [n_seq, k] int32 ascending, values in [0, n_vis)
 * seq_idx   dev [n_seq, seq_len - n_vis + k] int32, written
 */
civic_status_t civic_seq_indices(const int32_t* keep_idx, int32_t n_seq, int32_t k, int32_t seq_len,
                                 int32_t vis_start, int32_t n_vis, int32_t* seq_idx, void* stream);

/*
 * civic_compact_kv -- pack every layer's prefill K and V rows of the kept positions.
 *
 * Paper: the KV-cache storage term of Eq. 2 / Eq. 7 and the cache ratio (L+M_p)/(L+T_p) of
 * Eq. 14: the compact cache holds exactly the kept rows, contiguously, in source order.
 *   k_dst[l][s, j, :] = k_src[l][s, seq_idx[s, j], :]   (same for v), l < n_layers
 *
 * k_src, v_src  host arrays of n_layers dev pointers, each [n_seq, seq_len, row_bytes]
 * k_dst, v_dst  host arrays of n_layers dev pointers, each [n_seq, s_out,  row_bytes]
 * row_bytes     bytes of one token's row (kv_heads * head_dim * element size), multiple of 4
 * seq_idx       dev [n_seq, s_out] int32, values in [0, seq_len); shared by all layers
 * The pointer tables are read during the call only (copied into kernel parameters).  All
 * layers and both of K and V are moved by one launch per 80 layers.
 */
civic_status_t civic_compact_kv(const void* const* k_src, const void* const* v_src,
                                void* const* k_dst, void* const* v_dst, int32_t n_layers,
                                int32_t n_seq, int32_t seq_len, int32_t s_out, size_t row_bytes,
                                const int32_t* seq_idx, void* stream);

/*
 * civic_compact_kv_heads -- civic_compact_kv for head-major cache tensors.
 *
 * Paper: as civic_compact_kv (Eq. 2 / Eq. 7 storage term, Eq. 14 cache ratio); only the memory
 * layout differs: every tensor is [n_seq, n_heads, seq_len, head_bytes], so a token's row is
 * n_heads separate pieces of head_bytes (head_dim * element size, e.g. 256).
 *   k_dst[l][s, h, j, :] = k_src[l][s, h, seq_idx[s, j], :]   (same for v)
 *
 * k_src, v_src  host arrays of n_layers dev pointers, each [n_seq, n_heads, seq_len, head_bytes]
 * k_dst, v_dst  host arrays of n_layers dev pointers, each [n_seq, n_heads, s_out,  head_bytes]
 * head_bytes    multiple of 4; short pieces are packed several to a warp so that the moves stay
 *               16-byte vectorised
 * seq_idx       dev [n_seq, s_out] int32, values in [0, seq_len), shared by heads and layers
 */
civic_status_t civic_compact_kv_heads(const void* const* k_src, const void* const* v_src,
                                      void* const* k_dst, void* const* v_dst, int32_t n_layers,
                                      int32_t n_seq, int32_t n_heads, int32_t seq_len, int32_t s_out,
                                      size_t head_bytes, const int32_t* seq_idx, void* stream);

/*
 * civic_compact_kv_paged -- civic_compact_kv writing straight into a paged cache.
 *
 * Paper: as civic_compact_kv; the destination is the serving engine's block-structured cache
 * instead of a dense tensor, so the compact prefill cache never exists in a second copy.
 * Compact position j of sequence s goes to page block_table[s, j / page_size], slot
 * j % page_size:   k_cache[l][page, slot, :] = k_src[l][s, seq_idx[s, j], :]   (same for v)
 *
 * k_src, v_src      host arrays of n_layers dev pointers, each [n_seq, seq_len, row_bytes]
 * k_cache, v_cache  host arrays of n_layers dev pointers, each [n_pages, page_size, row_bytes];
 *                   only the addressed slots are written
 * block_table       dev [n_seq, max_pages_per_seq] int32, page numbers in [0, n_pages); the
 *                   first ceil(s_out / page_size) entries of every row are used.  Distinct
 *                   sequences must own distinct pages (the caller's contract, like index validity)
 * max_pages_per_seq * page_size < s_out is CIVIC_ERR_INVALID_ARG.
 */
civic_status_t civic_compact_kv_paged(const void* const* k_src, const void* const* v_src,
                                      void* const* k_cache, void* const* v_cache, int32_t n_layers,
                                      int32_t n_seq, int32_t seq_len, int32_t s_out, size_t row_bytes,
                                      const int32_t* seq_idx, const int32_t* block_table,
                                      int32_t max_pages_per_seq, int32_t page_size, int32_t n_pages,
                                      void* stream);

/*
 * civic_merge_embeddings -- the compact prefill sequence as data.
 *
 * Paper: Eq. 13, x_c = Merge(E_x, V_c): the text embeddings with the dense visual placeholder
 * span replaced by the compact visual rows (Eq. 12), length L + M_p.  Built in one pass from the
 * DENSE visual rows and the keep indices, without materialising V_c:
 *   merged[s, j, :] = text[s, j, :]                                  j <  vis_start
 *                   = visual[s, keep_idx[s, j - vis_start], :]       vis_start <= j < vis_start + k
 *                   = text[s, j - k + n_vis, :]                      otherwise
 *
 * text      dev [n_seq, seq_len, row_bytes]; rows inside [vis_start, vis_start + n_vis) are
 *           placeholders and are never read
 * visual    dev [n_seq, n_vis, row_bytes]
 * keep_idx  dev [n_seq, k] int32 ascending, values in [0, n_vis)
 * merged    dev [n_seq, seq_len - n_vis + k, row_bytes], written
 */
civic_status_t civic_merge_embeddings(const void* text, const void* visual, size_t row_bytes,
                                      const int32_t* keep_idx, int32_t n_seq, int32_t seq_len,
                                      int32_t vis_start, int32_t n_vis, int32_t k, void* merged,
                                      void* stream);

/*
 * civic_compact_pos_planes -- position ids of the compact sequence, plane-major layout.
 *
 * Paper: Section 3.5 (text positions preserved, compact visual positions inherited), for ids
 * stored as [n_planes, n_seq, seq_len] (planes t, h, w) over the FULL multimodal sequence:
 *   pos_out[c, s, j] = pos[c, s, seq_idx[s, j]]
 *
 * pos      dev [n_planes, n_seq, seq_len] int32
 * seq_idx  dev [n_seq, s_out] int32, values in [0, seq_len)
 * pos_out  dev [n_planes, n_seq, s_out] int32, written
 */
civic_status_t civic_compact_pos_planes(const int32_t* pos, int32_t n_planes, int32_t n_seq,
                                        int32_t seq_len, const int32_t* seq_idx, int32_t s_out,
                                        int32_t* pos_out, void* stream);

/*
 * civic_anchor_aggregate -- compact visual aggregation, the step that produces the compact
 * visual sequence (and a per-token importance score) upstream of the selection.
 *
 * Paper: Eq. 8 (Section 3.3):  K_0 = Norm(LN(X_0)),  Q_A = Norm(LN(A)),
 *        W_A = softmax(Q_A K_0^T / tau) over the dense tokens,  Z_0 = W_A X_0.
 * LN is layer normalisation over the features without learned scale or shift (eps 1e-5), Norm
 * the l2 normalisation of every row (eps 1e-12).  Both contractions run on the tensor cores in
 * bf16 with fp32 accumulation; W_A is rounded to bf16 before the second one, and its rows are
 * normalised by the sum of the rounded values, so they still add up to one.
 *
 * x0             dev  bf16 [n_img, t_e, d_v] dense patch embeddings, 16-byte aligned
 * anchors        dev  fp32 [m_e, d_v], shared by all images
 * tau            aggregation temperature, >= 0.025 (smaller: CIVIC_ERR_UNSUPPORTED)
 * z0             dev  bf16 [n_img, m_e, d_v], written
 * token_mass     dev  fp32 [n_img, t_e] or NULL, written: column sums of W_A, i.e. how much of
 *                the anchors' attention each dense token receives -- usable as the `scores` of
 *                civic_select
 * workspace      dev  scratch of civic_anchor_aggregate_workspace_bytes(...) bytes, 256-byte
 *                aligned (holds Q_A, the token statistics, W_A's unnormalised bf16 form and
 *                partial sums)
 * device_status  dev  int32, written: 0, or a non-zero code if a wait inside a kernel ran into
 *                its time limit (the kernels then stop cleanly and the outputs are invalid).
 *                Read it after synchronising the stream.
 * d_v must be a multiple of 64 (CIVIC_ERR_UNSUPPORTED otherwise); t_e and m_e are arbitrary.
 * Inputs must be finite.  Three launches (four with token_mass); the first one clears the status word.
 */
civic_status_t civic_anchor_aggregate(const void* x0, const float* anchors, int32_t n_img, int32_t t_e,
                                      int32_t m_e, int32_t d_v, float tau, void* z0, float* token_mass,
                                      void* workspace, size_t workspace_bytes, int32_t* device_status,
                                      void* stream);

/* Scratch bytes civic_anchor_aggregate needs; 0 if the shape is invalid or unsupported. */
size_t civic_anchor_aggregate_workspace_bytes(int32_t n_img, int32_t t_e, int32_t m_e, int32_t d_v);

/*
 * civic_kv_compressed_attention -- attention of the compact visual encoder with compressed keys
 * and values.
 *
 * Paper: Eq. 9 (Section 3.4), for already projected Q = H W_Q, K = H W_K, V = H W_V (the three
 * projections are plain GEMMs and are left to the caller's BLAS):
 *     K_c = Rbar^T K,  V_c = Rbar^T V,  Attn_c = softmax(Q K_c^T / sqrt(d)) V_c   per head,
 * R [m_e, s] the KV assignment matrix onto s memory anchors (non-negative, every column with a
 * positive sum), Rbar = R with every column divided by its sum, d = head_dim.  Heads split the
 * feature dimension into n_heads contiguous blocks of head_dim; the softmax runs over the s
 * anchors.  bf16 tensor-core products with fp32 accumulation; K_c and V_c are rounded to bf16
 * on the way, the unnormalised softmax weights are cut to bf16 and divided by the sum of the
 * cut values.
 *
 * q, k, v        dev  bf16 [n_img, m_e, n_heads * head_dim], 16-byte aligned
 * r              dev  fp32 [m_e, s], shared by the images
 * out            dev  bf16 [n_img, m_e, n_heads * head_dim], written
 * workspace      dev  scratch of civic_kv_compressed_attention_workspace_bytes(...) bytes,
 *                256-byte aligned (R in bf16, its column sums, K_c and V_c)
 * device_status  dev  int32, written: 0, or non-zero if a wait inside a kernel hit its time limit
 *                or a kernel found its shared memory misplaced (the kernels then stop cleanly and
 *                `out` is invalid).  Read it after synchronising the stream.
 * head_dim: a multiple of 8 up to 128 (64 and 128 are the fast cases; a width such as 72 -- 1152-wide
 * vision towers with 16 heads -- is handled by storing every head of K_c and V_c with zero
 * columns up to the next multiple of 16).  s: a multiple of 64 up to 512 (Table 2's "Anchors"
 * ablation uses 128 and 512).  CIVIC_ERR_UNSUPPORTED otherwise.  Up to 256 anchors a head's K_c
 * and V_c stay in shared memory while a block walks its query tiles; beyond that one block per SM
 * holds K_c and, for heads wider than 64, streams V_c from L2 for every query tile.
 * Three launches; the first one clears the status word.
 */
civic_status_t civic_kv_compressed_attention(const void* q, const void* k, const void* v, const float* r,
                                             int32_t n_img, int32_t m_e, int32_t n_heads, int32_t head_dim,
                                             int32_t s, void* out, void* workspace, size_t workspace_bytes,
                                             int32_t* device_status, void* stream);

/* Scratch bytes civic_kv_compressed_attention needs; 0 if the shape is invalid or unsupported. */
size_t civic_kv_compressed_attention_workspace_bytes(int32_t n_img, int32_t m_e, int32_t n_heads, int32_t head_dim,
                                                     int32_t s);

/*
 * Constants prepared once.
 *
 * Paper: the anchors A of Eq. 8 and the assignment R of Eq. 9 are learned parameters (Section 3.3,
 * 3.4): at inference they do not change from call to call.  What the two tensor-core calls derive
 * from them alone -- Q_A = Norm(LN(A)) in bf16 with its row sums; R in bf16 with its column sums --
 * can therefore be computed once and handed to the `_prepared` variants, which skip that work
 * (the conversion of R for Eq. 9; the anchor half of the preparation launch for Eq. 8) and give
 * bit-identical results to the plain calls.
 *
 * prepared        dev, caller-owned, 256-byte aligned, at least civic_anchor_prepared_bytes(m_e, d_v)
 *                 / civic_kv_attention_prepared_bytes(m_e, s) bytes (0 = unsupported shape); written
 *                 by the `_prepare` call, only read by the `_prepared` calls, opaque to the caller.
 *                 CIVIC_ERR_WORKSPACE if too small.
 * The `_prepared` calls take the same arguments as civic_anchor_aggregate /
 * civic_kv_compressed_attention with `prepared` in the place of `anchors` / `r`; their workspace is
 * sized by the same *_workspace_bytes functions.  One launch (two for R).
 */
size_t civic_anchor_prepared_bytes(int32_t m_e, int32_t d_v);
civic_status_t civic_anchor_prepare(const float* anchors, int32_t m_e, int32_t d_v, void* prepared,
                                    size_t prepared_bytes, void* stream);
civic_status_t civic_anchor_aggregate_prepared(const void* x0, const void* prepared, int32_t n_img, int32_t t_e,
                                               int32_t m_e, int32_t d_v, float tau, void* z0, float* token_mass,
                                               void* workspace, size_t workspace_bytes, int32_t* device_status,
                                               void* stream);
size_t civic_kv_attention_prepared_bytes(int32_t m_e, int32_t s);
civic_status_t civic_kv_attention_prepare(const float* r, int32_t m_e, int32_t s, void* prepared, size_t prepared_bytes,
                                          void* stream);
civic_status_t civic_kv_compressed_attention_prepared(const void* q, const void* k, const void* v, const void* prepared,
                                                      int32_t n_img, int32_t m_e, int32_t n_heads, int32_t head_dim,
                                                      int32_t s, void* out, void* workspace, size_t workspace_bytes,
                                                      int32_t* device_status, void* stream);

/*
 * Device-side validation of index arrays.
 *
 * Paper: the compact rows are "indexed by compact visual segments" with inherited positions
 * (Section 3.5); the paper has no counterpart to checking those indices, this is the library's
 * own safety net.  The compaction calls (civic_compact, civic_compact_kv, _kv_heads, _kv_paged,
 * civic_merge_embeddings, civic_compact_pos_planes) read `keep_idx` / `seq_idx` / `block_table`
 * on the device, so a wrong value cannot be caught by the host-side validation.  With a fault
 * record set, they run kernels that test every index they use: a row whose source index lies
 * outside [0, seq_len) (outside [0, n_vis) for the merge), or whose page lies outside
 * [0, n_pages), is NEITHER READ NOR WRITTEN, and the fault is recorded.  Nothing traps; all other
 * rows are moved as usual.
 *
 * fault record  dev int32[4] = {code, row, position, value}: code is a civic_index_fault_t, row the
 *               sequence / segment (index row) concerned, position the column of the index array
 *               (the page slot of the block table for CIVIC_INDEX_BAD_PAGE), value the offending
 *               entry.  The first kernel thread to meet a fault claims the record; later faults
 *               leave it alone, so it names ONE offending entry (which one is unspecified when
 *               there are several).  The library never clears it: zero it (cudaMemsetAsync)
 *               before the calls to be checked and read it after synchronising.
 *
 * civic_set_index_check   sets (NULL: clears) the record used by the CALLING THREAD's later
 *               compaction calls; returns CIVIC_ERR_ALIGNMENT for a pointer that is not 4-byte
 *               aligned.  Off by default; when off the calls launch the unchecked kernels and pay
 *               nothing.  The record must stay valid until those calls have completed.
 * civic_validate_indices  checks an index array [n_rows, row_len] on its own: every value in
 *               [0, limit) and, with require_ascending != 0, every row strictly ascending
 *               (CIVIC_INDEX_NOT_ASCENDING names the first position that is not larger than its
 *               predecessor).  One small launch; n_rows * row_len == 0 enqueues nothing.
 */
typedef enum {
    CIVIC_INDEX_OK = 0,
    CIVIC_INDEX_OUT_OF_RANGE = 1,
    CIVIC_INDEX_NOT_ASCENDING = 2,
    CIVIC_INDEX_BAD_PAGE = 3
} civic_index_fault_t;

civic_status_t civic_set_index_check(int32_t* fault_record);

civic_status_t civic_validate_indices(const int32_t* idx, int32_t n_rows, int32_t row_len, int32_t limit,
                                      int32_t require_ascending, int32_t* fault_record, void* stream);

/*
 * civic_selftest_bounded_wait -- shows that a wait inside the tensor-core kernels that never gets
 * its signal ends with a status instead of a hang.
 *
 * Paper: no counterpart.  The kernels of civic_anchor_aggregate and
 * civic_kv_compressed_attention wait on shared-memory barriers through one bounded wait routine
 * (limit about one second of SM cycles); when the limit runs out the thread records a code in the
 * call's device status word and raises a flag that makes the block's other waits return.  This
 * entry runs that same routine in a one-block kernel on a barrier that nothing ever signals, with
 * no copy and no tensor-core operation in flight: one thread waits with `limit_cycles` and times
 * out, a second thread waits with the ordinary limit and must leave through the flag.
 *
 * limit_cycles  1 .. 2^24 SM cycles (a few milliseconds at most)
 * record        dev int32[2], cleared and then written: [0] = 1 (the code a starved operand wait
 *               reports), [1] = 1 if the second waiter left because of the flag
 * One 8-byte memset and one launch; the context stays usable.
 */
civic_status_t civic_selftest_bounded_wait(uint64_t limit_cycles, int32_t* record, void* stream);

/* Static, human-readable name of a status. */
const char* civic_status_string(civic_status_t status);

/* Text of the CUDA error behind the calling thread's last CIVIC_ERR_CUDA ("" if none). */
const char* civic_last_cuda_error(void);

/* Kernels this library enqueued since it was loaded (all threads). */
uint64_t civic_launch_count(void);

/*
 * Kernels are enqueued with CUDA's programmatic-dependent-launch attribute: a kernel may become
 * resident while the previous kernel of the stream drains, and waits for that kernel's
 * completion before its first memory access, so stream-order semantics are unchanged while the
 * gap between the library's own consecutive kernels shrinks.  enable = 0 switches to plain
 * launches (process-wide); returns the previous setting.  Default: enabled.
 */
int32_t civic_set_programmatic_launch(int32_t enable);

#ifdef __cplusplus
}
#endif
#endif /* CIVIC_H_ */
