/*
 * CPU oracle for CIVIC's token selection and compaction  --  TEST INFRASTRUCTURE.
 *
 * A plain, slow, obviously-correct statement of what the hot path computes.  It is
 * used only by the test-suite, the smoke check and the benchmark's CPU-baseline leg;
 * the product (the CUDA library) neither links nor imports it, and it shares no code,
 * header, table or helper with the CUDA sources.
 *
 * What the paper fixes and what it leaves open
 * --------------------------------------------
 * The paper names the operations (score-rank token dropping: Table 1 caption;
 * selection and gather as the routing overheads of Eq. 3; the "adaptive spatial
 * retention floor" / "Min Keep Ratio" of Section 4.5 and Table 2) and fixes the
 * semantics of compaction (Section 3.5: compact rows are contiguous, text positions
 * are preserved, compact visual positions are inherited from the dense span;
 * Eq. 13: the compact sequence has L + M_p rows; Eq. 14: cache ratio
 * (L+M_p)/(L+T_p)).  It prints no algorithm and no worked example for the floor, so
 * agreement of the floor with the authors' unpublished code is "parity unpinned";
 * the definition implemented here is the benchmark definition's:
 *
 *   total order      a beats b  <=>  score[a] > score[b], or equal scores and a < b
 *                    (scores compared as IEEE-754 totalOrder on fp32 values)
 *   reserve          in every spatial region r (a region_h x region_w tile of one
 *                    temporal slice, ragged at the edges) the min(m, |r|) best tokens
 *   fill             the K - |reserved| best of the non-reserved tokens of the segment
 *   output           reserved U fill, as ascending token indices (exactly K of them)
 *   compaction       out[j] = in[index[j]] row by row (bytes, never interpreted)
 *   sequence index   text positions (always kept) and vis_start + kept visual
 *                    indices, ascending
 *   merge            Eq. 13: text rows with the visual span replaced by the kept visual rows
 *   other layouts    plane-major position ids, head-major K/V, paged K/V destinations:
 *                    the same row moves with other address arithmetic
 *   ragged batch     one selection per segment, each with its own grid, floor and budget
 *
 * Everything is done by sorting with the comparator above and by memcpy: no bit
 * tricks, no histograms, no scans.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum {
    ORACLE_OK = 0,
    ORACLE_ERR_ARG = 1,
    ORACLE_ERR_K_RANGE = 2,
    ORACLE_ERR_FLOOR_EXCEEDS_K = 3,
    ORACLE_ERR_INDEX = 4,
    ORACLE_ERR_NOMEM = 5
};

/* ---- ordering of fp32 scores: IEEE-754 totalOrder, written out by cases ---------- */

static uint32_t magnitude_bits(float x)
{
    uint32_t u;
    memcpy(&u, &x, sizeof u);
    return u & 0x7FFFFFFFu;
}

/* -1 if a orders below b, +1 if above, 0 if the two are the same datum.
 * negative NaN < -inf < negative finite < -0 < +0 < positive finite < +inf < positive NaN;
 * NaNs of one sign are ordered by payload magnitude (reversed for the negative ones). */
int oracle_score_cmp(float a, float b)
{
    int a_nan = isnan(a), b_nan = isnan(b);
    int a_neg = signbit(a) != 0, b_neg = signbit(b) != 0;
    if (!a_nan && !b_nan) {
        if (a < b) return -1;
        if (a > b) return 1;
        /* numerically equal: only -0 versus +0 differ */
        if (a_neg && !b_neg) return -1;
        if (!a_neg && b_neg) return 1;
        return 0;
    }
    if (a_nan && !b_nan) return a_neg ? -1 : 1;
    if (!a_nan && b_nan) return b_neg ? 1 : -1;
    /* both NaN */
    if (a_neg != b_neg) return a_neg ? -1 : 1;
    {
        uint32_t ma = magnitude_bits(a), mb = magnitude_bits(b);
        if (ma == mb) return 0;
        if (!a_neg) return ma < mb ? -1 : 1;
        return ma < mb ? 1 : -1;
    }
}

typedef struct {
    float score;
    int32_t index;
} token_t;

/* qsort comparator: best token first.  The order is total (indices are distinct),
 * so the sorted sequence is unique whatever the sort's stability. */
static int best_first(const void* pa, const void* pb)
{
    const token_t* a = (const token_t*)pa;
    const token_t* b = (const token_t*)pb;
    int c = oracle_score_cmp(a->score, b->score);
    if (c > 0) return -1; /* higher score first */
    if (c < 0) return 1;
    if (a->index < b->index) return -1; /* equal scores: lower index first */
    if (a->index > b->index) return 1;
    return 0;
}

static int ascending_i32(const void* pa, const void* pb)
{
    int32_t a = *(const int32_t*)pa, b = *(const int32_t*)pb;
    return (a > b) - (a < b);
}

static int ceil_div(int a, int b) { return (a + b - 1) / b; }

/* Number of tokens the floor reserves: depends on shapes only. */
int64_t oracle_reserved_count(int t, int h, int w, int region_h, int region_w, int m)
{
    int64_t total = 0;
    if (t <= 0 || h <= 0 || w <= 0 || region_h <= 0 || region_w <= 0 || m < 0) return -1;
    for (int tt = 0; tt < t; ++tt)
        for (int h0 = 0; h0 < h; h0 += region_h)
            for (int w0 = 0; w0 < w; w0 += region_w) {
                int hh = (h0 + region_h < h ? h0 + region_h : h) - h0;
                int ww = (w0 + region_w < w ? w0 + region_w : w) - w0;
                int size = hh * ww;
                total += size < m ? size : m;
            }
    return total;
}

/* Selection for ONE segment. scores[n], n = t*h*w, token i = (tt*h + hh)*w + ww.
 * Writes exactly k ascending indices. */
static int select_segment(const float* scores, int t, int h, int w, int region_h, int region_w,
                          int m, int k, int32_t* keep_idx)
{
    int n = t * h * w;
    int n_rh = ceil_div(h, region_h), n_rw = ceil_div(w, region_w);
    unsigned char* reserved = (unsigned char*)calloc((size_t)n, 1);
    token_t* buf = (token_t*)malloc((size_t)n * sizeof(token_t));
    int n_keep = 0, rc = ORACLE_OK;
    if (!reserved || !buf) { free(reserved); free(buf); return ORACLE_ERR_NOMEM; }

    /* reserve: per region, sort its members best-first and take the first min(m, size) */
    for (int tt = 0; tt < t && m > 0; ++tt)
        for (int rh = 0; rh < n_rh; ++rh)
            for (int rw = 0; rw < n_rw; ++rw) {
                int size = 0;
                for (int hh = rh * region_h; hh < (rh + 1) * region_h && hh < h; ++hh)
                    for (int ww = rw * region_w; ww < (rw + 1) * region_w && ww < w; ++ww) {
                        int i = (tt * h + hh) * w + ww;
                        buf[size].score = scores[i];
                        buf[size].index = i;
                        ++size;
                    }
                qsort(buf, (size_t)size, sizeof(token_t), best_first);
                for (int j = 0; j < size && j < m; ++j) {
                    reserved[buf[j].index] = 1;
                    keep_idx[n_keep++] = buf[j].index;
                    if (n_keep > k) { rc = ORACLE_ERR_FLOOR_EXCEEDS_K; goto done; }
                }
            }

    /* fill: sort the non-reserved tokens best-first, take the first k - n_reserved */
    {
        int n_rest = 0, need = k - n_keep;
        for (int i = 0; i < n; ++i)
            if (!reserved[i]) {
                buf[n_rest].score = scores[i];
                buf[n_rest].index = i;
                ++n_rest;
            }
        if (need > n_rest) { rc = ORACLE_ERR_K_RANGE; goto done; }
        qsort(buf, (size_t)n_rest, sizeof(token_t), best_first);
        for (int j = 0; j < need; ++j) keep_idx[n_keep++] = buf[j].index;
    }

    /* output in source order */
    qsort(keep_idx, (size_t)k, sizeof(int32_t), ascending_i32);
done:
    free(reserved);
    free(buf);
    return rc;
}

/* scores [n_seg, n] -> keep_idx [n_seg, k]; every segment has the same grid and budget. */
int oracle_select(const float* scores, int n_seg, int t, int h, int w, int region_h, int region_w,
                  int m, int k, int32_t* keep_idx)
{
    if (!scores || !keep_idx || n_seg < 0 || t <= 0 || h <= 0 || w <= 0 || region_h <= 0 ||
        region_w <= 0 || m < 0)
        return ORACLE_ERR_ARG;
    int64_t n = (int64_t)t * h * w;
    if (n > INT32_MAX) return ORACLE_ERR_ARG;
    if (k < 0 || k > n) return ORACLE_ERR_K_RANGE;
    if (oracle_reserved_count(t, h, w, region_h, region_w, m) > k) return ORACLE_ERR_FLOOR_EXCEEDS_K;
    for (int s = 0; s < n_seg; ++s) {
        int rc = select_segment(scores + (size_t)s * n, t, h, w, region_h, region_w, m, k,
                                keep_idx + (size_t)s * k);
        if (rc != ORACLE_OK) return rc;
    }
    return ORACLE_OK;
}

/* Section 3.5: compact rows are the kept dense rows in source order; positions are
 * inherited (copied), not renumbered.  hidden [n_seg, n, row_bytes] -> [n_seg, k, row_bytes],
 * pos_ids int32 [n_seg, n, 3] -> [n_seg, k, 3].  Either payload may be NULL. */
int oracle_compact(const void* hidden, size_t row_bytes, const int32_t* pos_ids,
                   const int32_t* keep_idx, int n_seg, int n, int k, void* hidden_out,
                   int32_t* pos_out)
{
    if (!keep_idx || n_seg < 0 || n < 0 || k < 0) return ORACLE_ERR_ARG;
    for (int s = 0; s < n_seg; ++s)
        for (int j = 0; j < k; ++j) {
            int32_t i = keep_idx[(size_t)s * k + j];
            if (i < 0 || i >= n) return ORACLE_ERR_INDEX;
            if (hidden && hidden_out)
                memcpy((char*)hidden_out + ((size_t)s * k + j) * row_bytes,
                       (const char*)hidden + ((size_t)s * n + i) * row_bytes, row_bytes);
            if (pos_ids && pos_out)
                memcpy(pos_out + ((size_t)s * k + j) * 3, pos_ids + ((size_t)s * n + i) * 3,
                       3 * sizeof(int32_t));
        }
    return ORACLE_OK;
}

/* Eq. 13 at index level: the compact sequence keeps every text position and the kept
 * visual positions, in source order.  The visual span is [vis_start, vis_start + n_vis).
 * seq_idx [n_seq, seq_len - n_vis + k]. */
int oracle_seq_indices(const int32_t* keep_idx, int n_seq, int k, int seq_len, int vis_start,
                       int n_vis, int32_t* seq_idx)
{
    if (!keep_idx || !seq_idx || n_seq < 0 || k < 0 || k > n_vis || vis_start < 0 ||
        vis_start + n_vis > seq_len)
        return ORACLE_ERR_ARG;
    int s_out = seq_len - n_vis + k;
    for (int s = 0; s < n_seq; ++s) {
        int32_t* out = seq_idx + (size_t)s * s_out;
        int c = 0;
        for (int p = 0; p < seq_len; ++p) {
            int is_text = p < vis_start || p >= vis_start + n_vis;
            int kept = is_text;
            if (!is_text)
                for (int j = 0; j < k; ++j)
                    if (keep_idx[(size_t)s * k + j] == p - vis_start) kept = 1;
            if (kept) {
                if (c >= s_out) return ORACLE_ERR_INDEX;
                out[c++] = p;
            }
        }
        if (c != s_out) return ORACLE_ERR_INDEX;
    }
    return ORACLE_OK;
}

/* Prefill KV cache of the compact sequence: for every layer and for K and V,
 * dst[l][s, j, :] = src[l][s, seq_idx[s, j], :].  src [n_seq, seq_len, row_bytes],
 * dst [n_seq, s_out, row_bytes].  The (layer, K|V, sequence) units are independent; with
 * OpenMP enabled they are spread over threads, each still a plain memcpy loop. */
int oracle_compact_kv(const void* const* k_src, const void* const* v_src, void* const* k_dst,
                      void* const* v_dst, int n_layers, int n_seq, int seq_len, int s_out,
                      size_t row_bytes, const int32_t* seq_idx)
{
    if (!k_src || !v_src || !k_dst || !v_dst || !seq_idx || n_layers < 0 || n_seq < 0 ||
        seq_len < 0 || s_out < 0)
        return ORACLE_ERR_ARG;
    for (int s = 0; s < n_seq; ++s)
        for (int j = 0; j < s_out; ++j) {
            int32_t i = seq_idx[(size_t)s * s_out + j];
            if (i < 0 || i >= seq_len) return ORACLE_ERR_INDEX;
        }
    int n_units = n_layers * 2 * n_seq;
#ifdef _OPENMP
#pragma omp parallel for schedule(static)
#endif
    for (int u = 0; u < n_units; ++u) {
        int l = u / (2 * n_seq), which = (u / n_seq) % 2, s = u % n_seq;
        const char* src = (const char*)(which ? v_src[l] : k_src[l]) + (size_t)s * seq_len * row_bytes;
        char* dst = (char*)(which ? v_dst[l] : k_dst[l]) + (size_t)s * s_out * row_bytes;
        for (int j = 0; j < s_out; ++j)
            memcpy(dst + (size_t)j * row_bytes,
                   src + (size_t)seq_idx[(size_t)s * s_out + j] * row_bytes, row_bytes);
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------------------
 * Steps adjacent to the core path (same semantics, other layouts)
 * ------------------------------------------------------------------------------------ */

/* Eq. 13: the compact prefill sequence is Merge(E_x, V_c) -- the text embeddings with the
 * dense visual placeholder span [vis_start, vis_start + n_vis) replaced by the compact visual
 * rows V_c, where V_c are the kept rows of the dense visual sequence in source order (Eq. 12,
 * Section 3.5).  text [n_seq, seq_len, row_bytes] (rows inside the span are placeholders and
 * are never read), visual [n_seq, n_vis, row_bytes], keep_idx [n_seq, k] ->
 * merged [n_seq, seq_len - n_vis + k, row_bytes]. */
int oracle_merge_embeddings(const void* text, const void* visual, size_t row_bytes,
                            const int32_t* keep_idx, int n_seq, int seq_len, int vis_start,
                            int n_vis, int k, void* merged)
{
    if (!text || !visual || !merged || n_seq < 0 || seq_len < 0 || vis_start < 0 || n_vis < 0 ||
        k < 0 || k > n_vis || vis_start + n_vis > seq_len || (k > 0 && !keep_idx))
        return ORACLE_ERR_ARG;
    int s_out = seq_len - n_vis + k;
    char* v_c = (char*)malloc((size_t)(k > 0 ? k : 1) * row_bytes);
    if (!v_c) return ORACLE_ERR_NOMEM;
    for (int s = 0; s < n_seq; ++s) {
        const char* e_x = (const char*)text + (size_t)s * seq_len * row_bytes;
        const char* v = (const char*)visual + (size_t)s * n_vis * row_bytes;
        char* out = (char*)merged + (size_t)s * s_out * row_bytes;
        /* V_c: the kept visual rows, in order */
        for (int j = 0; j < k; ++j) {
            int32_t i = keep_idx[(size_t)s * k + j];
            if (i < 0 || i >= n_vis) { free(v_c); return ORACLE_ERR_INDEX; }
            memcpy(v_c + (size_t)j * row_bytes, v + (size_t)i * row_bytes, row_bytes);
        }
        /* text before the span | V_c | text behind the span */
        memcpy(out, e_x, (size_t)vis_start * row_bytes);
        memcpy(out + (size_t)vis_start * row_bytes, v_c, (size_t)k * row_bytes);
        memcpy(out + (size_t)(vis_start + k) * row_bytes,
               e_x + (size_t)(vis_start + n_vis) * row_bytes,
               (size_t)(seq_len - vis_start - n_vis) * row_bytes);
    }
    free(v_c);
    return ORACLE_OK;
}

/* Section 3.5 for position ids stored plane-major, pos [n_planes, n_seq, seq_len] (the three
 * planes are t, h, w): text positions are preserved and compact visual positions inherited, so
 * out[c, s, j] = pos[c, s, seq_idx[s, j]].  out [n_planes, n_seq, s_out]. */
int oracle_compact_pos_planes(const int32_t* pos, int n_planes, int n_seq, int seq_len,
                              const int32_t* seq_idx, int s_out, int32_t* out)
{
    if (!pos || !seq_idx || !out || n_planes < 0 || n_seq < 0 || seq_len < 0 || s_out < 0)
        return ORACLE_ERR_ARG;
    for (int c = 0; c < n_planes; ++c)
        for (int s = 0; s < n_seq; ++s)
            for (int j = 0; j < s_out; ++j) {
                int32_t i = seq_idx[(size_t)s * s_out + j];
                if (i < 0 || i >= seq_len) return ORACLE_ERR_INDEX;
                out[((size_t)c * n_seq + s) * s_out + j] = pos[((size_t)c * n_seq + s) * seq_len + i];
            }
    return ORACLE_OK;
}

/* The prefill cache of Eq. 14 with head-major tensors: src[l] is [n_seq, n_heads, seq_len,
 * head_bytes], dst[l] is [n_seq, n_heads, s_out, head_bytes];
 * dst[l][s, h, j, :] = src[l][s, h, seq_idx[s, j], :] for K and for V. */
int oracle_compact_kv_heads(const void* const* k_src, const void* const* v_src, void* const* k_dst,
                            void* const* v_dst, int n_layers, int n_seq, int n_heads, int seq_len,
                            int s_out, size_t head_bytes, const int32_t* seq_idx)
{
    if (!k_src || !v_src || !k_dst || !v_dst || !seq_idx || n_layers < 0 || n_seq < 0 ||
        n_heads < 0 || seq_len < 0 || s_out < 0)
        return ORACLE_ERR_ARG;
    for (int s = 0; s < n_seq; ++s)
        for (int j = 0; j < s_out; ++j) {
            int32_t i = seq_idx[(size_t)s * s_out + j];
            if (i < 0 || i >= seq_len) return ORACLE_ERR_INDEX;
        }
    for (int l = 0; l < n_layers; ++l)
        for (int which = 0; which < 2; ++which)
            for (int s = 0; s < n_seq; ++s)
                for (int h = 0; h < n_heads; ++h) {
                    const char* src = (const char*)(which ? v_src[l] : k_src[l]) +
                                      ((size_t)s * n_heads + h) * seq_len * head_bytes;
                    char* dst = (char*)(which ? v_dst[l] : k_dst[l]) +
                                ((size_t)s * n_heads + h) * s_out * head_bytes;
                    for (int j = 0; j < s_out; ++j)
                        memcpy(dst + (size_t)j * head_bytes,
                               src + (size_t)seq_idx[(size_t)s * s_out + j] * head_bytes, head_bytes);
                }
    return ORACLE_OK;
}

/* The prefill cache of Eq. 14 written into a paged cache.  Every layer's K and V cache is
 * [n_pages, page_size, row_bytes]; sequence s owns the pages block_table[s, 0 .. ], and its
 * compact position j lives in page block_table[s, j / page_size] at slot j % page_size:
 * cache[l][page, slot, :] = src[l][s, seq_idx[s, j], :].  src [n_seq, seq_len, row_bytes].
 * Nothing else in the cache is written. */
int oracle_compact_kv_paged(const void* const* k_src, const void* const* v_src,
                            void* const* k_cache, void* const* v_cache, int n_layers, int n_seq,
                            int seq_len, int s_out, size_t row_bytes, const int32_t* seq_idx,
                            const int32_t* block_table, int max_pages_per_seq, int page_size,
                            int n_pages)
{
    if (!k_src || !v_src || !k_cache || !v_cache || !seq_idx || !block_table || n_layers < 0 ||
        n_seq < 0 || seq_len < 0 || s_out < 0 || page_size <= 0 || max_pages_per_seq < 0 ||
        n_pages < 0)
        return ORACLE_ERR_ARG;
    if ((int64_t)max_pages_per_seq * page_size < s_out) return ORACLE_ERR_ARG;
    for (int l = 0; l < n_layers; ++l)
        for (int which = 0; which < 2; ++which)
            for (int s = 0; s < n_seq; ++s) {
                const char* src = (const char*)(which ? v_src[l] : k_src[l]) +
                                  (size_t)s * seq_len * row_bytes;
                char* cache = (char*)(which ? v_cache[l] : k_cache[l]);
                for (int j = 0; j < s_out; ++j) {
                    int32_t i = seq_idx[(size_t)s * s_out + j];
                    int32_t page = block_table[(size_t)s * max_pages_per_seq + j / page_size];
                    int slot = j % page_size;
                    if (i < 0 || i >= seq_len || page < 0 || page >= n_pages) return ORACLE_ERR_INDEX;
                    memcpy(cache + ((size_t)page * page_size + slot) * row_bytes,
                           src + (size_t)i * row_bytes, row_bytes);
                }
            }
    return ORACLE_OK;
}

/* Table 2's "Min Keep Ratio" as a per-region token count: the smallest m with
 * m >= ratio * region_h * region_w for ratio = num / den (0.0 -> 0, plain top-K). */
int64_t oracle_floor_from_ratio(int region_h, int region_w, int num, int den)
{
    if (region_h <= 0 || region_w <= 0 || num < 0 || den <= 0 || num > den) return -1;
    int64_t size = (int64_t)region_h * region_w, m = 0;
    while (m * den < size * num) ++m;
    return m;
}

/* Ragged batch: segment s has its own grid, floor and budget, desc[s] = {t, h, w, region_h,
 * region_w, m, k}.  Scores are concatenated (segment s starts at the sum of the earlier
 * segments' n), keep_idx likewise (sum of the earlier k); indices are segment-local.  flat_idx
 * (optional) holds the same tokens numbered over the concatenated scores. */
int oracle_select_ragged(const float* scores, int n_seg, const int32_t* desc, int32_t* keep_idx,
                         int32_t* flat_idx)
{
    if (!desc || n_seg < 0) return ORACLE_ERR_ARG;
    int64_t tok0 = 0, out0 = 0;
    for (int s = 0; s < n_seg; ++s) {
        const int32_t* d = desc + (size_t)s * 7;
        int rc = oracle_select(scores + tok0, 1, d[0], d[1], d[2], d[3], d[4], d[5], d[6],
                               keep_idx + out0);
        if (rc != ORACLE_OK) return rc;
        if (flat_idx)
            for (int j = 0; j < d[6]; ++j) flat_idx[out0 + j] = (int32_t)(tok0 + keep_idx[out0 + j]);
        tok0 += (int64_t)d[0] * d[1] * d[2];
        out0 += d[6];
    }
    return ORACLE_OK;
}

/* Threads the K/V loop uses (1 when built without OpenMP). */
int oracle_set_threads(int n_threads)
{
#ifdef _OPENMP
    if (n_threads > 0) omp_set_num_threads(n_threads);
    return omp_get_max_threads();
#else
    (void)n_threads;
    return 1;
#endif
}
