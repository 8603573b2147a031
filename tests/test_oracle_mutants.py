"""Each planted mistake in a COPY of the oracle's source must trip at least one pin.

The copy is made by exact text replacement (the test fails if the text to replace is not
found), built in a temporary directory and loaded beside the real oracle.  This shows the
pins are sharp enough to notice a flipped tie-break, a transposed grid, a fill that ignores
the reservation, and the like.
"""
import ctypes
import os
import subprocess

import pytest

import oracle
from tests import pins

SRC = os.path.join(os.path.dirname(oracle.__file__), "civic_oracle.c")

MUTANTS = {
    "tie_prefers_higher_index": (
        "if (a->index < b->index) return -1; /* equal scores: lower index first */",
        "if (a->index < b->index) return 1;"),
    "lower_score_first": (
        "if (c > 0) return -1; /* higher score first */\n    if (c < 0) return 1;",
        "if (c > 0) return 1;\n    if (c < 0) return -1;"),
    "fill_ignores_reservation": (
        "if (!reserved[i]) {\n                buf[n_rest].score",
        "if (1) {\n                buf[n_rest].score"),
    "grid_transposed": (
        "int i = (tt * h + hh) * w + ww;",
        "int i = (tt * w + ww) * h + hh;"),
    "regions_span_time": (
        "int i = (tt * h + hh) * w + ww;",
        "int i = (0 * h + hh) * w + ww;"),
    "reserve_only_one": (
        "for (int j = 0; j < size && j < m; ++j) {",
        "for (int j = 0; j < size && j < 1; ++j) {"),
    "region_height_used_for_width": (
        "for (int ww = rw * region_w; ww < (rw + 1) * region_w && ww < w; ++ww) {",
        "for (int ww = rw * region_h; ww < (rw + 1) * region_h && ww < w; ++ww) {"),
    "output_not_sorted": (
        "qsort(keep_idx, (size_t)k, sizeof(int32_t), ascending_i32);",
        ";"),
    "zero_signs_ignored": (
        "if (a_neg && !b_neg) return -1;\n        if (!a_neg && b_neg) return 1;\n        return 0;",
        "return 0;"),
    "compact_wrong_segment_stride": (
        "(const char*)hidden + ((size_t)s * n + i) * row_bytes, row_bytes);",
        "(const char*)hidden + ((size_t)s * k + i) * row_bytes, row_bytes);"),
    "pos_renumbered_not_inherited": (
        "memcpy(pos_out + ((size_t)s * k + j) * 3, pos_ids + ((size_t)s * n + i) * 3,",
        "memcpy(pos_out + ((size_t)s * k + j) * 3, pos_ids + ((size_t)s * n + j) * 3,"),
    "seq_index_forgets_offset": (
        "if (keep_idx[(size_t)s * k + j] == p - vis_start) kept = 1;",
        "if (keep_idx[(size_t)s * k + j] == p) kept = 1;"),
    "kv_v_reads_k": (
        "const char* src = (const char*)(which ? v_src[l] : k_src[l]) + (size_t)s * seq_len * row_bytes;",
        "const char* src = (const char*)(which ? k_src[l] : k_src[l]) + (size_t)s * seq_len * row_bytes;"),
    "kv_wrong_sequence_index_row": (
        "src + (size_t)seq_idx[(size_t)s * s_out + j] * row_bytes, row_bytes);",
        "src + (size_t)seq_idx[j] * row_bytes, row_bytes);"),
    "merge_tail_text_from_wrong_offset": (
        "e_x + (size_t)(vis_start + n_vis) * row_bytes,",
        "e_x + (size_t)(vis_start + k) * row_bytes,"),
    "merge_visual_rows_not_gathered": (
        "memcpy(v_c + (size_t)j * row_bytes, v + (size_t)i * row_bytes, row_bytes);",
        "memcpy(v_c + (size_t)j * row_bytes, v + (size_t)j * row_bytes, row_bytes);"),
    "pos_planes_wrong_plane_stride": (
        "out[((size_t)c * n_seq + s) * s_out + j] = pos[((size_t)c * n_seq + s) * seq_len + i];",
        "out[((size_t)c * n_seq + s) * s_out + j] = pos[((size_t)s * n_seq + c) * seq_len + i];"),
    "kv_heads_source_uses_compact_stride": (
        "((size_t)s * n_heads + h) * seq_len * head_bytes;",
        "((size_t)s * n_heads + h) * s_out * head_bytes;"),
    "paged_slot_and_page_swapped": (
        "int slot = j % page_size;",
        "int slot = (j / page_size) % page_size;"),
    "paged_table_row_stride": (
        "block_table[(size_t)s * max_pages_per_seq + j / page_size];",
        "block_table[(size_t)s * (max_pages_per_seq - 1) + j / page_size];"),
    "ratio_floor_rounds_down": (
        "while (m * den < size * num) ++m;",
        "while ((m + 1) * den <= size * num) ++m;"),
    "ragged_flat_index_forgets_offset": (
        "flat_idx[out0 + j] = (int32_t)(tok0 + keep_idx[out0 + j]);",
        "flat_idx[out0 + j] = (int32_t)(keep_idx[out0 + j]);"),
    "ragged_scores_not_advanced": (
        "tok0 += (int64_t)d[0] * d[1] * d[2];",
        "tok0 += (int64_t)d[1] * d[2];"),
}


def _build_mutant(tmp_path, name):
    old, new = MUTANTS[name]
    text = open(SRC).read()
    assert text.count(old) == 1, f"mutation site for {name} not found exactly once"
    src = tmp_path / f"{name}.c"
    src.write_text(text.replace(old, new))
    out = tmp_path / f"lib{name}.so"
    subprocess.run(["gcc", "-std=gnu11", "-O2", "-fPIC", "-shared", "-fopenmp", "-o", str(out),
                    str(src), "-lm"], check=True)
    return oracle.Oracle(oracle._bind(str(out)))


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_mutant_is_caught(tmp_path, name):
    mutant = _build_mutant(tmp_path, name)
    caught = []
    for pin in pins.ALL_SELECT_PINS + pins.ALL_COMPACT_PINS + pins.ALL_ADJACENT_PINS:
        try:
            pin(mutant)
        except (AssertionError, oracle.OracleError):
            caught.append(pin.__name__)
    assert caught, f"no pin noticed the planted mistake '{name}'"
