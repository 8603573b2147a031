"""The Eq. 8 oracle against closed forms, invariances and library routines; planted mistakes in a
copy of its source must each trip a pin."""
import importlib.util
import os

import pytest

from oracle import aggregate
from tests import pins_aggregate as pins

SRC = os.path.join(os.path.dirname(aggregate.__file__), "aggregate.py")

MUTANTS = {
    "softmax_over_anchors": ("logits = logits - logits.max(axis=1, keepdims=True)  # softmax over the dense tokens (axis 1)\n"
                             "    e = np.exp(logits)\n    return e / e.sum(axis=1, keepdims=True)",
                             "e = np.exp(logits - logits.max())\n    return e / e.sum(axis=0, keepdims=True)"),
    "temperature_multiplies": ("logits = q_a @ k0.T / float(tau)", "logits = q_a @ k0.T * float(tau)"),
    "anchors_not_layer_normed": ("q_a = l2_normalize(layer_norm(anchors))", "q_a = l2_normalize(np.asarray(anchors, dtype=np.float64))"),
    "tokens_not_l2_normalized": ("k0 = l2_normalize(layer_norm(x0))", "k0 = layer_norm(x0)"),
    "averages_normalised_tokens": ("return w_a @ x0, w_a", "return w_a @ l2_normalize(layer_norm(x0)), w_a"),
    "layer_norm_over_tokens": ("mean = v.mean(axis=-1, keepdims=True)\n    var = ((v - mean) ** 2).mean(axis=-1, keepdims=True)",
                               "mean = v.mean(axis=0, keepdims=True)\n    var = ((v - mean) ** 2).mean(axis=0, keepdims=True)"),
    "unbiased_variance": ("var = ((v - mean) ** 2).mean(axis=-1, keepdims=True)",
                          "var = ((v - mean) ** 2).sum(axis=-1, keepdims=True) / (v.shape[-1] - 1)"),
    "assignment_rows_normalised": ("return r / r.sum(axis=0, keepdims=True)", "return r / r.sum(axis=1, keepdims=True)"),
    "values_not_compressed_with_normalised_r": ("v_c = rbar.T @ v", "v_c = np.asarray(r, dtype=np.float64).T @ v"),
    "attention_scaled_by_full_width": ("logits = q[:, cols] @ k_c[:, cols].T / np.sqrt(d)", "logits = q[:, cols] @ k_c[:, cols].T / np.sqrt(dim)"),
    "attention_softmax_over_queries": ("logits = logits - logits.max(axis=1, keepdims=True)  # softmax over the S memory anchors\n        e = np.exp(logits)\n        out[:, cols] = (e / e.sum(axis=1, keepdims=True)) @ v_c[:, cols]",
                                       "e = np.exp(logits - logits.max())\n        out[:, cols] = (e / e.sum(axis=0, keepdims=True)) @ v_c[:, cols]"),
    "heads_share_all_features": ("cols = slice(h * d, (h + 1) * d)", "cols = slice(0, dim)"),
    "keys_projected_with_value_weights": ("return kv_compressed_attention(h @ w_q, h @ w_k, h @ w_v, r, n_heads)[0]", "return kv_compressed_attention(h @ w_q, h @ w_v, h @ w_v, r, n_heads)[0]"),
    "mass_sums_over_tokens": ("mass.append(w_i.sum(axis=0))", "mass.append(np.full(w_i.shape[1], w_i.sum(axis=1).mean()))"),
}


@pytest.mark.parametrize("pin", pins.ALL_AGGREGATE_PINS + pins.ALL_ATTENTION_PINS, ids=lambda p: p.__name__)
def test_pin(pin):
    pin(aggregate)


@pytest.mark.parametrize("name", sorted(MUTANTS))
def test_mutant_is_caught(tmp_path, name):
    old, new = MUTANTS[name]
    text = open(SRC).read()
    assert text.count(old) == 1, f"mutation site for {name} not found exactly once"
    path = tmp_path / f"{name}.py"
    path.write_text(text.replace(old, new))
    spec = importlib.util.spec_from_file_location(f"mutant_{name}", path)
    mutant = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mutant)
    caught = []
    for pin in pins.ALL_AGGREGATE_PINS + pins.ALL_ATTENTION_PINS:
        try:
            pin(mutant)
        except (AssertionError, ValueError):
            caught.append(pin.__name__)
    assert caught, f"no pin noticed the planted mistake '{name}'"
