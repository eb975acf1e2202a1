"""Plausible mistakes planted in the CPU oracle (a dropped factor, a wrong axis, a swapped operand, a wrong
tie-break ...) must each make at least one of the oracle's pins fail: the pins are meant to be strong enough that the
oracle cannot be wrong in such a way and still pass.  Everything here runs on the CPU; the mistakes live in patched
copies of the oracle's functions for the duration of one check."""
import numpy as np
import pytest

from oracle import d3tom_oracle as orc

import test_oracle_pins as pins

PIN_TESTS = [(name, getattr(pins, name)) for name in sorted(dir(pins)) if name.startswith("test_")]


def _caught_by(monkeypatch, attr, replacement, keywords):
    """Name of the first pin (among those whose name contains one of `keywords`) that fails with the mistake in."""
    monkeypatch.setattr(orc, attr, replacement)
    try:
        for name, fn in PIN_TESTS:
            if not any(k in name for k in keywords):
                continue
            try:
                fn()
            except Exception:                      # an assertion, or the mistake breaking a shape
                return name
        return None
    finally:
        monkeypatch.undo()


def _attention_matrix_no_scale(q, k, scale):
    s = np.asarray(q, np.float64) @ np.asarray(k, np.float64).T
    s = s - s.max(axis=1, keepdims=True)
    p = np.exp(s)
    return p / p.sum(axis=1, keepdims=True)


def _attention_matrix_wrong_axis(q, k, scale):
    s = (np.asarray(q, np.float64) @ np.asarray(k, np.float64).T) * scale
    s = s - s.max(axis=0, keepdims=True)
    p = np.exp(s)
    return p / p.sum(axis=0, keepdims=True)


def _attention_values_from_keys(q, k, v, cu_seqlens, scale):
    return _ORIG["attention"](q, k, k, cu_seqlens, scale)


def _key_mass_all_rows(q, k, cu_seqlens, decider_pos, cu_deciders, scale):
    every = [np.arange(int(cu_seqlens[b + 1] - cu_seqlens[b])) for b in range(len(cu_seqlens) - 1)]
    cu = np.concatenate([[0], np.cumsum([len(e) for e in every])])
    return _ORIG["key_mass"](q, k, cu_seqlens, np.concatenate(every), cu, scale)


def _importance_last_entries(q, k, cu_seqlens, n_visual, decider_pos, cu_deciders, scale):
    c = orc.key_mass(q, k, cu_seqlens, decider_pos, cu_deciders, scale)
    return [c[b][len(c[b]) - int(n_visual[b]):] for b in range(len(c))]


def _select_ties_to_higher_index(scores, k):
    scores = np.asarray(scores)
    order = np.argsort(-scores.astype(np.float64)[::-1], kind="stable")
    order = len(scores) - 1 - order
    return np.sort(order[:k]).astype(np.int32)


def _select_rank_order(scores, k):
    scores = np.asarray(scores)
    return np.argsort(-scores.astype(np.float64), kind="stable")[:k].astype(np.int32)


def _cosine_is_dot_product(h_vis, kept_idx):
    h = np.asarray(h_vis, np.float64)
    kept_idx = np.asarray(kept_idx, dtype=np.int64)
    mask = np.zeros(h.shape[0], dtype=bool)
    mask[kept_idx] = True
    pruned = np.nonzero(~mask)[0]
    return h[pruned] @ h[kept_idx].T, pruned


def _argmax_last(sim):
    sim = np.asarray(sim)
    if sim.shape[0] == 0:
        return np.zeros(0, dtype=np.int64)
    return sim.shape[1] - 1 - np.argmax(sim[:, ::-1], axis=1)


def _aggregate_mean_by_members_only(h_vis, kept_idx, assignment, mode=orc.SUM):
    out, count = _ORIG["aggregate"](h_vis, kept_idx, assignment, orc.SUM)
    if mode == orc.MEAN:
        out = out / np.maximum(count, 1)[:, None]
    return out, count


def _compact_prompt_before_visual(hidden_req, n_visual, kept_idx, merged_rows):
    out, src = _ORIG["compact"](hidden_req, n_visual, kept_idx, merged_rows)
    k = len(kept_idx)
    return np.concatenate([out[k:], out[:k]]), np.concatenate([src[k:], src[:k]])


def _proj_k_and_v_swapped(x, w_qkv, H, dtype="bf16"):
    q, k, v = _ORIG["proj_qkv"](x, w_qkv, H, dtype)
    return q, v, k


def _schedule_high_to_low(s, T, alpha_min, alpha_max, reversed_=False):
    return _ORIG["schedule_alpha"](s, T, alpha_min, alpha_max, not reversed_)


def _keep_count_rounds(n_visual, keep_ratio):
    if n_visual <= 0:
        return 0
    return max(1, min(int(n_visual), int(round(keep_ratio * n_visual))))


def _round_bf16_truncates(x):
    x = np.asarray(x, dtype=np.float64)
    m, e = np.frexp(x)
    return np.ldexp(np.trunc(m * 256.0) / 256.0, e)


def _silu_is_sigmoid(g):
    g = np.asarray(g, np.float64)
    return 1.0 / (1.0 + np.exp(-g))


def _ffn_gate_up_swapped(x, w_gate_up, w_down, residual=None, dtype="bf16"):
    w = np.asarray(w_gate_up, np.float64)
    m = w.shape[0] // 2
    return _ORIG["ffn"](x, np.concatenate([w[m:], w[:m]]), w_down, residual, dtype)


def _linear_forgets_the_residual(x, w, residual=None, dtype="bf16"):
    return _ORIG["linear"](x, w, None, dtype)


def _merged_length_off(N, n_visual, k):
    return N - k


def _attention_heads_reversed(q, k, v, cu_seqlens, scale):
    out = _ORIG["attention"](q, k, v, cu_seqlens, scale)
    H = np.asarray(q).shape[1]
    dh = out.shape[1] // H
    return out.reshape(out.shape[0], H, dh)[:, ::-1].reshape(out.shape)


def _key_mass_averages_heads(q, k, cu_seqlens, decider_pos, cu_deciders, scale):
    H = np.asarray(q).shape[1]
    return [c / H for c in _ORIG["key_mass"](q, k, cu_seqlens, decider_pos, cu_deciders, scale)]


def _merge_kv_routes_on_values(k_cache, v_cache, cu_seqlens, n_visual, kept_idx_list, mode=orc.SUM, dtype="bf16",
                               assignment_list=None):
    res = _ORIG["merge_kv"](v_cache, k_cache, cu_seqlens, n_visual, kept_idx_list, mode, dtype, assignment_list)
    res["k_out"], res["v_out"] = res["v_out"], res["k_out"]
    return res


def _merge_rounds_before_it_adds(hidden, cu_seqlens, n_visual, kept_idx_list, mode=orc.SUM, dtype="bf16", assignment_list=None):
    coarse = np.round(np.asarray(hidden, np.float64) * 4.0) / 4.0          # a visibly coarser storage type
    return _ORIG["merge"](coarse, cu_seqlens, n_visual, kept_idx_list, mode, dtype, assignment_list)


_ORIG = {n: getattr(orc, n) for n in ("merge_kv", "merge","attention", "key_mass", "aggregate", "compact", "proj_qkv", "schedule_alpha", "ffn", "linear")}

MISTAKES = [
    ("attention_matrix", _attention_matrix_no_scale, ["attention"]),
    ("attention_matrix", _attention_matrix_wrong_axis, ["attention"]),
    ("attention", _attention_values_from_keys, ["attention"]),
    ("key_mass", _key_mass_all_rows, ["importance"]),
    ("importance", _importance_last_entries, ["importance"]),
    ("select", _select_ties_to_higher_index, ["select"]),
    ("select", _select_rank_order, ["select", "merge"]),
    ("cosine_matrix", _cosine_is_dot_product, ["assign"]),
    ("argmax_first", _argmax_last, ["assign"]),
    ("aggregate", _aggregate_mean_by_members_only, ["aggregate", "merge"]),
    ("compact", _compact_prompt_before_visual, ["merge"]),
    ("proj_qkv", _proj_k_and_v_swapped, ["proj_qkv", "post_layer"]),
    ("schedule_alpha", _schedule_high_to_low, ["schedule"]),
    ("keep_count", _keep_count_rounds, ["keep_count"]),
    ("round_bf16", _round_bf16_truncates, ["round_bf16"]),
    ("silu", _silu_is_sigmoid, ["silu", "ffn"]),
    ("ffn", _ffn_gate_up_swapped, ["ffn"]),
    ("linear", _linear_forgets_the_residual, ["linear"]),
    ("merged_length", _merged_length_off, ["merge"]),
    ("attention", _attention_heads_reversed, ["attention"]),
    ("key_mass", _key_mass_averages_heads, ["importance"]),
    ("merge_kv", _merge_kv_routes_on_values, ["merge_kv"]),
    ("merge", _merge_rounds_before_it_adds, ["merge"]),
]


@pytest.mark.parametrize("attr,replacement,keywords", MISTAKES, ids=[m[1].__name__.lstrip("_") for m in MISTAKES])
def test_a_planted_mistake_fails_a_pin(monkeypatch, attr, replacement, keywords):
    caught = _caught_by(monkeypatch, attr, replacement, keywords)
    assert caught is not None, "no pin notices %s" % replacement.__name__


def test_the_unpatched_oracle_passes_the_same_pins():
    for name, fn in PIN_TESTS:
        fn()
