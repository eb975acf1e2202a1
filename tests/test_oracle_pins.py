"""Pins of the CPU oracle against what the paper and the mathematics fix:
closed forms, brute force in pure Python on tiny inputs, invariants, special
cases that reduce to library routines, and the paper's printed FLOP totals.
None of these tests touches the CUDA path."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import d3tom_oracle as orc
from oracle import flops_model as fm

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rng(seed):
    return np.random.default_rng(seed)


# ------------------------------------------------------------------ rounding
def test_round_bf16_matches_torch_conversion():
    r = rng(0)
    x = np.concatenate([r.standard_normal(20000) * 10.0 ** r.integers(-6, 6, 20000),
                        np.array([0.0, 1.0, -1.0, 1.00390625, 1.01171875, 3.0e-5, 255.5, 256.5])])
    x32 = x.astype(np.float32)   # torch rounds fp32 -> bf16 with ties-to-even
    want = torch.from_numpy(x32).to(torch.bfloat16).to(torch.float64).numpy()
    got = orc.round_bf16(x32.astype(np.float64))
    assert np.array_equal(want, got)


def test_round_bf16_ties_to_even():
    # 1 + 2^-8 lies half-way between 1 and 1 + 2^-7 -> rounds to even mantissa (1.0)
    assert orc.round_bf16(1.0 + 2.0 ** -8) == 1.0
    assert orc.round_bf16(1.0 + 3 * 2.0 ** -8) == 1.0 + 2 * 2.0 ** -7


# ------------------------------------------------------------------ attention
def brute_attention_row(q, K, V, scale):
    logits = [sum(q[c] * K[j][c] for c in range(len(q))) * scale for j in range(len(K))]
    mx = max(logits)
    w = [math.exp(l - mx) for l in logits]
    z = sum(w)
    return [sum(w[j] / z * V[j][c] for j in range(len(K))) for c in range(len(V[0]))], [x / z for x in w]


def test_attention_equals_pure_python_brute_force():
    r = rng(1)
    n, H, dh = 7, 2, 4
    q, k, v = (r.standard_normal((n, H, dh)) for _ in range(3))
    out = orc.attention(q, k, v, [0, n], 0.5)
    for h in range(H):
        for i in range(n):
            o, _ = brute_attention_row(q[i, h].tolist(), k[:, h].tolist(), v[:, h].tolist(), 0.5)
            assert np.allclose(out[i, h * dh:(h + 1) * dh], o, rtol=1e-12, atol=1e-14)


def test_attention_two_key_closed_form():
    # one query, two keys: weights are the logistic function of the logit gap
    q = np.array([[[2.0, 0.0]]])
    k = np.array([[[1.0, 0.0]], [[-1.0, 0.0]]])
    v = np.array([[[1.0, 0.0]], [[0.0, 1.0]]])
    A = orc.attention_matrix(q[:, 0], k[:, 0], 0.25)      # logits +0.5, -0.5
    w0 = 1.0 / (1.0 + math.exp(-1.0))
    assert np.allclose(A, [[w0, 1 - w0]], atol=1e-15)
    # request of 2 tokens where both queries equal q
    out = orc.attention(np.repeat(q, 2, 0), k, v, [0, 2], 0.25)
    assert np.allclose(out, [[w0, 1 - w0], [w0, 1 - w0]], atol=1e-15)


def test_attention_rows_sum_to_one_and_uniform_keys_give_mean_of_values():
    r = rng(2)
    n, dh = 33, 8
    q = r.standard_normal((n, dh))
    A = orc.attention_matrix(q, r.standard_normal((n, dh)), 0.3)
    assert np.allclose(A.sum(axis=1), 1.0, atol=1e-14)
    k_same = np.tile(r.standard_normal((1, 1, dh)), (n, 1, 1))
    v = r.standard_normal((n, 1, dh))
    out = orc.attention(q[:, None], k_same, v, [0, n], 0.3)
    assert np.allclose(out, np.tile(v[:, 0].mean(axis=0), (n, 1)), atol=1e-13)


def test_attention_is_bidirectional_and_per_request():
    # permuting the keys together with the values changes nothing (no causal
    # mask), and a second request in the pack does not leak into the first
    r = rng(3)
    n, H, dh = 12, 2, 4
    q, k, v = (r.standard_normal((n, H, dh)) for _ in range(3))
    base = orc.attention(q, k, v, [0, n], 0.4)
    perm = r.permutation(n)
    assert np.allclose(orc.attention(q, k[perm], v[perm], [0, n], 0.4), base, atol=1e-13)
    q2, k2, v2 = (np.concatenate([x, r.standard_normal((5, H, dh))]) for x in (q, k, v))
    packed = orc.attention(q2, k2, v2, [0, n, n + 5], 0.4)
    assert np.allclose(packed[:n], base, atol=1e-13)
    # transposing the roles of q and k must change the result (catches q/k swap)
    assert not np.allclose(orc.attention(k, q, v, [0, n], 0.4), base)
    # heads are concatenated head-major
    one = orc.attention(q[:, 1:2], k[:, 1:2], v[:, 1:2], [0, n], 0.4)
    assert np.allclose(base[:, dh:], one, atol=1e-13)


def test_attention_rows_helper_equals_full():
    r = rng(4)
    n, H, dh = 20, 3, 4
    q, k, v = (r.standard_normal((n + 6, H, dh)) for _ in range(3))
    cu = [0, 6, n + 6]
    full = orc.attention(q, k, v, cu, 0.5)
    rows = [0, 7, 19]
    got = orc.attention_rows(q, k, v, cu, 0.5, 1, rows, 2)
    assert np.allclose(got, full[6 + np.array(rows), 2 * dh:3 * dh], atol=1e-13)


# ------------------------------------------------------------------ importance
def test_importance_is_column_sum_of_decider_rows_brute_force():
    r = rng(5)
    V, P, O, H, dh = 6, 2, 3, 2, 4
    n = V + P + O
    q, k = r.standard_normal((n, H, dh)), r.standard_normal((n, H, dh))
    dec = [V + P + 0, V + P + 2]
    want = [0.0] * n
    for h in range(H):
        for i in dec:
            _, w = brute_attention_row(q[i, h].tolist(), k[:, h].tolist(), [[0.0]] * n, 0.7)
            for j in range(n):
                want[j] += w[j]
    c = orc.key_mass(q, k, [0, n], np.array(dec), [0, 2], 0.7)[0]
    assert np.allclose(c, want, atol=1e-13)
    S = orc.importance(q, k, [0, n], [V], np.array(dec), [0, 2], 0.7)[0]
    assert S.shape == (V,) and np.allclose(S, want[:V], atol=1e-13)


def test_importance_total_mass_is_deciders_times_heads():
    r = rng(6)
    H, dh = 3, 8
    lens, vis = [19, 11], [10, 5]
    n = sum(lens)
    q, k = r.standard_normal((n, H, dh)), r.standard_normal((n, H, dh))
    dec = np.array([15, 17, 18, 6, 9])     # 3 deciders in request 0, 2 in request 1
    cu_d = [0, 3, 5]
    c = orc.key_mass(q, k, [0, 19, 30], dec, cu_d, 0.35)
    assert abs(c[0].sum() - 3 * H) < 1e-12 and abs(c[1].sum() - 2 * H) < 1e-12
    S = orc.importance(q, k, [0, 19, 30], vis, dec, cu_d, 0.35)
    assert S[0].sum() <= 3 * H and S[1].sum() <= 2 * H and (S[0] > 0).all()


def test_importance_empty_decider_set_is_zero():
    r = rng(7)
    q, k = r.standard_normal((9, 1, 4)), r.standard_normal((9, 1, 4))
    S = orc.importance(q, k, [0, 9], [5], np.zeros(0, dtype=np.int32), [0, 0], 1.0)[0]
    assert np.array_equal(S, np.zeros(5))


def test_importance_uses_only_decider_rows():
    # changing a non-decider query must not change S; changing a decider query must
    r = rng(8)
    q, k = r.standard_normal((10, 2, 4)), r.standard_normal((10, 2, 4))
    args = ([0, 10], [6], np.array([8]), [0, 1], 0.5)
    S0 = orc.importance(q, k, *args)[0]
    q1 = q.copy(); q1[9] += 1.0
    assert np.array_equal(orc.importance(q1, k, *args)[0], S0)
    q2 = q.copy(); q2[8] += 1.0
    assert not np.allclose(orc.importance(q2, k, *args)[0], S0)


# ------------------------------------------------------------------ keep count / select
def test_keep_count_values():
    assert orc.keep_count(1024, 0.10) == 102        # 102.4 -> 102 ranks satisfy Rank <= 102.4
    assert orc.keep_count(1000, 1 - 0.9) == 100     # 99.99999999999997 in binary
    assert orc.keep_count(256, 0.25) == 64
    assert orc.keep_count(4096, 0.25) == 1024
    # the number of integer ranks 1..|V| that satisfy Rank <= x is floor(x), not the nearest integer
    assert orc.keep_count(1026, 0.10) == 102        # 102.6
    assert orc.keep_count(15, 0.5) == 7             # 7.5
    assert orc.keep_count(7, 0.5) == 3              # 3.5
    assert orc.keep_count(2048, 0.4999) == 1023     # 1023.8
    assert orc.keep_count(10, 0.0) == 1             # clamp below
    assert orc.keep_count(10, 1.0) == 10 and orc.keep_count(10, 1.5) == 10


def test_select_equals_full_sort_with_index_tiebreak():
    r = rng(9)
    for V, k in [(1, 1), (17, 5), (64, 64), (100, 1), (257, 100)]:
        S = r.integers(0, 6, V).astype(np.float32) / 4      # many duplicates
        want = sorted(sorted(range(V), key=lambda j: (-float(S[j]), j))[:k])
        assert orc.select(S, k).tolist() == want
    S = np.full(33, 0.5, dtype=np.float32)
    assert orc.select(S, 7).tolist() == list(range(7))        # all equal -> lowest indices
    S = r.random(50).astype(np.float32)
    assert orc.select(S, 50).tolist() == list(range(50))      # r = 1 keeps everything
    got = orc.select(S, 10)
    assert len(got) == 10 and np.all(np.diff(got) > 0)
    assert S[got].min() >= np.delete(S, got).max()


# ------------------------------------------------------------------ assignment
def brute_assign(h, kept):
    V = len(h)
    out = [-1] * V
    for s, kk in enumerate(kept):
        out[kk] = s
    for m in range(V):
        if m in kept:
            continue
        best, best_s = None, -1
        for s, kk in enumerate(kept):
            dot = sum(a * b for a, b in zip(h[m], h[kk]))
            nm = math.sqrt(sum(a * a for a in h[m])); nk = math.sqrt(sum(a * a for a in h[kk]))
            c = dot / (nm * nk) if nm > 0 and nk > 0 else 0.0
            if best is None or c > best:
                best, best_s = c, s
        out[m] = best_s
    return out


def test_assign_equals_brute_force_cosine_argmax():
    r = rng(10)
    V, D = 23, 6
    h = r.standard_normal((V, D))
    kept = sorted(r.choice(V, 7, replace=False).tolist())
    assert orc.assign(h, kept).tolist() == brute_assign(h.tolist(), kept)


def test_assign_cosine_not_dot_product_and_scale_invariance():
    # kept 0 is long but at 45 degrees, kept 1 is short and collinear: cosine picks 1
    h = np.array([[10.0, 10.0], [0.1, 0.0], [1.0, 0.0]])
    assert orc.assign(h, [0, 1]).tolist() == [0, 1, 1]
    r = rng(11)
    h = r.standard_normal((30, 5))
    kept = [1, 4, 9, 20]
    a = orc.assign(h, kept)
    h2 = h * r.uniform(0.1, 10.0, (30, 1))
    assert np.array_equal(orc.assign(h2, kept), a)


def test_assign_duplicate_of_kept_row_goes_to_it_ties_to_lowest_and_zero_rows():
    r = rng(12)
    h = r.standard_normal((12, 4))
    kept = [2, 5, 7]
    h[9] = 3.0 * h[5]                       # cos = 1 with kept 5
    assert orc.assign(h, kept)[9] == 1
    h[7] = h[2]                             # two identical kept rows: tie -> lowest position
    h[10] = h[2]
    assert orc.assign(h, kept)[10] == 0
    h[11] = 0.0                             # zero-norm pruned row: all cosines 0 -> first kept
    assert orc.assign(h, kept)[11] == 0
    a = orc.assign(h, kept)
    assert all(0 <= s < 3 for s in a) and [a[i] for i in kept] == [0, 1, 2]


def test_assign_teacher_forced_similarity_matrix():
    h = np.zeros((5, 2))
    sim = np.array([[0.1, 0.9], [0.5, 0.5], [0.7, 0.2]], dtype=np.float32)   # pruned rows 0, 2, 4
    assert orc.assign(h, [1, 3], sim=sim).tolist() == [1, 0, 0, 1, 0]


# ------------------------------------------------------------------ aggregation / compaction
def test_aggregate_sum_is_kept_plus_onehot_transpose_times_merged():
    r = rng(13)
    V, D, k = 40, 7, 9
    h = r.standard_normal((V, D))
    kept = np.sort(r.choice(V, k, replace=False))
    a = orc.assign(h, kept)
    pruned = np.setdiff1d(np.arange(V), kept)
    M = np.zeros((len(pruned), k))
    M[np.arange(len(pruned)), a[pruned]] = 1.0
    out, cnt = orc.aggregate(h, kept, a, orc.SUM)
    assert np.allclose(out, h[kept] + M.T @ h[pruned], atol=1e-13)
    assert np.array_equal(cnt, M.sum(axis=0).astype(np.int32))
    # mass conservation of the paper's sum: column sums over visual rows are unchanged
    assert np.allclose(out.sum(axis=0), h.sum(axis=0), atol=1e-12)
    # mean: weights 1/(1+c) sum to one per kept token; sum of (1+c) is |V|
    mean, cnt2 = orc.aggregate(h, kept, a, orc.MEAN)
    assert np.allclose(mean * (1 + cnt2)[:, None], out, atol=1e-13)
    assert int((1 + cnt2).sum()) == V
    const = np.ones((V, D)) * 2.5
    mean_c, _ = orc.aggregate(const, kept, a, orc.MEAN)
    assert np.allclose(mean_c, 2.5)


def test_merge_lengths_sources_and_untouched_rows():
    r = rng(14)
    H = 1
    lens, vis = [15, 9], [10, 4]
    hidden = orc.round_bf16(r.standard_normal((24, 6)))
    kept = [np.array([0, 3, 4]), np.array([1, 2])]
    res = orc.merge(hidden, [0, 15, 24], vis, kept, orc.SUM, "bf16")
    assert res["cu_seqlens_out"].tolist() == [0, 15 - 10 + 3, 8 + 9 - 4 + 2]
    assert orc.merged_length(15, 10, 3) == 8
    src = res["src_of_dst"]
    assert src.tolist() == [0, 3, 4, 10, 11, 12, 13, 14, 16, 17, 19, 20, 21, 22, 23]
    # prompt and response rows are bit-identical copies
    assert np.array_equal(res["hidden_out"][3:8], hidden[10:15])
    assert np.array_equal(res["hidden_out"][10:], hidden[19:24])
    assert len(res["assign"]) == 14 and len(res["member_count"]) == 5
    assert res["member_count"][:3].sum() == 7 and res["member_count"][3:].sum() == 2
    # merged rows are representable in bf16 (rounded once)
    assert np.array_equal(orc.round_bf16(res["hidden_out"]), res["hidden_out"])


def test_merge_keep_ratio_one_is_identity():
    r = rng(15)
    hidden = orc.round_bf16(r.standard_normal((12, 5)))
    for mode in (orc.SUM, orc.MEAN):
        res = orc.merge(hidden, [0, 12], [8], [np.arange(8)], mode, "bf16")
        assert np.array_equal(res["hidden_out"], hidden)
        assert res["src_of_dst"].tolist() == list(range(12))
        assert res["member_count"].tolist() == [0] * 8


def test_merge_uses_pre_merge_states_for_every_cosine():
    # sequential in-place updating would route token 2 differently: after
    # adding token 1 into kept 0, kept 0 points along token 2.
    h = np.array([[1.0, 0.0], [0.0, 5.0], [0.3, 1.0], [0.5, 0.6]])
    kept = [0, 3]
    a = orc.assign(h, kept)
    # pre-merge cosines: token 1 -> kept 3 (cos .77 vs 0), token 2 -> kept 3
    assert a.tolist() == [0, 1, 1, 1]


# ------------------------------------------------------------------ post-merge layer
def test_post_layer_is_projection_then_attention():
    r = rng(16)
    n, H, dh = 9, 2, 4
    D = H * dh
    x = orc.round_bf16(r.standard_normal((n, D)))
    w = orc.round_bf16(r.standard_normal((3 * D, D)) * 0.2)
    q, k, v = orc.proj_qkv(x, w, H, "bf16")
    assert np.array_equal(q.reshape(n, D), orc.round_bf16(x @ w[:D].T))
    assert np.array_equal(v.reshape(n, D), orc.round_bf16(x @ w[2 * D:].T))
    y = orc.post_layer(x, w, [0, 4, n], H, "bf16")
    assert np.array_equal(y, orc.round_bf16(orc.attention(q, k, v, [0, 4, n], 1 / math.sqrt(dh))))


def test_proj_qkv_hand_computed_two_rows():
    # every number below is worked out by hand from Q = X W_q^T, K = X W_k^T, V = X W_v^T with
    # W = [W_q; W_k; W_v] stored [out, in]: rows 0-1 -> Q, rows 2-3 -> K, rows 4-5 -> V
    x = np.array([[1.0, 2.0], [3.0, -1.0]])
    w = np.array([[1.0, 2.0], [3.0, 4.0],        # W_q
                  [-1.0, 0.5], [0.0, -2.0],      # W_k
                  [0.5, 0.5], [2.0, -1.0]])      # W_v
    for H in (1, 2):                             # one head of width 2, two heads of width 1: same numbers, other shape
        q, k, v = orc.proj_qkv(x, w, H, "bf16")
        assert q.shape == k.shape == v.shape == (2, H, 2 // H)
        assert q.reshape(2, 2).tolist() == [[5.0, 11.0], [1.0, 5.0]]
        assert k.reshape(2, 2).tolist() == [[0.0, -4.0], [-3.5, 2.0]]
        assert v.reshape(2, 2).tolist() == [[1.5, 0.0], [1.0, 7.0]]
    q2 = orc.proj_qkv(x, w, 2, "bf16")[0]
    assert q2[0, 1, 0] == 11.0 and q2[1, 0, 0] == 1.0          # head h is column h when dh = 1
    # one product that the storage type changes: 1 + 3 * 2^-9 lies between the bf16 neighbours 1 and 1 + 2^-7
    # (closer to the upper one); fp32 holds it exactly
    xr = np.array([[1.0, 1.0]])
    wr = np.tile(np.array([[1.0, 3.0 / 512.0]]), (6, 1))
    assert orc.proj_qkv(xr, wr, 1, "bf16")[1][0, 0, 0] == 1.0078125
    assert orc.proj_qkv(xr, wr, 1, "fp32")[1][0, 0, 0] == 1.005859375
    # an exact tie (1 + 2^-8) goes to the even neighbour, 1
    wt = np.tile(np.array([[1.0, 1.0 / 256.0]]), (6, 1))
    assert orc.proj_qkv(xr, wt, 1, "bf16")[2][0, 0, 0] == 1.0


def test_post_layer_with_zero_query_weights_averages_the_values():
    # W_q = 0 makes every score 0, the softmax uniform, and the layer's output the mean of the request's V rows:
    # with the hand-computed V = [[1.5, 0], [1, 7]] of the case above that is [1.25, 3.5] for both rows
    x = np.array([[1.0, 2.0], [3.0, -1.0]])
    w = np.array([[0.0, 0.0], [0.0, 0.0], [-1.0, 0.5], [0.0, -2.0], [0.5, 0.5], [2.0, -1.0]])
    y = orc.post_layer(x, w, [0, 2], 1, "bf16")
    assert y.tolist() == [[1.25, 3.5], [1.25, 3.5]]
    # two requests of one row each: every row attends to itself only, the output is its own V row
    y = orc.post_layer(x, w, [0, 1, 2], 1, "bf16")
    assert y.tolist() == [[1.5, 0.0], [1.0, 7.0]]


# ------------------------------------------------------------------ schedule + FLOP tables
def test_schedule_endpoints_mean_direction():
    T = 64
    a = [orc.schedule_alpha(s, T, 0.5, 1.0) for s in range(T)]
    assert a[0] == 0.5 and a[-1] == 1.0
    assert abs(np.mean(a) - 0.75) < 1e-12
    assert all(y > x for x, y in zip(a, a[1:]))          # smallest at the beginning of decoding
    rev = [orc.schedule_alpha(s, T, 0.5, 1.0, True) for s in range(T)]
    assert np.allclose(rev, a[::-1])
    assert orc.schedule_alpha(0, 1, 0.3, 0.9) == 0.3


def test_flop_model_reproduces_paper_tables():
    rows = []
    with open(os.path.join(GOLDEN, "flops_tables.txt")) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                m, a, l, val, tol = line.split()
                rows.append((m, float(a), int(l), float(val), float(tol)))
    assert len(rows) == 19
    for method, alpha, l_star, val, tol in rows:
        if method == "baseline":
            got = fm.flops_baseline(fm.N_VIS + fm.N_PROMPT + fm.N_OUT)
        elif method == "d3tom":
            got = fm.flops_d3tom(alpha, l_star)
        else:
            got = fm.flops_d3tom_t(alpha, l_star)
        assert abs(got / 1e12 - val) <= tol, (method, alpha, l_star, got / 1e12, val)


def test_flop_model_is_sensitive_to_the_readings_it_pins():
    # merging the first step too, shifting l*, or a schedule of the same mean over a narrower range each miss the table
    N = fm.N_VIS + fm.N_PROMPT + fm.N_OUT
    all_merged = fm.T_STEPS * fm.flops_step(0.75, 3, N, fm.N_VIS)
    assert abs(all_merged / 1e12 - 109.12) > 0.5
    assert abs(fm.flops_d3tom(0.75, 4) / 1e12 - 109.12) > 0.5
    other = sum(fm.flops_step(orc.schedule_alpha(s, 32, 0.625, 0.875), 3, N, fm.N_VIS) for s in range(32)) / 32
    assert abs((fm.L_LAYERS * fm.flops_layer(N) + 31 * other) / 1e12 - 109.27) > 0.05


# ------------------------------------------------------------------ KV-cache merge (Sec. 4.4)
def test_merge_kv_equals_pure_python_brute_force():
    r = rng(31)
    V, P, D = 9, 3, 4
    K = r.standard_normal((V + P, D)); Vv = r.standard_normal((V + P, D))
    kept = np.array([1, 4, 7])
    res = orc.merge_kv(K, Vv, [0, V + P], [V], [kept], orc.SUM, "fp32")
    # brute force: cosine on K only, sums of K and V, dropped positions
    k_new = {int(k): list(K[k]) for k in kept}; v_new = {int(k): list(Vv[k]) for k in kept}
    for m in range(V):
        if m in kept:
            continue
        best, arg = -2.0, None
        for k in kept:
            dot = sum(K[m][c] * K[k][c] for c in range(D))
            cos = dot / math.sqrt(sum(x * x for x in K[m])) / math.sqrt(sum(x * x for x in K[k]))
            if cos > best:
                best, arg = cos, int(k)
        for c in range(D):
            k_new[arg][c] += K[m][c]; v_new[arg][c] += Vv[m][c]
    want_k = np.array([k_new[int(k)] for k in kept] + [list(x) for x in K[V:]])
    want_v = np.array([v_new[int(k)] for k in kept] + [list(x) for x in Vv[V:]])
    assert np.allclose(res["k_out"], want_k.astype(np.float32), rtol=1e-6, atol=1e-6)
    assert np.allclose(res["v_out"], want_v.astype(np.float32), rtol=1e-6, atol=1e-6)
    assert res["k_out"].shape[0] == P + len(kept) and list(res["src_of_dst"]) == [1, 4, 7, 9, 10, 11]


def test_merge_kv_routing_depends_on_keys_only_and_conserves_mass():
    r = rng(32)
    V, P, D = 40, 5, 8
    K, Va, Vb = (r.standard_normal((V + P, D)).astype(np.float32).astype(np.float64) for _ in range(3))   # storage precision
    kept = np.sort(r.choice(V, 7, replace=False))
    a = orc.merge_kv(K, Va, [0, V + P], [V], [kept], orc.SUM, "fp32")
    b = orc.merge_kv(K, Vb, [0, V + P], [V], [kept], orc.SUM, "fp32")
    assert np.array_equal(a["assign"], b["assign"])                      # values never influence the routing
    assert np.array_equal(a["assign"], orc.assign(K[:V], kept))          # it is the merge routing applied to K
    # SUM conserves the column sums of both caches over the visual rows
    assert np.allclose(a["k_out"][:7].sum(0), K[:V].sum(0), atol=1e-5)
    assert np.allclose(a["v_out"][:7].sum(0), Va[:V].sum(0), atol=1e-5)
    # MEAN divides both by 1 + members
    m = orc.merge_kv(K, Va, [0, V + P], [V], [kept], orc.MEAN, "fp32")
    assert np.allclose(m["v_out"][:7] * (1 + m["member_count"])[:, None], a["v_out"][:7], atol=1e-5)
    # keeping everything is the identity on both caches
    ident = orc.merge_kv(K, Va, [0, V + P], [V], [np.arange(V)], orc.SUM, "fp32")
    assert np.array_equal(ident["k_out"], K) and np.array_equal(ident["v_out"], Va)


# ------------------------------------------------------------------ rest of the block (Algorithm 1, FFN_l; layer-cost equation)
def test_linear_row_o_of_w_holds_output_feature_o_and_the_residual_is_added():
    w = np.array([[1.0, 2.0], [3.0, 4.0], [0.5, -1.0]])
    x = np.array([[1.0, 10.0], [0.0, 1.0]])
    y = orc.linear(x, w, dtype="fp32")
    assert np.array_equal(y, np.array([[21.0, 43.0, -9.5], [2.0, 4.0, -1.0]]))
    res = np.array([[1.0, 1.0, 1.0], [0.0, 0.0, 0.25]])
    assert np.array_equal(orc.linear(x, w, res, dtype="fp32"), y + res)
    # identity weights: the result is the storage rounding of x + residual
    r = rng(40)
    xb = orc.round_bf16(r.standard_normal((5, 8)))
    rb = orc.round_bf16(r.standard_normal((5, 8)))
    assert np.array_equal(orc.linear(xb, np.eye(8), rb, dtype="bf16"), orc.round_bf16(xb + rb))


def test_silu_closed_forms():
    # sigmoid(ln 3) = 3/4
    assert abs(orc.silu(math.log(3.0)) - 0.75 * math.log(3.0)) < 1e-15
    assert orc.silu(0.0) == 0.0
    assert abs(orc.silu(50.0) - 50.0) < 1e-12 and abs(orc.silu(-50.0)) < 1e-12
    assert orc.silu(-1000.0) == 0.0          # exp overflows to inf, the quotient is -0
    g = rng(41).standard_normal(1000) * 4
    want = torch.nn.functional.silu(torch.from_numpy(g)).numpy()
    assert np.allclose(orc.silu(g), want, rtol=1e-13, atol=1e-15)


def test_ffn_gate_and_up_are_not_interchangeable_closed_form():
    # one token, d = 1, m = 1: gate pre-activation ln 3, up 2, down 1 -> 0.75 ln3 * 2
    y, act = orc.ffn(np.array([[1.0]]), np.array([[math.log(3.0)], [2.0]]), np.array([[1.0]]), dtype="fp32")
    assert abs(y[0, 0] - 1.5 * math.log(3.0)) < 1e-6 and abs(act[0, 0] - 1.5 * math.log(3.0)) < 1e-6
    # zero gate matrix: silu(0) = 0, the block returns its residual
    r = rng(42)
    x = r.standard_normal((4, 6)); res = orc.round_bf16(r.standard_normal((4, 6)))
    w = np.concatenate([np.zeros((10, 6)), r.standard_normal((10, 6))])
    y, act = orc.ffn(x, w, r.standard_normal((6, 10)), res, dtype="bf16")
    assert np.array_equal(act, np.zeros((4, 10))) and np.array_equal(y, res)


def test_ffn_equals_pure_python_brute_force_and_torch_fp64():
    r = rng(43)
    n, d, m = 3, 5, 7
    x = r.standard_normal((n, d)); wgu = r.standard_normal((2 * m, d)) * 0.5
    wd = r.standard_normal((d, m)) * 0.5; res = r.standard_normal((n, d))
    want = np.zeros((n, d))
    for i in range(n):
        act = []
        for j in range(m):
            g = sum(x[i, c] * wgu[j, c] for c in range(d))
            u = sum(x[i, c] * wgu[m + j, c] for c in range(d))
            act.append(g / (1.0 + math.exp(-g)) * u)
        for o in range(d):
            want[i, o] = res[i, o] + sum(act[j] * wd[o, j] for j in range(m))
    y, _ = orc.ffn(x, wgu, wd, res, dtype="fp32")
    assert np.allclose(y, want, rtol=1e-6, atol=1e-6)      # fp32 storage rounding only
    F = torch.nn.functional
    tx, tw, td = torch.from_numpy(x), torch.from_numpy(wgu), torch.from_numpy(wd)
    t = F.linear(F.silu(F.linear(tx, tw[:m])) * F.linear(tx, tw[m:]), td) + torch.from_numpy(res)
    assert np.allclose(y, t.numpy(), rtol=1e-6, atol=1e-6)


def test_ffn_activation_is_rounded_to_storage_before_the_second_product():
    r = rng(44)
    n, d, m = 4, 8, 8
    x = orc.round_bf16(r.standard_normal((n, d)))
    wgu = orc.round_bf16(r.standard_normal((2 * m, d)) * 0.5)
    y, act = orc.ffn(x, wgu, np.eye(m), dtype="bf16")       # identity down projection: y is the activation
    assert np.array_equal(act, orc.round_bf16(act))
    assert np.array_equal(y, act)
    exact = orc.silu(x @ wgu[:m].T) * (x @ wgu[m:].T)
    assert np.array_equal(act, orc.round_bf16(exact)) and not np.array_equal(act, exact)


def test_keep_count_of_a_request_without_visual_tokens_is_zero():
    assert orc.keep_count(0, 0.5) == 0 and orc.keep_count(0, 1.0) == 0
    assert orc.keep_count(1, 0.01) == 1          # the clamp to one token needs a token
    assert len(orc.select(np.zeros(0), 0)) == 0
