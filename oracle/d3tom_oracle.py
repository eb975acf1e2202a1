"""Plain CPU oracle for the D3ToM merge-layer path (NumPy, float64).

TEST INFRASTRUCTURE ONLY: the product path never imports this module.

Every function follows one passage of the paper, named in its docstring, in
the paper's order and notation.  Floating point is float64 throughout; the
only library primitives used as steps are ``@`` (matmul), ``exp``, ``sort``.
There is no blocking, fusion or reordering.

Notation (Sec. 3.2): a request is the concatenation [V | P | X] of visual,
prompt and response tokens, N = |V| + |P| + |O|; ``D`` is the decider set
(response positions revealed in the previous step); ``alpha`` is the merge
ratio, ``r = 1 - alpha`` the keep ratio and ``k`` the number of kept tokens.

Readings of points the paper leaves open (each repeated where it is used):
  * multi-head: the paper writes one head; with H heads every head has its
    own softmax with scale 1/sqrt(dh) and the importance sums over heads.
  * k = floor(r*|V| + 1e-9) clamped to [1, |V|].
  * rank ties: lower index wins; argmax ties: lowest kept position wins.
  * all cosines use the pre-merge hidden states (vectorised reading).
  * aggregation: SUM is the paper's equation; MEAN divides by 1 + members.
  * kept tokens keep their original relative order in the output.
  * the schedule is indexed by decode order s = 0..T-1 (alpha grows with s).
  * FFN_l is the gated form (three d x m matrices, as the 3ndm cost term
    implies), without normalisation layers; the residual input is optional.

Pins: every function here is pinned by tests/test_oracle_*.py (closed forms,
brute force on tiny inputs, invariants, and the paper's printed FLOP tables
for the schedule).  The paper prints no worked numeric example of the
method's outputs, so the values of S, kept sets and merged activations are
pinned by definition + brute force + invariants only.
"""
from __future__ import annotations

import numpy as np

SUM = 0
MEAN = 1


# --------------------------------------------------------------------------
# storage rounding
# --------------------------------------------------------------------------
def round_bf16(x):
    """Round to the nearest bfloat16 (8 significant bits, ties to even) and
    return the value in float64.  One rounding, taken directly from float64."""
    x = np.asarray(x, dtype=np.float64)
    m, e = np.frexp(x)                 # x = m * 2**e, 0.5 <= |m| < 1
    q = np.rint(m * 256.0) / 256.0     # 8 significant bits, half-to-even
    return np.ldexp(q, e)


def round_storage(x, dtype: str):
    """Round to the storage type of a config: 'bf16' or 'fp32'."""
    if dtype == "bf16":
        return round_bf16(x)
    if dtype == "fp32":
        return np.asarray(x, dtype=np.float64).astype(np.float32).astype(np.float64)
    raise ValueError(dtype)


# --------------------------------------------------------------------------
# Sec. 3.2.1, self-attention matrix; Algorithm 1, SelfAttn_l
# --------------------------------------------------------------------------
def attention_matrix(q, k, scale):
    """A = softmax_j(q k^T * scale) for one head of one request.

    q: [n_q, dh], k: [n_k, dh] -> A: [n_q, n_k]; rows sum to 1.
    Full bidirectional attention: no mask of any kind."""
    s = (np.asarray(q, np.float64) @ np.asarray(k, np.float64).T) * scale
    s = s - s.max(axis=1, keepdims=True)
    p = np.exp(s)
    return p / p.sum(axis=1, keepdims=True)


def attention(q, k, v, cu_seqlens, scale):
    """Post-attention hidden states H~ of every request (Algorithm 1, SelfAttn_l).

    q, k, v: packed [total, H, dh]; cu_seqlens: [B+1].  Per request and head,
    O = A V with A from ``attention_matrix``; heads are concatenated.
    Returns [total, H*dh] float64."""
    q = np.asarray(q, np.float64)
    k = np.asarray(k, np.float64)
    v = np.asarray(v, np.float64)
    total, H, dh = q.shape
    out = np.zeros((total, H * dh))
    for b in range(len(cu_seqlens) - 1):
        lo, hi = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        for h in range(H):
            A = attention_matrix(q[lo:hi, h], k[lo:hi, h], scale)
            out[lo:hi, h * dh:(h + 1) * dh] = A @ v[lo:hi, h]
    return out


def attention_rows(q, k, v, cu_seqlens, scale, b, rows, h):
    """The same definition restricted to some query rows of one (request, head):
    softmax rows are independent, so this equals ``attention`` on those rows.
    rows: positions relative to the request start.  Returns [len(rows), dh]."""
    lo, hi = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
    rows = np.asarray(rows, dtype=np.int64)
    A = attention_matrix(np.asarray(q[lo:hi, h], np.float64)[rows], k[lo:hi, h], scale)
    return A @ np.asarray(v[lo:hi, h], np.float64)


# --------------------------------------------------------------------------
# Sec. 3.2.1, decider score S_j; Algorithm 1, the line computing S_j
# --------------------------------------------------------------------------
def key_mass(q, k, cu_seqlens, decider_pos, cu_deciders, scale):
    """c_j = sum over heads and over decider rows i in D of A_ij, for ALL keys j
    of each request.  Returns a list of [N_b] arrays.  sum_j c_j = |D| * H."""
    q = np.asarray(q, np.float64)
    k = np.asarray(k, np.float64)
    _, H, _ = q.shape
    res = []
    for b in range(len(cu_seqlens) - 1):
        lo, hi = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        dec = np.asarray(decider_pos[int(cu_deciders[b]):int(cu_deciders[b + 1])], dtype=np.int64)
        c = np.zeros(hi - lo)
        if len(dec):
            for h in range(H):
                A = attention_matrix(q[lo:hi, h][dec], k[lo:hi, h], scale)
                c += A.sum(axis=0)
        res.append(c)
    return res


def importance(q, k, cu_seqlens, n_visual, decider_pos, cu_deciders, scale):
    """S_j for the visual keys of each request: the first |V_b| entries of the
    key mass (visual tokens come first in [V | P | X]).  An empty decider set
    gives S = 0.  Returns a list of [V_b] float64 arrays."""
    c = key_mass(q, k, cu_seqlens, decider_pos, cu_deciders, scale)
    return [c[b][:int(n_visual[b])] for b in range(len(c))]


# --------------------------------------------------------------------------
# Sec. 3.2.1, the kept / merge partition; Algorithm 1, TopK
# --------------------------------------------------------------------------
def keep_count(n_visual: int, keep_ratio: float) -> int:
    """Number of tokens with Rank <= (1 - alpha)|V|: floor(r*|V| + 1e-9),
    clamped to [1, |V|].  The 1e-9 guards products such as (1-0.9)*1000 that
    land just below an integer in binary.  A request without visual tokens
    (|V| = 0, where the clamp has no meaning) keeps nothing."""
    if n_visual <= 0:
        return 0
    k = int(np.floor(keep_ratio * n_visual + 1e-9))
    return max(1, min(int(n_visual), k))


def select(scores, k: int):
    """V_kept: the k tokens of highest score, ties broken toward the lower
    index, returned ASCENDING by position (tokens are removed, not reordered).

    scores are compared as given (pass the float32 array to reproduce a
    float32 decision)."""
    scores = np.asarray(scores)
    order = np.argsort(-scores.astype(np.float64), kind="stable")  # score desc, index asc
    return np.sort(order[:k]).astype(np.int32)


# --------------------------------------------------------------------------
# Sec. 3.2.2, nearest kept neighbour by cosine similarity
# --------------------------------------------------------------------------
def cosine_matrix(h_vis, kept_idx):
    """cos(h~_m, h~_k) for every pruned m (ascending) against every kept k
    (ascending): [(V-k), k].  A zero-norm row has cosine 0 with everything.
    Uses the pre-merge hidden states for every m."""
    h = np.asarray(h_vis, np.float64)
    V = h.shape[0]
    kept_idx = np.asarray(kept_idx, dtype=np.int64)
    mask = np.zeros(V, dtype=bool)
    mask[kept_idx] = True
    pruned_idx = np.nonzero(~mask)[0]
    norm = np.sqrt((h * h).sum(axis=1))
    inv = np.where(norm > 0, 1.0 / np.where(norm > 0, norm, 1.0), 0.0)
    dots = h[pruned_idx] @ h[kept_idx].T
    return dots * inv[pruned_idx][:, None] * inv[kept_idx][None, :], pruned_idx


def argmax_first(sim):
    """k* per row: the first maximiser (lowest kept position)."""
    sim = np.asarray(sim)
    if sim.shape[0] == 0:
        return np.zeros(0, dtype=np.int64)
    return np.argmax(sim, axis=1)


def assign(h_vis, kept_idx, sim=None):
    """Destination slot of every visual token: a kept token maps to its own
    slot (its rank in the ascending kept list); a pruned token m maps to the
    slot of k* = argmax cos.  ``sim`` may supply the [(V-k), k] similarity
    matrix to decide from (teacher forcing); by default it is computed here.
    Returns int32 [V]."""
    V = np.asarray(h_vis).shape[0]
    kept_idx = np.asarray(kept_idx, dtype=np.int64)
    out = np.full(V, -1, dtype=np.int32)
    out[kept_idx] = np.arange(len(kept_idx), dtype=np.int32)
    if sim is None:
        sim, pruned_idx = cosine_matrix(h_vis, kept_idx)
    else:
        mask = np.zeros(V, dtype=bool)
        mask[kept_idx] = True
        pruned_idx = np.nonzero(~mask)[0]
    out[pruned_idx] = argmax_first(sim).astype(np.int32)
    return out


# --------------------------------------------------------------------------
# Sec. 3.2.2, aggregation h~_k* <- h~_k* + h~_m, and physical removal
# --------------------------------------------------------------------------
def aggregate(h_vis, kept_idx, assignment, mode=SUM):
    """Merged kept rows [k, D] and member counts c_k (pruned tokens routed to
    each kept token).  SUM: h~_k + sum of its members.  MEAN: that divided by
    1 + c_k."""
    h = np.asarray(h_vis, np.float64)
    kept_idx = np.asarray(kept_idx, dtype=np.int64)
    k = len(kept_idx)
    out = h[kept_idx].copy()
    count = np.zeros(k, dtype=np.int32)
    is_kept = np.zeros(h.shape[0], dtype=bool)
    is_kept[kept_idx] = True
    for m in range(h.shape[0]):          # ascending m, as in Algorithm 1's loop
        if not is_kept[m]:
            out[assignment[m]] += h[m]
            count[assignment[m]] += 1
    if mode == MEAN:
        out = out / (1.0 + count)[:, None]
    return out, count


def compact(hidden_req, n_visual, kept_idx, merged_rows):
    """Shortened request [merged kept visual rows (ascending position) | prompt
    | response], length N_m = N - |V| + k, and the original row of each output
    row (``src``, relative to the request start)."""
    hidden_req = np.asarray(hidden_req, np.float64)
    n = hidden_req.shape[0]
    kept_idx = np.asarray(kept_idx, dtype=np.int64)
    rest = np.arange(n_visual, n)
    out = np.concatenate([np.asarray(merged_rows, np.float64), hidden_req[rest]], axis=0)
    src = np.concatenate([kept_idx, rest]).astype(np.int32)
    return out, src


def merge(hidden, cu_seqlens, n_visual, kept_idx_list, mode=SUM, dtype="bf16", assignment_list=None):
    """Whole merge of a packed batch.  hidden: [total, D] (already in storage
    precision).  kept_idx_list[b]: ascending kept positions of request b.
    Visual rows are rounded once to ``dtype`` after aggregation; the other rows
    are copied.  Returns dict with hidden_out [sum N_m, D], cu_seqlens_out,
    src_of_dst (original PACKED row), assign (packed by visual offsets),
    member_count (packed by kept offsets)."""
    hidden = np.asarray(hidden, np.float64)
    outs, srcs, assigns, counts = [], [], [], []
    cu_out = [0]
    for b in range(len(cu_seqlens) - 1):
        lo, hi = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        Vb = int(n_visual[b])
        h_req = hidden[lo:hi]
        kept = np.asarray(kept_idx_list[b], dtype=np.int64)
        a = assign(h_req[:Vb], kept) if assignment_list is None else np.asarray(assignment_list[b])
        merged, cnt = aggregate(h_req[:Vb], kept, a, mode)
        merged = round_storage(merged, dtype)
        o, s = compact(h_req, Vb, kept, merged)
        outs.append(o)
        srcs.append(s + lo)
        assigns.append(a)
        counts.append(cnt)
        cu_out.append(cu_out[-1] + o.shape[0])
    return {
        "hidden_out": np.concatenate(outs, axis=0),
        "cu_seqlens_out": np.asarray(cu_out, dtype=np.int32),
        "src_of_dst": np.concatenate(srcs).astype(np.int32),
        "assign": np.concatenate(assigns).astype(np.int32),
        "member_count": np.concatenate(counts).astype(np.int32),
    }


# --------------------------------------------------------------------------
# Sec. 4.4, compatibility with KV-cache: route by cosine on K, add K and V, drop
# --------------------------------------------------------------------------
def merge_kv(k_cache, v_cache, cu_seqlens, n_visual, kept_idx_list, mode=SUM, dtype="bf16", assignment_list=None):
    """The merge applied to a cached [visual | prompt] prefix.  k_cache, v_cache:
    [total, D] (storage precision); per request the kept set K = kept_idx_list[b]
    and its complement M.  For every m in M, pi(m) = argmax_{k in K} cos(K_m, K_k)
    on the pre-merge keys (first maximiser); K_pi(m) += K_m and V_pi(m) += V_m
    (MEAN: both divided by 1 + members, the reading of "renormalise"); the
    positions in M are dropped.  Returns dict with k_out, v_out, cu_seqlens_out,
    src_of_dst, assign, member_count."""
    k_cache = np.asarray(k_cache, np.float64)
    v_cache = np.asarray(v_cache, np.float64)
    k_outs, v_outs, srcs, assigns, counts = [], [], [], [], []
    cu_out = [0]
    for b in range(len(cu_seqlens) - 1):
        lo, hi = int(cu_seqlens[b]), int(cu_seqlens[b + 1])
        Vb = int(n_visual[b])
        kept = np.asarray(kept_idx_list[b], dtype=np.int64)
        K, Vv = k_cache[lo:hi], v_cache[lo:hi]
        pi = assign(K[:Vb], kept) if assignment_list is None else np.asarray(assignment_list[b])   # routing from the keys only
        k_merged, cnt = aggregate(K[:Vb], kept, pi, mode)
        v_merged, cnt_v = aggregate(Vv[:Vb], kept, pi, mode)
        assert np.array_equal(cnt, cnt_v)
        ko, src = compact(K, Vb, kept, round_storage(k_merged, dtype))
        vo, _ = compact(Vv, Vb, kept, round_storage(v_merged, dtype))
        k_outs.append(ko); v_outs.append(vo); srcs.append(src + lo); assigns.append(pi); counts.append(cnt)
        cu_out.append(cu_out[-1] + ko.shape[0])
    return {
        "k_out": np.concatenate(k_outs, axis=0), "v_out": np.concatenate(v_outs, axis=0),
        "cu_seqlens_out": np.asarray(cu_out, dtype=np.int32),
        "src_of_dst": np.concatenate(srcs).astype(np.int32),
        "assign": np.concatenate(assigns).astype(np.int32),
        "member_count": np.concatenate(counts).astype(np.int32),
    }


# --------------------------------------------------------------------------
# layers after l*: attention over the shortened sequence (Sec. 3.2.2, last
# paragraph).  A "layer" here is attention only: X <- MHA(X; W_q, W_k, W_v).
# --------------------------------------------------------------------------
def proj_qkv(x, w_qkv, H, dtype="bf16"):
    """Q, K, V = X W_q, X W_k, X W_v.  w_qkv: [3*D, D], row o holds the weights
    of output feature o (rows 0..D-1 -> Q, D..2D-1 -> K, 2D..3D-1 -> V).
    Results are rounded to the storage type.  Returns three [n, H, dh]."""
    x = np.asarray(x, np.float64)
    w = np.asarray(w_qkv, np.float64)
    n, D = x.shape
    y = round_storage(x @ w.T, dtype)
    dh = D // H
    return (y[:, :D].reshape(n, H, dh), y[:, D:2 * D].reshape(n, H, dh), y[:, 2 * D:].reshape(n, H, dh))


def post_layer(x, w_qkv, cu_seqlens, H, dtype="bf16"):
    """One post-merge layer: projection, attention with scale 1/sqrt(dh),
    output rounded to storage."""
    q, k, v = proj_qkv(x, w_qkv, H, dtype)
    dh = q.shape[2]
    return round_storage(attention(q, k, v, cu_seqlens, 1.0 / np.sqrt(dh)), dtype)


# --------------------------------------------------------------------------
# Algorithm 1, H <- FFN_l(H^): the rest of a Transformer block on the shortened
# sequence.  The layer-cost equation of the FLOPs appendix counts 4 n d^2 for
# the four d x d projections (Q, K, V and the attention output projection) and
# 3 n d m for the feed-forward network, i.e. three d x m matrices.
# Readings: the paper does not write the FFN out; three matrices of d x m are
# the gated form, act = silu(x W_gate^T) * (x W_up^T), y = act W_down^T.  No
# normalisation layer (its weights belong to a trained model); the residual
# input is optional.
# --------------------------------------------------------------------------
def linear(x, w, residual=None, dtype="bf16"):
    """y = residual + x W^T, rounded to the storage type.  w: [N, K], row o
    holds the weights of output feature o.  With K = N = d this is the attention
    output projection, the fourth d x d matrix of the 4 n d^2 term."""
    y = np.asarray(x, np.float64) @ np.asarray(w, np.float64).T
    if residual is not None:
        y = y + np.asarray(residual, np.float64)
    return round_storage(y, dtype)


def silu(g):
    """silu(g) = g * sigmoid(g) = g / (1 + exp(-g))."""
    g = np.asarray(g, np.float64)
    with np.errstate(over="ignore"):
        return g / (1.0 + np.exp(-g))


def ffn(x, w_gate_up, w_down, residual=None, dtype="bf16"):
    """Gated feed-forward network, the 3 n d m term.  w_gate_up: [2m, d], rows
    0..m-1 the gate matrix, rows m..2m-1 the up matrix; w_down: [d, m].
    The activation act = silu(x W_gate^T) * (x W_up^T) is a stored tensor between
    the two products and is rounded to the storage type; y = residual + act W_down^T,
    rounded.  Returns (y, act)."""
    x = np.asarray(x, np.float64)
    w = np.asarray(w_gate_up, np.float64)
    m = w.shape[0] // 2
    gate = x @ w[:m].T
    up = x @ w[m:].T
    act = round_storage(silu(gate) * up, dtype)
    y = act @ np.asarray(w_down, np.float64).T
    if residual is not None:
        y = y + np.asarray(residual, np.float64)
    return round_storage(y, dtype), act


# --------------------------------------------------------------------------
# Sec. 3.2.3, timestep-dependent merge schedule (linear schedule)
# --------------------------------------------------------------------------
def schedule_alpha(s: int, T: int, alpha_min: float, alpha_max: float, reversed_: bool = False) -> float:
    """alpha at decode-order step s = 0..T-1: alpha_min + (alpha_max - alpha_min) * s/(T-1).

    The equation is written with t = 1..T and (t-1)/(T-1); the text fixes the
    direction (smallest at the beginning of decoding), so s = t-1 counts steps
    in the order they are executed.  ``reversed_`` gives the high->low ablation."""
    if T <= 1:
        return float(alpha_min)
    frac = s / (T - 1)
    if reversed_:
        frac = 1.0 - frac
    return float(alpha_min + (alpha_max - alpha_min) * frac)


def merged_length(N: int, n_visual: int, k: int) -> int:
    """N_m = N - alpha|V| with alpha|V| = |V| - k removed tokens."""
    return N - (n_visual - k)
