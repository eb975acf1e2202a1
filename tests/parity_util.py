"""Staged, teacher-forced comparison of the CUDA path with the CPU oracle.

Discrete decisions are checked in the precision they are taken in: the oracle's
select runs on the GPU's own fp32 importance, the oracle's arg-max runs on the
GPU's own fp32 similarity matrix, and the oracle's aggregation consumes the
GPU's kept sets / assignments, so a float tie can never cascade.  Floats are
compared against the fp64 oracle within the stated tolerances.
"""
from __future__ import annotations

import numpy as np
import torch

from oracle import d3tom_oracle as orc
from paper_2511_12280_b200 import binding as B_
from paper_2511_12280_b200.pipeline import MergeLayerStep

# |gpu - oracle| <= ATOL + RTOL * |oracle|
TOL = {
    "bf16": dict(atol=2e-2, rtol=1e-2),     # bf16 attention outputs and merged activations
    "fp32": dict(atol=1e-5, rtol=1e-4),     # fp32 storage, fp32 arithmetic against fp64
}


def f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


def assert_close(got, want, dtype, what):
    tol = TOL[dtype]
    got, want = np.asarray(got, np.float64), np.asarray(want, np.float64)
    assert got.shape == want.shape, (what, got.shape, want.shape)
    assert np.isfinite(got).all(), what + ": non-finite values"
    err = np.abs(got - want)
    bound = tol["atol"] + tol["rtol"] * np.abs(want)
    bad = err > bound
    if bad.any():
        i = np.unravel_index(np.argmax(err - bound), err.shape)
        raise AssertionError("%s: %d of %d outside tolerance; worst at %s: got %r want %r (max abs err %.3e)"
                             % (what, int(bad.sum()), err.size, i, got[i], want[i], err.max()))
    return float(err.max())


GUARD_ROWS = 5          # slack rows behind every output buffer; nothing may write there
POISON_INT, POISON_U8 = -1, 0xAB


def _output_buffers(step):
    """(name, tensor, rows the step may write) of every buffer a step writes."""
    bufs = [("attn_out", step.attn_out, step.total), ("importance", step.importance, step.total_vis),
            ("kept_idx", step.kept_idx, step.total_kept), ("keep_mask", step.keep_mask, step.total_vis),
            ("assign", step.assign, step.total_vis), ("member_count", step.member_count, step.total_kept),
            ("src_of_dst", step.src_of_dst, step.total_out), ("hidden_out", step.hidden_out, step.total_out)]
    if step.n_post:
        bufs += [("q2", step.q2, step.total_out), ("k2", step.k2, step.total_out), ("v2", step.v2, step.total_out)]
        bufs += [("layer_out%d" % l, t, step.total_out) for l, t in enumerate(step.layer_out)]
    return bufs


def _poison_value(t):
    return float("nan") if t.dtype.is_floating_point else (POISON_U8 if t.dtype == torch.uint8 else POISON_INT)


def poison_outputs(step):
    """Fills every output buffer (slack rows included) with NaN / -1 / 0xAB, so that an element the
    kernels forget to write cannot pass by holding an earlier run's correct value."""
    for _, t, _ in _output_buffers(step):
        t.fill_(_poison_value(t))


def assert_guard_rows_untouched(step):
    """The rows behind the part of each buffer that this problem owns still hold the poison."""
    for name, t, used in _output_buffers(step):
        tail = t[used:]
        assert tail.shape[0] >= GUARD_ROWS, name
        if t.dtype.is_floating_point:
            assert bool(torch.isnan(tail).all()), "%s: a kernel wrote past row %d" % (name, used)
        else:
            assert bool((tail == _poison_value(t)).all()), "%s: a kernel wrote past element %d" % (name, used)


def make_step(w, n_post=None, mode=B_.AGG_MEAN, sim_debug=True, decider_pos=None, keep_count=None) -> MergeLayerStep:
    """A step whose buffers are GUARD_ROWS rows longer than the problem and poisoned."""
    n_post = len(w.w_post) if n_post is None else n_post
    decider_pos = w.decider_pos if decider_pos is None else decider_pos
    if keep_count is None:
        keep_count = [B_.d3tom_keep_count(v, r) if len(d) else v
                      for v, r, d in zip(w.n_visual, w.keep_ratio, decider_pos)]
    total = int(w.cu_seqlens[-1])
    step = MergeLayerStep(w.H, w.dh, w.torch_dtype, total + GUARD_ROWS, w.B, sum(len(d) for d in decider_pos),
                          max(w.n_visual), n_post=n_post, mode=mode, sim_debug=sim_debug)
    step.set_problem(w.n_visual, w.n_prompt, w.n_resp, decider_pos, keep_count)
    poison_outputs(step)
    return step


def check_step(w, mode=B_.AGG_MEAN, full_attention=True, n_sample_rows=48, decider_pos=None, keep_count=None,
               reference_kernels=False, seed=0, check_post=True):
    """Runs one merge-layer step of workload ``w`` on the GPU and checks every
    output against the oracle.  Returns a dict of max-abs errors."""
    decider_pos = w.decider_pos if decider_pos is None else decider_pos
    step = make_step(w, mode=mode, sim_debug=True, decider_pos=decider_pos, keep_count=keep_count)
    if reference_kernels:
        step.ctx.set_reference_kernels(True)
    dev = step.dev
    q_h = w.q_for(decider_pos)
    q, k, v = q_h.to(dev), w.k.to(dev), w.v.to(dev)
    w_post = [x.to(dev) for x in w.w_post]
    step.run(q, k, v, w_post)
    torch.cuda.synchronize()
    assert step.ctx.device_status() == 0, "device status word reports a kernel-side problem"
    assert_guard_rows_untouched(step)

    rep = {}
    H, dh, D, dt = w.H, w.dh, w.D, w.dtype
    cu, cu_vis = w.cu_seqlens, w.cu_vis
    qn, kn, vn = f64(q_h), f64(w.k), f64(w.v)
    scale = 1.0 / np.sqrt(dh)
    total = int(cu[-1])

    # ---- (0) attention output H~
    attn_gpu = f64(step.attn_out[:total])
    assert np.isfinite(attn_gpu).all(), "attention output has unwritten (poisoned) elements"
    if full_attention:
        want = orc.round_storage(orc.attention(qn, kn, vn, cu, scale), dt)
        rep["attn"] = assert_close(attn_gpu, want, dt, "attention output")
    else:
        rng = np.random.default_rng(seed)
        worst = 0.0
        for _ in range(n_sample_rows):
            b = int(rng.integers(0, w.B)); h = int(rng.integers(0, H))
            nb = int(cu[b + 1] - cu[b])
            rows = np.unique(np.concatenate([rng.integers(0, nb, 3), [0, nb - 1]]))
            want = orc.round_storage(orc.attention_rows(qn, kn, vn, cu, scale, b, rows, h), dt)
            got = attn_gpu[int(cu[b]) + rows, h * dh:(h + 1) * dh]
            worst = max(worst, assert_close(got, want, dt, "attention rows (b=%d,h=%d)" % (b, h)))
        rep["attn"] = worst

    # ---- (i) importance: fp32, 1e-4 relative (+ 1e-7 per contributing row)
    dec_cat = np.concatenate([np.asarray(d, np.int64) for d in decider_pos]) if sum(map(len, decider_pos)) else np.zeros(0, np.int64)
    cu_d = w.cu_deciders(decider_pos)
    S = orc.importance(qn, kn, cu, w.n_visual, dec_cat, cu_d, scale)
    imp_gpu = step.importance[:int(cu_vis[-1])].cpu().numpy()
    for b in range(w.B):
        g = imp_gpu[cu_vis[b]:cu_vis[b + 1]].astype(np.float64)
        nd = len(decider_pos[b])
        bound = 1e-4 * np.abs(S[b]) + 1e-7 * nd * H
        assert np.isfinite(g).all()
        assert (np.abs(g - S[b]) <= bound).all(), "importance of request %d: max rel err %.3e" % (
            b, float(np.max(np.abs(g - S[b]) / np.maximum(np.abs(S[b]), 1e-30))))
        assert g.sum() <= nd * H * (1 + 1e-4)          # mass over visual keys cannot exceed deciders x heads
        if nd == 0:
            assert not g.any()

    # ---- (ii) select: the oracle's rule on the GPU's own fp32 scores, bit-exact
    kept_gpu = step.kept_idx[:step.total_kept].cpu().numpy()
    mask_gpu = step.keep_mask[:step.total_vis].cpu().numpy()
    kept_list = []
    for b in range(w.B):
        kb = step.keep_h[b]
        want = orc.select(imp_gpu[cu_vis[b]:cu_vis[b + 1]], kb)
        got = kept_gpu[step.cu_kept_h[b]:step.cu_kept_h[b + 1]]
        assert np.array_equal(got, want), "kept indices of request %d differ" % b
        m = np.zeros(w.n_visual[b], np.uint8); m[want] = 1
        assert np.array_equal(mask_gpu[cu_vis[b]:cu_vis[b + 1]], m)
        kept_list.append(want)

    # ---- (iii) assignment: oracle arg-max on the GPU's own similarity values, bit-exact;
    #      the similarity values themselves against the fp64 cosines
    assign_gpu = step.assign[:step.total_vis].cpu().numpy()
    sim_gpu = step.sim_debug.cpu().numpy() if step.sim_debug is not None else None
    assign_list = []
    worst_sim = 0.0
    for b in range(w.B):
        Vb, kb = w.n_visual[b], step.keep_h[b]
        a_gpu = assign_gpu[cu_vis[b]:cu_vis[b + 1]]
        h_vis = attn_gpu[int(cu[b]):int(cu[b]) + Vb]
        if kb < Vb:
            pruned = np.setdiff1d(np.arange(Vb), kept_list[b])
            sim = sim_gpu[cu_vis[b] + pruned][:, :kb]
            assert np.isfinite(sim).all(), "similarity dump has unwritten entries"
            want = orc.assign(h_vis, kept_list[b], sim=sim)
            cos, _ = orc.cosine_matrix(h_vis, kept_list[b])
            worst_sim = max(worst_sim, float(np.abs(sim - cos).max()))
            assert np.abs(sim - cos).max() <= 5e-5, "similarity values differ from fp64 cosines"
            # wherever the fp64 oracle has a clear winner the GPU must agree with it
            top2 = np.sort(cos, axis=1)[:, -2:] if kb > 1 else None
            clear = (top2[:, 1] - top2[:, 0] > 1e-4) if kb > 1 else np.ones(len(pruned), bool)
            assert np.array_equal(a_gpu[pruned][clear], np.argmax(cos, axis=1)[clear])
        else:
            want = orc.assign(h_vis, kept_list[b], sim=np.zeros((0, kb), np.float32))
        assert np.array_equal(a_gpu, want), "assignment of request %d differs" % b
        assign_list.append(want)
    rep["sim"] = worst_sim

    # ---- (iv) aggregation + compaction from the GPU's decisions
    res = orc.merge(attn_gpu, cu, w.n_visual, kept_list, orc.MEAN if mode == B_.AGG_MEAN else orc.SUM, dt,
                    assignment_list=assign_list)
    assert np.array_equal(res["cu_seqlens_out"], step.cu_out_h)
    assert np.array_equal(step.member_count[:step.total_kept].cpu().numpy(), res["member_count"])
    assert np.array_equal(step.src_of_dst[:step.total_out].cpu().numpy(), res["src_of_dst"])
    hid_gpu = f64(step.hidden_out[:step.total_out])
    rep["merge"] = assert_close(hid_gpu, res["hidden_out"], dt, "merged hidden states")
    # rows that are not merged are bit-identical copies
    src = res["src_of_dst"]
    cnt_of_row = np.zeros(step.total_out, np.int64)
    for b in range(w.B):
        o0 = step.cu_out_h[b]
        cnt_of_row[o0:o0 + step.keep_h[b]] = res["member_count"][step.cu_kept_h[b]:step.cu_kept_h[b + 1]]
    untouched = cnt_of_row == 0
    assert np.array_equal(hid_gpu[untouched], attn_gpu[src[untouched]])
    for b in range(w.B):
        o0, o1 = step.cu_out_h[b], step.cu_out_h[b + 1]
        assert np.all(np.diff(src[o0:o1]) > 0)
        assert o1 - o0 == orc.merged_length(step.seqlens_h[b], w.n_visual[b], step.keep_h[b])

    # ---- (v) post-merge layers, each fed the GPU's previous output
    if check_post and step.n_post:
        x = hid_gpu
        for l in range(step.n_post):
            wl = f64(w.w_post[l])
            got = f64(step.layer_out[l][:step.total_out])
            assert np.isfinite(got).all(), "post-merge layer %d has unwritten (poisoned) elements" % l
            if full_attention:
                want = orc.post_layer(x, wl, step.cu_out_h, H, dt)
                rep["post%d" % l] = assert_close(got, want, dt, "post-merge layer %d" % l)
            else:
                qq, kk, vv = orc.proj_qkv(x, wl, H, dt)
                rng = np.random.default_rng(seed + 1 + l)
                worst = 0.0
                for _ in range(max(8, n_sample_rows // 4)):
                    b = int(rng.integers(0, w.B)); h = int(rng.integers(0, H))
                    nb = int(step.cu_out_h[b + 1] - step.cu_out_h[b])
                    rows = np.unique(np.concatenate([rng.integers(0, nb, 3), [0, nb - 1]]))
                    want = orc.round_storage(orc.attention_rows(qq, kk, vv, step.cu_out_h, scale, b, rows, h), dt)
                    g = got[int(step.cu_out_h[b]) + rows, h * dh:(h + 1) * dh]
                    worst = max(worst, assert_close(g, want, dt, "post-merge layer %d rows" % l))
                rep["post%d" % l] = worst
            x = got
    step.ctx.close()
    return rep
