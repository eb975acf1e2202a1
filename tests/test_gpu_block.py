"""d3tom_linear and d3tom_ffn (Algorithm 1, FFN_l: the rest of a post-merge block) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import d3tom_oracle as orc
from paper_2511_12280_b200 import binding as B_
from paper_2511_12280_b200 import workload as wl

import parity_util as pu

pytestmark = pytest.mark.gpu


def make_ctx(rows, dtype):
    # the dense layers use no scratch of the context; head geometry only has to be valid
    return B_.Context(max(rows, 1), 1, 2, 64 if dtype == "bf16" else 8, 1, 1)


def run_linear(rows, K, N, dtype, residual, in_place=False, seed=0):
    dev = torch.device("cuda", 0)
    t = wl.block_inputs(seed, rows, max(K, N), 8, dtype)
    x = t["x"][:, :K].contiguous()
    w = t["w_o"][:N, :K].contiguous() * 4           # keeps outputs O(1) at small K
    res = t["residual"][:, :N].contiguous() if residual else None
    ctx = make_ctx(rows, dtype)
    xd, wd = x.to(dev), w.to(dev)
    if in_place:
        out = res.to(dev); resd = out
    else:
        out = torch.full((rows, N), float("nan"), dtype=x.dtype, device=dev)
        resd = res.to(dev) if residual else None
    ctx.d3tom_linear(xd, wd, resd, rows, K, N, out)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    want = orc.linear(pu.f64(x), pu.f64(w), pu.f64(res) if residual else None, dtype)
    pu.assert_close(pu.f64(out), want, dtype, "linear %dx%dx%d" % (rows, K, N))
    ctx.close()


@pytest.mark.parametrize("N", [128, 384, 512, 768])      # tile widths 128, 192 / 128, 256, 256 / 192
def test_linear_bf16_every_tile_width_ragged_rows(N):
    run_linear(300, 256, N, "bf16", residual=True)


def test_linear_bf16_without_residual_and_in_place():
    run_linear(300, 192, 256, "bf16", residual=False)
    run_linear(129, 320, 256, "bf16", residual=True, in_place=True)
    run_linear(1, 64, 128, "bf16", residual=True)


def test_linear_and_ffn_bf16_long_k_few_tiles_cut_into_k_slices():
    # six tiles for 148 SMs and 64 k-blocks: the tiles of the (only, incomplete) round are cut into K slices whose
    # partial sums meet in the workspace; the same for the gate/up pass of the feed-forward network
    run_linear(300, 4096, 512, "bf16", residual=True, seed=3)
    run_ffn(300, 4096, 256, "bf16", seed=4)


def test_linear_and_ffn_bf16_shapes_that_take_256_row_tiles():
    # 1500 rows x 48 column tiles: 256-row CTA tiles finish sooner than 128-row ones here (two rounds over the SMs
    # instead of four), for the linear layer and for the gate/up pass; the last tile has 220 of 256 rows
    run_linear(1500, 64, 12288, "bf16", residual=True, seed=5)
    run_linear(1500, 128, 12288, "bf16", residual=False, seed=6)
    run_ffn(1500, 128, 6144, "bf16", seed=7)
    # 1216 rows x 12288 columns: 256 x 224 tiles (275 of them fill two rounds over 148 SMs better than 240 tiles of
    # 256 x 256); 224 does not divide 12288, so the last column tile hangs over the edge of the matrix
    run_linear(1216, 64, 12288, "bf16", residual=True, seed=8)
    run_linear(1216, 128, 12288, "bf16", residual=False, seed=9)


def run_proj(rows, H, dh, seed=0):
    dev = torch.device("cuda", 0)
    D = H * dh
    t = wl.block_inputs(seed, rows, D, 8, "bf16")
    x = t["x"][:, :D].contiguous()
    g = torch.Generator().manual_seed(seed + 1)
    w = (torch.randn(3 * D, D, generator=g) * (4.0 / D ** 0.5)).to(torch.bfloat16)
    ctx = B_.Context(max(rows, 1), 1, H, dh, 1, 1)
    q, k, v = (torch.full((rows, D), float("nan"), dtype=torch.bfloat16, device=dev) for _ in range(3))
    ctx.d3tom_proj_qkv(x.to(dev), w.to(dev), rows, D, q, k, v)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    want = orc.proj_qkv(pu.f64(x), pu.f64(w), H, "bf16")
    for got, ref, name in zip((q, k, v), want, "qkv"):
        pu.assert_close(pu.f64(got), ref.reshape(rows, D), "bf16", "%s of the projection, %d rows, D = %d" % (name, rows, D))
    ctx.close()


def test_dense_layers_on_cta_pairs():
    # 256 x 256 tiles computed by two CTAs (each holds its 128 rows of x and half of the weight tile): a ragged last
    # row tile whose second CTA has no rows at all, whole tiles, more tiles than pairs (several rounds); the output
    # projection with and without residual and the gated feed-forward network (gate rows in one CTA, up rows in the other)
    B_.d3tom_set_pair_tiles(256)
    try:
        run_proj(64, 4, 128)
        run_proj(300, 4, 128, seed=1)
        run_proj(1216, 8, 128, seed=2)
        run_proj(5000, 2, 128, seed=3)
        run_linear(300, 256, 512, "bf16", residual=True)
        run_linear(129, 320, 256, "bf16", residual=True, in_place=True)
        run_linear(2500, 192, 768, "bf16", residual=False)
        run_ffn(300, 256, 512, "bf16", seed=5)
        run_ffn(2300, 128, 384, "bf16", seed=6)
    finally:
        B_.d3tom_set_pair_tiles(-1)


def test_long_dense_layers_take_cta_pairs_by_default():
    # from about two thousand rows on the library picks the pair tiles itself
    run_proj(2304, 4, 128, seed=7)
    run_linear(2100, 256, 512, "bf16", residual=True, seed=8)
    run_ffn(2100, 256, 256, "bf16", seed=9)


def test_linear_fp32_odd_sizes():
    run_linear(70, 50, 45, "fp32", residual=True)
    run_linear(33, 7, 3, "fp32", residual=False)


def run_ffn(rows, D, m, dtype, residual=True, seed=1, sample_rows=None):
    dev = torch.device("cuda", 0)
    t = wl.block_inputs(seed, rows, D, m, dtype)
    scale = 4.0 if D < 1024 else 1.0                  # keeps gate pre-activations O(1) at small D
    x, wgu, wdn = t["x"], t["w_gate_up"] * scale, t["w_down"] * scale
    res = t["residual"] if residual else None
    ctx = make_ctx(rows, dtype)
    act = torch.full((rows, m), float("nan"), dtype=x.dtype, device=dev)
    out = torch.full((rows, D), float("nan"), dtype=x.dtype, device=dev)
    ctx.d3tom_ffn(x.to(dev), wgu.to(dev), wdn.to(dev), res.to(dev) if residual else None, rows, D, m, act, out)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    sel = np.arange(rows) if sample_rows is None else np.asarray(sample_rows)
    xs, rs = pu.f64(x)[sel], (pu.f64(res)[sel] if residual else None)
    want_out, want_act = orc.ffn(xs, pu.f64(wgu), pu.f64(wdn), rs, dtype)
    act_g, out_g = pu.f64(act)[sel], pu.f64(out)[sel]
    pu.assert_close(act_g, want_act, dtype, "ffn activation")
    # second product fed the GPU's own activation (a bf16 rounding flip in act cannot cascade), then free-running
    pu.assert_close(out_g, orc.linear(act_g, pu.f64(wdn), rs, dtype), dtype, "ffn output, teacher-forced")
    pu.assert_close(out_g, want_out, dtype, "ffn output")
    if sample_rows is not None:
        assert torch.isfinite(out.float()).all() and torch.isfinite(act.float()).all()
    ctx.close()


def test_ffn_bf16_ragged_rows_several_tiles():
    run_ffn(300, 256, 384, "bf16")
    run_ffn(127, 128, 128, "bf16", residual=False)


def test_ffn_fp32_odd_sizes():
    run_ffn(37, 24, 20, "fp32")


def test_ffn_bf16_llada_shape_sampled_rows():
    # rows of the shortened sequence of the 4096-visual-token configuration, d = 4096, m = 12288;
    # the oracle computes a sample of rows (the layers act row by row)
    run_ffn(1216, 4096, 12288, "bf16", sample_rows=[0, 1, 127, 128, 640, 1151, 1152, 1215])


def test_linear_bf16_llada_shape_sampled_rows():
    dev = torch.device("cuda", 0)
    rows, D = 1216, 4096
    t = wl.block_inputs(2, rows, D, 8, "bf16")
    ctx = make_ctx(rows, "bf16")
    out = torch.full((rows, D), float("nan"), dtype=torch.bfloat16, device=dev)
    ctx.d3tom_linear(t["x"].to(dev), t["w_o"].to(dev), t["residual"].to(dev), rows, D, D, out)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0 and torch.isfinite(out.float()).all()
    sel = np.array([0, 127, 128, 1000, 1215])
    want = orc.linear(pu.f64(t["x"])[sel], pu.f64(t["w_o"]), pu.f64(t["residual"])[sel], "bf16")
    pu.assert_close(pu.f64(out)[sel], want, "bf16", "output projection")
    ctx.close()


def test_unsupported_shapes_and_bad_arguments_are_refused_on_the_host():
    dev = torch.device("cuda", 0)
    ctx = make_ctx(64, "bf16")
    z = lambda *s: torch.zeros(*s, dtype=torch.bfloat16, device=dev)
    lib = B_.load()
    with pytest.raises(RuntimeError, match="UNSUPPORTED|unsupported"):
        ctx.d3tom_linear(z(64, 64), z(100, 64), None, 64, 64, 100, z(64, 100))       # N not a multiple of 128
    with pytest.raises(RuntimeError, match="UNSUPPORTED|unsupported"):
        ctx.d3tom_linear(z(64, 40), z(128, 40), None, 64, 40, 128, z(64, 128))        # K not a multiple of 64
    with pytest.raises(RuntimeError, match="UNSUPPORTED|unsupported"):
        ctx.d3tom_ffn(z(64, 128), z(200, 128), z(128, 100), None, 64, 128, 100, z(64, 100), z(64, 128))
    x = z(64, 128)
    with pytest.raises(RuntimeError, match="INVALID|invalid"):
        ctx.d3tom_linear(x, z(128, 128), None, 64, 128, 128, x)                       # out must not be x
    ctx.d3tom_linear(x, z(128, 128), None, 0, 128, 128, z(64, 128))                  # no rows: nothing to do
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    ctx.close()


def test_whole_post_merge_block_after_a_merge_step():
    # merge-layer step, then one LLaDA-shaped block (attention, output projection, gated FFN, two residuals) on the
    # shortened ragged batch; every stage is checked against the oracle fed with the GPU's previous stage
    w = wl.make_workload("blk", "bf16", 2, 128, 41, 16, [dict(V=300, P=17, O=24, n_dec=5, r=0.3),
                                                          dict(V=200, P=9, O=8, n_dec=2, r=0.5)], post_layers=1)
    step = pu.make_step(w, sim_debug=False)
    dev = step.dev
    D, m = step.D, 384
    t = wl.block_inputs(7, 8, D, m, "bf16")
    w_o, w_gu, w_dn = t["w_o"] * 2, t["w_gate_up"] * 4, t["w_down"] * 4
    q, k, v = w.q_for().to(dev), w.k.to(dev), w.v.to(dev)
    step.attn_importance(q, k, v); step.select(); step.merge()
    x = step.hidden_out
    y = step.post_block(0, x, w.w_post[0].to(dev), w_o.to(dev), w_gu.to(dev), w_dn.to(dev))
    torch.cuda.synchronize()
    assert step.ctx.device_status() == 0
    n = step.total_out
    xg = pu.f64(x)[:n]
    attn = orc.post_layer(xg, pu.f64(w.w_post[0]), step.cu_out_h, w.H, "bf16").reshape(n, D)
    x1 = orc.linear(attn, pu.f64(w_o), xg, "bf16")
    pu.assert_close(pu.f64(step.block_x1)[:n], x1, "bf16", "x + attn W_o")
    x1g = pu.f64(step.block_x1)[:n]
    want, _ = orc.ffn(x1g, pu.f64(w_gu), pu.f64(w_dn), x1g, "bf16")
    pu.assert_close(pu.f64(y)[:n], want, "bf16", "block output")
    step.ctx.close()
