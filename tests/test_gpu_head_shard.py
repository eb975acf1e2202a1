"""The head-sharded variant on ONE GPU that plays two ranks one after the other (their kernels never wait for one
another): every rank's attention runs through the C ABI on its own heads, the exchange is the module's own combine
code, and the result must match the unsharded step on the same inputs and the oracle."""
import numpy as np
import pytest
import torch

from oracle import d3tom_oracle as orc
from paper_2511_12280_b200 import binding as B_
from paper_2511_12280_b200 import head_shard as hs
from paper_2511_12280_b200 import workload as wl
from paper_2511_12280_b200.pipeline import MergeLayerStep

import parity_util as pu

pytestmark = pytest.mark.gpu


def test_two_played_ranks_match_the_unsharded_step_and_the_oracle():
    G = 2
    w = wl.make_workload("shard_gpu", "bf16", 4, 128, 41, 16,
                         [dict(V=300, P=17, O=24, n_dec=5, r=0.3), dict(V=140, P=3, O=9, n_dec=2, r=0.5)], post_layers=1)
    keep = [B_.d3tom_keep_count(v, r) for v, r in zip(w.n_visual, w.keep_ratio)]
    total = int(w.cu_seqlens[-1])
    n_dec = sum(len(d) for d in w.decider_pos)
    dev = torch.device("cuda", 0)
    q, k, v = w.q_for().to(dev), w.k.to(dev), w.v.to(dev)
    w_post = w.w_post[0].to(dev)

    # the unsharded step
    ref = pu.make_step(w, sim_debug=False)
    ref.run(q, k, v, [w_post])
    torch.cuda.synchronize()

    ranks = []
    for r in range(G):
        h0, h1 = hs.shard_heads(w.H, r, G)
        local = MergeLayerStep(h1 - h0, w.dh, w.torch_dtype, total, w.B, n_dec, max(w.n_visual))
        full = MergeLayerStep(w.H, w.dh, w.torch_dtype, total, w.B, n_dec, max(w.n_visual))
        st = hs.HeadShardedStep(local, full, w.H, w.dh, h0, h1)
        st.set_problem(w.n_visual, w.n_prompt, w.n_resp, w.decider_pos, keep)
        ranks.append((st, h0, h1))
    # ---- attention + partial importance, rank after rank
    slices, parts = [], []
    for st, h0, h1 in ranks:
        hsl, sp = st.attention_local(hs.slice_heads(q, h0, h1), hs.slice_heads(k, h0, h1), hs.slice_heads(v, h0, h1))
        slices.append(hsl.clone()); parts.append(sp.clone())
    torch.cuda.synchronize()
    hidden, imp = hs.combine_hidden(slices), hs.combine_importance(parts)
    assert torch.equal(hidden, ref.attn_out[:total])                      # the same kernel per head: the same bits
    ref_imp = ref.importance[:ref.total_vis]
    assert torch.allclose(imp, ref_imp, rtol=1e-5, atol=1e-7)             # heads added in another order
    # against the oracle itself
    scale = 1.0 / np.sqrt(w.dh)
    want = orc.round_storage(orc.attention(pu.f64(w.q_for()), pu.f64(w.k), pu.f64(w.v), w.cu_seqlens, scale), w.dtype)
    pu.assert_close(pu.f64(hidden), want, w.dtype, "gathered attention output")
    # ---- replicated select + merge: both ranks take the same decisions, and the unsharded ones
    merged = [st.select_and_merge(hidden, imp).clone() for st, _, _ in ranks]
    torch.cuda.synchronize()
    assert torch.equal(merged[0], merged[1])
    for st, _, _ in ranks:
        assert torch.equal(st.full.kept_idx[:st.full.total_kept], ref.kept_idx[:ref.total_kept])
    assert torch.equal(merged[0], ref.hidden_out[:ref.total_out])
    # ---- a post-merge layer on the rank's heads (column-parallel projection), gathered again
    outs = []
    for st, h0, h1 in ranks:
        wl_ = hs.slice_qkv_weights(w_post, w.H, w.dh, h0, h1)
        outs.append(st.post_layer_local(merged[0], wl_).clone())
    torch.cuda.synchronize()
    post = hs.combine_hidden(outs)
    want = orc.post_layer(pu.f64(merged[0]), pu.f64(w.w_post[0]), ref.cu_out_h, w.H, w.dtype)
    pu.assert_close(pu.f64(post), want, w.dtype, "sharded post-merge layer")
    pu.assert_close(pu.f64(post), pu.f64(ref.layer_out[0][:ref.total_out]), w.dtype, "sharded against unsharded layer")
    for st, _, _ in ranks:
        assert st.local.ctx.device_status() == 0 and st.full.ctx.device_status() == 0
