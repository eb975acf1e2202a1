"""The head-sharded variant on two CPU ranks (gloo): every rank computes the oracle's attention and partial
importance for its own heads, the two exchanges run through paper_2511_12280_b200.head_shard, and what comes out
(kept sets, merged rows, a post-merge layer) must equal the single-rank oracle.  No GPU is involved."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import d3tom_oracle as orc
from paper_2511_12280_b200 import head_shard as hs
from paper_2511_12280_b200 import workload as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _workload():
    return wl.make_workload("shard", "fp32", 4, 8, 31, 6,
                            [dict(V=40, P=5, O=6, n_dec=3, r=0.3), dict(V=23, P=2, O=4, n_dec=2, r=0.5)], post_layers=1)


def _single_rank(w):
    q, k, v = (t.double().numpy() for t in (w.q_for(), w.k, w.v))
    scale = 1.0 / np.sqrt(w.dh)
    cu = w.cu_seqlens
    hidden = orc.round_storage(orc.attention(q, k, v, cu, scale), w.dtype)
    dec = np.concatenate(w.decider_pos).astype(np.int64)
    S = orc.importance(q, k, cu, w.n_visual, dec, w.cu_deciders(), scale)
    kept = [orc.select(S[b].astype(np.float32), orc.keep_count(w.n_visual[b], w.keep_ratio[b])) for b in range(w.B)]
    res = orc.merge(hidden, cu, w.n_visual, kept, orc.MEAN, w.dtype)
    post = orc.post_layer(res["hidden_out"], w.w_post[0].double().numpy(), res["cu_seqlens_out"], w.H, w.dtype)
    return hidden, np.concatenate(S), kept, res, post


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = _workload()
        h0, h1 = hs.shard_heads(w.H, rank, world)
        scale = 1.0 / np.sqrt(w.dh)
        cu = w.cu_seqlens
        # this rank's heads only (packed copies, as the kernels take them)
        ql, kl, vl = (hs.slice_heads(t, h0, h1).double().numpy() for t in (w.q_for(), w.k, w.v))
        h_slice = orc.round_storage(orc.attention(ql, kl, vl, cu, scale), w.dtype)
        dec = np.concatenate(w.decider_pos).astype(np.int64)
        s_part = np.concatenate(orc.importance(ql, kl, cu, w.n_visual, dec, w.cu_deciders(), scale))
        # ---- the exchange step
        hidden = hs.exchange_hidden(torch.from_numpy(h_slice)).numpy()
        S = hs.exchange_importance(torch.from_numpy(s_part)).numpy()
        # ---- replicated select + merge
        cv = w.cu_vis
        kept = [orc.select(S[cv[b]:cv[b + 1]].astype(np.float32), orc.keep_count(w.n_visual[b], w.keep_ratio[b]))
                for b in range(w.B)]
        res = orc.merge(hidden, cu, w.n_visual, kept, orc.MEAN, w.dtype)
        # ---- a post-merge layer on this rank's heads, gathered again
        wq, wk, wv = (t.double().numpy() for t in hs.slice_qkv_weights(w.w_post[0], w.H, w.dh, h0, h1))
        x = res["hidden_out"]
        n, Hl = x.shape[0], h1 - h0
        qq, kk, vv = (orc.linear(x, m, None, w.dtype).reshape(n, Hl, w.dh) for m in (wq, wk, wv))
        o_slice = orc.round_storage(orc.attention(qq, kk, vv, res["cu_seqlens_out"], scale), w.dtype)
        post = hs.exchange_hidden(torch.from_numpy(o_slice)).numpy()
        out[rank] = dict(hidden=hidden, S=S, kept=[k.tolist() for k in kept], merged=res["hidden_out"],
                         src=res["src_of_dst"], post=post)
    finally:
        dist.destroy_process_group()


def test_two_ranks_of_heads_reproduce_the_single_rank_step():
    world = 2
    out = mp.Manager().dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    hidden, S, kept, res, post = _single_rank(_workload())
    for r in range(world):
        got = out[r]
        assert np.array_equal(got["hidden"], hidden)                      # heads side by side, nothing mixed up
        assert np.allclose(got["S"], S, rtol=1e-12, atol=0)              # same terms, another order of addition
        assert got["kept"] == [k.tolist() for k in kept]
        assert np.array_equal(got["src"], res["src_of_dst"])
        assert np.array_equal(got["merged"], res["hidden_out"])
        assert np.array_equal(got["post"], post)
    # both ranks hold the same bits after the exchange (they must take the same decisions)
    assert np.array_equal(out[0]["S"], out[1]["S"]) and np.array_equal(out[0]["merged"], out[1]["merged"])


def test_head_ranges_and_weight_slices():
    assert [hs.shard_heads(32, r, 4) for r in range(4)] == [(0, 8), (8, 16), (16, 24), (24, 32)]
    with pytest.raises(ValueError):
        hs.shard_heads(6, 0, 4)
    with pytest.raises(ValueError):
        hs.shard_heads(8, 2, 2)
    H, dh = 4, 2
    D = H * dh
    w = torch.arange(3 * D * D, dtype=torch.float32).reshape(3 * D, D)
    wq, wk, wv = hs.slice_qkv_weights(w, H, dh, 1, 3)
    assert wq.shape == (4, D) and torch.equal(wq, w[2:6]) and torch.equal(wk, w[D + 2:D + 6]) and torch.equal(wv, w[2 * D + 2:2 * D + 6])
    x = torch.arange(2 * H * dh, dtype=torch.float32).reshape(2, H, dh)
    assert torch.equal(hs.slice_heads(x, 1, 3), x[:, 1:3])
    a, b = torch.ones(3, 2), 2 * torch.ones(3, 2)
    assert hs.combine_hidden([a, b]).tolist() == [[1, 1, 2, 2]] * 3
    assert hs.combine_importance([a[:, 0], b[:, 0]]).tolist() == [3, 3, 3]
    assert hs.exchange_importance(a)[0, 0] == 1                            # no process group: identity
