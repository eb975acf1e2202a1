"""d3tom_merge_kv (the merge applied to a cached K/V prefix, Sec. 4.4) against the oracle."""
import numpy as np
import pytest
import torch

from oracle import d3tom_oracle as orc
from paper_2511_12280_b200 import binding as B_
from paper_2511_12280_b200 import workload as wl

import parity_util as pu

pytestmark = pytest.mark.gpu


def run_case(w, mode, keep_ratio=0.25, seed=0):
    """The caches are the workload's K and V rows of each request's [visual | prompt] prefix;
    the kept set is a seeded random subset (the routing does not depend on how it was chosen)."""
    dev = torch.device("cuda", 0)
    rng = np.random.default_rng(seed)
    D, dt = w.D, w.dtype
    cu_full = w.cu_seqlens
    rows = np.concatenate([np.arange(cu_full[b], cu_full[b] + w.n_visual[b] + w.n_prompt[b]) for b in range(w.B)])
    k_h = w.k.reshape(-1, D)[rows].contiguous()
    v_h = w.v.reshape(-1, D)[rows].contiguous()
    lens = [v + p for v, p in zip(w.n_visual, w.n_prompt)]
    keep = [max(1, int(keep_ratio * v)) for v in w.n_visual]
    kept = [np.sort(rng.choice(v, k, replace=False)).astype(np.int32) for v, k in zip(w.n_visual, keep)]
    cs = lambda a: np.concatenate([[0], np.cumsum(a)]).astype(np.int32)
    cu, cu_vis, cu_kept = cs(lens), cs(w.n_visual), cs(keep)
    out_lens = [n - v + k for n, v, k in zip(lens, w.n_visual, keep)]
    cu_out = cs(out_lens)
    total, total_out = int(cu[-1]), int(cu_out[-1])
    t = lambda a: torch.as_tensor(np.asarray(a, np.int32), device=dev)
    ctx = B_.Context(total, w.B, w.H, w.dh, 1, max(w.n_visual))
    k_d, v_d = k_h.to(dev), v_h.to(dev)
    k_out = torch.full((total_out, D), float("nan"), dtype=k_d.dtype, device=dev)
    v_out = torch.full((total_out, D), float("nan"), dtype=k_d.dtype, device=dev)
    assign = torch.full((int(cu_vis[-1]),), -9, dtype=torch.int32, device=dev)
    member_count = torch.full((int(cu_kept[-1]),), -9, dtype=torch.int32, device=dev)
    src = torch.full((total_out,), -9, dtype=torch.int32, device=dev)
    sim = torch.full((int(cu_vis[-1]), max(keep)), float("nan"), dtype=torch.float32, device=dev)
    ctx.d3tom_merge_kv(mode, k_d, v_d, t(cu), t(w.n_visual), t(cu_vis), t(np.concatenate(kept)), t(cu_kept), w.B, D, total,
                       total_out, max(w.n_visual), max(keep), k_out, v_out, t(cu_out), assign, member_count, src, sim)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    # routing: the oracle's arg-max on the GPU's own similarity values, bit-exact; values against fp64 cosines
    kn, vn = pu.f64(k_h), pu.f64(v_h)
    a_gpu, sim_gpu = assign.cpu().numpy(), sim.cpu().numpy()
    assign_list = []
    for b in range(w.B):
        Vb, kb = w.n_visual[b], keep[b]
        Kb = kn[cu[b]:cu[b] + Vb]
        pruned = np.setdiff1d(np.arange(Vb), kept[b])
        s = sim_gpu[cu_vis[b] + pruned][:, :kb]
        assert np.isfinite(s).all()
        want = orc.assign(Kb, kept[b], sim=s)
        assert np.array_equal(a_gpu[cu_vis[b]:cu_vis[b + 1]], want)
        cos, _ = orc.cosine_matrix(Kb, kept[b])
        assert np.abs(s - cos).max() <= 5e-5
        assign_list.append(want)
    res = orc.merge_kv(kn, vn, cu, w.n_visual, kept, orc.MEAN if mode == B_.AGG_MEAN else orc.SUM, dt, assignment_list=assign_list)
    assert np.array_equal(res["cu_seqlens_out"], cu_out)
    assert np.array_equal(member_count.cpu().numpy(), res["member_count"])
    assert np.array_equal(src.cpu().numpy(), res["src_of_dst"])
    ek = pu.assert_close(pu.f64(k_out), res["k_out"], dt, "merged key cache")
    ev = pu.assert_close(pu.f64(v_out), res["v_out"], dt, "merged value cache")
    ctx.close()
    return ek, ev


@pytest.mark.parametrize("mode", [B_.AGG_SUM, B_.AGG_MEAN])
def test_merge_kv_small_ragged(mode):
    reqs = [dict(V=300, P=17, O=4, n_dec=1, r=0.3), dict(V=129, P=1, O=4, n_dec=1, r=0.1), dict(V=517, P=40, O=4, n_dec=1, r=0.5)]
    run_case(wl.make_workload("kv", "bf16", 2, 128, 41, 16, reqs), mode)


def test_merge_kv_fp32_path():
    reqs = [dict(V=200, P=9, O=4, n_dec=1, r=0.3), dict(V=77, P=3, O=4, n_dec=1, r=0.1)]
    run_case(wl.make_workload("kv32", "fp32", 2, 32, 42, 8, reqs), B_.AGG_SUM)


def test_merge_kv_llada_shape():
    # the prefix cache of the LLaDA-8B-shaped config: 1024 visual + 64 prompt rows of width 4096, keep 10 %
    run_case(wl.config("C1"), B_.AGG_MEAN, keep_ratio=0.10)
