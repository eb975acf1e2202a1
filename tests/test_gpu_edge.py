"""Edge cases of the CUDA path against the oracle: ragged tails, several tiles,
degenerate keep counts and decider sets, adversarial select inputs, host-made
argument errors."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import d3tom_oracle as orc
from paper_2511_12280_b200 import binding as B_
from paper_2511_12280_b200 import workload as wl

import parity_util as pu

pytestmark = pytest.mark.gpu


def small(dtype="bf16", H=2, dh=128, seed=11, reqs=None, post=1):
    reqs = reqs or [dict(V=300, P=17, O=24, n_dec=5, r=0.3), dict(V=129, P=1, O=8, n_dec=1, r=0.1),
                    dict(V=517, P=40, O=33, n_dec=33, r=0.5)]
    return wl.make_workload("small", dtype, H, dh, seed, 16, reqs, post_layers=post)


@pytest.mark.parametrize("dh", [128, 64])
@pytest.mark.parametrize("mode", [B_.AGG_MEAN, B_.AGG_SUM])
def test_ragged_batch_tensor_core_path(dh, mode):
    pu.check_step(small(dh=dh, H=2 if dh == 128 else 4), mode=mode)


def test_ragged_batch_fp32_path():
    pu.check_step(small(dtype="fp32", dh=32, H=2, post=1))


def test_lengths_around_tile_boundaries():
    # one, two and three 128-row tiles with 1-row tails, exact multiples, and a tiny request
    reqs = [dict(V=100, P=20, O=8, n_dec=2, r=0.25), dict(V=120, P=4, O=5, n_dec=5, r=0.25),
            dict(V=240, P=8, O=8, n_dec=3, r=0.25), dict(V=250, P=3, O=4, n_dec=1, r=0.25),
            dict(V=2, P=1, O=1, n_dec=1, r=0.5), dict(V=380, P=3, O=2, n_dec=2, r=0.25)]
    pu.check_step(small(reqs=reqs, post=1))


def test_many_rows_fp32_take_the_streaming_aggregation():
    # more than 4096 output rows: the aggregation runs as the bulk-copy pipeline (bf16 is covered by the ragged
    # serving config); narrow rows keep the oracle cheap
    reqs = [dict(V=3000, P=40, O=12, n_dec=3, r=0.8), dict(V=2600, P=9, O=8, n_dec=2, r=0.7)]
    w = wl.make_workload("rows", "fp32", 2, 32, 13, 16, reqs, post_layers=0)
    pu.check_step(w)
    pu.check_step(w, mode=B_.AGG_SUM)


def test_single_request_single_tile_ctas_with_deciders():
    # one request, few heads: every 128-row tile becomes a CTA of its own (the decider rows included)
    w = small(H=4, reqs=[dict(V=520, P=40, O=40, n_dec=7, r=0.25)], post=1)
    pu.check_step(w)
    w = small(H=2, dh=64, reqs=[dict(V=900, P=11, O=30, n_dec=30, r=0.5)], post=1)
    pu.check_step(w, mode=B_.AGG_SUM)


def test_single_request_balanced_walk_over_the_sms():
    # one request with more (head, 256-row) work items than SMs, in fewer than two rounds: every CTA takes an equal
    # share of the (item, key tile) steps, items are cut between CTAs and their halves merged.  Deciders sit in rows
    # whose items are cut; a ragged last key tile; head_dim 64 and 128; with and without the importance map.
    w = small(H=64, dh=64, reqs=[dict(V=600, P=40, O=60, n_dec=17, r=0.25)], post=1)       # 3 x 64 = 192 items, 6 key tiles
    pu.check_step(w)
    w = small(H=40, dh=128, reqs=[dict(V=900, P=33, O=70, n_dec=64, r=0.5)], post=1)       # 4 x 40 = 160 items, 8 key tiles
    pu.check_step(w)
    # (SUM: merged rows add up dozens of near-identical cluster members, the post-merge logits reach the hundreds and
    #  the softmax becomes an arg-max over near-ties, where one bf16 ulp in q or k picks another key: the post layer
    #  is not comparable within a tolerance there, for any kernel)
    pu.check_step(w, mode=B_.AGG_SUM, check_post=False)
    w = small(H=50, dh=128, reqs=[dict(V=700, P=3, O=66, n_dec=5, r=0.3)], post=0)         # 4 x 50 = 200 items, last block one tile
    pu.check_step(w)


def test_balanced_walk_gives_the_same_bits_on_every_run():
    # the halves of a cut item meet through global memory and a flag; the order of the two terms is fixed, so
    # repeated launches on the same inputs (with other launches in between, which shifts the timing between CTAs)
    # must agree bit for bit, for the rows and for the importance map
    w = small(H=40, dh=128, reqs=[dict(V=900, P=33, O=70, n_dec=64, r=0.5)], post=0)
    step = pu.make_step(w, sim_debug=False)
    dev = step.dev
    q, k, v = w.q_for().to(dev), w.k.to(dev), w.v.to(dev)
    first = None
    for it in range(25):
        step.attn_out.fill_(float("nan")); step.importance.fill_(float("nan"))
        step.attn_importance(q, k, v)
        if it % 3 == 0:
            step.ctx.d3tom_attn_varlen(q, k, v, step.cu_seqlens, 1, step.total, step.max_seqlen, step.scale, step.hidden_out)
        torch.cuda.synchronize()
        got = (step.attn_out[:step.total].clone(), step.importance[:step.total_vis].clone())
        if first is None:
            first = got
        assert torch.equal(got[0], first[0]) and torch.equal(got[1], first[1]), "run %d differs" % it
    assert step.ctx.device_status() == 0
    step.ctx.close()


def test_kept_set_larger_than_the_shared_memory_counters():
    # more than 12288 kept tokens in one request: the member counters live in global memory, the bitmap of a
    # sorting warp spans 13000 positions, and select stages 13000 keys
    w = small(H=1, dh=64, reqs=[dict(V=13000, P=8, O=8, n_dec=3, r=0.97)], post=0)
    # (attention on sampled rows: the oracle's full 13016 x 13016 fp64 matrix would take several GB of host memory)
    pu.check_step(w, full_attention=False, n_sample_rows=6)


@pytest.mark.parametrize("reqs", [
    [dict(V=900, P=9, O=12, n_dec=4, r=0.1)],       # 8 tiles of 128 kept columns: sixteen K slices each
    [dict(V=1500, P=5, O=8, n_dec=3, r=0.07)],      # 12 tiles of 128: eight slices each
    [dict(V=1000, P=7, O=9, n_dec=2, r=0.2)],       # 8 tiles of 256: sixteen slices each
    [dict(V=1000, P=7, O=9, n_dec=5, r=0.3)],       # 8 x 2 tiles of 256, the second 44 columns wide: eight slices
    [dict(V=500, P=3, O=6, n_dec=2, r=0.12), dict(V=300, P=8, O=4, n_dec=4, r=0.33)],   # two requests, 4 + 3 tiles
], ids=["128x16", "128x8", "256x16", "256x8", "batch"])
def test_few_similarity_tiles_are_cut_along_k_and_every_slice_reduces_its_columns(reqs):
    # a handful of (pruned rows x kept columns) tiles and a wide hidden vector: each tile's K range goes to 8 or 16
    # CTAs, which wait for one another and then add up a share of the columns each
    w = small(H=16, dh=128, reqs=reqs, post=0)
    pu.check_step(w, full_attention=False, n_sample_rows=24)
    pu.check_step(w, mode=B_.AGG_SUM, full_attention=False, n_sample_rows=24)


def run_attention_only(lens, H, seed=0):
    """d3tom_attn_varlen on random Q, K, V of a ragged batch against the oracle, every row."""
    dev = torch.device("cuda", 0)
    dh, total = 128, int(sum(lens))
    g = torch.Generator().manual_seed(seed)
    q, k, v = (torch.randn(total, H * dh, generator=g).to(torch.bfloat16) for _ in range(3))
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    ctx = B_.Context(total, len(lens), H, dh, 1, max(lens))
    out = torch.full((total, H * dh), float("nan"), dtype=torch.bfloat16, device=dev)
    scale = 1.0 / dh ** 0.5
    ctx.d3tom_attn_varlen(q.to(dev), k.to(dev), v.to(dev), torch.from_numpy(cu).to(dev), len(lens), total, max(lens), scale, out)
    torch.cuda.synchronize()
    assert ctx.device_status() == 0
    want = orc.round_storage(orc.attention(pu.f64(q).reshape(total, H, dh), pu.f64(k).reshape(total, H, dh),
                                           pu.f64(v).reshape(total, H, dh), cu, scale), "bf16")
    got = pu.f64(out)
    assert np.isfinite(got).all()
    pu.assert_close(got, want.reshape(total, H * dh), "bf16", "attention, one query tile per CTA, lengths %s" % (lens,))
    ctx.close()


def test_attention_with_one_query_tile_per_cta():
    # the kernel with three score buffers: one key block only (the second warpgroup has nothing to do), two, three, four
    # (the buffers come round), ragged last blocks, one-row requests, a batch of unequal lengths (longest first), and a
    # whole step whose post-merge layer runs on it
    B_.d3tom_set_single_tile_attention(1)
    try:
        run_attention_only([100], 2)
        run_attention_only([128], 2, seed=1)
        run_attention_only([129], 2, seed=2)
        run_attention_only([300], 3, seed=3)
        run_attention_only([513], 2, seed=4)
        run_attention_only([1216], 4, seed=5)
        run_attention_only([1, 700, 64, 257, 1000], 2, seed=6)
        pu.check_step(small())
    finally:
        B_.d3tom_set_single_tile_attention(-1)


def test_text_only_request_inside_a_batch():
    # a request without visual tokens between two ordinary ones: nothing to select or merge there, its rows are
    # copied, its attention runs as usual
    w = small(reqs=[dict(V=140, P=9, O=8, n_dec=2, r=0.5), dict(V=0, P=20, O=8, n_dec=2, r=0.5),
                    dict(V=130, P=5, O=8, n_dec=3, r=0.25)])
    pu.check_step(w)


def test_keep_ratio_one_is_identity():
    w = small(post=0)
    step = pu.make_step(w, keep_count=list(w.n_visual), sim_debug=False)
    dev = step.dev
    q, k, v = w.q_for().to(dev), w.k.to(dev), w.v.to(dev)
    step.run(q, k, v)
    torch.cuda.synchronize()
    total = step.total
    assert step.total_out == total
    assert torch.equal(step.hidden_out[:total], step.attn_out[:total])          # bit for bit
    assert step.src_of_dst[:total].cpu().tolist() == list(range(total))
    assert not step.member_count[:step.total_kept].any()
    assert step.keep_mask[:step.total_vis].all()
    step.ctx.close()


def test_keep_one_token_everything_merges_into_it():
    w = small(post=0)
    pu.check_step(w, keep_count=[1, 1, 1])
    pu.check_step(w, keep_count=[1, 1, 1], mode=B_.AGG_SUM)


def test_no_deciders_gives_zero_importance_and_identity():
    w = small(post=0)
    dec = [np.zeros(0, np.int32) for _ in range(w.B)]
    pu.check_step(w, decider_pos=dec)                      # keep_count defaults to |V| without deciders


def test_mixed_decider_counts_and_single_decider():
    w = small(post=0)
    dec = [w.decider_pos[0][:1], np.zeros(0, np.int32), w.decider_pos[2]]
    pu.check_step(w, decider_pos=dec)


def test_duplicate_rows_and_heavy_slots():
    # many identical visual rows: cosine ties resolve to the lowest kept position and
    # some kept tokens collect far more than 32 members (the long-list aggregation path)
    w = small(post=0, reqs=[dict(V=400, P=8, O=8, n_dec=4, r=0.02)])
    w.k[:400] = w.k[:1]
    w.v[5:400] = w.v[5:6]
    pu.check_step(w)
    pu.check_step(w, mode=B_.AGG_SUM)


def run_select(scores_list, ks):
    B = len(scores_list)
    V = [len(s) for s in scores_list]
    cu_vis = np.concatenate([[0], np.cumsum(V)]).astype(np.int32)
    cu_kept = np.concatenate([[0], np.cumsum(ks)]).astype(np.int32)
    ctx = B_.Context(max(8, int(cu_vis[-1])), B, 1, 64, 1, max(V))
    dev = torch.device("cuda", 0)
    imp = torch.as_tensor(np.concatenate(scores_list).astype(np.float32), device=dev)
    t = lambda a: torch.as_tensor(np.asarray(a, np.int32), device=dev)
    kept = torch.full((int(cu_kept[-1]) + 4,), -7, dtype=torch.int32, device=dev)     # 4 guard elements each
    mask = torch.full((int(cu_vis[-1]) + 4,), 9, dtype=torch.uint8, device=dev)
    ctx.d3tom_select(imp, t(cu_vis), t(ks), t(cu_kept), B, max(V), kept, mask)
    torch.cuda.synchronize()
    kept, mask = kept.cpu().numpy(), mask.cpu().numpy()
    assert (kept[cu_kept[-1]:] == -7).all() and (mask[cu_vis[-1]:] == 9).all()
    for b in range(B):
        want = orc.select(scores_list[b].astype(np.float32), ks[b])
        assert np.array_equal(kept[cu_kept[b]:cu_kept[b + 1]], want), b
        m = np.zeros(V[b], np.uint8); m[want] = 1
        assert np.array_equal(mask[cu_vis[b]:cu_vis[b + 1]], m), b
    ctx.close()


def test_select_adversarial_inputs():
    rng = np.random.default_rng(5)
    run_select([np.full(1000, 0.25), np.full(33, 0.0), np.full(1, 3.0)], [400, 33, 1])      # all equal
    run_select([rng.integers(0, 4, 5000) / 8.0, rng.integers(0, 2, 1025) * 1.0], [1234, 1])  # few distinct values
    run_select([rng.random(4096), rng.random(777) * 1e-30, rng.random(2048) * 1e30], [1024, 700, 2048])
    x = rng.random(3000).astype(np.float32)
    x[1000:2000] = x[1500]                               # a long run of ties straddling the threshold
    run_select([x], [int((x > x[1500]).sum()) + 37])
    # keys that differ only in the lowest mantissa bits
    base = np.float32(0.37)
    y = np.array([np.nextafter(base, np.float32(1), dtype=np.float32) if i % 3 == 0 else base for i in range(2000)], np.float32)
    run_select([y], [700])
    run_select([rng.random(70000)], [12345])             # larger than the shared-memory staging
    # between 8192 and 40960 tokens per request the keys are staged in shared memory; a keep count of 0 (nothing
    # kept: all-zero mask, no index written) and one of |V| (everything kept) in the same launch
    run_select([rng.random(20000), rng.integers(0, 3, 9000) / 4.0, rng.random(8193)], [5000, 0, 8193])
    run_select([rng.random(50000), rng.random(100)], [0, 100])
    run_select([rng.random(3000), rng.random(100)], [0, 7])                 # keys in registers, keep count 0


def test_host_made_failures_return_status_codes():
    w = small(post=0)
    step = pu.make_step(w, sim_debug=False)
    dev = step.dev
    q, k, v = w.q_for().to(dev), w.k.to(dev), w.v.to(dev)
    lib = B_.load()
    h = step.ctx._h
    s = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    P = lambda t: ctypes.c_void_p(t.data_ptr())
    # workspace limits
    assert lib.d3tom_attn_varlen(h, B_.BF16, P(q), P(k), P(v), P(step.cu_seqlens), step.nB, step.total + pu.GUARD_ROWS + 1,
                                 step.max_seqlen, 0.1, P(step.attn_out), s) == B_.ERR_WORKSPACE
    assert lib.d3tom_attn_varlen(h, B_.BF16, P(q), P(k), P(v), P(step.cu_seqlens), step.nB + 1, step.total,
                                 step.max_seqlen, 0.1, P(step.attn_out), s) == B_.ERR_WORKSPACE
    # invalid arguments
    assert lib.d3tom_attn_varlen(h, B_.BF16, None, P(k), P(v), P(step.cu_seqlens), step.nB, step.total,
                                 step.max_seqlen, 0.1, P(step.attn_out), s) == B_.ERR_INVALID_ARG
    assert lib.d3tom_attn_varlen(h, B_.BF16, P(q), P(k), P(v), P(step.cu_seqlens), step.nB, step.total,
                                 step.max_seqlen, -1.0, P(step.attn_out), s) == B_.ERR_INVALID_ARG
    assert lib.d3tom_attn_varlen(h, 7, P(q), P(k), P(v), P(step.cu_seqlens), step.nB, step.total,
                                 step.max_seqlen, 0.1, P(step.attn_out), s) == B_.ERR_UNSUPPORTED
    with pytest.raises(B_.D3tomError) as e:
        step.ctx.d3tom_merge(5, step.attn_out, step.cu_seqlens, step.n_visual_d, step.cu_vis, step.kept_idx,
                             step.cu_kept, step.nB, step.D, step.total, step.total_out, step.max_visual,
                             step.max_kept, step.hidden_out, step.cu_out, step.assign, step.member_count,
                             step.src_of_dst)
    assert e.value.status == B_.ERR_INVALID_ARG
    # unsupported head_dim for the tensor-core path
    with pytest.raises(B_.D3tomError) as e:
        bad = B_.Context(256, 1, 2, 96, 1, 128)
        x = torch.zeros(256, 2, 96, dtype=torch.bfloat16, device=dev)
        bad.d3tom_attn_varlen(x, x, x, step.cu_seqlens, 1, 256, 256, 0.1, x)
    assert e.value.status == B_.ERR_UNSUPPORTED
    # the context is still usable afterwards
    step.run(q, k, v)
    torch.cuda.synchronize()
    assert step.ctx.device_status() == 0
    step.ctx.close()


def test_results_are_reproducible_run_to_run():
    w = small(post=1)
    step = pu.make_step(w, sim_debug=False)
    dev = step.dev
    q, k, v = w.q_for().to(dev), w.k.to(dev), w.v.to(dev)
    wp = [x.to(dev) for x in w.w_post]
    outs = []
    for _ in range(3):
        y = step.run(q, k, v, wp)
        torch.cuda.synchronize()
        outs.append((step.importance[:step.total_vis].clone(), step.kept_idx[:step.total_kept].clone(),
                     step.assign[:step.total_vis].clone(), step.hidden_out[:step.total_out].clone(),
                     y[:step.total_out].clone()))
    for o in outs[1:]:
        for a, b in zip(outs[0], o):
            assert torch.equal(a, b)
    step.ctx.close()


def test_a_wait_that_cannot_end_reports_timeout_and_leaves_the_context_usable():
    # the library's wait routine on a barrier that nothing completes, with a 3 ms limit: the kernel returns, the status
    # word says so, and after clearing it the same context computes a correct step
    import time
    w = small(post=0)
    step = pu.make_step(w, sim_debug=False)
    dev = step.dev
    q, k, v = w.q_for().to(dev), w.k.to(dev), w.v.to(dev)
    assert step.ctx.device_status() == 0
    t0 = time.time()
    step.ctx.selftest_wait_timeout(3_000_000)
    torch.cuda.synchronize()
    assert time.time() - t0 < 1.0                       # it gave up after its limit: nothing hung
    assert step.ctx.device_status() == B_.ERR_TIMEOUT
    step.ctx.reset_device_status()
    assert step.ctx.device_status() == 0
    with pytest.raises(B_.D3tomError) as e:             # the limit is bounded on the host: at most one second
        step.ctx.selftest_wait_timeout(5_000_000_000)
    assert e.value.status == B_.ERR_INVALID_ARG
    step.run(q, k, v)
    torch.cuda.synchronize()
    assert step.ctx.device_status() == 0
    scale = 1.0 / np.sqrt(w.dh)
    want = orc.round_storage(orc.attention(pu.f64(w.q_for()), pu.f64(w.k), pu.f64(w.v), w.cu_seqlens, scale), w.dtype)
    pu.assert_close(pu.f64(step.attn_out[:step.total]), want, w.dtype, "attention output after a timed-out wait")
    pu.assert_guard_rows_untouched(step)
    step.ctx.close()
