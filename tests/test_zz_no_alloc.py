"""d3tom_attn_importance_static, the entry point for hosts that may not allocate
device memory (no context; scratch in a fixed array of the library image), must
give what d3tom_attn_importance gives, and what the CPU oracle gives.  Calls in
a row on different problems share that array, so each later one also shows that
nothing left over from the one before leaks into the results.  Batches of one
request take the launcher's own grid shapes (single-tile CTAs for a tiny grid or
for an incomplete last wave), so both of those are among the problems.  This
file is collected last on purpose."""
import numpy as np
import pytest
import torch

from oracle import d3tom_oracle as orc
from paper_2511_12280_b200 import binding as B_
from paper_2511_12280_b200 import workload as wl

import parity_util as pu

pytestmark = pytest.mark.gpu


def _problems():
    a = wl.make_workload("static_a", "bf16", 4, 128, 21, 16,
                         [dict(V=700, P=30, O=40, n_dec=9, r=0.3), dict(V=260, P=5, O=12, n_dec=3, r=0.3)])
    b = wl.make_workload("static_b", "bf16", 2, 64, 22, 8,
                         [dict(V=131, P=9, O=20, n_dec=2, r=0.3), dict(V=90, P=2, O=6, n_dec=0, r=0.3),
                          dict(V=300, P=1, O=3, n_dec=1, r=0.3)])
    # one request, few work items: every 128-row tile becomes a CTA of its own
    c = wl.make_workload("static_c", "bf16", 4, 128, 23, 8, [dict(V=200, P=20, O=30, n_dec=6, r=0.3)])
    # one request at the LLaDA-8B shape (the C1 configuration): 160 work items on 148 SMs, so the items of the
    # incomplete last wave are cut in two
    d = wl.config("C1")
    return [a, b, c, d]


def _run_both(w):
    step = pu.make_step(w, n_post=0, sim_debug=False)
    dev = step.dev
    q, k, v = w.q_for().to(dev), w.k.to(dev), w.v.to(dev)
    step.attn_importance(q, k, v)
    torch.cuda.synchronize()
    want_out = step.attn_out[:step.total].clone()
    want_imp = step.importance[:step.total_vis].clone()
    # poison the outputs of the second path so unwritten entries cannot pass
    out = torch.full_like(want_out, float("nan"))
    imp = torch.full_like(want_imp, float("nan"))
    status = torch.full((1,), 77, dtype=torch.int32, device=dev)
    B_.d3tom_attn_importance_static(w.H, w.dh, q, k, v, step.cu_seqlens, step.n_visual_d, step.dec_pos, step.cu_dec,
                                    step.nB, step.total, step.max_seqlen, step.max_visual, int(step.cu_dec_h[-1]),
                                    step.scale, out, imp, step.cu_vis, status)
    torch.cuda.synchronize()
    step.ctx.close()
    return want_out, want_imp, out, imp, int(status.item())


def test_static_entry_point_matches_the_context_one_on_two_calls_in_a_row():
    for w in _problems():
        want_out, want_imp, out, imp, status = _run_both(w)
        assert status == 0
        # same arithmetic, fixed reduction order: the tolerance of the parity tests holds with room to spare
        pu.assert_close(pu.f64(out), pu.f64(want_out), w.dtype, "static attention output")
        wi, gi = pu.f64(want_imp), pu.f64(imp)
        assert np.isfinite(gi).all()
        assert (np.abs(gi - wi) <= 1e-4 * np.abs(wi) + 1e-7 * w.H * max(1, max(map(len, w.decider_pos)))).all()
        # bit for bit wherever the context call runs the same whole-item kernel (a single request with more work
        # items than SMs is balanced over the SMs there, which cuts some items in two and rounds P differently)
        if not (w.B == 1 and w.H * ((w.seqlens[0] + 255) // 256) > 148):
            assert torch.equal(out, want_out)
            assert torch.equal(imp, want_imp)
        # and against the oracle itself, not only against the other entry point
        q, k, v = pu.f64(w.q_for()), pu.f64(w.k), pu.f64(w.v)
        scale = 1.0 / np.sqrt(w.dh)
        want = orc.round_storage(orc.attention(q, k, v, w.cu_seqlens, scale), w.dtype)
        pu.assert_close(pu.f64(out), want, w.dtype, "static attention output against the oracle")
        dec = np.concatenate([np.asarray(d, np.int64) for d in w.decider_pos])
        S = orc.importance(q, k, w.cu_seqlens, w.n_visual, dec, w.cu_deciders(), scale)
        for b in range(w.B):
            g = gi[w.cu_vis[b]:w.cu_vis[b + 1]]
            assert (np.abs(g - S[b]) <= 1e-4 * np.abs(S[b]) + 1e-7 * len(w.decider_pos[b]) * w.H).all()


def test_static_entry_point_rejects_sizes_beyond_its_array():
    dev = torch.device("cuda", 0)
    z = torch.zeros(8, dtype=torch.int32, device=dev)
    x = torch.zeros(64, 1, 64, dtype=torch.bfloat16, device=dev)
    f = torch.zeros(64, dtype=torch.float32, device=dev)
    with pytest.raises(B_.D3tomError) as e:       # heads * total_tokens beyond the per-head partial section
        B_.d3tom_attn_importance_static(64, 64, x, x, x, z, z, z, z, 1, 1 << 20, 1 << 20, 16, 1, 0.125, x, f, z)
    assert e.value.status == B_.ERR_WORKSPACE
    with pytest.raises(B_.D3tomError) as e:       # heads * deciders * visual beyond the score section
        B_.d3tom_attn_importance_static(32, 128, x, x, x, z, z, z, z, 1, 8192, 8192, 8000, 64, 0.125, x, f, z)
    assert e.value.status == B_.ERR_WORKSPACE
