"""HostFedStep: steps fed from pinned host memory on three overlapping streams give the results of plain runs."""
import numpy as np
import pytest
import torch

from paper_2511_12280_b200 import binding as B_
from paper_2511_12280_b200 import workload as wl
from paper_2511_12280_b200.pipeline import HostFedStep

import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("use_graphs", [False, True])
def test_overlapped_steps_equal_plain_runs(use_graphs):
    w = wl.make_workload("fed", "bf16", 2, 128, 31, 16, [dict(V=500, P=30, O=16, n_dec=6, r=0.3),
                                                          dict(V=260, P=8, O=16, n_dec=3, r=0.2)], post_layers=1)
    step = pu.make_step(w, sim_debug=False)
    dev = step.dev
    wp = [x.to(dev) for x in w.w_post]
    keep_a = [B_.d3tom_keep_count(v, r) for v, r in zip(w.n_visual, w.keep_ratio)]
    keep_b = [B_.d3tom_keep_count(v, 0.5) for v in w.n_visual]
    probs = [step.make_problem(w.n_visual, w.n_prompt, w.n_resp, w.decider_pos, kc) for kc in (keep_a, keep_b)]
    # six steps, every one with its own inputs (K and V are scaled so that a stale slot would show)
    rng = np.random.default_rng(5)
    ins = []
    for i in range(6):
        f = float(rng.uniform(0.5, 1.5))
        ins.append(tuple((t.float() * f).to(torch.bfloat16).contiguous().pin_memory() for t in (w.q_for(), w.k, w.v)))
    total = int(w.cu_seqlens[-1])
    want = []
    for i, (qh, kh, vh) in enumerate(ins):
        step.use_problem(probs[i & 1])
        y = step.run(qh.to(dev), kh.to(dev), vh.to(dev), wp)
        torch.cuda.synchronize()
        want.append(y[:step.total_out].cpu().clone())
    feed = HostFedStep(step, ins[0][0].to(dev), wp, use_graphs=use_graphs)
    outs = [torch.zeros(total, step.D, dtype=torch.bfloat16).pin_memory() for _ in ins]
    rows = []
    for i, (qh, kh, vh) in enumerate(ins):
        rows.append(feed.submit(qh, kh, vh, outs[i], probs[i & 1], key=i & 1))
    feed.wait()
    torch.cuda.synchronize()
    assert step.ctx.device_status() == 0
    for i in range(len(ins)):
        assert rows[i] == want[i].shape[0]
        assert torch.equal(outs[i][:rows[i]], want[i]), "step %d differs from the plain run" % i
    step.ctx.close()
