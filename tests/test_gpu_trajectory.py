"""The trajectory driver on the GPU: per-step graphs replay what host launches compute, and sampled steps of a
scheduled trajectory (forward and reversed, two tokens per step) agree with the oracle."""
import numpy as np
import pytest
import torch

from paper_2511_12280_b200 import binding as B_
from paper_2511_12280_b200 import trajectory as tr
from paper_2511_12280_b200 import workload as wl
from paper_2511_12280_b200.pipeline import MergeLayerStep

import parity_util as pu

pytestmark = pytest.mark.gpu


def workload():
    return wl.make_workload("traj", "bf16", 2, 128, 21, 16, [dict(V=400, P=20, O=8, n_dec=0, r=0.25)],
                            post_layers=1, T=4, mean_keep_ratio=0.25)


@pytest.mark.parametrize("reversed_", [False, True])
def test_graph_replay_equals_host_launches_and_steps_match_the_oracle(reversed_):
    w = workload()
    T, tps = 4, 2
    plan = tr.plan_schedule(w.n_visual, w.n_prompt, [w.decode_order], T, 0.5, 0.9, tokens_per_step=tps,
                            reversed_=reversed_)
    total = int(w.cu_seqlens[-1])
    step = MergeLayerStep(w.H, w.dh, w.torch_dtype, total, 1, tps, max(w.n_visual), n_post=1)
    dev = step.dev
    qs = [w.q_for(p.decider_pos).to(dev) for p in plan]
    k, v = w.k.to(dev), w.v.to(dev)
    w_post = [x.to(dev) for x in w.w_post]
    traj = tr.Trajectory(step, plan, w.n_visual, w.n_prompt, w.n_resp)
    host = []
    for s in range(T):
        y = traj.run_step(s, qs, k, v, w_post)
        torch.cuda.synchronize()
        host.append((y[:step.total_out].clone(), step.kept_idx[:step.total_kept].clone(), step.total_out))
    traj.capture(qs, k, v, w_post)
    for s in range(T):
        y = traj.run_step(s)
        torch.cuda.synchronize()
        assert step.total_out == host[s][2]
        assert torch.equal(y[:step.total_out], host[s][0]) and torch.equal(step.kept_idx[:step.total_kept], host[s][1])
    traj.run()
    torch.cuda.synchronize()
    assert step.ctx.device_status() == 0
    keeps = [p.keep_count[0] for p in plan]
    assert keeps[0] == w.n_visual[0] and (keeps[1:] == sorted(keeps[1:], reverse=not reversed_))
    assert traj.flops(step.D, 1) > 0
    # parity of two steps of the plan (first merged step and the last) against the oracle
    for s in (1, T - 1):
        pu.check_step(w, decider_pos=plan[s].decider_pos, keep_count=plan[s].keep_count)
