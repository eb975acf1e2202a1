"""Host-side driver of a denoising trajectory with the timestep-dependent merge
schedule (Sec. 3.2.3) and the decider set of Sec. 3.2.1.

A trajectory is T merge-layer steps over the same request.  Step s (decode
order, s = 0 first) uses
  * the merge ratio alpha_s of the linear schedule (``d3tom_schedule_alpha``;
    ``reversed_`` gives the high->low ablation),
  * the keep count k_s = ``d3tom_keep_count(|V|, 1 - alpha_s)``,
  * the decider set D_s: the response positions revealed in the previous step
    (``deciders="recent"``, the paper's definition) or all positions revealed
    so far (``deciders="all"``).  The first step has no decider and runs
    unmerged (Algorithm 1, else-branch).
Every size is known on the host before the first launch, so each step is
prepared ahead as one problem of ``MergeLayerStep`` and recorded as one CUDA
graph; running the trajectory is then T graph launches.

This module is marshalling and host arithmetic only (it calls the two host
helpers of the C ABI); every step of the path runs in the library's kernels.
"""
from __future__ import annotations

from types import SimpleNamespace
from typing import List, Optional, Sequence

import numpy as np

from . import binding as B_


def plan_schedule(n_visual: Sequence[int], n_prompt: Sequence[int], decode_order: Sequence[np.ndarray], T: int,
                  alpha_min: float, alpha_max: float, tokens_per_step: int = 1, reversed_: bool = False,
                  deciders: str = "recent", merged: bool = True) -> List[SimpleNamespace]:
    """One entry per step: ``alpha``, ``keep_count`` (per request) and ``decider_pos`` (per request, positions in
    the request, ascending).  decode_order[b] lists the response positions of request b (0-based within the
    response) in the order they are revealed, ``tokens_per_step`` per step.  ``merged=False`` plans the same
    trajectory without merging (every visual token kept): the baseline the saving is measured against."""
    if deciders not in ("recent", "all"):
        raise ValueError("deciders must be 'recent' or 'all'")
    if T < 1 or tokens_per_step < 1:
        raise ValueError("T and tokens_per_step must be positive")
    steps = []
    for s in range(T):
        alpha = B_.d3tom_schedule_alpha(s, T, alpha_min, alpha_max, reversed_)
        dec, keep = [], []
        for b, order in enumerate(decode_order):
            order = np.asarray(order, dtype=np.int64)
            hi = min(s * tokens_per_step, len(order))
            lo = max(0, hi - tokens_per_step) if deciders == "recent" else 0
            pos = np.sort(order[lo:hi]).astype(np.int32) + np.int32(n_visual[b] + n_prompt[b])
            dec.append(pos)
            if merged and len(pos):
                keep.append(B_.d3tom_keep_count(int(n_visual[b]), 1.0 - alpha))
            else:
                keep.append(int(n_visual[b]))          # no decider, or the unmerged baseline: nothing is pruned
        steps.append(SimpleNamespace(step=s, alpha=alpha, keep_count=keep, decider_pos=dec))
    return steps


class Trajectory:
    """The T steps of a plan on one ``MergeLayerStep``: problems are uploaded once, ``capture`` records one CUDA
    graph per step, ``run`` enqueues the whole trajectory in step order."""

    def __init__(self, step, plan: Sequence[SimpleNamespace], n_visual, n_prompt, n_resp):
        self.step = step
        self.plan = list(plan)
        self.problems = [step.make_problem(n_visual, n_prompt, n_resp, p.decider_pos, p.keep_count) for p in self.plan]
        self.graphs: Optional[list] = None
        self._args = None

    def __len__(self):
        return len(self.plan)

    def capture(self, qs, k, v, w_post=None):
        """qs: one Q tensor per step (the decider rows differ from step to step) or a single tensor."""
        qs = list(qs) if isinstance(qs, (list, tuple)) else [qs] * len(self.plan)
        self._args = (qs, k, v, w_post)
        self.graphs = []
        for pr, q in zip(self.problems, qs):
            self.step.use_problem(pr)
            self.graphs.append(self.step.capture(q, k, v, w_post))

    def run_step(self, s: int, qs=None, k=None, v=None, w_post=None):
        """Enqueues step s: its graph if captured, else the host-launched chain (needs the tensors)."""
        self.step.use_problem(self.problems[s])
        if self.graphs is not None:
            self.graphs[s].replay()
            return self.step.layer_out[-1] if self.step.n_post else self.step.hidden_out
        q = qs[s] if isinstance(qs, (list, tuple)) else qs
        return self.step.run(q, k, v, w_post)

    def run(self, qs=None, k=None, v=None, w_post=None):
        out = None
        for s in range(len(self.plan)):
            out = self.run_step(s, qs, k, v, w_post)
        return out

    def flops(self, D: int, n_post: int) -> float:
        """Floating-point operations of what the trajectory runs (2 per multiply-add): merge-layer attention
        4 N^2 D, similarity 2 (V - k) k D, and per post-merge layer the projection 6 N_m D^2 and attention
        4 N_m^2 D (FLOPs appendix, layer-cost and merge-overhead equations restricted to the built steps)."""
        total = 0.0
        for pr in self.problems:
            for n, nv, kc, nm in zip(pr.seqlens_h, pr.n_visual_h, pr.keep_h, pr.out_lens_h):
                total += 4.0 * n * n * D + 2.0 * (nv - kc) * kc * D
                total += n_post * (6.0 * nm * D * D + 4.0 * nm * nm * D)
        return total
