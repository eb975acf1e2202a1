"""One merge-layer step as a chain of C-ABI calls on one stream:

    d3tom_attn_importance -> d3tom_select -> d3tom_merge
        -> n_post x (d3tom_proj_qkv -> d3tom_attn_varlen)

This class only owns device buffers and marshals sizes; every step of the path
runs inside the library's kernels.  Sizes that the C ABI takes from the host
(keep counts, prefix sums of kept counts and of the shortened lengths) are
computed here from the request shapes; nothing is read back from the device
between the calls.
"""
from __future__ import annotations

from types import SimpleNamespace
from typing import List, Optional, Sequence

import numpy as np
import torch

from . import binding as B_


def _i32(a, device):
    return torch.as_tensor(np.asarray(a, dtype=np.int32), device=device)


class MergeLayerStep:
    def __init__(self, H: int, dh: int, dtype: torch.dtype, max_total_tokens: int, max_batch: int,
                 max_deciders: int, max_visual_per_request: int, n_post: int = 0, mode: int = B_.AGG_MEAN,
                 sim_debug: bool = False, device: int = 0):
        self.H, self.dh, self.D = H, dh, H * dh
        self.dtype = dtype
        self.dev = torch.device("cuda", device)
        self.mode = mode
        self.n_post = n_post
        self.want_sim_debug = sim_debug
        self.ctx = B_.Context(max_total_tokens, max_batch, H, dh, max(1, max_deciders), max_visual_per_request, device)
        T = max_total_tokens
        kw = dict(device=self.dev)
        self.attn_out = torch.empty(T, self.D, dtype=dtype, **kw)
        self.importance = torch.empty(T, dtype=torch.float32, **kw)
        self.kept_idx = torch.empty(T, dtype=torch.int32, **kw)
        self.keep_mask = torch.empty(T, dtype=torch.uint8, **kw)
        self.assign = torch.empty(T, dtype=torch.int32, **kw)
        self.member_count = torch.empty(T, dtype=torch.int32, **kw)
        self.src_of_dst = torch.empty(T, dtype=torch.int32, **kw)
        self.hidden_out = torch.empty(T, self.D, dtype=dtype, **kw)
        self.sim_debug = None
        if n_post:
            self.q2 = torch.empty(T, self.D, dtype=dtype, **kw)
            self.k2 = torch.empty(T, self.D, dtype=dtype, **kw)
            self.v2 = torch.empty(T, self.D, dtype=dtype, **kw)
            self.layer_out = [torch.empty(T, self.D, dtype=dtype, **kw) for _ in range(n_post)]
        self.scale = 1.0 / float(np.sqrt(dh))

    # ------------------------------------------------------------------ problem description (small index arrays)
    def make_problem(self, n_visual: Sequence[int], n_prompt: Sequence[int], n_resp: Sequence[int],
                     decider_pos: List[np.ndarray], keep_count: Sequence[int]) -> SimpleNamespace:
        """Uploads the index arrays of a batch and returns them with the host-side sizes the C ABI
        wants.  keep_count[b] = number of kept visual tokens of request b (from d3tom_keep_count); a
        request without deciders must be given keep_count = n_visual (Algorithm 1, else-branch).
        Several problems can be prepared ahead (one per denoising step) and switched with
        use_problem() without touching the device."""
        pr = SimpleNamespace()
        pr.nB = len(n_visual)
        pr.n_visual_h = [int(x) for x in n_visual]
        pr.seqlens_h = [int(v + p + o) for v, p, o in zip(n_visual, n_prompt, n_resp)]
        pr.keep_h = [int(x) for x in keep_count]
        pr.out_lens_h = [n - v + k for n, v, k in zip(pr.seqlens_h, pr.n_visual_h, pr.keep_h)]
        cs = lambda a: np.concatenate([[0], np.cumsum(a)]).astype(np.int32)
        pr.cu_seqlens_h, pr.cu_vis_h = cs(pr.seqlens_h), cs(pr.n_visual_h)
        pr.cu_kept_h, pr.cu_out_h = cs(pr.keep_h), cs(pr.out_lens_h)
        pr.cu_dec_h = cs([len(d) for d in decider_pos])
        dec = np.concatenate([np.asarray(d, dtype=np.int32) for d in decider_pos]) if pr.cu_dec_h[-1] else np.zeros(1, np.int32)
        d = self.dev
        pr.cu_seqlens, pr.cu_vis = _i32(pr.cu_seqlens_h, d), _i32(pr.cu_vis_h, d)
        pr.cu_kept, pr.cu_out = _i32(pr.cu_kept_h, d), _i32(pr.cu_out_h, d)
        pr.cu_dec, pr.dec_pos = _i32(pr.cu_dec_h, d), _i32(dec, d)
        pr.n_visual_d, pr.keep_d = _i32(pr.n_visual_h, d), _i32(pr.keep_h, d)
        pr.total = int(pr.cu_seqlens_h[-1])
        pr.total_vis = int(pr.cu_vis_h[-1])
        pr.total_kept = int(pr.cu_kept_h[-1])
        pr.total_out = int(pr.cu_out_h[-1])
        pr.max_seqlen, pr.max_visual = max(pr.seqlens_h), max(pr.n_visual_h)
        pr.max_kept, pr.max_out = max(pr.keep_h), max(pr.out_lens_h)
        return pr

    def use_problem(self, pr: SimpleNamespace):
        self.__dict__.update(vars(pr))
        if self.want_sim_debug:
            self.sim_debug = torch.full((self.total_vis, self.max_kept), float("nan"), dtype=torch.float32, device=self.dev)

    def set_problem(self, n_visual, n_prompt, n_resp, decider_pos, keep_count):
        self.use_problem(self.make_problem(n_visual, n_prompt, n_resp, decider_pos, keep_count))

    # ------------------------------------------------------------------ the calls
    def attn_importance(self, q, k, v, stream=None):
        self.ctx.d3tom_attn_importance(q, k, v, self.cu_seqlens, self.n_visual_d, self.dec_pos, self.cu_dec, self.nB,
                                       self.total, self.max_seqlen, self.max_visual, int(self.cu_dec_h[-1]),
                                       self.scale, self.attn_out, self.importance, self.cu_vis, stream)

    def select(self, stream=None):
        self.ctx.d3tom_select(self.importance, self.cu_vis, self.keep_d, self.cu_kept, self.nB, self.max_visual,
                              self.kept_idx, self.keep_mask, stream)

    def merge(self, hidden=None, stream=None):
        hidden = self.attn_out if hidden is None else hidden
        self.ctx.d3tom_merge(self.mode, hidden, self.cu_seqlens, self.n_visual_d, self.cu_vis, self.kept_idx,
                             self.cu_kept, self.nB, self.D, self.total, self.total_out, self.max_visual,
                             self.max_kept, self.hidden_out, self.cu_out, self.assign, self.member_count,
                             self.src_of_dst, self.sim_debug, stream)

    def post_layer(self, l: int, x, w_qkv, stream=None):
        self.ctx.d3tom_proj_qkv(x, w_qkv, self.total_out, self.D, self.q2, self.k2, self.v2, stream)
        self.ctx.d3tom_attn_varlen(self.q2, self.k2, self.v2, self.cu_out, self.nB, self.total_out, self.max_out,
                                   self.scale, self.layer_out[l], stream)

    def post_block(self, l: int, x, w_qkv, w_o, w_gate_up, w_down, stream=None):
        """A whole post-merge block on the shortened sequence (Algorithm 1, the layers after l*; layer-cost
        equation): attention as in post_layer, then x1 = x + attn W_o^T and y = x1 + FFN(x1), written to
        layer_out[l].  The activation scratch [rows, m] is allocated on first use."""
        m = w_down.shape[1]
        if getattr(self, "ffn_act", None) is None or self.ffn_act.shape[1] != m:
            self.ffn_act = torch.empty(self.attn_out.shape[0], m, dtype=self.dtype, device=self.dev)
            self.block_x1 = torch.empty_like(self.attn_out)
        self.post_layer(l, x, w_qkv, stream)
        n = self.total_out
        self.ctx.d3tom_linear(self.layer_out[l], w_o, x, n, self.D, self.D, self.block_x1, stream)
        self.ctx.d3tom_ffn(self.block_x1, w_gate_up, w_down, self.block_x1, n, self.D, m, self.ffn_act,
                           self.layer_out[l], stream)
        return self.layer_out[l]

    def run(self, q, k, v, w_post: Optional[Sequence[torch.Tensor]] = None, stream=None):
        """Enqueue the whole step.  Returns the last tensor of the chain."""
        self.attn_importance(q, k, v, stream)
        self.select(stream)
        self.merge(stream=stream)
        x = self.hidden_out
        for l in range(self.n_post):
            self.post_layer(l, x, w_post[l], stream)
            x = self.layer_out[l]
        return x

    def capture(self, q, k, v, w_post: Optional[Sequence[torch.Tensor]] = None):
        """Records run(q, k, v, w_post) for the current problem into a CUDA graph and returns it
        (call .replay() to enqueue the whole step with one launch).  The graph reads and writes
        the same buffers as run(); q, k, v may be refilled between replays.  One untimed run is
        made first on a side stream, as capture requires."""
        side = torch.cuda.Stream(device=self.dev)
        side.wait_stream(torch.cuda.current_stream(self.dev))
        with torch.cuda.stream(side):
            self.run(q, k, v, w_post)
        torch.cuda.current_stream(self.dev).wait_stream(side)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            self.run(q, k, v, w_post)
        return graph

    def launches_per_step(self) -> int:
        """Kernels of this library launched by one run(): attention 1 + importance finish 1,
        select 1, merge 1 (prepare) + 1 (similarity, when something is pruned) + 2 (members,
        aggregate/compact), and 2 per post-merge layer."""
        sim = 1 if self.total_out < self.total else 0
        return 2 + 1 + 1 + sim + 2 + 2 * self.n_post


class HostFedStep:
    """Runs merge-layer steps whose Q, K, V live in pinned host memory and whose result goes back to the host.

    Three streams: the inputs of step i + 1 are copied to the device (two input slots) while step i computes on
    the caller's current stream, and the result of step i leaves on a third stream while step i + 1 computes, so
    a sequence of steps costs max(copy, compute) per step instead of their sum.  ``submit`` only enqueues;
    ``wait`` makes the caller's current stream wait for the last result copy.  With ``use_graphs`` every
    (problem, slot) pair is recorded once as a CUDA graph and replayed."""

    def __init__(self, step: MergeLayerStep, like: torch.Tensor, w_post: Optional[Sequence[torch.Tensor]] = None,
                 use_graphs: bool = True):
        self.step, self.w_post, self.use_graphs = step, w_post, use_graphs
        dev = step.dev
        self.slots = [SimpleNamespace(q=torch.empty(like.shape, dtype=like.dtype, device=dev),
                                      k=torch.empty(like.shape, dtype=like.dtype, device=dev),
                                      v=torch.empty(like.shape, dtype=like.dtype, device=dev)) for _ in range(2)]
        self.copy_stream = torch.cuda.Stream(device=dev)
        self.out_stream = torch.cuda.Stream(device=dev)
        self.copied = [torch.cuda.Event() for _ in range(2)]
        self.consumed = [torch.cuda.Event() for _ in range(2)]
        self.computed, self.out_done = torch.cuda.Event(), torch.cuda.Event()
        self.graphs = {}
        self.n = 0

    def submit(self, q_h, k_h, v_h, out_h, problem, key=None):
        """q_h, k_h, v_h: pinned host tensors shaped like the slots; out_h: pinned host tensor that receives the
        rows of the last tensor of the chain; problem: from ``MergeLayerStep.make_problem``; key: a hashable
        name of the problem for the graph cache (defaults to its identity)."""
        step = self.step
        s = self.n & 1
        self.n += 1
        slot = self.slots[s]
        cur = torch.cuda.current_stream(step.dev)
        with torch.cuda.stream(self.copy_stream):
            self.copy_stream.wait_event(self.consumed[s])       # the step that last read this slot has run
            slot.q.copy_(q_h, non_blocking=True)
            slot.k.copy_(k_h, non_blocking=True)
            slot.v.copy_(v_h, non_blocking=True)
            self.copied[s].record(self.copy_stream)
        step.use_problem(problem)
        gkey = (id(problem) if key is None else key, s)
        if self.use_graphs and gkey not in self.graphs:
            # recorded once per (problem, slot); recording runs the step, so everything in flight finishes first
            torch.cuda.synchronize(step.dev)
            self.graphs[gkey] = step.capture(slot.q, slot.k, slot.v, self.w_post)
        cur.wait_event(self.copied[s])
        cur.wait_event(self.out_done)                           # the previous result has left the output buffers
        if self.use_graphs:
            self.graphs[gkey].replay()
            y = step.layer_out[-1] if step.n_post else step.hidden_out
        else:
            y = step.run(slot.q, slot.k, slot.v, self.w_post)
        self.consumed[s].record(cur)
        self.computed.record(cur)
        n = step.total_out
        with torch.cuda.stream(self.out_stream):
            self.out_stream.wait_event(self.computed)
            out_h[:n].copy_(y[:n], non_blocking=True)
            self.out_done.record(self.out_stream)
        return n

    def wait(self):
        torch.cuda.current_stream(self.step.dev).wait_event(self.out_done)
