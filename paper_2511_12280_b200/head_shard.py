"""One request over several GPUs: the heads of the merge layer are split across ranks.

Attention is independent per head (Sec. 3.2.1: A = softmax(Q K^T) is computed per
head; the importance score S_j sums the decider rows of every head), so rank r
runs the attention + importance kernels on its own heads only.  Select and
merge need full-width rows (the cosine of Sec. 3.2.2 is over the whole hidden
vector) and the complete S, so ONE exchange step sits between attention and
select:

  * the per-rank partial importance maps [sum V_b] fp32 are gathered and added
    in rank order (a fixed order: every rank holds the same bits, and so takes
    the same keep / merge decisions);
  * the per-rank slices of the post-attention states H~ [rows, D / G] are
    gathered into the full [rows, D] matrix in every rank's own memory.

Select and merge then run replicated on every rank.  A post-merge layer is
sharded the same way: the rank projects the full shortened X with the weight
rows of its own heads (three d3tom_linear calls), runs the ragged attention on
them, and the output slices are gathered again.

This module is host logic and marshalling only: slicing, the two gathers
(torch.distributed collectives on LOCAL buffers: NCCL on GPUs, gloo in the CPU
tests) and the order of the library calls.  The gathers land in local memory
before any kernel reads them; no kernel is ever handed another GPU's memory.
The paper has no multi-GPU part: this is an extension, built and tested on CPU
ranks and on one GPU that plays the ranks one after the other.
"""
from __future__ import annotations

from typing import List, Sequence, Tuple

import torch
import torch.distributed as dist


def shard_heads(n_heads: int, rank: int, world_size: int) -> Tuple[int, int]:
    """Heads [h0, h1) owned by ``rank``: equal contiguous blocks (n_heads must divide evenly, as the gathered
    slices have one width)."""
    if world_size <= 0 or not (0 <= rank < world_size):
        raise ValueError("bad rank / world size")
    if n_heads % world_size != 0:
        raise ValueError("the number of heads must be a multiple of the number of ranks")
    per = n_heads // world_size
    return rank * per, (rank + 1) * per


def slice_heads(x: torch.Tensor, h0: int, h1: int) -> torch.Tensor:
    """[rows, H, dh] -> the packed copy [rows, h1 - h0, dh] of one rank's heads."""
    return x[:, h0:h1].contiguous()


def slice_qkv_weights(w_qkv: torch.Tensor, n_heads: int, head_dim: int, h0: int, h1: int):
    """Rows of W_q, W_k, W_v ([3D, D], row o = output feature o) that produce heads [h0, h1): three [D_local, D]
    matrices (column-parallel projection: the input stays full width)."""
    D = n_heads * head_dim
    lo, hi = h0 * head_dim, h1 * head_dim
    return tuple(w_qkv[i * D + lo:i * D + hi].contiguous() for i in range(3))


def combine_importance(partials: Sequence[torch.Tensor]) -> torch.Tensor:
    """Sum of the per-rank partial importance maps, added in rank order."""
    total = partials[0].clone()
    for p in partials[1:]:
        total += p
    return total


def combine_hidden(slices: Sequence[torch.Tensor]) -> torch.Tensor:
    """[rows, D_local] per rank (rank r = heads r*H/G ..) -> [rows, D]: heads are contiguous along the row, so the
    slices are laid side by side in rank order."""
    return torch.cat(list(slices), dim=1).contiguous()


def gather_all(t: torch.Tensor) -> List[torch.Tensor]:
    """Every rank's copy of ``t`` (same shape on all ranks), in rank order, in local memory."""
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [t]
    out = [torch.empty_like(t) for _ in range(dist.get_world_size())]
    dist.all_gather(out, t.contiguous())
    return out


def exchange_importance(partial: torch.Tensor) -> torch.Tensor:
    return combine_importance(gather_all(partial))


def exchange_hidden(local_slice: torch.Tensor) -> torch.Tensor:
    return combine_hidden(gather_all(local_slice))


class HeadShardedStep:
    """One merge-layer step on the heads [h0, h1) of this rank.

    ``local`` is a MergeLayerStep built for H_local heads (its context's scratch is sized for them) and used for the
    attention calls; ``full`` is a MergeLayerStep built for all H heads and used for select, merge and the dense
    layers (their rows are full width).  Both get the same problem description.  ``gather`` turns this rank's tensor
    into the list of every rank's tensor (``gather_all`` by default; a test that plays several ranks on one device
    passes its own)."""

    def __init__(self, local, full, n_heads: int, head_dim: int, h0: int, h1: int, gather=gather_all):
        self.local, self.full = local, full
        self.H, self.dh, self.h0, self.h1 = n_heads, head_dim, h0, h1
        self.D, self.D_local = n_heads * head_dim, (h1 - h0) * head_dim
        self.gather = gather
        n_rows = full.attn_out.shape[0]
        dev, dt = full.dev, full.dtype
        self.q_l = torch.empty(n_rows, self.D_local, dtype=dt, device=dev)
        self.k_l = torch.empty_like(self.q_l)
        self.v_l = torch.empty_like(self.q_l)
        self.o_l = torch.empty_like(self.q_l)

    def set_problem(self, n_visual, n_prompt, n_resp, decider_pos, keep_count):
        pr = self.full.make_problem(n_visual, n_prompt, n_resp, decider_pos, keep_count)
        self.full.use_problem(pr)
        self.local.use_problem(pr)

    # ---- the two halves of the step, split at the exchange
    def attention_local(self, q_local, k_local, v_local):
        """Attention + importance over this rank's heads: (H~ slice [total, D_local], partial importance [sum V])."""
        lc = self.local
        lc.attn_importance(q_local, k_local, v_local)
        return lc.attn_out[:lc.total], lc.importance[:lc.total_vis]

    def select_and_merge(self, hidden_full, importance_full):
        """Replicated on every rank: needs the complete importance map and full-width rows."""
        fl = self.full
        fl.importance[:fl.total_vis].copy_(importance_full)
        fl.attn_out[:fl.total].copy_(hidden_full)
        fl.select()
        fl.merge()
        return fl.hidden_out[:fl.total_out]

    def post_layer_local(self, x_full, w_qkv_local):
        """A post-merge layer on this rank's heads: column-parallel projection of the full-width rows, ragged
        attention, returns the output slice [total_out, D_local]."""
        fl, n = self.full, self.full.total_out
        wq, wk, wv = w_qkv_local
        ctx = self.local.ctx
        ctx.d3tom_linear(x_full, wq, None, n, self.D, self.D_local, self.q_l)
        ctx.d3tom_linear(x_full, wk, None, n, self.D, self.D_local, self.k_l)
        ctx.d3tom_linear(x_full, wv, None, n, self.D, self.D_local, self.v_l)
        ctx.d3tom_attn_varlen(self.q_l, self.k_l, self.v_l, fl.cu_out, fl.nB, n, fl.max_out, fl.scale, self.o_l)
        return self.o_l[:n]

    def run(self, q_local, k_local, v_local, w_post_local=()):
        """The whole step; returns the full-width output of the last layer (identical on every rank)."""
        h_slice, s_part = self.attention_local(q_local, k_local, v_local)
        hidden = combine_hidden(self.gather(h_slice))
        importance = combine_importance(self.gather(s_part))
        x = self.select_and_merge(hidden, importance)
        for w_l in w_post_local:
            x = combine_hidden(self.gather(self.post_layer_local(x, w_l)))
        return x
