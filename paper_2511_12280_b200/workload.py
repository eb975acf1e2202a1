"""Seeded synthetic workloads shaped like the paper's LaViDa / LLaDA-8B runs.

This module only DRAWS inputs.  It holds none of the method's arithmetic (no
softmax, no top-k, no keep counts, no merging) and imports neither the CUDA
binding nor the CPU oracle, so both sides can consume the very same tensors.

The paper's own inputs (images, prompts, trained weights) are not available;
these tensors stand in for them with the published shapes: about a thousand
visual tokens per image crop (more for multi-crop images), 64-token prompts,
16-100 response tokens, hidden width 4096 = 32 heads x 128.

Recipe (one ``numpy.random.Generator(PCG64(seed))`` per workload, draws in
this order):
  1. ragged config only: per request |V|, |P|, decider count, keep ratio, from
     a generator of their own with the same seed;
  2. merge-layer weights W_q, W_k, W_v ~ N(0, 0.02), each [D, D] stored
     [out, in];
  3. per request: cluster centres ~ N(0,1) [n_clusters, D]; a uniform cluster
     id per visual token; X_vis = centre + 0.1 N(0,1); X_prompt, X_resp ~
     N(0,1); the decided (decider) positions = a uniform random subset of the
     response positions, ascending (for the step-schedule config a random
     decode ORDER instead); a uniform random 10 % "salient" subset of visual
     positions; one unit vector u_h per head;
  4. Q, K, V = X W^T in fp32; K rows of salient tokens get + 4 u_h per head;
     Q rows of decider tokens get + 4 u_h per head (so decider queries put
     extra mass on the salient keys);
  5. everything is rounded to the storage type (bf16 or fp32);
  6. post-merge layer weights W^l ~ N(0, 0.02), [3D, D], drawn last.
``block_inputs`` draws the tensors of the rest of a block (output projection,
feed-forward network) from a generator of its own.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np
import torch

SALIENT_FRACTION = 0.10
SALIENT_NORM = 4.0
CLUSTER_SIGMA = 0.1
WEIGHT_SIGMA = 0.02


@dataclass
class Workload:
    name: str
    dtype: str                      # "bf16" | "fp32" (storage type)
    H: int
    dh: int
    n_visual: List[int]
    n_prompt: List[int]
    n_resp: List[int]
    keep_ratio: List[float]         # r_b = 1 - alpha_b (constant-ratio configs)
    decider_pos: List[np.ndarray]   # per request, positions relative to request start, ascending
    salient: List[np.ndarray]       # per request, planted salient visual positions
    q_base: torch.Tensor            # [total, H, dh] storage dtype, WITHOUT the decider boost
    k: torch.Tensor                 # [total, H, dh]
    v: torch.Tensor                 # [total, H, dh]
    u: List[torch.Tensor]           # per request [H, dh] fp32 unit vectors
    w_post: List[torch.Tensor] = field(default_factory=list)   # each [3D, D] storage dtype
    # step-schedule config only
    T: int = 0
    decode_order: Optional[np.ndarray] = None     # permutation of response offsets 0..O-1
    mean_keep_ratio: float = 0.0

    @property
    def B(self):
        return len(self.n_visual)

    @property
    def D(self):
        return self.H * self.dh

    @property
    def seqlens(self):
        return [v + p + o for v, p, o in zip(self.n_visual, self.n_prompt, self.n_resp)]

    @property
    def cu_seqlens(self):
        return np.concatenate([[0], np.cumsum(self.seqlens)]).astype(np.int32)

    @property
    def cu_vis(self):
        return np.concatenate([[0], np.cumsum(self.n_visual)]).astype(np.int32)

    @property
    def torch_dtype(self):
        return torch.bfloat16 if self.dtype == "bf16" else torch.float32

    def cu_deciders(self, decider_pos=None):
        dp = self.decider_pos if decider_pos is None else decider_pos
        return np.concatenate([[0], np.cumsum([len(d) for d in dp])]).astype(np.int32)

    def q_for(self, decider_pos=None) -> torch.Tensor:
        """Q with the salience boost applied to the given decider rows (default:
        the workload's own decider lists).  Rounded to storage after the add."""
        dp = self.decider_pos if decider_pos is None else decider_pos
        q = self.q_base.to(torch.float32).clone()
        cu = self.cu_seqlens
        for b in range(self.B):
            rows = torch.as_tensor(np.asarray(dp[b], dtype=np.int64)) + int(cu[b])
            if len(rows):
                q[rows] += SALIENT_NORM * self.u[b][None]
        return q.to(self.torch_dtype)

    def step_deciders(self, s: int) -> List[np.ndarray]:
        """Step-schedule config: the decider list of decode-order step s = the
        response tokens decoded in steps 0..s-1 (one more per step)."""
        assert self.decode_order is not None
        b = 0
        off = self.n_visual[b] + self.n_prompt[b]
        return [np.sort(self.decode_order[:s]).astype(np.int32) + off]


def _normal(rng, shape, sigma=1.0):
    return (rng.standard_normal(size=shape, dtype=np.float32) * np.float32(sigma))


def make_workload(name, dtype, H, dh, seed, n_clusters, requests, post_layers=0, T=0, mean_keep_ratio=0.0) -> Workload:
    """requests: list of dicts with V, P, O, n_dec, r."""
    rng = np.random.Generator(np.random.PCG64(seed))
    D = H * dh
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    wq, wk, wv = (torch.from_numpy(_normal(rng, (D, D), WEIGHT_SIGMA)) for _ in range(3))
    qs, ks, vs, us, decs, sals = [], [], [], [], [], []
    decode_order = None
    for rq in requests:
        V, P, O, n_dec = rq["V"], rq["P"], rq["O"], rq["n_dec"]
        centres = _normal(rng, (n_clusters, D))
        ids = rng.integers(0, n_clusters, size=V)
        x_vis = centres[ids] + _normal(rng, (V, D), CLUSTER_SIGMA)
        x_prompt = _normal(rng, (P, D))
        x_resp = _normal(rng, (O, D))
        if T:
            decode_order = rng.permutation(O).astype(np.int32)
            dec = np.zeros(0, dtype=np.int32)
        else:
            dec = np.sort(rng.choice(O, size=n_dec, replace=False)).astype(np.int32) + (V + P)
        if V > 0:
            sal = np.sort(rng.choice(V, size=max(1, int(round(SALIENT_FRACTION * V))), replace=False)).astype(np.int32)
        else:
            sal = np.zeros(0, dtype=np.int32)       # a text-only request: nothing to merge
        u = _normal(rng, (H, dh))
        u /= np.linalg.norm(u, axis=1, keepdims=True)
        u = torch.from_numpy(u)
        x = torch.from_numpy(np.concatenate([x_vis, x_prompt, x_resp], axis=0)).to(tdt).to(torch.float32)
        q = (x @ wq.T).reshape(-1, H, dh)
        k = (x @ wk.T).reshape(-1, H, dh)
        v = (x @ wv.T).reshape(-1, H, dh)
        k[torch.as_tensor(sal.astype(np.int64))] += SALIENT_NORM * u[None]
        qs.append(q.to(tdt)); ks.append(k.to(tdt)); vs.append(v.to(tdt))
        us.append(u); decs.append(dec); sals.append(sal)
    w_post = [torch.from_numpy(_normal(rng, (3 * D, D), WEIGHT_SIGMA)).to(tdt) for _ in range(post_layers)]
    return Workload(
        name=name, dtype=dtype, H=H, dh=dh,
        n_visual=[r["V"] for r in requests], n_prompt=[r["P"] for r in requests], n_resp=[r["O"] for r in requests],
        keep_ratio=[float(r["r"]) for r in requests], decider_pos=decs, salient=sals,
        q_base=torch.cat(qs), k=torch.cat(ks), v=torch.cat(vs), u=us, w_post=w_post,
        T=T, decode_order=decode_order, mean_keep_ratio=mean_keep_ratio)


def block_inputs(seed: int, rows: int, D: int, m: int, dtype: str = "bf16"):
    """Inputs for the rest of a post-merge block (output projection + gated feed-forward network) at LLaDA-8B
    shapes (D = 4096, m = 12288) or smaller: x, residual ~ N(0,1) [rows, D]; W_o [D, D], W_gate_up [2m, D],
    W_down [D, m] ~ N(0, 0.02), one generator, drawn in this order, rounded to the storage type."""
    rng = np.random.Generator(np.random.PCG64(seed))
    tdt = torch.bfloat16 if dtype == "bf16" else torch.float32
    draw = lambda shape, sigma: torch.from_numpy(_normal(rng, shape, sigma)).to(tdt)
    return dict(x=draw((rows, D), 1.0), residual=draw((rows, D), 1.0), w_o=draw((D, D), WEIGHT_SIGMA),
                w_gate_up=draw((2 * m, D), WEIGHT_SIGMA), w_down=draw((D, m), WEIGHT_SIGMA))


def config(name: str) -> Workload:
    """The five benchmark configurations, C0..C4."""
    if name == "C0":   # tiny fp32 merge layer
        return make_workload("C0", "fp32", 4, 64, 0, 32, [dict(V=256, P=16, O=16, n_dec=8, r=0.25)])
    if name == "C1":   # LLaDA-8B-shaped merge layer
        return make_workload("C1", "bf16", 32, 128, 1, 128, [dict(V=1024, P=64, O=64, n_dec=32, r=0.10)])
    if name == "C2":   # multi-crop image + 3 post-merge layers
        return make_workload("C2", "bf16", 32, 128, 2, 128, [dict(V=4096, P=128, O=64, n_dec=32, r=0.25)], post_layers=3)
    if name == "C3":   # step-dependent schedule, T = 64
        return make_workload("C3", "bf16", 32, 128, 3, 128, [dict(V=2048, P=64, O=64, n_dec=0, r=0.25)],
                             post_layers=3, T=64, mean_keep_ratio=0.25)
    if name == "C4":   # batched ragged serving
        rng = np.random.Generator(np.random.PCG64(4))
        reqs = []
        for _ in range(8):
            reqs.append(dict(V=int(rng.integers(1024, 4097)), P=int(rng.integers(32, 257)), O=64,
                             n_dec=int(rng.integers(8, 49)), r=float(rng.choice([0.1, 0.25, 0.5]))))
        return make_workload("C4", "bf16", 32, 128, 4, 128, reqs, post_layers=3)
    raise KeyError(name)
