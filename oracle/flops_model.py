"""Theoretical cost model of the paper (Sec. 4.3 "Efficiency Analysis" and the
appendix "Detailed Theoretical FLOPs Analysis"), written out term by term.

TEST INFRASTRUCTURE ONLY.  It exists to pin the oracle's schedule and
step-structure readings against the totals the paper prints (efficiency
table and merge-layer ablation table): l* counts the full-length layers
before the merge layer, the first denoising step runs unmerged because its
decider set is empty, and the D3ToM-t rows follow a linear schedule over
alpha in [2*mean-1, 1].

The paper counts one multiply-accumulate as one operation; so does this file.
"""
from __future__ import annotations

from .d3tom_oracle import schedule_alpha

# fixed analysis configuration (appendix, "Scope of FLOPs Reporting")
D_MODEL, M_FFN, L_LAYERS, T_STEPS = 4096, 12288, 32, 32
N_VIS, N_PROMPT, N_OUT = 1000, 64, 64


def flops_attn(n, d=D_MODEL):
    """Self-attention part of Eq. layer_cost: 4 n d^2 + 2 n^2 d."""
    return 4 * n * d * d + 2 * n * n * d


def flops_ffn(n, d=D_MODEL, m=M_FFN):
    """FFN part of Eq. layer_cost: 3 n d m."""
    return 3 * n * d * m


def flops_layer(n, d=D_MODEL, m=M_FFN):
    return flops_attn(n, d) + flops_ffn(n, d, m)


def flops_baseline(N, d=D_MODEL, m=M_FFN, L=L_LAYERS, T=T_STEPS):
    """Eq. baseline_cost: T * L * FLOPs_layer(N)."""
    return T * L * flops_layer(N, d, m)


def flops_merge(alpha, V, d=D_MODEL):
    """Eq. merge_overhead: 2 a (1-a) |V|^2 d + a |V| d."""
    return 2 * alpha * (1 - alpha) * V * V * d + alpha * V * d


def flops_step(alpha, l_star, N, V, d=D_MODEL, m=M_FFN, L=L_LAYERS):
    """Eq. step_cost_new: l* full layers, the split layer (attention at N, FFN
    at N_m), L - l* - 1 layers at N_m, plus the merge overhead."""
    n_m = N - alpha * V
    return (l_star * flops_layer(N, d, m)
            + flops_attn(N, d) + flops_ffn(n_m, d, m)
            + (L - l_star - 1) * flops_layer(n_m, d, m)
            + flops_merge(alpha, V, d))


def flops_d3tom(alpha, l_star=3, V=N_VIS, P=N_PROMPT, O=N_OUT, d=D_MODEL, m=M_FFN, L=L_LAYERS, T=T_STEPS):
    """Constant ratio: the first step has no deciders and runs unmerged
    (Algorithm 1, else-branch), the other T-1 steps are merged."""
    N = V + P + O
    return L * flops_layer(N, d, m) + (T - 1) * flops_step(alpha, l_star, N, V, d, m, L)


def flops_d3tom_t(alpha_mean, l_star=3, V=N_VIS, P=N_PROMPT, O=N_OUT, d=D_MODEL, m=M_FFN, L=L_LAYERS, T=T_STEPS):
    """Linear schedule with mean ``alpha_mean`` spanning [2*mean-1, 1]: one
    unmerged step plus (T-1) merged steps costed at the schedule's average
    step cost."""
    N = V + P + O
    a_min, a_max = 2 * alpha_mean - 1, 1.0
    mean_step = sum(flops_step(schedule_alpha(s, T, a_min, a_max), l_star, N, V, d, m, L) for s in range(T)) / T
    return L * flops_layer(N, d, m) + (T - 1) * mean_step
