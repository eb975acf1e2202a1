"""Parity of the CUDA path with the CPU oracle on the benchmark configurations
(through the C ABI, on a B200)."""
import numpy as np
import pytest
import torch

from paper_2511_12280_b200 import binding as B_
from paper_2511_12280_b200 import workload as wl

import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def configs():
    cache = {}

    def get(name):
        if name not in cache:
            cache[name] = wl.config(name)
        return cache[name]
    return get


@pytest.mark.parametrize("mode", [B_.AGG_MEAN, B_.AGG_SUM])
def test_c0_tiny_fp32(configs, mode):
    rep = pu.check_step(configs("C0"), mode=mode, full_attention=True)
    assert rep["attn"] < 1e-4


@pytest.mark.parametrize("mode", [B_.AGG_MEAN, B_.AGG_SUM])
def test_c1_llada_shape(configs, mode):
    pu.check_step(configs("C1"), mode=mode, full_attention=True)


def test_c1_reference_kernels_agree_with_oracle_too(configs):
    # the plain CUDA-core kernels are a second, independent GPU implementation
    pu.check_step(configs("C1"), full_attention=False, reference_kernels=True)


def test_c2_multicrop_with_post_layers(configs):
    # the configuration and launch shape the benchmark times.  Every output row of the merge-layer
    # attention and of the three post-merge layers is compared (the oracle needs about 7 s for this step
    # on 16 host threads)
    pu.check_step(configs("C2"), full_attention=True)


def test_c2_sum_mode(configs):
    pu.check_step(configs("C2"), mode=B_.AGG_SUM, full_attention=True, check_post=False)


def test_c4_batched_ragged(configs):
    # all eight requests in full (about 40 s of oracle time on 16 host threads)
    pu.check_step(configs("C4"), full_attention=True)


@pytest.mark.parametrize("s", [0, 1, 21, 42, 63])
def test_c3_schedule_steps(configs, s):
    w = configs("C3")
    T = w.T
    a_min, a_max = 2 * (1 - w.mean_keep_ratio) - 1, 1.0
    alpha = B_.d3tom_schedule_alpha(s, T, a_min, a_max)
    dec = w.step_deciders(s)
    # a step without deciders runs unmerged (Algorithm 1, else-branch)
    k = B_.d3tom_keep_count(w.n_visual[0], 1.0 - alpha) if len(dec[0]) else w.n_visual[0]
    pu.check_step(w, full_attention=True, decider_pos=dec, keep_count=[k])    # about 2.5 s of oracle time per step
