"""Host logic of the trajectory driver (Sec. 3.2.3 schedule, Sec. 3.2.1 decider set): no GPU needed."""
import numpy as np
import pytest

from oracle import d3tom_oracle as orc
from paper_2511_12280_b200 import trajectory as tr


def order(O, seed):
    return np.random.default_rng(seed).permutation(O).astype(np.int32)


@pytest.mark.parametrize("reversed_", [False, True])
def test_alphas_and_keep_counts_follow_the_schedule(reversed_):
    V, P, O, T = 2048, 64, 64, 32
    plan = tr.plan_schedule([V], [P], [order(O, 0)], T, 0.5, 1.0, tokens_per_step=2, reversed_=reversed_)
    assert len(plan) == T
    for s, p in enumerate(plan):
        assert p.alpha == pytest.approx(orc.schedule_alpha(s, T, 0.5, 1.0, reversed_), abs=1e-15)
        want = orc.keep_count(V, 1.0 - orc.schedule_alpha(s, T, 0.5, 1.0, reversed_)) if s > 0 else V
        assert p.keep_count == [want]
    # the first step has no decider and runs unmerged (Algorithm 1, else-branch)
    assert len(plan[0].decider_pos[0]) == 0 and plan[0].keep_count == [V]
    alphas = [p.alpha for p in plan]
    assert alphas == sorted(alphas, reverse=reversed_)
    assert np.mean(alphas) == pytest.approx(0.75)


def test_recent_deciders_are_the_tokens_of_the_previous_step():
    V, P, O, T, tps = 100, 7, 12, 6, 2
    od = order(O, 1)
    plan = tr.plan_schedule([V], [P], [od], T, 0.2, 0.8, tokens_per_step=tps, deciders="recent")
    seen = []
    for s, p in enumerate(plan):
        want = np.sort(od[(s - 1) * tps:s * tps]) + V + P if s else np.zeros(0, np.int32)
        assert np.array_equal(p.decider_pos[0], want)
        assert p.decider_pos[0].dtype == np.int32
        seen.extend(p.decider_pos[0].tolist())
    # every set is new; after T steps all but the last group have served as deciders
    assert len(seen) == len(set(seen)) == (T - 1) * tps
    assert set(seen) == set((od[:(T - 1) * tps] + V + P).tolist())


def test_all_deciders_grow_by_the_step_size_and_are_nested():
    V, P, O, T = 50, 3, 10, 10
    od = order(O, 2)
    plan = tr.plan_schedule([V], [P], [od], T, 0.0, 0.9, deciders="all")
    prev = set()
    for s, p in enumerate(plan):
        cur = set(p.decider_pos[0].tolist())
        assert len(cur) == s and prev <= cur
        assert list(p.decider_pos[0]) == sorted(cur)
        prev = cur


def test_unmerged_plan_keeps_every_visual_token_and_batches_are_per_request():
    plan = tr.plan_schedule([40, 90], [5, 6], [order(8, 3), order(8, 4)], 4, 0.5, 0.9, tokens_per_step=2, merged=False)
    assert all(p.keep_count == [40, 90] for p in plan)
    plan = tr.plan_schedule([40, 90], [5, 6], [order(8, 3), order(8, 4)], 4, 0.5, 0.9, tokens_per_step=2)
    for s, p in enumerate(plan[1:], start=1):
        a = orc.schedule_alpha(s, 4, 0.5, 0.9)
        assert p.keep_count == [orc.keep_count(40, 1 - a), orc.keep_count(90, 1 - a)]
        assert p.decider_pos[0].min() >= 45 and p.decider_pos[1].min() >= 96


def test_bad_arguments():
    with pytest.raises(ValueError):
        tr.plan_schedule([4], [1], [order(4, 0)], 2, 0.1, 0.2, deciders="none")
    with pytest.raises(ValueError):
        tr.plan_schedule([4], [1], [order(4, 0)], 0, 0.1, 0.2)
