"""Host logic of the grouped GEMM launches: the static tile schedule (longest-processing-time
assignment of work items to persistent CTAs / CTA pairs).  No GPU needed."""
import ctypes

import numpy as np
import pytest

from paper_1910_04732_b200 import build as B


@pytest.fixture(scope="module")
def b():
    B.build()
    from paper_1910_04732_b200 import binding
    binding.load_library()
    return binding


def loads(cost, unit_of, units):
    out = np.zeros(units)
    for c, u in zip(cost, unit_of):
        out[u] += c
    return out


def test_every_item_assigned_once_and_makespan_reported(b):
    rng = np.random.default_rng(0)
    cost = rng.uniform(1.0, 50.0, size=500)
    unit_of, ms, rr = b.plan_tile_schedule(cost, 74)
    assert len(unit_of) == 500 and min(unit_of) >= 0 and max(unit_of) < 74
    ld = loads(cost, unit_of, 74)
    assert np.isclose(ld.max(), ms)
    assert np.isclose(loads(cost, [i % 74 for i in range(500)], 74).max(), rr)
    assert ms <= rr + 1e-9
    # longest-processing-time guarantee: within 4/3 of the lower bound max(mean load, longest item)
    assert ms <= (4.0 / 3.0) * max(cost.sum() / 74, cost.max()) + 1e-9


def test_bert_forward_mix_is_balanced(b):
    # H' = X Q^T of one BERT-shaped layer on 74 CTA pairs: 240 tiles of 12 k-blocks, 48 tiles of 48
    cost = [12.0] * 192 + [12.0] * 48 + [48.0] * 48
    unit_of, ms, rr = b.plan_tile_schedule(cost, 74)
    assert rr == 84.0            # round-robin: 3 short tiles + 1 long one on 48 pairs
    assert ms == 72.0            # 48 + 2 x 12, or 6 x 12: the mean load is 70.05
    ld = loads(cost, unit_of, 74)
    assert ld.min() >= 60.0


def test_equal_costs_keep_list_order_round_robin(b):
    unit_of, ms, rr = b.plan_tile_schedule([5.0] * 20, 8)
    assert unit_of == [i % 8 for i in range(20)]
    assert ms == rr == 15.0


def test_edges_and_argument_checks(b):
    assert b.plan_tile_schedule([], 4) == ([], 0.0, 0.0)
    unit_of, ms, _ = b.plan_tile_schedule([3.0, 1.0], 148)
    assert unit_of == [0, 1] and ms == 3.0
    lib = b.load_library()
    one = (ctypes.c_double * 1)(1.0)
    assert lib.flop_plan_tile_schedule(one, 1, 0, None, None, None) == b.ERR_INVALID_ARG
    assert lib.flop_plan_tile_schedule(one, 1, 149, None, None, None) == b.ERR_INVALID_ARG
    assert lib.flop_plan_tile_schedule(one, 2049, 4, None, None, None) == b.ERR_INVALID_ARG
    assert lib.flop_plan_tile_schedule(None, 1, 4, None, None, None) == b.ERR_INVALID_ARG
    assert lib.flop_plan_tile_schedule(one, 1, 4, None, None, None) == b.OK


def test_round_robin_is_kept_when_it_is_within_three_per_cent_of_the_bound(b):
    # 740 equal tiles and 74 slightly longer ones on 74 units: round-robin gives 10 short + 1 long each, the optimum
    cost = [10.0] * 740 + [10.2] * 74
    unit_of, ms, rr = b.plan_tile_schedule(cost, 74)
    assert unit_of == [i % 74 for i in range(len(cost))]
    assert ms == rr
