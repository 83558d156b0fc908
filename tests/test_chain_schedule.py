"""Host logic of the chained launches: the queue the persistent CTA pairs draw their tiles from.  What makes
the device-side waits safe is a property of this order (every stage-0 tile before every stage-1 tile), so it is
checked here, without a GPU."""
import numpy as np
import pytest

from paper_1910_04732_b200 import build as B


@pytest.fixture(scope="module")
def b():
    B.build()
    from paper_1910_04732_b200 import binding
    binding.load_library()
    return binding


def test_stage_order_key_order_and_every_item_once(b):
    rng = np.random.default_rng(1)
    n = 1500
    stage = rng.integers(0, 2, size=n)
    key = rng.integers(0, 50, size=n)
    pos = b.plan_chain_queue(stage, key)
    assert sorted(pos) == list(range(n))                                   # a permutation
    order = np.argsort(pos)
    st, ky = stage[order], key[order]
    first_late = np.nonzero(st == 1)[0].min()
    assert np.all(st[:first_late] == 0) and np.all(st[first_late:] == 1)     # all of stage 0, then all of stage 1
    for s in (0, 1):
        k = ky[st == s]
        assert np.all(np.diff(k) >= 0)                                      # inside a stage: by key
        idx = order[st == s]
        same = np.diff(k) == 0
        assert np.all(np.diff(idx)[same] > 0)                               # ties keep list order


def test_small_and_bad_arguments(b):
    assert b.plan_chain_queue([1, 0, 0], [0, 5, 1]) == [2, 1, 0]
    lib = b.load_library()
    assert lib.flop_plan_chain_queue(None, None, 3, None) == b.ERR_INVALID_ARG
    assert lib.flop_plan_chain_queue(None, None, 0, None) == b.OK
    assert lib.flop_plan_chain_queue(None, None, 4000, None) == b.ERR_INVALID_ARG
