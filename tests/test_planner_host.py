"""The library's host-side pipeline planner (Section 3.4) against the planning oracle: load orders and
budget steps item for item, simulated times to rounding.  Host code only: runs without a GPU."""
import numpy as np
import pytest

from oracle import planner
from paper_2504_15299_b200 import binding, build


@pytest.fixture(scope="module", autouse=True)
def lib():
    build.build_library()
    return binding.lib()


@pytest.mark.parametrize("seed", range(20))
def test_load_orders_and_simulation_match_the_oracle(seed):
    r = np.random.default_rng(seed)
    E, K = int(r.integers(1, 12)), int(r.integers(1, 5))
    B = (r.integers(0, 5, size=(E, K)) * (r.random((E, K)) < 0.6)).astype(int).tolist()
    t_io = (r.random(K) * 3 + 0.1).tolist()
    t_comp = (r.random(K) * 2 + 0.05).tolist()
    for policy, ref in ((binding.PLAN_HEBF, planner.hebf_order(B)), (binding.PLAN_BY_ID, planner.id_order(B))):
        got = binding.plan_load_order(B, policy)
        assert got == ref
        span, wait = binding.plan_simulate(B, got, t_io, t_comp)
        rs, rw = planner.simulate(B, ref, t_io, t_comp)
        assert span == pytest.approx(rs, rel=1e-13, abs=1e-13) and wait == pytest.approx(rw, rel=1e-13, abs=1e-13)


def test_mixtral_sized_layer_and_argument_checks():
    # the realised B of a 64-token Mixtral-shaped batch: 8 experts x 4 widths
    B = [[1, 3, 6, 5], [0, 4, 7, 4], [2, 2, 8, 6], [1, 5, 5, 3], [3, 3, 6, 6], [0, 2, 9, 4], [2, 4, 4, 5], [1, 3, 7, 5]]
    order = binding.plan_load_order(B)
    assert order == planner.hebf_order(B) and len(order) == 32
    with pytest.raises(binding.D2MoEError):
        binding.plan_simulate(B, [(0, 1), (0, 0)], [1.0] * 4, [1.0] * 4)          # a segment before the one below it
    with pytest.raises(binding.D2MoEError):
        binding.plan_load_order([[1, -1]])


@pytest.mark.parametrize("seed", range(10))
def test_budget_steps_match_the_oracle_over_a_trace(seed):
    r = np.random.default_rng(100 + seed)
    sizes = [8, 4, 4, 16]
    budget = int(r.integers(4, 9)) * 32
    res_o, res_c = [], []
    for step in range(12):
        layer = step % 3
        B = r.integers(0, 3, size=(4, 4)).tolist()
        need = [(layer, j, k, sizes[k]) for j, q in planner.load_items(B).items() for _, k in q]
        ro, lo, eo = planner.budget_step(res_o, need, budget)
        rc, lc, ec = binding.plan_budget_step(res_c, need, budget)
        assert (rc, lc, ec) == (ro, lo, eo)
        res_o, res_c = ro, rc
    with pytest.raises(binding.D2MoEError):
        binding.plan_budget_step([], [(0, 0, 0, 100)], 10)
