"""Pins for the pipeline-planning oracle (Section 3.4): the paper's own example, the constraints of Eq. 6,
closed forms, and brute force over every admissible order on tiny instances."""
import itertools

import numpy as np
import pytest

from oracle import planner


def all_orders(B):
    """Every interleaving of the experts' ascending-width queues (constraint 6b)."""
    queues = planner.load_items(B)
    tags = [j for j, q in queues.items() for _ in q]
    for perm in set(itertools.permutations(tags)):
        pos = {j: 0 for j in queues}
        out = []
        for j in perm:
            out.append(queues[j][pos[j]])
            pos[j] += 1
        yield out


def test_paper_example_reuse_counts_and_queue():
    # Section 3.4: three requests on one expert, one at INT2 and two at INT3: the INT2 segment is read by all
    # three, the INT3 segment by two; nothing of a higher width is loaded
    B = [[0, 0, 0], [1, 2, 0]]
    assert planner.load_items(B) == {1: [(1, 0), (1, 1)]}
    assert planner.frequency(B, (1, 0)) == 3 and planner.frequency(B, (1, 1)) == 2
    assert planner.hebf_order(B) == [(1, 0), (1, 1)]


def test_intermediate_segments_are_loaded_even_without_their_own_requests():
    B = [[0, 0, 2]]                     # only width index 2 requested: segments 0, 1, 2 are all needed
    assert planner.id_order(B) == [(0, 0), (0, 1), (0, 2)]
    span, wait = planner.simulate(B, planner.id_order(B), [1.0, 2.0, 4.0], [0.5, 0.5, 0.5])
    assert span == pytest.approx(7.0 + 2 * 0.5) and wait == pytest.approx(7.0)


def test_hebf_picks_the_hottest_head_and_keeps_widths_ascending():
    B = [[1, 0, 0], [2, 3, 0], [0, 0, 4]]
    order = planner.hebf_order(B)
    # heads: (0,0) f=1, (1,0) f=5, (2,0) f=4 -> (1,0); then (1,1) f=3 vs (2,0) f=4 -> (2,0); (2,1) f=4; (2,2) f=4; (1,1) f=3; (0,0)
    assert order == [(1, 0), (2, 0), (2, 1), (2, 2), (1, 1), (0, 0)]
    seen = set()
    for j, k in order:
        assert k == 0 or (j, k - 1) in seen
        seen.add((j, k))
    assert sorted(order) == sorted(planner.id_order(B))
    # ties go to the lower expert id
    assert planner.hebf_order([[1, 0], [1, 0]]) == [(0, 0), (1, 0)]


def test_simulation_closed_forms():
    B = [[2, 1], [0, 3]]
    order = planner.id_order(B)
    comp = 2 * 0.3 + 1 * 0.4 + 3 * 0.4
    # free loading: the compute queue never waits
    span, wait = planner.simulate(B, order, [0.0, 0.0], [0.3, 0.4])
    assert span == pytest.approx(comp) and wait == 0.0
    # free compute: the makespan is the I/O queue
    span, wait = planner.simulate(B, order, [1.0, 2.0], [0.0, 0.0])
    assert span == pytest.approx(1.0 + 2.0 + 1.0 + 2.0)
    # makespan = total compute + total wait whenever the last item computes (Eq. 6c summed over the queue)
    span, wait = planner.simulate(B, order, [1.0, 2.0], [0.3, 0.4])
    assert span == pytest.approx(comp + wait)
    # lower bounds: no order beats the I/O queue length plus the last compute, nor the first load plus all compute
    for o in all_orders(B):
        s, _ = planner.simulate(B, o, [1.0, 2.0], [0.3, 0.4])
        assert s >= 6.0 - 1e-12 and s >= 1.0 + comp - 1e-12


def test_order_violating_constraint_6b_is_rejected():
    with pytest.raises(AssertionError):
        planner.simulate([[1, 1]], [(0, 1), (0, 0)], [1.0, 1.0], [1.0, 1.0])


@pytest.mark.parametrize("seed", range(12))
def test_hebf_against_brute_force_on_tiny_instances(seed):
    """Brute force over every admissible order: HEBF is never better than the optimum (sanity of the simulator)
    and, on these compute-heavy instances, never worse than the sequential ID order and within 25 % of optimal."""
    r = np.random.default_rng(seed)
    E, K = 3, 3
    B = r.integers(0, 4, size=(E, K)).tolist()
    if not planner.load_items(B):
        B[0][0] = 1
    t_io = [1.0, 1.5, 2.5]
    t_comp = [1.2, 1.3, 1.5]
    best = min(planner.simulate(B, o, t_io, t_comp)[0] for o in all_orders(B))
    hebf = planner.simulate(B, planner.hebf_order(B), t_io, t_comp)[0]
    seq = planner.simulate(B, planner.id_order(B), t_io, t_comp)[0]
    assert hebf >= best - 1e-12
    assert hebf <= seq + 1e-12
    assert hebf <= 1.25 * best


def test_budget_step_releases_high_widths_first_and_respects_the_budget():
    seg = lambda l, e, k: (l, e, k, [10, 5, 20][k])
    resident = [seg(0, 0, 0), seg(0, 0, 1), seg(0, 0, 2), seg(0, 1, 0), seg(0, 1, 1)]     # 50 bytes
    need = [seg(1, 0, 0), seg(1, 0, 1)]                                                # 15 bytes
    # enough room: nothing is released
    res, loads, ev = planner.budget_step(resident, need, 70)
    assert ev == [] and loads == need and sum(b for *_, b in res) == 65
    # 60 bytes: 5 must go -> the highest width segment (20 bytes) is released first
    res, loads, ev = planner.budget_step(resident, need, 60)
    assert ev == [seg(0, 0, 2)] and sum(b for *_, b in res) <= 60
    # 30 bytes: all high widths, then the width-1 segments, then base segments until it fits
    res, loads, ev = planner.budget_step(resident, need, 30)
    assert ev[:3] == [seg(0, 0, 2), seg(0, 0, 1), seg(0, 1, 1)] and sum(b for *_, b in res) <= 30
    assert all(x in res for x in need)
    # segments the layer needs and already holds are neither reloaded nor released
    res, loads, ev = planner.budget_step(resident + [seg(1, 0, 0)], need, 60)
    assert loads == [seg(1, 0, 1)] and seg(1, 0, 0) not in ev
    with pytest.raises(AssertionError):
        planner.budget_step([], need, 10)


def test_larger_budget_never_loads_more():
    # replay a fixed request trace (4 layers, repeated 6 times) under growing budgets: bytes loaded fall monotonically,
    # and with room for everything each segment is loaded exactly once
    r = np.random.default_rng(5)
    sizes = [8, 4, 4, 16]
    trace = []
    for step in range(6):
        for layer in range(4):
            B = r.integers(0, 3, size=(4, 4)).tolist()
            trace.append([(layer, j, k, sizes[k]) for j, q in planner.load_items(B).items() for _, k in q])
    total = 4 * 4 * sum(sizes)
    loaded = []
    for budget in (4 * sum(sizes), 2 * 4 * sum(sizes), total):
        resident, n = [], 0
        for need in trace:
            resident, loads, _ = planner.budget_step(resident, need, budget)
            assert sum(b for *_, b in resident) <= budget
            n += sum(b for *_, b in loads)
        loaded.append(n)
    assert loaded[0] >= loaded[1] >= loaded[2]
    assert loaded[2] == sum(x[3] for x in {x for need in trace for x in need})
