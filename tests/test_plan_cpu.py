"""schedules.plan_rounds: every plan it makes is a legal regrouping of the schedule."""
import pytest

from paper_2609_23536_b200.schedules import peak_live, plan_rounds, sched


def _check(schedule, n, slots, rounds, max_group):
    acts = [x for g in rounds for x in g]
    assert sorted(acts) == sorted((a, l, m) for a, m in schedule for l in range(n))  # every action exactly once
    when = {x: r for r, g in enumerate(rounds) for x in g}
    order = {}
    for a, m in schedule:
        order.setdefault(a, []).append(m)
    live = [0] * n
    for r, g in enumerate(rounds):
        assert 1 <= len(g) <= max_group
        assert len({(a, l) for a, l, m in g}) == len(g) and len({(l, m) for a, l, m in g}) == len(g)
        for a, l, m in g:
            if a == "F" and l > 0:
                assert when[("F", l - 1, m)] < r            # a unit walks the linears in chain order
            if a == "dI":
                assert when[("F", l, m)] < r and (l == n - 1 or when[("dI", l + 1, m)] < r)
            if a == "dW":
                assert when[("dI", l, m)] < r
            i = order[a].index(m)
            if i:
                assert when[(a, l, order[a][i - 1])] < r    # each linear sees the microbatches in schedule order
        for a, l, m in g:
            if a == "F":
                live[l] += 1
                assert live[l] <= slots
        for a, l, m in g:  # released slots are available to later rounds only
            if a == "dW":
                live[l] -= 1


@pytest.mark.parametrize("M,w,d", [(4, 1, 0), (8, 3, 3), (8, 1, 2), (6, 2, 1), (32, 3, 3), (5, 5, 5)])
@pytest.mark.parametrize("n", [1, 3, 4])
@pytest.mark.parametrize("window,group", [(1, 4), (2, 4), (4, 8), (6, 8)])
def test_plans_are_legal(M, w, d, n, window, group):
    s = sched(M, w, d)
    slots = peak_live(s)
    rounds = plan_rounds(s, n, slots, group, window)
    _check(s, n, slots, rounds, group)
    if window == 1 and n == 1:
        assert [g[0] for g in rounds] == [(a, 0, m) for a, m in s]  # nothing to regroup: the schedule itself
    assert len(rounds) <= 3 * n * M


def test_plan_for_the_benchmark_schedule_groups_most_actions():
    s = sched(8, 3, 3)
    rounds = plan_rounds(s, 4, peak_live(s), 4, 4)
    assert len(rounds) <= 32 and sum(len(g) >= 3 for g in rounds) >= 20
    assert rounds[0] == [("F", 0, 0)] and rounds[1] == [("F", 1, 0), ("F", 0, 1)]  # warm-up wavefront
    with pytest.raises(RuntimeError):
        plan_rounds(s, 4, 2, 4, 4)  # two slots cannot hold this schedule


# ------------------------------------------------------------------------------------------ the library's own planner
@pytest.fixture(scope="module")
def qe():
    from paper_2609_23536_b200 import build

    build.build()
    from paper_2609_23536_b200 import binding

    return binding


def _actions(schedule, n):
    return [(a, l, m) for a, m in schedule for l in (range(n) if a == "F" else range(n - 1, -1, -1))]


@pytest.mark.parametrize("M,w,d", [(4, 1, 0), (8, 3, 3), (8, 1, 2), (6, 2, 1), (32, 3, 3)])
@pytest.mark.parametrize("n", [1, 3, 4])
@pytest.mark.parametrize("window,group", [(1, 4), (2, 4), (4, 8), (6, 8)])
def test_native_planner_makes_the_same_legal_plan(qe, M, w, d, n, window, group):
    """qe_plan_rounds (what qe_step_run uses; host logic, no device) against schedules.plan_rounds (what bench.py uses)."""
    s = sched(M, w, d)
    slots = peak_live(s)
    native = qe.plan_rounds(_actions(s, n), n, M, slots, window, group)
    _check(s, n, slots, native, group)
    assert native == plan_rounds(s, n, slots, group, window)


def test_native_planner_refuses_lists_without_a_plan(qe):
    s = sched(8, 3, 3)
    with pytest.raises(qe.QEError) as e:
        qe.plan_rounds(_actions(s, 4), 4, 8, 2, 4, 8)  # two slots cannot hold seven live tapes
    assert e.value.code == "ORDER"
    with pytest.raises(qe.QEError) as e:
        qe.plan_rounds([("dI", 0, 0), ("F", 0, 0), ("dW", 0, 0)], 1, 1, 1, 1, 8)  # dI before its forward, no look-ahead
    assert e.value.code == "ORDER"
    with pytest.raises(qe.QEError) as e:
        qe.plan_rounds([("F", 3, 0)], 1, 1, 1, 4, 8)
    assert e.value.code == "BAD_ARG"
    # (with look-ahead the forward is simply taken first)
    assert qe.plan_rounds([("dI", 0, 0), ("F", 0, 0), ("dW", 0, 0)], 1, 1, 1, 4, 8) == [[("F", 0, 0)], [("dI", 0, 0)], [("dW", 0, 0)]]
    # tapes alive before the list count against the pool
    assert len(qe.plan_rounds([("F", 0, 0), ("dI", 0, 0), ("dW", 0, 0)], 1, 1, 2, 4, 8, live_now=[1])) == 3
    with pytest.raises(qe.QEError):
        qe.plan_rounds([("F", 0, 0), ("dI", 0, 0), ("dW", 0, 0)], 1, 1, 2, 4, 8, live_now=[2])
