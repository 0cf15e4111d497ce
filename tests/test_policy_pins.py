"""Pins of the policy oracle (oracle/hg_policy.py) against hand-written expectations, so that the oracle the
host library is compared with is itself fixed by something other than the library: Algorithm 1's branches one
by one, the top-K rule (Section 4.3) on ties, NaN and short rows, and the position rule (Section 4.5)."""
import itertools
import math

from oracle import hg_policy as P

POST, PRE = P.POST_QK, P.PRE_QK


def test_algorithm_1_initial_state():
    assert P.feedback_scheduler_init(128) == (128, POST)
    assert P.feedback_scheduler_init(7) == (7, POST)


def test_algorithm_1_branch_by_branch():
    step = lambda k, s, tg, tc, tx: P.feedback_scheduler_step(k, s, tg, tc, tx, 128, 1024, 100)
    # T_cpu + T_tx <= T_gpu: increase K (either strategy; the boundary counts as hidden; K_max caps it)
    assert step(128, POST, 1.0, 0.5, 0.2) == (228, POST)
    assert step(128, POST, 1.0, 0.5, 0.5) == (228, POST)
    assert step(990, POST, 1.0, 0.1, 0.1) == (1024, POST)
    assert step(1024, POST, 1.0, 0.1, 0.1) == (1024, POST)
    assert step(300, PRE, 1.0, 0.2, 0.2) == (400, PRE)          # hidden while in Pre-QK^T: K grows, strategy stays
    # else, K > K_min: decrease K, never below K_min
    assert step(500, POST, 1.0, 0.9, 0.2) == (400, POST)
    assert step(150, POST, 1.0, 0.9, 0.2) == (128, POST)
    assert step(500, PRE, 1.0, 0.9, 0.2) == (400, PRE)
    # else, K == K_min: strategy <- Pre-QK^T, K untouched
    assert step(128, POST, 1.0, 0.9, 0.2) == (128, PRE)
    assert step(128, PRE, 1.0, 0.9, 0.2) == (128, PRE)
    # the sum decides, not either term alone
    assert step(128, POST, 1.0, 0.6, 0.6) == (128, PRE)
    assert step(128, POST, 1.0, 0.0, 1.0000001) == (128, PRE)


def test_latencies_around_the_balance_point_do_not_flip_the_strategy_back_and_forth():
    """CPU stage alternately just hidden and just exposed: K moves by one step around its value, and the
    strategy changes at most once over the whole run (Post -> Pre, at K_min)."""
    for k0, strat0 in ((128, POST), (128, PRE), (528, POST)):
        k, s = k0, strat0
        flips, ks = 0, []
        for i in range(200):
            t_cpu = 0.79 if i % 2 == 0 else 0.81
            k2, s2 = P.feedback_scheduler_step(k, s, 1.0, t_cpu, 0.2, 128, 1024, 100)
            flips += s2 != s
            k, s = k2, s2
            ks.append(k)
        assert flips <= 1
        assert max(ks) - min(ks) <= 100 and all(128 <= x <= 1024 for x in ks)
    # and a cost model in which Post-QK^T is far more expensive than Pre-QK^T (the measured case: 13 ms against
    # 0.4 ms at K_min): once in Pre-QK^T the policy stays there and K climbs to where the CPU stage stops hiding
    k, s = P.feedback_scheduler_init(128)
    seen = []
    for _ in range(60):
        t_cpu = 13.0 if s == POST else 0.4 * k / 128
        k, s = P.feedback_scheduler_step(k, s, 2.0, t_cpu, 0.2, 128, 1024, 128)
        seen.append((k, s))
    assert seen[0] == (128, PRE) and all(st == PRE for _, st in seen)
    assert {kk for kk, _ in seen[10:]} == {512, 640}            # 0.4 * K / 128 + 0.2 <= 2.0 holds up to K = 576


def test_topk_rule():
    # the K largest, reported in ascending index order
    assert P.topk([0.1, 5.0, -2.0, 3.0, 4.0], 2) == [1, 4]
    assert P.topk([0.1, 5.0, -2.0, 3.0, 4.0], 3) == [1, 3, 4]
    # ties go to the lower index
    assert P.topk([1.0, 2.0, 2.0, 2.0, 0.0], 2) == [1, 2]
    assert P.topk([7.0] * 6, 4) == [0, 1, 2, 3]
    # k larger than the row: everything that is a number; k = 0: nothing
    assert P.topk([3.0, 1.0, 2.0], 10) == [0, 1, 2]
    assert P.topk([3.0, 1.0, 2.0], 0) == []
    assert P.topk([], 5) == []
    # NaN is never selected; infinities order like numbers
    nan, inf = float("nan"), float("inf")
    assert P.topk([nan, 1.0, nan, 0.5], 3) == [1, 3]
    assert P.topk([nan, nan], 1) == []
    assert P.topk([-inf, 0.0, inf, 1.0], 2) == [2, 3]
    assert P.topk([-inf, -inf, 0.0], 2) == [0, 2]
    # brute force on every small row: the chosen set has the k largest values, smallest indices among equals
    for row in itertools.product([0.0, 1.0, 2.0], repeat=5):
        for k in range(0, 6):
            got = P.topk(list(row), k)
            assert got == sorted(got) and len(got) == min(k, 5)
            rest = [i for i in range(5) if i not in got]
            for i in got:
                for j in rest:
                    assert row[i] > row[j] or (row[i] == row[j] and i < j)


def test_position_rule():
    # the first `sinks` and the last `window` tokens, sinks first, at most k, ascending
    assert P.positions(100, 4, 8, 12) == [0, 1, 2, 3] + list(range(92, 100))
    assert P.positions(100, 4, 8, 6) == [0, 1, 2, 3, 98, 99]           # k cuts the window to its most recent part
    assert P.positions(100, 4, 8, 3) == [0, 1, 2]                      # k below the sinks
    assert P.positions(100, 4, 8, 500) == [0, 1, 2, 3] + list(range(92, 100))
    # sinks and window overlapping on a short context: no token twice
    assert P.positions(10, 4, 8, 100) == list(range(10))
    assert P.positions(3, 4, 1024, 100) == [0, 1, 2]
    assert P.positions(5, 0, 2, 9) == [3, 4]
    assert P.positions(5, 2, 0, 9) == [0, 1]
    assert P.positions(0, 4, 8, 9) == []
    assert P.positions(6, 4, 8, 0) == []
    for n, s, w, k in itertools.product(range(0, 9), range(0, 5), range(0, 5), range(0, 9)):
        got = P.positions(n, s, w, k)
        assert got == sorted(set(got)) and len(got) == min(k, min(n, s + w) if s + w <= n else n) and all(0 <= t < n for t in got)
        assert all(t < s or t >= n - w for t in got)
        assert math.isclose(len([t for t in got if t < s]), min(s, n, k))


def test_ranked_rule():
    # every head takes the same number of leading candidates: K, the host token count and the shortest list bound it
    assert P.ranked([[5, 3, 9, 1], [2, 8, 7, 0]], 3, 10) == [[5, 3, 9], [2, 8, 7]]
    assert P.ranked([[5, 3, 9, 1], [2, 8, -1, -1]], 3, 10) == [[5, 3], [2, 8]]        # the shorter list sets the count
    assert P.ranked([[5, 3, 9, 1]], 10, 10) == [[5, 3, 9, 1]]
    assert P.ranked([[5, 3, 9, 1]], 10, 2) == [[]]                                   # 5 is not a host token
    assert P.ranked([[1, 0, 9, 1]], 10, 2) == [[1, 0]]                               # an entry beyond the host rows ends the list
    assert P.ranked([[-1, 4]], 2, 10) == [[]]
    assert P.ranked([[4, 2], [1, 3]], 0, 10) == [[], []]
