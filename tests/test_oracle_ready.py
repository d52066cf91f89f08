"""Pins of the readiness model (Section 4.3, asynchronous swap-in): expected values below are worked by hand."""
import itertools

from oracle.ready import InFlight


def test_worked_example():
    m = InFlight()
    reqs = [[1, 2, 3], [4, 5], [], [3, 9]]
    assert m.ready(reqs) == [True, True, True, True]          # nothing in flight
    m.mark([3, 4], "a")
    assert m.ready(reqs) == [False, False, True, False] and m.count() == 2
    m.mark([9], "b")
    m.complete("a")
    assert m.ready(reqs) == [True, True, True, False] and m.count() == 1
    m.complete("b")
    assert m.ready(reqs) == [True, True, True, True] and m.count() == 0


def test_block_marked_again_follows_the_newer_copy():
    m = InFlight()
    m.mark([7], "old")
    m.mark([7], "new")
    m.complete("old")
    assert m.ready([[7]]) == [False]       # the newer copy has not landed yet
    m.complete("new")
    assert m.ready([[7]]) == [True]


def test_ready_is_disjointness_for_every_subset():
    blocks = [0, 1, 2, 3]
    reqs = [[0], [1, 2], [2, 3], [0, 3], []]
    for k in range(len(blocks) + 1):
        for pending in itertools.combinations(blocks, k):
            m = InFlight()
            m.mark(pending, "t")
            want = [not (set(r) & set(pending)) for r in reqs]
            assert m.ready(reqs) == want
            assert m.count() == len(pending)
