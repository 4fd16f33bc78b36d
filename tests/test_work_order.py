"""The order in which the Newton-Schulz kernel hands out its work items, walked on the host with the scheduler's own
cursor (mona_work_order; no device needed).  The kernel cannot deadlock because every item comes after all items it
depends on - GEMM q of a matrix after every item of GEMM q - 1 of that matrix - whatever the launch shape and the
delay; a CTA pair sees an arbitrary increasing subsequence of the order and must decode it to the same items."""
import random

import pytest

from paper_2605_26842_b200 import binding

CASES = [  # (matrices, delay, items per phase)
    (1, 1, [1]),
    (1, 6, [6, 6, 12] * 5),                 # one matrix: most values of tau hold no item at all
    (7, 20, [6, 6, 12] * 5),                # delay larger than the chunk
    (93, 20, [6, 6, 12] * 5),               # the benchmark's 768 x 2048 expert chunk
    (93, 1, [6, 6, 12] * 5),
    (40, 3, [3, 3, 4] * 2 + [3]),           # a launch that ends in the middle of an iteration
    (5, 2, [1, 1, 2] * 5),
    (512, 7, [1, 1, 1] * 5),
    (3, 1024, [10, 10, 8]),
]


def reference_order(C, delay, items):
    """The definition, written out: tau ascending, then phase, then item; matrix = tau - delay * phase."""
    P = len(items)
    out = []
    for tau in range(C + delay * (P - 1)):
        for q in range(P):
            c = tau - delay * q
            if 0 <= c < C:
                out += [(c, q, t) for t in range(items[q])]
    return out


@pytest.mark.parametrize("C,delay,items", CASES)
def test_order_is_the_definition_and_respects_dependencies(C, delay, items):
    got = binding.work_order(C, delay, items)
    assert got == reference_order(C, delay, items)
    assert len(set(got)) == len(got) == C * sum(items)            # every item exactly once
    done = {}                                                       # (c, q) -> items seen so far
    for c, q, t in got:
        if q > 0:
            assert done.get((c, q - 1), 0) == items[q - 1], (c, q, t)     # the previous GEMM of this matrix is complete
        done[(c, q)] = done.get((c, q), 0) + 1


@pytest.mark.parametrize("C,delay,items", CASES)
def test_a_pair_decodes_its_subsequence_to_the_same_items(C, delay, items):
    full = binding.work_order(C, delay, items)
    for start, stride in ((0, 74), (73, 74), (5, 1000), (0, 2)):
        assert binding.work_order(C, delay, items, start=start, stride=stride) == full[start::stride]
    # irregular gaps, as the shared counter produces them: ask item by item with a fresh cursor up to each index
    rnd = random.Random(C * 1000 + delay)
    picks = sorted(rnd.sample(range(len(full)), min(20, len(full))))
    for idx in picks:
        assert binding.work_order(C, delay, items, start=idx, stride=len(full) + 1) == [full[idx]]


def test_bad_arguments_are_refused():
    for args in ((0, 1, [1]), (1, 0, [1]), (1, 1, []), (1, 1, [1] * 16)):
        with pytest.raises(binding.MonaError) as e:
            binding.work_order(*args, capacity=4)
        assert e.value.status == 1
    with pytest.raises(binding.MonaError):
        binding.work_order(2, 1, [1, 1], stride=0, capacity=4)
    assert binding.work_order(2, 1, [1, 1], start=100) == []       # beyond the last item: nothing, no error
