"""A host-side model of the split-K combine (pairwise exchanges along a fixed binary tree): for any number
of segments and any order of arrival exactly one participant finishes with the sum of all partials, every
meeting place is used by exactly two participants and is left empty, and the association of the additions
(hence the rounding) does not depend on the order of arrival.  The device code follows the same walk."""
import itertools
import random

import numpy as np


def walk(nseg, my_seg, part, nodes, log):
    """One participant's walk; nodes maps meeting place (first segment of the right-hand node) -> value."""
    idx, n, level = my_seg, nseg, 0
    while n > 1:
        right = idx | 1
        if right < n:
            place = right << level
            log.setdefault(place, []).append(my_seg)
            if place not in nodes:
                nodes[place] = part
                return None                      # first: leaves its sum
            part = np.float32(part + nodes.pop(place))     # second: takes it, empties the node, moves up
        idx >>= 1
        n = (n + 1) >> 1
        level += 1
    return part


def reference_tree_sum(parts):
    """The fixed association: neighbours are added pairwise, level by level."""
    vals = [np.float32(p) for p in parts]
    while len(vals) > 1:
        nxt = [np.float32(vals[i] + vals[i + 1]) for i in range(0, len(vals) - 1, 2)]
        if len(vals) % 2:
            nxt.append(vals[-1])
        vals = nxt
    return vals[0]


def run(nseg, order, parts):
    nodes, log, done = {}, {}, []
    for s in order:
        r = walk(nseg, s, np.float32(parts[s]), nodes, log)
        if r is not None:
            done.append(r)
    assert len(done) == 1, "exactly one participant completes the root"
    assert not nodes, "every meeting place is empty again"
    assert all(len(v) == 2 for v in log.values()), "two participants per meeting place"
    assert all(1 <= place < nseg for place in log), "meeting places are rows of CTAs that start inside the row tile"
    assert len(log) == nseg - 1
    return done[0]


def test_all_orders_small():
    rng = np.random.Generator(np.random.PCG64(5))
    for nseg in range(1, 7):
        parts = rng.standard_normal(nseg).astype(np.float32) * np.float32(1e3)
        want = reference_tree_sum(parts)
        for order in itertools.permutations(range(nseg)):
            assert run(nseg, order, parts) == want


def test_random_orders_up_to_1024_segments():
    rnd = random.Random(7)
    rng = np.random.Generator(np.random.PCG64(6))
    for nseg in [2, 3, 5, 8, 9, 31, 32, 33, 100, 148, 511, 1000, 1024]:
        parts = (rng.standard_normal(nseg) * 10.0 ** rng.integers(-3, 4, nseg)).astype(np.float32)
        want = reference_tree_sum(parts)
        for _ in range(5):
            order = list(range(nseg))
            rnd.shuffle(order)
            assert run(nseg, order, parts) == want       # bit-identical whatever the order of arrival
