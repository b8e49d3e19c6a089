"""Tree discovery (Section "Discovering performant decoding trees"): the greedy growth against brute force over all
valid trees of small sizes, the expected length against exhaustive enumeration of the acceptance outcomes, and the
committed benchmark trees."""
import itertools

from paper_2402_05109_b200.tree_search import (grow_trees, to_parent_list, expected_accept_length, accept_probability,
                                                rank_paths_of, pick_tree_size)
from synth import load_tree, ALPHA, BETA


def model(depth, r):                       # the synthetic acceptance model of the benchmarks, normalised over the ranks
    return ALPHA[depth - 1] * (1.0 - BETA) * BETA ** r


def raw_model(depth, r):                   # the unnormalised scores the committed trees were grown with
    return ALPHA[depth - 1] * BETA ** r


def valid_trees(n, max_depth, width):
    """Every set of n rank paths closed under parents and earlier siblings (brute force)."""
    universe = [p for k in range(1, max_depth + 1) for p in itertools.product(range(width), repeat=k)]
    for combo in itertools.combinations(universe, n):
        s = set(combo)
        if all((len(p) == 1 or p[:-1] in s) and (p[-1] == 0 or p[:-1] + (p[-1] - 1,) in s) for p in combo):
            yield combo


def test_greedy_growth_maximises_expected_length():
    trees = grow_trees(5, 3, model, max_children=3)
    for n in range(1, 6):
        best = max(sum(accept_probability(p, model) for p in t) for t in valid_trees(n, 3, 3))
        got = sum(accept_probability(p, model) for p in trees[n - 1])
        assert abs(got - best) < 1e-12, (n, got, best)
        assert trees[n - 1][:n - 1] == trees[n - 2] if n > 1 else True          # nested: T_n = T_{n-1} + one node


def test_expected_length_against_outcome_enumeration():
    """Draw, for every depth, which rank (or none) is the right token; the accepted length of a tree is the depth of the
    deepest node whose whole path was drawn.  Sum over all outcomes = closed form."""
    parent = to_parent_list(grow_trees(9, 3, model, max_children=4)[-1])
    paths = set(rank_paths_of(parent)[1:])
    R = 5                                                       # ranks 0..R-1 explicit, "none of them" as the rest
    exp = 0.0
    for draw in itertools.product(range(R + 1), repeat=3):      # draw[k] = right rank at depth k+1, R = not in the list
        prob, length = 1.0, 0
        for k, r in enumerate(draw, start=1):
            prob *= (1.0 - sum(model(k, q) for q in range(R))) if r == R else model(k, r)
        path = ()
        for k, r in enumerate(draw, start=1):
            if r == R or path + (r,) not in paths:
                break
            path += (r,)
            length = k
        exp += prob * length
    assert abs(exp - expected_accept_length(parent, model)) < 1e-12


def test_committed_trees_are_the_greedy_trees_of_the_synthetic_model():
    for name, n, depth, cap in (("tree15_d3", 15, 3, None), ("tree63_d4", 63, 4, 10)):
        parent = load_tree(name)
        if cap is None:                                         # per-level caps (4, 2, 1): grow with a rank limit per depth
            capped = lambda d, r: raw_model(d, r) if r < (4, 2, 1)[d - 1] else 0.0
            grown = [p for p in grow_trees(40, depth, capped, max_children=4) if True][-1]
            grown = [p for p in grown if accept_probability(p, capped) > 0][:n]
        else:
            grown = grow_trees(n, depth, raw_model, max_children=cap)[-1]
        assert to_parent_list(grown) == parent, name
        assert rank_paths_of(parent)[1:] == sorted(grown, key=lambda p: (len(p), p))


def test_pick_tree_size_prefers_small_trees_when_steps_get_expensive():
    trees = grow_trees(63, 4, model)
    elen = lambda n: expected_accept_length(to_parent_list(trees[n - 1]), model) if n else 0.0
    sizes = [0, 3, 7, 15, 31, 63]
    cheap = lambda n: 1.0 + 0.001 * n          # memory-bound: extra rows are almost free -> the largest tree wins
    dear = lambda n: 1.0 + 0.05 * n            # compute-bound: every row costs -> a smaller tree wins
    assert pick_tree_size(sizes, elen, cheap, 1)[0] == 63
    assert pick_tree_size(sizes, elen, dear, 8)[0] < 63
    lens = [elen(n) for n in sizes]
    assert all(b > a for a, b in zip(lens, lens[1:]))       # more nodes, longer expected acceptance
