"""Discovery of decoding trees (Section "Discovering performant decoding trees" and its appendix).

The paper grows a sequence of trees T_1, T_2, ... by adding, at every step, the candidate node that raises the expected
acceptance length most, then picks the tree size whose measured throughput is best for the deployment at hand.
Host-side logic, no GPU arithmetic: the acceptance statistics come in as a function (the paper estimates them on a
corpus; the benchmarks here pass a synthetic model), the step latencies come from timing the engine.

A tree is a `parent` list in the library's row order: row 0 is the root, parent[i] < i, rows sorted by (depth, rank
path); the rank path (r_1..r_k) of a node says it is the r_k-th most likely child of the node with rank path
(r_1..r_{k-1}).
"""
import heapq
from typing import Callable, Dict, List, Sequence, Tuple

RankPath = Tuple[int, ...]


def accept_probability(path: RankPath, rank_prob: Callable[[int, int], float]) -> float:
    """Probability that the node with this rank path is accepted: every node on its path must be, and rank_prob(depth, r)
    is the chance that the r-th most likely token of the head at that depth is the right one given that its parent was."""
    p = 1.0
    for depth, r in enumerate(path, start=1):
        p *= rank_prob(depth, r)
    return p


def grow_trees(n_max: int, max_depth: int, rank_prob: Callable[[int, int], float], max_children: int = 64) -> List[List[RankPath]]:
    """T_1 .. T_n_max as lists of rank paths (the root excluded): T_n = T_{n-1} plus the eligible node of the highest
    acceptance probability.  A node is eligible when its parent and its next-more-likely sibling are in the tree
    (children are the top tokens in order, so rank r needs ranks 0..r-1).  The expected acceptance length of a tree is
    the sum of its nodes' probabilities, so this greedy choice is the one the paper describes: the node that raises
    the expected length most.  Ties: shallower first, then the smaller rank path."""
    heap: List[Tuple[float, int, RankPath]] = []

    def push(path: RankPath):
        if len(path) <= max_depth and path[-1] < max_children:
            heapq.heappush(heap, (-accept_probability(path, rank_prob), len(path), path))

    push((0,))
    chosen: List[RankPath] = []
    trees: List[List[RankPath]] = []
    while len(chosen) < n_max and heap:
        _, _, path = heapq.heappop(heap)
        chosen.append(path)
        trees.append(list(chosen))
        push(path[:-1] + (path[-1] + 1,))        # its next sibling becomes eligible
        push(path + (0,))                        # and its first child
    return trees


def to_parent_list(paths: Sequence[RankPath]) -> List[int]:
    """The library's tree description of a set of rank paths (closed under parents and earlier siblings)."""
    rows = sorted([()] + list(paths), key=lambda p: (len(p), p))
    index: Dict[RankPath, int] = {p: i for i, p in enumerate(rows)}
    return [-1] + [index[p[:-1]] for p in rows[1:]]


def rank_paths_of(parent: Sequence[int]) -> List[RankPath]:
    kids: Dict[int, int] = {}
    paths: List[RankPath] = [()] * len(parent)
    for i in range(1, len(parent)):
        r = kids.get(parent[i], 0)
        kids[parent[i]] = r + 1
        paths[i] = paths[parent[i]] + (r,)
    return paths


def expected_accept_length(parent: Sequence[int], rank_prob: Callable[[int, int], float]) -> float:
    """Expected number of accepted candidates per step: the accepted nodes form one path, so the expectation of its
    length is the sum over the nodes of their acceptance probabilities."""
    return sum(accept_probability(p, rank_prob) for p in rank_paths_of(parent)[1:])


def pick_tree_size(sizes: Sequence[int], expected_len: Callable[[int], float], step_seconds: Callable[[int], float], batch: int):
    """Throughput of every candidate size (tokens emitted per second = batch * (1 + expected accepted length) / step
    time) and the best one.  Returns (best_size, {size: tokens_per_second})."""
    table = {n: batch * (1.0 + expected_len(n)) / step_seconds(n) for n in sizes}
    return max(table, key=lambda n: (table[n], -n)), table
