"""Static candidate-tree topologies.

A tree is a `parent` list: row 0 is the root (parent -1, the committed-but-unprocessed token), every
other row is one candidate token, parent[i] < i, rows ordered by (depth, rank path).  The committed
JSON files under synth/trees/ are the authority; `grow_tree` documents how they were made: greedy
growth by expected acceptance (Section "Discovering performant decoding trees" of the paper) under
a synthetic acceptance model instead of a text corpus.
"""
import json
import os
from typing import List, Sequence

_DIR = os.path.join(os.path.dirname(os.path.abspath(__file__)), "trees")


ALPHA = (0.70, 0.55, 0.45, 0.38)     # synthetic acceptance model: chance that head j's list holds the right token at all
BETA = 0.45                          # ... and how fast it falls with the rank inside the list


def node_score(path: Sequence[int], alpha=ALPHA, beta=BETA, normalised=False) -> float:
    """Acceptance score of the candidate with rank path (r_1..r_k): prod_j alpha[j] * beta**r_j; `normalised` makes every
    factor a probability over the ranks (times 1 - beta), so that the scores of a tree add up to an expected length."""
    s = 1.0
    for j, r in enumerate(path):
        s *= alpha[j] * beta ** r * ((1.0 - beta) if normalised else 1.0)
    return s


def rank_paths(parent: Sequence[int]) -> List[tuple]:
    """Rank path of every row (the root's is empty): index among the siblings, level by level."""
    kids = {}
    paths = [()] * len(parent)
    for i in range(1, len(parent)):
        r = kids.get(parent[i], 0)
        kids[parent[i]] = r + 1
        paths[i] = paths[parent[i]] + (r,)
    return paths


def grow_tree(n_candidates: int, caps: Sequence[int], alpha=ALPHA, beta=BETA, normalised=False) -> List[int]:
    """Greedy tree growth: repeatedly add the eligible node with the largest acceptance score.

    A candidate with rank path (r_1..r_k) scores prod_j alpha[j] * beta**r_j.  A node is eligible when
    its parent and its previous sibling are in the tree, r_k < caps[k-1] and k <= len(caps).
    Ties go to the shallower node, then to the lexicographically smaller rank path.
    """
    def score(path):
        return node_score(path, alpha, beta, normalised)

    chosen = {()}
    while len(chosen) - 1 < n_candidates:
        best = None
        for p in chosen:
            if len(p) >= len(caps):
                continue
            r = 0
            while p + (r,) in chosen:
                r += 1
            if r >= caps[len(p)]:
                continue
            c = p + (r,)
            key = (-score(c), len(c), c)
            if best is None or key < best[0]:
                best = (key, c)
        if best is None:
            raise ValueError("tree cannot grow to the requested size under these caps")
        chosen.add(best[1])
    rows = sorted(chosen, key=lambda p: (len(p), p))
    index = {p: i for i, p in enumerate(rows)}
    return [-1] + [index[p[:-1]] for p in rows[1:]]


def chain_tree(depth: int) -> List[int]:
    """Root followed by a single chain of `depth` candidates."""
    return [-1] + list(range(depth))


def star_tree(n_children: int) -> List[int]:
    """Root with n_children depth-1 candidates."""
    return [-1] + [0] * n_children


def load_tree(name: str) -> List[int]:
    with open(os.path.join(_DIR, name + ".json")) as f:
        return json.load(f)["parent"]


def _write_committed():
    os.makedirs(_DIR, exist_ok=True)
    for name, n, caps in (("tree15_d3", 15, (4, 2, 1)), ("tree63_d4", 63, (10, 10, 10, 10))):
        parent = grow_tree(n, caps)
        with open(os.path.join(_DIR, name + ".json"), "w") as f:
            json.dump({"name": name, "n_candidates": n, "caps": list(caps), "parent": parent}, f)
            f.write("\n")


if __name__ == "__main__":
    _write_committed()
