"""Accept-exercise mode: overlay a teacher continuation on one seeded root-to-node path.

plant[i] = -1 keeps the drafted token of row i; plant[i] >= 0 replaces it.  Planting the base
model's own greedy continuation on a depth-m path makes greedy acceptance accept (at least) m
candidates, so a schedule cycling m through 0..K exercises every accepted length.
"""
from typing import List, Sequence
from .rng import uniform_ids


def planted_length(step: int, b: int, K: int) -> int:
    return (step + b) % (K + 1)


def plant_row(parent: Sequence[int], teacher: Sequence[int], m: int, seed: int, step: int, b: int,
              vocab: int = 0) -> List[int]:
    """teacher[k-1] is the token the base model would emit k places after the root (k = 1..m+1).

    The chosen path gets teacher[0..m-1].  With vocab > 0 the other children of the path's rows (the root
    included) are overwritten with tokens that differ from the teacher's, so that exactly m candidates are
    accepted; this needs teacher[m] as well.
    """
    T = len(parent)
    depth = [0] * T
    for i in range(1, T):
        depth[i] = depth[parent[i]] + 1
    plant = [-1] * T
    nodes = [i for i in range(T) if depth[i] == m]
    node = nodes[int(uniform_ids(seed, 7000 + 131 * step + b, 1, len(nodes))[0])]
    on_path = set()
    while node != -1:
        on_path.add(node)
        if node != 0:
            plant[node] = int(teacher[depth[node] - 1])
        node = parent[node]
    if vocab > 0:
        rank = 0
        for i in range(1, T):
            rank = rank + 1 if parent[i] == parent[i - 1] else 0
            if i not in on_path and parent[i] in on_path:
                plant[i] = (int(teacher[depth[i] - 1]) + 1 + rank) % vocab
    return plant
