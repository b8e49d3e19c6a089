"""Accept-exercise mode: overlay a teacher continuation on one seeded root-to-node path.

plant[i] = -1 keeps the drafted token of row i; plant[i] >= 0 replaces it.  Planting the base
model's own greedy continuation on a depth-m path makes greedy acceptance accept (at least) m
candidates, so a schedule cycling m through 0..K exercises every accepted length.
"""
from typing import List, Sequence
from .rng import uniform_ids


def planted_length(step: int, b: int, K: int) -> int:
    return (step + b) % (K + 1)


def plant_row(parent: Sequence[int], teacher: Sequence[int], m: int, seed: int, step: int, b: int) -> List[int]:
    """teacher[k-1] is the token the base model would emit k places after the root (k = 1..m)."""
    T = len(parent)
    depth = [0] * T
    for i in range(1, T):
        depth[i] = depth[parent[i]] + 1
    plant = [-1] * T
    if m == 0:
        return plant
    nodes = [i for i in range(T) if depth[i] == m]
    node = nodes[int(uniform_ids(seed, 7000 + 131 * step + b, 1, len(nodes))[0])]
    while node != 0:
        plant[node] = int(teacher[depth[node] - 1])
        node = parent[node]
    return plant
