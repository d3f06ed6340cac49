"""Oracle for Stage 2 of LExI (paper, Algorithm 2): TEST INFRASTRUCTURE ONLY, plain Python.

``brute_force`` is the definition: enumerate every feasible k and take the smallest phi.
``evolutionary`` walks Algorithm 2 in the paper's order (initialise, then per generation: fitness,
tournament selection, crossover, mutation, projection, add to the population; finally arg min), with
the choices the paper leaves open made as follows, each consuming the caller's stream of uniform
uint32 numbers in order:
  below(n) = next % n;  coin = next & 1;  chance(p) = next / 2**32 < p
  initial member: all k_min, then each remaining unit goes to the below(#open)-th layer still under k_max
  parent: best of `tournament` members drawn with below(|P|), the first drawn wins ties
  crossover: child_j = p1_j if coin else p2_j
  mutation: if chance(eta): a = below(L); b = below(L-1), stepping over a; child_a += 1; child_b -= 1
  projection: clip; then move single units where that costs least / gains most, lowest index on ties
The library's implementation is separate code; the two share nothing but this description.

``evolutionary`` can record what it did (``trace``): the initial members and, per generation, the
two parents' positions in the population and the child after crossover, after mutation and after
projection.  The pins in the tests read that record against generations worked out by hand, so
that the steps themselves - not only the final allocation - are held to Algorithm 2.
"""
from __future__ import annotations

import itertools
from typing import List, Sequence, Tuple

import numpy as np


def phi(D: np.ndarray, k: Sequence[int]) -> float:
    return float(sum(D[j, kj - 1] for j, kj in enumerate(k)))


def brute_force(D: np.ndarray, k_min: int, budget: int) -> Tuple[List[int], float]:
    L, k_max = D.shape
    best, best_phi = None, float("inf")
    for k in itertools.product(range(k_min, k_max + 1), repeat=L):
        if sum(k) != budget:
            continue
        v = phi(D, k)
        if v < best_phi:
            best, best_phi = list(k), v
    return best, best_phi


class _Stream:
    def __init__(self, rnd):
        self.v = [int(x) for x in rnd]
        self.pos = 0

    def next(self) -> int:
        x = self.v[self.pos]
        self.pos += 1
        return x

    def below(self, n: int) -> int:
        return self.next() % n

    def coin(self) -> bool:
        return bool(self.next() & 1)

    def chance(self, p: float) -> bool:
        return self.next() / 4294967296.0 < p


def _project(D, k, k_min, k_max, budget):
    L = len(k)
    k = [min(max(v, k_min), k_max) for v in k]
    while sum(k) > budget:
        cands = [(D[j, k[j] - 2] - D[j, k[j] - 1], j) for j in range(L) if k[j] > k_min]
        cost, j = min(cands, key=lambda c: (c[0], c[1]))
        k[j] -= 1
    while sum(k) < budget:
        cands = [(D[j, k[j] - 1] - D[j, k[j]], j) for j in range(L) if k[j] < k_max]
        gain, j = max(cands, key=lambda c: (c[0], -c[1]))
        k[j] += 1
    return k


def evolutionary(D: np.ndarray, k_min: int, budget: int, rnd, *, n_pop: int = 32, g_max: int = 2000,
                 eta_mut: float = 0.3, tournament: int = 3, trace: list = None) -> Tuple[List[int], float]:
    D = np.asarray(D, dtype=np.float64)
    L, k_max = D.shape
    r = _Stream(rnd)
    pop, fit = [], []
    for _ in range(n_pop):
        k = [k_min] * L
        for _unit in range(budget - L * k_min):
            open_layers = [j for j in range(L) if k[j] < k_max]
            k[open_layers[r.below(len(open_layers))]] += 1
        pop.append(k)
        fit.append(phi(D, k))
    if trace is not None:
        trace.append({"init": [list(k) for k in pop]})
    for _g in range(g_max):
        parents = []
        for _q in range(2):
            best = None
            for _c in range(tournament):
                m = r.below(len(pop))
                if best is None or fit[m] < fit[best]:
                    best = m
            parents.append(best)
        p1, p2 = pop[parents[0]], pop[parents[1]]
        child = [p1[j] if r.coin() else p2[j] for j in range(L)]
        crossed = list(child)
        if L >= 2 and r.chance(eta_mut):
            a = r.below(L)
            b = r.below(L - 1)
            if b >= a:
                b += 1
            child[a] += 1
            child[b] -= 1
        mutated = list(child)
        child = _project(D, child, k_min, k_max, budget)
        if trace is not None:
            trace.append({"parents": tuple(parents), "crossed": crossed, "mutated": mutated,
                          "projected": list(child)})
        pop.append(child)
        fit.append(phi(D, child))
    best = min(range(len(pop)), key=lambda m: (fit[m], m))
    return list(pop[best]), fit[best]
