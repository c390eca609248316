"""Host-side placement helpers that turn the histograms of ``director_placement_cost`` into a new
placement matrix.  They are simple greedy heuristics operating on the quantities the paper's optimiser
uses (Section VI-A: workload matrix W, per-rank load of Eq. 1, capacity C_max) - not the paper's LP
relaxation.  Pure integer host code; the placement is tiny (E*R bytes) and is consumed by
``director_set_placement``.
"""
from __future__ import annotations

import heapq

import numpy as np


def expert_counts(workload) -> np.ndarray:
    """N_i = sum_j W[j, i]: tokens routed to expert i over all source ranks."""
    return np.asarray(workload, dtype=np.int64).sum(axis=0)


def single_copy_loads(N, X) -> np.ndarray:
    """Eq. 1 for a single-copy placement: lambda_j = sum of N_i over the experts hosted on rank j."""
    return np.asarray(X, dtype=np.int64).T @ np.asarray(N, dtype=np.int64)


def _share(n: int, q: int, r: int) -> int:
    """Rows the q-th of r round-robin replicas receives out of n."""
    return (n - q + r - 1) // r if n > q else 0


def replicate_hottest(N, X, n_hot: int = 2) -> np.ndarray:
    """Adds one replica of each of the n_hot most loaded experts (ties: lower id) on the least loaded
    rank (loads of the given placement, ties: lower rank) that neither hosts it nor received another
    new replica."""
    N = np.asarray(N, dtype=np.int64)
    out = np.array(X, dtype=np.uint8, copy=True)
    E, R = out.shape
    lam = single_copy_loads(N, out)
    order = np.lexsort((np.arange(E), -N))[:n_hot]
    used = np.zeros(R, dtype=bool)
    for e in order:
        ranks = np.lexsort((np.arange(R), lam))
        for j in ranks:
            if not out[e, j] and not used[j]:
                out[e, j] = 1
                used[j] = True
                break
    return out


def greedy_balanced(N, R: int, C_max: int, primary=None) -> np.ndarray:
    """Replica counts by repeatedly splitting the expert with the largest per-replica load, then
    largest-first packing of all copies onto the least loaded rank with a free slot.

    Spare slots (R*C_max - E) go one at a time to the expert maximising N_i / r_i (ties: lower id; never
    more than R copies; never to an expert without tokens).  Copies are then placed in the order
    (rows descending, expert ascending, copy ascending) on the least loaded rank (ties: lower rank) that
    has a free slot and does not host that expert; a copy that fits nowhere is dropped.  With `primary`
    (rank per expert) copy 0 of every expert is fixed there beforehand."""
    N = np.asarray(N, dtype=np.int64)
    E = len(N)
    reps = np.ones(E, dtype=np.int64)
    spare = R * C_max - E
    if spare < 0:
        raise ValueError("more experts than slots")
    # max-heap on N_i / r_i with exact rational comparison
    class Key:
        __slots__ = ("n", "r", "e")

        def __init__(self, n, r, e):
            self.n, self.r, self.e = n, r, e

        def __lt__(self, o):       # "smaller" == higher priority
            a, b = self.n * o.r, o.n * self.r
            return a > b if a != b else self.e < o.e

    heap = [Key(int(N[e]), 1, e) for e in range(E) if N[e] > 0 and R > 1]
    heapq.heapify(heap)
    while spare > 0 and heap:
        k = heapq.heappop(heap)
        reps[k.e] += 1
        spare -= 1
        if reps[k.e] < R:
            heapq.heappush(heap, Key(k.n, int(reps[k.e]), k.e))

    X = np.zeros((E, R), dtype=np.uint8)
    load = np.zeros(R, dtype=np.int64)
    free = np.full(R, C_max, dtype=np.int64)
    todo = []
    for e in range(E):
        first = 0
        if primary is not None:
            j = int(primary[e])
            X[e, j] = 1
            free[j] -= 1
            load[j] += _share(int(N[e]), 0, int(reps[e]))
            first = 1
        todo += [(-_share(int(N[e]), q, int(reps[e])), e, q) for q in range(first, int(reps[e]))]
    for neg_rows, e, _q in sorted(todo):
        ok = (free > 0) & (X[e] == 0)
        if not ok.any():
            continue
        cand = np.flatnonzero(ok)
        j = int(cand[np.argmin(load[cand])])     # argmin returns the first (lowest rank) minimum
        X[e, j] = 1
        free[j] -= 1
        load[j] -= neg_rows
    return X
