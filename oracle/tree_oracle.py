"""Oracle for the optimal draft tree (TEST INFRASTRUCTURE, not product code).

Section 4 ("Markov Chain Simulation") defines the optimal tree with k + 1 vertices as the one that
maximises the sum of its vertices' acceptance probabilities R(j); because a vertex can only be
accepted when its ancestors are, R never grows along a path, and the optimum is the set of the k
vertices of highest R.  This file writes that definition out -- enumerate, sort, take k -- for
the 0-th order model the paper's experiments use, R(j_1..j_m) = a[j_1] * ... * a[j_m] with a[r]
the acceptance probability of a node's child of rank r.  It does not follow Algorithm 3's
priority queue (the library does); `best_tree_by_search` is an exhaustive search over all trees
for tiny k that pins the definition itself.
"""
from __future__ import annotations

from typing import Dict, List, Sequence, Tuple


def vertex_probability(path: Tuple[int, ...], accept: Sequence[float]) -> float:
    r = 1.0
    for j in path:
        r *= accept[j] if j < len(accept) else 0.0
    return r


def top_k_vertices(accept: Sequence[float], k: int) -> List[Tuple[float, Tuple[int, ...]]]:
    """The k vertices of highest R (ties: shallower first, then lexicographic), each (R, path)."""
    C = len(accept)
    cand = []

    def extend(path, need):
        # `need` = vertices a valid tree must hold to contain `path` (it with its ancestors and
        # all their earlier siblings); only vertices with need <= k can be in a k-vertex tree
        for j in range(C):
            if need + j + 1 > k:
                break
            child = path + (j,)
            cand.append((vertex_probability(child, accept), child))
            extend(child, need + j + 1)

    extend((), 0)
    cand.sort(key=lambda t: (-t[0], len(t[1]), t[1]))
    return cand[:k]


def expected_accepted(paths, accept: Sequence[float]) -> float:
    return sum(vertex_probability(tuple(p), accept) for p in paths)


def is_valid_tree(paths) -> bool:
    """Prefix-closed and sibling-closed: a vertex needs its parent and its previous sibling."""
    s = {tuple(p) for p in paths}
    for p in s:
        if len(p) > 1 and p[:-1] not in s:
            return False
        if p[-1] > 0 and p[:-1] + (p[-1] - 1,) not in s:
            return False
    return True


def best_tree_by_search(accept: Sequence[float], k: int) -> float:
    """Largest expected number of accepted tokens over ALL valid trees with k drafted vertices."""
    C = len(accept)
    best = 0.0

    seen: Dict[frozenset, bool] = {}

    def grow_memo(tree: frozenset, total: float):
        if tree in seen:
            return
        seen[tree] = True
        nonlocal best
        if len(tree) == k:
            best = max(best, total)
            return
        frontier = set()
        for p in list(tree) + [()]:
            child = p + (0,)
            if child not in tree:
                frontier.add(child)
            if p:
                sib = p[:-1] + (p[-1] + 1,)
                if sib[-1] < C and sib not in tree:
                    frontier.add(sib)
        for v in frontier:
            grow_memo(tree | {v}, total + vertex_probability(v, accept))

    grow_memo(frozenset(), 0.0)
    return best


def parent_array(paths) -> List[int]:
    """Vertices in lexicographic order (the paper's order) as a parent-index array, root first."""
    order = [()] + sorted(tuple(p) for p in paths)
    index = {p: n for n, p in enumerate(order)}
    return [-1] + [index[p[:-1]] for p in order[1:]]


def acceptance_profile(paths, parent: Sequence[int], max_children: int):
    """Empirical per-rank acceptance (Section 5: R estimated from observed acceptances as a 0-th
    order Markov source).  `paths`: per sequence the accepted node ids, root first (-1 padding
    allowed).  A node on a path was verified: each of its children is one trial of its rank; the
    next node on the path is the child that was accepted.  Returns (accept, trials) per rank, with
    accept[r] = hits[r] / trials[r] (0 where never tried), uncapped."""
    n = len(parent)
    kids = [[] for _ in range(n)]
    for m in range(1, n):
        kids[parent[m]].append(m)
    hits = [0] * max_children
    trials = [0] * max_children
    for path in paths:
        path = [int(v) for v in path if int(v) >= 0]
        for d, node in enumerate(path):
            for r in range(min(len(kids[node]), max_children)):
                trials[r] += 1
            if d + 1 < len(path):
                r = kids[node].index(path[d + 1])
                if r < max_children:
                    hits[r] += 1
    return [hits[r] / trials[r] if trials[r] else 0.0 for r in range(max_children)], trials
