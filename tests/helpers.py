"""Helpers shared by the tests: golden-file parsing and small independent reference
computations written directly in the tests' own terms (none of them calls the oracle or the
CUDA library)."""
from __future__ import annotations

import os
from typing import Dict, List

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def load_accept_cases() -> List[Dict]:
    cases, cur = [], None
    with open(os.path.join(GOLDEN, "accept_cases.txt")) as f:
        for raw in f:
            line = raw.strip()
            if not line or line.startswith("#"):
                continue
            if line.startswith("case "):
                cur = {"name": line[5:].strip()}
                cases.append(cur)
                continue
            key, val = line.split(":", 1)
            val = val.strip()
            if key == "parents":
                cur["parents"] = [[] if p.strip() == "-" else [int(x) for x in p.split(",")]
                                  for p in val.split(";")]
            else:
                cur[key] = [int(x) for x in val.split()]
    return cases


def logits_with_argmax(argmax, V: int, rng=None) -> np.ndarray:
    """[N, V] fp32 rows whose unique maximum sits at argmax[n]."""
    n = len(argmax)
    if rng is None:
        out = np.zeros((n, V), dtype=np.float32)
    else:
        out = rng.standard_normal((n, V)).astype(np.float32)
    for i, a in enumerate(argmax):
        out[i, a] = 50.0
    return out


def mask_bits(mask_row: np.ndarray, N: int) -> List[int]:
    """Indices j < N whose bit is set in a row of uint32 words (word j // 32, bit j % 32)."""
    return [j for j in range(N) if (int(mask_row[j // 32]) >> (j % 32)) & 1]


def dp_longest_accepted(tok, amax, parents):
    """Longest accepted path by dynamic programming over the topological order, with the
    tie-break 'lowest end node, then lowest predecessor carrying length-1'.  Independent of
    the oracle's brute-force enumeration.  Returns the node list v0..vm."""
    N = len(tok)
    best = [-1] * N
    best[0] = 0
    for v in range(1, N):
        for p in parents[v]:
            if best[p] >= 0 and tok[v] == amax[p]:
                best[v] = max(best[v], best[p] + 1)
    m = max(best)
    end = min(v for v in range(N) if best[v] == m)
    path = [end]
    while path[-1] != 0:
        v = path[-1]
        path.append(min(p for p in parents[v]
                        if best[p] == best[v] - 1 and tok[v] == amax[p]))
    return path[::-1]


def verification_parents(tree_parent, merge_to, n):
    """Parent lists of the verification DAG of a grown token graph: a node reaches the children
    of its tree parent's merged copies too, i.e. parents(x) = {tree_parent[x]} + {r : merge_to[r]
    == tree_parent[x]} (sorted; node 0 is the root)."""
    merged_into = {}
    for r in range(n):
        if merge_to[r] >= 0:
            merged_into.setdefault(int(merge_to[r]), []).append(r)
    parents = [[]]
    for x in range(1, n):
        p = int(tree_parent[x])
        parents.append(sorted([p] + [r for r in merged_into.get(p, []) if r < x]))
    return parents


def root_paths(parents, max_depth):
    """Every root path (as a tuple of node ids) of a DAG given by parent lists, up to max_depth
    edges, by explicit depth-first enumeration over child lists."""
    n = len(parents)
    children = [[] for _ in range(n)]
    for v, ps in enumerate(parents):
        for p in ps:
            children[p].append(v)
    out, stack = [], [(0,)]
    while stack:
        path = stack.pop()
        out.append(path)
        if len(path) - 1 < max_depth:
            for c in children[path[-1]]:
                stack.append(path + (c,))
    return out
