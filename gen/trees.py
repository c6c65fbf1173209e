"""Draft-tree topologies and accepted-path choices (index work only).

A tree configuration T = (N_1, ..., N_gamma) in the paper's notation (Section
4.1) expands every node of generation i-1 into N_i children, so generation i
holds N_1*...*N_i nodes.  Here the root (the last verified token) is node 0 and
nodes are numbered in breadth-first order; ``parents[i]`` is the tree-local
index of node i's parent, -1 for the root (whose parent is the sequence's
committed state).
"""

from __future__ import annotations

from dataclasses import dataclass
from typing import List, Sequence

import numpy as np

from .configs import Config
from .draw import rng_for


@dataclass
class Tree:
    parents: np.ndarray        # (M,) int32, BFS order, parents[0] == -1
    level_offsets: np.ndarray  # (n_levels+1,) int32; level l = nodes [off[l], off[l+1])

    @property
    def n_nodes(self) -> int:
        return int(self.parents.shape[0])

    @property
    def n_levels(self) -> int:
        return int(self.level_offsets.shape[0] - 1)

    def depth(self) -> np.ndarray:
        d = np.zeros(self.n_nodes, dtype=np.int32)
        for i in range(1, self.n_nodes):
            d[i] = d[self.parents[i]] + 1
        return d

    def children(self) -> List[List[int]]:
        ch: List[List[int]] = [[] for _ in range(self.n_nodes)]
        for i in range(1, self.n_nodes):
            ch[int(self.parents[i])].append(i)
        return ch

    def path_to(self, node: int) -> List[int]:
        p = []
        v = int(node)
        while v >= 0:
            p.append(v)
            v = int(self.parents[v])
        return p[::-1]


def _from_levels(levels: List[List[int]]) -> Tree:
    parents = np.array([p for lvl in levels for p in lvl], dtype=np.int32)
    off = np.zeros(len(levels) + 1, dtype=np.int32)
    off[1:] = np.cumsum([len(l) for l in levels])
    return Tree(parents, off)


def full_tree(branching: Sequence[int]) -> Tree:
    """Root plus one level per entry of ``branching``."""
    levels = [[-1]]
    first = 0
    for b in branching:
        prev = levels[-1]
        levels.append([first + j for j in range(len(prev)) for _ in range(int(b))])
        first += len(prev)
    return _from_levels(levels)


def paper_tree(config: Sequence[int]) -> Tree:
    """A tree configuration as the paper writes it, e.g. (3,2,2,1,1)."""
    return full_tree(config)


def chain_tree(length: int) -> Tree:
    return full_tree([1] * (int(length) - 1))


def capped_tree(branching: Sequence[int], node_budget: int, seed: int, cid: int = 2, rnd: int = 0) -> Tree:
    """Full tree, but only a seeded random subset of the deepest level is kept
    so that the node count equals ``node_budget`` (BFS order preserved)."""
    t = full_tree(branching)
    if t.n_nodes <= node_budget:
        return t
    last0, last1 = int(t.level_offsets[-2]), int(t.level_offsets[-1])
    keep = node_budget - last0
    if keep <= 0:
        raise ValueError("node budget smaller than the tree above its deepest level")
    g = rng_for(seed, cid, 0, rnd, "tree")
    sel = np.sort(g.choice(last1 - last0, size=keep, replace=False)) + last0
    parents = np.concatenate([t.parents[:last0], t.parents[sel]]).astype(np.int32)
    off = t.level_offsets.copy()
    off[-1] = last0 + keep
    return Tree(parents, off)


def random_branching_tree(n_nodes: int, n_levels: int, seed: int, cid: int = 4, rnd: int = 0, seq: int = 0,
                          max_children: int = 3) -> Tree:
    """Every node draws 1..max_children children, level by level, for
    ``n_levels`` levels; the result is cut (BFS order) or grown (extra children
    under random nodes above the last level that still have room) to exactly
    ``n_nodes`` nodes."""
    g = rng_for(seed, cid, seq, rnd, "tree")
    levels = [[-1]]
    first = 0
    for _ in range(n_levels - 1):
        prev = levels[-1]
        nxt = []
        for j in range(len(prev)):
            nxt += [first + j] * int(g.integers(1, max_children + 1))
        first += len(prev)
        levels.append(nxt)
    t = _from_levels(levels)
    parents = list(t.parents)
    depth = list(t.depth())
    if len(parents) > n_nodes:
        parents, depth = parents[:n_nodes], depth[:n_nodes]
    while len(parents) < n_nodes:
        counts = np.bincount([p for p in parents if p >= 0], minlength=len(parents))
        cand = [i for i in range(len(parents)) if depth[i] < n_levels - 1 and counts[i] < max_children]
        if not cand:
            raise ValueError("cannot grow the tree to the requested size")
        p = int(cand[int(g.integers(0, len(cand)))])
        parents.append(p)
        depth.append(depth[p] + 1)
    # renumber breadth-first (stable within a level: by parent's new index, then insertion order)
    order = sorted(range(len(parents)), key=lambda i: (depth[i],))
    order_levels: List[List[int]] = [[] for _ in range(max(depth) + 1)]
    for i in order:
        order_levels[depth[i]].append(i)
    new_index = {}
    out_levels: List[List[int]] = []
    for l, nodes in enumerate(order_levels):
        if l > 0:
            nodes = sorted(nodes, key=lambda i: (new_index[parents[i]], i))
        for i in nodes:
            new_index[i] = len(new_index)
        out_levels.append([-1 if parents[i] < 0 else new_index[parents[i]] for i in nodes])
    return _from_levels(out_levels)


def random_accepted_node(tree: Tree, seed: int, cid: int, rnd: int, seq: int = 0) -> int:
    """Accepted depth a ~ U{0..levels-1}; walk down from the root picking a
    uniformly random child at each level (stopping early at a leaf)."""
    g = rng_for(seed, cid, seq, rnd, "accept")
    a = int(g.integers(0, tree.n_levels))
    ch = tree.children()
    v = 0
    for _ in range(a):
        if not ch[v]:
            break
        v = ch[v][int(g.integers(0, len(ch[v])))]
    return v


def config_tree(cfg: Config, rnd: int = 0, seq: int = 0, seed=None) -> Tree:
    """The draft tree a configuration uses in round ``rnd`` for sequence ``seq``."""
    seed = cfg.seed if seed is None else seed
    if cfg.tree == "full:2x4":
        return full_tree([2, 2, 2])
    if cfg.tree == "capped150":
        return capped_tree([4, 4, 2, 2, 2], 150, seed, cfg.cid, rnd)
    if cfg.tree == "chain16":
        return chain_tree(16)
    if cfg.tree == "rand32":
        return random_branching_tree(32, 5, seed, cfg.cid, rnd, seq)
    raise ValueError(f"configuration {cfg.cid} has no tree")
