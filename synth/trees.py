"""Draft-candidate tree templates (shape only: which node hangs under which).

A template lists, for every node of the candidate tree (root excluded) in
flattened order, its parent (-1 = the root, i.e. the last accepted token) and
its rank (which of the top-k predictions of that depth's mask token fills the
node), plus the attach points of the mask-token groups.  Nodes are flattened
depth by depth, as the paper flattens its tree (Appendix B).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List

from .rng import uniform_ints


@dataclass(frozen=True)
class Template:
    parent: tuple   # N ints, -1 = root, parent[i] < i
    rank: tuple     # N ints, 0-based
    attach: tuple   # G ints, -1 = root or node index

    @property
    def N(self) -> int:
        return len(self.parent)

    @property
    def G(self) -> int:
        return len(self.attach)

    def depths(self) -> List[int]:
        d = []
        for p in self.parent:
            d.append(1 if p < 0 else d[p] + 1)
        return d


def product_rule_template(K, B, *, per_node_groups: bool = False) -> Template:
    """Rank tuples (a_1..a_m), 1-based, kept iff a_i <= K_i and prod_{i<=j} a_i <= B_j for all j<=m."""
    levels = [[()]]
    for depth in range(len(K)):
        nxt = []
        for t in levels[-1]:
            prod = 1
            for a in t:
                prod *= a
            for a in range(1, K[depth] + 1):
                if prod * a <= B[depth]:
                    nxt.append(t + (a,))
        nxt.sort()
        levels.append(nxt)
    flat = [t for lvl in levels[1:] for t in lvl]
    index = {t: i for i, t in enumerate(flat)}
    parent = tuple(-1 if len(t) == 1 else index[t[:-1]] for t in flat)
    rank = tuple(t[-1] - 1 for t in flat)
    attach = (-1,) + tuple(range(len(flat))) if per_node_groups else (-1,)
    return Template(parent, rank, attach)


def comb_template(n: int, k: int, *, per_node_groups: bool = True) -> Template:
    """The paper's efficient tree (Sec. 3.2, Fig. 4): k candidates per depth, children only under the top-1."""
    parent, rank = [], []
    for depth in range(n):
        top1_prev = -1 if depth == 0 else (depth - 1) * k
        for j in range(k):
            parent.append(top1_prev)
            rank.append(j)
    N = n * k
    attach = (-1,) + tuple(range(N)) if per_node_groups else (-1,)
    return Template(tuple(parent), tuple(rank), attach)


def full_tree_template(n: int, k: int, *, per_node_groups: bool = True) -> Template:
    """Fully tree-based decoding (Sec. 4.3, Table 4): every candidate of a depth has k children."""
    return product_rule_template((k,) * n, (k ** n,) * n, per_node_groups=per_node_groups)


def chain_template(n: int) -> Template:
    """Straightforward decoding (Sec. 3.2, Fig. 3): the top-1 draft of each mask, one group at the end."""
    return Template(tuple(range(-1, n - 1)), (0,) * n, (-1,))


def empty_template(with_group: bool = True) -> Template:
    return Template((), (), (-1,) if with_group else ())


def random_recursive_template(seed: int, N: int, *, max_depth: int = 8, max_rank: int = 16) -> Template:
    """Node i picks its parent uniformly from {root} + {j < i : depth(j) < max_depth}; ranks count siblings."""
    draws = uniform_ints(seed, 7001, N, 1 << 30).tolist()
    parent, depth, nchild = [], [], {}
    for i in range(N):
        while True:
            cands = [-1] + [j for j in range(i) if depth[j] < max_depth]
            cands = [c for c in cands if nchild.get(c, 0) < max_rank]
            p = cands[draws[i] % len(cands)]
            break
        parent.append(p)
        depth.append(1 if p < 0 else depth[p] + 1)
        nchild[p] = nchild.get(p, 0) + 1
    # flatten by depth (stable), remap parents
    order = sorted(range(N), key=lambda i: (depth[i], i))
    new = {old: k for k, old in enumerate(order)}
    par2 = [(-1 if parent[o] < 0 else new[parent[o]]) for o in order]
    seen, rank2 = {}, []
    for p in par2:
        rank2.append(seen.get(p, 0))
        seen[p] = seen.get(p, 0) + 1
    return Template(tuple(par2), tuple(rank2), (-1,))
