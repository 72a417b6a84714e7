"""Planted-acceptance draft trees.

Random-init mask tokens predict nothing useful, so the acceptance regime of a
tuned model (about 2.4-2.7 emitted tokens per pass, the paper's Table 1) is
imitated by overwriting one root-to-leaf path of the candidate tree with the
model's true greedy continuation on a seeded fraction of the steps.
"""
from __future__ import annotations

from typing import List, Sequence

from .rng import uniform_ints, uniform_unit
from .trees import Template


def plant_tree(template: Template, tree_tokens: Sequence[int], continuation: Sequence[int],
               seed: int, step: int, fraction: float, vocab: int) -> List[int]:
    """Return the tree tokens for ``step``.

    ``continuation[j]`` is the true greedy token that follows the root after j
    more tokens (continuation[0] is the token the root predicts).  With
    probability ``fraction`` (seeded) one leaf is chosen uniformly and the nodes
    on its path get continuation[0..depth-1]; a sibling that happens to hold the
    same token is moved to another id so siblings stay distinct.
    """
    toks = list(tree_tokens)
    N = template.N
    if N == 0:
        return toks
    u = float(uniform_unit(seed, 9001, 1, offset=step)[0])
    if u >= fraction:
        return toks
    has_child = [False] * N
    for p in template.parent:
        if p >= 0:
            has_child[p] = True
    leaves = [i for i in range(N) if not has_child[i]]
    leaf = leaves[int(uniform_ints(seed, 9002, 1, len(leaves), offset=step)[0])]
    path = []
    x = leaf
    while x >= 0:
        path.append(x)
        x = template.parent[x]
    path.reverse()
    for j, node in enumerate(path):
        if j >= len(continuation):
            break
        want = int(continuation[j])
        toks[node] = want
        for sib in range(N):
            if sib != node and template.parent[sib] == template.parent[node] and toks[sib] == want:
                toks[sib] = (want + 1 + sib) % vocab
    return toks
