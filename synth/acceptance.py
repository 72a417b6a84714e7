"""A stated, synthetic model of draft acceptance, for comparing tree templates without a tuned model.

Random-init mask tokens predict nothing, and none of the paper's datasets or tuned weights exist
here, so the acceptance side of the paper's template comparison (Sec. 4.3, Table 4) is replaced
by a model with three stated numbers.  It describes the drafts only (an input of the workload);
it holds none of the decoding method's arithmetic: the acceptance rule it walks is "the true next
token is among this node's children", which is what any draft tree means.

Model.  A mask token that stands `dist` positions after the last token it can see (dist = 1 for the
first mask of a group attached to the last accepted token) ranks the true token of its position
at rank rho (1-based) with probability

    P(rho | dist) = h0 * gamma**(dist - 1) * r**(rho - 1)        (capped so that the sum over rho <= 1)

independently per position: the top-1 hit rate decays with the distance by `gamma` per position and
each further rank is `r` times as likely as the one before.  Defaults h0 = 0.62, gamma = 0.80,
r = 0.35 give the paper's tree of 5 candidates x 3 mask tokens with a group per node about 2.6
tokens per pass, the range the speedups of its Table 1 imply for a 7B model.

A template whose groups hang on every node always drafts from dist = 1, 2, ...; with a single
group on the last token, the masks left after c accepted drafts stand c positions further away
and only n - c of them are left (Fig. 3 caption), which the simulation follows.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List

from .rng import uniform_unit
from .trees import Template


@dataclass(frozen=True)
class AcceptanceModel:
    h0: float = 0.62
    gamma: float = 0.80
    r: float = 0.35

    def rank_cdf(self, dist: int, k: int) -> List[float]:
        """cdf[j] = P(true token is among the first j + 1 ranks) for a mask at distance `dist`."""
        top = self.h0 * self.gamma ** (dist - 1)
        out, acc, p = [], 0.0, top
        for _ in range(k):
            acc = min(1.0, acc + p)
            out.append(acc)
            p *= self.r
        return out


def tokens_per_pass(tmpl: Template, n_mask: int, model: AcceptanceModel = AcceptanceModel(), *, passes: int = 20000,
                    seed: int = 0x5EED3001) -> Dict[str, float]:
    """Seeded simulation of `passes` decoding passes; returns mean tokens per pass and mean accepted drafts."""
    N = tmpl.N
    depth = tmpl.depths()
    children: Dict[int, Dict[int, int]] = {}
    for i in range(N):
        children.setdefault(tmpl.parent[i], {})[tmpl.rank[i]] = i
    group_at = set(tmpl.attach)
    k_max = (max(tmpl.rank) + 1) if N else 1
    u = uniform_unit(seed, 11, passes * (max(depth, default=0) + 1)).tolist()
    ui = 0
    shift = 0                      # masks of the drafting group that the accepted text had already used up
    total = 0
    for _ in range(passes):
        cur, c = -1, 0
        while True:
            d = c + 1                                           # depth of the candidates now under test
            if d + shift > n_mask:                              # no mask was left to draft this depth
                break
            kids = children.get(cur, {})
            if not kids:
                break
            cdf = model.rank_cdf(d + shift, k_max)
            x = u[ui]
            ui += 1
            rho = next((j for j, v in enumerate(cdf) if x < v), None)
            if rho is None or rho not in kids:
                break
            cur = kids[rho]
            c += 1
        total += 1 + c
        # the group that drafts the next tree: attached to the last accepted node, else to the
        # nearest ancestor that carries one (distance = masks of it that the accepted text used up)
        at, s = cur, 0
        while at not in group_at and at >= 0:
            at = tmpl.parent[at]
            s += 1
        if at not in group_at:
            shift = n_mask                                      # no group at all: nothing drafted
        else:
            shift = s
    return {"tokens_per_pass": total / passes, "accepted_per_pass": total / passes - 1.0}
