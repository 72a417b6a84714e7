"""The seeded input generators beyond the tensors: tree templates and the synthetic acceptance model."""
import synth
from synth import AcceptanceModel, tokens_per_pass


def test_full_tree_template_counts():
    for n, k in [(3, 1), (3, 2), (3, 3), (4, 2)]:
        t = synth.full_tree_template(n, k)
        assert t.N == sum(k ** d for d in range(1, n + 1))
        assert t.G == t.N + 1
        d = t.depths()
        for i, p in enumerate(t.parent):
            assert p < i and (p < 0) == (d[i] == 1)
        # every node of depth < n has exactly k children with ranks 0..k-1
        for x in range(-1, t.N):
            kids = sorted(t.rank[i] for i in range(t.N) if t.parent[i] == x)
            assert kids == (list(range(k)) if x < 0 or d[x] < n else [])


def test_acceptance_model_limits():
    sure = AcceptanceModel(h0=1.0, gamma=1.0, r=0.0)        # every top-1 draft is right
    n = 3
    # a group per node: every pass accepts all n drafts
    assert tokens_per_pass(synth.full_tree_template(n, 1), n, sure, passes=200)["tokens_per_pass"] == n + 1
    # one group on the last token: a full acceptance leaves no mask for the next pass (Fig. 3: 4, 1, 4, 1, ...)
    assert tokens_per_pass(synth.chain_template(n), n, sure, passes=200)["tokens_per_pass"] == (n + 1 + 1) / 2
    never = AcceptanceModel(h0=0.0)
    assert tokens_per_pass(synth.comb_template(n, 5), n, never, passes=200)["tokens_per_pass"] == 1.0
    assert tokens_per_pass(synth.empty_template(), n, sure, passes=50)["tokens_per_pass"] == 1.0


def test_acceptance_grows_with_candidates_and_groups():
    n = 3
    m = AcceptanceModel()
    straight = tokens_per_pass(synth.chain_template(n), n, m)["tokens_per_pass"]
    full = [tokens_per_pass(synth.full_tree_template(n, k), n, m)["tokens_per_pass"] for k in (1, 2, 3)]
    comb = tokens_per_pass(synth.comb_template(n, 5), n, m)["tokens_per_pass"]
    assert straight < full[0] < full[1] < full[2]               # more candidates, more acceptance
    assert full[0] < comb < full[2]                             # the comb tree sits between k = 1 and the full k = 3 tree
    cdf = m.rank_cdf(1, 5)
    assert abs(cdf[0] - m.h0) < 1e-12 and all(a < b for a, b in zip(cdf, cdf[1:])) and cdf[-1] <= 1.0
