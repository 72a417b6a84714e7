"""Pins of the CPU oracle against what the paper and the mathematics fix (no GPU needed).

Each test is chosen so that a plausible mistake in the oracle (a dropped term, a wrong sign or
index, a transposed operand, a wrong visibility bit) fails at least one of them.
"""
import math
import os

import numpy as np
import pytest

from helpers import MICRO, block_for, oracle_model, orc, prompt_tokens, synth

import torch

GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ primitives: closed forms

def test_rmsnorm_closed_forms():
    g = np.array([1.0, 2.0, -3.0, 0.5])
    x = np.full((1, 4), 7.0)
    # constant row: x / sqrt(x^2) = 1 -> output equals the gain
    np.testing.assert_allclose(orc.rmsnorm(x, g, 0.0), g[None], rtol=1e-15)
    # 3-4-0-0 row: mean square = 25/4
    y = orc.rmsnorm(np.array([[3.0, 4.0, 0.0, 0.0]]), np.ones(4), 0.0)
    np.testing.assert_allclose(y, [[1.2, 1.6, 0.0, 0.0]], rtol=1e-15)
    # eps enters under the root
    y = orc.rmsnorm(np.array([[0.0, 0.0]]), np.ones(2), 1e-5)
    assert np.all(y == 0.0)
    y = orc.rmsnorm(np.array([[1.0, 1.0]]), np.ones(2), 3.0)
    np.testing.assert_allclose(y, [[0.5, 0.5]], rtol=1e-15)


def test_silu_values():
    assert orc.silu(np.array([0.0]))[0] == 0.0
    np.testing.assert_allclose(orc.silu(np.array([1.0]))[0], 1.0 / (1.0 + math.exp(-1.0)), rtol=1e-15)
    np.testing.assert_allclose(orc.silu(np.array([-1.0]))[0], -1.0 / (1.0 + math.e), rtol=1e-15)
    np.testing.assert_allclose(orc.silu(np.array([40.0]))[0], 40.0, rtol=1e-15)


def test_rope_worked_cases():
    # D = 2: one pair, frequency 1 -> a plane rotation by `pos` radians, counter-clockwise
    x = np.array([[[1.0, 0.0]], [[0.0, 1.0]]])
    y = orc.rope(x, np.array([0.5, 0.5]), 10000.0)
    np.testing.assert_allclose(y[0, 0], [math.cos(0.5), math.sin(0.5)], rtol=1e-15)
    np.testing.assert_allclose(y[1, 0], [-math.sin(0.5), math.cos(0.5)], rtol=1e-15)
    # D = 4, half-split pairing: dims (0,2) rotate with frequency 1, dims (1,3) with theta^(-1/2)
    x = np.array([[[1.0, 1.0, 0.0, 0.0]]])
    y = orc.rope(x, np.array([3.0]), 100.0)
    np.testing.assert_allclose(y[0, 0], [math.cos(3.0), math.cos(0.3), math.sin(3.0), math.sin(0.3)], rtol=1e-14)
    # position 0 is the identity
    z = np.random.default_rng(0).normal(size=(3, 2, 8))
    np.testing.assert_array_equal(orc.rope(z, np.zeros(3), 10000.0), z)


def test_rope_relative_property():
    rng = np.random.default_rng(1)
    q, k = rng.normal(size=(1, 1, 16)), rng.normal(size=(1, 1, 16))
    ref = np.sum(orc.rope(q, np.array([9]), 1e4) * orc.rope(k, np.array([4]), 1e4))
    for shift in (1, 17, 1000):
        got = np.sum(orc.rope(q, np.array([9 + shift]), 1e4) * orc.rope(k, np.array([4 + shift]), 1e4))
        assert abs(got - ref) < 1e-9 * (1 + abs(ref))
    # and norms are preserved
    np.testing.assert_allclose(np.linalg.norm(orc.rope(q, np.array([123]), 1e4)), np.linalg.norm(q), rtol=1e-14)


def test_masked_softmax_and_attention_special_cases():
    s = np.array([[1.0, 2.0, 3.0]])
    p = orc.masked_softmax(s, np.array([[True, False, True]]))
    np.testing.assert_allclose(p, [[1 / (1 + math.e ** 2), 0.0, math.e ** 2 / (1 + math.e ** 2)]], rtol=1e-15)
    # a single visible key returns that key's value whatever the scores
    m = oracle_model(MICRO, 3)
    rng = np.random.default_rng(2)
    q = rng.normal(size=(2, m.H, m.D))
    keys = rng.normal(size=(m.H_kv, 5, m.D))
    vals = rng.normal(size=(m.H_kv, 5, m.D))
    allowed = np.zeros((2, 5), dtype=bool)
    allowed[0, 3] = allowed[1, 1] = True
    out = orc._attention(m, q, keys, vals, allowed).reshape(2, m.H, m.D)
    rep = m.H // m.H_kv
    for h in range(m.H):
        np.testing.assert_allclose(out[0, h], vals[h // rep, 3], rtol=1e-14)   # grouped heads: h -> h // rep
        np.testing.assert_allclose(out[1, h], vals[h // rep, 1], rtol=1e-14)
    # zero queries -> uniform average over the visible keys
    allowed = np.array([[True, True, False, True, False], [True] * 5])
    out = orc._attention(m, np.zeros_like(q), keys, vals, allowed).reshape(2, m.H, m.D)
    np.testing.assert_allclose(out[0, 0], vals[0, [0, 1, 3]].mean(0), rtol=1e-13)
    np.testing.assert_allclose(out[1, m.H - 1], vals[m.H_kv - 1].mean(0), rtol=1e-13)


def test_score_scale_is_inverse_sqrt_head_dim():
    m = oracle_model(MICRO, 3)
    q = np.zeros((1, m.H, m.D))
    q[0, :, 0] = 1.0
    keys = np.zeros((m.H_kv, 2, m.D))
    keys[:, 1, 0] = math.sqrt(m.D) * math.log(3.0)       # score difference = log 3 after scaling
    vals = np.zeros((m.H_kv, 2, m.D))
    vals[:, 1, :] = 1.0
    out = orc._attention(m, q, keys, vals, np.ones((1, 2), dtype=bool))
    np.testing.assert_allclose(out, 0.75, rtol=1e-13)      # softmax(0, log 3) = (1/4, 3/4)


def test_topk_and_argmax_ties_go_to_lowest_id():
    v = np.array([1.0, 5.0, 5.0, 0.0, 5.0, 3.0])
    assert orc.argmax_lowest(v) == 1
    ids, vals = orc.topk_sorted(v, 5)
    assert ids.tolist() == [1, 2, 4, 5, 0]
    assert vals.tolist() == [5.0, 5.0, 5.0, 3.0, 1.0]


# ------------------------------------------------------------------ reduction to a library routine

def test_causal_forward_matches_eager_torch_single_layer():
    """Empty tree, no masks = a standard LLaMA decode; the causal forward against torch's own ops."""
    shape = MICRO
    w = synth.make_weights(shape, 11, dtype=torch.float32)
    m = oracle_model(shape, 11, weights=w)
    toks = prompt_tokens(11, 7, shape.V)
    got = orc.causal_logits(m, toks)
    # torch: scaled_dot_product_attention + rms_norm + silu, float64
    import torch.nn.functional as Fn
    x = w["tok_emb"].double()[toks]
    T = len(toks)
    half = shape.D // 2
    inv = shape.rope_theta ** (-torch.arange(half, dtype=torch.float64) * 2 / shape.D)
    ang = torch.arange(T, dtype=torch.float64)[:, None] * inv[None]
    cos, sin = torch.cos(ang), torch.sin(ang)

    def rot(t):  # [T, h, D]
        a, b = t[..., :half], t[..., half:]
        return torch.cat([a * cos[:, None] - b * sin[:, None], b * cos[:, None] + a * sin[:, None]], -1)

    for lw in w["layers"]:
        xn = Fn.rms_norm(x, (shape.d,), lw["g_attn"].double(), shape.rms_eps)
        qkv = Fn.linear(xn, lw["wqkv"].double())
        q, k, v = torch.split(qkv, [shape.H * shape.D, shape.H_kv * shape.D, shape.H_kv * shape.D], dim=-1)
        q = rot(q.view(T, shape.H, shape.D)).transpose(0, 1)
        k = rot(k.view(T, shape.H_kv, shape.D)).transpose(0, 1).repeat_interleave(shape.H // shape.H_kv, 0)
        v = v.view(T, shape.H_kv, shape.D).transpose(0, 1).repeat_interleave(shape.H // shape.H_kv, 0)
        a = Fn.scaled_dot_product_attention(q, k, v, is_causal=True).transpose(0, 1).reshape(T, -1)
        x = x + Fn.linear(a, lw["wo"].double())
        xn = Fn.rms_norm(x, (shape.d,), lw["g_ffn"].double(), shape.rms_eps)
        x = x + Fn.linear(Fn.silu(Fn.linear(xn, lw["wg"].double())) * Fn.linear(xn, lw["wu"].double()),
                          lw["wd"].double())
    ref = Fn.linear(Fn.rms_norm(x, (shape.d,), w["g_final"].double(), shape.rms_eps), w["lm_head"].double())
    np.testing.assert_allclose(got, ref.numpy(), rtol=1e-9, atol=1e-11)


# ------------------------------------------------------------------ counting facts and the printed figures

def _read_gold(name):
    rows = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def test_comb_tree_counts_and_ancestors_fig4_fig6():
    rows = _read_gold("fig4_fig6_comb_tree.txt")
    kv = {r[0]: int(r[1]) for r in rows if r[0] != "ancestors"}
    t = synth.comb_template(kv["n"], kv["k"])
    blk = block_for(t, kv["n"])
    assert blk.N == kv["nodes"] and blk.G == kv["groups"] and blk.M == kv["rows"]
    for r in rows:
        if r[0] != "ancestors":
            continue
        node = int(r[1])
        anc = sorted(int(a) for a in r[3:])
        row = 1 + node
        seen_nodes = sorted(int(c) - 1 for c in np.nonzero(blk.vis[row, 1: 1 + blk.N])[0] + 1)
        assert seen_nodes == sorted(anc + [node])
        assert blk.vis[row, 0]                                  # every node sees the last accepted token
        assert not blk.vis[row, 1 + blk.N:].any()               # a candidate never sees a mask token
        assert not blk.sees_prompt[row]                         # nor a prompt token (Sec. 3.1)
        # its attached masks see the same tree nodes (incl. the node), earlier masks of their own group only
        g = blk.group_of[node]
        for i in range(blk.n):
            mr = blk.mask_row(g, i)
            assert sorted(np.nonzero(blk.vis[mr, 1: 1 + blk.N])[0].tolist()) == sorted(anc + [node])
            own = np.nonzero(blk.vis[mr, 1 + blk.N:])[0] + 1 + blk.N
            assert own.tolist() == [blk.mask_row(g, j) for j in range(i + 1)]
            assert blk.sees_prompt[mr]
            assert blk.rel_pos[mr] == blk.depth[node] + i + 1


def test_fig3_emitted_per_pass_pattern():
    rows = _read_gold("fig3_passes.txt")
    n = int([r for r in rows if r[0] == "n_mask"][0][1])
    want = [int(v) for v in [r for r in rows if r[0] == "emitted_per_pass"][0][1:]]
    blk = block_for(synth.chain_template(n), n)
    # scripted predictions: the true continuation is 10, 11, 12, ...; drafts of pass 1 all right,
    # drafts of pass 3 right, right, wrong.
    emitted = [1]                                               # pass 1 (t = 1) emits the AR token only
    tree = [11, 12, 13]
    # pass 2
    acc, out, cur = orc.verify_walk(blk, tree, [11, 12, 13, 14])
    emitted.append(len(out))
    assert out == [11, 12, 13, 14] and acc == [0, 1, 2]
    topk = np.array([[[21], [22], [23]]])
    tree = orc.next_tree(blk, topk, cur)
    assert tree == [-1, -1, -1]                                 # all masks used up: no drafts left
    # pass 3
    acc, out, cur = orc.verify_walk(blk, tree, [15, 0, 0, 0])
    emitted.append(len(out))
    assert out == [15] and cur == -1
    tree = orc.next_tree(blk, np.array([[[16], [17], [99]]]), cur)
    assert tree == [16, 17, 99]
    # pass 4
    acc, out, cur = orc.verify_walk(blk, tree, [16, 17, 18, 0])
    emitted.append(len(out))
    assert out == [16, 17, 18] and acc == [0, 1]
    assert emitted == want
    # partial acceptance shifts which masks are still usable
    assert orc.next_tree(blk, np.array([[[31], [32], [33]]]), cur) == [33, -1, -1]


def _gold_cases(name):
    """(header dict, [(case fields, expected tree)]) of a next-tree golden file."""
    rows = _read_gold(name)
    head = {r[0]: int(r[1]) for r in rows if r[0] in ("n", "k")}
    cases, cur = [], None
    for r in rows:
        if r[0] == "case":
            cur = {r[i]: int(r[i + 1]) for i in range(1, len(r), 2)}
        elif r[0] == "tree":
            cases.append((cur, [int(v) for v in r[1:]]))
    return head, cases


def test_next_tree_takes_the_group_of_the_last_accepted_node_alg1_golden():
    """Algorithm 1, last step of each branch, on the Fig. 4 tree with a mask group per node: the
    expected trees were written out by hand in the golden file; every scripted prediction is a
    distinct id, so a wrong group, a swapped mask/candidate index or a shifted depth changes a token."""
    head, cases = _gold_cases("alg1_next_tree_comb_n4k3.txt")
    n, k = head["n"], head["k"]
    blk = block_for(synth.comb_template(n, k), n)
    assert blk.G == n * k + 1
    topk = np.zeros((blk.G, n, k), dtype=np.int64)
    for g, at in enumerate(blk.attach):
        for r in range(1, n + 1):
            for j in range(1, k + 1):
                topk[g, r - 1, j - 1] = 100 * (at + 1) + 10 * r + j
    assert len(set(topk.ravel().tolist())) == topk.size
    assert len(cases) == 5
    for case, want in cases:
        assert orc.next_tree(blk, topk, case["last"]) == want
    # the same through the walk: accepting exactly the path to `last` selects that group
    for case, want in cases:
        path, x = [], case["last"]
        while x >= 0:
            path.append(x)
            x = blk.parent[x]
        path.reverse()
        tree = list(range(500, 500 + blk.N))                    # distinct draft tokens
        am = [499] * (1 + blk.N)                                # predictions that match nothing ...
        prev = -1
        for x in path:                                          # ... except along the path
            am[1 + prev] = tree[x]
            prev = x
        acc, out, cur = orc.verify_walk(blk, tree, am)
        assert acc == path and cur == case["last"]
        assert orc.next_tree(blk, topk, cur) == want


def test_next_tree_single_group_drops_the_first_c_masks_fig3_golden():
    """One mask group after the last token and k > 1 candidates per mask: after c accepted drafts
    depth r of the next tree holds the candidates of mask c + r (Fig. 3 caption), by hand in the
    golden file."""
    head, cases = _gold_cases("fig3_single_group_shift.txt")
    n, k = head["n"], head["k"]
    blk = block_for(synth.comb_template(n, k, per_node_groups=False), n)
    assert blk.G == 1
    topk = np.array([[[10 * r + j for j in range(1, k + 1)] for r in range(1, n + 1)]])
    assert len(cases) == 6
    for case, want in cases:
        assert blk.depth[case["last"]] == case["c"] if case["last"] >= 0 else case["c"] == 0
        assert orc.next_tree(blk, topk, case["last"]) == want


def test_first_pass_drafts_the_top_k_of_each_mask_alg1_t1():
    """Algorithm 1, t = 1: the last query token's top-1 is emitted and C^1 holds the top k of each
    mask token.  A scripted model (one layer whose attention and FFN add nothing, mask embedding i
    = unit vector 1 + i, LM-head column 1 + i = the scores of mask i) makes the logits of every
    mask row known in advance; the expected tree is the c = 0 case of the hand-written golden."""
    head, cases = _gold_cases("fig3_single_group_shift.txt")
    n, k = head["n"], head["k"]
    want = [t for c, t in cases if c["c"] == 0][0]
    d, V = 8, 64
    lm = np.zeros((V, d))
    lm[7, 0] = 1.0                                              # every query token embeds to e_0: its argmax is 7
    for r in range(1, n + 1):
        for j in range(1, k + 1):
            lm[10 * r + j, r] = 4.0 - j                         # mask r: candidate j has the j-th largest score
    z = lambda *s: np.zeros(s)
    layer = dict(wqkv=z(3 * d, d), wo=z(d, d), wg=z(8, d), wu=z(8, d), wd=z(d, 8), g_attn=np.ones(d),
                 g_ffn=np.ones(d), prompt_k=z(1, 0, d), prompt_v=z(1, 0, d))
    tok = z(V, d)
    tok[:, 0] = 1.0
    me = z(n, d)
    for i in range(n):
        me[i, 1 + i] = 1.0
    m = orc.Model(L=1, d=d, H=1, H_kv=1, D=d, F=8, V=V, P=0, n_mask=n, rms_eps=1e-5, rope_theta=1e4,
                  weights=dict(tok_emb=tok, mask_emb=me, g_final=np.ones(d), lm_head=lm, layers=[layer]))
    for tmpl in (synth.comb_template(n, k), synth.comb_template(n, k, per_node_groups=False)):
        blk = block_for(tmpl, n)
        st = orc.State(m)
        rec = orc.prefill(m, blk, st, [3, 1, 4, 1, 5])
        assert rec["out_tokens"] == [7] and rec["n_out"] == 1
        assert rec["next_tree"] == want and st.tree == want and st.root == 7 and st.C == 5


def _algorithm1_flat_walk(n, k, cand, logits_argmax):
    """Independent restatement of the paper's verification for its comb tree, on flattened row indices.

    cand[i][j] : j-th candidate of mask i (0-based); logits_argmax[r] : argmax of flattened row r
    (row 0 = last token, row 1 + i*k + j = candidate (i, j)).  Returns emitted tokens.
    """
    out = []
    base = 0                      # row of the token whose prediction is being checked
    a = logits_argmax[base]
    offset = 0                    # rows of the depths already passed
    for i in range(n):
        hit = None
        for j in range(k):
            if cand[i][j] == a:
                hit = j
                break
        if hit is None:
            break
        out.append(a)
        a = logits_argmax[1 + offset + hit]
        if hit != 0:
            break                 # only the top-1 candidate has children
        offset += k
    out.append(a)
    return out


def test_walk_equals_algorithm1_on_comb_trees():
    rng = np.random.default_rng(5)
    for n, k in [(3, 5), (4, 3), (4, 5), (2, 1)]:
        blk = block_for(synth.comb_template(n, k), n)
        for trial in range(300):
            vocab = 4                                           # tiny vocabulary -> many matches
            cand = [rng.permutation(vocab + k)[:k].tolist() for _ in range(n)]   # distinct siblings
            tree = [cand[i][j] for i in range(n) for j in range(k)]
            am = rng.integers(0, vocab + k, size=1 + n * k).tolist()
            _, out, _ = orc.verify_walk(blk, tree, am)
            assert out == _algorithm1_flat_walk(n, k, cand, am)
            assert 1 <= len(out) <= n + 1


# ------------------------------------------------------------------ tree attention == per-path causal attention

@pytest.mark.parametrize("seed", [0, 1, 2])
def test_tree_rows_equal_per_path_causal_forward(seed):
    shape = MICRO
    m = oracle_model(shape, 20 + seed, dtype=torch.float32)
    tmpl = synth.random_recursive_template(seed, 12, max_depth=5)
    tmpl = synth.Template(tmpl.parent, tmpl.rank, (-1,) + tuple(range(0, 12, 3)))
    blk = block_for(tmpl, shape.n_mask)
    prompt = prompt_tokens(seed, 5, shape.V)
    st = orc.State(m)
    orc.prefill(m, blk, st, prompt)
    tree = synth.uniform_ints(seed, 77, blk.N, shape.V).tolist()
    rec = orc.bita_step(m, blk, st, tree, keep=False)
    for x in range(-1, blk.N):
        path, y = [], x
        while y >= 0:
            path.append(tree[y])
            y = blk.parent[y]
        seq = prompt + [st.root] + path[::-1]
        ref = orc.causal_logits(m, seq)[-1]
        np.testing.assert_allclose(rec["logits"][1 + x], ref, rtol=1e-10, atol=1e-12)


def test_prompts_and_masks_do_not_touch_token_rows():
    shape = MICRO
    m = oracle_model(shape, 31, dtype=torch.float32)
    tmpl = synth.product_rule_template((3, 3, 3), (3, 3, 3), per_node_groups=True)
    blk_full = block_for(tmpl, shape.n_mask)
    blk_bare = block_for(synth.Template(tmpl.parent, tmpl.rank, ()), shape.n_mask)
    prompt = prompt_tokens(31, 6, shape.V)
    tree = synth.uniform_ints(31, 78, blk_full.N, shape.V).tolist()
    recs = []
    for blk in (blk_full, blk_bare):
        st = orc.State(m)
        orc.prefill(m, blk_full, st, prompt)
        recs.append(orc.bita_step(m, blk, st, tree, keep=False))
    rows = 1 + blk_full.N
    # (equal up to the last bit: BLAS blocks a 28-row and a 76-row product differently)
    np.testing.assert_allclose(recs[0]["logits"][:rows], recs[1]["logits"][:rows], rtol=1e-12, atol=1e-14)
    # while the mask rows do depend on the prompt prefix
    m2 = oracle_model(shape, 31, dtype=torch.float32)
    for lw in m2.w["layers"]:
        lw["prompt_v"] = lw["prompt_v"] * 0.0
    st = orc.State(m2)
    orc.prefill(m2, blk_full, st, prompt)
    rec2 = orc.bita_step(m2, blk_full, st, tree, keep=False)
    np.testing.assert_allclose(rec2["logits"][:rows], recs[0]["logits"][:rows], rtol=1e-12, atol=1e-14)
    assert np.abs(rec2["logits"][rows:] - recs[0]["logits"][rows:]).max() > 1e-6


# ------------------------------------------------------------------ lossless property

TEMPLATES = {
    "product-1group": lambda n: synth.product_rule_template((3, 3, 3), (3, 3, 3)),
    "product-pernode": lambda n: synth.product_rule_template((3, 3, 3), (3, 3, 3), per_node_groups=True),
    "comb-k3": lambda n: synth.comb_template(n, 3),
    "comb-k3-1group": lambda n: synth.comb_template(n, 3, per_node_groups=False),
    "chain": lambda n: synth.chain_template(n),
    "empty": lambda n: synth.empty_template(),
    "random": lambda n: synth.random_recursive_template(9, 10, max_depth=4),
}


@pytest.mark.parametrize("name", sorted(TEMPLATES))
@pytest.mark.parametrize("drafts", ["model", "random", "planted"])
def test_lossless_equals_autoregressive_greedy(name, drafts):
    shape = MICRO
    m = oracle_model(shape, 41, dtype=torch.float32)
    tmpl = TEMPLATES[name](shape.n_mask)
    blk = block_for(tmpl, shape.n_mask)
    prompt = prompt_tokens(41, shape.prompt_len, shape.V)
    n_new = 14
    ref = orc.ar_greedy(m, prompt, n_new + 6)

    def tree_fn(step, st):
        if drafts == "model":
            return None
        rnd = synth.uniform_ints(43, 100 + step, blk.N, shape.V).tolist()
        if drafts == "random":
            return rnd
        done = st.C - len(prompt) + 1                           # tokens emitted so far
        return synth.plant_tree(tmpl, rnd, ref[done: done + 6], 43, step, 0.7, shape.V)

    out, per_pass, st = orc.generate(m, blk, prompt, n_new, tree_fn)
    assert out == ref[:n_new]
    assert per_pass[0] == 1
    assert all(1 <= c <= blk.max_depth + 1 for c in per_pass)
    if name == "empty":
        assert all(c == 1 for c in per_pass)
    if drafts == "planted" and blk.N:
        assert max(per_pass) > 1                                # planted paths are really accepted
    # the cache after compaction is the cache of the same tokens run causally in one go
    total = st.C
    seq = (prompt + out + ref[n_new:])[:total]                  # tokens now in the cache
    emitted_all = prompt + ref
    seq = emitted_all[:total]
    st2 = orc.State(m)
    orc.prefill(m, blk, st2, seq)
    for l in range(m.L):
        np.testing.assert_allclose(st.k[l], st2.k[l], rtol=1e-9, atol=1e-11)
        np.testing.assert_allclose(st.v[l], st2.v[l], rtol=1e-9, atol=1e-11)


def test_step_after_full_acceptance_has_no_drafts_single_group():
    """With one mask group, accepting n drafts leaves nothing to draft from: the next pass emits 1 token."""
    shape = MICRO
    m = oracle_model(shape, 41, dtype=torch.float32)
    tmpl = synth.chain_template(shape.n_mask)
    blk = block_for(tmpl, shape.n_mask)
    prompt = prompt_tokens(41, shape.prompt_len, shape.V)
    ref = orc.ar_greedy(m, prompt, 10)
    st = orc.State(m)
    orc.prefill(m, blk, st, prompt)
    rec = orc.bita_step(m, blk, st, ref[1:1 + blk.N])
    assert rec["n_out"] == shape.n_mask + 1 and rec["next_tree"] == [-1] * blk.N
    rec = orc.bita_step(m, blk, st)
    assert rec["n_out"] == 1


def test_mask_position_ids_and_prefill_layout():
    blk = block_for(synth.product_rule_template((3, 3, 3), (3, 3, 3), per_node_groups=True), 3)
    assert blk.rel_pos[0] == 0
    for i in range(blk.N):
        assert blk.rel_pos[1 + i] == blk.depth[i]
    for g, a in enumerate(blk.attach):
        q = 0 if a < 0 else blk.depth[a]
        assert [blk.rel_pos[blk.mask_row(g, i)] for i in range(3)] == [q + 1, q + 2, q + 3]
