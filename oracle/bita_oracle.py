"""CPU oracle for the BiTA tree-decoding step (arXiv 2401.12522).

TEST INFRASTRUCTURE ONLY.  This file is a plain, slow, fp64 restatement of what
one decoding pass of the method computes, written from the paper so that the
CUDA library can be checked against it element by element.  It is imported by
the tests, by the smoke check and by the benchmark's CPU-baseline leg, never by
the product path, and it shares no code with the CUDA path (it does not import
the package, and the package does not import it).

What follows the paper and where:

* ``causal_logits`` / ``ar_greedy`` - the definition of the output: greedy
  autoregressive decoding of the frozen model (Abstract, Sec. 3.2 "lossless").
* ``block_layout`` - the packed input of one pass: last accepted token,
  flattened candidate tree, groups of n mask tokens (Sec. 3.2; Appendix B;
  Algorithm 1 "M x (n k + 1)").
* visibility rule - tree-based attention (Sec. 3.2, Fig. 6 caption) and the
  bi-directional-tuning mask: prompts are seen by mask tokens only (Sec. 3.1,
  Fig. 3 caption).
* ``verify_walk`` - greedy verification (Algorithm 1, else-branch) in its
  general-tree form.
* ``next_tree`` - draft candidates for the next pass from the top-k predictions
  of the selected mask group (Algorithm 1, last step of each branch).
* ``bita_step`` / ``prefill`` - one pass for t > 1 and for t = 1 (Algorithm 1).

Readings of points the paper leaves open (all repeated in the design notes):
masks of one group are causal among themselves; a node's masks see the node;
a "deep" prompt token is a per-layer key/value prefix used as is (no projection,
no rotary embedding); position ids are C for the root, C + depth for a node and
q + i for mask i attached at position q; ties go to the lowest token id.
PARITY UNPINNED for exactly these readings of the mask/prompt rows (mask-group
causality, prefix mechanics, mask position ids): nothing the paper prints fixes
them and they cannot change the emitted tokens; everything else is pinned by
the tests under ``tests/`` that do not need a GPU.

Model constants (the paper only says "LLaMA-2"): RMSNorm, rotary embedding with
half-split pairing (dims j and j + D/2), SwiGLU, no biases, untied LM head,
score scale 1/sqrt(D), grouped-query attention with H/H_kv consecutive query
heads per KV head.
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------- primitives

def f64(a) -> np.ndarray:
    return np.asarray(a, dtype=F64)


def rmsnorm(x: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """x * g / sqrt(mean(x^2) + eps), row-wise."""
    ms = np.mean(x * x, axis=-1, keepdims=True)
    return x * f64(g) / np.sqrt(ms + eps)


def rope(x: np.ndarray, pos: np.ndarray, theta: float) -> np.ndarray:
    """Rotary embedding, half-split pairing.  x: [rows, heads, D]; pos: [rows]."""
    D = x.shape[-1]
    half = D // 2
    j = np.arange(half, dtype=F64)
    inv_freq = theta ** (-2.0 * j / D)
    ang = f64(pos)[:, None] * inv_freq[None, :]          # [rows, half]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def silu(x: np.ndarray) -> np.ndarray:
    return x / (1.0 + np.exp(-x))


def masked_softmax(scores: np.ndarray, allowed: np.ndarray) -> np.ndarray:
    s = np.where(allowed, scores, -np.inf)
    s = s - np.max(s, axis=-1, keepdims=True)
    e = np.where(allowed, np.exp(s), 0.0)
    return e / np.sum(e, axis=-1, keepdims=True)


def argmax_lowest(v: np.ndarray) -> int:
    return int(np.argmax(v))           # first maximum = lowest id


def topk_sorted(v: np.ndarray, k: int):
    """k largest entries, ordered by (value descending, id ascending)."""
    order = np.argsort(-v, kind="stable")[:k]
    return order.astype(np.int64), v[order]


# --------------------------------------------------------------------------- model container

class Model:
    """Dimensions + weights.  ``w["layers"]`` may be any object with ``__getitem__`` (lazily generated)."""

    def __init__(self, *, L, d, H, H_kv, D, F, V, P, n_mask, rms_eps, rope_theta, weights):
        self.L, self.d, self.H, self.H_kv, self.D, self.F, self.V = L, d, H, H_kv, D, F, V
        self.P, self.n_mask, self.rms_eps, self.rope_theta = P, n_mask, rms_eps, rope_theta
        self.w = weights


def _project(x: np.ndarray, W) -> np.ndarray:
    return x @ f64(W).T


def _attention(model: Model, q, keys, values, allowed) -> np.ndarray:
    """q: [M,H,D]; keys/values: [H_kv, S, D]; allowed: [M,S] -> [M, H*D]."""
    M = q.shape[0]
    out = np.zeros((M, model.H, model.D), dtype=F64)
    rep = model.H // model.H_kv
    for h in range(model.H):
        kh = h // rep
        scores = (q[:, h, :] @ keys[kh].T) / math.sqrt(model.D)
        p = masked_softmax(scores, allowed)
        out[:, h, :] = p @ values[kh]
    return out.reshape(M, model.H * model.D)


def _layer(model: Model, lw: Dict, x, pos, ctx_k, ctx_v, vis, sees_prompt):
    """One decoder block over packed rows.  Returns (x_out, k_rows, v_rows)."""
    M = x.shape[0]
    H, Hk, D = model.H, model.H_kv, model.D
    xn = rmsnorm(x, lw["g_attn"], model.rms_eps)
    qkv = _project(xn, lw["wqkv"])
    q = qkv[:, : H * D].reshape(M, H, D)
    k = qkv[:, H * D: (H + Hk) * D].reshape(M, Hk, D)
    v = qkv[:, (H + Hk) * D:].reshape(M, Hk, D)
    q = rope(q, pos, model.rope_theta)
    k = rope(k, pos, model.rope_theta)
    C = ctx_k.shape[1]
    keys = np.concatenate([ctx_k, k.transpose(1, 0, 2)], axis=1)
    vals = np.concatenate([ctx_v, v.transpose(1, 0, 2)], axis=1)
    allowed = np.concatenate([np.ones((M, C), dtype=bool), vis], axis=1)
    if model.P > 0 and sees_prompt is not None and sees_prompt.any():
        keys = np.concatenate([keys, f64(lw["prompt_k"])], axis=1)
        vals = np.concatenate([vals, f64(lw["prompt_v"])], axis=1)
        allowed = np.concatenate([allowed, np.repeat(sees_prompt[:, None], model.P, axis=1)], axis=1)
    att = _attention(model, q, keys, vals, allowed)
    x = x + _project(att, lw["wo"])
    xn = rmsnorm(x, lw["g_ffn"], model.rms_eps)
    hf = silu(_project(xn, lw["wg"])) * _project(xn, lw["wu"])
    x = x + _project(hf, lw["wd"])
    return x, k, v


def forward_rows(model: Model, x, pos, ctx_k: List, ctx_v: List, vis, sees_prompt,
                 want_logits: bool = True, n_layers: Optional[int] = None):
    """Packed rows through the layer stack.  Returns dict(hidden=[L] of [M,d], logits, k=[L], v=[L])."""
    hidden, ks, vs = [], [], []
    L = model.L if n_layers is None else n_layers
    for l in range(L):
        x, k, v = _layer(model, model.w["layers"][l], x, pos, ctx_k[l], ctx_v[l], vis, sees_prompt)
        hidden.append(x)
        ks.append(k)
        vs.append(v)
    logits = None
    if want_logits:
        logits = _project(rmsnorm(x, model.w["g_final"], model.rms_eps), model.w["lm_head"])
    return dict(hidden=hidden, logits=logits, k=ks, v=vs)


# --------------------------------------------------------------------------- the definition: AR greedy decoding

def causal_logits(model: Model, tokens: Sequence[int]) -> np.ndarray:
    """Logits of every position of a plain causal forward over ``tokens`` (no cache, no tree, no prompts)."""
    T = len(tokens)
    x = f64(model.w["tok_emb"])[np.asarray(tokens, dtype=np.int64)]
    pos = np.arange(T)
    tril = np.tril(np.ones((T, T), dtype=bool))
    H, Hk, D = model.H, model.H_kv, model.D
    rep = H // Hk
    for l in range(model.L):
        lw = model.w["layers"][l]
        xn = rmsnorm(x, lw["g_attn"], model.rms_eps)
        qkv = xn @ f64(lw["wqkv"]).T
        q = rope(qkv[:, : H * D].reshape(T, H, D), pos, model.rope_theta)
        k = rope(qkv[:, H * D: (H + Hk) * D].reshape(T, Hk, D), pos, model.rope_theta)
        v = qkv[:, (H + Hk) * D:].reshape(T, Hk, D)
        att = np.zeros((T, H, D), dtype=F64)
        for h in range(H):
            s = q[:, h] @ k[:, h // rep].T / math.sqrt(D)
            att[:, h] = masked_softmax(s, tril) @ v[:, h // rep]
        x = x + att.reshape(T, H * D) @ f64(lw["wo"]).T
        xn = rmsnorm(x, lw["g_ffn"], model.rms_eps)
        x = x + (silu(xn @ f64(lw["wg"]).T) * (xn @ f64(lw["wu"]).T)) @ f64(lw["wd"]).T
    return rmsnorm(x, model.w["g_final"], model.rms_eps) @ f64(model.w["lm_head"]).T


def ar_greedy(model: Model, prompt: Sequence[int], n_new: int) -> List[int]:
    """The reference output: n_new tokens of greedy autoregressive decoding, recomputed from scratch each time."""
    seq = list(prompt)
    out = []
    for _ in range(n_new):
        t = argmax_lowest(causal_logits(model, seq)[-1])
        out.append(t)
        seq.append(t)
    return out


# --------------------------------------------------------------------------- packed block of one pass

class Block:
    """Row layout of one pass: row 0 root, rows 1..N tree nodes, then G groups of n mask rows."""

    def __init__(self, parent: Sequence[int], rank: Sequence[int], attach: Sequence[int], n_mask: int):
        self.parent, self.rank, self.attach, self.n = list(parent), list(rank), list(attach), n_mask
        N, G = len(parent), len(attach)
        self.N, self.G = N, G
        self.M = 1 + N + G * n_mask
        self.depth = []
        for i, p in enumerate(self.parent):
            assert -1 <= p < i
            self.depth.append(1 if p < 0 else self.depth[p] + 1)
        self.max_depth = max(self.depth, default=0)
        self.children = {x: [i for i in range(N) if self.parent[i] == x] for x in range(-1, N)}
        # row-level ancestors (row index = node index + 1, root = row 0)
        anc_rows = [[0]]                                   # row 0: itself
        for i in range(N):
            p = self.parent[i]
            anc_rows.append(anc_rows[p + 1] + [i + 1])      # root..parent chain + itself
        vis = np.zeros((self.M, self.M), dtype=bool)
        rel = np.zeros(self.M, dtype=np.int64)              # position id minus C
        sees_prompt = np.zeros(self.M, dtype=bool)
        for r in range(1 + N):
            vis[r, anc_rows[r]] = True
            rel[r] = 0 if r == 0 else self.depth[r - 1]
        for g, a in enumerate(self.attach):
            arow = a + 1
            for i in range(n_mask):                         # mask i+1 of the paper
                r = 1 + N + g * n_mask + i
                vis[r, anc_rows[arow]] = True               # attach point, its ancestors, the root
                first = 1 + N + g * n_mask
                vis[r, first: r + 1] = True                 # masks 1..i of its own group (causal)
                rel[r] = rel[arow] + (i + 1)
                sees_prompt[r] = True
        self.vis, self.rel_pos, self.sees_prompt = vis, rel, sees_prompt
        self.k_max = (max(self.rank) + 1) if N else 1
        self.group_of = {a: g for g, a in reversed(list(enumerate(self.attach)))}

    def mask_row(self, g: int, i: int) -> int:
        return 1 + self.N + g * self.n + i


def embed_block(model: Model, blk: Block, root: int, tree_tokens: Sequence[int]) -> np.ndarray:
    emb = f64(model.w["tok_emb"])
    x = np.zeros((blk.M, model.d), dtype=F64)
    x[0] = emb[root]
    for i, t in enumerate(tree_tokens):
        if t >= 0:                                          # token -1 = disabled node: zero row
            x[1 + i] = emb[t]
    me = f64(model.w["mask_emb"])
    for g in range(blk.G):
        for i in range(blk.n):
            x[blk.mask_row(g, i)] = me[i]
    return x


def verify_walk(blk: Block, tree_tokens: Sequence[int], row_argmax: Sequence[int]):
    """Greedy verification.  Returns (accepted node indices, emitted tokens, last accepted node or -1)."""
    cur = -1
    a = int(row_argmax[0])
    accepted, out = [], []
    while True:
        nxt = None
        for x in blk.children[cur]:                         # lowest index first
            if tree_tokens[x] >= 0 and tree_tokens[x] == a:
                nxt = x
                break
        if nxt is None:
            break
        accepted.append(nxt)
        out.append(a)
        cur = nxt
        a = int(row_argmax[1 + cur])
    out.append(a)                                           # the AR prediction of the last accepted token
    return accepted, out, cur


def next_tree(blk: Block, topk_ids: np.ndarray, cur: int) -> List[int]:
    """Tokens of the next pass's tree.  topk_ids: [G, n, k_max]."""
    # the group attached to the last accepted node, else to its nearest ancestor that has one
    a, shift = cur, 0
    while a not in blk.group_of:
        if a < 0:
            return [-1] * blk.N                             # no group at all: no drafts
        a = blk.parent[a]
        shift += 1
    g = blk.group_of[a]
    toks = []
    for i in range(blk.N):
        m = blk.depth[i] - 1 + shift                        # 0-based mask index that predicts this depth
        toks.append(int(topk_ids[g, m, blk.rank[i]]) if m < blk.n else -1)
    return toks


class State:
    """Decoding state between passes: cache (per layer [H_kv, C, D] keys/values), last accepted token."""

    def __init__(self, model: Model):
        self.k = [np.zeros((model.H_kv, 0, model.D), dtype=F64) for _ in range(model.L)]
        self.v = [np.zeros((model.H_kv, 0, model.D), dtype=F64) for _ in range(model.L)]
        self.root = -1
        self.tree: List[int] = []

    @property
    def C(self) -> int:
        return self.k[0].shape[1]

    def append(self, ks, vs, rows: Sequence[int]):
        rows = list(rows)
        for l in range(len(self.k)):
            self.k[l] = np.concatenate([self.k[l], ks[l][rows].transpose(1, 0, 2)], axis=1)
            self.v[l] = np.concatenate([self.v[l], vs[l][rows].transpose(1, 0, 2)], axis=1)


def bita_step(model: Model, blk: Block, st: State, tree_tokens: Optional[Sequence[int]] = None,
              keep: bool = True) -> Dict:
    """One pass for t > 1 (Algorithm 1, else-branch): verify the tree, emit tokens, draft the next tree."""
    toks = list(st.tree if tree_tokens is None else tree_tokens)
    assert len(toks) == blk.N
    C = st.C
    x = embed_block(model, blk, st.root, toks)
    pos = C + blk.rel_pos
    fw = forward_rows(model, x, pos, st.k, st.v, blk.vis, blk.sees_prompt)
    logits = fw["logits"]
    row_argmax = [argmax_lowest(logits[r]) for r in range(1 + blk.N)]
    topk_ids = np.zeros((blk.G, blk.n, blk.k_max), dtype=np.int64)
    topk_val = np.zeros((blk.G, blk.n, blk.k_max), dtype=F64)
    for g in range(blk.G):
        for i in range(blk.n):
            topk_ids[g, i], topk_val[g, i] = topk_sorted(logits[blk.mask_row(g, i)], blk.k_max)
    accepted, out, cur = verify_walk(blk, toks, row_argmax)
    nt = next_tree(blk, topk_ids, cur)
    rec = dict(n_out=len(out), out_tokens=out, accepted_idx=accepted, next_tree=nt,
               new_len=C + 1 + len(accepted), hidden=fw["hidden"], logits=logits,
               row_argmax=row_argmax, topk_ids=topk_ids, topk_val=topk_val, k=fw["k"], v=fw["v"],
               tree_tokens=toks, cur=cur)
    if keep:
        commit_step(st, rec)
    return rec


def commit_step(st: State, rec: Dict):
    """Keep root + accepted path in the cache (rejected drafts and all masks are dropped: Fig. 3 caption)."""
    st.append(rec["k"], rec["v"], [0] + [1 + i for i in rec["accepted_idx"]])
    st.root = rec["out_tokens"][-1]
    st.tree = list(rec["next_tree"])


def prefill(model: Model, blk: Block, st: State, tokens: Sequence[int]) -> Dict:
    """First pass (Algorithm 1, t = 1): the query, one mask group after its last token, no tree."""
    T = len(tokens)
    assert T >= 1
    n = blk.n
    C = st.C
    M = T + n
    x = np.zeros((M, model.d), dtype=F64)
    x[:T] = f64(model.w["tok_emb"])[np.asarray(tokens, dtype=np.int64)]
    x[T:] = f64(model.w["mask_emb"])[:n]
    vis = np.tril(np.ones((M, M), dtype=bool))
    sees_prompt = np.zeros(M, dtype=bool)
    sees_prompt[T:] = True
    pos = C + np.arange(M)
    fw = forward_rows(model, x, pos, st.k, st.v, vis, sees_prompt)
    logits = fw["logits"]
    a = argmax_lowest(logits[T - 1])
    topk_ids = np.zeros((1, n, blk.k_max), dtype=np.int64)
    topk_val = np.zeros((1, n, blk.k_max), dtype=F64)
    for i in range(n):
        topk_ids[0, i], topk_val[0, i] = topk_sorted(logits[T + i], blk.k_max)
    # the only group of this pass hangs on the last query token, which plays the root's role
    tree = []
    for i in range(blk.N):
        m = blk.depth[i] - 1
        tree.append(int(topk_ids[0, m, blk.rank[i]]) if m < n else -1)
    st.append(fw["k"], fw["v"], range(T))
    st.root = a
    st.tree = tree
    return dict(n_out=1, out_tokens=[a], next_tree=tree, new_len=C + T, logits=logits, hidden=fw["hidden"],
                topk_ids=topk_ids, topk_val=topk_val)


def generate(model: Model, blk: Block, prompt: Sequence[int], n_new: int, tree_fn=None):
    """Algorithm 1's outer loop without the EOS cut.  ``tree_fn(step, state) -> tokens`` may replace the drafts."""
    st = State(model)
    out = list(prefill(model, blk, st, prompt)["out_tokens"])
    per_pass = [1]
    step = 0
    while len(out) < n_new:
        toks = None if tree_fn is None else tree_fn(step, st)
        rec = bita_step(model, blk, st, toks)
        out.extend(rec["out_tokens"])
        per_pass.append(rec["n_out"])
        step += 1
    return out[:n_new], per_pass, st
