"""Lockstep comparison of the CUDA library with the CPU oracle on the same seeded inputs.

Both sides start every pass from the same (cache, last token, tree).  Random-init logits are nearly
flat, so an argmax or a top-k slot may legitimately differ where the oracle's own margin is below
the logit tolerance; such a choice is validated against the oracle's logits and then adopted by the
oracle so that the run stays in lockstep.  Everything else must match exactly (tokens, accepted
length, accepted indices, next tree, cache length) or within the stated tolerances (hidden states,
logits, cache contents).
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from helpers import block_for, oracle_model, oracle_model_from_device, orc, prompt_tokens, synth

@dataclass(frozen=True)
class Tolerances:
    """Bounds of the floating-point comparison; the defaults are the parity target as stated.

    layer_rel_l2    error ONE layer adds: the GPU's output of layer l against the oracle's layer l
                    applied to the GPU's own input of that layer (its residual stream after layer
                    l - 1 and its cache), relative L2 over the block.  Independent of what the
                    earlier layers did, so it cannot hide behind, or be loosened by, their error.
    hidden_rel_l2   accumulated distance of the two residual streams after any layer, relative L2.
    logit_rms       max |delta| over the block's logits in units of RMS(oracle logits).  The same
                    number, times that RMS, is the margin below which a differing argmax / top-k
                    slot counts as a tie; it never depends on an error measured on the GPU side.
    kv_rel_l2       cache contents (bf16 roundings of the oracle's fp64 values).
    """
    layer_rel_l2: float = 1e-2
    hidden_rel_l2: float = 1e-2
    logit_rms: float = 3e-2
    kv_rel_l2: float = 1e-2


TARGET = Tolerances()


def rel_l2(a: np.ndarray, b: np.ndarray) -> float:
    den = float(np.linalg.norm(b))
    return float(np.linalg.norm(a - b)) / (den if den > 0 else 1.0)


class Lockstep:
    def __init__(self, shape, seed: int, template, *, C_max: int, device="cuda:0", lazy_oracle=False,
                 check_hidden=True, tol: Tolerances = TARGET, weights=None, model=None, gpu=None, seq: int = 0):
        """`gpu`, `seq`: compare sequence `seq` of an existing context of several sequences (the
        caller drives that context's passes and hands each sequence's record to `after_step`)."""
        from paper_2401_12522_b200 import Bita

        self.shape, self.template, self.tol = shape, template, tol
        w = weights if weights is not None else synth.make_weights(shape, seed, dtype=torch.bfloat16, device=device)
        if model is not None:
            self.model = model
        elif lazy_oracle:
            self.model = oracle_model_from_device(shape, w)
        else:
            self.model = oracle_model(shape, seed)
        self.blk = block_for(template, shape.n_mask)
        self.st = orc.State(self.model)
        self.seq = seq
        self.row0 = 0             # first row of this sequence in the debug buffers of the pass being compared
        self.owns_gpu = gpu is None
        self.gpu = Bita(shape, w, template, C_max=C_max, device=device) if gpu is None else gpu
        self.check_hidden = check_hidden
        if self.owns_gpu:
            self.gpu.enable_debug(True)
        self.adopted = 0          # passes where a sub-tolerance choice of the GPU was adopted
        self.exact = 0            # passes where every margin was above tolerance and records matched bit for bit
        self.layer_err = np.zeros(shape.L)    # per layer, worst pass: error the layer adds (see Tolerances)
        self.acc_err = np.zeros(shape.L)      # per layer, worst pass: accumulated distance of the streams
        self.max_logit = 0.0      # in units of RMS(logits)
        self.logit_per_pass: List[float] = []
        self.emitted: List[int] = []

    @property
    def max_hidden(self) -> float:
        return float(self.layer_err.max()) if len(self.layer_err) else 0.0

    @property
    def max_hidden_acc(self) -> float:
        return float(self.acc_err.max()) if len(self.acc_err) else 0.0

    def report(self) -> Dict:
        """The plain numbers of the run, for the parity table."""
        return dict(config=self.shape.name, layers=self.shape.L, rows=self.blk.M, passes=self.exact + self.adopted,
                    exact=self.exact, adopted=self.adopted, layer_rel_l2_max=self.max_hidden,
                    hidden_rel_l2_final=float(self.acc_err[-1]), hidden_rel_l2_max=self.max_hidden_acc,
                    hidden_rel_l2_per_layer=[float(f"{v:.3e}") for v in self.acc_err],
                    logit_max_over_rms=self.max_logit, tolerances=dict(self.tol.__dict__))

    # ------------------------------------------------------------------ pieces
    def _gpu_hidden(self, l: int, rows: int) -> np.ndarray:
        return self.gpu.debug_hidden(l, self.row0 + rows)[self.row0:].cpu().numpy().astype(np.float64)

    def _slab(self, cache: torch.Tensor, l: int) -> torch.Tensor:
        """[H_kv][C_max][D] of this sequence in layer l (the cache of a batch context has a sequence axis)."""
        return cache[l] if cache.dim() == 4 else cache[l, self.seq]

    def _layer_on_gpu_input(self, l, lw, rows, x0, pos, C, vis, sees_prompt) -> np.ndarray:
        """The oracle's layer l applied to the GPU's own input of that layer (its residual stream
        after layer l - 1, its cache as context)."""
        x_in = x0 if l == 0 else self._gpu_hidden(l - 1, rows)
        ck = self._slab(self.gpu.k_cache, l)[:, :C, :].double().cpu().numpy()
        cv = self._slab(self.gpu.v_cache, l)[:, :C, :].double().cpu().numpy()
        return orc._layer(self.model, lw, x_in, pos, ck, cv, vis, sees_prompt)[0]

    def _observe_layers(self, rows, x0, pos, C, vis, sees_prompt) -> Optional[Dict]:
        """With lazily converted weights (full-depth models) the per-layer references are computed as
        the oracle's own pass touches each layer, so that every layer is converted once per pass.
        Returns the dict that fills up during that pass, or None when the weights are plain lists."""
        layers = self.model.w["layers"]
        if not self.check_hidden or not hasattr(layers, "observer"):
            return None
        got: Dict[int, np.ndarray] = {}

        def see(l, lw):
            got[l] = self._layer_on_gpu_input(l, lw, rows, x0, pos, C, vis, sees_prompt)
        layers._cache = (None, None)
        layers.observer = see
        return got

    def _stop_observing(self):
        layers = self.model.w["layers"]
        if hasattr(layers, "observer"):
            layers.observer = None

    def _compare_float(self, rec_o: Dict, rows: int, x0: np.ndarray, pos: np.ndarray, C: int, vis: np.ndarray,
                       sees_prompt: np.ndarray, teacher: Optional[Dict] = None):
        """Hidden states per layer and logits of one pass.  x0/pos/C/vis/sees_prompt are the inputs the
        oracle's layer stack was given for these rows (C = cache slots every row sees)."""
        tol = self.tol
        if self.check_hidden:
            for l in range(self.shape.L):
                g = self._gpu_hidden(l, rows)
                acc = rel_l2(g, rec_o["hidden"][l])
                ref = teacher[l] if teacher is not None and l in teacher else \
                    self._layer_on_gpu_input(l, self.model.w["layers"][l], rows, x0, pos, C, vis, sees_prompt)
                own = rel_l2(g, ref)
                self.layer_err[l] = max(self.layer_err[l], own)
                self.acc_err[l] = max(self.acc_err[l], acc)
                assert own <= tol.layer_rel_l2, f"hidden layer {l}: the layer adds rel L2 {own:.3e} (allowed {tol.layer_rel_l2:.1e})"
                assert acc <= tol.hidden_rel_l2, f"hidden layer {l}: accumulated rel L2 {acc:.3e} (allowed {tol.hidden_rel_l2:.1e})"
        gl = self.gpu.debug_logits(self.row0 + rows)[self.row0:].cpu().numpy()
        ol = rec_o["logits"]
        rms = float(np.sqrt(np.mean(ol * ol)))
        err = float(np.abs(gl.astype(np.float64) - ol).max()) / rms
        self.max_logit = max(self.max_logit, err)
        self.logit_per_pass.append(err)
        assert err <= tol.logit_rms, f"logits: max|delta| = {err:.3e} x RMS (allowed {tol.logit_rms:.1e})"
        return gl, rms * tol.logit_rms

    @staticmethod
    def _select(gl_row: np.ndarray, k: int):
        order = np.argsort(-gl_row, kind="stable")[:k]
        return order.astype(np.int64)

    def _validate_choice(self, ol_row: np.ndarray, ids: Sequence[int], tol: float) -> bool:
        """True when the choice is the oracle's own; asserts it is at least within tolerance of it."""
        k = len(ids)
        o_ids, o_vals = orc.topk_sorted(ol_row, k)
        same = list(o_ids) == [int(i) for i in ids]
        for j, i in enumerate(ids):
            assert abs(ol_row[int(i)] - o_vals[j]) <= tol, "selected token is not within tolerance of the oracle's"
        if not same:
            # a differing pick is only legitimate where the oracle's own margin is below tolerance
            nxt = np.sort(ol_row)[::-1][: k + 1]
            gaps = nxt[:-1] - nxt[1:]
            assert gaps.min() <= tol, "selection differs although every oracle margin exceeds the tolerance"
        return same

    def _check_cache(self, upto: int, since: int = 0):
        L = self.shape.L
        for l in range(L):
            for name, gcache, ocache in (("k", self.gpu.k_cache, self.st.k), ("v", self.gpu.v_cache, self.st.v)):
                g = self._slab(gcache, l)[:, since:upto, :].float().cpu().numpy().astype(np.float64)
                o = ocache[l][:, since:upto, :]
                e = rel_l2(g, o)
                assert e <= self.tol.kv_rel_l2, f"cache {name} layer {l}: rel L2 {e:.3e}"

    # ------------------------------------------------------------------ passes
    def prefill(self, prompt: Sequence[int]):
        rec_g = self.gpu.prefill(prompt, seq=self.seq)
        self.row0 = 0             # the first pass takes one sequence at a time: its rows start the buffers
        T = len(prompt)
        n = self.shape.n_mask
        # the library runs the first pass in equal blocks of at most MAX_ROWS - 8 query rows; the debug
        # buffers hold the last block only
        from paper_2401_12522_b200 import MAX_ROWS
        cap = MAX_ROWS - 8
        blocks_left, last_start = -(-T // cap), 0
        while blocks_left > 1:
            last_start += -(-(T - last_start) // blocks_left)
            blocks_left -= 1
        rows = T - last_start + n
        # inputs of the last block as the oracle's first pass sets them up: token and mask embeddings,
        # consecutive positions, causal visibility inside the block, the earlier blocks as context
        x0 = np.concatenate([np.asarray(self.model.w["tok_emb"], dtype=np.float64)[np.asarray(prompt[last_start:])],
                             np.asarray(self.model.w["mask_emb"], dtype=np.float64)[:n]])
        sp = np.zeros(rows, dtype=bool)
        sp[rows - n:] = True
        layer_in = (rows, x0, last_start + np.arange(rows), last_start, np.tril(np.ones((rows, rows), dtype=bool)), sp)
        teacher = self._observe_layers(*layer_in)
        try:
            rec_o = orc.prefill(self.model, self.blk, self.st, prompt)
        finally:
            self._stop_observing()
        sub = dict(hidden=[h[last_start:] for h in rec_o["hidden"]], logits=rec_o["logits"][last_start:])
        gl, tol = self._compare_float(sub, *layer_in, teacher=teacher)
        ol = sub["logits"]
        a_g = int(self._select(gl[T - last_start - 1], 1)[0])
        same = self._validate_choice(ol[T - last_start - 1], [a_g], tol)
        topk = np.zeros((1, n, self.blk.k_max), dtype=np.int64)
        for i in range(n):
            topk[0, i] = self._select(gl[T - last_start + i], self.blk.k_max)
            same &= self._validate_choice(ol[T - last_start + i], topk[0, i], tol)
        tree = []
        for i in range(self.blk.N):
            m = self.blk.depth[i] - 1
            tree.append(int(topk[0, m, self.blk.rank[i]]) if m < n else -1)
        assert rec_g["n_out"] == 1 and rec_g["out_tokens"] == [a_g]
        assert rec_g["next_tree"] == tree
        assert rec_g["new_len"] == self.st.C == T
        if not same:
            self.adopted += 1
            self.st.root, self.st.tree = a_g, tree
        else:
            assert self.st.root == a_g and self.st.tree == tree
            self.exact += 1
        self._check_cache(T)
        self.emitted.append(a_g)
        return rec_g

    def step(self, tree_tokens: Optional[Sequence[int]] = None):
        blk = self.blk
        toks = list(self.st.tree if tree_tokens is None else tree_tokens)
        C0 = self.st.C
        rec_g = self.gpu.step(None if tree_tokens is None else toks)
        return self.after_step(rec_g, toks, C0)

    def after_step(self, rec_g: Dict, toks: Sequence[int], C0: int, row0: int = 0):
        """Compares one sequence's share of a finished pass (its record, its rows of the debug
        buffers from `row0` on, its cache) with the oracle's pass from the same state."""
        blk = self.blk
        self.row0 = row0
        layer_in = (blk.M, orc.embed_block(self.model, blk, self.st.root, toks), C0 + blk.rel_pos, C0, blk.vis,
                    blk.sees_prompt)
        teacher = self._observe_layers(*layer_in)
        try:
            rec_o = orc.bita_step(self.model, blk, self.st, toks, keep=False)
        finally:
            self._stop_observing()
        gl, tol = self._compare_float(rec_o, *layer_in, teacher=teacher)
        ol = rec_o["logits"]
        same = True
        row_argmax = []
        for r in range(1 + blk.N):
            a = int(self._select(gl[r], 1)[0])
            row_argmax.append(a)
            if r == 0 or toks[r - 1] >= 0:          # rows of disabled nodes carry no meaning
                same &= self._validate_choice(ol[r], [a], tol)
        topk = np.zeros((blk.G, blk.n, blk.k_max), dtype=np.int64)
        for g in range(blk.G):
            for i in range(blk.n):
                topk[g, i] = self._select(gl[blk.mask_row(g, i)], blk.k_max)
                same &= self._validate_choice(ol[blk.mask_row(g, i)], topk[g, i], tol)
        # integer work must be exact given the selections
        acc, out, cur = orc.verify_walk(blk, toks, row_argmax)
        nt = orc.next_tree(blk, topk, cur)
        assert rec_g["n_out"] == len(out)
        assert rec_g["out_tokens"] == out
        assert rec_g["accepted_idx"] == acc
        assert rec_g["next_tree"] == nt
        assert rec_g["new_len"] == C0 + 1 + len(acc)
        assert rec_g["status"] == 0
        assert 1 <= rec_g["n_out"] <= blk.max_depth + 1
        if same:
            # every margin above tolerance: the oracle's own record must be identical
            assert rec_o["out_tokens"] == out and rec_o["accepted_idx"] == acc and rec_o["next_tree"] == nt
            self.exact += 1
        else:
            self.adopted += 1
            rec_o = dict(rec_o, out_tokens=out, accepted_idx=acc, next_tree=nt, n_out=len(out))
        orc.commit_step(self.st, rec_o)
        assert self.st.C == rec_g["new_len"]
        self._check_cache(self.st.C, since=C0)
        self.emitted.extend(out)
        return rec_g

    def close(self):
        if self.owns_gpu:
            self.gpu.close()


class BatchLockstep:
    """Several sequences decoded together by one context, each compared with its own oracle run:
    every sequence has its own prompt (different lengths), cache, tree and accepted length."""

    def __init__(self, shape, seed: int, template, batch: int, *, C_max: int, device="cuda:0", tol: Tolerances = TARGET,
                 lazy_oracle=False, weights=None):
        from paper_2401_12522_b200 import Bita
        w = weights if weights is not None else synth.make_weights(shape, seed, dtype=torch.bfloat16, device=device)
        self.gpu = Bita(shape, w, template, C_max=C_max, device=device, batch=batch)
        self.gpu.enable_debug(True)
        model = oracle_model_from_device(shape, w) if lazy_oracle else oracle_model(shape, seed)
        self.seqs = [Lockstep(shape, seed, template, C_max=C_max, device=device, tol=tol, weights=w, model=model,
                              gpu=self.gpu, seq=b) for b in range(batch)]
        self.M = self.seqs[0].blk.M

    def prefill(self, prompts: Sequence[Sequence[int]]):
        return [ls.prefill(p) for ls, p in zip(self.seqs, prompts)]

    def step(self, trees: Optional[Sequence[Optional[Sequence[int]]]] = None):
        """`trees`: per sequence a token list, or None = all sequences verify the trees they drafted."""
        toks = [list(ls.st.tree) for ls in self.seqs] if trees is None else [list(t) for t in trees]
        C0 = [ls.st.C for ls in self.seqs]
        recs = self.gpu.step_batch(None if trees is None else toks)
        for b, ls in enumerate(self.seqs):
            ls.after_step(recs[b], toks[b], C0[b], row0=b * self.M)
        return recs

    def close(self):
        self.gpu.close()


def run_lockstep(shape, seed, template, n_steps, *, prompt=None, tree_fn=None, C_max=None, **kw) -> Lockstep:
    if prompt is None:
        prompt = prompt_tokens(seed, shape.prompt_len, shape.V)
    blk_rows = 1 + template.N + template.G * shape.n_mask
    if C_max is None:
        C_max = len(prompt) + n_steps * 17 + blk_rows + 64
    ls = Lockstep(shape, seed, template, C_max=C_max, **kw)
    ls.prefill(prompt)
    for s in range(n_steps):
        toks = None if tree_fn is None else tree_fn(s, ls)
        ls.step(toks)
    return ls
