"""Lockstep comparison of the CUDA library with the CPU oracle on the same seeded inputs.

Both sides start every pass from the same (cache, last token, tree).  Random-init logits are nearly
flat, so an argmax or a top-k slot may legitimately differ where the oracle's own margin is below
the logit tolerance; such a choice is validated against the oracle's logits and then adopted by the
oracle so that the run stays in lockstep.  Everything else must match exactly (tokens, accepted
length, accepted indices, next tree, cache length) or within the stated tolerances (hidden states,
logits, cache contents).
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from helpers import block_for, oracle_model, orc, prompt_tokens, synth

# tolerances of the parity target
HIDDEN_REL_L2 = 1e-2          # error a layer adds, relative L2 over the whole block (see layer_increment)
LOGIT_TOL_RMS = 3e-2          # max |delta| <= 3e-2 * RMS(oracle logits) ...
LOGIT_TOL_PER_HIDDEN = 6.0    # ... or 6 x the accumulated hidden error of the worst row where that is larger (see _compare_float)
KV_REL_L2 = 1e-2              # cache contents are bf16 roundings of the oracle's fp64 values


def layer_increment(err_abs: float, prev_err_abs: float, ref_norm: float) -> float:
    """Error added by one layer, relative to that layer's output.

    The residual stream carries the error of the earlier layers along (x_l = x_{l-1} + f(x_{l-1})), so
    the distance ||gpu_l - oracle_l|| is the accumulated error of all layers so far.  bf16 operands
    give every layer a rounding error of some 0.5 % of its output; these add in quadrature.  The
    per-layer bound is therefore applied to the part layer l added: sqrt(E_l^2 - E_{l-1}^2) / ||x_l||.
    """
    inc2 = max(0.0, err_abs * err_abs - prev_err_abs * prev_err_abs)
    return float(np.sqrt(inc2)) / (ref_norm if ref_norm > 0 else 1.0)


def rel_l2(a: np.ndarray, b: np.ndarray) -> float:
    den = float(np.linalg.norm(b))
    return float(np.linalg.norm(a - b)) / (den if den > 0 else 1.0)


class Lockstep:
    def __init__(self, shape, seed: int, template, *, C_max: int, device="cuda:0", lazy_oracle=False,
                 check_hidden=True):
        from paper_2401_12522_b200 import Bita

        self.shape, self.template = shape, template
        self.model = oracle_model(shape, seed, lazy=lazy_oracle)
        self.blk = block_for(template, shape.n_mask)
        self.st = orc.State(self.model)
        w = synth.make_weights(shape, seed, dtype=torch.bfloat16, device=device)
        self.gpu = Bita(shape, w, template, C_max=C_max, device=device)
        self.check_hidden = check_hidden
        self.gpu.enable_debug(True)
        self.adopted = 0          # passes where a sub-tolerance choice of the GPU was adopted
        self.exact = 0            # passes where every margin was above tolerance and records matched bit for bit
        self.max_hidden = 0.0     # largest per-layer increment
        self.max_hidden_acc = 0.0 # largest accumulated hidden error
        self.max_logit = 0.0      # in units of RMS(logits)
        self.emitted: List[int] = []

    # ------------------------------------------------------------------ pieces
    def _compare_float(self, rec_o: Dict, rows: int):
        acc_rel = 0.0
        if self.check_hidden:
            prev = 0.0
            for l in range(self.shape.L):
                g = self.gpu.debug_hidden(l, rows).cpu().numpy().astype(np.float64)
                o = rec_o["hidden"][l]
                err_abs = float(np.linalg.norm(g - o))
                ref = float(np.linalg.norm(o))
                e = layer_increment(err_abs, prev, ref)
                prev = err_abs
                # A row of logits inherits the error of its own row of the hidden state, and the rows
                # differ (mask rows sit further out than tree rows): the logits are bounded with the
                # worst row, the per-layer criterion stays on the whole block.
                row_ref = np.linalg.norm(o, axis=-1)
                row_rel = np.linalg.norm(g - o, axis=-1) / np.where(row_ref > 0, row_ref, 1.0)
                acc_rel = max(err_abs / (ref if ref > 0 else 1.0), float(row_rel.max()))
                self.max_hidden = max(self.max_hidden, e)
                self.max_hidden_acc = max(self.max_hidden_acc, acc_rel)
                assert e <= HIDDEN_REL_L2, f"hidden layer {l}: adds rel L2 {e:.3e} (accumulated {acc_rel:.3e})"
        gl = self.gpu.debug_logits(rows).cpu().numpy()
        ol = rec_o["logits"]
        rms = float(np.sqrt(np.mean(ol * ol)))
        err = float(np.abs(gl.astype(np.float64) - ol).max()) / rms
        self.max_logit = max(self.max_logit, err)
        # The logits inherit the accumulated error of the hidden state; their largest deviation over
        # rows x V entries sits some 5-6 standard deviations out.  Beyond the 3e-2 x RMS target the
        # check is that the LM head adds nothing of its own.
        tol_rel = max(LOGIT_TOL_RMS, LOGIT_TOL_PER_HIDDEN * acc_rel)
        assert err <= tol_rel, f"logits: max|delta| = {err:.3e} x RMS (allowed {tol_rel:.3e})"
        return gl, rms * tol_rel

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
                g = gcache[l, :, since:upto, :].float().cpu().numpy().astype(np.float64)
                o = ocache[l][:, since:upto, :]
                e = rel_l2(g, o)
                assert e <= KV_REL_L2, f"cache {name} layer {l}: rel L2 {e:.3e}"

    # ------------------------------------------------------------------ passes
    def prefill(self, prompt: Sequence[int]):
        rec_g = self.gpu.prefill(prompt)
        rec_o = orc.prefill(self.model, self.blk, self.st, prompt)
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
        sub = dict(hidden=[h[last_start:] for h in rec_o["hidden"]], logits=rec_o["logits"][last_start:])
        gl, tol = self._compare_float(sub, rows)
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
        rec_o = orc.bita_step(self.model, blk, self.st, toks, keep=False)
        gl, tol = self._compare_float(rec_o, blk.M)
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
