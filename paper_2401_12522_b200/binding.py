"""ctypes binding of ``include/bita.h``.  Names and argument order follow the header."""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libbita.so")

MAX_NODES, MAX_ROWS, MAX_DEPTH, MAX_TOPK, MAX_MASK, MAX_BATCH = 160, 352, 16, 16, 8, 16


class BitaError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib.bita_strerror(code).decode() if lib is not None else str(code)
        extra = f" (cudaError {lib.bita_last_cuda_error()})" if code == -5 else ""
        super().__init__(f"{where}: {msg}{extra}")


class ModelDims(C.Structure):
    _fields_ = [(k, C.c_int32) for k in ("L", "d", "H", "H_kv", "D", "F", "V", "P", "C_max")] + \
               [("rms_eps", C.c_float), ("rope_theta", C.c_float)]


class Weights(C.Structure):
    _fields_ = [(k, C.c_void_p) for k in ("tok_emb", "mask_emb", "g_final", "lm_head")] + \
               [(k, C.POINTER(C.c_void_p)) for k in
                ("wqkv", "wo", "wg", "wu", "wd", "g_attn", "g_ffn", "prompt_k", "prompt_v")]


class TreeTemplate(C.Structure):
    _fields_ = [("N", C.c_int32), ("parent", C.POINTER(C.c_int32)), ("rank", C.POINTER(C.c_int32)),
                ("G", C.c_int32), ("attach", C.POINTER(C.c_int32))]


class KV(C.Structure):
    _fields_ = [("k", C.c_void_p), ("v", C.c_void_p), ("C_max", C.c_int32)]


class StepOut(C.Structure):
    _fields_ = [("status", C.c_int32), ("n_out", C.c_int32), ("new_len", C.c_int32),
                ("out_tokens", C.c_int32 * (MAX_DEPTH + 1)), ("accepted_idx", C.c_int32 * MAX_DEPTH),
                ("next_tree", C.c_int32 * MAX_NODES)]


def _signatures():
    vp, i32, sz = C.c_void_p, C.c_int32, C.c_size_t
    return {
        "bita_workspace_bytes": [C.POINTER(ModelDims), C.POINTER(TreeTemplate), C.c_int, C.POINTER(sz)],
        "bita_init": [C.POINTER(vp), C.POINTER(ModelDims), C.POINTER(Weights), C.POINTER(TreeTemplate), C.c_int,
                      vp, sz, vp],
        "bita_workspace_bytes_batch": [C.POINTER(ModelDims), C.POINTER(TreeTemplate), C.c_int, i32, C.POINTER(sz)],
        "bita_init_batch": [C.POINTER(vp), C.POINTER(ModelDims), C.POINTER(Weights), C.POINTER(TreeTemplate), C.c_int,
                            i32, vp, sz, vp],
        "bita_prefill_seq": [vp, C.POINTER(KV), i32, C.POINTER(i32), i32, C.POINTER(StepOut)],
        "bita_step_batch": [vp, C.POINTER(KV), C.POINTER(i32), C.POINTER(StepOut)],
        "bita_step_batch_enqueue": [vp, C.POINTER(KV), vp],
        "bita_step_batch_finish": [vp, C.POINTER(StepOut)],
        "bita_rewind_seq": [vp, C.POINTER(KV), i32, i32, i32],
        "bita_batch": [vp],
        "bita_prefill": [vp, C.POINTER(KV), C.POINTER(i32), i32, C.POINTER(StepOut)],
        "bita_step": [vp, C.POINTER(KV), C.POINTER(i32), C.POINTER(StepOut)],
        "bita_step_enqueue": [vp, C.POINTER(KV), vp],
        "bita_step_finish": [vp, C.POINTER(StepOut)],
        "bita_reset": [vp, C.POINTER(KV)],
        "bita_rewind": [vp, C.POINTER(KV), i32, i32],
        "bita_set_debug_buffer": [vp, vp, sz],
        "bita_debug_fetch": [vp, C.c_int, vp, sz],
        "bita_set_wait_limit": [vp, C.c_uint64],
        "bita_probe_wait_timeout": [vp, C.c_uint64],
        "bita_set_attention_route": [C.c_int],
        "bita_set_kernel_timing": [vp, C.c_int],
        "bita_get_kernel_timing": [vp, C.POINTER(C.c_float), C.POINTER(i32)],
        "bita_block_rows": [vp],
        "bita_last_launch_count": [vp],
        "bita_last_cuda_error": [],
        "bita_gemm_workspace_bytes": [i32, i32, i32, C.POINTER(sz)],
        "bita_gemm_bf16": [vp, vp, vp, i32, i32, i32, vp, sz, vp],
        "bita_attention_workspace_bytes": [i32, i32, i32, i32, C.POINTER(sz)],
        "bita_attention_workspace_bytes_long": [i32, i32, i32, i32, i32, C.POINTER(sz)],
        "bita_tree_attention": [vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, vp, sz, vp],
        "bita_tree_attention_static": [vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, vp],
    }


def _load():
    if not os.path.exists(_LIB_PATH):
        raise ImportError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2401_12522_b200.build` "
            "(there is no fallback path)")
    L = C.CDLL(_LIB_PATH)
    for name, args in _signatures().items():
        fn = getattr(L, name)
        fn.argtypes = args
        fn.restype = C.c_int
    L.bita_destroy.argtypes = [C.c_void_p]
    L.bita_destroy.restype = None
    L.bita_strerror.argtypes = [C.c_int]
    L.bita_strerror.restype = C.c_char_p
    return L


lib = None
lib = _load()


def _check(code: int, where: str):
    if code != 0:
        raise BitaError(code, where)


def _ptr(t: Optional[torch.Tensor]):
    return C.c_void_p(0 if t is None else t.data_ptr())


def _stream_handle(stream) -> C.c_void_p:
    return C.c_void_p(0 if stream is None else stream.cuda_stream)


def _i32_array(vals: Sequence[int]):
    return (C.c_int32 * max(1, len(vals)))(*[int(v) for v in vals])


class Bita:
    """One decoding context: owns (through torch) the workspace and the KV cache it hands to the library."""

    def __init__(self, shape, weights: Dict, template, *, C_max: int, stream=None, device="cuda:0", batch: int = 1):
        self.device = torch.device(device)
        self.batch = batch
        self.stream = stream
        self.shape = shape
        self.template = template
        self.weights = weights                       # keep the tensors alive
        self.n_mask = shape.n_mask
        L = shape.L
        self.dims = ModelDims(L, shape.d, shape.H, shape.H_kv, shape.D, shape.F, shape.V, shape.P, C_max,
                              shape.rms_eps, shape.rope_theta)
        self._parent = _i32_array(template.parent)
        self._rank = _i32_array(template.rank)
        self._attach = _i32_array(template.attach)
        self.tmpl = TreeTemplate(template.N, self._parent, self._rank, template.G, self._attach)
        for name, t in self._all_tensors(weights):
            if t.dtype != torch.bfloat16 or not t.is_cuda or not t.is_contiguous():
                raise ValueError(f"weight {name} must be a contiguous bf16 CUDA tensor")
        self._arrs = {}
        w = Weights()
        for k in ("tok_emb", "mask_emb", "g_final", "lm_head"):
            setattr(w, k, weights[k].data_ptr())
        for k in ("wqkv", "wo", "wg", "wu", "wd", "g_attn", "g_ffn", "prompt_k", "prompt_v"):
            arr = (C.c_void_p * L)(*[weights["layers"][l][k].data_ptr() for l in range(L)])
            self._arrs[k] = arr
            setattr(w, k, C.cast(arr, C.POINTER(C.c_void_p)))
        self._w = w
        need = C.c_size_t(0)
        _check(lib.bita_workspace_bytes_batch(C.byref(self.dims), C.byref(self.tmpl), self.n_mask, batch,
                                              C.byref(need)), "bita_workspace_bytes_batch")
        self.workspace = torch.empty(need.value + 256, dtype=torch.uint8, device=self.device)
        ws_ptr = (self.workspace.data_ptr() + 255) // 256 * 256
        # [L][B][H_kv][C_max][D]; with one sequence the B axis is left out
        kv_shape = (L, shape.H_kv, C_max, shape.D) if batch == 1 else (L, batch, shape.H_kv, C_max, shape.D)
        self.k_cache = torch.zeros(kv_shape, dtype=torch.bfloat16, device=self.device)
        self.v_cache = torch.zeros(kv_shape, dtype=torch.bfloat16, device=self.device)
        self.kv = KV(self.k_cache.data_ptr(), self.v_cache.data_ptr(), C_max)
        self._ctx = C.c_void_p(0)
        torch.cuda.synchronize(self.device)
        _check(lib.bita_init_batch(C.byref(self._ctx), C.byref(self.dims), C.byref(w), C.byref(self.tmpl), self.n_mask,
                                   batch, C.c_void_p(ws_ptr), need.value, _stream_handle(stream)), "bita_init_batch")
        self.rows = lib.bita_block_rows(self._ctx)
        self._debug = None
        self._out = StepOut()
        self._outs = (StepOut * batch)()

    @staticmethod
    def _all_tensors(weights):
        for k, v in weights.items():
            if k == "layers":
                for l, lw in enumerate(v):
                    for kk, t in lw.items():
                        yield f"layers[{l}].{kk}", t
            else:
                yield k, v

    # ---- the three calls -------------------------------------------------------------------
    def prefill(self, tokens: Sequence[int], seq: int = 0) -> Dict:
        arr = _i32_array(tokens)
        _check(lib.bita_prefill_seq(self._ctx, C.byref(self.kv), seq, arr, len(tokens), C.byref(self._out)),
               "bita_prefill_seq")
        return self._record()

    # ---- several sequences in one pass ------------------------------------------------------
    def step_batch(self, tree_tokens: Optional[Sequence[Sequence[int]]] = None):
        """One pass over all sequences; `tree_tokens` = one token list per sequence, or None."""
        arr = None if tree_tokens is None else _i32_array([t for seq in tree_tokens for t in seq])
        _check(lib.bita_step_batch(self._ctx, C.byref(self.kv), arr, self._outs), "bita_step_batch")
        return [self._record(self._outs[b]) for b in range(self.batch)]

    def step_batch_enqueue(self, tree_tokens_dev: Optional[torch.Tensor] = None):
        if tree_tokens_dev is not None:
            assert tree_tokens_dev.dtype == torch.int32 and tree_tokens_dev.is_cuda and tree_tokens_dev.is_contiguous()
        _check(lib.bita_step_batch_enqueue(self._ctx, C.byref(self.kv), _ptr(tree_tokens_dev)), "bita_step_batch_enqueue")

    def step_batch_finish(self):
        _check(lib.bita_step_batch_finish(self._ctx, self._outs), "bita_step_batch_finish")
        return [self._record(self._outs[b]) for b in range(self.batch)]

    def step(self, tree_tokens: Optional[Sequence[int]] = None) -> Dict:
        arr = None if tree_tokens is None else _i32_array(tree_tokens)
        _check(lib.bita_step(self._ctx, C.byref(self.kv), arr, C.byref(self._out)), "bita_step")
        return self._record()

    def step_enqueue(self, tree_tokens_dev: Optional[torch.Tensor] = None):
        if tree_tokens_dev is not None:
            assert tree_tokens_dev.dtype == torch.int32 and tree_tokens_dev.is_cuda
        _check(lib.bita_step_enqueue(self._ctx, C.byref(self.kv), _ptr(tree_tokens_dev)), "bita_step_enqueue")

    def step_finish(self) -> Dict:
        _check(lib.bita_step_finish(self._ctx, C.byref(self._out)), "bita_step_finish")
        return self._record()

    def reset(self):
        _check(lib.bita_reset(self._ctx, C.byref(self.kv)), "bita_reset")

    def rewind(self, new_len: int, last_token: int, seq: int = 0):
        _check(lib.bita_rewind_seq(self._ctx, C.byref(self.kv), seq, new_len, last_token), "bita_rewind_seq")

    # ---- helpers ---------------------------------------------------------------------------
    def _record(self, o=None) -> Dict:
        o = self._out if o is None else o
        n = o.n_out
        return dict(status=o.status, n_out=n, new_len=o.new_len, out_tokens=list(o.out_tokens[:n]),
                    accepted_idx=list(o.accepted_idx[:max(0, n - 1)]), next_tree=list(o.next_tree[:self.template.N]))

    def enable_debug(self, on: bool = True):
        if on:
            n = self.shape.L * MAX_ROWS * self.shape.d + MAX_ROWS * self.shape.V
            self._debug = torch.zeros(n, dtype=torch.float32, device=self.device)
            _check(lib.bita_set_debug_buffer(self._ctx, _ptr(self._debug), n * 4), "bita_set_debug_buffer")
        else:
            _check(lib.bita_set_debug_buffer(self._ctx, C.c_void_p(0), 0), "bita_set_debug_buffer")
            self._debug = None

    def debug_hidden(self, layer: int, rows: int) -> torch.Tensor:
        d = self.shape.d
        off = layer * MAX_ROWS * d
        return self._debug[off: off + rows * d].view(rows, d)

    def debug_logits(self, rows: int) -> torch.Tensor:
        off = self.shape.L * MAX_ROWS * self.shape.d
        return self._debug[off: off + rows * self.shape.V].view(rows, self.shape.V)

    DEBUG_LOGITS, DEBUG_TOPK, DEBUG_HIDDEN = 1, 2, 1000

    def debug_fetch(self, what: int, rows: int) -> torch.Tensor:
        """What the last pass left behind, read back to the host through bita_debug_fetch."""
        if what == self.DEBUG_TOPK:
            out = torch.empty((rows, MAX_TOPK), dtype=torch.int32)
        elif what == self.DEBUG_LOGITS:
            out = torch.empty((rows, self.shape.V), dtype=torch.float32)
        else:
            out = torch.empty((rows, self.shape.d), dtype=torch.float32)
        _check(lib.bita_debug_fetch(self._ctx, what, C.c_void_p(out.data_ptr()), out.numel() * out.element_size()),
               "bita_debug_fetch")
        return out

    def set_wait_limit(self, limit_ns: int):
        _check(lib.bita_set_wait_limit(self._ctx, int(limit_ns)), "bita_set_wait_limit")

    def probe_wait_timeout(self, limit_ns: int) -> int:
        """Returns the status the self-check leaves (-6 = the bounded wait gave up, as it must)."""
        return lib.bita_probe_wait_timeout(self._ctx, int(limit_ns))

    def set_kernel_timing(self, on: bool):
        _check(lib.bita_set_kernel_timing(self._ctx, 1 if on else 0), "bita_set_kernel_timing")

    def kernel_timing(self):
        """(ms, launches) per family of the most recent pass: [projections, attention]."""
        ms = (C.c_float * 2)()
        n = (C.c_int32 * 2)()
        _check(lib.bita_get_kernel_timing(self._ctx, ms, n), "bita_get_kernel_timing")
        return list(ms), list(n)

    @property
    def last_launch_count(self) -> int:
        return lib.bita_last_launch_count(self._ctx)

    def close(self):
        if self._ctx:
            lib.bita_destroy(self._ctx)
            self._ctx = C.c_void_p(0)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def bita_gemm_bf16(X: torch.Tensor, W: torch.Tensor, stream=None) -> torch.Tensor:
    """Y[m][n] = sum_k X[m][k] W[n][k]; X [M,K] bf16, W [N,K] bf16 -> fp32 [M,N]."""
    M, K = X.shape
    N = W.shape[0]
    need = C.c_size_t(0)
    _check(lib.bita_gemm_workspace_bytes(M, N, K, C.byref(need)), "bita_gemm_workspace_bytes")
    ws = torch.empty(need.value + 256, dtype=torch.uint8, device=X.device)
    Y = torch.empty((M, N), dtype=torch.float32, device=X.device)
    wp = (ws.data_ptr() + 255) // 256 * 256
    _check(lib.bita_gemm_bf16(_ptr(X), _ptr(W), _ptr(Y), M, N, K, C.c_void_p(wp), need.value, _stream_handle(stream)),
           "bita_gemm_bf16")
    return Y


def bita_tree_attention(q, k, v, vis, prompt_k, prompt_v, sees_prompt, ctx_len, *, H_kv, P, workspace=None,
                        out=None, stream=None):
    """q [B,M,H,D] bf16; k,v [B,H_kv,C_max,D]; vis int32 [B,M,W] (bit patterns); ctx_len int32 [B] -> [B,M,H*D]."""
    B, M, H, D = q.shape
    C_max = k.shape[2]
    need = C.c_size_t(0)
    _check(lib.bita_attention_workspace_bytes_long(B, M, H, D, C_max, C.byref(need)),
           "bita_attention_workspace_bytes_long")
    if workspace is None and need.value:
        workspace = torch.empty(need.value + 256, dtype=torch.uint8, device=q.device)
    wp = 0 if workspace is None else (workspace.data_ptr() + 255) // 256 * 256
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size() - (wp - workspace.data_ptr())
    if out is None:
        out = torch.empty((B, M, H * D), dtype=torch.bfloat16, device=q.device)
    _check(lib.bita_tree_attention(_ptr(q), _ptr(k), _ptr(v), _ptr(vis), _ptr(prompt_k), _ptr(prompt_v),
                                   _ptr(sees_prompt), _ptr(ctx_len), _ptr(out), B, M, H, H_kv, D, P, C_max,
                                   C.c_void_p(wp), max(0, ws_bytes), _stream_handle(stream)), "bita_tree_attention")
    return out


def set_attention_route(route: int):
    """0 = key slices merge inside a thread-block cluster (default), 1 = always through the workspace."""
    _check(lib.bita_set_attention_route(int(route)), "bita_set_attention_route")


STATIC_SCRATCH_BYTES = 8 << 20


def bita_tree_attention_static(q, k, v, vis, prompt_k, prompt_v, sees_prompt, ctx_len, out, *, H_kv, P, stream=None):
    """Tree attention without any device allocation by the library: the caller passes inputs and
    the output tensor, the split-KV scratch is the library's built-in array (8 MiB per GPU).

    For callers that cannot allocate at call time (frozen memory pool, foreign allocator, no
    device-wide sync allowed).  Raises BitaError(-8) when the problem needs more scratch than the
    array holds.  Calls that overlap on the GPU share the array and race; keep them ordered.
    """
    B, M, H, D = q.shape
    C_max = k.shape[2]
    _check(lib.bita_tree_attention_static(_ptr(q), _ptr(k), _ptr(v), _ptr(vis), _ptr(prompt_k), _ptr(prompt_v),
                                          _ptr(sees_prompt), _ptr(ctx_len), _ptr(out), B, M, H, H_kv, D, P, C_max,
                                          _stream_handle(stream)), "bita_tree_attention_static")
    return out
