"""The no-allocation tree-attention entry point: right results out of its built-in scratch.

Some users of the library run where device memory cannot be allocated at call time (a frozen
memory pool, someone else's allocator, a latency path that must not trigger the device-wide
synchronisation an allocation brings).  For them the library keeps an 8 MiB scratch array in its
device image, and `bita_tree_attention_static` sends the partial results of its key slices through
that array to the merge kernel.  This file checks, through the C ABI, on two calls in a row - the
second with other shapes, so that what the first call left in the shared array cannot leak into the
result - that the output agrees with the CPU oracle and with the regular entry point, that the
call leaves the device's free memory and torch's allocation counters untouched, that a problem
whose partial results exceed the array is refused cleanly, and that one needing no scratch at all
is accepted whatever its size.  It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

import synth
from lockstep import rel_l2
from test_gpu_parity import _random_attention_case, check_attention_against_oracle

pytestmark = pytest.mark.gpu


def test_static_scratch_attention_matches_oracle_and_regular_entry_twice():
    from paper_2401_12522_b200 import bita_tree_attention, bita_tree_attention_static
    from paper_2401_12522_b200.binding import lib
    import ctypes as C
    # both shapes take several key slices (6 and 8), so the array is written and read back
    cases = [(2, 16, 8, 2, 128, 16, 300), (1, 40, 4, 4, 64, 16, 77)]
    for call, (B, N, H, H_kv, D, P, Cn) in enumerate(cases):
        tmpl = synth.random_recursive_template(N + 1, N)
        M = 1 + N + 4
        need = C.c_size_t(0)
        assert lib.bita_attention_workspace_bytes(B, M, H, D, C.byref(need)) == 0 and need.value > 0
        q, k, v, pk, pv, vis, sp, ctx, blk = _random_attention_case(11 + call, B, M, H, H_kv, D, P, Cn, tmpl)
        ref = bita_tree_attention(q, k, v, vis, pk, pv, sp, ctx, H_kv=H_kv, P=P)
        out = torch.full_like(ref, float("nan"))
        torch.cuda.synchronize()
        free0, _ = torch.cuda.mem_get_info()
        alloc0, reserved0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
        bita_tree_attention_static(q, k, v, vis, pk, pv, sp, ctx, out, H_kv=H_kv, P=P)
        torch.cuda.synchronize()
        if call > 0:                                           # the first call on a device may load the kernels' code
            assert torch.cuda.mem_get_info()[0] == free0
        assert (torch.cuda.memory_allocated(), torch.cuda.memory_reserved()) == (alloc0, reserved0)
        check_attention_against_oracle(out, q, k, v, pk, pv, ctx, blk, H_kv, P)
        a = out.float().cpu().numpy().astype(np.float64)
        b = ref.float().cpu().numpy().astype(np.float64)
        assert rel_l2(a, b) < 6e-3
        assert np.abs(a - b).max() < 3e-2


def _zeros_case(B, M, H, D):
    dev = "cuda:0"
    q = torch.zeros((B, M, H, D), dtype=torch.bfloat16, device=dev)
    k = torch.zeros((B, H, M + 8, D), dtype=torch.bfloat16, device=dev)
    vis = torch.zeros((B, M, (M + 31) // 32), dtype=torch.int32, device=dev)
    ctx = torch.zeros(B, dtype=torch.int32, device=dev)
    out = torch.zeros((B, M, H * D), dtype=torch.bfloat16, device=dev)
    return q, k, vis, ctx, out


def test_static_scratch_refuses_what_does_not_fit_and_accepts_what_needs_none():
    from paper_2401_12522_b200 import BitaError, bita_tree_attention_static
    # 32 heads x 4 key slices x 133 rows of partial results: 8.4 MiB, more than the array holds
    q, k, vis, ctx, out = _zeros_case(1, 133, 32, 128)
    with pytest.raises(BitaError) as e:
        bita_tree_attention_static(q, k, k, vis, None, None, None, ctx, out, H_kv=32, P=0)
    assert e.value.code == -8
    # 8 sequences x 32 heads: one key slice each, no scratch needed, accepted at any size
    q, k, vis, ctx, out = _zeros_case(8, 133, 32, 128)
    bita_tree_attention_static(q, k, k, vis, None, None, None, ctx, out, H_kv=32, P=0)
    torch.cuda.synchronize()
