"""The no-allocation tree-attention entry point gives the same output as the regular one.

Some users of the library run where device memory cannot be allocated at call time (a frozen
memory pool, someone else's allocator, a latency path that must not trigger the device-wide
synchronisation an allocation brings).  For them the library keeps an 8 MiB scratch array in its
device image.  This file checks, through the C ABI, that the variant agrees with the regular entry
point on two calls in a row - the second with other shapes, so that what the first call left in the
shared array cannot leak into the result - and that an oversized problem is refused cleanly.
It is collected last on purpose.
"""
import numpy as np
import pytest
import torch

import synth
from lockstep import rel_l2
from test_gpu_parity import _random_attention_case

pytestmark = pytest.mark.gpu


def test_static_scratch_attention_matches_regular_entry_point_twice():
    from paper_2401_12522_b200 import bita_tree_attention, bita_tree_attention_static
    cases = [(2, 16, 8, 2, 128, 16, 300), (1, 40, 4, 4, 64, 16, 77)]
    for call, (B, N, H, H_kv, D, P, C) in enumerate(cases):
        tmpl = synth.random_recursive_template(N + 1, N)
        M = 1 + N + 4
        q, k, v, pk, pv, vis, sp, ctx, blk = _random_attention_case(11 + call, B, M, H, H_kv, D, P, C, tmpl)
        ref = bita_tree_attention(q, k, v, vis, pk, pv, sp, ctx, H_kv=H_kv, P=P)
        out = torch.full_like(ref, float("nan"))
        bita_tree_attention_static(q, k, v, vis, pk, pv, sp, ctx, out, H_kv=H_kv, P=P)
        torch.cuda.synchronize()
        a = out.float().cpu().numpy().astype(np.float64)
        b = ref.float().cpu().numpy().astype(np.float64)
        assert np.isfinite(a).all()
        assert rel_l2(a, b) < 6e-3
        assert np.abs(a - b).max() < 3e-2


def test_static_scratch_refuses_what_does_not_fit():
    from paper_2401_12522_b200 import BitaError, bita_tree_attention_static
    B, M, H, D = 8, 133, 32, 128                       # needs far more than 8 MiB of partials
    dev = "cuda:0"
    q = torch.zeros((B, M, H, D), dtype=torch.bfloat16, device=dev)
    k = torch.zeros((B, H, M + 8, D), dtype=torch.bfloat16, device=dev)
    vis = torch.zeros((B, M, (M + 31) // 32), dtype=torch.int32, device=dev)
    ctx = torch.zeros(B, dtype=torch.int32, device=dev)
    out = torch.zeros((B, M, H * D), dtype=torch.bfloat16, device=dev)
    with pytest.raises(BitaError) as e:
        bita_tree_attention_static(q, k, k, vis, None, None, None, ctx, out, H_kv=H, P=0)
    assert e.value.code == -8
