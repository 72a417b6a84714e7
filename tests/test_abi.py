"""The C-ABI library loads, exports every symbol the header declares, and rejects bad arguments on
the host before anything is launched (no GPU needed: none of these calls touches the device)."""
import ctypes as C
import os
import re

import pytest

import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "bita.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bita_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2401_12522_b200 import binding
    names = _declared_symbols()
    assert "bita_init" in names and "bita_step" in names and "bita_reset" in names
    raw = C.CDLL(os.path.join(ROOT, "paper_2401_12522_b200", "libbita.so"))
    for n in names:
        assert hasattr(raw, n), f"{n} declared in bita.h but not exported"
    # and the binding covers them
    covered = set(binding._signatures()) | {"bita_destroy", "bita_strerror"}
    assert set(names) <= covered


def test_struct_sizes_match_header_constants():
    from paper_2401_12522_b200 import binding as b
    text = open(os.path.join(ROOT, "include", "bita.h")).read()
    consts = {k: int(v) for k, v in re.findall(r"#define (BITA_MAX_[A-Z]+) (\d+)", text)}
    assert consts == {"BITA_MAX_NODES": b.MAX_NODES, "BITA_MAX_ROWS": b.MAX_ROWS, "BITA_MAX_DEPTH": b.MAX_DEPTH,
                      "BITA_MAX_TOPK": b.MAX_TOPK, "BITA_MAX_MASK": b.MAX_MASK, "BITA_MAX_BATCH": b.MAX_BATCH}
    assert C.sizeof(b.StepOut) == 4 * (3 + b.MAX_DEPTH + 1 + b.MAX_DEPTH + b.MAX_NODES)
    assert C.sizeof(b.ModelDims) == 44


def _dims(shape, C_max=256):
    from paper_2401_12522_b200 import binding as b
    return b.ModelDims(shape.L, shape.d, shape.H, shape.H_kv, shape.D, shape.F, shape.V, shape.P, C_max,
                       shape.rms_eps, shape.rope_theta)


def _tmpl(parent, rank, attach):
    from paper_2401_12522_b200 import binding as b
    keep = (b._i32_array(parent), b._i32_array(rank), b._i32_array(attach))
    return b.TreeTemplate(len(parent), keep[0], keep[1], len(attach), keep[2]), keep


def test_host_side_validation():
    from paper_2401_12522_b200 import binding as b
    lib = b.lib
    shape = synth.CONFIGS["tiny"]
    t = synth.product_rule_template(shape.tree_K, shape.tree_B)
    tm, keep = _tmpl(t.parent, t.rank, t.attach)
    need = C.c_size_t(0)
    d = _dims(shape)
    assert lib.bita_workspace_bytes(C.byref(d), C.byref(tm), shape.n_mask, C.byref(need)) == 0
    assert need.value > 0 and need.value % 256 == 0
    # unsupported head dimension
    bad = _dims(shape)
    bad.D = 96
    assert lib.bita_workspace_bytes(C.byref(bad), C.byref(tm), shape.n_mask, C.byref(need)) == -1
    # a parent that does not precede its child
    tm2, keep2 = _tmpl([-1, 1], [0, 0], [-1])
    assert lib.bita_workspace_bytes(C.byref(d), C.byref(tm2), shape.n_mask, C.byref(need)) == -2
    # two groups on one attach point
    tm3, keep3 = _tmpl([-1], [0], [-1, -1])
    assert lib.bita_workspace_bytes(C.byref(d), C.byref(tm3), shape.n_mask, C.byref(need)) == -2
    # a mask group on every node of the 64-node tree: 1 + 64 + 65 * 4 = 325 rows fit, 65 * 5 + 65 = 390 do not
    big = synth.product_rule_template((10, 6, 4, 2), (10, 6, 6, 4), per_node_groups=True)
    tm4, keep4 = _tmpl(big.parent, big.rank, big.attach)
    assert lib.bita_workspace_bytes(C.byref(d), C.byref(tm4), 4, C.byref(need)) == 0
    assert lib.bita_workspace_bytes(C.byref(d), C.byref(tm4), 5, C.byref(need)) == -2
    # rank beyond the top-k width
    tm5, keep5 = _tmpl([-1], [16], [-1])
    assert lib.bita_workspace_bytes(C.byref(d), C.byref(tm5), shape.n_mask, C.byref(need)) == -2
    # several sequences: the rows of all of them share one block (19 rows each here)
    assert lib.bita_workspace_bytes_batch(C.byref(d), C.byref(tm), shape.n_mask, 16, C.byref(need)) == 0
    assert lib.bita_workspace_bytes_batch(C.byref(d), C.byref(tm), shape.n_mask, 17, C.byref(need)) == -1
    assert lib.bita_workspace_bytes_batch(C.byref(d), C.byref(tm), shape.n_mask, 0, C.byref(need)) == -1
    assert lib.bita_workspace_bytes_batch(C.byref(d), C.byref(tm4), 4, 2, C.byref(need)) == -2     # 2 x 325 rows
    assert lib.bita_step_batch(None, None, None, C.byref(out0 := b.StepOut())) == -1
    # null context
    out = b.StepOut()
    assert lib.bita_step(None, None, None, C.byref(out)) == -1
    assert lib.bita_step_finish(None, C.byref(out)) == -1
    assert lib.bita_strerror(-3) == b"KV cache full"
    assert lib.bita_gemm_workspace_bytes(400, 8, 8, C.byref(need)) == -1
    assert lib.bita_gemm_workspace_bytes(4, 8, 12, C.byref(need)) == -1
    assert lib.bita_attention_workspace_bytes(1, 19, 4, 96, C.byref(need)) == -1
