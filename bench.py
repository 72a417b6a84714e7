"""Benchmark of the BiTA decoding pass on B200: accepted tokens/s and bita_step latency at batch 1.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 7b|13b|70b|tiny] [--planted F]
    python bench.py --impl reference ...      # the CPU oracle, timed on the host cores

One "step" is one bita_step: the whole pass (pack, layer stack with tree attention, LM head,
selection, verification walk, next tree, cache compaction) over one packed block.  Inputs are
seeded and synthetic (random-init weights of the named shape, uniform-random prompt, draft trees
with a planted fraction of true continuations).  Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

import synth  # noqa: E402

MODEL_SEED = 0x5EED0001
PROMPT_SEED = 0x5EED1001
PLANT_SEED = 0x5EED2001
METRIC = "accepted_tokens_per_s"
UNIT = "tokens/s"


# DRAM bytes (read + write) per projection launch with the 69-row block (q/k/v, O, gate/up, down per
# layer; LM head), from the ncu captures of small cases of the same kernels summarised in
# profiles/k_gemm_tc_k_attn_umma_7b_ncu_full.md and profiles/k_gemm_tc_70b_width_ncu_full.md (one or two
# layers of the width; traffic per launch does not depend on the depth, so a pass is L x the layer's
# launches + the head's).  The 13B width has no capture: its `traffic` is null.
NCU_TRAFFIC = {
    "7b": {"per_layer": 105.16e6 + 35.45e6 + 184.81e6 + 96.93e6, "head": 266.94e6},
    "70b": {"per_layer": 173.88e6 + 141.25e6 + 944.74e6 + 480.06e6, "head": 529.02e6},
}


def _traffic_per_mean_launch(shape, tmpl):
    t = NCU_TRAFFIC.get(shape.name.split("-")[0])
    if t is None or (1 + tmpl.N + tmpl.G * shape.n_mask) != 69:
        return None
    return (shape.L * t["per_layer"] + t["head"]) / (4 * shape.L + 1)


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
    return 6650.0, "fallback (earlier measurement on this pool)"


def _tensor_peak():
    """Sustained dense bf16 TFLOP/s (the figure for a kernel timed inside a long step)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["bf16_tflops_sustained"])
    return 1400.0


def _pass_roofline(shape, rows, ms):
    """A pass against the larger of its two floors: streaming the weights once (HBM) and 2 x params x
    rows flops on the tensor cores.  Past about 210 rows the second is the larger."""
    peak, _ = _peaks()
    t_hbm = shape.streamed_params * 2 / (peak * 1e9) * 1e3
    t_tc = 2.0 * shape.streamed_params * rows / (_tensor_peak() * 1e12) * 1e3
    return {"floor_hbm_ms": t_hbm, "floor_tensor_ms": t_tc, "bound": "hbm" if t_hbm >= t_tc else "tensor",
            "frac_of_floor": max(t_hbm, t_tc) / ms}


def _expected_tokens_per_step(tmpl, fraction):
    has_child = [False] * tmpl.N
    for p in tmpl.parent:
        if p >= 0:
            has_child[p] = True
    depth = tmpl.depths()
    leaves = [depth[i] for i in range(tmpl.N) if not has_child[i]]
    return 1.0 + fraction * (sum(leaves) / len(leaves) if leaves else 0.0)


# ----------------------------------------------------------------------------------------------
# clocks
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.idx}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1]))
                    mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                                     f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), samples=len(sm))
        out["reasons"] = sorted(reasons)
        return out


# ----------------------------------------------------------------------------------------------
# CPU oracle legs: `cpu_baseline` of our arm and the whole of `--impl reference`
def _seeded_state(orc, model, shape, C):
    """Oracle decoding state with C cached tokens of seeded random keys/values (the time of a pass
    does not depend on their values) and an arbitrary last token."""
    st = orc.State(model)
    for l in range(shape.L):
        st.k[l] = synth.pseudo_normal(PROMPT_SEED, 1000 + 2 * l, (shape.H_kv, C, shape.D), 1.0).double().numpy()
        st.v[l] = synth.pseudo_normal(PROMPT_SEED, 1001 + 2 * l, (shape.H_kv, C, shape.D), 1.0).double().numpy()
    st.root = 1
    return st


def _gen_device():
    return "cuda:0" if torch.cuda.is_available() else "cpu"


def oracle_whole_steps(shape, tmpl, n_steps, n_warm, fraction):
    """Times whole oracle passes (`orc.bita_step`: pack, every layer, LM head, selection, walk, next
    tree, cache append) of the workload's block, the oracle exactly as the tests call it.
    Returns (tokens/s, ms per pass, description, cores)."""
    from oracle import bita_oracle as orc
    from oracle.inputs import block_for, oracle_model
    cores = len(os.sched_getaffinity(0))
    torch.set_num_threads(cores)
    # the model's weights as fp32 host arrays, generated off the clock (on the GPU when there is one)
    weights = synth.make_weights(shape, MODEL_SEED, dtype=torch.bfloat16, device=_gen_device())
    model = oracle_model(shape, MODEL_SEED, weights=weights)
    del weights
    if torch.cuda.is_available():
        torch.cuda.empty_cache()
    blk = block_for(tmpl, shape.n_mask)
    st = _seeded_state(orc, model, shape, shape.prompt_len)
    tree = synth.uniform_ints(PLANT_SEED, 77, blk.N, shape.V).tolist()
    times = []
    for i in range(n_warm + n_steps):
        t0 = time.perf_counter()
        rec = orc.bita_step(model, blk, st, tree)
        times.append(time.perf_counter() - t0)
        tree = rec["next_tree"]
    ms = 1e3 * sum(times[n_warm:]) / max(1, n_steps)
    tps = _expected_tokens_per_step(tmpl, fraction) / (ms * 1e-3)
    desc = (f"{n_steps} whole oracle passes (orc.bita_step, all {shape.L} layers + LM head + selection + walk) of the "
            f"{shape.name} block ({blk.M} rows) on a cache of {shape.prompt_len} seeded random tokens; fp64 numpy; "
            f"tokens per pass = expectation of the planting recipe")
    return tps, ms, desc, cores


def oracle_layer_samples(shape, tmpl, n_steps, n_warm, fraction):
    """For models whose whole oracle pass takes minutes (70B): a sample is ONE decoder layer of the
    pass; the whole pass is ESTIMATED as L x (mean layer time) + (LM head + selection + walk, timed once).
    Returns (tokens/s of the estimate, ms per sample, ms per estimated pass, description, cores)."""
    import numpy as np
    from oracle import bita_oracle as orc
    from oracle.inputs import block_for, oracle_model
    cores = len(os.sched_getaffinity(0))
    torch.set_num_threads(cores)
    one = shape.with_layers(1)
    weights = synth.make_weights(one, MODEL_SEED, dtype=torch.bfloat16, device=_gen_device())
    model = oracle_model(one, MODEL_SEED, weights=weights)
    del weights
    if torch.cuda.is_available():
        torch.cuda.empty_cache()
    blk = block_for(tmpl, shape.n_mask)
    st = _seeded_state(orc, model, one, shape.prompt_len)
    x = synth.pseudo_normal(PROMPT_SEED, 33, (blk.M, shape.d), 1.0).double().numpy()
    pos = shape.prompt_len + blk.rel_pos

    def layer():
        return orc._layer(model, model.w["layers"][0], x, pos, st.k[0], st.v[0], blk.vis, blk.sees_prompt)

    def head():
        logits = orc.rmsnorm(x, model.w["g_final"], model.rms_eps) @ np.asarray(model.w["lm_head"], dtype=np.float64).T
        am = [orc.argmax_lowest(logits[r]) for r in range(1 + blk.N)]
        tk = np.zeros((blk.G, blk.n, blk.k_max), dtype=np.int64)
        for g in range(blk.G):
            for i in range(blk.n):
                tk[g, i], _ = orc.topk_sorted(logits[blk.mask_row(g, i)], blk.k_max)
        _, _, cur = orc.verify_walk(blk, [1] * blk.N, am)
        orc.next_tree(blk, tk, cur)

    t0 = time.perf_counter()
    head()
    t_head = time.perf_counter() - t0
    for _ in range(n_warm):
        layer()
    t0 = time.perf_counter()
    for _ in range(n_steps):
        layer()
    t_layer = (time.perf_counter() - t0) / max(1, n_steps)
    full = shape.L * t_layer + t_head
    tps = _expected_tokens_per_step(tmpl, fraction) / full
    desc = (f"ESTIMATE: {n_steps} samples of one decoder layer of the {shape.name} pass ({blk.M} rows, cache of "
            f"{shape.prompt_len} seeded random tokens; orc._layer as it stands), scaled x{shape.L} layers + LM head / "
            f"selection / walk timed once ({t_head * 1e3:.0f} ms); a whole fp64 pass of this model takes minutes; "
            f"tokens per pass = expectation of the planting recipe")
    return tps, t_layer * 1e3, full * 1e3, desc, cores


def oracle_leg(shape, tmpl, n_steps, n_warm, fraction, whole_steps=None):
    """cpu_baseline record of a workload: whole passes where one takes seconds, the labelled
    layer-sample estimate where it takes minutes."""
    if shape.streamed_params > 20e9:
        tps, ms_sample, ms_full, desc, cores = oracle_layer_samples(shape, tmpl, n_steps, n_warm, fraction)
        return {"value": tps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc,
                "ms_per_step": ms_full, "ms_per_sample": ms_sample, "estimated": True}
    tps, ms, desc, cores = oracle_whole_steps(shape, tmpl, n_steps if whole_steps is None else whole_steps, n_warm,
                                              fraction)
    return {"value": tps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc, "ms_per_step": ms,
            "ms_per_sample": ms, "estimated": False}


def _config(shape, tmpl, fraction, world):
    """The `config` object, identical in our arm and in the reference arm."""
    return {"workload": _workload_name(shape, tmpl, fraction), "l2": "inputs (weights) larger than L2",
            "tokens_per_step_expected": _expected_tokens_per_step(tmpl, fraction),
            "parallelism": f"replicas x{world}"}


def run_reference(args, shape, tmpl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    leg = oracle_leg(shape, tmpl, args.steps, args.warmup, args.planted)
    # `ms_per_step` is the wall time of one timed sample, so that steps x ms_per_step is the timed
    # region of this run; for the 70B shape the sample is one layer and `value` the labelled estimate
    line = {
        "impl": "reference", "metric": METRIC, "value": leg["value"], "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": leg["ms_per_sample"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": _config(shape, tmpl, args.planted, max(1, args.gpus)),
        "cpu_baseline": {k: leg[k] for k in ("value", "unit", "cores", "kind", "sample", "estimated")},
        "estimated_full_step_ms": leg["ms_per_step"],
        "e2e": {"value": leg["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def _workload_name(shape, tmpl, fraction):
    return (f"LLaMA-2-{shape.name} shape bf16 random-init, {tmpl.N}-node tree + {shape.n_mask} mask tokens "
            f"({1 + tmpl.N + tmpl.G * shape.n_mask} rows), {shape.prompt_len}-token prompt, batch 1, "
            f"planted acceptance {fraction:.2f}")


# ----------------------------------------------------------------------------------------------
def build_trees(ctx, shape, tmpl, n_steps, fraction):
    """Untimed dry run: per step, look ahead with one-token passes to learn the true continuation from
    the current state, rewind, plant it on a seeded fraction of the steps, take the step.
    Returns (list of per-step tree token lists, emitted tokens per step)."""
    trees, emitted = [], []
    depth = max(tmpl.depths(), default=0)
    disabled = [-1] * tmpl.N
    rec = None
    for s in range(n_steps):
        state_len = ctx_len(ctx) if rec is None else rec["new_len"]
        root = ctx._root if rec is None else rec["out_tokens"][-1]
        base = list(ctx._tree if rec is None else rec["next_tree"])
        u = float(synth.uniform_unit(PLANT_SEED, 9001, 1, offset=s)[0])
        if fraction > 0 and u < fraction and tmpl.N:
            cont = []
            for _ in range(depth):
                cont += ctx.step(disabled)["out_tokens"]
            ctx.rewind(state_len, root)
            toks = synth.plant_tree(tmpl, base, cont, PLANT_SEED, s, 1.1, shape.V)
        else:
            toks = base
        rec = ctx.step(toks)
        trees.append(toks)
        emitted.append(rec["n_out"])
    return trees, emitted


def ctx_len(ctx):
    return ctx._len


def replica_plan(rank: int, shape):
    """What differs between the independent replicas of a multi-GPU run: only the prompt seed."""
    return {"prompt_seed": PROMPT_SEED + rank, "model_seed": MODEL_SEED, "plant_seed": PLANT_SEED}


def aggregate_over_ranks(dist_mod, world: int, dev_ms: float, e2e_ms: float, tokens: float, device):
    """Whole-job numbers of a replica run: the slowest rank's times, the sum of the tokens."""
    times = torch.tensor([dev_ms, e2e_ms], dtype=torch.float64, device=device)
    toks = torch.tensor([float(tokens)], dtype=torch.float64, device=device)
    if world > 1:
        dist_mod.all_reduce(times, op=dist_mod.ReduceOp.MAX)
        dist_mod.all_reduce(toks, op=dist_mod.ReduceOp.SUM)
    dev_ms, e2e_ms = times.tolist()
    return dev_ms, e2e_ms, float(toks[0])


def measure_workload(shape, tmpl, K, W, fraction, rank, world, local, dist):
    """All device-side measurements of one workload on this rank's GPU.  Returns a dict of raw numbers
    (times are this rank's; `aggregate_over_ranks` combines them)."""
    from paper_2401_12522_b200 import Bita
    dev = torch.device(f"cuda:{local}")
    total_steps = K + W
    depth = max(tmpl.depths(), default=0)
    rows = 1 + tmpl.N + tmpl.G * shape.n_mask
    C_max = shape.prompt_len + total_steps * (depth + 1) + depth + rows + 64
    # replicas: every rank decodes its own sequence with its own seeds; no data-path collective
    weights = synth.make_weights(shape, MODEL_SEED, dtype=torch.bfloat16, device=dev)
    prompt = synth.uniform_ints(replica_plan(rank, shape)["prompt_seed"], 5001, shape.prompt_len, shape.V).tolist()
    ctx = Bita(shape, weights, tmpl, C_max=C_max, device=dev)

    def start(c=ctx):
        c.reset()
        r = c.prefill(prompt)
        c._len, c._root, c._tree = r["new_len"], r["out_tokens"][-1], r["next_tree"]

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    start()
    trees, emitted = build_trees(ctx, shape, tmpl, total_steps, fraction)
    trees_dev = torch.tensor(trees, dtype=torch.int32, device=dev) if tmpl.N else None
    tokens_timed = sum(emitted[W:])

    # ---- device-resident timing: inputs already in HBM, no host sync inside the timed region
    start()
    for s in range(W):
        ctx.step_enqueue(None if trees_dev is None else trees_dev[s])
    sampler = ClockSampler(local)
    barrier()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for s in range(W, total_steps):
        ctx.step_enqueue(None if trees_dev is None else trees_dev[s])
    e1.record()
    barrier()
    clocks = sampler.stop()
    dev_ms = e0.elapsed_time(e1)
    final = ctx.step_finish()
    launches = ctx.last_launch_count * K
    assert final["new_len"] == shape.prompt_len + sum(emitted), "replay diverged from the dry run"

    # ---- end to end through bita_step with host buffers (H2D of the tree, D2H of the record per step)
    start()
    for s in range(W):
        ctx.step(trees[s])
    barrier()
    t0 = time.perf_counter()
    e0.record()
    got = 0
    step_wall = []
    for s in range(W, total_steps):
        t_s = time.perf_counter()
        got += ctx.step(trees[s])["n_out"]
        step_wall.append((time.perf_counter() - t_s) * 1e3)
    e1.record()
    barrier()
    e2e_ms = max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3)
    assert got == tokens_timed

    # ---- per-family timing pass for the roofline: one CUDA event on the library's stream wherever the
    # kernel family changes (runs of consecutive projections are timed as they overlap in a normal pass)
    start()
    ctx.set_kernel_timing(True)
    fam_ms, fam_n = [0.0, 0.0], [0, 0]
    n_prof = min(K, 16)
    for s in range(n_prof):
        ctx.step_enqueue(None if trees_dev is None else trees_dev[s])
        ms, n = ctx.kernel_timing()
        fam_ms = [a + b for a, b in zip(fam_ms, ms)]
        fam_n = [a + b for a, b in zip(fam_n, n)]
    ctx.set_kernel_timing(False)
    ctx.step_finish()
    ctx.close()

    # ---- the same library in autoregressive mode (no tree, no mask tokens: one row, one token per pass),
    # the denominator of the paper's speedup metric (Sec. 4.1, "Evaluation Settings")
    ar = Bita(shape, weights, synth.empty_template(with_group=False), C_max=shape.prompt_len + total_steps + 80,
              device=dev)
    start(ar)
    for s in range(W):
        ar.step_enqueue(None)
    barrier()
    e0.record()
    for s in range(K):
        ar.step_enqueue(None)
    e1.record()
    barrier()
    ar_ms = e0.elapsed_time(e1) / K
    ar.step_finish()
    ar.close()
    del ctx, ar, weights, trees_dev
    torch.cuda.empty_cache()
    return dict(dev_ms=dev_ms, e2e_ms=e2e_ms, tokens=tokens_timed, emitted=emitted, step_wall=step_wall,
                launches=launches, fam_ms=fam_ms, fam_n=fam_n, n_prof=n_prof, clocks=clocks, ar_ms=ar_ms, rows=rows)


def summarise(shape, tmpl, K, W, fraction, world, m, dev_ms, e2e_ms, total_tokens):
    """Numbers of one workload as they go into the JSON line."""
    peak, peak_src = _peaks()
    weight_bytes = shape.streamed_params * 2
    fam_ms, fam_n, n_prof, emitted = m["fam_ms"], m["fam_n"], m["n_prof"], m["emitted"]
    gemm_ms = fam_ms[0] / max(1, fam_n[0])                    # average projection launch
    gemm_bytes = weight_bytes / (fam_n[0] / n_prof)            # algorithmic bytes of an average launch
    achieved = gemm_bytes / (gemm_ms * 1e-3) / 1e9
    mean_C = shape.prompt_len + sum(emitted[:W]) + sum(emitted[W:]) / 2
    step_bytes = weight_bytes + shape.kv_bytes_per_token() * mean_C
    step_ms = dev_ms / K
    value = total_tokens / (dev_ms * 1e-3)
    ar_tps = world * 1e3 / m["ar_ms"]
    return {
        "value": value, "ms_per_step": step_ms, "tokens_per_step": m["tokens"] / K,
        "tokens_per_step_expected": _expected_tokens_per_step(tmpl, fraction),
        "step_hbm_frac": (step_bytes / (step_ms * 1e-3) / 1e9) / peak,
        "step_algorithmic_bytes": step_bytes,
        "autoregressive": {"ms_per_token": m["ar_ms"], "tokens_per_s": ar_tps, "rows": 1,
                           "hbm_frac": (weight_bytes + shape.kv_bytes_per_token() * mean_C) / (m["ar_ms"] * 1e-3) / 1e9 / peak},
        "greedy_speedup": value / ar_tps,
        "e2e": {"value": total_tokens / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms / K,
                "p50_ms": statistics.median(m["step_wall"]),
                "p90_ms": sorted(m["step_wall"])[int(0.9 * (len(m["step_wall"]) - 1))],
                "h2d_bytes_per_step": 4 * tmpl.N, "d2h_bytes_per_step": 4 * (5 + 2 * 16 + 1 + 160)},
        "gpu_launches": m["launches"],
        "clocks": m["clocks"],
        "roofline": {"bound": "hbm",
                     "kernel": "k_gemm_tc (weight-streaming projection), mean over the step's launches; CUDA events on "
                               "the library's stream at the boundaries of runs of consecutive projections",
                     "achieved": achieved, "peak": peak, "peak_source": peak_src, "unit": "GB/s",
                     "frac": achieved / peak, "algorithmic_bytes_per_launch": gemm_bytes,
                     "traffic": _traffic_per_mean_launch(shape, tmpl),
                     "traffic_source": "dram bytes of an earlier ncu capture (profiles/), not measured by this run"
                                       if _traffic_per_mean_launch(shape, tmpl) else None,
                     "attention_ms_per_step": fam_ms[1] / n_prof, "projection_ms_per_step": fam_ms[0] / n_prof},
    }


def run_ours(args, names):
    """`names`: workloads to measure; the LAST one is the headline of the JSON line, the others are
    reported under `other_workloads`."""
    from paper_2401_12522_b200.build import build
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    if rank == 0:
        build()
    if world > 1:
        dist.barrier()
    dev = torch.device(f"cuda:{local}")
    torch.cuda.set_device(dev)
    K, W = args.steps, args.warmup
    results = {}
    for name in names:
        shape = synth.CONFIGS[name]
        if args.layers:
            shape = shape.with_layers(args.layers)
        tmpl = synth.product_rule_template(shape.tree_K, shape.tree_B)
        m = measure_workload(shape, tmpl, K, W, args.planted, rank, world, local, dist)
        dev_ms, e2e_ms, total_tokens = aggregate_over_ranks(dist, world, m["dev_ms"], m["e2e_ms"], m["tokens"], dev)
        if rank == 0:
            r = summarise(shape, tmpl, K, W, args.planted, world, m, dev_ms, e2e_ms, total_tokens)
            r["config"] = _config(shape, tmpl, args.planted, world)
            if world == 1 and not args.no_cpu_baseline:
                r["cpu_baseline"] = oracle_leg(shape, tmpl, args.cpu_samples, 1, args.planted, whole_steps=2)
            results[name] = r
    if rank == 0:
        head = results[names[-1]]
        line = {"metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
                "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "bf16", "data": "synthetic"}
        line.update({k: v for k, v in head.items() if k not in ("value", "ms_per_step")})
        line["other_workloads"] = {n: results[n] for n in names[:-1]}
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_attn_sweep():
    """Tree-attention kernel alone: bf16 q of (1 + 4 + N) rows x 32 heads x 128 against caches of C tokens,
    seeded random trees, batch 1 and 8.  Prints one JSON line per case (latency, KV GB/s)."""
    from paper_2401_12522_b200 import bita_tree_attention
    from paper_2401_12522_b200.build import build
    build()
    dev = torch.device("cuda:0")
    peak, _ = _peaks()
    H = H_kv = 32
    D, P = 128, 16
    for B in (1, 8):
        for N in (16, 64, 128):
            M = 1 + N + 4
            tmpl = synth.random_recursive_template(N + 1, N)
            W = (M + 31) // 32
            depth = tmpl.depths()
            vis = torch.zeros((M, W), dtype=torch.int64)
            anc = [[0]]
            for i, p_ in enumerate(tmpl.parent):
                anc.append(anc[p_ + 1] + [i + 1])
            rows = anc + [anc[0] + list(range(1 + N, 1 + N + i + 1)) for i in range(4)]
            for r, cols in enumerate(rows):
                for c in cols:
                    vis[r, c >> 5] |= 1 << (c & 31)
            vis = (vis & 0xFFFFFFFF).to(torch.int64)
            vis32 = torch.where(vis >= 2 ** 31, vis - 2 ** 32, vis).to(torch.int32)
            vis_d = vis32[None].repeat(B, 1, 1).contiguous().to(dev)
            sp = torch.zeros((B, M), dtype=torch.uint8)
            sp[:, 1 + N:] = 1
            sp = sp.to(dev)
            for C in (512, 2048, 8192, 32768):
                C_max = C + M + 8
                q = synth.pseudo_normal(1, 1, (B, M, H, D), 1.0, dtype=torch.bfloat16, device=dev)
                k = synth.pseudo_normal(1, 2, (B, H_kv, C_max, D), 1.0, dtype=torch.bfloat16, device=dev)
                v = synth.pseudo_normal(1, 3, (B, H_kv, C_max, D), 1.0, dtype=torch.bfloat16, device=dev)
                pk = synth.pseudo_normal(1, 4, (H_kv, P, D), 1.0, dtype=torch.bfloat16, device=dev)
                pv = synth.pseudo_normal(1, 5, (H_kv, P, D), 1.0, dtype=torch.bfloat16, device=dev)
                ctx = torch.full((B,), C, dtype=torch.int32, device=dev)
                out = torch.empty((B, M, H * D), dtype=torch.bfloat16, device=dev)
                flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
                ws = None
                times = []
                for it in range(8):
                    flush.zero_()                                # caches smaller than L2 would otherwise stay in it
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    bita_tree_attention(q, k, v, vis_d, pk, pv, sp, ctx, H_kv=H_kv, P=P, out=out)
                    e1.record()
                    torch.cuda.synchronize()
                    if it >= 3:
                        times.append(e0.elapsed_time(e1))
                ms = statistics.median(times)
                kv_bytes = B * 2 * (C + M) * H_kv * D * 2
                print(json.dumps({"metric": "tree_attention_latency", "B": B, "rows": M, "C": C, "ms": ms,
                                  "kv_gb_per_s": kv_bytes / ms / 1e6, "hbm_frac": kv_bytes / ms / 1e6 / peak,
                                  "l2": "flushed before each launch"}))
                del q, k, v, flush


def _time_steps(ctx, steps, warm=4):
    for _ in range(warm):
        ctx.step_batch_enqueue(None)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        ctx.step_batch_enqueue(None)
    e1.record()
    torch.cuda.synchronize()
    ctx.step_batch_finish()
    return e0.elapsed_time(e1) / steps


def run_next_rows(args, shape):
    """Measurements beyond the headline step, one JSON line each (device-resident, CUDA events):

    * the first pass (Algorithm 1, t = 1) as a timed path;
    * the cost side of the paper's comparison of decoding methods (Sec. 4.3, Table 4): step latency
      of every tree template at this model shape - straightforward decoding, fully tree-based
      decoding with k = 1..4 candidates per mask, the efficient (comb) tree, each with a mask group
      per node as the paper attaches them, plus the configuration's product-rule tree - next to
      the library in autoregressive mode.  The acceptance side comes from the stated synthetic model
      in synth/acceptance.py (no tuned model or dataset exists here): tokens per pass by seeded
      simulation, tokens/s = tokens per pass / measured latency, speedup = tokens/s over AR tokens/s;
    * several sequences in one pass (a context of batch > 1): latency of the pass and aggregate
      tokens/s for 1..5 sequences of the configuration's 69-row block, prompts of different lengths.
    """
    from paper_2401_12522_b200 import Bita, BitaError
    from paper_2401_12522_b200.build import build
    build()
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    peak, _ = _peaks()
    weights = synth.make_weights(shape, MODEL_SEED, dtype=torch.bfloat16, device=dev)
    prompt = synth.uniform_ints(replica_plan(0, shape)["prompt_seed"], 5001, shape.prompt_len, shape.V).tolist()
    steps = 24
    model = synth.AcceptanceModel()
    # ---- autoregressive mode: one row, one token per pass
    ar = Bita(shape, weights, synth.empty_template(with_group=False), C_max=shape.prompt_len + steps + 80, device=dev)
    ar.prefill(prompt)
    ar_ms = _time_steps(ar, steps)
    ar.close()
    print(json.dumps({"metric": "step_latency_by_template", "workload": shape.name, "template": "autoregressive (no tree, no masks)",
                      "n_mask": 0, "nodes": 0, "groups": 0, "rows": 1, "ms_per_step": ar_ms, "tokens_per_pass_model": 1.0,
                      "tokens_per_s": 1e3 / ar_ms, "speedup_vs_autoregressive": 1.0}))
    # ---- first pass
    ctx = Bita(shape, weights, synth.product_rule_template(shape.tree_K, shape.tree_B),
               C_max=shape.prompt_len + 400, device=dev)
    times = []
    for it in range(3):
        ctx.reset()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ctx.prefill(prompt)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    ctx.close()
    pre_ms = min(times)
    flops = 2.0 * shape.streamed_params * shape.prompt_len
    print(json.dumps({"metric": "first_pass", "workload": shape.name, "tokens": shape.prompt_len, "ms": pre_ms,
                      "tokens_per_s": shape.prompt_len / pre_ms * 1e3, "tflops": flops / pre_ms / 1e9}))
    # ---- templates; n = 3 is the paper's setting for 7B-class models (Sec. 4.1), n = 4 this configuration's
    cases = []
    for n in sorted({3, shape.n_mask}):
        cases += [(n, "straightforward decoding (chain of top-1 drafts, one group after the last token)", synth.chain_template(n))]
        cases += [(n, f"fully tree-based decoding k={k}, a group per node", synth.full_tree_template(n, k)) for k in (1, 2, 3, 4)]
        cases += [(n, "efficient tree-based decoding (comb tree k=5, a group per node: the paper's default)",
                   synth.comb_template(n, 5))]
    cases += [(shape.n_mask, "product-rule tree of the measured configuration (64 nodes, one group)",
               synth.product_rule_template(shape.tree_K, shape.tree_B))]
    for n, name, tmpl in cases:
        from dataclasses import replace
        sh = replace(shape, n_mask=n)
        rows = 1 + tmpl.N + tmpl.G * n
        acc = synth.tokens_per_pass(tmpl, n, model)["tokens_per_pass"]
        line = {"metric": "step_latency_by_template", "workload": shape.name, "template": name, "n_mask": n,
                "nodes": tmpl.N, "groups": tmpl.G, "rows": rows, "tokens_per_pass_model": acc,
                "acceptance_model": {"h0": model.h0, "gamma": model.gamma, "r": model.r}}
        depth = max(tmpl.depths(), default=0)
        try:
            w = dict(weights, mask_emb=weights["mask_emb"][:n].contiguous())
            ctx = Bita(sh, w, tmpl, C_max=shape.prompt_len + (steps + 8) * (depth + 1) + rows + 64, device=dev)
        except BitaError as e:
            line.update(ms_per_step=None, refused=str(e))
            print(json.dumps(line))
            continue
        ctx.prefill(prompt)
        ms = _time_steps(ctx, steps)
        ctx.close()
        line.update(ms_per_step=ms, tokens_per_s=acc / ms * 1e3, speedup_vs_autoregressive=(acc / ms) / (1.0 / ar_ms),
                    weights_hbm_frac=shape.streamed_params * 2 / ms / 1e6 / peak, roofline=_pass_roofline(shape, rows, ms))
        print(json.dumps(line))
    # ---- several sequences in one pass: each with its own prompt length, cache, tree and accepted length
    tmpl = synth.product_rule_template(shape.tree_K, shape.tree_B)
    rows = 1 + tmpl.N + tmpl.G * shape.n_mask
    depth = max(tmpl.depths(), default=0)
    acc = synth.tokens_per_pass(tmpl, shape.n_mask, model)["tokens_per_pass"]
    B = 1
    while B * rows <= 352 and B <= 16:
        lens = [max(16, shape.prompt_len - 37 * b) for b in range(B)]
        ctx = Bita(shape, weights, tmpl, C_max=shape.prompt_len + (steps + 8) * (depth + 1) + rows + 64, device=dev,
                   batch=B)
        for b in range(B):
            ctx.prefill(prompt[:lens[b]], seq=b)
        ms = _time_steps(ctx, steps)
        ctx.close()
        flops = 2.0 * shape.streamed_params * B * rows
        print(json.dumps({"metric": "step_latency_by_batch", "workload": shape.name, "sequences": B, "rows": B * rows,
                          "prompt_lens": lens, "ms_per_step": ms, "tokens_per_pass_model": acc * B,
                          "tokens_per_s": acc * B / ms * 1e3, "speedup_vs_autoregressive": (acc * B / ms) / (1.0 / ar_ms),
                          "weights_hbm_frac": shape.streamed_params * 2 / ms / 1e6 / peak,
                          "tflops": flops / ms / 1e9, "roofline": _pass_roofline(shape, B * rows, ms)}))
        B += 1


def _spawn_ranks(n: int):
    """`python bench.py --gpus N` without a launcher: start the N ranks ourselves (one process per GPU)."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    sys.exit(subprocess.call(cmd))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=64)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="all", choices=sorted(synth.CONFIGS) + ["all"],
                    help="all (default): the 70B shape is the headline, 7B and 13B ride along under other_workloads")
    ap.add_argument("--layers", type=int, default=0, help="truncate the layer stack (debugging only)")
    ap.add_argument("--planted", type=float, default=0.6)
    ap.add_argument("--cpu-samples", type=int, default=12,
                    help="cpu_baseline: layer samples of the 70B estimate (whole passes of smaller models: 2)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--attn-sweep", action="store_true", help="time the tree-attention kernel alone over the sweep shapes")
    ap.add_argument("--next-rows", action="store_true",
                    help="first pass as a timed path and step latency per tree template (one JSON line per template)")
    args = ap.parse_args()
    if args.attn_sweep:
        run_attn_sweep()
        return
    if args.next_rows:
        shape = synth.CONFIGS["7b" if args.workload == "all" else args.workload]
        run_next_rows(args, shape.with_layers(args.layers) if args.layers else shape)
        return
    if args.warmup < 3:
        args.warmup = 3
    world = os.environ.get("WORLD_SIZE")
    if world is None and args.gpus > 1:
        _spawn_ranks(args.gpus)
    if world is not None and int(world) != args.gpus:
        sys.exit(f"bench.py: --gpus {args.gpus} but the launcher started WORLD_SIZE={world} ranks")
    names = ["7b", "13b", "70b"] if args.workload == "all" else [args.workload]
    if args.impl == "reference":
        shape = synth.CONFIGS[names[-1]]
        if args.layers:
            shape = shape.with_layers(args.layers)
        run_reference(args, shape, synth.product_rule_template(shape.tree_K, shape.tree_B))
    else:
        run_ours(args, names)


if __name__ == "__main__":
    main()
