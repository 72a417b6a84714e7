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


# DRAM bytes (read + write) per projection launch at the 7B width with the 69-row block, from the ncu
# capture summarised in profiles/k_gemm_tc_k_attn_umma_7b_ncu_full.md (q/k/v, O, gate/up, down per
# layer; LM head).  Other shapes have no capture: their `traffic` is null.
NCU_TRAFFIC_7B = {"per_layer": 105.57e6 + 35.54e6 + 184.55e6 + 96.89e6, "head": 266.14e6}


def _traffic_per_mean_launch(shape, tmpl):
    if not shape.name.startswith("7b") or (1 + tmpl.N + tmpl.G * shape.n_mask) != 69:
        return None
    return (shape.L * NCU_TRAFFIC_7B["per_layer"] + NCU_TRAFFIC_7B["head"]) / (4 * shape.L + 1)


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured (MEASURED_PEAKS.json)"
    return 6650.0, "fallback (earlier measurement on this pool)"


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
# reference arm: the CPU oracle as it stands, on a bounded sample of the same workload
def _oracle_sample(shape, tmpl, n_steps, n_warm, fraction):
    """Times `n_steps` oracle samples; a sample is ONE decoder layer of the step's packed block.

    The full-step time is estimated as L x (layer time) + (final norm + LM head + selection + walk),
    the latter measured once.  Returns (tokens/s, ms per estimated full step, description, cores).
    """
    import numpy as np
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from helpers import block_for, oracle_model  # noqa
    from oracle import bita_oracle as orc

    cores = len(os.sched_getaffinity(0))
    torch.set_num_threads(cores)
    one = shape.with_layers(1)
    model = oracle_model(one, MODEL_SEED)
    # fp64 copies of the sampled layer, so that a sample times the arithmetic and not the conversion
    model.w["layers"][0] = {k: np.asarray(v, dtype=np.float64) for k, v in model.w["layers"][0].items()}
    lm64 = np.asarray(model.w["lm_head"], dtype=np.float64)
    blk = block_for(tmpl, shape.n_mask)
    C = shape.prompt_len
    rng_k = synth.pseudo_normal(PROMPT_SEED, 31, (shape.H_kv, C, shape.D), 1.0).double().numpy()
    rng_v = synth.pseudo_normal(PROMPT_SEED, 32, (shape.H_kv, C, shape.D), 1.0).double().numpy()
    x = synth.pseudo_normal(PROMPT_SEED, 33, (blk.M, shape.d), 1.0).double().numpy()
    pos = C + blk.rel_pos

    def layer():
        return orc._layer(model, model.w["layers"][0], x, pos, rng_k, rng_v, blk.vis, blk.sees_prompt)

    def head():
        logits = orc.rmsnorm(x, model.w["g_final"], model.rms_eps) @ lm64.T
        am = [orc.argmax_lowest(logits[r]) for r in range(1 + blk.N)]
        tk = np.zeros((blk.G, blk.n, blk.k_max), dtype=np.int64)
        for g in range(blk.G):
            for i in range(blk.n):
                tk[g, i], _ = orc.topk_sorted(logits[blk.mask_row(g, i)], blk.k_max)
        acc, out, cur = orc.verify_walk(blk, [1] * blk.N, am)
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
    desc = (f"{n_steps} samples of one decoder layer of the {shape.name} step ({blk.M} rows, random KV context of "
            f"{C} tokens, weights held in fp64), scaled x{shape.L} layers + LM head/selection/walk measured once; "
            f"tokens per step = expectation of the planting recipe")
    return tps, full * 1e3, desc, cores


def run_reference(args, shape, tmpl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    tps, ms, desc, cores = _oracle_sample(shape, tmpl, args.steps, args.warmup, args.planted)
    line = {
        "impl": "reference", "metric": METRIC, "value": tps, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": _workload_name(shape, tmpl, args.planted)},
        "cpu_baseline": {"value": tps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": tps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
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


def run_ours(args, shape, tmpl):
    from paper_2401_12522_b200 import Bita
    from paper_2401_12522_b200.build import build
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
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
    total_steps = K + W
    depth = max(tmpl.depths(), default=0)
    rows = 1 + tmpl.N + tmpl.G * shape.n_mask
    C_max = shape.prompt_len + total_steps * (depth + 1) + depth + rows + 64
    # replicas: every rank decodes its own sequence with its own seeds; no data-path collective
    weights = synth.make_weights(shape, MODEL_SEED, dtype=torch.bfloat16, device=dev)
    prompt = synth.uniform_ints(replica_plan(rank, shape)["prompt_seed"], 5001, shape.prompt_len, shape.V).tolist()
    ctx = Bita(shape, weights, tmpl, C_max=C_max, device=dev)

    def start():
        ctx.reset()
        r = ctx.prefill(prompt)
        ctx._len, ctx._root, ctx._tree = r["new_len"], r["out_tokens"][-1], r["next_tree"]

    start()
    trees, emitted = build_trees(ctx, shape, tmpl, total_steps, args.planted)
    trees_dev = torch.tensor(trees, dtype=torch.int32, device=dev) if tmpl.N else None
    tokens_timed = sum(emitted[W:])

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

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

    # ---- per-kernel timing pass for the roofline (events around every projection / attention launch)
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

    dev_ms, e2e_ms, total_tokens = aggregate_over_ranks(dist if world > 1 else None, world, dev_ms, e2e_ms,
                                                        tokens_timed, dev)

    if rank == 0:
        peak, peak_src = _peaks()
        weight_bytes = shape.streamed_params * 2
        gemm_ms = fam_ms[0] / max(1, fam_n[0])                    # average projection launch
        gemm_bytes = weight_bytes / (fam_n[0] / n_prof)            # algorithmic bytes of an average launch
        achieved = gemm_bytes / (gemm_ms * 1e-3) / 1e9
        mean_C = shape.prompt_len + sum(emitted[:W]) + sum(emitted[W:]) / 2
        step_bytes = weight_bytes + shape.kv_bytes_per_token() * mean_C
        step_ms = dev_ms / K
        line = {
            "metric": METRIC, "value": total_tokens / (dev_ms * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": W, "ms_per_step": step_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": _workload_name(shape, tmpl, args.planted), "l2": "inputs (weights) larger than L2",
                       "tokens_per_step": tokens_timed / K, "parallelism": f"replicas x{world}"},
            "e2e": {"value": total_tokens / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms / K,
                    "p50_ms": statistics.median(step_wall), "p90_ms": sorted(step_wall)[int(0.9 * (len(step_wall) - 1))],
                    "h2d_bytes_per_step": 4 * tmpl.N, "d2h_bytes_per_step": 4 * (5 + 2 * 16 + 1 + 160)},
            "gpu_launches": launches,
            "clocks": clocks,
            "step_hbm_frac": (step_bytes / (step_ms * 1e-3) / 1e9) / peak,
            "roofline": {"bound": "hbm", "kernel": "projection (weight-streaming GEMM), mean over the step's launches; events at the boundaries of runs of consecutive projections",
                         "achieved": achieved, "peak": peak, "peak_source": peak_src, "unit": "GB/s",
                         "frac": achieved / peak, "algorithmic_bytes_per_launch": gemm_bytes,
                         "traffic": _traffic_per_mean_launch(shape, tmpl),
                         "attention_ms_per_step": fam_ms[1] / n_prof, "projection_ms_per_step": fam_ms[0] / n_prof},
        }
        if world == 1 and not args.no_cpu_baseline:
            tps, ms, desc, cores = _oracle_sample(shape, tmpl, args.cpu_samples, 1, args.planted)
            line["cpu_baseline"] = {"value": tps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc,
                                    "ms_per_step": ms}
        print(json.dumps(line))
    ctx.close()
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


def run_next_rows(args, shape):
    """Measurements beyond the headline step: the first pass (Algorithm 1, t = 1) as a timed path, and
    the cost side of the template comparison (Sec. 4.3): step latency per tree template at this
    model shape.  One JSON line each; device-resident, CUDA events, no planted acceptance."""
    from paper_2401_12522_b200 import Bita
    from paper_2401_12522_b200.build import build
    build()
    dev = torch.device("cuda:0")
    torch.cuda.set_device(dev)
    peak, _ = _peaks()
    weights = synth.make_weights(shape, MODEL_SEED, dtype=torch.bfloat16, device=dev)
    prompt = synth.uniform_ints(replica_plan(0, shape)["prompt_seed"], 5001, shape.prompt_len, shape.V).tolist()
    n, steps = shape.n_mask, 24
    templates = [
        ("straightforward (chain of top-1 drafts, one group)", synth.chain_template(n)),
        ("product-rule tree of the configuration, one group", synth.product_rule_template(shape.tree_K, shape.tree_B)),
        ("efficient comb tree k=5, a group per node (paper default)", synth.comb_template(n, 5)),
        ("efficient comb tree k=3, a group per node", synth.comb_template(n, 3)),
    ]
    for name, tmpl in templates:
        rows = 1 + tmpl.N + tmpl.G * n
        depth = max(tmpl.depths(), default=0)
        C_max = shape.prompt_len + (steps + 8) * (depth + 1) + rows + 64
        ctx = Bita(shape, weights, tmpl, C_max=C_max, device=dev)
        ctx.reset()
        # ---- first pass: equal blocks of up to 248 rows through the same kernels, then the first tree
        times = []
        for it in range(3):
            ctx.reset()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            ctx.prefill(prompt)
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        pre_ms = min(times)
        flops = 2.0 * shape.streamed_params * shape.prompt_len
        # ---- steps with the model's own drafts (random-init masks: acceptance ~ 0, so this is cost only)
        for s in range(4):
            ctx.step_enqueue(None)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for s in range(steps):
            ctx.step_enqueue(None)
        e1.record()
        torch.cuda.synchronize()
        ctx.step_finish()
        ms = e0.elapsed_time(e1) / steps
        print(json.dumps({"metric": "step_latency_by_template", "workload": shape.name, "template": name,
                          "nodes": tmpl.N, "groups": tmpl.G, "rows": rows, "ms_per_step": ms,
                          "weights_gb_per_s": shape.streamed_params * 2 / ms / 1e6,
                          "hbm_frac": shape.streamed_params * 2 / ms / 1e6 / peak,
                          "prefill": {"tokens": shape.prompt_len, "ms": pre_ms, "tokens_per_s": shape.prompt_len / pre_ms * 1e3,
                                      "tflops": flops / pre_ms / 1e9}}))
        ctx.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="7b", choices=sorted(synth.CONFIGS))
    ap.add_argument("--layers", type=int, default=0, help="truncate the layer stack (debugging only)")
    ap.add_argument("--planted", type=float, default=0.6)
    ap.add_argument("--cpu-samples", type=int, default=12)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--attn-sweep", action="store_true", help="time the tree-attention kernel alone over the sweep shapes")
    ap.add_argument("--next-rows", action="store_true",
                    help="first pass as a timed path and step latency per tree template (one JSON line per template)")
    args = ap.parse_args()
    if args.attn_sweep:
        run_attn_sweep()
        return
    if args.next_rows:
        shape = synth.CONFIGS[args.workload]
        run_next_rows(args, shape.with_layers(args.layers) if args.layers else shape)
        return
    if args.warmup < 3:
        args.warmup = 3
    shape = synth.CONFIGS[args.workload]
    if args.layers:
        shape = shape.with_layers(args.layers)
    tmpl = synth.product_rule_template(shape.tree_K, shape.tree_B)
    if args.impl == "reference":
        run_reference(args, shape, tmpl)
    else:
        run_ours(args, shape, tmpl)


if __name__ == "__main__":
    main()
