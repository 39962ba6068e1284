#!/usr/bin/env python
"""Benchmark of the tree-verification hot path (verify -> accept -> commit) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--no-sweep]

One step = one pass of the whole hot path over one synthetic batch: ssd_verify_tree of a
32-node tree against a 256-token cache on the GPT-2-Large shape (36 x 1280, vocab 50257, bf16,
random N(0, 0.02) weights), ssd_accept_tree on the produced logits, ssd_kv_commit of the accepted
path; the cache is then rolled back (host-side length only) so that every step sees the same
prefix length.  A few token sets are prepared before the timed region: random ids, with the
verifier's own arg-max token planted on each child with probability 0.6 (level by level, from
untimed verifications of the same prefix), so that the timed steps accept paths of several nodes
and the commit really gathers rows.  Prints ONE JSON line.

At one GPU the line also carries a `sweep` measured in the same process: the 16- and 64-node
trees on the same model, the stage-two verification of the GPT-2-small-shaped draft (512-token
prefix, eight-node trigram tree) with a warm L2 and with an L2-evicting pass between steps, and the
GPT-2-XL-shaped model over tree sizes 8..256 with the fractions of the HBM and tensor-core
roofs and the tree size at which the tensor bound overtakes the HBM bound, and the full staged loop
(target, draft, trigram) at three controlled acceptance levels: tokens per target step and tokens/s.

N > 1 runs N independent replicas (one process per GPU, no data-path collective): the path is a
single sequence at batch 1 and does not shard.  Without torchrun's environment the script starts
the N replica processes itself.
"""
from __future__ import annotations

import argparse
import json
import os
import socket
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import ssd_synth  # noqa: E402

METRIC = "GPT-2-L-shape tree-verify us/step (verify+accept+commit)"
UNIT = "us/step"
NOMINAL_HBM_GBS = 8000.0
PLANT_PROBABILITY = 0.6
# DRAM bytes (read + write) of one forward: sums over the forward's kernels in the ncu launch lists under profiles/
# (bench_step_gpt2_large_n32_launch_list.md - a later capture of the same forward, in the sampling list, gives 1760.7 MB -
# and bench_step_gpt2_large_n256_launch_list.md); per forward, like `achieved`
NCU_TRAFFIC_BYTES = {("gpt2_large", 32, 256): 1758.2e6, ("gpt2_large", 256, 256): 2894.2e6}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            return json.load(open(p)), "measured"
        except Exception:
            pass
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.path = index, None, None

    def start(self):
        try:
            f = tempfile.NamedTemporaryFile("w", suffix=".csv", delete=False)
            self.path = f.name
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"], stdout=f, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def count(self) -> int:
        try:
            return sum(1 for line in open(self.path) if line.count(",") >= 6)
        except Exception:
            return 0

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0,
               "window": "warm-up steps, the timed region and identical untimed steps after it (the timed region alone is shorter than one sampling period)"}
        if not self.proc:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        try:
            for line in open(self.path):
                parts = [x.strip() for x in line.split(",")]
                if len(parts) < 7:
                    continue
                try:
                    sm.append(float(parts[0]))
                    mx.append(float(parts[1]))
                except ValueError:
                    continue
                for nm, val in zip(names, parts[3:7]):
                    if val.lower().startswith("active"):
                        reasons.add(nm)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


def tree_rule(n_nodes):
    """Children per node by depth of the benchmark's breadth-first tree."""
    return (4, 2, 2, 1, 1) if n_nodes <= 32 else (4, 2, 2, 2, 1, 1) if n_nodes <= 64 else (4, 3, 2, 2, 2, 2, 2)


def workload(args):
    cfg = ssd_synth.config(args.model, dtype=getattr(args, "weights", "bf16"))
    parent = ssd_synth.tree_branching(args.nodes, tree_rule(args.nodes))
    return cfg, parent


def gemm_flops(cfg: dict, n_nodes: int) -> float:
    """Multiply-add flops of the dense projections of one forward over n_nodes rows."""
    d, F, L, V = cfg["d_model"], cfg["d_ff"], cfg["n_layer"], cfg["vocab"]
    return 2.0 * n_nodes * (L * (4 * d * d + 2 * d * F) + V * d)


def percentiles(values) -> dict:
    v = np.asarray(values, dtype=np.float64)
    return {"median": float(np.median(v)), "p10": float(np.percentile(v, 10)), "p90": float(np.percentile(v, 90)), "mean": float(v.mean())}


def max_over_ranks(values, device="cuda"):
    """Element-wise maximum of `values` over all ranks (the job is as slow as its slowest replica)."""
    import torch
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def replica_value(ms_per_step: float, world: int) -> float:
    """Whole-job microseconds per step of `world` independent replicas: each replica finishes one
    step per `ms_per_step`, so the job finishes `world` steps in that time."""
    return ms_per_step * 1e3 / world


def replica_env(rank: int, world: int, port: int) -> dict:
    """Environment of one replica process started by this script (what torchrun would have set)."""
    env = dict(os.environ)
    env.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    return env


def spawn_replicas(world: int, argv, script=None) -> int:
    """Start `world` copies of this script, one per GPU; rank 0's output (the JSON line) is this process's output."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = [subprocess.Popen([sys.executable, script or os.path.abspath(__file__)] + list(argv), env=replica_env(r, world, port),
                              stdout=None if r == 0 else subprocess.DEVNULL) for r in range(world)]
    rc = 0
    for p in procs:
        rc = p.wait() or rc
    return rc


def omp_threads() -> int:
    v = os.environ.get("OMP_NUM_THREADS")
    return int(v) if v and v.isdigit() else (os.cpu_count() or 1)


# ------------------------------------------------------------------------------------------------
# CPU oracle (the reference arm and the cpu_baseline leg): the only code here that touches oracle/
# ------------------------------------------------------------------------------------------------
def oracle_steps(cfg, weights, parent, prefix_len, rng, max_steps, warmup, budget_s):
    """Times full oracle steps (verify + accept + commit of the whole tree at the full prefix).  Returns the step times (s)."""
    from oracle import ssd_oracle
    model = ssd_oracle.Model(cfg, weights)
    kv = model.new_kv()
    V, n = cfg["vocab"], len(parent)
    deadline = time.time() + budget_s
    kv.prefill(ssd_synth.uniform_tokens(prefix_len, V, rng), chunk=min(prefix_len, 256) or 1)

    def step():
        tokens = ssd_synth.uniform_tokens(n, V, rng)
        logits = kv.verify_tree(tokens, parent)
        path, nxt, _ = ssd_oracle.accept_tree(logits, None, tokens, parent, mode=0)
        kv.commit(path)
        kv.rollback(prefix_len)

    for _ in range(warmup):
        if time.time() > deadline:
            break
        step()
    times = []
    for _ in range(max_steps):
        t0 = time.perf_counter()
        step()
        times.append(time.perf_counter() - t0)
        if time.time() > deadline:
            break
    return times


def run_reference(args):
    """The CPU oracle, as it stands, timed on the host cores (rank 0 only) on the metric's full workload."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    cfg, parent = workload(args)
    rng = np.random.default_rng(1002)
    weights = ssd_synth.make_weights(cfg, seed=0)
    times = oracle_steps(cfg, weights, parent, args.prefix, rng, args.steps, min(args.warmup, 1), args.ref_budget_s)
    us = float(np.median(times)) * 1e6
    sample = ("full oracle steps (verify + accept + commit of the %d-node tree at prefix %d), median of %d of %d steps "
              "(time budget %g s)" % (args.nodes, args.prefix, len(times), args.steps, args.ref_budget_s))
    line = {"impl": "reference", "metric": METRIC, "value": us, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": us / 1e3, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic",
            "config": {"workload": "%s verify n=%d prefix=%d, greedy accept, commit (CPU oracle)" % (args.model, args.nodes, args.prefix)},
            "cpu_baseline": {"value": us, "unit": UNIT, "cores": omp_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# GPU arm
# ------------------------------------------------------------------------------------------------
class Runner:
    """One model on the device with a prefilled cache; times steps of a given tree."""

    def __init__(self, model, prefix_len, device, tune=(), seed=0, rng_seed=1002, dtype=None):
        import torch
        import paper_2308_04623_b200 as ssd
        self.torch, self.ssd = torch, ssd
        self.cfg = ssd_synth.config(model, **({"dtype": dtype} if dtype else {}))
        self.model, self.P, self.V = model, prefix_len, self.cfg["vocab"]
        self.rng = np.random.default_rng(rng_seed)
        self.weights = ssd_synth.make_weights(self.cfg, seed=seed)
        self.stream = torch.cuda.current_stream()
        self.ctx = ssd.Context(self.cfg, device=device, stream=self.stream.cuda_stream)
        self.ctx.load_weights(ssd_synth.bf16_bits(self.weights) if self.cfg["dtype"] != "fp32" else self.weights)
        for spec in tune:
            knob, value = spec.split("=")
            self.ctx.set_tuning(int(knob), int(value))
        self.kv = self.ctx.new_kv()
        self.logits = torch.empty((256, self.V), dtype=torch.float32, device="cuda")
        self.prefix = ssd_synth.uniform_tokens(prefix_len, self.V, self.rng)
        for s in range(0, prefix_len, 256):  # prefix through hot-path calls only: chain trees, every node committed
            t = self.prefix[s:s + 256]
            self.ctx.verify_tree(t, ssd_synth.tree_chain(len(t)), self.kv, self.logits.data_ptr())
            self.ctx.kv_commit(self.kv, np.arange(len(t), dtype=np.int32))
        self.srng = ssd.binding.ssd_rng(1, 0)
        self.evict = None

    def planted_tokens(self, parent, sets, probability):
        """Random token ids with the verifier's arg-max planted on children, level by level (untimed)."""
        torch = self.torch
        n = len(parent)
        depth = ssd_synth.tree_depths(parent)
        out = []
        for _ in range(sets):
            tokens = ssd_synth.uniform_tokens(n, self.V, self.rng)
            for lvl in range(1, int(depth.max()) + 1 if n > 1 else 0):
                self.ctx.verify_tree(tokens, parent, self.kv, self.logits.data_ptr())
                best = torch.argmax(self.logits[:n], dim=1).cpu().numpy()
                for c in np.nonzero(depth == lvl)[0]:
                    if self.rng.random() < probability:
                        tokens[c] = int(best[parent[c]])
            out.append(tokens)
        return out

    def time_steps(self, parent, token_sets, steps, warmup, draft=None, sampling=None, evict_l2=False):
        """Runs warmup + steps full steps; device time of the whole loop and of every verify call."""
        torch, ssd, ctx, kv = self.torch, self.ssd, self.ctx, self.kv
        if evict_l2 and self.evict is None:
            self.evict = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")  # larger than the 126 MB L2

        def one(i, ev=None):
            tokens = token_sets[i % len(token_sets)]
            if evict_l2:
                self.evict.add_(1)
            if ev is not None:
                ev[0].record(self.stream)
            ctx.verify_tree(tokens, parent, kv, self.logits.data_ptr())
            if ev is not None:
                ev[1].record(self.stream)
            if sampling:
                path, nxt = ctx.accept_tree(self.logits.data_ptr(), draft.data_ptr(), tokens, parent, mode=ssd.SSD_SAMPLING,
                                            temperature=sampling[0], top_k=sampling[1], rng=self.srng)
            else:
                path, nxt = ctx.accept_tree(self.logits.data_ptr(), None, tokens, parent, mode=ssd.SSD_GREEDY, rng=self.srng)
            ctx.kv_commit(kv, path)
            kv.rollback(self.P)
            return len(path)

        for i in range(warmup):
            one(i)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        vev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        lengths = []
        launches0 = ctx.kernel_launches()
        t0 = time.perf_counter()
        e0.record(self.stream)
        for k in range(steps):
            lengths.append(one(warmup + k, vev[k]))
        e1.record(self.stream)
        torch.cuda.synchronize()
        wall = time.perf_counter() - t0
        return {"dev_ms": e0.elapsed_time(e1), "wall_ms": wall * 1e3, "verify_us": [a.elapsed_time(b) * 1e3 for a, b in vev],
                "lengths": lengths, "launches": ctx.kernel_launches() - launches0}

    def kernel_timeline(self, parent, tokens):
        """Per-kernel device time of one forward from the library's timeline (nanosecond timer stamps taken inside the
        kernels): for every kernel the time from its dependencies being met to its latest CTA's end."""
        ssd, ctx = self.ssd, self.ctx
        ctx.set_tuning(ssd.SSD_TUNE_KERNEL_TRACE, 1)
        for _ in range(3):
            ctx.verify_tree(tokens, parent, self.kv, self.logits.data_ptr())
        self.torch.cuda.synchronize()
        t = ctx.phase_trace().astype(np.int64).reshape(-1, 8)
        ctx.set_tuning(ssd.SSD_TUNE_KERNEL_TRACE, 0)
        return t

    def close(self):
        self.kv.close()
        self.ctx.close()


def per_kernel_roofline(run: Runner, parent, tokens, peak_gbs):
    """Achieved HBM GB/s of each projection kernel of a layer and of the LM head, from the device-side timeline."""
    cfg = run.cfg
    L, d, F, V = cfg["n_layer"], cfg["d_model"], cfg["d_ff"], cfg["vocab"]
    t = run.kernel_timeline(parent, tokens)
    setup = 3  # tree preparation, clearing of the logits and embedding are not traced
    per = (len(t) - setup - 2) // L
    if per not in (5, 8) or len(t) != setup + per * L + 2:
        return None
    body = t[setup:setup + per * L].reshape(L, per, 8)
    dur = (body[:, :, 6] - body[:, :, 1]) / 1e3  # dependencies met -> latest end, us
    med = np.median(dur[2:], axis=0)
    names = ["ln1", "qkv", "attention", "o_proj", "ln2", "fc", "gelu", "proj"] if per == 8 else ["qkv", "attention", "o_proj", "fc", "proj"]
    mb = 1 if cfg["dtype"] == "bf16_w8" else 2   # bytes per matrix entry (8-bit codes carry 4 more bytes per output row)
    rows_of = {"qkv": 3 * d, "o_proj": d, "fc": F, "proj": d}
    weight_bytes = {"qkv": mb * 3 * d * d, "o_proj": mb * d * d, "fc": mb * d * F, "proj": mb * d * F}
    if mb == 1:
        weight_bytes = {k: v + 4 * rows_of[k] for k, v in weight_bytes.items()}
    out = {}
    for name, us in zip(names, med):
        e = {"us": float(us)}
        if name in weight_bytes:
            e["algorithmic_bytes"] = weight_bytes[name]
            e["achieved_gbs"] = weight_bytes[name] / (us * 1e-6) / 1e9
            e["frac"] = e["achieved_gbs"] / peak_gbs
        out[name] = e
    head_us = float(t[-1, 6] - t[-1, 1]) / 1e3
    head_bytes = mb * V * d + (4 * V if mb == 1 else 0) + 4 * len(parent) * V
    out["lm_head"] = {"us": head_us, "algorithmic_bytes": head_bytes, "achieved_gbs": head_bytes / (head_us * 1e-6) / 1e9,
                      "frac": head_bytes / (head_us * 1e-6) / 1e9 / peak_gbs}
    deps = body[:, 0, 1].astype(np.float64)
    out["layer_us"] = float((deps[-1] - deps[2]) / (L - 3) / 1e3)
    out["how"] = ("device timer stamps taken inside the kernels of one traced forward (dependencies met -> latest CTA end), "
                  "median over layers; tracing itself slows the forward by a few percent")
    # The chain itself: from one kernel's dependencies being met to the next one's (median over layers), and one middle layer's
    # stamps relative to its first kernel's dependencies (first CTA: entry, dependencies met, first accumulator complete - the
    # projections only - and end; then the latest end over all CTAs).
    flat = np.concatenate([body[:, :, 1].reshape(-1), [t[setup + per * L, 1]]]).astype(np.float64)
    step = np.diff(flat).reshape(L, per)
    out["phase_us"] = {name: float(v) for name, v in zip(names, np.median(step[2:], axis=0) / 1e3)}
    mid = body[L // 2]
    t0 = mid[0, 1]
    rel = lambda v: None if v == 0 else round(float(v - t0) / 1e3, 2)
    out["timeline_us"] = {"layer": L // 2, "columns": ["entry", "dependencies_met", "accumulator", "end", "latest_end"],
                          "rows": {name: [rel(r[0]), rel(r[1]), rel(r[3]), rel(r[2]), rel(r[6])] for name, r in zip(names, mid)}}
    return out


def sweep_entry(label, cfg, n, P, res, peaks):
    v = percentiles(res["verify_us"])
    alg = ssd_synth.algorithmic_bytes(cfg, P, n)
    fl = gemm_flops(cfg, n)
    gbs = alg / (v["median"] * 1e-6) / 1e9
    return {"workload": label, "n_nodes": n, "prefix": P, "verify_us": v, "step_us": res["dev_ms"] * 1e3 / len(res["verify_us"]),
            "algorithmic_bytes": alg, "achieved_gbs": gbs, "frac_hbm_measured": gbs / peaks["hbm_gbs"], "frac_hbm_8TBs": gbs / NOMINAL_HBM_GBS,
            "gemm_flops": fl, "frac_tensor_sustained": fl / (v["median"] * 1e-6) / 1e12 / peaks["bf16_tflops_sustained"],
            "bound_us": {"hbm": alg / peaks["hbm_gbs"] / 1e3, "tensor": fl / peaks["bf16_tflops_sustained"] / 1e6},
            "accepted_nodes_per_step": float(np.mean(res["lengths"]))}


def run_sweep(args, local, peaks):
    """The other configurations the benchmark is defined on, measured in the same process (one GPU only)."""
    out = {}
    steps, warm = max(10, min(args.steps, 30)), 3
    # ---- GPT-2-small-shaped draft verified in the second stage: 512-token prefix, eight-node trigram tree
    run = Runner("gpt2_small", 512, local, args.tune)
    tokens, parent, rows = ssd_synth.trigram_tree(11, 22, 33, run.V)
    warm_res = run.time_steps(parent, [tokens], steps, warm)
    cold_res = run.time_steps(parent, [tokens], steps, warm, evict_l2=True)
    e = sweep_entry("gpt2_small stage-two verify, trigram tree", run.cfg, len(parent), 512, warm_res, peaks)
    e["verify_us_l2_evicted"] = percentiles(cold_res["verify_us"])
    e["l2_note"] = "268 MB of algorithmic bytes against a 126 MB L2: 'evicted' writes a 256 MB buffer between steps"
    out["config3"] = e
    run.close()
    del run
    # ---- GPT-2-XL-shaped model: tree sizes 8..256, random parents with depth <= 8
    # (one model, prefilled to the longest prefix; the shorter prefixes are the same cache rolled back)
    run = Runner("gpt2_xl", 960, local, args.tune)
    rows_xl, other_prefixes = [], []
    trees = {n: (ssd_synth.tree_random(n, 8, run.rng), [ssd_synth.uniform_tokens(n, run.V, run.rng) for _ in range(4)]) for n in (8, 16, 32, 64, 128, 256)}
    for P in (960, 512, 128):
        run.kv.rollback(P)
        run.P = P
        for n, (parent, toks) in trees.items():
            e = sweep_entry("gpt2_xl verify, random tree of depth <= 8", run.cfg, n, P, run.time_steps(parent, toks, steps if P == 512 else 10, warm), peaks)
            (rows_xl if P == 512 else other_prefixes).append(e if P == 512 else {k: e[k] for k in ("n_nodes", "prefix", "verify_us", "frac_hbm_measured", "frac_tensor_sustained", "bound_us")})
    cfg = run.cfg
    run.close()
    del run
    # the tree size at which the tensor bound (at the sustained bf16 peak) overtakes the HBM bound (at the measured copy bandwidth)
    cross = None
    for n in range(1, 1025):
        if gemm_flops(cfg, n) / (peaks["bf16_tflops_sustained"] * 1e12) > ssd_synth.algorithmic_bytes(cfg, 512, n) / (peaks["hbm_gbs"] * 1e9):
            cross = n
            break
    t = [r["verify_us"]["median"] for r in rows_xl]
    out["config5"] = {"rows": rows_xl, "rows_prefix_960_and_128": other_prefixes, "crossover_nodes_of_the_bounds": cross,
                      "measured_us_per_node_beyond_64": (t[5] - t[3]) / (256 - 64),
                      "note": "below the crossover the forward can at best run at the HBM bound, above it at the tensor bound; measured times "
                              "are several times either bound (a chain of dependent kernels), and grow roughly linearly in the tree size from 64 nodes on"}
    return out


def run_w8(args, local, peaks):
    """8-bit weight streaming (the paper's closing list of next steps, item 2) beside the bf16 model, same trees and tokens: verify time, the
    algorithmic bytes of each (codes of one byte and a scale per row against two bytes) and the fraction of the copy bandwidth."""
    out = []
    steps = max(10, min(args.steps, 30))
    for model, P, n in ((args.model, args.prefix, 32), ("gpt2_xl", 512, 32)):
        par = ssd_synth.tree_branching(n, tree_rule(n))
        row = {"workload": "%s verify n=%d prefix=%d" % (model, n, P)}
        for dtype in ("bf16", "bf16_w8"):
            run = Runner(model, P, local, args.tune, dtype=dtype)
            toks = [ssd_synth.uniform_tokens(n, run.V, run.rng) for _ in range(4)]
            e = sweep_entry(model, run.cfg, n, P, run.time_steps(par, toks, steps, 3), peaks)
            row[dtype] = {k: e[k] for k in ("verify_us", "algorithmic_bytes", "achieved_gbs", "frac_hbm_measured", "bound_us")}
            run.close()
            del run
        row["w8_time_over_bf16"] = row["bf16_w8"]["verify_us"]["median"] / row["bf16"]["verify_us"]["median"]
        out.append(row)
    return {"rows": out, "note": "codes go to the 8-bit tensor-core kind unconverted; activations as four e4m3 planes; the forward is a chain of "
                                 "dependent kernels, so halving the streamed bytes moves the LM head (HBM-bound) and little else"}


def run_staged(args, local, peaks, alphas=(0.3, 0.6, 0.9), n_tokens=256):
    """The full staged loop at the benchmark's sizes with the acceptance made controllable: GPT-2-Large-shaped target,
    GPT-2-small-shaped draft, a trigram table built from a synthetic stream.  Random-weight models never agree, so - as
    the configuration defines it - every proposal row of the target's tree is alpha * softmax(target logits at the parent)
    + (1 - alpha) * Dirichlet(0.5), children drawn independently from it; the harness obtains those rows by running the
    target level by level (untimed).  What is timed, with CUDA events around each stage, is the method's own work per
    step: the draft speculated by the trigram (rounds x [table look-up, draft verify of the eight-node tree, acceptance
    with one-entry rows, the draft's laws and sibling picks, commit]), and the target's verify of the 32-node tree,
    sampling acceptance and commit.  The draft's outputs do not feed the synthetic tree: this is the cost of the pipeline
    at a controlled acceptance, not a language-model run."""
    import torch
    import paper_2308_04623_b200 as ssd
    tgt = Runner(args.model, 64, local, args.tune, rng_seed=4004)
    drf = Runner("gpt2_small", 64, local, args.tune, rng_seed=4004)
    V = tgt.V
    stream_tokens = np.random.default_rng(4).zipf(1.3, size=200000) % V
    tri = ssd.Trigram(stream_tokens.astype(np.int32), V, device=local, stream=tgt.stream.cuda_stream)
    parent = ssd_synth.tree_branching(32, tree_rule(32))
    depth = ssd_synth.tree_depths(parent)
    n = len(parent)
    kids = {p: [c for c in range(n) if parent[c] == p] for p in range(n)}
    tri_parent = ssd_synth.tree_chain_plus_branch()
    rows = torch.zeros((n, V), dtype=torch.float32, device="cuda")
    dlogits = torch.empty((16, V), dtype=torch.float32, device="cuda")
    drows = torch.empty((16, V), dtype=torch.float32, device="cuda")
    gen = torch.Generator(device="cuda")
    out = {}
    # (a short untimed run first: graph captures, first launches of the sampling kernels and buffer growth happen there)
    for alpha, n_tokens_run in [(0.5, 16)] + [(a, n_tokens) for a in alphas]:
        gen.manual_seed(int(alpha * 1000))
        tgt.kv.rollback(64)
        drf.kv.rollback(64)
        srng = ssd.binding.ssd_rng(int(alpha * 100), 0)
        seq = list(tgt.prefix) + [int(tgt.rng.integers(V))]
        emitted, steps, t_draft, t_target, lengths = 0, 0, 0.0, 0.0, []
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        while emitted < n_tokens_run and len(tgt.kv) + 40 < tgt.cfg["n_ctx"]:
            root = seq[-1]
            # ---- timed: the draft stage (its results are not used for the synthetic tree)
            base = len(drf.kv)
            ev[0].record(tgt.stream)
            for _ in range(2):
                ttok, _ = tri.propose(seq[-2], root, tri_parent)
                drf.ctx.verify_tree(ttok, tri_parent, drf.kv, dlogits.data_ptr())
                idx = np.concatenate([[-1], ttok[1:]]).astype(np.int32).reshape(-1, 1)
                path1, _ = drf.ctx.accept_tree_sparse(dlogits.data_ptr(), idx, np.ones((8, 1), dtype=np.float32), ttok, tri_parent,
                                                       mode=ssd.SSD_SAMPLING, rng=srng)
                drf.ctx.propose_children(dlogits.data_ptr(), path1, 1, mode=ssd.SSD_SAMPLING, rng=srng, rows_out_ptr=drows.data_ptr())
                drf.ctx.kv_commit(drf.kv, path1)
                drf.kv.rollback(base)
            ev[1].record(tgt.stream)
            # ---- untimed harness: the synthetic tree, level by level
            tokens = np.zeros(n, dtype=np.int32)
            tokens[0] = root
            for d in range(int(depth.max())):
                nd = int((depth <= d).sum())
                tgt.ctx.verify_tree(tokens[:nd], parent[:nd], tgt.kv, tgt.logits.data_ptr())
                for p in np.nonzero(depth == d)[0]:
                    if not kids[int(p)]:
                        continue
                    g = 0.5 * torch.randn(V, device="cuda", generator=gen) ** 2      # Gamma(1/2) draws: a Dirichlet(1/2) row once normalised
                    q = alpha * torch.softmax(tgt.logits[int(p)].double(), 0) + (1.0 - alpha) * (g / g.sum()).double()
                    picks = torch.multinomial(q, len(kids[int(p)]), replacement=True, generator=gen).cpu().numpy()
                    for c, t in zip(kids[int(p)], picks):
                        tokens[c] = int(t)
                        rows[c] = q.float()
            # ---- timed: the target stage
            ev[2].record(tgt.stream)
            tgt.ctx.verify_tree(tokens, parent, tgt.kv, tgt.logits.data_ptr())
            path0, next0 = tgt.ctx.accept_tree(tgt.logits.data_ptr(), rows.data_ptr(), tokens, parent, mode=ssd.SSD_SAMPLING, rng=srng)
            tgt.ctx.kv_commit(tgt.kv, path0)
            ev[3].record(tgt.stream)
            torch.cuda.synchronize()
            t_draft += ev[0].elapsed_time(ev[1])
            t_target += ev[2].elapsed_time(ev[3])
            new = [int(tokens[c]) for c in path0[1:]] + [int(next0)]
            # (untimed) the draft's cache follows the emitted sequence
            chain = np.asarray([root] + new[:-1], dtype=np.int32)
            drf.ctx.verify_tree(chain, ssd_synth.tree_chain(len(chain)), drf.kv, dlogits.data_ptr())
            drf.ctx.kv_commit(drf.kv, np.arange(len(chain), dtype=np.int32))
            seq += new
            emitted += len(new)
            lengths.append(len(new))
            steps += 1
        method_ms = t_draft + t_target
        if n_tokens_run != n_tokens:
            continue
        out["alpha_%g" % alpha] = {
            "emitted_tokens": emitted, "target_steps": steps, "tokens_per_target_step": emitted / steps,
            "tokens_per_s": emitted / (method_ms * 1e-3), "us_per_step": {"draft_stage": t_draft * 1e3 / steps, "target_stage": t_target * 1e3 / steps},
            "accepted_length_histogram": {str(k): int(lengths.count(k)) for k in sorted(set(lengths))}}
    out["note"] = ("synthetic acceptance: proposal rows = alpha * softmax(target logits at the parent) + (1 - alpha) * Dirichlet(0.5), built by "
                   "untimed level-by-level target forwards; timed = draft stage (2 rounds of trigram look-up, 8-node draft verify, acceptance, "
                   "proposals, commit) + target stage (32-node verify, sampling acceptance, commit); prefix 64 growing with the emitted tokens")
    tri.close()
    tgt.close()
    drf.close()
    return out


def run_staged_decoder(local, n_tokens=192, prompt_len=64, table_tokens=320):
    """The three-stage loop itself (target <- draft <- trigram table) through the public API, set up so that all three stages
    contribute tokens although the weights are random: the GPT-2-small-shaped model is the target AND its own draft, decoding is
    deterministic, and the trigram table is built from the model's own continuation of the prompt (as the paper builds its
    table from samples of the draft).  Reports which stage every emitted token came from, tokens per target forward and the
    loop's tokens/s (host bookkeeping of the loop included), and whether the output equals plain one-token-at-a-time decoding."""
    import torch
    import paper_2308_04623_b200 as ssd
    from paper_2308_04623_b200.staged import StagedDecoder
    cfg = ssd_synth.config("gpt2_small")
    V = cfg["vocab"]
    bits = ssd_synth.bf16_bits(ssd_synth.make_weights(cfg, seed=11))
    stream = torch.cuda.current_stream()
    c0 = ssd.Context(cfg, device=local, stream=stream.cuda_stream)
    c1 = ssd.Context(cfg, device=local, stream=stream.cuda_stream)
    c0.load_weights(bits)
    c1.load_weights(bits)
    prompt = [int(t) for t in ssd_synth.uniform_tokens(prompt_len, V, np.random.default_rng(12))]
    # plain decoding: one node per forward
    kv = c0.new_kv()
    buf = torch.empty((64, V), dtype=torch.float32, device="cuda")
    body = np.asarray(prompt[:-1], dtype=np.int32)
    c0.verify_tree(body, ssd_synth.tree_chain(len(body)), kv, buf.data_ptr())
    c0.kv_commit(kv, np.arange(len(body), dtype=np.int32))
    plain, tok = [], prompt[-1]
    one, root_only = np.zeros(1, dtype=np.int32), np.array([-1], dtype=np.int32)
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for i in range(table_tokens):
        if i == 32:   # (the first steps carry the graph capture of the one-node forward)
            p0.record(stream)
        one[0] = tok
        c0.verify_tree(one, root_only, kv, buf.data_ptr())
        c0.kv_commit(kv, np.zeros(1, dtype=np.int32))
        tok = int(torch.argmax(buf[0]).item())
        plain.append(tok)
    p1.record(stream)
    torch.cuda.synchronize()
    plain_tok_s = (table_tokens - 32) / (p0.elapsed_time(p1) * 1e-3)
    kv.close()
    tri = ssd.Trigram(np.asarray(prompt + plain, dtype=np.int32), V, device=local, stream=stream.cuda_stream)
    res = None
    for timed in (False, True):   # (an untimed pass first: graph captures and first launches)
        dec = StagedDecoder(c0, c1, tri, mode=ssd.SSD_GREEDY, rounds=2, siblings=1, seed=3)
        dec.prefill(prompt)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        got = dec.generate(n_tokens if timed else 24)
        e1.record(stream)
        torch.cuda.synchronize()
        if timed:
            ms = e0.elapsed_time(e1)
            st = dec.stats
            res = {"emitted_tokens": len(got), "target_forwards": st["target_steps"], "draft_forwards": st["draft_forwards"],
                   "tokens_per_target_forward": st["emitted"] / max(1, st["target_steps"]), "tokens_per_s": len(got) / (ms * 1e-3),
                   "token_origin": dict(st["origin"]), "equals_plain_decoding": got == plain[:len(got)],
                   "plain_decoding_tokens_per_s": plain_tok_s,
                   "note": "GPT-2-small-shaped random weights as target and as its own draft, deterministic decoding, trigram table "
                           "built from the model's own continuation of the 64-token prompt; the loop's host bookkeeping is inside the time"}
        dec.close()
    tri.close()
    c0.close()
    c1.close()
    return res


def run_gpu(args):
    import torch

    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    cfg, parent = workload(args)
    n, P = len(parent), args.prefix
    run = Runner(args.model, P, local, args.tune, rng_seed=1002 + rank, dtype=args.weights)
    sampling = (args.temperature, args.top_k) if args.accept == "sampling" else None
    draft = torch.from_numpy(ssd_synth.draft_rows_gamma(n, run.V, run.rng)).cuda() if sampling else None
    token_sets = run.planted_tokens(parent, args.plant_sets, PLANT_PROBABILITY)

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    run.time_steps(parent, token_sets, 1, args.warmup, draft, sampling)  # warm-up
    barrier()
    res = run.time_steps(parent, token_sets, args.steps, 0, draft, sampling)  # ---- the timed region: exactly K steps
    barrier()
    if rank == 0:  # the same steps, untimed, until the sampler has seen the GPU under this load a few times
        t_end = time.perf_counter() + 2.0
        while sampler.proc and sampler.count() < 4 and time.perf_counter() < t_end:
            run.time_steps(parent, token_sets, 20, 0, draft, sampling)
    clocks = sampler.stop() if rank == 0 else {}
    status = run.ctx.device_status()
    v = percentiles(res["verify_us"])
    dev_ms, wall_ms, verify_med = max_over_ranks([res["dev_ms"], res["wall_ms"], v["median"]])
    if rank != 0:
        run.close()
        return
    ms_per_step = dev_ms / args.steps
    peaks, peak_kind = measured_peaks()
    alg_bytes = ssd_synth.algorithmic_bytes(cfg, P, n)
    achieved = alg_bytes / (verify_med * 1e-6) / 1e9
    lengths = np.asarray(res["lengths"])
    hist = {str(k): int((lengths == k).sum()) for k in sorted(set(lengths.tolist()))}
    line = {
        "metric": METRIC, "value": replica_value(ms_per_step, world), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16" if cfg["dtype"] != "fp32" else "f32", "data": "synthetic",
        "config": {"workload": "%s%s verify n=%d prefix=%d, %s accept, commit" % (
                       args.model, " (matrices as 8-bit codes)" if cfg["dtype"] == "bf16_w8" else "", n, P, ("sampling (T=%g, top-k=%d)" % (args.temperature, args.top_k)) if sampling else "greedy"),
                   "tree": "branching %s BFS truncated at %d" % (list(tree_rule(n)), n),
                   "tokens": "uniform ids, the verifier's arg-max planted on each child with probability %g" % PLANT_PROBABILITY,
                   "l2": "inputs larger than L2 (%.0f MB of weights per step)" % (alg_bytes / 1e6), "replicas": world,
                   "aggregate": "per-replica step time / n_gpus", "accepted_nodes_per_step": float(lengths.mean()),
                   "accepted_path_length_histogram": hist},
        "verify_us": verify_med, "verify_us_percentiles": v, "steps_per_s": world * 1e3 / ms_per_step,
        # every node of the accepted path (the root included) emits one token: tokens[path[1:]] and the extra one
        "emitted_tokens_per_s": world * 1e3 / ms_per_step * float(lengths.mean()),
        "roofline": {"bound": "hbm", "kernel": "ssd_verify_tree (all launches of one forward; per-kernel figures under roofline_per_kernel)",
                     "achieved": achieved, "peak": peaks["hbm_gbs"], "peak_kind": "of " + peak_kind, "unit": "GB/s",
                     "frac": achieved / peaks["hbm_gbs"], "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS, "algorithmic_bytes": alg_bytes,
                     "traffic": NCU_TRAFFIC_BYTES.get((args.model, n, P))},
        "e2e": {"value": wall_ms * 1e3 / args.steps / world, "unit": UNIT, "h2d_bytes_per_step": 4 * n * 4 + 4 * n,
                "d2h_bytes_per_step": 4 * (n + 4)},
        "gpu_launches": int(res["launches"]), "clocks": clocks, "device_status": status,
    }
    if world == 1:
        line["roofline_per_kernel"] = per_kernel_roofline(run, parent, token_sets[0], peaks["hbm_gbs"])
    weights = run.weights
    run.close()
    del run
    if world == 1 and not args.no_sweep:
        sweep = {}
        for nn in (16, 64):
            r2 = Runner(args.model, P, local, args.tune)
            par = ssd_synth.tree_branching(nn, tree_rule(nn))
            toks = r2.planted_tokens(par, 4, PLANT_PROBABILITY)
            sweep["n%d" % nn] = sweep_entry("%s verify" % args.model, cfg, nn, P, r2.time_steps(par, toks, max(10, min(args.steps, 30)), 3), peaks)
            r2.close()
            del r2
        sweep.update(run_sweep(args, local, peaks))
        sweep["config4"] = run_staged(args, local, peaks)
        sweep["config4"]["staged_decoder_self_draft"] = run_staged_decoder(local)
        sweep["w8"] = run_w8(args, local, peaks)
        line["sweep"] = sweep
    if world == 1 and not args.no_cpu_baseline:
        times = oracle_steps(cfg, weights, parent, P, np.random.default_rng(7), 3, 0, 60.0)
        line["cpu_baseline"] = {"value": float(np.median(times)) * 1e6, "unit": UNIT, "cores": omp_threads(), "kind": "oracle",
                                "sample": "%d full oracle steps (the whole %d-node tree at prefix %d), median" % (len(times), n, P)}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ssd", choices=["ssd", "reference"])
    ap.add_argument("--model", default="gpt2_large")
    ap.add_argument("--nodes", type=int, default=32)
    ap.add_argument("--prefix", type=int, default=256)
    ap.add_argument("--ref-budget-s", type=float, default=150.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="skip the other configurations (16 / 64 nodes, draft model, XL sweep)")
    ap.add_argument("--plant-sets", type=int, default=8, help="token sets prepared before the timed region (fewer = fewer launches before it, for profiling)")
    ap.add_argument("--weights", default="bf16", choices=["bf16", "bf16_w8"],
                    help="how the library holds the matrices it streams: bf16 (the benchmark's configuration) or 8-bit codes with per-row scales")
    ap.add_argument("--tune", action="append", default=[], help="knob=value for ssd_set_tuning (experiments)")
    ap.add_argument("--accept", default="greedy", choices=["greedy", "sampling"],
                    help="acceptance rule of the step (the metric's workload is greedy; sampling draws draft rows from a Dirichlet)")
    ap.add_argument("--top-k", type=int, default=0, help="top-k warp of the verifier's distribution (sampling only; 0 = off)")
    ap.add_argument("--temperature", type=float, default=1.0)
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ssd" else args.warmup
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_replicas(args.gpus, sys.argv[1:]))  # one process per GPU; under torchrun the ranks exist already
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
