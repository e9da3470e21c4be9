#!/usr/bin/env python
"""Benchmark of the GXPO active step on B200.

A "step" is one whole active step of Algorithm 1's parameter-space update over
the workload's tensor list: probe step 0, probe step 1, extrapolate + reposition,
slow step with the in-sweep norm, gate update.  By default that is 3 sweeps + 1 tiny
kernel moving 68 bytes per parameter (--flow deferred: the first probe step and, since
the benchmark's g0 and g1 buffers stay intact, the fused second-probe + extrapolation
sweep too leave m, v to the slow step's sweep; 72 with --no-persist); --flow fused moves
84, --flow unfused (the four separate calls) 94.  The three gradient buffers are
synthetic and already resident.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
With --gpus N > 1 every GPU runs the step on a list of its own (the update shards without
any exchange but the 8-byte sum behind the gate).  Under a launcher that has set
WORLD_SIZE (torch.distributed.run) this process is one of its ranks; without one it starts
the N ranks itself, one process per GPU.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "GXPO active-step params/sec"
UNIT = "params/s"
# Which kernel serves a call, and how many bytes per parameter it has to move, is the
# library's decision (list length, optimizer, promise, diagnostics, tuning): the benchmark
# asks it after each call of a warm-up step (gxpo_last_sweep) and repeats none of its rules.


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="qwen25_7b",
                    choices=["qwen25_7b", "llama31_8b", "flat_1p54b", "flat_2p5b", "lora_qwen25_7b", "surrogate_1e8", "small", "flat"])
    ap.add_argument("--params", type=int, default=1 << 26, help="size of the 'flat' workload")
    ap.add_argument("--layers", type=int, default=0, help="override the decoder depth (0 = full)")
    ap.add_argument("--K", type=int, default=5)
    ap.add_argument("--alpha", type=float, default=0.5)
    ap.add_argument("--lr", type=float, default=1e-7)
    ap.add_argument("--placement", type=int, default=0)
    ap.add_argument("--variant", type=int, default=0)
    ap.add_argument("--ctas", type=int, default=0)
    ap.add_argument("--unit-tiles", type=int, default=0)
    ap.add_argument("--fallback", action="store_true", help="time the single-pass fallback step")
    ap.add_argument("--flow", default="deferred", choices=["deferred", "fused", "unfused"],
                    help="deferred: probe_step_deferred + probe_extrapolate (68 B/param on long lists, default); "
                         "fused: probe_step(0) + probe_extrapolate (84); unfused: the four separate sweeps (94)")
    ap.add_argument("--emit-bf16", action="store_true",
                    help="also keep bfloat16 model-weight copies (gxpo_bind_model_weights), so that the caller needs no "
                         "cast sweeps: theta1 and theta-tilde as bfloat16 only, theta-tilde recomputed by the slow step "
                         "(16 + 18 + 32 = 66 B/param); with --no-persist only theta1 is bfloat16-only (16 + 30 + 28 = 74)")
    ap.add_argument("--no-persist", action="store_true",
                    help="do not promise that g0 and g1 outlive the slow step (72 instead of 68 B/param in the deferred flow)")
    ap.add_argument("--clip", type=float, default=0.0,
                    help="global-norm clipping of every gradient at this value (gxpo_clip_grad_norm: one 2 B/param "
                         "norm pass per gradient, the coefficient applied inside the sweeps); 0 = off")
    ap.add_argument("--diagnostics", action="store_true",
                    help="gather the per-step diagnostics too (adds a 4 B/param <g0, g_slow> pass after the slow step)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-params", type=int, default=1 << 26)
    ap.add_argument("--e2e-staging", type=int, default=1 << 23, help="parameters per staged piece in the e2e leg")
    ap.add_argument("--cpu-params", type=int, default=1 << 24)
    return ap.parse_args()


def workload_shapes(args):
    from paper_2605_06755_b200 import workloads as w
    if args.workload == "qwen25_7b":
        return w.qwen25_7b_shapes(args.layers or 28), "Qwen2.5-7B-shaped tensor list"
    if args.workload == "llama31_8b":
        return w.llama31_8b_shapes(args.layers or 32), "Llama-3.1-8B-shaped tensor list"
    if args.workload == "lora_qwen25_7b":
        return w.lora_qwen25_7b_shapes(), "rank-128 LoRA adapters (q, k, v, o) of a Qwen2.5-7B-shaped decoder"
    if args.workload == "flat":
        return [("flat", args.params)], f"flat {args.params}-parameter buffer"
    if args.workload == "flat_2p5b":
        return [("flat", 2_500_000_007)], "flat 2,500,000,007-parameter buffer (offsets beyond 2^31 elements)"
    if args.workload == "flat_1p54b":
        return [("flat", w.FLAT_QWEN25_1P5B)], "flat 1.54e9-parameter buffer"
    return w.qwen25_7b_shapes(args.layers or 1), "Qwen2.5-7B-shaped list, reduced depth"


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def recorded_traffic_per_param(kernel_fn, calls):
    """DRAM bytes per parameter of `kernel_fn`, averaged over the named calls, from the
    committed ncu summary profiles/<kernel_fn>_adamw_bf16_flat*.txt (lines
    "dram_bytes_per_param[<call>]: X").  The summary records the hash of the kernel source
    it was taken from; once that source has changed the counters no longer describe the
    kernel and None is returned."""
    import hashlib
    import re
    import glob
    source = os.path.join(ROOT, "paper_2605_06755_b200", "csrc", "gxpo_kernels.cuh")
    try:
        summary = sorted(glob.glob(os.path.join(ROOT, "profiles", f"{kernel_fn}_adamw_bf16_flat*.txt")))[0]
        text = open(summary).read()
        want = re.search(r"^kernel_source_sha256:\s*([0-9a-f]{64})", text, re.M).group(1)
        have = hashlib.sha256(open(source, "rb").read()).hexdigest()
        if have != want:
            return None
        bulk = re.search(r"^bulk_source_sha256:\s*([0-9a-f]{64})", text, re.M)
        if bulk and bulk.group(1) != hashlib.sha256(
                open(os.path.join(os.path.dirname(source), "gxpo_bulk.cuh"), "rb").read()).hexdigest():
            return None
        vals = [float(re.search(r"^dram_bytes_per_param\[%s\]:\s*([0-9.]+)" % re.escape(c), text, re.M).group(1))
                for c in calls]
        return statistics.mean(vals)
    except Exception:
        return None


# ----------------------------------------------------------------------------
# clocks
# ----------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("uuid,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, uuid: str):
        self.uuid = uuid
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) == 8:
                self.rows.append((time.time(), parts))

    def stop(self, t0: float, t1: float):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        mine = [p for (ts, p) in self.rows if (self.uuid in p[0] or not self.uuid) and t0 - 0.05 <= ts <= t1 + 0.15]
        if not mine:
            mine = [p for (ts, p) in self.rows if self.uuid in p[0] or not self.uuid]
        sm = [float(p[1]) for p in mine if p[1].replace(".", "").isdigit()]
        mx = [float(p[2]) for p in mine if p[2].replace(".", "").isdigit()]
        pw = [float(p[3]) for p in mine if p[3].replace(".", "").isdigit()]
        reasons = [n for i, n in enumerate(self.NAMES) if any(p[4 + i].lower().startswith("active") for p in mine)]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "reasons": reasons, "samples": len(mine)}


# ----------------------------------------------------------------------------
# CPU oracle legs
# ----------------------------------------------------------------------------
def oracle_sample(n, seed, K, alpha, lr):
    """Inputs of one active step on an n-parameter slice, as the oracle's float64 arrays."""
    import numpy as np
    from oracle import gxpo_oracle as ora
    from paper_2605_06755_b200 import workloads as w
    th, m, v, g0, g1, gs = w.llm_inputs_numpy(n, seed, "bf16")
    grads = [ora.bf16_bits_to_f64(g) for g in (g0, g1, gs)]
    opt = ora.OptCfg(kind="adamw", lr=lr, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.01)
    cfg = ora.GxpoCfg(K=K, alpha=alpha, delta=float(np.float32(1e-8)))
    st = ora.State(th, opt, m, v)
    return ora, st, cfg, grads


def time_oracle_steps(n, K, alpha, lr, steps, warmup, min_seconds=0.0):
    ora, st, cfg, grads = oracle_sample(n, 1234, K, alpha, lr)
    gate = ora.Gate(cfg)
    fn = lambda which, theta: grads[which]
    import numpy as np
    with np.errstate(all="ignore"):
        for _ in range(warmup):
            ora.train_step(st, gate, cfg, fn, round_f32=True)
        done, t0 = 0, time.perf_counter()
        while done < steps or (time.perf_counter() - t0) < min_seconds:
            ora.train_step(st, gate, cfg, fn, round_f32=True)
            done += 1
        dt = time.perf_counter() - t0
    return done, dt


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    shapes, desc = workload_shapes(args)
    n = args.cpu_params
    done, dt = time_oracle_steps(n, args.K, args.alpha, args.lr, args.steps, args.warmup)
    value = n * done / dt
    sample = (f"{n}-parameter slice drawn with the workload's recipe, one oracle active step "
              f"(double arithmetic, fp32 rounding between calls) per bench step")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": done, "warmup": args.warmup, "ms_per_step": 1e3 * dt / done, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": desc, "params": sum(k for _, k in shapes), "tensors": len(shapes),
                   "optimizer": "AdamW", "K": args.K, "alpha": args.alpha, "lr": args.lr, "grad_dtype": "bf16"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------
# the CUDA path
# ----------------------------------------------------------------------------
def build_device_workload(torch, b, shapes, seed, alias_gslow, with_work=True):
    """with_work=False: no `work` buffer at all (bound as NULL): the step with bfloat16-only
    probe points keeps no point there."""
    from paper_2605_06755_b200 import workloads as w
    d = sum(k for _, k in shapes)
    dev = torch.device("cuda", torch.cuda.current_device())
    theta = torch.empty(d, dtype=torch.float32, device=dev)
    work = torch.empty(d if with_work else 0, dtype=torch.float32, device=dev)
    m = torch.empty(d, dtype=torch.float32, device=dev)
    v = torch.empty(d, dtype=torch.float32, device=dev)
    g0 = torch.empty(d, dtype=torch.bfloat16, device=dev)
    g1 = torch.empty(d, dtype=torch.bfloat16, device=dev)
    gs = g0 if alias_gslow else torch.empty(d, dtype=torch.bfloat16, device=dev)
    w.fill_llm_inputs_torch(theta, m, v, g0, g1, None if alias_gslow else gs, seed)
    work.zero_()
    ptrs, off = [], 0
    for _, k in shapes:
        ptrs.append(b.TensorPtrs(theta.data_ptr() + 4 * off, (work.data_ptr() + 4 * off) if with_work else 0,
                                 m.data_ptr() + 4 * off, v.data_ptr() + 4 * off,
                                 g0.data_ptr() + 2 * off, g1.data_ptr() + 2 * off,
                                 gs.data_ptr() + 2 * off, k))
        off += k
    return d, ptrs, (theta, work, m, v, g0, g1, gs)


def plan_workload(args, free_bytes, margin=6 << 30, extra_bytes=0):
    """Shapes of the workload and whether g_slow has to share g0's buffer (legal: g0 is
    dead once the extrapolation has run) so that 22 -> 20 bytes per parameter fit into
    the free device memory; as a last resort the decoder depth is reduced, and the
    description says so."""
    shapes, desc = workload_shapes(args)
    d = sum(k for _, k in shapes)
    alias = (22 + extra_bytes) * d + margin > free_bytes
    while ((20 if alias else 22) + extra_bytes) * d + margin > free_bytes and args.workload in ("qwen25_7b", "llama31_8b"):
        args.layers = (args.layers or (28 if args.workload == "qwen25_7b" else 32)) - 1
        if args.layers < 1:
            raise SystemExit("not enough free device memory for even one decoder layer")
        shapes, desc = workload_shapes(args)
        desc += f" (reduced to {args.layers} layers: not enough free device memory)"
        d = sum(k for _, k in shapes)
    return shapes, desc, alias


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2605_06755_b200 import build
    build.build_library()
    from paper_2605_06755_b200 import binding as b

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library is the only compute path")
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but {world} rank(s) are running")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        world = dist.get_world_size()        # what the communicator really spans
    props = torch.cuda.get_device_properties(local)
    stream = torch.cuda.current_stream()

    free, total = torch.cuda.mem_get_info()
    emit = bool(getattr(args, "emit_bf16", False)) and args.flow == "deferred" and not args.fallback
    diag = bool(getattr(args, "diagnostics", False)) and not args.fallback
    # bfloat16-only probe points need no `work` buffer: 20 + 2 instead of 24 + 2 bytes per parameter
    # resident.  Possible when the step can run in that mode at all (promise, no diagnostics,
    # staged sweeps) and g_slow then still gets a buffer of its own.
    only16 = False
    if emit and not getattr(args, "no_persist", False) and not diag and args.variant in (0, 3):
        shapes, desc, alias = plan_workload(args, free, extra_bytes=2 - 4)
        only16 = not alias and "reduced" not in desc
    if not only16:
        shapes, desc, alias = plan_workload(args, free, extra_bytes=2 if emit else 0)
    d, ptrs, keep = build_device_workload(torch, b, shapes, 1000 + rank, alias, with_work=not only16)
    sumsq = torch.zeros(1, dtype=torch.float64, device="cuda")

    cfg, opt = b.make_cfg(K=args.K, alpha=args.alpha, lr=args.lr, placement=args.placement)
    ctx = b.Context(cfg, opt, b.BF16)
    ctx.tune(args.ctas, args.variant, args.unit_tiles)
    ctx.bind(ptrs)
    ctx.enable_diagnostics(diag)
    # the benchmark's g0 and g1 are buffers of their own that nothing overwrites: say so
    persist = not getattr(args, "no_persist", False) and args.flow == "deferred" and not alias and not args.fallback
    ctx.set_gradients_persist(persist)
    if emit:
        weights = torch.empty(d, dtype=torch.bfloat16, device="cuda")
        offs, acc = [], 0
        for _, k in shapes:
            offs.append(acc)
            acc += k
        assert persist or not only16
        ctx.bind_model_weights([weights.data_ptr() + 2 * o for o in offs],
                               bf16_only=b.BF16_ONLY_PROBE_POINTS if only16 else b.BF16_ONLY_THETA1)
    if world > 1:
        ctx.set_sumsq_buffer(sumsq.data_ptr())

    flow = args.flow
    names = {"deferred": ["probe_step0_deferred", "probe_extrapolate_deferred", "slow_step"],
             "fused": ["probe_step0", "probe_extrapolate", "slow_step"],
             "unfused": ["probe_step0", "probe_step1", "extrapolate", "slow_step"]}[flow]
    if args.fallback:
        names = ["fallback_step"]
    # the calls behind the names, in order; with --clip a norm pass goes in front of each
    # sweep that consumes a new gradient (the recipe's global-norm clipping)
    calls = {"fallback_step": lambda: ctx.probe_step(-1, stream),
             "probe_step0_deferred": lambda: ctx.probe_step_deferred(stream),
             "probe_step0": lambda: ctx.probe_step(0, stream),
             "probe_step1": lambda: ctx.probe_step(1, stream),
             "extrapolate": lambda: ctx.extrapolate(stream),
             "probe_extrapolate": lambda: ctx.probe_extrapolate(stream),
             "probe_extrapolate_deferred": lambda: ctx.probe_extrapolate(stream),
             "slow_step": lambda: ctx.slow_step(stream)}
    clip = float(getattr(args, "clip", 0.0) or 0.0)
    if clip > 0.0:
        consumes = {"fallback_step": 0, "probe_step0_deferred": 0, "probe_step0": 0, "probe_step1": 1,
                    "probe_extrapolate": 1, "probe_extrapolate_deferred": 1, "slow_step": 2}
        with_clip = []
        for nm in names:
            if nm in consumes:
                k = consumes[nm]
                cn = f"clip_norm_g{k}"
                calls[cn] = (lambda k=k: ctx.clip_grad_norm(k, clip, stream))
                with_clip.append(cn)
            with_clip.append(nm)
        names = with_clip
    n_ev = len(names) + 1

    def one_step(evs=None, sweeps=None):
        if evs:
            evs[0].record(stream)
        for i, nm in enumerate(names):
            calls[nm]()
            if sweeps is not None:
                sweeps[nm] = ctx.last_sweep()
            if evs:
                evs[i + 1].record(stream)
        if args.fallback:
            return None
        if world > 1:
            dist.all_reduce(sumsq)        # the one exchange of a sharded step: 8 bytes
        return ctx.gate_update(stream, allow_nonfinite=True)

    sweeps = {}
    for i in range(max(args.warmup, 3)):
        one_step(sweeps=sweeps if i == 0 else None)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    # Label the calls by what the library launched for them: the summaries under profiles/
    # are keyed by these labels.
    G = 2                                                     # bfloat16 gradients
    relabel = {}
    if "probe_extrapolate_deferred" in sweeps and sweeps["probe_extrapolate_deferred"].kernel == b"fused_bulk_light_kernel":
        relabel["probe_extrapolate_deferred"] = ("probe_extrapolate_nostate"     # m, v left unwritten
                                                 if sweeps["probe_extrapolate_deferred"].bytes_written_per_param >= 4 else
                                                 "probe_extrapolate_bf16only")   # and theta-tilde as bfloat16 only
    if "slow_step" in sweeps and sweeps["slow_step"].kernel == b"slow_recompute_bulk_kernel":
        relabel["slow_step"] = "slow_step_recompute"                             # theta-tilde redone from theta^t, g0, g1
    elif "slow_step" in sweeps and sweeps["slow_step"].bytes_read_per_param - sweeps["slow_step"].extra_launches * 2 * G == 12 + 3 * G:
        relabel["slow_step"] = "slow_step_replay"                                # g0 and g1 read once more
    lag = bool(relabel)
    for old, new in relabel.items():
        calls[new] = calls[old]
        sweeps[new] = sweeps[old]
    names = [relabel.get(nm, nm) for nm in names]
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(n_ev)] for _ in range(args.steps)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(str(getattr(props, "uuid", "")))
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = ctx.launch_count()
    torch.cuda.synchronize()
    t_wall0 = time.time()
    e0.record(stream)
    res = None
    for s in range(args.steps):
        res = one_step(evs[s])
    e1.record(stream)
    torch.cuda.synchronize()
    t_wall1 = time.time()
    if world > 1:
        dist.barrier()
    launches = ctx.launch_count() - launches0
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    ms_total = e0.elapsed_time(e1)
    if world > 1:
        t = torch.tensor([ms_total], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms_total = float(t.item())
    ms_step = ms_total / args.steps

    # per-kernel durations from the events inside the timed region
    per = {nm: statistics.mean(evs[s][i].elapsed_time(evs[s][i + 1]) for s in range(args.steps))
           for i, nm in enumerate(names)}
    peak, peak_kind = measured_peak_gbs()
    # algorithmic bytes per parameter and kernel function of every call, as the library reports them
    alg_bytes = {nm: sweeps[nm].bytes_read_per_param + sweeps[nm].bytes_written_per_param for nm in names}
    kernel_of = {nm: sweeps[nm].kernel.decode() for nm in names}
    kernels = {nm: {"kernel": kernel_of[nm], "ms": ms, "bytes_per_param": alg_bytes[nm],
                    "gbs": alg_bytes[nm] * d / (ms * 1e-3) / 1e9} for nm, ms in per.items()}
    # dominant kernel = the kernel function with the largest share of the step; its figures
    # are averages over its launches in one step (algorithmic bytes and duration alike)
    by_fn = {}
    for nm, ms in per.items():
        by_fn.setdefault(kernel_of[nm], []).append(nm)
    dom_fn = max(by_fn, key=lambda f: sum(per[nm] for nm in by_fn[f]))
    dom = by_fn[dom_fn]
    dom_bytes = statistics.mean(alg_bytes[nm] for nm in dom) * d
    dom_ms = statistics.mean(per[nm] for nm in dom)
    achieved = dom_bytes / (dom_ms * 1e-3) / 1e9
    tpp = recorded_traffic_per_param(dom_fn, dom)
    roofline = {"bound": "hbm", "kernel": dom_fn, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": f"of {peak_kind}",
                "traffic": (tpp * d if tpp else None),
                "algorithmic_bytes_per_launch": dom_bytes, "ms_per_launch": dom_ms,
                "launches_averaged": dom, "share_of_step": sum(per[nm] for nm in dom) / sum(per.values())}
    step_bytes = sum(alg_bytes[nm] for nm in names) * d
    whole_gbs = step_bytes / (ms_step * 1e-3) / 1e9

    total_params = d * world
    line = {
        "metric": METRIC, "value": total_params / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": desc, "params_per_gpu": d, "tensors": len(shapes), "optimizer": "AdamW",
                   "K": args.K, "alpha": args.alpha, "lr": args.lr, "grad_dtype": "bf16",
                   "placement": ["pingpong", "snapshot"][args.placement],
                   "step": "fallback (single pass)" if args.fallback else
                   {"deferred": ("active (probe with deferred state writing bfloat16 theta1 only, probe+extrapolate in one sweep "
                                 "writing bfloat16 theta-tilde only, slow step recomputing theta-tilde, gate)") if only16 else
                                ("active (probe with deferred state, probe+extrapolate in one sweep with m, v still unwritten, "
                                 "slow step replaying both moment updates, gate)") if lag else
                                "active (probe with deferred state, probe+extrapolate in one sweep, slow step, gate)",
                    "fused": "active (probe, probe+extrapolate in one sweep, slow step, gate)",
                    "unfused": "active (probe, probe, extrapolate, slow step, gate)"}[flow],
                   "bf16_model_weight_copies": (("theta1 and theta-tilde as bfloat16 only (theta-tilde recomputed by the slow step)"
                                                 if only16 else "theta1 as bfloat16 only") if emit else False),
                   "diagnostics": diag, "gradients_persist": persist,
                   "clip_grad_norm": clip if clip > 0.0 else None, "g_slow_aliases_g0": alias,
                   "work_buffer": not only16, "resident_bytes_per_param": 12 + (0 if only16 else 4) + (4 if alias else 6) + (2 if emit else 0), "l2": "inputs larger than L2 (no flush needed)",
                   "parallelism": f"dp{world} (independent shards, one 8-byte all-reduce per step)" if world > 1 else "1 GPU"},
        "hbm_gbs_whole_step": whole_gbs, "hbm_frac_whole_step": whole_gbs / peak,
        "hbm_frac_of_8tbs_nominal": whole_gbs / 8000.0,
        "bytes_per_param_per_step": step_bytes / d,
        "kernels": kernels, "roofline": roofline, "clocks": clocks, "gpu_launches": launches,
        "gate": None if res is None else {"norm": res.norm, "t": res.t, "active": res.active},
    }

    if not args.no_e2e:
        # every rank streams its own slice through its own link; the job's figure is all
        # slices over the slowest rank's time
        e2e = run_e2e(torch, b, args, cfg, opt)
        if world > 1:
            t = torch.tensor([e2e["ms_per_step"]], dtype=torch.float64, device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e2e["ms_per_step"] = float(t.item())
            e2e["value"] = args.e2e_params * world / (e2e["ms_per_step"] * 1e-3)
            e2e["h2d_bytes_per_step"] *= world
            e2e["d2h_bytes_per_step"] *= world
            e2e["sample"] += f"; one such slice per rank, {world} ranks, max over ranks"
        line["e2e"] = e2e
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        n = args.cpu_params
        done, dt = time_oracle_steps(n, args.K, args.alpha, args.lr, 2, 1, min_seconds=10.0)
        line["cpu_baseline"] = {
            "value": n * done / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{done} oracle active steps on a {n}-parameter slice drawn with the workload's recipe "
                      f"({dt:.1f} s on one of {os.cpu_count()} host cores)"}
    ctx.close()
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_e2e(torch, b, args, cfg, opt):
    """The same step through gxpo_step_host: parameters, optimizer state and the
    three gradients start in pinned HOST memory; results are copied back."""
    n = args.e2e_params
    from paper_2605_06755_b200 import workloads as w
    import numpy as np
    th, m, v, g0, g1, gs = w.llm_inputs_numpy(n, 4321, "bf16")
    pin = [torch.from_numpy(x.view(np.int16) if x.dtype == np.uint16 else x).pin_memory()
           for x in (th, m, v, g0, g1, gs)]
    ctx = b.Context(cfg, opt, b.BF16)
    ctx.tune(args.ctas, args.variant, args.unit_tiles)
    t = [b.tensor_ptrs(pin[0], None, pin[1], pin[2], pin[3], pin[4], pin[5])]
    l0 = None
    for i in range(2 + 3):
        if i == 2:
            torch.cuda.synchronize()
            l0 = ctx.launch_count()
            t0 = time.perf_counter()
        ctx.step_host(t, staging_elems=args.e2e_staging, allow_nonfinite=True)
    torch.cuda.synchronize()
    dt = (time.perf_counter() - t0) / 3
    launches = (ctx.launch_count() - l0) // 3
    ctx.close()
    return {"value": n / dt, "unit": UNIT, "h2d_bytes_per_step": 18 * n, "d2h_bytes_per_step": 12 * n + 64,
            "ms_per_step": dt * 1e3, "gpu_launches_per_step": launches,
            "sample": f"{n}-parameter flat slice; theta, m, v, g0, g1, g_slow in pinned host memory, "
                      f"streamed through gxpo_step_host in {args.e2e_staging}-parameter pieces"}


def run_surrogate(args):
    """The diagonal-quadratic surrogate at n = 1e8 (plain GD, eta = 0.1, gradients computed
    in-kernel): `--steps` consecutive active steps, once through the fused harness kernel
    (16 B/param) and once through the library calls with the harness gradient kernel standing
    in for the backward passes (3 x 16 + 12 + 12 + 20 + 12 = 104 B/param, fp32 gradients)."""
    import torch

    from paper_2605_06755_b200 import build
    build.build_library()
    from paper_2605_06755_b200 import binding as b
    from paper_2605_06755_b200 import workloads as w
    torch.cuda.set_device(0)
    n, eta = 100_000_000, 0.1
    a_np, b_np, t0_np = w.quadratic_surrogate(n, 0)
    a, bb, t0 = (torch.from_numpy(x).cuda() for x in (a_np, b_np, t0_np))
    peak, peak_kind = measured_peak_gbs()
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # fused harness kernel
    theta = t0.clone()
    scratch = torch.zeros(b.quad_scratch_bytes(), dtype=torch.uint8, device="cuda")
    sumsq = torch.zeros(1, dtype=torch.float64, device="cuda")
    def fused_step():
        b.quad_active_step(theta.data_ptr(), a.data_ptr(), bb.data_ptr(), n, eta, args.K, 1.0, 1e-8, 0.0,
                           sumsq.data_ptr(), scratch.data_ptr(), stream)
    for _ in range(max(args.warmup, 3)):
        fused_step()
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(args.steps):
        fused_step()
    e1.record(stream)
    torch.cuda.synchronize()
    ms_fused = e0.elapsed_time(e1) / args.steps
    # the library calls
    theta2, work = t0.clone(), torch.empty_like(t0)
    g0, g1, gs = (torch.empty_like(t0) for _ in range(3))
    cfg, opt = b.make_cfg(kind=b.OPT_GD, lr=eta, K=args.K, alpha=1.0, delta=1e-8)
    ctx = b.Context(cfg, opt, b.F32)
    ctx.bind([b.tensor_ptrs(theta2, work, None, None, g0, g1, gs)])
    def api_step():
        b.quad_grad(theta2.data_ptr(), a.data_ptr(), bb.data_ptr(), g0.data_ptr(), n, stream)
        ctx.probe_step(0, stream)
        b.quad_grad(work.data_ptr(), a.data_ptr(), bb.data_ptr(), g1.data_ptr(), n, stream)
        ctx.probe_step(1, stream)
        ctx.extrapolate(stream)
        b.quad_grad(theta2.data_ptr(), a.data_ptr(), bb.data_ptr(), gs.data_ptr(), n, stream)
        ctx.slow_step(stream)
        return ctx.gate_update(stream)
    for _ in range(max(args.warmup, 3)):
        api_step()
    torch.cuda.synchronize()
    l0 = ctx.launch_count()
    e0.record(stream)
    for _ in range(args.steps):
        res = api_step()
    e1.record(stream)
    torch.cuda.synchronize()
    ms_api = e0.elapsed_time(e1) / args.steps
    launches = ctx.launch_count() - l0 + 3 * args.steps
    gbs = 16 * n / (ms_fused * 1e-3) / 1e9
    line = {"metric": METRIC, "value": n / (ms_fused * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_fused, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "diagonal-quadratic surrogate, n = 1e8, plain GD eta = 0.1, gradients in-kernel",
                       "K": args.K, "alpha": 1.0, "step": "fused harness kernel (16 B/param)",
                       "l2": "inputs larger than L2 (no flush needed)"},
            "roofline": {"bound": "hbm", "kernel": "quad_active_kernel", "achieved": gbs, "peak": peak, "unit": "GB/s",
                         "frac": gbs / peak, "peak_kind": f"of {peak_kind}", "traffic": None,
                         "algorithmic_bytes_per_launch": 16 * n},
            "library_calls": {"ms_per_step": ms_api, "bytes_per_param": 104,
                              "gbs": 104 * n / (ms_api * 1e-3) / 1e9, "gate_norm": res.norm},
            "gpu_launches": launches + args.steps}
    ctx.close()
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------
# several GPUs: one process per GPU
# ----------------------------------------------------------------------------
def rank_environment(rank, world, port, base=None):
    """Environment of one rank: what torch.distributed.run would set for a single node."""
    env = dict(os.environ if base is None else base)
    env.update({"RANK": str(rank), "LOCAL_RANK": str(rank), "WORLD_SIZE": str(world),
                "LOCAL_WORLD_SIZE": str(world), "MASTER_ADDR": "127.0.0.1", "MASTER_PORT": str(port)})
    return env


def free_port():
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(world, cmd, poll_s=0.2):
    """Start `cmd` once per rank (ranks 0..world-1, LOCAL_RANK = RANK, one node, rendezvous on
    127.0.0.1) and wait for all of them.  Every rank inherits stdout and stderr, so rank 0's one
    JSON line and the communication library's own log reach the caller untouched.  When a rank
    fails the others are terminated (exactly the processes started here).  Returns the list of
    exit codes."""
    port = free_port()
    procs = [subprocess.Popen(cmd, env=rank_environment(r, world, port)) for r in range(world)]
    codes = [None] * world
    failed = False
    while any(c is None for c in codes):
        for r, p in enumerate(procs):
            if codes[r] is None:
                codes[r] = p.poll()
                if codes[r] not in (None, 0):
                    failed = True
        if failed:
            for r, p in enumerate(procs):
                if codes[r] is None:
                    p.terminate()
            for r, p in enumerate(procs):
                if codes[r] is None:
                    try:
                        codes[r] = p.wait(timeout=30)
                    except subprocess.TimeoutExpired:
                        p.kill()
                        codes[r] = p.wait()
            break
        time.sleep(poll_s)
    return codes


def main():
    args = parse_args()
    if args.gpus < 1:
        raise SystemExit("--gpus must be >= 1")
    if args.impl == "reference":
        run_reference(args)
        return
    launched = "WORLD_SIZE" in os.environ
    if launched and int(os.environ["WORLD_SIZE"]) != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} contradicts WORLD_SIZE={os.environ['WORLD_SIZE']} of the launcher")
    if args.gpus > 1 and args.workload == "surrogate_1e8":
        raise SystemExit("the surrogate workload is a one-GPU harness")
    if args.gpus > 1 and not launched:
        # no launcher around us: be the launcher
        import torch
        have = torch.cuda.device_count()
        if have < args.gpus:
            raise SystemExit(f"--gpus {args.gpus} but only {have} CUDA device(s) are visible")
        codes = spawn_ranks(args.gpus, [sys.executable, os.path.abspath(__file__)] + sys.argv[1:])
        bad = [(r, c) for r, c in enumerate(codes) if c != 0]
        if bad:
            raise SystemExit(f"rank(s) failed (rank, exit code): {bad}")
        return
    if args.workload == "surrogate_1e8":
        run_surrogate(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
