#!/usr/bin/env python
"""Benchmark of the D3 decode hot path on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--alpha A] [--impl d3|reference]

One "step" is one decode step of the whole hot path (schedule, every retained
block, KV fill, final norm + LM head) for the batch.  The workload is the
Llama-2-7B-shaped decoder (random-init bf16, seeded), batch 1, prompt 512
uniform-random token ids, generate 256; the K timed steps take their generation
indices i evenly over 1..255 (K = 255, the default, is the run itself).  The
timed region of K steps is repeated (--reps, default 5); the median repetition
is the reported value, the best one rides along.

Prints ONE JSON line: decode tokens/s (device-timed, inputs resident in HBM),
the HBM roofline of the dominant kernel and of the whole step, the same metric
end to end through the C ABI with host buffers, the alpha = 1 run of the same
kernels, time to first token of the prompt, the batched workloads C3 / C4, and
the CPU oracle timed on the host cores as a baseline.
`--impl reference` times the CPU oracle alone on a bounded sample.
`--gpus N` without a torchrun environment starts the N replica processes itself.
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

import numpy as np
import torch

from paper_2503_08524_b200 import inputs as I

PROMPT, GENERATE, BATCH = 512, 256, 1
START_FRACTION = 0.2          # the paper's GSM8K value of `start`
METRIC = "decode tokens/s at 1 B200 and % of HBM roofline (retained-layer bytes/step)"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
ORACLE_PROMPT = 32            # bounded sample for the CPU oracle
# dram__bytes_read + dram__bytes_write of one k_step_b1 launch over its algorithmic bytes, from the
# ncu capture summarised in profiles/fused_step_k_step_b1_7bshape_L4.md (4-block case of the same
# kernel: 1.8960 GB moved for 1.881 GB algorithmic; traffic grows with the blocks executed, so the
# full launch is scaled by its own algorithmic bytes).  Set to None when the kernel changes.
FUSED_TRAFFIC_RATIO = 1.0080


def gen_indices(k: int):
    """Generation index of each of k steps, spread evenly over the run 1..GENERATE-1."""
    n = GENERATE - 1
    if k >= n:
        return [1 + (j % n) for j in range(k)]
    return [1 + (j * n) // k for j in range(k)]


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int, period_ms: int = 50):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        sel = str(device_index)
        try:
            sel = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid)
        except Exception:
            pass
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", sel, "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", str(period_ms)],
                stdout=self.tmp, stderr=subprocess.DEVNULL)
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
        self.tmp.flush()
        self.tmp.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.tmp.read().splitlines():
            p = [v.strip() for v in line.split(",")]
            if len(p) < 7:
                continue
            try:
                sm.append(float(p[0]))
                mx.append(float(p[1]))
            except ValueError:
                continue
            for n, v in zip(names, p[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        self.tmp.close()
        os.unlink(self.tmp.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons),
                       samples=len(sm))
        return out


ORACLE_STEPS, ORACLE_PASSES = 40, 2


def oracle_steps(k):
    """Timed oracle steps per pass for a run of k GPU steps (the same rule in both arms)."""
    return max(8, min(int(k), ORACLE_STEPS))


def time_oracle(shape, w_cpu, alpha, start_id, steps):
    """CPU oracle on a bounded sample, the same in both arms: ORACLE_PROMPT-token prefill
    (untimed), one warm-up step, then ORACLE_PASSES passes of ORACLE_STEPS timed decode steps
    with generation indices spread over the run like the GPU's.  The host is shared with other
    jobs, so a pass can be disturbed: the fastest pass is the value, every pass is reported.
    Returns (tokens/s of the best pass, [seconds per pass], threads used)."""
    import oracle as O
    orc = O.Oracle(shape, w_cpu, 1, ORACLE_PROMPT + ORACLE_PASSES * steps + 4, start_id=start_id)
    prompt = I.prompt_tokens(shape, I.BASE_SEED, 0, ORACLE_PROMPT).numpy()
    orc.prefill(0, prompt)
    toks = I.token_ids(I.BASE_SEED, 999, steps + 1, shape.vocab).numpy()
    gi = gen_indices(steps)
    orc.decode_step([0], [int(toks[steps])], [gi[0]], alpha)
    passes = []
    for _ in range(ORACLE_PASSES):
        t0 = time.perf_counter()
        for j in range(steps):
            orc.decode_step([0], [int(toks[j])], [gi[j]], alpha)
        passes.append(time.perf_counter() - t0)
    orc.close()
    return steps * BATCH / min(passes), passes, O.threads()


def host_mem_available_gb():
    try:
        for line in open("/proc/meminfo"):
            if line.startswith("MemAvailable"):
                return int(line.split()[1]) / 1e6
    except Exception:
        pass
    return 0.0


def oracle_shape_and_scale(shape):
    """The full 32-block model if host RAM holds its bf16 weights, else 8 blocks
    (the result is then scaled by the block count and says so)."""
    need_gb = (shape.n_layers * shape.layer_weight_bytes + 2 * shape.head_weight_bytes) / 1e9
    if host_mem_available_gb() > need_gb + 16:
        return shape, 1.0, f"{shape.n_layers} blocks"
    small = shape.with_layers(8)
    return small, 8.0 / shape.n_layers, "8 of 32 blocks, tokens/s scaled by 8/32"


def oracle_baseline(w, shape, alpha, start_id, steps):
    """cpu_baseline object of either arm (w: weights on any device)."""
    oshape, scale, note = oracle_shape_and_scale(shape)
    w_cpu = I.weights_to({k: (v[:oshape.n_layers] if isinstance(v, list) else v) for k, v in w.items()}, "cpu")
    tps, passes, cores = time_oracle(oshape, w_cpu, alpha, min(start_id, oshape.n_layers), steps)
    return {"value": tps * scale, "unit": "tokens/s", "cores": cores, "kind": "oracle",
            "omp_threads": cores, "host_cpus": os.cpu_count(),
            "pass_seconds": [round(p, 2) for p in passes],
            "sample": f"fp64 C oracle, 7B shape, {note}, prompt {ORACLE_PROMPT}, best of {ORACLE_PASSES} passes of "
                      f"{steps} decode steps at alpha={alpha} ({sum(passes):.1f} s of CPU work in all)"}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    shape = I.LLAMA_7B
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    w = I.make_weights(shape, I.BASE_SEED, device=dev)
    start_id = int(START_FRACTION * shape.n_layers)
    steps = oracle_steps(args.steps)
    cb = oracle_baseline(w, shape, args.alpha, start_id, steps)
    tps = cb["value"]
    line = {
        "impl": "reference", "metric": METRIC, "value": tps, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": steps, "warmup": 1,
        "ms_per_step": 1e3 / tps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "llama2-7b-shape batch 1, prompt 512, generate 256 (oracle: bounded sample)",
                   "alpha": args.alpha, "start_id": start_id},
        "cpu_baseline": cb,
        "e2e": {"value": tps, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)
    return 0


def spawn_replicas(args):
    """`--gpus N` outside a torchrun environment: start the N replica processes (one per GPU)
    with the standard launcher and pass the flags through; rank 0 prints the line."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def median(v):
    return statistics.median(v)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=GENERATE - 1)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--alpha", type=float, default=0.995)
    ap.add_argument("--reps", type=int, default=5, help="repetitions of the K-step timed region (>= 5)")
    ap.add_argument("--impl", default="d3", choices=["d3", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--workloads", default="c3,c4",
                    help="batched workloads reported beside the main line (c3,c4,c5 or none); "
                         "c5 holds ~140 GB of weights and is off by default")
    ap.add_argument("--layers", type=int, default=0,
                    help="profiling aid: keep only this many blocks (same kernel shapes, less memory); "
                         "numbers from such a run are not benchmark values")
    ap.add_argument("--prompt", type=int, default=PROMPT, help="profiling aid: shorter prompt")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    args.reps = max(args.reps, 1)
    if args.impl == "reference":
        return run_reference(args)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        return spawn_replicas(args)

    from paper_2503_08524_b200 import binding as B   # raises if libd3 is missing

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback)")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev))

    from paper_2503_08524_b200.replicas import Replicas
    reps = Replicas(dist, dev)
    barrier = reps.barrier
    max_over_ranks = reps.max_ms
    profiling_aid = args.layers > 0 or args.prompt != PROMPT

    shape = I.LLAMA_7B if args.layers <= 0 else I.LLAMA_7B.with_layers(args.layers)
    start_id = int(START_FRACTION * shape.n_layers)
    K, W = args.steps, args.warmup
    max_seq = args.prompt + K + W + 8
    w = I.make_weights(shape, I.BASE_SEED, device=dev)
    model = B.D3Model(shape, w, 1, max_seq, 128, start_id=start_id, device=dev)
    model.zero_kv()
    prompt = I.prompt_tokens(shape, I.BASE_SEED, 0, args.prompt).numpy()
    toks = I.token_ids(I.BASE_SEED, 999, K + W, shape.vocab).numpy()
    gi = gen_indices(K)
    logits = torch.empty((BATCH, shape.vocab), dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()

    def timed_run(alpha, profile=False):
        """Prefill, W warm-up steps, K timed steps.  Returns (ms, stats totals, profile, prefill ms)."""
        model.d3_reset_slot(0)
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        p0.record(stream)
        model.d3_prefill(0, prompt, logits=logits[0])
        p1.record(stream)
        for j in range(W):
            model.d3_decode_step([0], [int(toks[j])], [gi[0]], alpha, logits=logits)
        model.d3_profile(profile)
        if profile:
            model.d3_read_profile()
        tot = {"bytes": 0, "rows_layers": 0, "launches": 0, "touched": 0}
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for j in range(K):
            _, st = model.d3_decode_step([0], [int(toks[W + j])], [gi[j]], alpha, logits=logits,
                                         want_stats=True)
            tot["bytes"] += st["algorithmic_bytes"]
            tot["rows_layers"] += st["rows_layers"]
            tot["launches"] += st["kernel_launches"]
            tot["touched"] += st["layers_touched"]
        e1.record(stream)
        barrier()
        ms = e0.elapsed_time(e1)
        prof = model.d3_read_profile() if profile else None
        model.d3_profile(False)
        return ms, tot, prof, p0.elapsed_time(p1)

    def repeated(alpha, n):
        """n repetitions of the K-step region; per repetition the slowest rank's time."""
        ms_list, ttft, tot = [], [], None
        for _ in range(n):
            ms, tot, _, pf = timed_run(alpha)
            ms_list.append(max_over_ranks(ms))
            ttft.append(pf)
        return ms_list, tot, ttft

    # ---- main timed region: args.reps repetitions, clock samples taken across all of them
    sampler = ClockSampler(local) if rank == 0 else None
    ms_reps, tot, ttft_ms = repeated(args.alpha, args.reps)
    clocks = sampler.stop() if sampler else None
    ms = median(ms_reps)
    value = world * BATCH * K / (ms / 1e3)

    # ---- the same kernels at alpha = 1 (full depth) and 0.999
    others = {}
    for a in (1.0, 0.999):
        if abs(a - args.alpha) < 1e-12:
            continue
        ms_a, tot_a, _ = repeated(a, 3 if args.reps >= 3 else args.reps)
        others[a] = (median(ms_a), min(ms_a), tot_a)

    # ---- per-kernel-class device times of the same K steps (events around each launch)
    _, _, prof, _ = timed_run(args.alpha, profile=True)

    # ---- end to end through the C ABI, every step: host token in (pinned), the call's result out
    # (the [vocab] fp32 logits, 128 KB, to pinned host memory) plus the greedy token chosen on the
    # device, which is the next step's input.  Second variant: only the 4-byte token comes back.
    tok_dev = torch.empty(BATCH, dtype=torch.int32, device=dev)
    tok_host = torch.empty(BATCH, dtype=torch.int32).pin_memory()
    logits_host = torch.empty((BATCH, shape.vocab), dtype=torch.float32).pin_memory()

    def e2e_run(copy_logits):
        model.d3_reset_slot(0)
        model.d3_prefill(0, prompt)
        cur = int(toks[0])
        for j in range(W):
            model.d3_decode_step([0], [cur], [gi[0]], args.alpha, logits=logits)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for j in range(K):
            model.d3_decode_one(0, cur, gi[j], args.alpha, logits)                  # host arrays -> device
            model.d3_argmax(logits, tok_dev)
            if copy_logits:
                logits_host.copy_(logits, non_blocking=True)                        # device -> host
            tok_host.copy_(tok_dev, non_blocking=True)
            stream.synchronize()
            cur = int(tok_host[0])
        e1.record(stream)
        barrier()
        return max_over_ranks(e0.elapsed_time(e1))

    e2e_ms = median([e2e_run(True) for _ in range(3)])
    e2e_tok_ms = median([e2e_run(False) for _ in range(3)])
    e2e_value = world * BATCH * K / (e2e_ms / 1e3)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return 0

    peak, peak_kind = measured_peak()
    # dominant kernel class and its algorithmic bytes per launch
    d, f = shape.d_model, shape.d_ffn
    nq = shape.n_q_heads * shape.head_dim
    class_bytes = {
        "norm+qkv": 2 * shape.qkv_rows * d + 2 * d + 4 * d + 4 * shape.qkv_rows,
        "o_proj+resid": 2 * d * nq + 4 * nq + 8 * d,
        "norm+gate_up+swiglu": 2 * 2 * f * d + 2 * d + 4 * d + 4 * f,
        "down+resid": 2 * d * f + 4 * f + 8 * d,
        "norm+lm_head": 2 * shape.vocab * d + 2 * d + 4 * d + 4 * shape.vocab,
    }
    kernels = {k: v for k, v in prof.items() if not k.startswith("fused:")}
    top = max(kernels.items(), key=lambda kv: kv[1]["ms"])
    top_name, top_ms, top_n = top[0], top[1]["ms"], top[1]["launches"]
    prof_total = sum(v["ms"] for v in kernels.values())
    # the single-kernel step moves the whole step's algorithmic bytes per launch
    class_bytes["fused_step"] = tot["bytes"] / K
    roofline = {"bound": "hbm", "kernel": top_name, "unit": "GB/s", "peak": peak,
                "peak_kind": f"of {peak_kind} (STREAM-style copy)", "traffic": None,
                "share_of_kernel_time": top_ms / prof_total, "launches": top_n}
    if top_name in class_bytes:
        launch_ms = top_ms / top_n
        timed = "per-launch CUDA events of the profiled pass (a synchronize after every step)"
        if top_name == "fused_step" and tot["launches"] == K:
            # one launch per step: the timed region itself (median repetition, events around its K
            # launches back to back, the 1 KiB counter memsets included) is the launch duration
            launch_ms = ms / K
            timed = "CUDA events around the K launches of the timed region (median repetition)"
        ach = class_bytes[top_name] * BATCH / 1e9 / (launch_ms / 1e3)
        roofline.update(achieved=ach, frac=ach / peak, frac_of_nominal_8TBs=ach / NOMINAL_HBM_GBS,
                        bytes_per_launch=class_bytes[top_name], avg_launch_us=1e3 * launch_ms,
                        avg_launch_us_profiled_pass=1e3 * top_ms / top_n, timed=timed)
        if top_name == "fused_step" and FUSED_TRAFFIC_RATIO is not None:
            roofline["traffic"] = FUSED_TRAFFIC_RATIO * class_bytes[top_name]
    else:
        roofline.update(achieved=None, frac=None)
    step_gbs = tot["bytes"] / 1e9 / (ms / 1e3)
    best_gbs = tot["bytes"] / 1e9 / (min(ms_reps) / 1e3)
    step_roofline = {"bytes_per_step": tot["bytes"] / K, "achieved": step_gbs, "unit": "GB/s",
                     "frac_of_measured": step_gbs / peak, "frac_of_nominal_8TBs": step_gbs / NOMINAL_HBM_GBS,
                     "best_rep_frac_of_measured": best_gbs / peak,
                     "avg_layers_per_token": tot["rows_layers"] / K}
    alphas = {str(args.alpha): {"tokens_per_s": value, "ms_per_step": ms / K,
                                "avg_layers": tot["rows_layers"] / K,
                                "frac_of_measured": step_gbs / peak,
                                "frac_of_nominal_8TBs": step_gbs / NOMINAL_HBM_GBS}}
    for a, (ms_a, best_a, tot_a) in others.items():
        g = tot_a["bytes"] / 1e9 / (ms_a / 1e3)
        alphas[str(a)] = {"tokens_per_s": world * BATCH * K / (ms_a / 1e3), "ms_per_step": ms_a / K,
                          "ms_per_step_best": best_a / K,
                          "avg_layers": tot_a["rows_layers"] / K, "frac_of_measured": g / peak,
                          "frac_of_nominal_8TBs": g / NOMINAL_HBM_GBS}
    if 1.0 in others:
        full = alphas["1.0"]
        alphas["speedup_vs_alpha_1"] = value / full["tokens_per_s"]
        alphas["layer_ratio_vs_alpha_1"] = full["avg_layers"] / (tot["rows_layers"] / K)
        alphas["bytes_ratio_vs_alpha_1"] = others[1.0][2]["bytes"] / tot["bytes"]

    # ---- time to first token: the prompt through all blocks (d3_prefill), device-timed
    pf = median(ttft_ms)
    flops = 2.0 * args.prompt * shape.n_layers * (shape.layer_weight_bytes / 2) + 2.0 * shape.vocab * shape.d_model
    ttft = {"prompt_tokens": args.prompt, "ms": pf, "ms_best": min(ttft_ms),
            "prompt_tokens_per_s": args.prompt / (pf / 1e3), "projection_tflops": flops / 1e12 / (pf / 1e3)}

    # ---- batched workloads (mixed depths, tensor-core projections), each with its own clock record
    model.close()
    del model, w
    torch.cuda.empty_cache()
    workloads = {}
    wl_launches = 0
    if world == 1 and not profiling_aid:
        from paper_2503_08524_b200 import workloads as WL
        for name in [n for n in args.workloads.split(",") if n in WL.WORKLOADS]:
            box = {}

            def on_timed(start, box=box):
                if start:
                    box["s"] = ClockSampler(local)
                else:
                    box["clocks"] = box.pop("s").stop()
            try:
                r = WL.run_workload(name, steps=24 if name != "c5" else 12, reps=3, device=dev, on_timed=on_timed)
            except Exception as exc:     # the main line must still be printed
                if "s" in box:
                    box.pop("s").stop()
                workloads[name] = {"workload": name, "error": f"{type(exc).__name__}: {exc}"[:300]}
                torch.cuda.empty_cache()
                continue
            r["clocks"] = box.get("clocks")
            r.pop("kernel_classes", None)
            workloads[name] = r
            wl_launches += int(r["launches_per_step"] * r["steps"] * r["reps"])

    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        try:
            w = I.make_weights(shape, I.BASE_SEED, device=dev)
            cpu_baseline = oracle_baseline(w, shape, args.alpha, start_id, oracle_steps(K))
            del w
        except Exception as exc:         # the main line must still be printed
            cpu_baseline = {"value": None, "unit": "tokens/s", "cores": None, "kind": "oracle",
                            "sample": f"failed: {type(exc).__name__}: {exc}"[:300]}

    line = {
        "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": K,
        "warmup": W, "ms_per_step": ms / K, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 weights+KV, f32 activations/accumulate", "data": "synthetic",
        "config": {"workload": f"llama2-7b-shape (L={shape.n_layers},d=4096,32x128,ffn 11008,V=32000), "
                               f"batch 1, prompt {args.prompt}, generate 256", "alpha": args.alpha, "start_id": start_id,
                   "anchor": "start", "kv_fill": "copy", "gen_index_schedule": "1 + floor(j*255/K)",
                   "l2": "inputs_exceed_l2 (weights of one step >> 126 MB)",
                   "multi_gpu": "independent replicas"},
        "repetitions": {"n": len(ms_reps), "reported": "median", "ms_per_step_median": ms / K,
                        "ms_per_step_best": min(ms_reps) / K, "ms_per_step_all": [m / K for m in ms_reps]},
        "roofline": roofline, "step_roofline": step_roofline, "alphas": alphas,
        "kernel_classes": prof, "ttft": ttft, "workloads": workloads, "cpu_baseline": cpu_baseline,
        "e2e": {"value": e2e_value, "unit": "tokens/s", "ms_per_step": e2e_ms / K,
                "h2d_bytes_per_step": 12 * BATCH, "d2h_bytes_per_step": (4 * shape.vocab + 4) * BATCH,
                "result": "fp32 logits [vocab] to pinned host memory + the greedy token",
                "token_only": {"value": world * BATCH * K / (e2e_tok_ms / 1e3), "ms_per_step": e2e_tok_ms / K,
                               "d2h_bytes_per_step": 4 * BATCH}},
        "gpu_launches": tot["launches"], "clocks": clocks,
    }
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
