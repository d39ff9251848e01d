"""Batched decode workloads (several sequences per step, mixed depths).

  python -m paper_2503_08524_b200.workloads c3|c4|c5 [--layers N] [--steps K] [--alpha A]
                                                     [--exec auto|kernels|tensor|fused] [--rows R] [--profile]

The workloads follow the batched configurations the paper's runs suggest
(static batches of a few sequences, prompts of a few hundred to ~1k tokens,
Sec. 4.1 and its efficiency discussion in Sec. 4.2):

  c3  Llama-2-7B shape, 32 rows, prompt lengths uniform in [128, 1024], row b at
      generation index 1 + (8 b mod 256) + step: one step mixes many depths
  c4  Llama-2-13B shape, 8 rows, prompt 1024, all rows at the same index
  c5  Llama-2-70B shape (GQA 64/8), 4 rows, prompt 512, all rows at the same index

Weights are random-init bf16 from the seeded generator, token ids uniform over
the vocabulary.  Prints one JSON line: ms/step, tokens/s, the step's algorithmic
bytes over time against the measured HBM copy rate, and (with --profile) the
device time of every kernel class.  `--layers` keeps only N blocks (same kernel
shapes, less memory) for profiler captures; its numbers are not whole-model ones.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import torch

from . import inputs as I

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKLOADS = {
    #        shape        rows  prompt lo/hi  stagger  alpha   steps
    "c3": (I.LLAMA_7B, 32, 128, 1024, 8, 0.997, 64),
    "c4": (I.LLAMA_13B, 8, 1024, 1024, 0, 0.998, 64),
    "c5": (I.LLAMA_70B, 4, 512, 512, 0, 0.998, 32),
}
EXEC = {"auto": 0, "kernels": 1, "tensor": 2, "fused": 3}


def measured_hbm_gbs():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


def run_workload(name, layers=0, steps=0, warmup=3, alpha=0.0, gen_offset=0, exec_mode="auto", rows=0,
                 profile=False, reps=1, device="cuda:0", on_timed=None):
    """Run one workload and return its result line (a dict).  `reps` repeats the timed region
    of K steps (the sequences simply go on) and reports the median and the best repetition;
    `on_timed(True/False)` brackets the timed part (a clock sampler hooks in there)."""
    from . import binding as B   # raises if libd3 is missing
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device (no CPU fallback)")
    base, wrows, plo, phi, stagger, walpha, wsteps = WORKLOADS[name]
    rows = rows if rows > 0 else wrows
    shape = base.with_layers(layers) if layers > 0 else base
    alpha = alpha if alpha > 0 else walpha
    K, W = (steps if steps > 0 else wsteps), max(warmup, 3)
    reps = max(1, reps)
    seed = I.BASE_SEED + int(name[1])
    start_id = int(0.2 * shape.n_layers)
    w = I.make_weights(shape, seed, device=device)
    extra = 2 * (K * reps + W) + 16
    model = B.D3Model(shape, w, rows, phi + extra, 128, start_id=start_id, device=device)
    model.zero_kv()
    lens = I.uniform_ints(seed, 3, rows, plo, phi)
    stream = torch.cuda.current_stream()
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    p0.record(stream)
    for b in range(rows):
        model.d3_prefill(b, I.prompt_tokens(shape, seed, b, lens[b]).numpy())
    p1.record(stream)
    model.d3_set_exec(EXEC[exec_mode])
    slots = list(range(rows))
    gi0 = [1 + gen_offset + (stagger * b) % 256 for b in range(rows)]
    logits = torch.empty((rows, shape.vocab), dtype=torch.float32, device=device)
    counter = [0]

    def step(want_stats=False):
        s = counter[0]
        counter[0] += 1
        toks = I.token_ids(seed, 100 + s, rows, shape.vocab).numpy()
        return model.d3_decode_step(slots, toks, [g + s for g in gi0], alpha, logits=logits,
                                    want_stats=want_stats)

    for _ in range(W):
        step()
    torch.cuda.synchronize()
    prefill_ms = p0.elapsed_time(p1)
    if on_timed:
        on_timed(True)
    rep_ms, tot = [], {"bytes": 0, "rows_layers": 0, "launches": 0, "touched": 0}
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(K):
            _, st = step(True)
            tot["bytes"] += st["algorithmic_bytes"]
            tot["rows_layers"] += st["rows_layers"]
            tot["launches"] += st["kernel_launches"]
            tot["touched"] += st["layers_touched"]
        e1.record(stream)
        torch.cuda.synchronize()
        rep_ms.append(e0.elapsed_time(e1) / K)
    if on_timed:
        on_timed(False)
    rep_sorted = sorted(rep_ms)
    ms = rep_sorted[len(rep_sorted) // 2]
    n_steps = K * reps
    prof = None
    if profile:
        model.d3_profile(True)
        model.d3_read_profile()
        n = min(K, 8)
        for _ in range(n):
            step()
        prof = {k: {"ms_per_step": v["ms"] / n, "launches_per_step": v["launches"] / n}
                for k, v in model.d3_read_profile().items() if v["launches"]}
        model.d3_profile(False)
    model.d3_sync()
    peak, kind = measured_hbm_gbs()
    gbs = tot["bytes"] / n_steps / 1e6 / ms
    line = {
        "workload": name, "shape": shape.name, "rows": rows, "prompt": [plo, phi], "alpha": alpha,
        "exec": exec_mode, "steps": K, "warmup": W, "reps": reps, "ms_per_step": ms,
        "ms_per_step_best": rep_sorted[0], "tokens_per_s": rows / ms * 1e3,
        "algorithmic_gb_per_step": tot["bytes"] / n_steps / 1e9, "achieved_gbs": gbs,
        "frac_of_hbm_peak": gbs / peak, "frac_of_nominal_8TBs": gbs / 8000.0, "peak_gbs": peak, "peak_kind": kind,
        "rows_layers_per_step": tot["rows_layers"] / n_steps, "layers_touched_per_step": tot["touched"] / n_steps,
        "launches_per_step": tot["launches"] / n_steps, "prefill_ms_all_rows": prefill_ms,
        "prompt_tokens_all_rows": int(sum(int(v) for v in lens)), "kernel_classes": prof,
    }
    model.close()
    del model, w
    torch.cuda.empty_cache()
    return line


def main(argv=None) -> int:
    ap = argparse.ArgumentParser()
    ap.add_argument("workload", choices=sorted(WORKLOADS))
    ap.add_argument("--layers", type=int, default=0)
    ap.add_argument("--steps", type=int, default=0)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--alpha", type=float, default=0.0)
    ap.add_argument("--gen-offset", type=int, default=0, help="added to every row's generation index")
    ap.add_argument("--exec", dest="exec_mode", default="auto", choices=sorted(EXEC))
    ap.add_argument("--rows", type=int, default=0, help="override the workload's row count (1 = single-kernel step)")
    ap.add_argument("--reps", type=int, default=1, help="repetitions of the timed region (median reported)")
    ap.add_argument("--profile", action="store_true")
    args = ap.parse_args(argv)
    line = run_workload(args.workload, args.layers, args.steps, args.warmup, args.alpha, args.gen_offset,
                        args.exec_mode, args.rows, args.profile, args.reps)
    print(json.dumps(line), flush=True)
    return 0


if __name__ == "__main__":
    sys.exit(main())
