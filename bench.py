#!/usr/bin/env python
"""Benchmark of recurrent-pipeline decoding on B200.

One "step" is one pass of the whole hot path over one batch of synthetic input: every sample's
first visit (prompt through all partitions) followed by the recurrent pipeline until each sample
has n_new greedy tokens.  Headline workload: the Llama-7B shape (32 layers, d 4096, bf16 seeded
weights, 8 partitions of 4 layers, 64 samples in flight, 128-token prompts, 512 new tokens), the
largest of the five named workloads; the other four are timed in the same run with fewer
repetitions and reported under `per_workload`.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

Prints ONE JSON line.  `value` = generated tokens/s over all samples with the prompts already in
device memory (device time from library-side CUDA events on its own streams); `e2e` = the same
through the host-pointer entry points, prompts copied in and tokens copied out every step;
`roofline` = decode phase against the measured HBM copy bandwidth; `cpu_baseline` = the CPU
checker timed on a bounded sample of the same workload.  With N > 1 every rank runs an
independent replica (the path does not shard) and the values add up.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2505_18164_b200 import inputs as I  # noqa: E402

HEADLINE = "llama_7b"
METRIC = "generated tokens/s (all in-flight samples)"
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0

# DRAM traffic of the decode phase relative to its algorithmic bytes, from the ncu captures kept with the profiler
# summaries of this repository (see profiles/): per workload and scheduler the ratio (dram bytes read + written) /
# (algorithmic bytes) of the dominant kernel on a short capture.  Weights are ~90-99% of both and are read once per
# group and pass, so traffic grows with the number of passes like the algorithmic bytes do.  None where no capture of
# the current kernel exists.
# llama_7b, stream scheduler: three consecutive k_tc_gemm launches on the workload's widths (8 positions, tiled weights)
# read 226.1 MB and wrote 7.6 MB for 224.4 MB of matrices (profiles/stream_scheduler_llama_7b_launch_list.md).
TRAFFIC_RATIO: dict = {("llama_7b", 0): 1.04, ("llama_7b", 1): 1.04}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return float(d["hbm_gbs"]), "measured"
        except Exception:
            pass
    return FALLBACK_HBM_GBS, "fallback"


def decode_bytes(w: I.Workload, n_samples: int, kv_bpe: int) -> dict:
    """Algorithmic bytes of the decode phase of one step (what the schedule must move).

    Per pass (every sample gains one token) each of the G groups streams every block matrix and
    vector once and the output projection once; each sample reads its whole cache (keys and values
    of every layer, rows 0..t) and writes one row per layer, kv_bpe bytes per element.  Embedding
    rows and activations are negligible and left out."""
    s = w.shape
    bpe = 4 if s.weight_dtype == I.DT_F32 else 2
    specs = I.tensor_specs(s)
    block = sum(int(np.prod(shp)) for n, shp, _ in specs if n.startswith("h."))
    head = s.vocab * s.d_model + s.d_model * (2 if s.arch == I.ARCH_GPT else 1)
    G = min(n_samples, w.n_partitions)
    per_pass_w = G * (block + head) * bpe
    kvw = s.n_kv_head * s.head_dim
    n_pass = w.n_new - 1
    kv = 0
    for i in range(n_pass):
        t = w.n_prompt + i                       # rows cached before this pass
        kv += n_samples * s.n_layer * (2 * (t + 1) * kvw + 2 * kvw) * kv_bpe
    return {"weights": per_pass_w * n_pass, "kv": kv, "total": per_pass_w * n_pass + kv, "passes": n_pass,
            "per_pass_weights": per_pass_w}


def workload_config(w: I.Workload, world: int) -> dict:
    s = w.shape
    return {"workload": w.name, "n_layer": s.n_layer, "d_model": s.d_model, "vocab": s.vocab,
            "partitions": list(w.part_bounds), "samples_in_flight": w.n_samples, "n_prompt": w.n_prompt, "n_new": w.n_new,
            "l2": "the weights streamed per tick (one pass over the model per round and group, plus caches) exceed the "
                  "126 MB L2 except on tiny_gpt_fp32, which is L2-resident by construction; no flush between steps",
            "multi_gpu": "replicas only" if world > 1 else "single"}


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "200", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def stop(self) -> dict:
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
                pw.append(float(f[2]))
            except ValueError:
                continue
            for nm, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w": statistics.median(pw) if pw else None, "reasons": sorted(reasons), "samples": len(sm)}


# ---- the CPU checker as a timed baseline ---------------------------------------------------------------

def oracle_sample_plan(w: I.Workload, cores: int):
    """What the CPU checker is timed on: the whole workload where that costs seconds, else one sample's shortened
    prompt and first new tokens, sized for about 5-8 s from rough per-core rates of the checker (measured once:
    about 1.5e9 parameters per second and core, decoding and per prompt position alike; small models run below that)."""
    n_params = I.param_bytes(w.shape) / (4 if w.shape.weight_dtype == I.DT_F32 else 2)
    dec_rate = cores * 1.5e9 / n_params
    pf_rate = cores * 1.5e9 / n_params
    full_cost = w.n_samples * (w.n_prompt / pf_rate + w.n_new / dec_rate)
    if full_cost <= 12.0:
        return ("full",)
    p_s = int(min(w.n_prompt, max(min(w.n_prompt, 8), 3.0 * pf_rate)))
    n_s = int(min(w.n_new - 1, max(8, 4.0 * dec_rate)))
    return ("slot0", p_s, n_s)


def cpu_baseline(w: I.Workload, weights):
    """The CPU checker, as it stands, on a bounded sample of the workload -> (cpu_baseline object, seconds of CPU work).

    "full": all samples, full prompts, all new tokens, scheduled by the checker's own recurrent-pipeline simulation;
    the value is tokens / time.  "slot0": sample 0 alone, the first p_s tokens of its prompt and its first n_s + 1
    new tokens; the prompt visit and the decode steps are timed separately and the value is the whole workload
    projected from those two rates: S N / (S P t_position + S (N - 1) / r_decode)."""
    from oracle import mdi_oracle as O
    cores = O.num_threads()
    plan = oracle_sample_plan(w, cores)
    orc = O.Oracle(w.shape, weights)
    prompts = I.make_prompts(w.shape.vocab, w.n_samples, w.n_prompt, w.prompt_seed)
    S, P, N = w.n_samples, w.n_prompt, w.n_new
    t0 = time.perf_counter()
    if plan[0] == "full":
        toks, _, _ = orc.generate_pipeline([[int(t) for t in p] for p in prompts], N, list(w.part_bounds), head_on_starter=False)
        dt = time.perf_counter() - t0
        value = sum(len(t) for t in toks) / dt
        sample = f"the whole workload: {S} samples, {P}-token prompts, {N} new tokens each, {dt:.1f} s of CPU work"
    else:
        _, p_s, n_s = plan
        prompt = [int(t) for t in prompts[0][:p_s]]
        orc.generate_sequential(prompt, 1, list(w.part_bounds))
        t_pf = time.perf_counter() - t0
        t1 = time.perf_counter()
        orc.generate_sequential(prompt, 1 + n_s, list(w.part_bounds))
        t_all = time.perf_counter() - t1
        dt = time.perf_counter() - t0
        t_pos = t_pf / p_s
        r_dec = n_s / max(t_all - t_pf, 1e-9)
        value = S * N / (S * P * t_pos + S * (N - 1) / r_dec)
        sample = (f"sample 0 alone: first {p_s} of its {P} prompt tokens ({t_pos * 1e3:.0f} ms per position) and its first "
                  f"{n_s + 1} new tokens ({r_dec:.2f} tokens/s decoding), {dt:.1f} s of CPU work; value = the whole workload "
                  f"({S} samples x ({P} prompt positions + {N} tokens)) projected from these two rates")
    return {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample}, dt


def run_reference(args, w: I.Workload):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    world = int(os.environ.get("WORLD_SIZE", "1"))
    weights = I.make_weights(w.shape, w.weight_seed)
    times, vals, cb = [], [], None
    for i in range(args.warmup + args.steps):
        cb, dt = cpu_baseline(w, weights)
        if i >= args.warmup:
            times.append(dt)
            vals.append(cb["value"])
    v = len(vals) / sum(1.0 / x for x in vals)          # steps are equal amounts of work: harmonic mean of the rates
    cb["value"] = v
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": v, "unit": "tokens/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w, world),
        "cpu_baseline": cb,
        "e2e": {"value": v, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0}))


def max_over_ranks(values, world: int, device: str = "cpu"):
    """Per-rank totals -> the slowest rank's (replicas run independently; the job is as slow as its slowest)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def aggregate_tokens_per_s(world: int, n_samples: int, n_new: int, steps: int, total_ms: float) -> float:
    """Whole-job throughput: every rank generated n_samples * n_new tokens per step."""
    return world * n_samples * n_new * steps / (total_ms * 1e-3)


# ---- one workload on this rank's GPU --------------------------------------------------------------------

def run_workload(w: I.Workload, args, steps: int, warmup: int, e2e_steps: int, world: int, rank: int, want_cpu: bool,
                 sampler_index=None):
    """Times `steps` steps after `warmup`, then `e2e_steps` through the host-pointer entry points.
    Returns a dict of measurements (times are this rank's; the caller reduces over ranks)."""
    import torch
    import torch.distributed as dist
    from paper_2505_18164_b200 import mdi

    s = w.shape
    S, P, N = w.n_samples, w.n_prompt, w.n_new
    ctx = mdi.Context(s, list(w.part_bounds), S, kv_pool_tokens=S * ((P + N + 15) // 16 * 16), rounds_per_graph=args.rounds_per_graph,
                      scheduler=args.scheduler, tc_min_group=args.tc_min_group, kv_cache_dtype=args.kv_cache_dtype,
                      in_kernel_timing=1 if args.in_kernel_timing else 0, td_b_kblocks=args.td_b_kblocks,
                      fused_blocks_per_head=args.fused_blocks_per_head)
    weights = {}
    for name, a in I.iter_weights(s, w.weight_seed):
        ctx.load_weights(name, a)
        if want_cpu:
            weights[name] = a
    prompts_host = torch.from_numpy(I.make_prompts(s.vocab, S, P, w.prompt_seed)).pin_memory()
    prompts_dev = prompts_host.cuda()
    out_dev = torch.empty((S, N), dtype=torch.int32, device="cuda")
    out_host = torch.empty((S, N), dtype=torch.int32).pin_memory()
    out_np = out_host.numpy()
    prompts_np = prompts_host.numpy()

    def step_device():
        for smp in range(S):
            ctx.reset_sample(smp)
        for smp in range(S):
            ctx.prefill_dev(smp, prompts_dev[smp], P)
        ctx.generate_dev(S, N, out_dev)

    def step_host():
        for smp in range(S):
            ctx.reset_sample(smp)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for smp in range(S):
            ctx.prefill(smp, prompts_np[smp])
        ctx.generate(S, N, out_np)
        return time.perf_counter() - t0

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warmup):
        step_device()
    barrier()
    sampler = ClockSampler(sampler_index) if sampler_index is not None else None
    if sampler:
        sampler.start()
    st0 = ctx.stats()
    run_ms, gen_ms, pf_ms = [], [], []
    for _ in range(steps):
        step_device()
        st = ctx.stats()
        run_ms.append(st.last_run_ms)
        gen_ms.append(st.last_generate_ms)
        pf_ms.append(st.last_prefill_ms)
    barrier()
    st1 = ctx.stats()
    clocks = sampler.stop() if sampler else None
    tokens_dev = out_dev.cpu().numpy().copy()

    # end to end through the host-pointer entry points
    e2e_s = []
    if e2e_steps > 0:
        step_host()
        barrier()
        e2e_s = [step_host() for _ in range(e2e_steps)]
        barrier()
        assert np.array_equal(out_np, tokens_dev), "host and device entry points disagree"
    kv_stored_bpe = int(st1.kv_element_bytes)
    ptimes = None
    if args.in_kernel_timing:
        try:
            ptimes = [dict(zip(("blocks", "ms"), ctx.partition_times(p))) for p in range(w.n_partitions)]
        except Exception as e:  # the stream scheduler has no in-kernel timing
            ptimes = str(e)
    res = {"run_ms": run_ms, "gen_ms": gen_ms, "pf_ms": pf_ms, "e2e_s": e2e_s, "clocks": clocks, "partition_times_ms": ptimes,
           "launches": int(st1.kernel_launches - st0.kernel_launches), "kv_stored_bpe": kv_stored_bpe}
    ctx.close()
    del ctx
    torch.cuda.empty_cache()
    if want_cpu:
        res["cpu_baseline"], _ = cpu_baseline(w, weights)
    return res


def roofline_of(w: I.Workload, gen_avg_ms: float, kv_stored_bpe: int, peak: float, peak_kind: str, traffic_key) -> dict:
    """Decode phase against the HBM copy bandwidth.  `algorithmic_bytes` counts the cache at the weights' width
    (2 bytes for the bf16 workloads, 4 for the fp32 one), which is what the method needs; `stored_bytes` counts it at
    the width the library stores (fp32 unless asked otherwise), which is what this implementation moves."""
    kv_alg_bpe = 4 if w.shape.weight_dtype == I.DT_F32 else 2
    db = decode_bytes(w, w.n_samples, kv_alg_bpe)
    ds = decode_bytes(w, w.n_samples, kv_stored_bpe)
    achieved = db["total"] / (gen_avg_ms * 1e-3) / 1e9
    ratio = TRAFFIC_RATIO.get(traffic_key)
    return {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "peak_kind": f"of {peak_kind}", "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
            "frac_on_stored_bytes": ds["total"] / (gen_avg_ms * 1e-3) / 1e9 / peak,
            "traffic": ratio * ds["total"] if ratio else None,
            "traffic_note": ("scaled from a short ncu capture of the same kernels (see profiles/)" if ratio else
                             "no ncu capture of the current kernels for this workload"),
            "scope": "decode phase of one step (all kernels of mdi_generate)",
            "algorithmic_bytes": db["total"], "weight_bytes": db["weights"], "kv_bytes": db["kv"],
            "stored_bytes": ds["total"], "kv_stored_bytes_per_element": kv_stored_bpe}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="mdi", choices=["mdi", "reference"])
    ap.add_argument("--workload", default=None, choices=list(I.ALL_WORKLOADS),
                    help=f"time this workload only (default: {HEADLINE}, plus the other named workloads under per_workload)")
    ap.add_argument("--no-per-workload", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--e2e-steps", type=int, default=-1, help="steps of the end-to-end leg (default: min(steps, 3))")
    ap.add_argument("--rounds-per-graph", type=int, default=0)
    ap.add_argument("--scheduler", type=int, default=0, help="0 auto (a persistent kernel when the shape fits), 1 streams, 2 phase-per-matrix persistent kernel, 3 fused-phase persistent kernel")
    ap.add_argument("--tc-min-group", type=int, default=0, help="smallest group whose decode steps run on the tensor cores (0 = library default)")
    ap.add_argument("--kv-cache-dtype", type=int, default=0, help="0 library default, 1 bf16, 2 fp16, 3 fp32")
    ap.add_argument("--in-kernel-timing", action="store_true", help="persistent kernels time themselves; adds partition_times_ms "
                    "(per partition: blocks, milliseconds per category of the last generate call) to the line")
    ap.add_argument("--fused-blocks-per-head", type=int, default=0, help="scheduler 3: 1 = one block per head (no clusters), 0 = library default")
    ap.add_argument("--td-b-kblocks", type=int, default=0, help="scheduler 4: k-blocks of the resident activation operand")
    ap.add_argument("--n-new", type=int, default=0, help="shorter generation (profiler captures only; not the headline)")
    ap.add_argument("--n-prompt", type=int, default=0, help="shorter prompts (profiler captures only)")
    ap.add_argument("--n-layer", type=int, default=0, help="fewer blocks (profiler captures only)")
    ap.add_argument("--partitions", type=int, default=1, help="with --n-layer: partitions of equal size")
    ap.add_argument("--n-samples", type=int, default=0, help="fewer samples in flight (profiler captures only)")
    args = ap.parse_args()
    headline_only = args.workload is not None or args.no_per_workload
    w = I.ALL_WORKLOADS[args.workload or HEADLINE]
    if args.n_new or args.n_prompt:
        w = I.scaled(w, n_new=args.n_new or w.n_new, n_prompt=args.n_prompt or w.n_prompt)
    if args.n_layer:
        w = I.scaled(w, n_layer=args.n_layer, part_bounds=tuple(range(0, args.n_layer + 1, args.n_layer // args.partitions)))
    if args.n_samples:
        w = I.scaled(w, n_samples=args.n_samples)
    from paper_2505_18164_b200 import build
    build.build_inputs()

    if args.impl == "reference":
        run_reference(args, w)
        return

    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decoding path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    want_cpu = rank == 0 and not args.no_cpu_baseline
    e2e_steps = args.e2e_steps if args.e2e_steps >= 0 else min(args.steps, 3)
    r = run_workload(w, args, args.steps, args.warmup, e2e_steps, world, rank, want_cpu, sampler_index=local if rank == 0 else None)
    S, N = w.n_samples, w.n_new
    tot_run_ms, tot_e2e_ms = max_over_ranks([sum(r["run_ms"]), sum(r["e2e_s"]) * 1e3], world, "cuda")

    per = []
    if not headline_only and world == 1:
        for name in I.WORKLOAD_ORDER:
            if name == w.name:
                continue
            ww = I.ALL_WORKLOADS[name]
            try:
                rr = run_workload(ww, args, 3, 3, 1, 1, 0, want_cpu)
            except Exception as e:  # the headline must not be lost to a secondary workload
                per.append({"workload": name, "error": f"{type(e).__name__}: {e}"})
                continue
            per.append((ww, rr))

    if rank == 0:
        peak, peak_kind = measured_peaks()
        gen_avg_ms = sum(r["gen_ms"]) / len(r["gen_ms"])
        value = aggregate_tokens_per_s(world, S, N, args.steps, tot_run_ms)
        line = {
            "metric": METRIC, "value": value, "unit": "tokens/s",
            "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": tot_run_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if w.shape.weight_dtype == I.DT_BF16 else "f32", "data": "synthetic",
            "config": workload_config(w, world),
            "decode_tokens_per_s": world * S * (N - 1) / (gen_avg_ms * 1e-3),
            "prefill_ms": sum(r["pf_ms"]) / len(r["pf_ms"]), "decode_ms": gen_avg_ms,
            "roofline": roofline_of(w, gen_avg_ms, r["kv_stored_bpe"], peak, peak_kind, (w.name, args.scheduler)),
            "e2e": ({"value": aggregate_tokens_per_s(world, S, N, e2e_steps, tot_e2e_ms), "unit": "tokens/s",
                     "h2d_bytes_per_step": int(S * w.n_prompt * 4), "d2h_bytes_per_step": int(S * N * 4), "steps": e2e_steps}
                    if e2e_steps > 0 else None),
            "gpu_launches": r["launches"],
            "clocks": r["clocks"],
            "cpu_baseline": r.get("cpu_baseline"),
        }
        if r.get("partition_times_ms") is not None:
            line["partition_times_ms"] = r["partition_times_ms"]
        if per:
            out = []
            for item in per:
                if isinstance(item, dict):
                    out.append(item)
                    continue
                ww, rr = item
                g = sum(rr["gen_ms"]) / len(rr["gen_ms"])
                run = sum(rr["run_ms"]) / len(rr["run_ms"])
                rl = roofline_of(ww, g, rr["kv_stored_bpe"], peak, peak_kind, (ww.name, args.scheduler))
                out.append({"workload": ww.name, "steps": 3, "warmup": 3,
                            "value": ww.n_samples * ww.n_new / (run * 1e-3), "unit": "tokens/s", "ms_per_step": run,
                            "prefill_ms": sum(rr["pf_ms"]) / len(rr["pf_ms"]), "decode_ms": g,
                            "frac": rl["frac"], "frac_on_stored_bytes": rl["frac_on_stored_bytes"],
                            "achieved_gbs": rl["achieved"], "algorithmic_bytes": rl["algorithmic_bytes"],
                            "e2e_value": ww.n_samples * ww.n_new / rr["e2e_s"][0] if rr["e2e_s"] else None,
                            "gpu_launches_per_step": rr["launches"] / 3,
                            "served_from": "L2 (the whole model is 42.7 MB)" if ww.name == "tiny_gpt_fp32" else "HBM",
                            "cpu_baseline": rr.get("cpu_baseline")})
            line["per_workload"] = out
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
