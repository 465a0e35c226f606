#!/usr/bin/env python
"""Throughput of the Kangaroo batch-1 self-speculative decode step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 7b] [--impl kangaroo|reference]

One step = one generation job of the named workload: reset, prefill of the prompt, then draft /
verify / accept rounds until n_gen tokens exist (Figure 2 of the paper), all on the device.
`value` is generated tokens per second over the whole step (prefill included) with the prompt
already resident in HBM; `e2e` is the same job through kg_generate with pinned host buffers
(prompt copied in, tokens copied out, every step).  The roofline object describes the decode
launch (all rounds of a step run inside one persistent kernel launch): algorithmic bytes from the
device's own per-round log divided by its CUDA-event duration.  Its `draft_step` and `verify_step`
entries time single launches of one draft step (layers 1..l, adapter, LM head on one row) and of
one verify pass (layers l+1..L and the LM head on M rows) against a KV cache of 512 tokens:
>= 20 warm-up and >= 100 timed launches each, median with p10 / p90.

With --gpus N > 1 (launched by torchrun) every rank runs an independent replica of the job: the
batch-1 chain has no exchange step, so there is no collective on the data path.

--impl reference times the CPU oracle on a bounded sample of the same workload.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) over algorithmic bytes of the decode launch, from an ncu
# capture of a 4-layer case of the same kernel (the traffic is weights + KV and grows in proportion to the bytes a
# launch streams).  Set to None when the kernel changes.
NCU_TRAFFIC_RATIO = 0.995

METRIC = "batch-1 generated tokens/s"
UNIT = "tokens/s"


# ------------------------------------------------------------------------------------ helpers

def _dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def _measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            with open(p) as f:
                d = json.load(f)
            return float(d["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
        except Exception:
            pass
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons every 200 ms while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "200", "-i", str(self.gpu_index)],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
            if self.thread is not None:
                self.thread.join(timeout=2)

    def summary(self, t0, t1):
        rows = [r for (t, r) in self.rows if t0 <= t <= t1 and len(r) >= 9] or [r for (_, r) in self.rows if len(r) >= 9]
        if not rows:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0}
        sm = []
        for r in rows:
            try:
                sm.append(float(r[1]))
            except ValueError:
                pass
        try:
            smax = float(rows[0][2])
        except ValueError:
            smax = None
        reasons = set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            for name, v in zip(names, r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        power = []
        for r in rows:
            try:
                power.append(float(r[3]))
            except ValueError:
                pass
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": smax, "reasons": sorted(reasons),
                "samples": len(rows), "power_w_max": max(power) if power else None}


def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    if dist is None:
        return [float(v) for v in values]
    import torch
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def job_throughput(units_per_rank_step, steps, world, ms_max):
    """Whole-job throughput of `world` independent replicas: all units processed / the slowest rank's time."""
    return world * units_per_rank_step * steps / (ms_max * 1e-3)


# ------------------------------------------------------------------------------------ CPU oracle legs

def _oracle_sample(shape_name, n_prompt_s, n_gen_s):
    """Builds the oracle for the workload's shape and returns a callable running one bounded sample:
    prefill of the first n_prompt_s prompt tokens, then Kangaroo rounds until n_gen_s tokens exist."""
    import numpy as np
    import kg_inputs as ki
    from oracle import kangaroo_oracle as ko
    shape = ki.get_config(shape_name)
    shape_s = shape.with_(max_seq=n_prompt_s + n_gen_s + shape.gamma + 8)
    dtype = np.float64 if shape.d_model <= 512 else np.float32   # 8 bytes per weight do not fit for the large shapes
    o = ko.KangarooOracle(shape_s, ki.make_weights(shape_s), dtype)
    prompt = ki.make_prompt(shape, n_prompt_s).tolist()

    def run():
        t0 = time.perf_counter()
        toks = o.generate(prompt, n_gen_s, shape.eta, shape.gamma)
        return len(toks), time.perf_counter() - t0
    return shape, run


def _host_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([int(p.get("num_threads", 1)) for p in threadpool_info()] or [1])
        return n
    except Exception:
        return len(os.sched_getaffinity(0))


def _sample_sizes(shape_name):
    # sized so that one sample is a few seconds of host work on the 7B shape
    return {"tiny": (32, 64), "7b": (32, 8), "13b": (32, 6), "33b": (32, 4)}[shape_name]


def cpu_baseline(shape_name, repeats=1):
    n_prompt_s, n_gen_s = _sample_sizes(shape_name)
    shape, run = _oracle_sample(shape_name, n_prompt_s, n_gen_s)
    best = None
    for _ in range(repeats):
        n, dt = run()
        best = dt if best is None else min(best, dt)
    return {"value": n_gen_s / best, "unit": UNIT, "cores": _host_threads(), "kind": "oracle",
            "sample": f"{shape_name} shape, first {n_prompt_s} prompt tokens, {n_gen_s} generated tokens "
                      f"(eta={shape.eta}, gamma={shape.gamma}), prefill included, {best:.2f} s"}


def run_reference(args):
    rank, _, world = _dist_env()
    if rank != 0:
        return 0
    n_prompt_s, n_gen_s = _sample_sizes(args.workload)
    shape, run = _oracle_sample(args.workload, n_prompt_s, n_gen_s)
    for _ in range(args.warmup):
        run()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run()
    dt = time.perf_counter() - t0
    value = n_gen_s * args.steps / dt
    sample = (f"each step: {args.workload} shape, first {n_prompt_s} prompt tokens, {n_gen_s} generated tokens, "
              f"prefill included")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32" if shape.d_model > 512 else "f64", "data": "synthetic",
            "config": dict(_config(shape, args, 1), sample=sample), "gpu_launches": 0,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": _host_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)
    return 0


def _percentile(xs, q):
    xs = sorted(xs)
    return xs[min(len(xs) - 1, max(0, int(round(q * (len(xs) - 1)))))]


def step_rooflines(model, shape, binding, traffic, torch, peak, T=512, Ms=(1, 4, 7), warm=20, reps=100):
    """Single launches of one draft step and of one verify pass on the microbenchmark state (seeded N(0,1) KV cache of
    length T, N(0,1) early features): algorithmic bytes / CUDA-event time of the launch, against the copy peak."""
    def timed(prepare, launch, nbytes):
        ms = []
        for r in range(warm + reps):
            prepare(r)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); launch(); e1.record()
            torch.cuda.synchronize()
            if r >= warm:
                ms.append(e0.elapsed_time(e1))
        med = statistics.median(ms)
        return {"ms": med, "ms_p10": _percentile(ms, 0.1), "ms_p90": _percentile(ms, 0.9), "bytes": nbytes,
                "achieved": nbytes / (med * 1e-3) / 1e9, "frac": nbytes / (med * 1e-3) / 1e9 / peak,
                "frac_of_8TBs": nbytes / (med * 1e-3) / 1e9 / 8000.0, "launches": reps}
    out = {"kv_len": T, "warmup": warm, "unit": "GB/s", "peak": peak}
    # one draft step exactly: with eta > 1 in the stop mode that drops the low-confidence token the loop runs one
    # shallow pass, one adapter + LM-head pass, and stops
    out["draft_step"] = timed(lambda r: model.fill_state(T, -1, 100 + r),
                              lambda: model.draft(2.0, 1, binding.STOP_DROP, sync=False), traffic.draft_step_bytes(shape, T))
    out["verify_step"] = {}
    for M in Ms:
        out["verify_step"][f"M={M}"] = timed(lambda r, M=M: model.fill_state(T, M - 1, 200 + r),
                                             lambda: model.verify(sync=False), traffic.verify_bytes(shape, T, M))
    return out


def _config(shape, args, world):
    return {"workload": f"{shape.name}: L={shape.n_layers} d={shape.d_model} H={shape.n_heads}x{shape.head_dim} "
                        f"F={shape.d_ffn} V={shape.vocab} l={shape.exit_layer} {shape.dtype}; batch 1, prompt "
                        f"{shape.n_prompt}, generate {shape.n_gen} greedy, eta={shape.eta}, gamma={shape.gamma}, stop=keep",
            "timed_region": "reset + prefill + decode rounds (draft loop, verify, accept) per step",
            "l2": "inputs larger than L2: every pass streams >= 1.2 GB of weights (L2 is 126 MB)",
            "parallelism": "1 GPU" if world == 1 else f"{world} independent replicas"}


# ------------------------------------------------------------------------------------ the CUDA arm

def run_kangaroo(args):
    import numpy as np
    import torch
    import kg_inputs as ki
    import __graft_entry__ as ge
    from paper_2404_18911_b200 import binding, traffic

    rank, local_rank, world = _dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_
        dist = dist_
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        ge.build()
    if dist is not None:
        dist.barrier()
    binding.load()

    shape = ki.get_config(args.workload)
    if args.n_gen:
        shape = shape.with_(n_gen=args.n_gen)
    if args.n_prompt:
        shape = shape.with_(n_prompt=args.n_prompt)
    if args.layers:
        shape = shape.with_(n_layers=args.layers, name=f"{shape.name}-{args.layers}layers")
    if shape.n_prompt + shape.n_gen + shape.gamma + 8 > shape.max_seq:
        shape = shape.with_(max_seq=shape.n_prompt + shape.n_gen + shape.gamma + 8)
    mode = binding.STOP_DROP if args.stop == "drop" else binding.STOP_KEEP
    model = binding.KangarooModel(shape, device=f"cuda:{local_rank}")
    prompt_np = ki.make_prompt(shape)
    prompt_dev = torch.from_numpy(prompt_np).to(f"cuda:{local_rank}")
    prompt_pin = torch.from_numpy(prompt_np).pin_memory()
    out_pin = torch.empty(shape.n_gen, dtype=torch.int32).pin_memory()
    torch.cuda.synchronize()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    ev = lambda: torch.cuda.Event(enable_timing=True)

    def step_device(marks=None):
        a = ev(); a.record()
        model.reset()
        model.prefill_device(prompt_dev)
        b = ev(); b.record()
        model.decode(shape.n_gen, shape.eta, shape.gamma, mode, sync=False)
        c = ev(); c.record()
        if marks is not None:
            marks.append((a, b, c))

    for _ in range(args.warmup):
        step_device()
    barrier()
    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.25)

    # ---- timed region 1: device-resident job
    marks = []
    barrier()
    t_wall0 = time.time()
    e0 = ev(); e0.record()
    for _ in range(args.steps):
        step_device(marks)
    e1 = ev(); e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    prefill_ms = [a.elapsed_time(b) for (a, b, c) in marks]
    decode_ms = [b.elapsed_time(c) for (a, b, c) in marks]
    toks_dev = model.read_tokens(shape.n_gen)
    st_log = model.read_round_log()

    # ---- timed region 2: through kg_generate with pinned host buffers
    for _ in range(min(2, args.warmup)):
        model.generate_into(prompt_pin, out_pin, shape.n_gen, shape.eta, shape.gamma, mode)
    barrier()
    f0 = ev(); f0.record()
    for _ in range(args.steps):
        _, stats = model.generate_into(prompt_pin, out_pin, shape.n_gen, shape.eta, shape.gamma, mode)
    f1 = ev(); f1.record()
    barrier()
    t_wall1 = time.time()
    ms_e2e = f0.elapsed_time(f1)
    sampler.stop()
    assert out_pin.tolist() == toks_dev, "kg_generate and prefill_device + decode disagree"

    ms_total, ms_e2e = max_over_ranks([ms_total, ms_e2e], dist, f"cuda:{local_rank}")

    if rank == 0:
        n_tok = shape.n_gen
        value = job_throughput(n_tok, args.steps, world, ms_total)
        e2e = job_throughput(n_tok, args.steps, world, ms_e2e)
        peak, peak_src = _measured_peaks()
        dec_bytes = traffic.decode_bytes(shape, st_log)
        dec_ms = statistics.mean(decode_ms)
        achieved = dec_bytes / (dec_ms * 1e-3) / 1e9
        rounds = len(st_log)
        n_steps_total = sum(r[1] for r in st_log)
        drafted = sum(r[0] for r in st_log)
        accepted = sum(r[2] for r in st_log)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16 weights and KV, f32 accumulate" if shape.dtype == "bf16" else "f32", "data": "synthetic",
            "config": _config(shape, args, world),
            "e2e": {"value": e2e, "unit": UNIT, "h2d_bytes_per_step": int(prompt_np.nbytes), "d2h_bytes_per_step": int(4 * n_tok)},
            "gpu_launches": 2 * args.steps,
            "clocks": sampler.summary(t_wall0, t_wall1),
            "roofline": {"bound": "hbm", "kernel": "kg_persistent_kernel (decode program: all rounds of one step)",
                         "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "frac_of_8TBs": achieved / 8000.0, "peak_source": peak_src,
                         "bytes_per_launch": dec_bytes, "ms_per_launch": dec_ms,
                         "traffic": None if NCU_TRAFFIC_RATIO is None else int(NCU_TRAFFIC_RATIO * dec_bytes),
                         "traffic_source": None if NCU_TRAFFIC_RATIO is None else
                         f"ncu dram bytes of a 4-layer launch of the same kernel, scaled by algorithmic bytes (x{NCU_TRAFFIC_RATIO})"},
            "breakdown": {"prefill_ms": statistics.mean(prefill_ms), "decode_ms": dec_ms,
                          "decode_only_tokens_per_s": (n_tok - 1) / (dec_ms * 1e-3),
                          "rounds": rounds, "cr": (n_tok - 1) / max(rounds, 1), "draft_steps": n_steps_total,
                          "drafted": drafted, "accepted": accepted,
                          "accept_rate": accepted / max(drafted, 1)},
        }
        if not args.no_step_rooflines and not args.layers:
            steps = step_rooflines(model, shape, binding, traffic, torch, peak)
            line["roofline"]["draft_step"] = steps.pop("draft_step")
            line["roofline"]["verify_step"] = steps.pop("verify_step")
            line["roofline"]["step_timing"] = steps
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(args.workload)
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="kangaroo", choices=["kangaroo", "reference"])
    ap.add_argument("--workload", default="7b", choices=["tiny", "7b", "13b", "33b"])
    ap.add_argument("--stop", default="keep", choices=["keep", "drop"])
    ap.add_argument("--n-gen", type=int, default=0, help="override the number of generated tokens (debugging)")
    ap.add_argument("--n-prompt", type=int, default=0, help="override the prompt length (profiling on a small case)")
    ap.add_argument("--layers", type=int, default=0, help="override the number of layers (profiling on a small case)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-step-rooflines", action="store_true", help="skip the single-launch draft-step / verify-step timings")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "kangaroo" else args.warmup
    if args.impl == "reference":
        return run_reference(args)
    return run_kangaroo(args)


if __name__ == "__main__":
    sys.exit(main())
