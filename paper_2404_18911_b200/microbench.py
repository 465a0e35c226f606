"""Step and operator microbenchmarks of the decode path (the verify-step / draft-step evaluation shapes).

    python -m paper_2404_18911_b200.microbench [--workload 7b] [--what steps|ops|all] [--T 128,512,2048,4096]
                                               [--M 1,2,3,4,5,6,7,8,9,10,11,16] [--warmup 20] [--reps 100]

steps: the verify pass (layers l+1..L + head on M rows) against a seeded N(0,1) KV cache of length T,
       the draft loop with eta = 0 (gamma full draft steps + one shallow pass), and plain AR steps;
ops:   each linear operator of a layer and the LM head as a single launch, rotating over enough
       weight copies that no launch finds its weights in L2.
Prints one JSON object per point: median time with p10 / p90 over the timed launches (after the warm-up launches),
algorithmic bytes, achieved GB/s.
"""
from __future__ import annotations

import argparse
import json
import statistics
import sys


def _events(torch):
    return torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)


def _pct(xs, q):
    xs = sorted(xs)
    return xs[min(len(xs) - 1, max(0, int(round(q * (len(xs) - 1)))))]


def bench_steps(args, shape, torch, binding, traffic):
    Ts = [int(t) for t in args.T.split(",")]
    Ms = [int(m) for m in args.M.split(",")]
    max_T = max(Ts)
    shape = shape.with_(max_seq=max_T + 64 + 2 * shape.gamma_max, gamma_max=max(shape.gamma_max, max(Ms) - 1))
    model = binding.KangarooModel(shape)
    out = []
    for T in Ts:
        for M in Ms:
            ms = []
            for r in range(args.reps + args.warmup):
                model.fill_state(T, M - 1, 7 + r)
                e0, e1 = _events(torch)
                e0.record()
                model.verify(sync=False)
                e1.record()
                torch.cuda.synchronize()
                if r >= args.warmup:
                    ms.append(e0.elapsed_time(e1))
            b = traffic.verify_bytes(shape, T, M)
            t = statistics.median(ms)
            out.append({"point": "verify", "T": T, "M": M, "ms": t, "ms_p10": _pct(ms, 0.1), "ms_p90": _pct(ms, 0.9), "bytes": b,
                        "GBps": b / t / 1e6, "launches": len(ms)})
            print(json.dumps(out[-1]), flush=True)
        # draft loop, eta = 0: gamma adapter+head steps and gamma+1 shallow passes
        g = min(shape.gamma_max, 10)
        ms = []
        for r in range(args.reps + args.warmup):
            model.fill_state(T, -1, 7 + r)
            e0, e1 = _events(torch)
            e0.record()
            model.draft(0.0, g, binding.STOP_KEEP, sync=False)
            e1.record()
            torch.cuda.synchronize()
            if r >= args.warmup:
                ms.append(e0.elapsed_time(e1))
        b = sum(traffic.shallow_pass_bytes(shape, T + j) for j in range(g + 1)) + \
            sum(traffic.adapter_head_bytes(shape, T + j, 1) for j in range(g))
        t = statistics.median(ms)
        out.append({"point": "draft_loop", "T": T, "gamma": g, "ms": t, "ms_per_draft_step": t / (g + 0.5), "bytes": b,
                    "GBps": b / t / 1e6})
        print(json.dumps(out[-1]), flush=True)
        # one draft step exactly (one shallow pass, one adapter + LM-head pass): eta > 1, low-confidence token dropped
        ms = []
        for r in range(args.reps + args.warmup):
            model.fill_state(T, -1, 7 + r)
            e0, e1 = _events(torch)
            e0.record()
            model.draft(2.0, 1, binding.STOP_DROP, sync=False)
            e1.record()
            torch.cuda.synchronize()
            if r >= args.warmup:
                ms.append(e0.elapsed_time(e1))
        b = traffic.draft_step_bytes(shape, T)
        t = statistics.median(ms)
        out.append({"point": "draft_step", "T": T, "ms": t, "ms_p10": _pct(ms, 0.1), "ms_p90": _pct(ms, 0.9), "bytes": b,
                    "GBps": b / t / 1e6, "launches": len(ms)})
        print(json.dumps(out[-1]), flush=True)
        # plain AR
        n = 8
        ms = []
        for r in range(3):
            model.fill_state(T, -1, 7 + r)
            e0, e1 = _events(torch)
            e0.record()
            model.decode_ar(1 + n, sync=False)
            e1.record()
            torch.cuda.synchronize()
            ms.append(e0.elapsed_time(e1))
        b = sum(traffic.ar_step_bytes(shape, T + j) for j in range(n))
        t = statistics.median(ms)
        out.append({"point": "ar", "T": T, "steps": n, "ms_per_step": t / n, "bytes_per_step": b / n, "GBps": b / t / 1e6})
        print(json.dumps(out[-1]), flush=True)
    return out


def bench_ops(args, shape, torch, binding):
    d, F, V = shape.d_model, shape.d_ffn, shape.vocab
    ops = [("qkv", 3 * d, d, False), ("o", d, d, False), ("gate_up", F, d, True), ("down", d, F, False), ("head", V, d, False)]
    Ms = [int(m) for m in args.M.split(",")]
    scratch = binding.op_scratch(torch)
    for name, N, K, dual in ops:
        per = N * K * 2 * (2 if dual else 1)
        n_buf = max(2, int(600e6 // per) + 1)
        Ws = [torch.randn(N, K, device="cuda", dtype=torch.float32).mul_(0.02).to(torch.bfloat16) for _ in range(n_buf)]
        W2s = [torch.randn(N, K, device="cuda", dtype=torch.float32).mul_(0.02).to(torch.bfloat16) for _ in range(n_buf)] if dual else None
        gain = torch.ones(K, device="cuda")
        for M in Ms:
            x = torch.randn(M, K, device="cuda")
            resid = torch.randn(M, N, device="cuda")
            def call(i):
                if name == "head":
                    binding.op_lm_head(Ws[i % n_buf], x, gain, 1e-6, 8.0, want_logits=False, scratch=scratch)
                elif dual:
                    binding.op_linear(Ws[i % n_buf], x, gain=gain, W2=W2s[i % n_buf], scratch=scratch)
                else:
                    binding.op_linear(Ws[i % n_buf], x, resid=resid, scratch=scratch)
            for i in range(n_buf):
                call(i)
            reps = max(args.reps, n_buf) * 2
            e0, e1 = _events(torch)
            torch.cuda.synchronize()
            e0.record()
            for i in range(reps):
                call(i)
            e1.record()
            torch.cuda.synchronize()
            t = e0.elapsed_time(e1) / reps
            print(json.dumps({"point": "op", "op": name, "N": N, "K": K, "M": M, "us": 1e3 * t, "bytes": per,
                              "GBps": per / t / 1e6, "note": "includes launch gap and output allocation"}), flush=True)
        del Ws, W2s


def bench_sweep(args, shape, torch, binding):
    """End-to-end decode of the workload for a grid of (eta, gamma): decode-only tokens/s (device time of the decode
    launch), compression rate (Eq. 1), draft steps, and the speed-up over plain greedy decoding on the same kernels."""
    import kg_inputs as ki
    model = binding.KangarooModel(shape)
    prompt = ki.make_prompt(shape).tolist()
    n = shape.n_gen
    # plain greedy baseline
    model.reset(); model.prefill(prompt)
    e0, e1 = _events(torch)
    e0.record(); model.decode_ar(n, sync=False); e1.record(); torch.cuda.synchronize()
    ar_ms = e0.elapsed_time(e1)
    ref = model.read_tokens(n)
    print(json.dumps({"point": "greedy", "tokens": n, "ms": ar_ms, "tokens_per_s": (n - 1) / ar_ms * 1e3}), flush=True)
    for gamma in (2, 4, 6, 10):
        for eta in (0.0, 0.2, 0.4, 0.6, 0.8):
            toks, st = model.generate(prompt, n, eta, gamma)
            assert toks == ref, "speculative output differs from greedy decoding"
            print(json.dumps({"point": "kangaroo", "eta": eta, "gamma": gamma, "ms_decode": st["ms_decode"],
                              "tokens_per_s": (n - 1) / st["ms_decode"] * 1e3, "speedup_vs_greedy": ar_ms / st["ms_decode"],
                              "cr": st["cr"], "rounds": st["rounds"], "draft_steps": st["draft_steps"],
                              "accept_rate": st["accepted"] / max(st["drafted"], 1)}), flush=True)


def main():
    import torch
    import kg_inputs as ki
    from paper_2404_18911_b200 import binding, traffic, build_library
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="7b")
    ap.add_argument("--what", default="steps", choices=["steps", "ops", "sweep", "all"])
    ap.add_argument("--T", default="128,512,2048,4096")
    ap.add_argument("--M", default="1,2,3,4,5,6,7,8,9,10,11,16")
    ap.add_argument("--reps", type=int, default=100, help="timed launches per point")
    ap.add_argument("--warmup", type=int, default=20, help="untimed launches per point")
    args = ap.parse_args()
    build_library()
    binding.load()
    shape = ki.get_config(args.workload)
    if args.what in ("steps", "all"):
        bench_steps(args, shape, torch, binding, traffic)
    if args.what in ("ops", "all"):
        bench_ops(args, shape, torch, binding)
    if args.what == "sweep":
        bench_sweep(args, shape, torch, binding)
    return 0


if __name__ == "__main__":
    sys.exit(main())
