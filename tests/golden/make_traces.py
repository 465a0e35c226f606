#!/usr/bin/env python
"""Writes the oracle traces under tests/golden/ that the GPU parity tests replay.

    python tests/golden/make_traces.py [case ...]        # default: every case

Only `oracle/` (the CPU definition of the method) and `kg_inputs/` (seeded inputs) are used; nothing here
touches the CUDA library.  Each case runs the fp64 oracle with weights regenerated tensor by tensor from the
counter-based generator, so that nothing larger than a few layers is resident even for the 33B shape, and stores
what a replay has to reproduce: token ids, the accepted-length list S, per round (P, n_d, n_steps, k), the
drafts, every confidence, the target's tokens, the top-2 logit gap of every arg max, the two leading logits and
a fixed sample of logit entries per row.

Cases
  7b_full     the benchmark job: 7B shape, prompt 512, 256 tokens, eta 0.6, gamma 6, low-confidence draft kept
  13b_short   13B shape, 40-token prompt, 24 tokens, eta 0.6, gamma 6
  33b_short   33B shape, 44-token prompt, 28 tokens, eta 0.6, gamma 8 (with a 40-token prompt the second round already
              holds a verify row whose two leading logits are 0.014 apart, which ends a replay there)
  7b_verify   verify passes of the 7B shape on the microbenchmark state (seeded N(0,1) KV cache of length T and
              N(0,1) early features): (T, rows) = (128, 1), (512, 4), (2048, 8), (4096, 7), (4096, 11)
"""
import json
import os
import sys
import time

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import kg_inputs as ki                                   # noqa: E402
from oracle import kangaroo_oracle as ko                 # noqa: E402

N_SAMPLES = 10
BUDGET_BYTES = int(os.environ.get("KG_TRACE_BUDGET_GB", "36")) << 30     # fp64 tensors kept resident


def lazy_weights(shape):
    """Weights for the fp64 oracle; the draft path's tensors (read most often) are the ones kept resident."""
    w = ki.LazyWeights(shape, np.float64, BUDGET_BYTES)
    w["embed"], w["head"], w["g_final"]
    for blk in [w["adapter"]] + [w["layers"][i] for i in range(shape.exit_layer)]:
        for n in blk.keys():
            blk[n]
    return w


def sample_indices(V):
    """The logit entries every row records: a fixed spread over the vocabulary."""
    return [int((7919 * j + 13) % V) for j in range(N_SAMPLES)]


def row_record(z, idx):
    """Leading two entries (index, value), their gap, and the sampled entries of one logit row."""
    order = np.argsort(-z, kind="stable")[:2]
    return {"top": [[int(order[0]), float(z[order[0]])], [int(order[1]), float(z[order[1]])]],
            "gap": ko.top2_gap(z), "samples": [float(z[i]) for i in idx]}


def generation_case(name, config, n_prompt, n_new, eta, gamma, mode):
    shape = ki.get_config(config).with_(max_seq=n_prompt + n_new + gamma + 8)
    o = ko.KangarooOracle(shape, lazy_weights(shape), np.float64)
    prompt = ki.make_prompt(shape, n_prompt).tolist()
    idx = sample_indices(shape.vocab)
    t0 = time.time()
    x0 = o.prefill(prompt)
    out = [x0]
    trace = {"case": name, "config": config, "n_prompt": n_prompt, "n_new": n_new, "eta": eta, "gamma": gamma,
             "stop_mode": mode, "arithmetic": "float64", "sample_indices": idx,
             "prefill": {"x0": int(x0), **row_record(o.last_logits, idx)}, "rounds": []}
    print(f"[{name}] prefill done in {time.time() - t0:.0f} s, x0 = {x0}", flush=True)
    while len(out) < n_new:
        em = o.round(eta, gamma, mode)
        r = o.log[-1]
        trace["rounds"].append({
            "P": r["P"], "n_d": r["n_drafted"], "n_steps": r["n_steps"], "k": r["k"],
            "drafts": [int(t) for t in r["drafts"]], "conf": [float(p) for p in r["conf"]],
            "target": [int(t) for t in r["target"]], "emitted": [int(t) for t in r["emitted"]],
            "adapter_len_before": r["adapter_len_before"], "adapter_len_after": r["adapter_len_after"],
            "draft_rows": [row_record(z, idx) for z in r["draft_logits"]],
            "verify_rows": [row_record(r["verify_logits"][i], idx) for i in range(r["M"])]})
        r["draft_logits"] = r["verify_logits"] = None     # the full rows are not needed again
        out.extend(em)
        print(f"[{name}] round {len(trace['rounds'])}: n_d={r['n_drafted']} k={r['k']} tokens={len(out)} "
              f"({time.time() - t0:.0f} s)", flush=True)
    S = list(o.S)
    S[-1] -= len(out) - n_new                             # the last round counts only the tokens that are returned
    trace["tokens"] = [int(t) for t in out[:n_new]]
    trace["S"] = S
    trace["cr"] = ko.compression_rate(S)
    return trace


def verify_case(name, config, points, seed):
    base = ki.get_config(config)
    idx = sample_indices(base.vocab)
    trace = {"case": name, "config": config, "seed": seed, "arithmetic": "float64", "sample_indices": idx, "points": []}
    t0 = time.time()
    w = ki.LazyWeights(base, np.float64, BUDGET_BYTES // 2)
    for T, M in points:
        shape = base.with_(max_seq=T + M + 8, gamma_max=max(base.gamma_max, M - 1))
        o = ko.KangarooOracle(shape, w, np.float64)
        st = ki.microbench_state(shape, T, M - 1, seed)
        for i in range(shape.n_layers):
            o.cache[i].k[:T], o.cache[i].v[:T], o.cache[i].length = st["k"][i], st["v"][i], T
        feats = [st["feat"][1 + j].astype(np.float64) for j in range(M)]
        t, z = o._verify_tokens(feats, T)
        trace["points"].append({"T": T, "M": M, "target": [int(v) for v in t],
                                "rows": [row_record(z[i], idx) for i in range(M)]})
        print(f"[{name}] T={T} M={M} done ({time.time() - t0:.0f} s)", flush=True)
        del o, st
    return trace


CASES = {
    "13b_short": lambda: generation_case("13b_short", "13b", 40, 24, 0.6, 6, ko.STOP_KEEP),
    "33b_short": lambda: generation_case("33b_short", "33b", 44, 28, 0.6, 8, ko.STOP_KEEP),
    "7b_verify": lambda: verify_case("7b_verify", "7b", [(128, 1), (512, 4), (2048, 8), (4096, 7), (4096, 11)], 11),
    "7b_full": lambda: generation_case("7b_full", "7b", 512, 256, 0.6, 6, ko.STOP_KEEP),
}


def main():
    names = sys.argv[1:] or list(CASES)
    for n in names:
        tr = CASES[n]()
        path = os.path.join(HERE, f"trace_{n}.json")
        with open(path, "w") as f:
            json.dump(tr, f, separators=(",", ":"))
            f.write("\n")
        print(f"wrote {path}", flush=True)


if __name__ == "__main__":
    main()
