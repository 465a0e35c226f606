"""Round-by-round lockstep comparison of the CUDA path (through the C ABI) with the CPU oracle.

Token ids and accept lengths must agree exactly; logits within LOGIT_TOL, confidences within
CONF_TOL.  A decision may differ only where the oracle itself is nearly tied (top-2 logit gap
below LOGIT_TOL, or a confidence within CONF_TOL of eta); such positions are logged and the
oracle is re-seeded from the CUDA path's prefix so that the comparison can continue."""
import numpy as np

from oracle import kangaroo_oracle as ko

LOGIT_TOL = 2e-2
CONF_TOL = 1e-3


class Mismatch(AssertionError):
    pass


def _resync(o, prompt, gpu_tokens):
    """Fresh oracle state holding prompt + gpu_tokens[:-1], with x_0 := gpu_tokens[-1]."""
    o.reset()
    o.prefill(list(prompt) + list(gpu_tokens[:-1]))
    o.x0 = int(gpu_tokens[-1])
    o.tokens[-1] = o.x0


def lockstep(g, o, prompt, n_new, eta, gamma, mode, check_logits=True, conf_tol=CONF_TOL):
    """g: binding.KangarooModel (debug_logits on when check_logits), o: KangarooOracle.
    Returns dict(tokens, S, flips, max_logit_err, max_conf_err)."""
    flips = []
    max_le = 0.0
    max_ce = 0.0
    g.reset()
    o.reset()
    x0g = g.prefill(prompt)
    x0o = o.prefill(prompt)
    if check_logits:
        err = float(np.max(np.abs(g.debug_logits(1, 0).astype(np.float64) - o.last_logits)))
        max_le = max(max_le, err)
        if err > LOGIT_TOL:
            raise Mismatch(f"prefill logits differ by {err}")
    out = [x0g]
    if x0g != x0o:
        if ko.top2_gap(o.last_logits) >= LOGIT_TOL:
            raise Mismatch(f"x_0 differs: {x0g} vs {x0o}")
        flips.append(("prefill", len(prompt) - 1))
        _resync(o, prompt, out)
    S = []
    while len(out) < n_new:
        d = g.draft(eta, gamma, mode)
        v = g.verify()
        o.round(eta, gamma, mode)
        r = o.log[-1]
        ok = True
        why = None
        # drafts
        nst = min(d["n_steps"], r["n_steps"])
        for j in range(nst):
            if check_logits:
                err = float(np.max(np.abs(g.debug_logits(0, j).astype(np.float64) - r["draft_logits"][j])))
                max_le = max(max_le, err)
                if err > LOGIT_TOL:
                    raise Mismatch(f"draft logits step {j} differ by {err}")
            ce = abs(d["conf"][j] - r["conf"][j])
            max_ce = max(max_ce, ce)
            if ce > conf_tol:
                raise Mismatch(f"confidence step {j}: {d['conf'][j]} vs {r['conf'][j]}")
            tg = d["tokens"][j] if j < len(d["tokens"]) else None
            to = r["drafts"][j] if j < len(r["drafts"]) else None
            if tg != to:
                near_tie = ko.top2_gap(r["draft_logits"][j]) < LOGIT_TOL
                near_eta = abs(r["conf"][j] - eta) < conf_tol
                if not (near_tie or near_eta):
                    raise Mismatch(f"draft token step {j}: {tg} vs {to}")
                ok, why = False, ("draft", r["P"] + j)
                break
        if ok and (d["n_steps"] != r["n_steps"] or d["n_drafted"] != r["n_drafted"]):
            near_eta = any(abs(p - eta) < conf_tol for p in r["conf"])
            if not near_eta:
                raise Mismatch(f"draft counts differ: {d} vs n_d={r['n_drafted']} steps={r['n_steps']}")
            ok, why = False, ("eta", r["P"])
        if ok:
            for i in range(r["M"]):
                if check_logits:
                    err = float(np.max(np.abs(g.debug_logits(1, i).astype(np.float64) - r["verify_logits"][i])))
                    max_le = max(max_le, err)
                    if err > LOGIT_TOL:
                        raise Mismatch(f"verify logits row {i} differ by {err}")
                if v["target"][i] != r["target"][i]:
                    if ko.top2_gap(r["verify_logits"][i]) >= LOGIT_TOL:
                        raise Mismatch(f"target token row {i}: {v['target'][i]} vs {r['target'][i]}")
                    ok, why = False, ("verify", r["P"] + i)
                    break
        if ok:
            if v["k"] != r["k"] or v["emitted"] != r["emitted"] or v["n_rows"] != r["M"]:
                raise Mismatch(f"accept differs: {v} vs k={r['k']} emitted={r['emitted']}")
        out.extend(v["emitted"])
        S.append(len(v["emitted"]))
        if not ok:
            flips.append(why)
            _resync(o, prompt, out)
    return dict(tokens=out, S=S, flips=flips, max_logit_err=max_le, max_conf_err=max_ce)
