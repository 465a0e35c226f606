"""The oracle's model path pinned against (a) a brute-force full-sequence recompute, (b) an
independent torch CPU composition of the same decoder, and (c) the paper's invariants:
greedy Kangaroo == plain greedy decoding (lossless), 1..gamma+1 tokens per round, eta = 0
drafts gamma, eta > 1 drafts none (or one, when the stopped token is kept)."""
import numpy as np
import pytest
import torch

import kg_inputs as ki
from oracle import kangaroo_oracle as ko

MICRO = ki.KgShape("micro", 2, 64, 2, 32, 96, 128, 1, "f32", logit_scale=12.0, max_seq=96,
                   gamma_max=6, gain_std=0.2, deep_resid_scale=0.3, adapter_resid_scale=0.3,
                   n_prompt=9, n_gen=24)
MICRO_BF = MICRO.with_(name="micro_bf", dtype="bf16", seed=3)
TINY = ki.get_config("tiny")
TINY_G = TINY.with_(gain_std=0.2, seed=1)


def build(shape, dtype=np.float64):
    w = ki.make_weights(shape)
    return ko.KangarooOracle(shape, w, dtype), w


# ---------------------------------------------------------------- independent torch composition

def torch_forward(shape, w, tokens, adapter=False):
    """LLaMA-style forward written directly on torch CPU float64 ops (matmul, softmax, silu).
    Returns target logits [T, V] (adapter=False) or draft logits [T, V] (adapter=True)."""
    T = len(tokens)
    d, H, hd = shape.d_model, shape.n_heads, shape.head_dim
    tt = lambda a: torch.from_numpy(np.asarray(a)).double()

    def norm(x, g):
        return x * torch.rsqrt((x * x).mean(-1, keepdim=True) + shape.rms_eps) * tt(g)

    def rot(x):                                   # x [T, H, hd] -> rotate via complex multiplication
        half = hd // 2
        freqs = shape.rope_theta ** (-torch.arange(0, half).double() * 2.0 / hd)
        ang = torch.arange(T).double()[:, None] * freqs[None]          # [T, half]
        z = torch.complex(x[..., :half], x[..., half:]) * torch.polar(torch.ones_like(ang), ang)[:, None, :]
        return torch.cat([z.real, z.imag], -1)

    def quant(x):
        return x.float().bfloat16().double() if shape.dtype == "bf16" else x

    def attn(x, wqkv, wo):
        qkv = x @ tt(wqkv).T
        q, k, v = [qkv[:, i * d:(i + 1) * d].reshape(T, H, hd) for i in range(3)]
        q, k, v = rot(q), quant(rot(k)), quant(v)
        sc = torch.einsum("qhe,khe->hqk", q, k) / hd ** 0.5
        sc = sc.masked_fill(torch.ones(T, T).triu(1).bool()[None], float("-inf"))
        o = torch.einsum("hqk,khe->qhe", torch.softmax(sc, -1), v).reshape(T, d)
        return o @ tt(wo).T

    def block(h, lw):
        h = h + attn(norm(h, lw["g1"]), lw["wqkv"], lw["wo"])
        n = norm(h, lw["g2"])
        return h + (torch.nn.functional.silu(n @ tt(lw["wgate"]).T) * (n @ tt(lw["wup"]).T)) @ tt(lw["wdown"]).T

    h = tt(w["embed"])[torch.tensor(tokens)]
    n_l = shape.exit_layer if adapter else shape.n_layers
    for i in range(n_l):
        h = block(h, w["layers"][i])
    if adapter:
        a = h + attn(norm(h, w["adapter"]["g_in"]), w["adapter"]["wqkv"], w["adapter"]["wo"])
        y = norm(a, w["adapter"]["g_last"])
    else:
        y = norm(h, w["g_final"])
    return (y @ tt(w["head"]).T * shape.logit_scale).numpy()


@pytest.mark.parametrize("shape", [MICRO, MICRO_BF, TINY_G])
def test_cached_forward_matches_torch_and_bruteforce(shape):
    o, w = build(shape)
    prompt = ki.make_prompt(shape, 7).tolist()
    toks = o.generate_ar(prompt, 6)
    seq = prompt + toks
    # logits of every AR step, collected again step by step
    o.reset()
    o.prefill(prompt)
    step_logits = [o.last_logits]
    for _ in range(5):
        o.ar_step()
        step_logits.append(o.last_logits)
    ref_t = torch_forward(shape, w, seq[:-1])
    ref_b = o.full_recompute_logits(seq[:-1])
    # the references round K/V to bf16 at the same point (after the rotation), so fp64 summation order is the only
    # difference; a forgotten rounding, or one applied before the rotation, moves logits by ~1e-2 and fails here
    tol = 1e-9
    for i, z in enumerate(step_logits):
        row = len(prompt) - 1 + i
        assert np.max(np.abs(z - ref_t[row])) < tol, (i, np.max(np.abs(z - ref_t[row])))
        assert np.max(np.abs(z - ref_b[row])) < tol
        assert int(np.argmax(ref_t[row])) == toks[i] or ko.top2_gap(ref_t[row]) < 2 * tol
    if shape.dtype == "f32":
        assert [int(np.argmax(ref_b[len(prompt) - 1 + i])) for i in range(6)] == toks


def test_draft_logits_match_torch():
    """The adapter + shared head path (M^s = A o M^b[:l]) against the torch composition."""
    shape = MICRO
    o, w = build(shape)
    prompt = ki.make_prompt(shape, 8).tolist()
    o.prefill(prompt)
    o.round(0.0, 4, ko.STOP_KEEP)                     # eta = 0: four draft steps from x_0
    r = o.log[-1]
    seq = prompt + [o.tokens[len(prompt)]] + r["drafts"]
    ref = torch_forward(shape, w, seq, adapter=True)
    for j, z in enumerate(r["draft_logits"]):
        assert np.max(np.abs(z - ref[len(prompt) + j])) < 1e-9
    reft = torch_forward(shape, w, seq)
    for j in range(r["M"]):
        assert np.max(np.abs(r["verify_logits"][j] - reft[len(prompt) + j])) < 1e-9


GRID = [(eta, gamma, mode) for eta in (0.0, 0.3, 0.6, 0.9, 1.5) for gamma in (1, 2, 6) for mode in (ko.STOP_KEEP, ko.STOP_DROP)]


@pytest.mark.parametrize("shape", [MICRO, MICRO_BF, TINY])
def test_lossless_and_invariants(shape):
    o, w = build(shape)
    prompt = ki.make_prompt(shape).tolist()
    n = shape.n_gen if shape.name != "tiny" else 40
    ar = o.generate_ar(prompt, n)
    for eta, gamma, mode in GRID:
        kg = o.generate(prompt, n, eta, gamma, mode)
        assert kg == ar, (eta, gamma, mode)                                    # lossless (title; Section 3)
        assert sum(o.S) == n - 1
        for r in o.log:
            assert 1 <= r["k"] + 1 <= gamma + 1                                # Section 1: 1 .. gamma+1 tokens
            assert r["n_drafted"] <= gamma and r["n_steps"] <= gamma
            assert r["M"] == r["n_drafted"] + 1
            assert all(1.0 / shape.vocab <= p <= 1.0 for p in r["conf"])
            if eta == 0.0:
                assert r["n_drafted"] == gamma                                 # fixed-step drafting
            if eta > 1.0:
                assert r["n_drafted"] == (1 if mode == ko.STOP_KEEP else 0)
            if r["k"] < r["n_drafted"]:
                assert r["drafts"][r["k"]] != r["target"][r["k"]]
            assert r["adapter_len_after"] in (r["P"] + r["k"] + 1, r["P"] + r["k"])
        cr = ko.compression_rate(o.S)
        assert abs(cr - (n - 1) / len(o.S)) < 1e-12
        assert abs(cr - sum(ko.ctar(o.S, w_) for w_ in range(gamma + 1))) < 1e-12


def test_prefix_nesting_in_eta():
    """From the same state a lower threshold drafts a superset prefix, so it accepts at least as many."""
    shape = TINY
    o, w = build(shape)
    prompt = ki.make_prompt(shape).tolist()
    for mode in (ko.STOP_KEEP, ko.STOP_DROP):
        res = {}
        for eta in (0.0, 0.4, 0.8):
            o.reset(); o.prefill(prompt)
            o.round(eta, 6, mode)
            res[eta] = o.log[-1]
        for a, b in ((0.0, 0.4), (0.4, 0.8)):
            da, db = res[a]["drafts"], res[b]["drafts"]
            assert da[: len(db)] == db
            assert res[a]["k"] >= res[b]["k"]


def test_rollback_equals_fresh_prefill():
    """After a round (with rejected drafts), continuing must equal a fresh prefill of the accepted prefix."""
    shape = TINY
    o, w = build(shape)
    prompt = ki.make_prompt(shape).tolist()
    o.prefill(prompt)
    seen_reject = seen_all = False
    gammas = [1, 4, 2, 1, 3, 1, 4, 2, 1, 1, 2, 4, 1, 1]
    for it in range(len(gammas) - 1):
        o.round(0.0, gammas[it], ko.STOP_KEEP)
        r = o.log[-1]
        seen_reject |= r["k"] < r["n_drafted"]
        seen_all |= r["k"] == r["n_drafted"]
        g_next = gammas[it + 1]
        prefix = o.tokens[:-1]                      # everything before the current x_0
        o2 = ko.KangarooOracle(shape, w)
        assert o2.prefill(prefix) == o.x0
        nxt = o2.round(0.0, g_next, ko.STOP_KEEP)
        # o's own next round, replayed on a copy so the loop is not disturbed
        o3 = ko.KangarooOracle(shape, w)
        o3.prefill(prompt)
        for j in range(it + 1):
            o3.round(0.0, gammas[j], ko.STOP_KEEP)
        assert o3.tokens == o.tokens
        assert o3.round(0.0, g_next, ko.STOP_KEEP) == nxt
        assert o3.log[-1]["drafts"] == o2.log[-1]["drafts"]
        assert np.allclose(o3.log[-1]["conf"], o2.log[-1]["conf"], atol=1e-9)
    assert seen_reject and seen_all


def test_fp32_oracle_agrees_with_fp64():
    shape = TINY
    o64, w = build(shape)
    o32 = ko.KangarooOracle(shape, w, np.float32)
    prompt = ki.make_prompt(shape).tolist()
    a = o64.generate(prompt, 32, 0.6, 6)
    b = o32.generate(prompt, 32, 0.6, 6)
    assert a == b and o64.S == o32.S
    for r64, r32 in zip(o64.log, o32.log):
        assert np.allclose(r64["conf"], r32["conf"], atol=1e-4)
        assert np.max(np.abs(r64["verify_logits"] - r32["verify_logits"])) < 1e-3


def test_workload_calibration_recorded_range():
    """Not a property of the method: the synthetic tiny model should exercise both accepts and
    rejects and a wide confidence range at the paper's eta = 0.6, gamma = 6 (parity unpinned by the paper)."""
    shape = TINY
    o, w = build(shape)
    prompt = ki.make_prompt(shape).tolist()
    o.generate(prompt, shape.n_gen, shape.eta, shape.gamma)
    conf = [p for r in o.log for p in r["conf"]]
    assert min(conf) < 0.35 and max(conf) > 0.9
    ks = [r["k"] for r in o.log]
    assert any(r["k"] < r["n_drafted"] for r in o.log) and any(r["k"] == r["n_drafted"] for r in o.log)
    assert 1.2 < ko.compression_rate(o.S) < 4.0


# ---------------------------------------------------------------- where K and V are rounded for bf16 models

def _bf16_by_hand(x: float) -> float:
    """Nearest-even rounding of a Python float to bfloat16, on the bits of its fp32 value."""
    import struct
    bits = struct.unpack("<I", struct.pack("<f", x))[0]
    bits = (bits + 0x7FFF + ((bits >> 16) & 1)) & 0xFFFF0000
    return struct.unpack("<f", struct.pack("<I", bits))[0]


def test_kv_cache_stores_bf16_of_rotated_k_and_of_v():
    """bf16 models keep K and V in bf16: K is rotated first and rounded when stored, V is rounded when stored, and
    nothing else is rounded.  Two heads of four dimensions, position 3, every value worked out with scalar
    arithmetic; the inputs are chosen so that leaving the rounding out, or rounding K before the rotation, gives
    different stored values."""
    import math
    H, hd, d, pos, theta = 2, 4, 8, 3, 10000.0
    shape = MICRO_BF.with_(d_model=d, n_heads=H, head_dim=hd, max_seq=8, rope_theta=theta)
    o = ko.KangarooOracle.__new__(ko.KangarooOracle)
    o.s, o.dt, o.d, o.H, o.hd = shape, np.dtype(np.float64), d, H, hd
    cache = ko.KVCache(8, H, hd, np.float64, True)
    cache.length = pos                                    # rows 0..2 stay zero: they only add exp(0) terms below
    q = [0.3, -1.1, 0.7, 0.2, -0.4, 0.9, 1.3, -0.6]
    k = [1.2345678, -0.7654321, 2.3456789, 0.1234567, -1.1111111, 0.3333333, 0.9876543, -2.2222222]
    v = [0.1111111, 1.7777777, -0.5555555, 3.1415926, -2.7182818, 0.5772156, 1.4142135, -1.7320508]
    qkv = np.array([q + k + v], np.float64)
    out = o.attention_core(qkv, pos, cache)
    assert cache.length == pos + 1

    def rot(x, h):                                        # pairs (i, i + hd/2), angle pos * theta^(-2i/hd)
        r = [0.0] * hd
        for i in range(hd // 2):
            a = pos * theta ** (-2.0 * i / hd)
            x1, x2 = x[h * hd + i], x[h * hd + i + hd // 2]
            r[i] = x1 * math.cos(a) - x2 * math.sin(a)
            r[i + hd // 2] = x2 * math.cos(a) + x1 * math.sin(a)
        return r

    k_rot = [rot(k, h) for h in range(H)]
    k_exp = [[_bf16_by_hand(x) for x in k_rot[h]] for h in range(H)]
    v_exp = [[_bf16_by_hand(v[h * hd + e]) for e in range(hd)] for h in range(H)]
    assert np.array_equal(cache.k[pos], np.array(k_exp)) and np.array_equal(cache.v[pos], np.array(v_exp))
    # the two plausible mistakes give other values on this input
    k_unrounded = np.array(k_rot)
    k_round_first = np.array([rot([_bf16_by_hand(x) for x in k], h) for h in range(H)])
    assert not np.array_equal(cache.k[pos], k_unrounded) and np.max(np.abs(cache.k[pos] - k_unrounded)) > 1e-4
    assert np.max(np.abs(cache.k[pos] - k_round_first)) > 1e-4
    assert np.max(np.abs(cache.v[pos] - np.array(v).reshape(H, hd))) > 1e-4
    # and the attention output uses the stored (rounded) row: softmax over three zero keys and the new key
    for h in range(H):
        qr = rot(q, h)
        s_new = sum(a * b for a, b in zip(qr, k_exp[h])) / math.sqrt(hd)
        w_new = math.exp(s_new) / (3.0 + math.exp(s_new))
        for e in range(hd):
            assert abs(out[0, h * hd + e] - w_new * v_exp[h][e]) < 1e-12
