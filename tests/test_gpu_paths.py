"""Kernel paths and host branches that the other GPU tests do not reach, each against the oracle element by
element: attention with many KV splits, the 33B head count and the longest KV lengths; linear operators whose
CTAs own more accumulator rows than fit in shared memory at once (several superchunks, the LM head's merge across
them); a model built on borrowed caller weights; the device-side check of prompt ids; the bounded device waits."""
import numpy as np
import pytest

import kg_inputs as ki
from kg_inputs import synth
from oracle import kangaroo_oracle as ko

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    import __graft_entry__ as ge
    ge.build()
    from paper_2404_18911_b200 import binding as b
    b.load()
    return torch, b


def _mat(seed, tid, r, c, std, bf16):
    return synth.fill_f32(seed, tid, r * c, std, bf16).reshape(r, c)


def _dev(torch, a, bf16=False):
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(torch.bfloat16) if bf16 else t


def _lin_ref(x, W):
    return x.astype(np.float64) @ W.astype(np.float64).T


# ---- attention: few heads and long KV (many splits per head), 52 heads (the 33B shape), KV 2048 / 4096 ----------

class _S:
    pass


@pytest.mark.parametrize("H,hd,M,pos0,ps", [(4, 64, 1, 600, 16), (4, 64, 7, 1500, 16), (2, 128, 16, 900, 8),
                                            (52, 128, 9, 4100, 16), (32, 128, 1, 2048, 16), (32, 128, 5, 4096, 16),
                                            (32, 128, 11, 4090, 16), (32, 128, 1, 0, 16), (32, 128, 16, 0, 16)])
def test_attention_many_splits_and_long_kv(env, H, hd, M, pos0, ps):
    torch, b = env
    d, T = H * hd, pos0 + M
    n_pages = (T + ps - 1) // ps + 2
    sh = _S()
    sh.rope_theta, sh.dtype = 10000.0, "bf16"
    o = ko.KangarooOracle.__new__(ko.KangarooOracle)
    o.s, o.dt, o.d, o.H, o.hd = sh, np.dtype(np.float64), d, H, hd
    cache = ko.KVCache(T + 1, H, hd, np.float64, True)
    kpast = _mat(5, 90, max(pos0, 1), d, 1.0, True)[:pos0].reshape(pos0, H, hd)
    vpast = _mat(5, 91, max(pos0, 1), d, 1.0, True)[:pos0].reshape(pos0, H, hd)
    cache.k[:pos0], cache.v[:pos0], cache.length = kpast, vpast, pos0
    qkv = _mat(6, 92, M, 3 * d, 1.0, False)
    ref = o.attention_core(qkv.astype(np.float64), pos0, cache)
    perm = np.random.default_rng(1).permutation(n_pages).astype(np.int32)
    kc = np.zeros((n_pages, H, ps, hd), np.float32)
    vc = np.zeros((n_pages, H, ps, hd), np.float32)
    pg, sl = perm[np.arange(pos0) // ps], np.arange(pos0) % ps
    kc[pg, :, sl, :] = kpast
    vc[pg, :, sl, :] = vpast
    kcd, vcd = _dev(torch, kc, True), _dev(torch, vc, True)
    out = b.op_attention(_dev(torch, qkv), pos0, H, hd, 10000.0, kcd, vcd, _dev(torch, perm), ps).cpu().numpy()
    assert np.max(np.abs(out - ref)) < 2e-3, float(np.max(np.abs(out - ref)))
    # a second call on the same scratch gives the same bits (fixed merge order, counters left clean)
    kcd2, vcd2 = _dev(torch, kc, True), _dev(torch, vc, True)
    out2 = b.op_attention(_dev(torch, qkv), pos0, H, hd, 10000.0, kcd2, vcd2, _dev(torch, perm), ps).cpu().numpy()
    assert np.array_equal(out, out2)


# ---- linear operators with more than 256 accumulator rows per CTA ----------------------------------------------

@pytest.mark.parametrize("M", [1, 7, 12])
def test_linear_and_head_with_several_superchunks(env, M):
    torch, b = env
    N, K, F = 40000, 512, 20000
    W = _mat(1, 50, N, K, 0.02, True)
    x = _mat(2, 51, M, K, 1.0, False)
    gain = (1.0 + _mat(3, 52, 1, K, 0.1, False)[0]).astype(np.float32)
    resid = _mat(4, 53, M, N, 1.0, False)
    Wd, xd, gd = _dev(torch, W, True), _dev(torch, x), _dev(torch, gain)
    n = ko.rmsnorm(x.astype(np.float64), gain.astype(np.float64), 1e-6)
    scale = float(np.sqrt(K) * 0.02)
    y = b.op_linear(Wd, xd, gain=gd, eps=1e-6, resid=_dev(torch, resid)).cpu().numpy()
    assert np.max(np.abs(y - (resid + _lin_ref(n, W)))) < 2e-4 * scale
    # SwiGLU pair: 20000 features = 136 feature pairs per CTA, above the 128 that fit at once
    Wg, Wu = W[:F], W[F:2 * F]
    y = b.op_linear(_dev(torch, Wg, True), xd, gain=gd, eps=1e-6, W2=_dev(torch, Wu, True)).cpu().numpy()
    assert np.max(np.abs(y - ko.silu(_lin_ref(n, Wg)) * _lin_ref(n, Wu))) < 5e-4
    # LM head: the running (max, sum, arg max) is merged across a CTA's superchunks
    s = 9.0
    tok, p, z = b.op_lm_head(Wd, xd, gd, 1e-6, s)
    tok, p, z = tok.cpu().numpy(), p.cpu().numpy(), z.cpu().numpy()
    zr = s * _lin_ref(n, W)
    assert np.max(np.abs(z - zr)) < 2e-3
    for m in range(M):
        t_ref, p_ref = ko.top1_confidence(zr[m])
        assert tok[m] == t_ref or ko.top2_gap(zr[m]) < 2e-2
        assert abs(p[m] - p_ref) < 1e-3
        assert tok[m] == int(np.argmax(z[m]))


# ---- a model on borrowed caller weights -------------------------------------------------------------------------

def test_lockstep_parity_on_borrowed_weights(env):
    from parity_harness import lockstep
    from test_gpu_parity import SMALL_BF
    torch, b = env
    shape = SMALL_BF
    w = ki.make_weights(shape)
    g = b.KangarooModel(shape, debug_logits=True, weights=w)
    o = ko.KangarooOracle(shape, w, np.float64)
    prompt = ki.make_prompt(shape).tolist()
    res = lockstep(g, o, prompt, shape.n_gen, shape.eta, shape.gamma, 0)
    print("flips:", res["flips"], "max logit err", res["max_logit_err"], "max conf err", res["max_conf_err"])
    assert len(res["flips"]) <= 2, res["flips"]
    assert res["max_logit_err"] < 2e-2 and res["max_conf_err"] < 1e-3
    # the same tokens as the model that generated its own weights from the same seed
    g2 = b.KangarooModel(shape)
    t2, _ = g2.generate(prompt, shape.n_gen, shape.eta, shape.gamma)
    t1, _ = g.generate(prompt, shape.n_gen, shape.eta, shape.gamma)
    assert t1 == t2


# ---- prompt ids that arrive in device memory --------------------------------------------------------------------

def test_out_of_range_device_prompt_is_an_error_not_a_fault(env):
    torch, b = env
    shape = ki.get_config("tiny")
    g = b.KangarooModel(shape)
    prompt = ki.make_prompt(shape).tolist()
    ref, _ = g.generate(prompt, 16, shape.eta, shape.gamma)
    for bad_id in (shape.vocab, -1, 2 ** 31 - 1):
        bad = list(prompt)
        bad[5] = bad_id
        g.reset()
        g.prefill_device(torch.tensor(bad, dtype=torch.int32, device="cuda"))
        with pytest.raises(b.KgError) as e:
            g.read_tokens()
        assert e.value.status == b.KG_E_ARG
        torch.cuda.synchronize()                            # the context is intact
        with pytest.raises(b.KgError) as e:
            g.draft(shape.eta, shape.gamma)
        assert e.value.status == b.KG_E_STATE               # the sequence must be reset first
    toks, _ = g.generate(prompt, 16, shape.eta, shape.gamma)
    assert toks == ref


# ---- bounded device waits ---------------------------------------------------------------------------------------

def test_expired_device_wait_returns_timeout_and_leaves_the_context_usable(env):
    """One CTA leaves out a grid-barrier arrival (host-set test hook), so every CTA's wait runs into a budget of a
    few milliseconds: the launch ends by itself, the call reports KG_E_TIMEOUT, the model stays refused, and a
    model re-initialised in the same arena passes the lock-step comparison with the oracle."""
    import time
    from parity_harness import lockstep
    torch, b = env
    shape = ki.get_config("tiny")
    prompt = ki.make_prompt(shape).tolist()
    g = b.KangarooModel(shape, debug_logits=True)
    g.prefill(prompt)
    g.set_wait_budget(5.0)
    g.skip_barrier_arrival(1)
    t0 = time.time()
    with pytest.raises(b.KgError) as e:
        g.draft(shape.eta, shape.gamma)
    assert e.value.status == b.KG_E_TIMEOUT
    assert "timed out" in str(e.value)
    torch.cuda.synchronize()                                # every CTA has left; the stream answers
    assert time.time() - t0 < 5.0
    for call in (lambda: g.verify(), lambda: g.draft(0.6, 6), lambda: g.reset(), lambda: g.prefill(prompt)):
        with pytest.raises(b.KgError) as e:
            call()
        assert e.value.status == b.KG_E_TIMEOUT             # refused on the host, nothing launched
    arena = g.arena
    g.close()
    g2 = b.KangarooModel(shape, debug_logits=True, arena=arena)
    o = ko.KangarooOracle(shape, ki.make_weights(shape), np.float64)
    res = lockstep(g2, o, prompt, 24, shape.eta, shape.gamma, 0)
    assert not res["flips"] and res["max_logit_err"] < 2e-2
    # the streamed (bf16) path: the producer warp and the weight ring leave their waits too
    from test_gpu_parity import SMALL_BF
    gb = b.KangarooModel(SMALL_BF)
    pb = ki.make_prompt(SMALL_BF).tolist()
    ref, _ = gb.generate(pb, 16, 0.6, 6)
    gb.reset()
    gb.prefill(pb)
    gb.set_wait_budget(5.0)
    gb.skip_barrier_arrival(3)
    with pytest.raises(b.KgError) as e:
        gb.decode(16, 0.6, 6)
    assert e.value.status == b.KG_E_TIMEOUT
    torch.cuda.synchronize()
    gb2 = b.KangarooModel(SMALL_BF, arena=gb.arena)
    toks, _ = gb2.generate(pb, 16, 0.6, 6)
    assert toks == ref
