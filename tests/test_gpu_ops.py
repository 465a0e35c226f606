"""Single operators of the CUDA path against the oracle's definitions, element by element."""
import numpy as np
import pytest

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


# (N, K, M): ragged row counts per CTA, several chunks, K phases (M*K*4 > staging budget), tiny N
LIN_CASES = [(4096, 4096, 1), (4096, 4096, 7), (1000, 512, 3), (333, 96, 2), (12288, 4096, 8), (4096, 11008, 8),
             (4096, 11008, 11), (2048, 1376, 16), (64, 64, 1), (5000, 6656, 9)]


@pytest.mark.parametrize("N,K,M", LIN_CASES)
def test_linear_bf16_plain_norm_resid(env, N, K, M):
    torch, b = env
    W = _mat(1, 50, N, K, 0.02, True)
    x = _mat(2, 51, M, K, 1.0, False)
    gain = (1.0 + _mat(3, 52, 1, K, 0.1, False)[0]).astype(np.float32)
    resid = _mat(4, 53, M, N, 1.0, False)
    Wd, xd, gd, rd = _dev(torch, W, True), _dev(torch, x), _dev(torch, gain), _dev(torch, resid)
    scale = float(np.sqrt(K) * 0.02)                      # typical magnitude of an output
    y = b.op_linear(Wd, xd).cpu().numpy()
    assert np.max(np.abs(y - _lin_ref(x, W))) < 2e-4 * scale
    y = b.op_linear(Wd, xd, gain=gd, eps=1e-6, resid=rd).cpu().numpy()
    ref = resid + _lin_ref(ko.rmsnorm(x.astype(np.float64), gain.astype(np.float64), 1e-6), W)
    assert np.max(np.abs(y - ref)) < 2e-4 * scale


@pytest.mark.parametrize("F,K,M", [(11008, 4096, 1), (11008, 4096, 6), (1376, 512, 16), (100, 64, 3)])
def test_linear_swiglu(env, F, K, M):
    torch, b = env
    Wg, Wu = _mat(1, 60, F, K, 0.02, True), _mat(1, 61, F, K, 0.02, True)
    x = _mat(2, 62, M, K, 1.0, False)
    gain = (1.0 + _mat(3, 63, 1, K, 0.1, False)[0]).astype(np.float32)
    y = b.op_linear(_dev(torch, Wg, True), _dev(torch, x), gain=_dev(torch, gain), eps=1e-6, W2=_dev(torch, Wu, True)).cpu().numpy()
    n = ko.rmsnorm(x.astype(np.float64), gain.astype(np.float64), 1e-6)
    ref = ko.silu(_lin_ref(n, Wg)) * _lin_ref(n, Wu)
    assert np.max(np.abs(y - ref)) < 5e-4


@pytest.mark.parametrize("N,K,M", [(256, 256, 1), (688, 256, 5), (256, 688, 16), (1024, 256, 7)])
def test_linear_f32_weights(env, N, K, M):
    torch, b = env
    W = _mat(1, 70, N, K, 0.02, False)
    x = _mat(2, 71, M, K, 1.0, False)
    resid = _mat(4, 73, M, N, 1.0, False)
    y = b.op_linear(_dev(torch, W), _dev(torch, x), resid=_dev(torch, resid)).cpu().numpy()
    assert np.max(np.abs(y - (resid + _lin_ref(x, W)))) < 1e-4


@pytest.mark.parametrize("V,K,M,bf", [(32000, 4096, 1, True), (32000, 4096, 7, True), (1024, 256, 3, False), (2048, 512, 16, True), (50, 64, 2, True)])
def test_lm_head(env, V, K, M, bf):
    torch, b = env
    W = _mat(1, 80, V, K, 0.02, bf)
    x = _mat(2, 81, M, K, 1.0, False)
    gain = (1.0 + _mat(3, 82, 1, K, 0.1, False)[0]).astype(np.float32)
    s = 9.0
    tok, p, z = b.op_lm_head(_dev(torch, W, bf), _dev(torch, x), _dev(torch, gain), 1e-6, s)
    tok, p, z = tok.cpu().numpy(), p.cpu().numpy(), z.cpu().numpy()
    zr = s * _lin_ref(ko.rmsnorm(x.astype(np.float64), gain.astype(np.float64), 1e-6), W)
    assert np.max(np.abs(z - zr)) < 2e-3
    for m in range(M):
        t_ref, p_ref = ko.top1_confidence(zr[m])
        assert tok[m] == t_ref or ko.top2_gap(zr[m]) < 2e-2
        assert abs(p[m] - p_ref) < 1e-3
        assert tok[m] == int(np.argmax(z[m]))               # consistent with its own logits, lowest index on ties


def test_lm_head_tie_takes_lowest_index(env):
    torch, b = env
    V, K = 4096, 64
    W = np.zeros((V, K), np.float32)
    W[[7, 300, 4000], 0] = 1.0                              # three identical maximal rows
    x = np.zeros((2, K), np.float32); x[:, 0] = 1.0
    tok, p, z = b.op_lm_head(_dev(torch, W, True), _dev(torch, x), None, 0.0, 1.0)
    assert tok.cpu().tolist() == [7, 7]
    ref = 1.0 / (3.0 + (V - 3) * np.exp(-1.0))
    assert np.allclose(p.cpu().numpy(), ref, rtol=1e-5)


class _S:  # minimal shape for the oracle's attention
    pass


@pytest.mark.parametrize("H,hd,M,pos0,ps,bf", [(32, 128, 1, 512, 16, True), (32, 128, 7, 300, 16, True), (4, 64, 16, 0, 16, False),
                                               (4, 64, 5, 37, 8, False), (2, 32, 3, 150, 4, True), (40, 128, 9, 1000, 16, True)])
def test_attention(env, H, hd, M, pos0, ps, bf):
    torch, b = env
    d = H * hd
    T = pos0 + M
    n_pages = (T + ps - 1) // ps + 2
    sh = _S()
    sh.n_layers, sh.exit_layer, sh.d_model, sh.n_heads, sh.head_dim = 2, 1, d, H, hd
    sh.rope_theta, sh.dtype, sh.max_seq = 10000.0, "bf16" if bf else "f32", T + 1
    o = ko.KangarooOracle.__new__(ko.KangarooOracle)
    o.s, o.dt, o.d, o.H, o.hd = sh, np.dtype(np.float64), d, H, hd
    cache = ko.KVCache(T + 1, H, hd, np.float64, bf)
    kpast = _mat(5, 90, pos0, d, 1.0, bf).reshape(pos0, H, hd)
    vpast = _mat(5, 91, pos0, d, 1.0, bf).reshape(pos0, H, hd)
    cache.k[:pos0], cache.v[:pos0], cache.length = kpast, vpast, pos0
    qkv = _mat(6, 92, M, 3 * d, 1.0, False)
    ref = o.attention_core(qkv.astype(np.float64), pos0, cache)
    # device cache [page][head][slot][hd] with a permuted page table
    perm = np.random.default_rng(0).permutation(n_pages).astype(np.int32)
    kc = np.zeros((n_pages, H, ps, hd), np.float32)
    vc = np.zeros((n_pages, H, ps, hd), np.float32)
    for pos in range(pos0):
        kc[perm[pos // ps], :, pos % ps, :] = kpast[pos]
        vc[perm[pos // ps], :, pos % ps, :] = vpast[pos]
    kcd, vcd = _dev(torch, kc, bf), _dev(torch, vc, bf)
    out = b.op_attention(_dev(torch, qkv), pos0, H, hd, 10000.0, kcd, vcd, _dev(torch, perm), ps).cpu().numpy()
    assert np.max(np.abs(out - ref)) < 2e-3
    # the new rows were appended to the cache, rotated and rounded like the oracle's
    kcn, vcn = kcd.float().cpu().numpy(), vcd.float().cpu().numpy()
    for i in range(M):
        pos = pos0 + i
        kk, vv = kcn[perm[pos // ps], :, pos % ps, :], vcn[perm[pos // ps], :, pos % ps, :]
        tol = 0.05 if bf else 1e-5                       # one bf16 ulp at |k| ~ 4
        assert np.max(np.abs(kk - cache.k[pos])) < tol and np.max(np.abs(vv - cache.v[pos])) < tol
        if bf:                                           # identical bf16 values except where rounding flipped
            assert np.mean(kk == cache.k[pos].astype(np.float32)) > 0.98
