"""Closed forms and library special cases that pin the oracle's primitives."""
import math

import numpy as np
import pytest
import torch

from oracle import kangaroo_oracle as ko


def test_rmsnorm_closed_forms():
    g = np.array([1.0, 2.0, 3.0, 4.0])
    x = np.full(4, 5.0)                     # constant vector: x / sqrt(25 + eps) ~ 1
    y = ko.rmsnorm(x, g, 0.0)
    assert np.allclose(y, g)
    x = np.array([3.0, 4.0, 0.0, 0.0])      # mean square = 25/4
    assert np.allclose(ko.rmsnorm(x, np.ones(4), 0.0), x / 2.5)
    assert np.allclose(ko.rmsnorm(x, np.ones(4), 1.0), x / math.sqrt(25 / 4 + 1))
    # scale invariance (eps = 0) and per-row independence
    X = np.random.default_rng(0).normal(size=(3, 8))
    assert np.allclose(ko.rmsnorm(7.0 * X, np.ones(8), 0.0), ko.rmsnorm(X, np.ones(8), 0.0))
    assert np.allclose(ko.rmsnorm(X, np.ones(8), 1e-6)[1], ko.rmsnorm(X[1], np.ones(8), 1e-6))
    assert np.allclose(np.mean(ko.rmsnorm(X, np.ones(8), 0.0) ** 2, axis=-1), 1.0)


def test_rmsnorm_matches_torch():
    X = np.random.default_rng(1).normal(size=(4, 16))
    g = np.random.default_rng(2).normal(size=16)
    t = torch.nn.functional.rms_norm(torch.from_numpy(X), (16,), torch.from_numpy(g), eps=1e-6).numpy()
    assert np.allclose(ko.rmsnorm(X, g, 1e-6), t, atol=1e-12)


def test_rope_properties():
    rng = np.random.default_rng(3)
    x = rng.normal(size=(2, 8))
    assert np.array_equal(ko.rope(x, 0, 10000.0), x)                       # position 0 is the identity
    y = ko.rope(x, 5, 10000.0)
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1))   # rotations keep the norm
    assert np.allclose(ko.rope(ko.rope(x, 3, 10000.0), 4, 10000.0), ko.rope(x, 7, 10000.0))  # angles add
    # hand case: hd = 2, one pair, angle = pos * theta^0 = pos
    v = np.array([[1.0, 0.0]])
    assert np.allclose(ko.rope(v, 2, 10000.0), [[math.cos(2.0), math.sin(2.0)]])
    # pairing is (i, i + hd/2), frequency theta^(-2i/hd): hd = 4, pairs (0,2) and (1,3)
    v = np.array([[1.0, 1.0, 0.0, 0.0]])
    a1 = 3 * 10000.0 ** (-2 * 1 / 4)
    assert np.allclose(ko.rope(v, 3, 10000.0), [[math.cos(3.0), math.cos(a1), math.sin(3.0), math.sin(a1)]])
    # relative-position property: <rope(q,m), rope(k,n)> depends on m - n only
    q, k = rng.normal(size=(1, 8)), rng.normal(size=(1, 8))
    d1 = float(np.sum(ko.rope(q, 9, 1e4) * ko.rope(k, 4, 1e4)))
    d2 = float(np.sum(ko.rope(q, 25, 1e4) * ko.rope(k, 20, 1e4)))
    assert abs(d1 - d2) < 1e-12


def test_rope_matches_complex_rotation():
    rng = np.random.default_rng(4)
    hd, pos, theta = 16, 11, 10000.0
    x = rng.normal(size=(3, hd))
    zc = x[:, :hd // 2] + 1j * x[:, hd // 2:]
    ang = pos * theta ** (-2.0 * np.arange(hd // 2) / hd)
    r = zc * np.exp(1j * ang)
    assert np.allclose(ko.rope(x, pos, theta), np.concatenate([r.real, r.imag], -1))


def test_round_bf16_matches_torch():
    rng = np.random.default_rng(5)
    x = np.concatenate([rng.normal(size=1000), [1.00390625, 1.01171875, -1.00390625, 0.0, 3.0e38, 1e-40]]).astype(np.float32)
    t = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(ko.round_bf16(x), t)
    # ties go to even: 1 + 2^-8 is exactly between 1 and 1 + 2^-7
    assert ko.round_bf16(np.array([1.00390625], np.float32))[0] == 1.0
    assert ko.round_bf16(np.array([1.01171875], np.float32))[0] == np.float32(1.015625)


def test_silu_and_softmax():
    x = np.linspace(-6, 6, 25)
    assert np.allclose(ko.silu(x), torch.nn.functional.silu(torch.from_numpy(x)).numpy())
    assert ko.silu(np.array([0.0]))[0] == 0.0
    s = np.random.default_rng(6).normal(size=(3, 7))
    p = ko.softmax_rows(s)
    assert np.allclose(p.sum(-1), 1.0)
    assert np.allclose(p, torch.softmax(torch.from_numpy(s), -1).numpy())
    assert np.allclose(ko.softmax_rows(s + 100.0), p)


def test_confidence_closed_forms():
    V = 1024
    tok, p = ko.top1_confidence(np.zeros(V))
    assert tok == 0 and abs(p - 1.0 / V) < 1e-15             # uniform logits: p = 1/V, lowest index wins
    z = np.zeros(V); z[17] = 50.0
    tok, p = ko.top1_confidence(z)
    assert tok == 17 and 1 - p < 1e-15
    z = np.zeros(4); z[2] = math.log(3.0)                    # p = 3 / (3 + 3) = 0.5
    tok, p = ko.top1_confidence(z)
    assert tok == 2 and abs(p - 0.5) < 1e-15
    z = np.array([1.0, 5.0, 5.0, 2.0])                       # tie: lowest index
    assert ko.argmax_lowest(z) == 1
    assert ko.top2_gap(z) == 0.0
    assert ko.top2_gap(np.array([1.0, 4.0, 2.5])) == 1.5
    rng = np.random.default_rng(7)
    z = rng.normal(size=50) * 3
    tok, p = ko.top1_confidence(z)
    assert abs(p - float(torch.softmax(torch.from_numpy(z), 0).max())) < 1e-14
    assert 1.0 / 50 <= p <= 1.0


def test_metrics_eq1_eq2():
    S = [1, 3, 2, 7, 1, 4]
    g = 6
    assert ko.compression_rate(S) == 18 / 6                                   # Eq. 1; also N / |S|
    assert ko.ctar(S, 0) == 1.0 and ko.ctar(S, g + 1) == 0.0
    c = [ko.ctar(S, w) for w in range(0, g + 2)]
    assert all(c[i] >= c[i + 1] for i in range(len(c) - 1))                  # decreasing in w (Section 3)
    assert ko.ctar(S, 1) == 4 / 6 and ko.ctar(S, 3) == 2 / 6                 # Eq. 2 by hand
    assert abs(ko.compression_rate(S) - sum(c[: g + 1])) < 1e-12             # s_k = sum_w I(s_k > w)
