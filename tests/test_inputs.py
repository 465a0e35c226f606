"""The seeded input generator: determinism, bit-identity of its implementations, distribution,
and the closed-form parameter counts the paper quotes (Table 2; abstract)."""
import numpy as np
import pytest

import kg_inputs as ki
from kg_inputs import synth


def test_splitmix64_published_vector():
    # First outputs of the SplitMix64 stream started from state 0 (widely published test vector).
    s, out = 0, []
    for _ in range(3):
        out.append(synth.splitmix64(s))
        s = (s + 0x9E3779B97F4A7C15) & ((1 << 64) - 1)
    assert out == [0xE220A8397B1DCDAF, 0x6E789E6AA1B965F4, 0x06C45D188009454F]


def test_scalar_and_vector_mix_agree():
    xs = [0, 1, 2**63, 2**64 - 1, 123456789]
    v = synth.splitmix64(np.array(xs, dtype=np.uint64))
    assert [int(a) for a in v] == [synth.splitmix64(x) for x in xs]


def test_gauss_ints_definition():
    seed, tid = 7, 42
    base = synth.stream_base(seed, tid)
    g = synth.gauss_ints(seed, tid, 5, 4)
    for j in range(4):
        u = synth.splitmix64((base + 5 + j) & (2**64 - 1))
        assert int(g[j]) == sum((u >> (8 * b)) & 0xFF for b in range(8)) - 1020


def test_distribution_and_range():
    x = synth.gauss_f32(0, 9, 0, 1 << 20, 0.02)
    assert abs(float(x.mean())) < 1e-4
    assert abs(float(x.std()) - 0.02) < 2e-4
    assert float(np.abs(x).max()) <= 1020 * float(synth.scale_f32(0.02)) + 1e-9
    kurt = float(((x / x.std()) ** 4).mean())
    assert 2.7 < kurt < 3.0           # Irwin-Hall(8): 3 - 1.2/8


def test_c_fill_matches_numpy_bitwise():
    if not synth._load_fill_lib():
        pytest.skip("libkg_inputs_fill.so not built")
    for bf in (False, True):
        a = synth.fill_f32(3, 17, 100003, 0.02, bf)
        b = synth.fill_f32(3, 17, 100003, 0.02, bf, force_numpy=True)
        assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


def test_bf16_values_are_representable_and_nearest():
    import torch
    x = synth.gauss_f32(1, 2, 0, 4096, 0.02)
    r = synth.round_to_bf16_f32(x)
    assert np.all((r.view(np.uint32) & 0xFFFF) == 0)
    t = torch.from_numpy(x.copy()).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(t, r)


def test_streams_differ_and_are_deterministic():
    a = synth.gauss_ints(0, 100, 0, 64)
    assert np.array_equal(a, synth.gauss_ints(0, 100, 0, 64))
    assert not np.array_equal(a, synth.gauss_ints(0, 101, 0, 64))
    assert not np.array_equal(a, synth.gauss_ints(1, 100, 0, 64))
    assert np.array_equal(synth.gauss_ints(0, 100, 10, 20), synth.gauss_ints(0, 100, 0, 64)[10:30])


def test_prompt_tokens():
    c = ki.get_config("tiny")
    p = ki.make_prompt(c)
    assert p.shape == (32,) and p.dtype == np.int32
    assert p.min() >= 0 and p.max() < c.vocab
    assert len(set(p.tolist())) > 20


def test_deep_and_adapter_output_scales():
    c = ki.get_config("tiny")
    w = ki.make_weights(c)
    s0 = float(w["layers"][0]["wo"].std())
    s2 = float(w["layers"][2]["wo"].std())
    sa = float(w["adapter"]["wo"].std())
    assert abs(s0 - 0.02) < 1e-3
    assert abs(s2 - 0.02 * c.deep_resid_scale) < 1e-4
    assert abs(sa - 0.02 * c.adapter_resid_scale) < 1e-4
    assert abs(float(w["layers"][2]["wdown"].std()) - 0.02 * c.deep_resid_scale) < 1e-4
    assert abs(float(w["layers"][2]["wgate"].std()) - 0.02) < 1e-3


def test_paper_parameter_counts():
    # Table 2 / abstract for Vicuna-7B (d=4096, F=11008, V=32000): adapter 67M, +head 198M,
    # one transformer layer 202M, 11.3 % of Medusa's 591M heads, 88.7 % fewer; FFN = 67 % of a block.
    pc = ki.param_counts(4096, 11008, 32000)
    assert pc["adapter"] == 67_117_056
    assert round(pc["adapter"] / 1e6) == 67
    assert round((pc["adapter"] + pc["head"]) / 1e6) == 198
    assert round(pc["layer"] / 1e6) == 202
    assert round(100 * 67 / 591, 1) == 11.3
    assert round(100 * (1 - 67 / 591), 1) == 88.7
    assert round(100 * pc["ffn"] / pc["layer"]) == 67


def test_shapes_match_the_five_configs():
    c = ki.CONFIGS
    assert (c["tiny"].n_layers, c["tiny"].d_model, c["tiny"].n_heads, c["tiny"].head_dim, c["tiny"].d_ffn, c["tiny"].vocab, c["tiny"].exit_layer) == (4, 256, 4, 64, 688, 1024, 1)
    assert (c["7b"].n_layers, c["7b"].d_model, c["7b"].n_heads, c["7b"].head_dim, c["7b"].d_ffn, c["7b"].vocab, c["7b"].exit_layer) == (32, 4096, 32, 128, 11008, 32000, 2)
    assert (c["13b"].n_layers, c["13b"].d_model, c["13b"].d_ffn, c["13b"].exit_layer) == (40, 5120, 13824, 2)
    assert (c["33b"].n_layers, c["33b"].d_model, c["33b"].n_heads, c["33b"].d_ffn, c["33b"].exit_layer, c["33b"].gamma) == (60, 6656, 52, 17920, 3, 8)
    for s in c.values():
        assert s.n_heads * s.head_dim == s.d_model
        assert s.max_seq >= s.n_prompt + s.n_gen + s.gamma_max + 1


def test_lazy_weights_equal_the_eager_recipe():
    """Tensors regenerated on demand are bit-identical to make_weights, whether they are kept or rebuilt into the
    reusable buffers (budget 0: nothing is kept)."""
    shape = ki.get_config("tiny").with_(gain_std=0.1)
    w = ki.make_weights(shape)
    for budget in (0, 600_000, 1 << 40):
        lw = ki.LazyWeights(shape, np.float64, budget)
        assert getattr(lw, "lazy_weights", False)
        for i in range(shape.n_layers):
            for n in ("wqkv", "wo", "wgate", "wup", "wdown", "g1", "g2"):
                a = lw["layers"][i][n]
                assert a.dtype == np.float64 and np.array_equal(a, w["layers"][i][n].astype(np.float64)), (budget, i, n)
        for n in ("wqkv", "wo", "g_in", "g_last"):
            assert np.array_equal(lw["adapter"][n], w["adapter"][n].astype(np.float64))
        for n in ("embed", "head", "g_final"):
            assert np.array_equal(lw[n], w[n].astype(np.float64))
        assert lw._bytes <= budget
    # two tensors of one shape read back to back stay valid together (two buffers per shape)
    lw = ki.LazyWeights(shape, np.float64, 0)
    g, u = lw["layers"][0]["wgate"], lw["layers"][0]["wup"]
    assert np.array_equal(g, w["layers"][0]["wgate"]) and np.array_equal(u, w["layers"][0]["wup"])
