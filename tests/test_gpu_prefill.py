"""The tensor-core prompt pass (GEMMs on tcgen05 over blocks of prompt rows) against the oracle and against the
16-row chunked pass of the decode kernels: prefill logits, then lock-step rounds that read the K / V caches it wrote."""
import numpy as np
import pytest

import kg_inputs as ki
from oracle import kangaroo_oracle as ko

pytestmark = pytest.mark.gpu

# bf16 model whose sides are whole GEMM tiles (d, F multiples of 128), several k blocks, two layers before the exit
TC_BF = ki.KgShape("tc_bf", 4, 512, 4, 128, 1408, 2048, 2, "bf16", logit_scale=10.0, max_seq=256, page_size=16,
                   gamma_max=10, gain_std=0.1, deep_resid_scale=0.1, adapter_resid_scale=0.1, n_prompt=70, n_gen=24, seed=9)


@pytest.fixture(scope="module")
def binding():
    import __graft_entry__ as ge
    ge.build()
    from paper_2404_18911_b200 import binding as b
    b.load()
    return b


@pytest.mark.parametrize("n_prompt", [32, 70, 128, 150])
def test_tensor_core_prefill_matches_oracle_and_chunked_pass(binding, n_prompt):
    from parity_harness import lockstep
    shape = TC_BF
    g = binding.KangarooModel(shape, debug_logits=True)
    o = ko.KangarooOracle(shape, ki.make_weights(shape), np.float64)
    prompt = ki.make_prompt(shape, n_prompt).tolist()
    # prefill logits of both passes against the oracle
    x0_ref = o.prefill(prompt)
    z_ref = o.last_logits
    g.set_prefill_mode(1)
    x0_chunk = g.prefill(prompt)
    z_chunk = g.debug_logits(1, 0).astype(np.float64)
    g.reset()
    g.set_prefill_mode(0)
    x0_tc = g.prefill(prompt)
    z_tc = g.debug_logits(1, 0).astype(np.float64)
    e_tc, e_chunk = float(np.max(np.abs(z_tc - z_ref))), float(np.max(np.abs(z_chunk - z_ref)))
    print(f"n={n_prompt}: prefill logit deviation tensor-core {e_tc:.2e}, chunked {e_chunk:.2e}")
    assert e_tc < 2e-2 and e_chunk < 2e-2
    assert x0_tc == x0_ref or ko.top2_gap(z_ref) < 2e-2
    assert x0_tc == x0_chunk or ko.top2_gap(z_ref) < 2e-2
    # rounds on top of the caches the tensor-core pass wrote (the harness prefills again, in the default mode)
    res = lockstep(g, o, prompt, shape.n_gen, shape.eta, shape.gamma, 0)
    assert len(res["flips"]) <= 2, res["flips"]
    assert res["max_logit_err"] < 2e-2 and res["max_conf_err"] < 1e-3


def test_tensor_core_prefill_of_the_7b_shape_matches_the_trace(binding):
    """The benchmark's prompt (512 tokens, one block of rows): x_0 and the recorded prefill logits of the fp64 oracle."""
    import json
    import os
    tr = json.load(open(os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "trace_7b_full.json")))
    shape = ki.get_config("7b")
    g = binding.KangarooModel(shape, debug_logits=True)
    prompt = ki.make_prompt(shape, tr["n_prompt"]).tolist()
    for mode in (0, 1):
        g.reset()
        g.set_prefill_mode(mode)
        x0 = g.prefill(prompt)
        z = g.debug_logits(1, 0)
        err = max(abs(float(z[i]) - v) for i, v in zip(tr["sample_indices"], tr["prefill"]["samples"]))
        err = max([err] + [abs(float(z[i]) - v) for i, v in tr["prefill"]["top"]])
        print(f"7B prefill, mode {mode}: logit deviation {err:.2e}")
        assert err < 2e-2 and x0 == tr["prefill"]["x0"]


@pytest.mark.parametrize("N,K,M", [(128, 64, 1), (256, 4096, 128), (4096, 4096, 100), (1408, 512, 70), (512, 2752, 37), (12288, 4096, 128), (4096, 11008, 128), (11008, 4096, 77)])
def test_gemm_against_fp64(binding, N, K, M):
    """out = resid + x W^T of the tensor-core GEMM, element by element against float64, at the tolerance of the
    decode path's linear operator; and its error next to that operator's on the first 16 rows."""
    import torch
    from kg_inputs import synth
    W = synth.fill_f32(1, 50, N * K, 0.02, True).reshape(N, K)
    x = synth.fill_f32(2, 51, M * K, 1.0, False).reshape(M, K)
    resid = synth.fill_f32(4, 53, M * N, 1.0, False).reshape(M, N)
    Wd = torch.from_numpy(W).cuda().to(torch.bfloat16)
    xd, rd = torch.from_numpy(x).cuda(), torch.from_numpy(resid).cuda()
    ref = resid.astype(np.float64) + x.astype(np.float64) @ W.astype(np.float64).T
    scale = float(np.sqrt(K) * 0.02)
    y = binding.op_gemm(Wd, xd, resid=rd).cpu().numpy()
    e_tc = float(np.max(np.abs(y - ref)))
    m16 = min(M, 16)
    y16 = binding.op_linear(Wd, xd[:m16].contiguous(), resid=rd[:m16].contiguous()).cpu().numpy()
    e_lin = float(np.max(np.abs(y16 - ref[:m16])))
    print(f"N={N} K={K} M={M}: max error tensor-core GEMM {e_tc:.2e}, decode-path linear (first {m16} rows) {e_lin:.2e}, bound {2e-4 * scale:.2e}")
    assert e_tc < 2e-4 * scale
    y2 = binding.op_gemm(Wd, xd).cpu().numpy()
    assert np.max(np.abs(y2 - (ref - resid))) < 2e-4 * scale
