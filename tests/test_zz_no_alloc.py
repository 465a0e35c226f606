"""The allocation-free LM-head entry point against the ordinary one.

kg_op_lm_head_noalloc serves callers that cannot get device memory when they need a token (a frozen or
exhausted pool, a host application that forbids cudaMalloc in its plugins, an error path): its scratch is a
fixed array inside the library.  The test calls it twice in a row through the C ABI, with different inputs,
and checks each result against kg_op_lm_head within the tolerances the other operator tests use; the second
call would expose stale partials left in the shared array by the first.  The file name keeps it last in the
collection order, so a run that stops at the first failure has already run every other test."""
import numpy as np
import pytest

from kg_inputs import synth
from oracle import kangaroo_oracle as ko

pytestmark = pytest.mark.gpu


def _mat(seed, tid, r, c, std, bf16):
    return synth.fill_f32(seed, tid, r * c, std, bf16).reshape(r, c)


def test_noalloc_lm_head_matches_scratch_version_twice():
    import torch
    import __graft_entry__ as ge
    ge.build()
    from paper_2404_18911_b200 import binding as b
    b.load()
    V, K = 32000, 4096
    W = torch.from_numpy(_mat(1, 80, V, K, 0.02, True)).cuda().to(torch.bfloat16)
    gain = torch.from_numpy((1.0 + _mat(3, 82, 1, K, 0.1, False)[0]).astype(np.float32)).cuda()
    # outputs are made before the calls: the entry point itself must not need an allocator
    for call, (M, seed) in enumerate([(7, 2), (3, 9)]):
        x = torch.from_numpy(_mat(seed, 81, M, K, 1.0, False)).cuda()
        tok = torch.full((M,), -1, dtype=torch.int32, device="cuda")
        p = torch.zeros(M, dtype=torch.float32, device="cuda")
        z = torch.zeros(M, V, dtype=torch.float32, device="cuda")
        b.op_lm_head_noalloc(W, x, gain, 1e-6, 9.0, tok, p, z)
        tok_r, p_r, z_r = b.op_lm_head(W, x, gain, 1e-6, 9.0)
        torch.cuda.synchronize()
        assert torch.equal(tok, tok_r), (call, tok.tolist(), tok_r.tolist())
        assert float((p - p_r).abs().max()) < 1e-3, call
        assert float((z - z_r).abs().max()) < 2e-3, call
        assert int(tok.min()) >= 0
        # and against the definition, on both calls: z = s * RMSNorm(x; g) W^T, lowest arg max, p = 1 / sum exp(z - z_max)
        xn = ko.rmsnorm(x.cpu().numpy().astype(np.float64), gain.cpu().numpy().astype(np.float64), 1e-6)
        zr = 9.0 * (xn @ W.float().cpu().numpy().astype(np.float64).T)
        assert np.max(np.abs(z.cpu().numpy() - zr)) < 2e-3, call
        for m in range(M):
            t_ref, p_ref = ko.top1_confidence(zr[m])
            assert int(tok[m]) == t_ref or ko.top2_gap(zr[m]) < 2e-2, (call, m)
            assert abs(float(p[m]) - p_ref) < 1e-3, (call, m)


def test_noalloc_at_the_edge_of_its_capacity_and_on_the_plain_path():
    """The largest rows the static scratch holds (16 rows of 8192), an fp32 head (plain path, no packed rows), and
    one element beyond the row limit."""
    import torch
    import __graft_entry__ as ge
    ge.build()
    from paper_2404_18911_b200 import binding as b
    b.load()
    for (V, K, M, bf) in [(3000, 8192, 16, True), (1024, 256, 5, False)]:
        W = torch.from_numpy(_mat(1, 83, V, K, 0.02, bf)).cuda()
        W = W.to(torch.bfloat16) if bf else W
        x = torch.from_numpy(_mat(4, 84, M, K, 1.0, False)).cuda()
        gain = torch.from_numpy((1.0 + _mat(3, 85, 1, K, 0.1, False)[0]).astype(np.float32)).cuda()
        tok = torch.full((M,), -1, dtype=torch.int32, device="cuda")
        p = torch.zeros(M, dtype=torch.float32, device="cuda")
        z = torch.zeros(M, V, dtype=torch.float32, device="cuda")
        b.op_lm_head_noalloc(W, x, gain, 1e-6, 7.0, tok, p, z)
        tok_r, p_r, z_r = b.op_lm_head(W, x, gain, 1e-6, 7.0)
        torch.cuda.synchronize()
        assert torch.equal(tok, tok_r) and float((p - p_r).abs().max()) < 1e-3 and float((z - z_r).abs().max()) < 2e-3
        xn = ko.rmsnorm(x.cpu().numpy().astype(np.float64), gain.cpu().numpy().astype(np.float64), 1e-6)
        zr = 7.0 * (xn @ W.float().cpu().numpy().astype(np.float64).T)
        assert np.max(np.abs(z.cpu().numpy() - zr)) < 2e-3
    K = 8192 + 16
    W = torch.zeros(64, K, dtype=torch.bfloat16, device="cuda")
    x = torch.zeros(2, K, dtype=torch.float32, device="cuda")
    tok = torch.zeros(2, dtype=torch.int32, device="cuda")
    p = torch.zeros(2, dtype=torch.float32, device="cuda")
    with pytest.raises(b.KgError) as e:
        b.op_lm_head_noalloc(W, x, None, 0.0, 1.0, tok, p)
    assert e.value.status == b.KG_E_LIMIT


def test_noalloc_rejects_sizes_beyond_its_capacity():
    import torch
    import __graft_entry__ as ge
    ge.build()
    from paper_2404_18911_b200 import binding as b
    b.load()
    V, K, M = 64, 64, b.KG_M_MAX + 1
    W = torch.zeros(V, K, dtype=torch.bfloat16, device="cuda")
    x = torch.zeros(M, K, dtype=torch.float32, device="cuda")
    tok = torch.zeros(M, dtype=torch.int32, device="cuda")
    p = torch.zeros(M, dtype=torch.float32, device="cuda")
    with pytest.raises(b.KgError) as e:
        b.op_lm_head_noalloc(W, x, None, 0.0, 1.0, tok, p)
    assert e.value.status == b.KG_E_LIMIT
    assert "static scratch" in b.strerror(b.KG_E_LIMIT)
