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
