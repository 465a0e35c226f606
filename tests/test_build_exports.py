"""The C-ABI library builds for sm_100a, loads without a GPU and exports every declared symbol."""
import os
import re


def test_library_exports_every_declared_symbol():
    import __graft_entry__ as ge
    ge.build()
    from paper_2404_18911_b200 import binding
    lib = binding.load()
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    hdr = open(os.path.join(root, "include", "kangaroo.h")).read()
    declared = set(re.findall(r"\b(kg_[a-z_A-Z0-9]+)\s*\(", hdr))
    assert declared, "no declarations found"
    for name in sorted(declared):
        assert hasattr(lib, name), name
    assert set(binding.EXPORTS) == declared


def test_config_validation_without_gpu():
    import ctypes as C
    import kg_inputs as ki
    from paper_2404_18911_b200 import binding
    lib = binding.load()
    for name in ("tiny", "7b", "13b", "33b"):
        c = binding.config_from_shape(ki.get_config(name))
        assert lib.kg_workspace_bytes(C.byref(c), 1) > lib.kg_workspace_bytes(C.byref(c), 0) > 0
    c = binding.config_from_shape(ki.get_config("33b"))
    assert lib.kg_workspace_bytes(C.byref(c), 1) < 100e9          # fits one 180 GB B200 with room to spare
    bad = binding.config_from_shape(ki.get_config("tiny").with_(exit_layer=4))
    assert lib.kg_workspace_bytes(C.byref(bad), 1) == 0           # l must be < L
    bad = binding.config_from_shape(ki.get_config("tiny").with_(gamma_max=16))
    assert lib.kg_workspace_bytes(C.byref(bad), 1) == 0
    assert binding.strerror(0) == "ok" and "timed out" in binding.strerror(-6)


def test_misaligned_device_pointers_are_refused_before_anything_is_launched():
    """The kernels read caller memory with 16-byte bulk copies and vector loads; a pointer that is not 16-byte
    aligned must come back as KG_E_ARG from the host-side checks (no CUDA call is reached: this runs without a GPU).
    The addresses are never dereferenced."""
    import ctypes as C
    import kg_inputs as ki
    from paper_2404_18911_b200 import binding as b
    lib = b.load()
    ok, bad = 0x7f0000001000, 0x7f0000001002
    st = C.c_void_p(0)
    # single operators: weight, second weight, input, gain, residual, output, scratch in turn
    base = dict(W=ok, W2=None, x=ok, gain=ok, resid=ok, out=ok, scratch=ok)
    for key in ("W", "x", "gain", "resid", "out", "scratch"):
        a = dict(base); a[key] = bad
        r = lib.kg_op_linear(b.KG_BF16, a["W"], a["W2"], 64, 64, a["x"], 1, a["gain"], 1e-6, a["resid"], 0, a["out"], a["scratch"], st)
        assert r == b.KG_E_ARG, key
    assert lib.kg_op_linear(b.KG_BF16, ok, bad, 64, 64, ok, 1, ok, 1e-6, None, 1, ok, ok, st) == b.KG_E_ARG
    for i in range(5):                                              # W, x, gain, logits, scratch
        ptrs = [ok] * 5; ptrs[i] = bad
        W, x, g, z, sc = ptrs
        assert lib.kg_op_lm_head(b.KG_BF16, W, 64, 64, x, 1, g, 1e-6, 1.0, ok, ok, z, sc, st) == b.KG_E_ARG, i
    for i in range(4):                                              # W, x, gain, logits
        ptrs = [ok] * 4; ptrs[i] = bad
        W, x, g, z = ptrs
        assert lib.kg_op_lm_head_noalloc(b.KG_BF16, W, 64, 64, x, 1, g, 1e-6, 1.0, ok, ok, z, st) == b.KG_E_ARG, i
    for i in range(5):                                              # qkv, K cache, V cache, out, scratch
        ptrs = [ok] * 5; ptrs[i] = bad
        q, kc, vc, out, sc = ptrs
        assert lib.kg_op_attention(b.KG_BF16, q, 1, 0, 2, 64, 10000.0, kc, vc, ok, 16, out, sc, st) == b.KG_E_ARG, i
    # borrowed weights: one misaligned matrix among otherwise plausible pointers
    shape = ki.get_config("tiny")
    cfg = b.config_from_shape(shape)
    L = shape.n_layers
    arr = lambda v: (C.c_void_p * (L + 1))(*([v] * (L + 1)))
    for field in ("embed_dev", "wqkv_dev", "wdown_dev", "g2_dev"):
        w = b.KgWeights()
        w.embed_dev = w.head_dev = w.g_final_dev = ok
        keep = []
        for f in ("wqkv_dev", "wo_dev", "wgate_dev", "wup_dev", "wdown_dev", "g1_dev", "g2_dev"):
            a = arr(ok); keep.append(a); setattr(w, f, a)
        if field == "embed_dev":
            w.embed_dev = bad
        else:
            a = arr(ok); a[1] = bad; keep.append(a); setattr(w, field, a)
        h = C.c_void_p()
        assert lib.kg_init_model(C.byref(cfg), C.byref(w), ok, 1 << 40, None, C.byref(h)) == b.KG_E_ARG, field
        assert not h.value
