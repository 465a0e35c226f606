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
