"""The C-ABI library loads and exports every entry point the header declares (no GPU needed)."""
import ctypes
import os
import re

from paper_2603_09215_b200 import binding, build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in os.listdir(inc):
        if f.endswith(".h"):
            text = open(os.path.join(inc, f)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(sparsk_[a-z_0-9]+)\s*\(", text))
    return names


def test_library_builds_and_exports_the_header():
    lib_path = build.build()
    lib = ctypes.CDLL(lib_path)
    declared = _declared()
    assert declared, "no declarations found"
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in include/ but not exported"
    assert declared == set(binding.EXPORTS), declared ^ set(binding.EXPORTS)


def test_workspace_size_and_dims_validation_on_host():
    """sparsk_workspace_bytes is pure host arithmetic: 0 for bad dims, and it grows with the
    KV cache ([L][slots][H_kv][S][hd] bf16, twice)."""
    from paper_2603_09215_b200 import synth
    L = binding.load()
    dims = synth.model_dims("tiny", 2, 3, 0)
    d1 = binding.make_dims(dims, 2, 128, 2)
    d2 = binding.make_dims(dims, 2, 256, 2)
    a, b = L.sparsk_workspace_bytes(ctypes.byref(d1)), L.sparsk_workspace_bytes(ctypes.byref(d2))
    assert a > 0 and b > a
    kv = 2 * 4 * 2 * 2 * 128 * 64 * 2
    assert b - a >= kv
    for field, bad in (("exit_layer", 5), ("refresh_phase", 3), ("head_dim", 48), ("d_model", 250),
                       ("max_seqs", 0), ("n_kv_heads", 3)):
        d = binding.make_dims(dims, 2, 128, 2)
        setattr(d, field, bad)
        assert L.sparsk_workspace_bytes(ctypes.byref(d)) == 0, field
    out = ctypes.c_void_p()
    assert L.sparsk_create(ctypes.byref(d1), None, None, 0, None, ctypes.byref(out)) == binding.EINVAL
