"""CPU-only checks of the C-ABI library: it loads, exports every symbol the public header declares, and
its host-side argument validation returns status codes without needing a GPU."""
import ctypes as C
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    """Every function declared in include/*.h (the product header and the debug-hook header)."""
    names = set()
    inc = os.path.join(ROOT, "include")
    for f in sorted(os.listdir(inc)):
        if f.endswith(".h"):
            text = re.sub(r"/\*.*?\*/", "", open(os.path.join(inc, f)).read(), flags=re.S)
            names |= set(re.findall(r"\b(cats_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def _lib():
    from paper_2605_11186_b200 import build
    return C.CDLL(build.build())


def test_header_declares_the_five_core_calls():
    names = _declared_functions()
    for n in ("cats_build_tree_mask", "cats_verify_layer", "cats_tree_attention", "cats_accept_path", "cats_compact_kv"):
        assert n in names


def test_library_exports_every_declared_symbol():
    lib = _lib()
    names = _declared_functions()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), n


def test_status_strings_and_version():
    lib = _lib()
    lib.cats_status_string.restype = C.c_char_p
    assert lib.cats_version() >= 100
    seen = {lib.cats_status_string(s) for s in range(0, -8, -1)}
    assert len(seen) == 8 and b"ok" in seen


def test_host_side_validation_needs_no_gpu():
    lib = _lib()

    class Cfg(C.Structure):
        _fields_ = [("hidden", C.c_int32), ("n_heads", C.c_int32), ("head_dim", C.c_int32), ("ffn", C.c_int32),
                    ("vocab", C.c_int32), ("n_layers", C.c_int32), ("max_seq", C.c_int32), ("rms_eps", C.c_float),
                    ("rope_base", C.c_float)]
    lib.cats_workspace_bytes.restype = C.c_size_t
    good = Cfg(4096, 32, 128, 11008, 32000, 32, 640, 1e-5, 10000.0)
    n = lib.cats_workspace_bytes(C.byref(good), 128, 512)
    assert 10 << 20 < n < 200 << 20
    assert lib.cats_workspace_bytes(C.byref(good), 129, 512) == 0
    assert lib.cats_workspace_bytes(C.byref(good), 0, 512) == 0
    bad = Cfg(4096, 32, 96, 11008, 32000, 32, 640, 1e-5, 10000.0)
    assert lib.cats_workspace_bytes(C.byref(bad), 16, 512) == 0
    # null pointers and out-of-range T are refused before anything is launched
    assert lib.cats_build_tree_mask(None, 4, 0, None, None, None, None, None) == -1
    assert lib.cats_accept_path(None, None, None, 4, None, None, None, None, None, None) == -1
    assert lib.cats_compact_kv(None, None, 1, C.c_int64(8), C.c_int64(8), 0, None, None, None, None, None, None, None) == -1
    assert lib.cats_verify_forward(None, None, None, None) == -1
