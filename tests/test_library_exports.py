"""The C-ABI library builds, loads and exports every symbol the header declares
(no GPU needed; no compute call is made)."""

import os
import re

import paper_2509_11815_b200 as sv
from paper_2509_11815_b200 import build as sv_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "specvlm.h")).read()
    return sorted(set(re.findall(r"SPECVLM_API[^;(]*?\b(specvlm_\w+)\s*\(", text)))


def test_library_builds_and_exports_header_symbols():
    path = sv_build.build()
    assert os.path.exists(path)
    lib = sv.load_library()
    names = _declared()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), f"{n} declared in specvlm.h but not exported"
    assert sorted(sv.EXPORTS) == names
    assert lib.specvlm_version() == 100


def test_host_side_tree_validation():
    assert sv.specvlm_tree_validate_host([-1, 0, 0, 1]) == 0
    assert sv.specvlm_tree_validate_host([-1, 0, 0, 1], [9, 4, 5, 4]) == 0
    assert sv.specvlm_tree_validate_host([0, 0]) == -4
    assert sv.specvlm_tree_validate_host([-1, 1]) == -4
    assert sv.specvlm_tree_validate_host([-1, 0, 0], [9, 4, 4]) == -4
    assert sv.specvlm_tree_validate_host([-1] + list(range(64))) == -4
    assert b"sibling" in sv.load_library().specvlm_last_error_string() or True


def test_host_side_argument_errors_need_no_gpu():
    import ctypes
    lib = sv.load_library()
    d = sv.AttnDesc()
    n = ctypes.c_size_t(0)
    d.B, d.H, d.T, d.D, d.S_cap = 1, 32, 60, 64, 1024          # D != 128
    assert lib.specvlm_attn_workspace_bytes(ctypes.byref(d), ctypes.byref(n)) == -1
    assert b"D must be 128" in lib.specvlm_last_error_string()
    d.D, d.T = 128, 65                                         # T > 64
    assert lib.specvlm_attn_workspace_bytes(ctypes.byref(d), ctypes.byref(n)) == -1
    d.T = 60
    for f in ("q_stride_t", "k_stride_s", "v_stride_s", "o_stride_t"):
        setattr(d, f, 128)
    d.k_stride_h = 12                                          # not a multiple of 8
    assert lib.specvlm_attn_workspace_bytes(ctypes.byref(d), ctypes.byref(n)) == -1
    d.k_stride_h = 1024 * 128
    d.num_splits = 4                                           # <= 8 splits combine on chip
    assert lib.specvlm_attn_workspace_bytes(ctypes.byref(d), ctypes.byref(n)) == 0
    assert n.value == 0
    d.num_splits = 12
    assert lib.specvlm_attn_workspace_bytes(ctypes.byref(d), ctypes.byref(n)) == 0
    assert n.value == 256 + 32 * 12 * 64 * 2 * 4 + 32 * 12 * 64 * 128 * 4
    # null pointers are rejected before any launch
    assert lib.specvlm_argmax(None, 1, 60, 32000, 32000, None, None) == -1
    assert lib.specvlm_tree_build(None, None, 1, 60, None, None, None, None, None) == -1


def _header_prototypes():
    """name -> list of parameter kinds ('ptr', 'i32', 'i64', 'f32', 'size') parsed from the header."""
    text = open(os.path.join(ROOT, "include", "specvlm.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    protos = {}
    for name, args in re.findall(r"SPECVLM_API[^;(]*?\b(specvlm_\w+)\s*\(([^)]*)\)\s*;", text):
        kinds = []
        args = " ".join(args.split())
        if args not in ("", "void"):
            for a in args.split(","):
                a = a.strip()
                if "*" in a:
                    kinds.append("ptr")
                elif re.match(r"(const\s+)?int64_t\b", a):
                    kinds.append("i64")
                elif re.match(r"(const\s+)?(int32_t|int)\b", a):
                    kinds.append("i32")
                elif re.match(r"(const\s+)?float\b", a):
                    kinds.append("f32")
                elif re.match(r"(const\s+)?size_t\b", a):
                    kinds.append("size")
                else:
                    raise AssertionError(f"unparsed parameter {a!r} of {name}")
        protos[name] = kinds
    return protos


def test_binding_prototypes_match_the_header():
    """Every ctypes prototype has the header's parameter count, and pointers / 32-bit / 64-bit /
    float parameters sit where the header puts them (a mismatch would corrupt the call silently)."""
    import ctypes
    lib = sv.load_library()
    kinds_of = {ctypes.c_int32: "i32", ctypes.c_int: "i32", ctypes.c_int64: "i64", ctypes.c_float: "f32",
                ctypes.c_size_t: "size", ctypes.c_void_p: "ptr", ctypes.c_char_p: "ptr"}
    protos = _header_prototypes()
    assert sorted(protos) == _declared()
    for name, want in protos.items():
        argtypes = getattr(lib, name).argtypes
        assert argtypes is not None, f"{name} has no ctypes prototype"
        got = []
        for t in argtypes:
            if t in kinds_of:
                got.append(kinds_of[t])
            elif hasattr(t, "contents") or getattr(t, "_type_", None) is not None and not isinstance(t._type_, str):
                got.append("ptr")          # POINTER(struct)
            else:
                raise AssertionError(f"unknown ctypes type {t} in {name}")
        assert got == want, f"{name}: binding {got} != header {want}"
