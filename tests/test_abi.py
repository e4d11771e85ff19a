"""The C-ABI library loads without a GPU and exports every function the headers under include/ declare
(taot.h: the planner; taot_measure.h: measurement aids)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = "".join(open(os.path.join(ROOT, "include", f)).read() for f in sorted(os.listdir(os.path.join(ROOT, "include")))
                   if f.endswith(".h"))
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(taot_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    from paper_2608_03676_b200.build import build
    lib_path = build()
    lib = ctypes.CDLL(lib_path)
    names = _declared()
    assert "taot_plan" in names and "taot_sinkhorn" in names and len(names) >= 13
    for name in names:
        assert hasattr(lib, name), name
    import paper_2608_03676_b200 as P
    assert sorted(P.exported_symbols()) == names                 # the binding covers the whole header
    lib.taot_status_string.restype = ctypes.c_char_p
    assert lib.taot_status_string(0) == b"ok"
    assert b"NULL" in lib.taot_status_string(-1)


def test_host_side_validation_needs_no_gpu():
    import paper_2608_03676_b200 as P
    lib = P.load_library()
    p = P.TaotParams(ctypes.sizeof(P.TaotParams), 1, 8, 32, 2, 2, 4096, 0.4, 200, 0.0, 1, 1e-8, 0.1, 0)
    h = ctypes.c_void_p()
    assert lib.taot_create(ctypes.byref(h), ctypes.byref(p), None, None, None) == -1          # NULL pointers
    e2r = (ctypes.c_int32 * 32)(*[e // 4 for e in range(32)])
    C = (ctypes.c_float * 64)(*([1.0] * 64))
    bad = P.TaotParams(ctypes.sizeof(P.TaotParams), 1, 8, 32, 2, 2, 4097, 0.4, 200, 0.0, 1, 1e-8, 0.1, 0)
    assert lib.taot_create(ctypes.byref(h), ctypes.byref(bad), e2r, C, None) == -2            # T % R != 0
    bad = P.TaotParams(ctypes.sizeof(P.TaotParams), 1, 8, 32, 2, 2, 4096, 0.0, 200, 0.0, 1, 1e-8, 0.1, 0)
    assert lib.taot_create(ctypes.byref(h), ctypes.byref(bad), e2r, C, None) == -2            # eps <= 0
    big = P.TaotParams(ctypes.sizeof(P.TaotParams), 1, 2048, 4096, 2, 2, 4096, 0.4, 200, 0.0, 1, 1e-8, 0.1, 0)
    e2r_big = (ctypes.c_int32 * 4096)()
    C_big = (ctypes.c_float * (2048 * 2048))()
    assert lib.taot_create(ctypes.byref(h), ctypes.byref(big), e2r_big, C_big, None) == -3    # beyond this build
    e2r[5] = 99
    assert lib.taot_create(ctypes.byref(h), ctypes.byref(p), e2r, C, None) == -2              # home rank out of range
    assert not h.value
    assert lib.taot_destroy(None) == 0
    size = ctypes.c_size_t()
    assert lib.taot_workspace_bytes(None, ctypes.byref(size)) == -1


def test_layer_groups_of_the_pipelined_host_call():
    import paper_2608_03676_b200 as P
    assert P.split_layers(24, 4) == [(0, 6), (6, 12), (12, 18), (18, 24)]
    assert P.split_layers(7, 3) == [(0, 3), (3, 5), (5, 7)]
    assert P.split_layers(2, 8) == [(0, 1), (1, 2)]                 # never an empty group
    assert P.split_layers(5, 0) == [(0, 5)]
    for L in range(1, 40):
        for g in range(1, 10):
            b = P.split_layers(L, g)
            assert b[0][0] == 0 and b[-1][1] == L and all(x[1] == y[0] for x, y in zip(b, b[1:]))
            sizes = [hi - lo for lo, hi in b]
            assert min(sizes) >= 1 and max(sizes) - min(sizes) <= 1


def test_ablation_bits_are_validated_on_the_host():
    import paper_2608_03676_b200 as P
    lib = P.load_library()
    e2r = (ctypes.c_int32 * 32)(*[e // 4 for e in range(32)])
    C = (ctypes.c_float * 64)(*([1.0] * 64))
    h = ctypes.c_void_p()
    bad = P.TaotParams(ctypes.sizeof(P.TaotParams), 1, 8, 32, 2, 2, 4096, 0.4, 200, 0.0, 1, 1e-8, 0.1, 0, 4)
    assert lib.taot_create(ctypes.byref(h), ctypes.byref(bad), e2r, C, None) == -2            # unknown ablation bit
    assert ctypes.sizeof(P.ReportRow) == 128
