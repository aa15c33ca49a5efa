"""CPU-only checks of the C-ABI library: it builds, loads, exports every symbol the header
declares, and its host-side validation rejects bad arguments without launching anything."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def pkg():
    from paper_2607_04244_b200 import build
    build.build_library()
    import paper_2607_04244_b200 as p
    p.load()
    return p


def _declared_functions():
    names = set()
    inc = os.path.join(ROOT, "include")
    for fn in os.listdir(inc):
        if not fn.endswith(".h"):
            continue
        src = open(os.path.join(inc, fn)).read()
        src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
        for m in re.finditer(r"^[A-Za-z_][\w\s\*]*?\b(\w+)\s*\([^;{]*\)\s*;", src, flags=re.M):
            names.add(m.group(1))
    return names


def test_library_exports_every_declared_symbol(pkg):
    declared = _declared_functions()
    assert {"qpack_w4_g128", "qlinear_w4a16", "qlinear_stack_w4a16"} <= declared
    lib = ctypes.CDLL(pkg.LIB_PATH)
    for name in sorted(declared):
        assert hasattr(lib, name), f"{name} declared in include/ but not exported"
    assert declared == set(pkg.EXPORTS), declared ^ set(pkg.EXPORTS)


def test_size_queries(pkg):
    # packed bytes = codes + bf16 scales + 4-bit zeros, no padding
    for K, N, g in [(2560, 9728, 128), (9728, 2560, 128), (2560, 6144, 64), (2560, 151936, 128), (512, 256, 128)]:
        assert pkg.ql_packed_bytes(K, N, g) == K * N // 2 + (K // g) * N * 2 + (K // g) * N // 2
    assert pkg.ql_packed_bytes(2560, 9728, 100) == 0
    assert pkg.ql_packed_bytes(2560, 9700, 128) == 0
    assert pkg.ql_packed_bytes(2500, 9728, 128) == 0
    assert pkg.ql_workspace_bytes(16, 9728) > 0
    assert pkg.ql_workspace_bytes(64, 151936) >= pkg.ql_workspace_bytes(16, 151936)
    assert pkg.ql_workspace_bytes(0, 128) == 0 and pkg.ql_workspace_bytes(65, 128) == 0
    assert pkg.ql_workspace_bytes(16, 100) == 0
    assert pkg.ql_select_path(16, 2560, 9728, 128) in (pkg.QL_PATH_MMA, pkg.QL_PATH_TC5)
    assert pkg.ql_select_path(16, 2560, 9728, 96) < 0


def test_attention_plan_and_argument_checks_without_a_device(pkg):
    # the union of the queries' windows and its split into pieces of 64-key sub-blocks (paper Section 3.3)
    assert pkg.ql_attn_plan(16, 8208, 32, 8, 128, 8192, 1024) == dict(key_lo=8192 - 512, key_hi=8208, n_pieces=9, sub_per_piece=1)
    assert pkg.ql_attn_plan(16, 2064, 32, 8, 128, 2048, 2048) == dict(key_lo=1024, key_hi=2064, n_pieces=17, sub_per_piece=1)
    assert pkg.ql_attn_plan(16, 80, 32, 8, 128, 64, 1024) == dict(key_lo=0, key_hi=80, n_pieces=1, sub_per_piece=2)      # fits: everything, one piece
    p = pkg.ql_attn_plan(16, 4096, 32, 8, 128, 2000, 1024)
    assert (p["key_lo"], p["key_hi"]) == (1488, 2528)                                   # both sides of the block
    p = pkg.ql_attn_plan(16, 40016, 32, 8, 128, 40000, 65536)
    assert p["n_pieces"] * p["sub_per_piece"] * 64 >= 40016 and p["n_pieces"] <= 18
    for bad in [(17, 100, 32, 8, 128, 0, 64), (16, 100, 32, 8, 128, 90, 64), (16, 100, 32, 5, 128, 0, 64), (0, 100, 32, 8, 128, 0, 64)]:
        with pytest.raises(pkg.QlError) as e:
            pkg.ql_attn_plan(*bad)
        assert e.value.status == pkg.QL_ERR_SHAPE
    with pytest.raises(pkg.QlError) as e:
        pkg.ql_attn_plan(16, 100, 32, 8, 64, 0, 64)
    assert e.value.status == pkg.QL_ERR_UNSUPPORTED
    assert pkg.ql_attn_workspace_bytes(32, 8) >= 256 + 32 * 18 * 16 * 132 * 4
    assert pkg.ql_attn_workspace_bytes(32, 5) == 0


def test_status_strings(pkg):
    lib = pkg.load()
    seen = {lib.ql_status_str(i).decode() for i in range(8)}
    assert len(seen) == 8 and "ok" in seen


def test_argument_errors_launch_nothing(pkg):
    """Fake (never dereferenced) pointers: every call must be rejected by validation."""
    lib = pkg.load()
    P = 0x10000          # 16-byte aligned, non-null
    ws_bytes = pkg.ql_workspace_bytes(16, 256)
    before = pkg.ql_launch_count()
    lin = lambda **kw: lib.qlinear_w4a16(kw.get("packed", P), kw.get("X", P), kw.get("Y", P), kw.get("am", None),
                                         kw.get("M", 16), kw.get("K", 512), kw.get("N", 256), kw.get("g", 128),
                                         kw.get("ws", P), kw.get("wsb", ws_bytes), None)
    assert lin(packed=None) == pkg.QL_ERR_NULL
    assert lin(X=None) == pkg.QL_ERR_NULL
    assert lin(Y=None, am=None) == pkg.QL_ERR_NULL
    assert lin(ws=None) == pkg.QL_ERR_NULL
    assert lin(M=0) == pkg.QL_ERR_SHAPE
    assert lin(M=65) == pkg.QL_ERR_SHAPE
    assert lin(K=500) == pkg.QL_ERR_SHAPE
    assert lin(N=200) == pkg.QL_ERR_SHAPE
    assert lin(g=32) == pkg.QL_ERR_SHAPE
    assert lin(X=P + 2) == pkg.QL_ERR_ALIGN
    assert lin(Y=P + 8) == pkg.QL_ERR_ALIGN
    assert lin(wsb=1024) == pkg.QL_ERR_WORKSPACE
    pk = lambda **kw: lib.qpack_w4_g128(kw.get("wq", P), kw.get("scale", P), kw.get("zero", P), kw.get("K", 512),
                                        kw.get("N", 256), kw.get("g", 128), kw.get("packed", P),
                                        kw.get("pb", pkg.ql_packed_bytes(512, 256, 128)), None)
    assert pk(wq=None) == pkg.QL_ERR_NULL
    assert pk(packed=None) == pkg.QL_ERR_NULL
    assert pk(K=520) == pkg.QL_ERR_SHAPE
    assert pk(pb=100) == pkg.QL_ERR_WORKSPACE
    assert pk(packed=P + 4) == pkg.QL_ERR_ALIGN
    assert lib.qlinear_w4a16_path(P, P, P, None, 16, 512, 256, 128, P, ws_bytes, None, 9) == pkg.QL_ERR_UNSUPPORTED
    # stack: a bad operation anywhere rejects the whole list
    good = dict(kind=pkg.QL_OP_LINEAR, M=16, K=512, N=256, g=128, ld_in=512, ld_out=256, packed=P, in0=P, out=P)
    bad = dict(good, K=100)
    ops = pkg.make_ops([good, bad])
    assert lib.qlinear_stack_w4a16(ops, 2, P, ws_bytes, None) == pkg.QL_ERR_SHAPE
    ops = pkg.make_ops([dict(kind=77, M=16, N=256, ld_in=256, ld_out=256, in0=P, out=P)])
    assert lib.qlinear_stack_w4a16(ops, 1, P, ws_bytes, None) == pkg.QL_ERR_UNSUPPORTED
    ops = pkg.make_ops([dict(kind=pkg.QL_OP_SILU_MUL_UNIT_RMS, M=16, N=256, ld_in=256, ld_out=256, in0=P, out=P)])
    assert lib.qlinear_stack_w4a16(ops, 1, P, ws_bytes, None) == pkg.QL_ERR_NULL
    assert lib.qlinear_stack_w4a16(None, 0, P, ws_bytes, None) == pkg.QL_ERR_NULL
    assert lib.ql_workspace_init(None, 100, None) == pkg.QL_ERR_NULL
    assert lib.ql_workspace_init(P, 100, None) == pkg.QL_ERR_WORKSPACE
    assert pkg.ql_launch_count() == before


def test_missing_library_fails_loudly(tmp_path):
    import importlib
    import paper_2607_04244_b200 as p
    saved = p._lib
    try:
        p._lib = None
        with pytest.raises(OSError):
            p.load(str(tmp_path / "nope.so"))
    finally:
        p._lib = saved
