"""Python binding of the qlinear_w4a16 C-ABI library (argument marshalling only).

Every function has the name and the meaning of the entry point declared in
include/qlinear_w4a16.h; torch is used for device memory and streams, nothing else.  There is no
fallback: if the shared library is missing, `load()` raises.
"""
from __future__ import annotations

import ctypes
import os

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG_DIR, "libqlinear_w4a16.so")

QL_OK = 0
QL_ERR_NULL, QL_ERR_SHAPE, QL_ERR_ALIGN, QL_ERR_UNSUPPORTED = 1, 2, 3, 4
QL_ERR_WORKSPACE, QL_ERR_CUDA, QL_ERR_DEVICE_TIMEOUT = 5, 6, 7
QL_PATH_AUTO, QL_PATH_MMA, QL_PATH_TC5 = 0, 2, 3
PATH_NAMES = {QL_PATH_MMA: "mma", QL_PATH_TC5: "tcgen05"}
QL_OP_LINEAR, QL_OP_UNIT_RMS, QL_OP_SILU_MUL_UNIT_RMS = 0, 1, 2

EXPORTS = [
    "ql_status_str", "ql_packed_bytes", "ql_workspace_bytes", "ql_workspace_init", "ql_device_status",
    "ql_device_status_raw",
    "qpack_w4_g128", "qrequant_pack_w4", "qlinear_w4a16", "qlinear_w4a16_path", "ql_select_path", "qlinear_stack_w4a16",
    "qlinear_stack_w4a16_host", "ql_launch_count", "qlinear_w4a16_static", "ql_static_status", "ql_stack_plan", "ql_linear_plan", "ql_plan_first_chunk", "ql_plan_chunk_owner",
    "ql_plan_chain_split", "ql_debug_set_owner_extra",
    "ql_attn_workspace_bytes", "qattn_swa_bf16", "ql_attn_plan",
    "ql_debug_set_wait_budget_ns", "ql_debug_no_release", "ql_debug_set_timeline", "ql_debug_timeline_enabled", "ql_debug_set_ablate",
]


class ql_op(ctypes.Structure):
    _fields_ = [
        ("kind", ctypes.c_int32), ("M", ctypes.c_int32), ("K", ctypes.c_int32), ("N", ctypes.c_int32),
        ("g", ctypes.c_int32), ("ld_in", ctypes.c_int32), ("ld_out", ctypes.c_int32), ("reserved", ctypes.c_int32),
        ("packed", ctypes.c_void_p), ("in0", ctypes.c_void_p), ("in1", ctypes.c_void_p),
        ("out", ctypes.c_void_p), ("argmax_out", ctypes.c_void_p),
        ("draft_ids", ctypes.c_void_p), ("accept_out", ctypes.c_void_p),
    ]


class QlError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = _lib.ql_status_str(status).decode() if _lib is not None else str(status)
        super().__init__(f"{where}: status {status} ({msg})")


_lib = None


def load(path: str | None = None):
    """Load the shared library (once).  Raises OSError if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    path = path or LIB_PATH
    if not os.path.exists(path):
        raise OSError(f"{path} not found: build it with `python -m paper_2607_04244_b200.build` "
                      "(there is no fallback implementation)")
    lib = ctypes.CDLL(path)
    vp, sz, i32 = ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int
    lib.ql_status_str.restype = ctypes.c_char_p
    lib.ql_status_str.argtypes = [i32]
    lib.ql_packed_bytes.restype = sz
    lib.ql_packed_bytes.argtypes = [i32, i32, i32]
    lib.ql_workspace_bytes.restype = sz
    lib.ql_workspace_bytes.argtypes = [i32, i32]
    lib.ql_workspace_init.restype = i32
    lib.ql_workspace_init.argtypes = [vp, sz, vp]
    lib.ql_device_status.restype = i32
    lib.ql_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int), vp]
    lib.ql_device_status_raw.restype = i32
    lib.ql_device_status_raw.argtypes = [vp, ctypes.POINTER(ctypes.c_int), vp]
    lib.qpack_w4_g128.restype = i32
    lib.qpack_w4_g128.argtypes = [vp, vp, vp, i32, i32, i32, vp, sz, vp]
    lib.qrequant_pack_w4.restype = i32
    lib.qrequant_pack_w4.argtypes = [vp, vp, vp, i32, i32, i32, vp, sz, vp]
    lib.qlinear_w4a16.restype = i32
    lib.qlinear_w4a16.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp, sz, vp]
    lib.qlinear_w4a16_path.restype = i32
    lib.qlinear_w4a16_path.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp, sz, vp, i32]
    lib.ql_select_path.restype = i32
    lib.ql_select_path.argtypes = [i32, i32, i32, i32]
    lib.qlinear_stack_w4a16.restype = i32
    lib.qlinear_stack_w4a16.argtypes = [ctypes.POINTER(ql_op), i32, vp, sz, vp]
    lib.qlinear_stack_w4a16_host.restype = i32
    lib.qlinear_stack_w4a16_host.argtypes = [ctypes.POINTER(ql_op), i32, vp, vp, sz, vp, vp, sz, vp, sz, vp]
    lib.qlinear_w4a16_static.restype = i32
    lib.qlinear_w4a16_static.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp]
    lib.ql_static_status.restype = i32
    lib.ql_static_status.argtypes = [ctypes.POINTER(ctypes.c_int), vp]
    lib.ql_stack_plan.restype = i32
    lib.ql_stack_plan.argtypes = [ctypes.POINTER(ql_op), i32, vp, sz, ctypes.POINTER(ctypes.c_int)]
    lib.ql_linear_plan.restype = i32
    lib.ql_linear_plan.argtypes = [i32, i32, i32, i32, i32, ctypes.POINTER(ctypes.c_int)]
    lib.ql_attn_workspace_bytes.restype = sz
    lib.ql_attn_workspace_bytes.argtypes = [i32, i32]
    lib.qattn_swa_bf16.restype = i32
    lib.qattn_swa_bf16.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, i32, i32, i32, vp, sz, vp]
    lib.ql_attn_plan.restype = i32
    lib.ql_attn_plan.argtypes = [i32, i32, i32, i32, i32, i32, i32, ctypes.POINTER(ctypes.c_int)]
    for fn in (lib.ql_plan_first_chunk, lib.ql_plan_chunk_owner):
        fn.restype = ctypes.c_uint32
        fn.argtypes = [ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32]
    lib.ql_plan_chain_split.restype = i32
    lib.ql_plan_chain_split.argtypes = [i32, i32, i32, i32, ctypes.POINTER(ctypes.c_uint32)]
    lib.ql_debug_set_owner_extra.restype = None
    lib.ql_debug_set_owner_extra.argtypes = [i32]
    lib.ql_debug_set_wait_budget_ns.restype = None
    lib.ql_debug_set_wait_budget_ns.argtypes = [ctypes.c_uint64]
    lib.ql_debug_no_release.restype = None
    lib.ql_debug_no_release.argtypes = [i32]
    lib.ql_debug_set_timeline.restype = None
    lib.ql_debug_set_timeline.argtypes = [vp]
    lib.ql_debug_set_ablate.restype = None
    lib.ql_debug_set_ablate.argtypes = [i32]
    lib.ql_debug_timeline_enabled.restype = i32
    lib.ql_debug_timeline_enabled.argtypes = []
    lib.ql_launch_count.restype = ctypes.c_uint64
    lib.ql_launch_count.argtypes = []
    _lib = lib
    return lib


def _check(status: int, where: str):
    if status != QL_OK:
        raise QlError(status, where)


def _ptr(t):
    return None if t is None else t.data_ptr()


def _stream(stream=None):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


# ---- host-only helpers ------------------------------------------------------------------------

def ql_packed_bytes(K: int, N: int, g: int) -> int:
    return load().ql_packed_bytes(K, N, g)


def ql_workspace_bytes(M_max: int, N_max: int) -> int:
    return load().ql_workspace_bytes(M_max, N_max)


def ql_select_path(M: int, K: int, N: int, g: int) -> int:
    return load().ql_select_path(M, K, N, g)


def ql_launch_count() -> int:
    return int(load().ql_launch_count())


def ql_debug_set_wait_budget_ns(ns: int) -> None:
    load().ql_debug_set_wait_budget_ns(ns)


def ql_plan_chain_split(n_tiles: int, n_groups: int, ncta: int, cta: int) -> dict:
    """The chunks [lo, hi) thread block `cta` gets of a chained operation, whether the split is the
    aligned one, and the last thread block of the tile of chunk hi - 1."""
    r = (ctypes.c_uint32 * 4)()
    _check(load().ql_plan_chain_split(n_tiles, n_groups, ncta, cta, r), "ql_plan_chain_split")
    return {"lo": int(r[0]), "hi": int(r[1]), "aligned": bool(r[2]), "last_cta": int(r[3])}


def ql_debug_set_owner_extra(chunks: int = -1) -> None:
    load().ql_debug_set_owner_extra(chunks)


def ql_debug_no_release(fused_op: int) -> None:
    load().ql_debug_no_release(fused_op)


def ql_debug_set_timeline(buf) -> None:
    """buf: an int64 device tensor of at least 160 * n_ops * 8 elements, or None."""
    load().ql_debug_set_timeline(None if buf is None else buf.data_ptr())


def ql_debug_set_ablate(mask: int) -> None:
    load().ql_debug_set_ablate(mask)


def ql_debug_timeline_enabled() -> bool:
    return bool(load().ql_debug_timeline_enabled())


# ---- device entry points ----------------------------------------------------------------------

def new_workspace(M_max: int, N_max: int, device="cuda", stream=None):
    """Allocate (with torch) and initialise a workspace for calls with M <= M_max, N <= N_max."""
    import torch
    nbytes = ql_workspace_bytes(M_max, N_max)
    if nbytes == 0:
        raise QlError(QL_ERR_SHAPE, "ql_workspace_bytes")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
    ql_workspace_init(ws, stream)
    return ws


def ql_workspace_init(ws, stream=None):
    _check(load().ql_workspace_init(ws.data_ptr(), ws.numel(), _stream(stream)), "ql_workspace_init")


def ql_device_status(ws, stream=None) -> int:
    out = ctypes.c_int(-1)
    _check(load().ql_device_status(ws.data_ptr(), ctypes.byref(out), _stream(stream)), "ql_device_status")
    return out.value


def ql_device_status_raw(ws, stream=None) -> int:
    out = ctypes.c_int(-1)
    _check(load().ql_device_status_raw(ws.data_ptr(), ctypes.byref(out), _stream(stream)), "ql_device_status_raw")
    return out.value


def qpack_w4_g128(wq, scale, zero, K: int, N: int, g: int, packed=None, stream=None):
    """wq int32/uint32-as-int32 [K/8,N], scale int16 (bf16 bits) [K/g,N], zero uint8 [K/g,N] or None.
    Returns the packed uint8 tensor (allocated with torch if not given)."""
    import torch
    if packed is None:
        packed = torch.empty(ql_packed_bytes(K, N, g), dtype=torch.uint8, device=wq.device)
    _check(load().qpack_w4_g128(wq.data_ptr(), scale.data_ptr(), _ptr(zero), K, N, g, packed.data_ptr(),
                                packed.numel(), _stream(stream)), "qpack_w4_g128")
    return packed


def qrequant_pack_w4(w, scale, zero, K: int, N: int, g: int, packed=None, stream=None):
    """w int16 (bf16 bits) [K,N], scale int16 (bf16 bits) [K/g,N], zero uint8 [K/g,N] or None.
    Returns the packed uint8 tensor holding the re-quantised codes."""
    import torch
    if packed is None:
        packed = torch.empty(ql_packed_bytes(K, N, g), dtype=torch.uint8, device=w.device)
    _check(load().qrequant_pack_w4(w.data_ptr(), scale.data_ptr(), _ptr(zero), K, N, g, packed.data_ptr(),
                                   packed.numel(), _stream(stream)), "qrequant_pack_w4")
    return packed


def qlinear_w4a16(packed, X, Y, argmax_out, M: int, K: int, N: int, g: int, ws, stream=None, path: int = QL_PATH_AUTO):
    lib = load()
    if path == QL_PATH_AUTO:
        st = lib.qlinear_w4a16(packed.data_ptr(), X.data_ptr(), _ptr(Y), _ptr(argmax_out), M, K, N, g,
                               ws.data_ptr(), ws.numel(), _stream(stream))
    else:
        st = lib.qlinear_w4a16_path(packed.data_ptr(), X.data_ptr(), _ptr(Y), _ptr(argmax_out), M, K, N, g,
                                    ws.data_ptr(), ws.numel(), _stream(stream), path)
    _check(st, "qlinear_w4a16")


def make_ops(op_list):
    """list of dicts -> ctypes array of ql_op (tensors are turned into device pointers)."""
    arr = (ql_op * len(op_list))()
    for o, d in zip(arr, op_list):
        o.kind = d["kind"]
        o.M, o.K, o.N, o.g = d["M"], d.get("K", 0), d["N"], d.get("g", 0)
        o.ld_in, o.ld_out, o.reserved = d["ld_in"], d["ld_out"], 0
        for name in ("packed", "in0", "in1", "out", "argmax_out", "draft_ids", "accept_out"):
            t = d.get(name)
            setattr(o, name, None if t is None else (t if isinstance(t, int) else t.data_ptr()))
    return arr


def qlinear_stack_w4a16(ops, ws, stream=None):
    """ops: a ctypes array from make_ops (kept alive by the caller for the duration of the call)."""
    _check(load().qlinear_stack_w4a16(ops, len(ops), ws.data_ptr(), ws.numel(), _stream(stream)),
           "qlinear_stack_w4a16")


def qlinear_stack_w4a16_host(ops, host_in, dev_in, dev_out, host_out, ws, stream=None):
    """host_in/host_out: CPU tensors (pinned for asynchronous copies); synchronises the stream."""
    in_b = 0 if host_in is None else host_in.numel() * host_in.element_size()
    out_b = 0 if host_out is None else host_out.numel() * host_out.element_size()
    _check(load().qlinear_stack_w4a16_host(ops, len(ops), _ptr(host_in), _ptr(dev_in), in_b, _ptr(dev_out),
                                           _ptr(host_out), out_b, ws.data_ptr(), ws.numel(), _stream(stream)),
           "qlinear_stack_w4a16_host")


def qlinear_w4a16_static(packed, X, Y, argmax_out, M: int, K: int, N: int, g: int, stream=None):
    """qlinear_w4a16 with the library's own static scratch array instead of a workspace: for callers
    that have no way to allocate device memory.  M <= 16, N <= 16384."""
    _check(load().qlinear_w4a16_static(packed.data_ptr(), X.data_ptr(), _ptr(Y), _ptr(argmax_out), M, K, N, g,
                                       _stream(stream)), "qlinear_w4a16_static")


def ql_static_status(stream=None) -> int:
    out = ctypes.c_int(-1)
    _check(load().ql_static_status(ctypes.byref(out), _stream(stream)), "ql_static_status")
    return out.value


def ql_attn_workspace_bytes(Hq: int, Hkv: int) -> int:
    return int(load().ql_attn_workspace_bytes(Hq, Hkv))


def new_attn_workspace(Hq: int, Hkv: int, device="cuda", stream=None):
    """Allocate (with torch) and zero a workspace for qattn_swa_bf16."""
    import torch
    nbytes = ql_attn_workspace_bytes(Hq, Hkv)
    if nbytes == 0:
        raise QlError(QL_ERR_SHAPE, "ql_attn_workspace_bytes")
    ws = torch.empty(nbytes, dtype=torch.uint8, device=device)
    ql_workspace_init(ws, stream)
    return ws


def qattn_swa_bf16(Q, K, V, out, n_q: int, T: int, Hq: int, Hkv: int, d: int, p0: int, window: int, ws,
                   ld_q=None, ld_kv=None, ld_out=None, stream=None):
    """Q int16 (bf16 bits) [n_q,Hq,d], K / V [T,Hkv,d], out [n_q,Hq,d]; leading dimensions default to dense."""
    _check(load().qattn_swa_bf16(Q.data_ptr(), K.data_ptr(), V.data_ptr(), out.data_ptr(), n_q, T, Hq, Hkv, d, p0, window,
                                 Hq * d if ld_q is None else ld_q, Hkv * d if ld_kv is None else ld_kv,
                                 Hq * d if ld_out is None else ld_out, ws.data_ptr(), ws.numel(), _stream(stream)),
           "qattn_swa_bf16")
    return out


def ql_attn_plan(n_q: int, T: int, Hq: int, Hkv: int, d: int, p0: int, window: int) -> dict:
    """What qattn_swa_bf16 would do (no launch, no device needed)."""
    c = (ctypes.c_int * 4)()
    _check(load().ql_attn_plan(n_q, T, Hq, Hkv, d, p0, window, c), "ql_attn_plan")
    return dict(zip(["key_lo", "key_hi", "n_pieces", "sub_per_piece"], list(c)))


def ql_linear_plan(M: int, K: int, N: int, g: int, path: int = QL_PATH_AUTO) -> dict:
    """How qlinear_w4a16 would set up this linear (no launch, no device needed)."""
    c = (ctypes.c_int * 4)()
    _check(load().ql_linear_plan(M, K, N, g, path, c), "ql_linear_plan")
    return dict(zip(["path", "n_stages", "n_x", "x_phase"], list(c)))


def ql_stack_plan(ops, ws_ptr: int, ws_bytes: int) -> dict:
    """What qlinear_stack_w4a16 would launch for `ops` (a ctypes array from make_ops); no device needed."""
    c = (ctypes.c_int * 8)()
    _check(load().ql_stack_plan(ops, len(ops), ws_ptr, ws_bytes, c), "ql_stack_plan")
    names = ["stack_launches", "fused_ops", "dual_ops", "folded_glue", "independent", "single_linears", "single_glue", "batch_launches"]
    return dict(zip(names, list(c)))
