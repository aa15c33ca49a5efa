"""The entry point for callers that cannot allocate device memory (an embedded callback, a
real-time loop, a plugin without access to the host program's allocator): qlinear_w4a16_static
keeps the kernel's scratch in a static device array of the library.  Its result must be the one of
the ordinary entry point on the same path, on two calls in a row (the second call finds the first
call's leftovers in the array)."""
import numpy as np
import pytest
import torch

import qsynth
from oracle import w4a16_oracle as orc
from gpu_util import check_against_oracle, dev_u16, host_u16, pack_on_device

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_point_matches_workspace_entry_point(ql):
    g = 128
    cases = [qsynth.make_linear([120, 0], 16, 1024, 2560, g), qsynth.make_linear([120, 1], 5, 2560, 1152, g)]
    for d in cases:
        M, K, N = d["M"], d["K"], d["N"]
        packed = pack_on_device(ql, d)
        X = dev_u16(d["x"])
        # reference: the ordinary entry point on the same compute path, with a caller-owned workspace
        ws = ql.new_workspace(M, N)
        y_ref = torch.zeros((M, N), dtype=torch.int16, device="cuda")
        tok_ref = torch.zeros((M,), dtype=torch.int32, device="cuda")
        ql.qlinear_w4a16(packed, X, y_ref, tok_ref, M, K, N, g, ws, path=ql.QL_PATH_MMA)
        torch.cuda.synchronize()
        y64 = orc.qlinear_f64(d["x"], d["wq"], d["scale"], d["zero"], g)
        for call in range(2):
            y = torch.full((M, N), 0x7FC0, dtype=torch.int16, device="cuda")
            tok = torch.full((M,), -1, dtype=torch.int32, device="cuda")
            ql.qlinear_w4a16_static(packed, X, y, tok, M, K, N, g)
            torch.cuda.synchronize()
            assert ql.ql_static_status() == ql.QL_OK
            check_against_oracle(host_u16(y), y64, f"static call {call}")
            assert torch.equal(y, y_ref), f"call {call}: differs from the workspace entry point"
            assert torch.equal(tok, tok_ref)


def test_static_scratch_entry_point_g64_and_tokens_only(ql):
    """Group size 64, and the form that returns only the greedy tokens (Y == NULL); the launch
    counter of the library counts these calls like any other."""
    M, K, N, g = 16, 1024, 1280, 64
    d = qsynth.make_linear([120, 2], M, K, N, g)
    packed = pack_on_device(ql, d)
    X = dev_u16(d["x"])
    ws = ql.new_workspace(M, N)
    y_ref = torch.zeros((M, N), dtype=torch.int16, device="cuda")
    tok_ref = torch.zeros((M,), dtype=torch.int32, device="cuda")
    ql.qlinear_w4a16(packed, X, y_ref, tok_ref, M, K, N, g, ws, path=ql.QL_PATH_MMA)
    torch.cuda.synchronize()
    y64 = orc.qlinear_f64(d["x"], d["wq"], d["scale"], d["zero"], g)
    check_against_oracle(host_u16(y_ref), y64, "workspace entry point, g=64")
    before = ql.ql_launch_count()
    for call in range(2):
        y = torch.full((M, N), 0x7FC0, dtype=torch.int16, device="cuda")
        ql.qlinear_w4a16_static(packed, X, y, None, M, K, N, g)
        tok = torch.full((M,), -1, dtype=torch.int32, device="cuda")
        ql.qlinear_w4a16_static(packed, X, None, tok, M, K, N, g)
        torch.cuda.synchronize()
        assert ql.ql_static_status() == ql.QL_OK
        assert torch.equal(y, y_ref) and torch.equal(tok, tok_ref), f"call {call}"
    assert ql.ql_launch_count() - before == 4


def test_static_scratch_entry_point_rejects_sizes_beyond_its_array(ql):
    P = 0x10000
    lib = ql.load()
    assert lib.qlinear_w4a16_static(P, P, P, None, 17, 512, 256, 128, None) == ql.QL_ERR_WORKSPACE
    assert lib.qlinear_w4a16_static(P, P, P, None, 16, 512, 128 * 129, 128, None) == ql.QL_ERR_WORKSPACE
    assert lib.qlinear_w4a16_static(P, P, P, None, 16, 500, 256, 128, None) == ql.QL_ERR_SHAPE
    assert lib.qlinear_w4a16_static(None, P, P, None, 16, 512, 256, 128, None) == ql.QL_ERR_NULL
