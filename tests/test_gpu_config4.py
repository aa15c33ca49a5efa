"""Parity at points of the M-sweep (configuration 4) at full size, through the calls the sweep
times: M in {1, 8, 64} x the three sweep shapes x g in {64, 128} x asymmetric / symmetric zero
points; plus the mode of the warp-level kernel that reloads X in phases (M = 64 with long K)."""
import numpy as np
import pytest
import torch

import qsynth
from oracle import w4a16_oracle as orc
from gpu_util import check_against_oracle, dev_u16, host_u16, pack_on_device, run_linear

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("sym", [False, True], ids=["asym", "sym"])
@pytest.mark.parametrize("g", [64, 128])
@pytest.mark.parametrize("shape_idx", [0, 1, 2])
def test_sweep_points_full_size(ql, shape_idx, g, sym):
    """The sweep's shapes at M = 1, 8 and 64 through both calls: qlinear_w4a16 (the path it selects)
    and a two-linear qlinear_stack_w4a16 list, which is what the sweep times (above 16 rows the
    launcher cuts every linear into slabs of 16 rows)."""
    K, N = qsynth.SWEEP_SHAPES[shape_idx]
    packed = None
    for M in (1, 8, 64):
        d = qsynth.config4_point(shape_idx, M, g, sym)
        if packed is None:
            packed = pack_on_device(ql, d, zero_none=sym)           # the weights do not depend on M
        y64 = orc.qlinear_f64(d["x"], d["wq"], d["scale"], d["zero"], g, col_block=4096)
        y_bits, _ = run_linear(ql, packed, d["x"], M, K, N, g)       # the path qlinear_w4a16 selects
        rf, me = check_against_oracle(y_bits, y64, f"shape {K}x{N} M{M} g{g} {'sym' if sym else 'asym'}")
        print(f"{K}x{N} M={M} g={g} {'sym' if sym else 'asym'}: path {ql.PATH_NAMES[ql.ql_select_path(M, K, N, g)]}, relF {rf:.3e}")
        X = dev_u16(d["x"])
        ys = [torch.full((M, N), 0x7FC0, dtype=torch.int16, device="cuda") for _ in range(2)]
        ws = ql.new_workspace(M, N)
        ops = ql.make_ops([dict(kind=ql.QL_OP_LINEAR, M=M, K=K, N=N, g=g, ld_in=K, ld_out=N, packed=packed, in0=X, out=y) for y in ys])
        plan = ql.ql_stack_plan(ops, ws.data_ptr(), ws.numel())
        assert plan["stack_launches"] == 1 and plan["batch_launches"] == 1 and plan["single_linears"] == 0
        assert plan["fused_ops"] == 2 * ((M + 15) // 16)
        ql.qlinear_stack_w4a16(ops, ws)
        torch.cuda.synchronize()
        assert ql.ql_device_status(ws) == ql.QL_OK
        for y in ys:
            check_against_oracle(host_u16(y), y64, f"stack list, shape {K}x{N} M{M} g{g} {'sym' if sym else 'asym'}")


@pytest.mark.parametrize("K,N", [(2560, 9728), (9728, 2560)])
def test_phased_x_mode_of_the_warp_level_kernel(ql, K, N):
    """At M = 64 the X columns of the groups a thread block touches do not fit beside the ring, so
    the warp-level MMA kernel reloads them every few chunks: the plan must say so, and the result
    must match the oracle."""
    M, g = 64, 128
    plan = ql.ql_linear_plan(M, K, N, g, ql.QL_PATH_MMA)
    assert plan["path"] == ql.QL_PATH_MMA and plan["x_phase"] > 0, plan
    d = qsynth.make_linear([44, K, N], M, K, N, g)
    packed = pack_on_device(ql, d)
    y_bits, am = run_linear(ql, packed, d["x"], M, K, N, g, want_argmax=True, path=ql.QL_PATH_MMA)
    y64 = orc.qlinear_f64(d["x"], d["wq"], d["scale"], d["zero"], g, col_block=4096)
    check_against_oracle(y_bits, y64, f"phased X {K}x{N}")
    idx, gap = orc.argmax_rows(y64)
    ok = gap >= 1e-3
    assert np.array_equal(am.astype(np.int64)[ok], idx[ok])
