"""The bounded waits of the persistent kernel, exercised without hanging or faulting anything: a
test hook makes the first operation of a two-operation chain keep its finished tiles to itself, so
the second operation's wait for it runs out of its (shortened) budget.  The launch must return, the
status word must say QL_ERR_DEVICE_TIMEOUT and name the polling site, and after ql_workspace_init
the same workspace must serve an ordinary call again."""
import numpy as np
import pytest
import torch

import qsynth
from oracle import w4a16_oracle as orc
from gpu_util import check_against_oracle, dev_u16, host_u16, pack_on_device

pytestmark = pytest.mark.gpu


def test_wait_runs_out_reports_and_recovers(ql):
    M, g = 16, 128
    a = qsynth.make_linear([55, 0], M, 512, 1024, g)
    b = qsynth.make_linear([55, 1], M, 1024, 512, g, with_x=False)
    pa, pb = pack_on_device(ql, a), pack_on_device(ql, b)
    x = dev_u16(a["x"])
    y1 = torch.zeros((M, 1024), dtype=torch.int16, device="cuda")
    y2 = torch.zeros((M, 512), dtype=torch.int16, device="cuda")
    ops = ql.make_ops([
        dict(kind=ql.QL_OP_LINEAR, M=M, K=512, N=1024, g=g, ld_in=512, ld_out=1024, packed=pa, in0=x, out=y1),
        dict(kind=ql.QL_OP_LINEAR, M=M, K=1024, N=512, g=g, ld_in=1024, ld_out=512, packed=pb, in0=y1, out=y2)])
    ws = ql.new_workspace(M, 1024)
    plan = ql.ql_stack_plan(ops, ws.data_ptr(), ws.numel())
    assert plan["stack_launches"] == 1 and plan["fused_ops"] == 2 and plan["independent"] == 0
    try:
        ql.ql_debug_set_wait_budget_ns(2_000_000)        # 2 ms instead of 2 s
        ql.ql_debug_no_release(0)                        # operation 0 never publishes its tiles
        ql.qlinear_stack_w4a16(ops, ws)
        torch.cuda.synchronize()                         # the kernel ends by itself
    finally:
        ql.ql_debug_no_release(-1)
        ql.ql_debug_set_wait_budget_ns(0)
    assert ql.ql_device_status(ws) == ql.QL_ERR_DEVICE_TIMEOUT
    raw = ql.ql_device_status_raw(ws)
    site = (raw >> 8) & 0xFF
    assert site == 7, f"expected the watcher's poll of the predecessor (site 7), got site {site}"
    # a launch on the workspace as the timeout left it (hook off, full 2 s budget) must not wait for
    # anything: it runs through at once and the status keeps reporting the timeout
    import time
    t0 = time.perf_counter()
    ql.qlinear_stack_w4a16(ops, ws)
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 1.0
    assert ql.ql_device_status(ws) == ql.QL_ERR_DEVICE_TIMEOUT
    # recovery: re-initialise the workspace, run the same list for real
    ql.ql_workspace_init(ws)
    y1.zero_(); y2.zero_()
    ql.qlinear_stack_w4a16(ops, ws)
    torch.cuda.synchronize()
    assert ql.ql_device_status(ws) == ql.QL_OK
    check_against_oracle(host_u16(y1), orc.qlinear_f64(a["x"], a["wq"], a["scale"], a["zero"], g), "first linear")
    check_against_oracle(host_u16(y2), orc.qlinear_f64(host_u16(y1), b["wq"], b["scale"], b["zero"], g), "second linear")
