"""GPU parity of qlinear_stack_w4a16 on lists of INDEPENDENT linears (no two share a buffer other
than inputs both only read).  Such a list is not a chain: the launcher lays the operations' chunks
end to end and cuts them into one contiguous piece per thread block; the X operand follows the
chunks through a ring of slots.
Every output is compared with the oracle element by element at the library's tolerances."""
import numpy as np
import pytest
import torch

import qsynth
from oracle import w4a16_oracle as orc
from gpu_util import check_against_oracle, dev_u16, host_u16, pack_on_device

pytestmark = pytest.mark.gpu


def run_independent(ql, lins, M, g, n_max, shared_x=None, runs=1):
    packed = [pack_on_device(ql, d, zero_none=d.get("symmetric", False)) for d in lins]
    xs = [dev_u16(d["x"]) if shared_x is None else shared_x for d in lins]
    ys = [torch.full((M, d["N"]), 0x7FC0, dtype=torch.int16, device="cuda") for d in lins]   # NaN pattern
    ops = [dict(kind=ql.QL_OP_LINEAR, M=M, K=d["K"], N=d["N"], g=g, ld_in=d["K"], ld_out=d["N"], packed=p, in0=x, out=y)
           for d, p, x, y in zip(lins, packed, xs, ys)]
    ws = ql.new_workspace(M, n_max)
    arr = ql.make_ops(ops)
    plan = ql.ql_stack_plan(arr, ws.data_ptr(), ws.numel())
    outs = []
    for _ in range(runs):
        for y in ys:
            y.fill_(0x7FC0)
        before = ql.ql_launch_count()
        ql.qlinear_stack_w4a16(arr, ws)
        torch.cuda.synchronize()
        assert ql.ql_launch_count() - before == plan["stack_launches"]
        assert ql.ql_device_status(ws) == ql.QL_OK
        outs.append([host_u16(y).copy() for y in ys])
    return plan, outs


@pytest.mark.parametrize("name", ["gate", "qkv", "o"])
def test_bench_shapes_one_stream(ql, name):
    """The benchmark's gate/up, fused-qkv and o shapes at M=16, g=128, four distinct weight sets each:
    one launch, the operations run as one stream of chunks (thread blocks' pieces cross operation
    boundaries and split tiles in the middle)."""
    M, g = 16, 128
    K, N = qsynth.LAYER_SHAPES[name]
    lins = [qsynth.make_linear([77, i, K, N], M, K, N, g) for i in range(4)]
    plan, outs = run_independent(ql, lins, M, g, N, runs=2)
    assert plan["stack_launches"] == 1 and plan["batch_launches"] == 1 and plan["fused_ops"] == 4 and plan["single_linears"] == 0
    for i, d in enumerate(lins):
        y64 = orc.qlinear_f64(d["x"], d["wq"], d["scale"], d["zero"], g, col_block=4096)
        rf, me = check_against_oracle(outs[0][i], y64, f"{name} #{i}")
        print(f"{name} #{i}: relF {rf:.3e} max scaled {me:.3e}")
        assert np.array_equal(outs[0][i], outs[1][i]), "second run differs"


@pytest.mark.parametrize("n_lin", [3, 7])
def test_down_shape_long_k(ql, n_lin):
    """down (K = 76 groups): the X operand of a whole tile (330 KB) cannot be resident, it comes through
    the ring of X slots chunk by chunk.  Three linears give every thread block a piece of 31 chunks,
    seven a piece of 72: both shorter than a tile, the pieces cross tile and operation boundaries."""
    M, g = 16, 128
    K, N = qsynth.LAYER_SHAPES["down"]
    lins = [qsynth.make_linear([78, i, K, N], M, K, N, g) for i in range(n_lin)]
    plan, outs = run_independent(ql, lins, M, g, N, runs=2)
    assert plan["stack_launches"] == 1 and plan["batch_launches"] == 1 and plan["independent"] == n_lin - 1
    for i, d in enumerate(lins):
        y64 = orc.qlinear_f64(d["x"], d["wq"], d["scale"], d["zero"], g, col_block=4096)
        check_against_oracle(outs[0][i], y64, f"down #{i} of {n_lin}")
        assert np.array_equal(outs[0][i], outs[1][i]), "second run differs"


def test_small_shapes_ragged_m_g64(ql):
    """M = 5, g = 64, mixed small shapes (some with fewer chunks than thread blocks), symmetric and
    asymmetric zero points, one shared input for the operations of equal K."""
    M, g = 5, 64
    shapes = [(512, 1024), (512, 256), (512, 2560), (512, 128), (512, 1280), (512, 384)]
    lins = [qsynth.make_linear([79, i, K, N], M, K, N, g, symmetric=(i % 2 == 1)) for i, (K, N) in enumerate(shapes)]
    x = lins[0]["x"]
    for d in lins:
        d["x"] = x
    plan, outs = run_independent(ql, lins, M, g, 2560, shared_x=dev_u16(x), runs=1)
    assert plan["batch_launches"] == 1
    for i, d in enumerate(lins):
        y64 = orc.qlinear_f64(x, d["wq"], d["scale"], d["zero"], g)
        check_against_oracle(outs[0][i], y64, f"small #{i}")


def test_exact_case_bit_identical(ql):
    """Power-of-two scales and small-integer activations: every partial sum is exact in fp32 in any
    order, so each output must equal the rounded oracle bit for bit."""
    M, K, g = 16, 1024, 128
    rng = np.random.default_rng(15)
    lins = []
    for i, N in enumerate([512, 1536, 256]):
        codes = rng.integers(0, 16, (K, N), dtype=np.uint8)
        zero = rng.integers(0, 16, (K // g, N), dtype=np.uint8)
        xi = rng.integers(-2, 3, (M, K))
        lins.append(dict(wq=qsynth.pack_codes_k8(codes), scale=np.full((K // g, N), 0x3E00, dtype=np.uint16), zero=zero,
                         x=qsynth.f32_to_bf16_bits(xi.astype(np.float32)), M=M, K=K, N=N, g=g))
    plan, outs = run_independent(ql, lins, M, g, 1536)
    assert plan["batch_launches"] == 1
    for i, d in enumerate(lins):
        y64 = orc.qlinear_f64(d["x"], d["wq"], d["scale"], d["zero"], g)
        assert np.array_equal(outs[0][i], orc.f64_to_bf16_bits(y64)), f"operation {i}"
