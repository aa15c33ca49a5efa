"""GPU parity of qlinear_stack_w4a16: every linear of the chained stack is checked teacher-forced
(the oracle recomputes it from the bf16 input the GPU actually fed it), the glue operations are
checked against the oracle within one bf16 unit in the last place."""
import numpy as np
import pytest
import torch

import qsynth
from oracle import w4a16_oracle as orc
from gpu_util import check_against_oracle, dev_u16, host_u16, pack_on_device

pytestmark = pytest.mark.gpu

NAMES = ("qkv", "o", "gate", "up", "down")


def build_stack(ql, n_layers, shapes, M, g, q_dim, layer_ids=None, lm_head=None, drafter=False):
    """Allocates activations, packs weights and returns (ops list, buffers, weights per layer)."""
    hid = shapes["qkv"][0]
    mlp = shapes["gate"][1]
    dev = "cuda"
    bufs = {"h": [torch.zeros((M, hid), dtype=torch.int16, device=dev) for _ in range(n_layers + 1)]}
    for nm, width in (("qkv", shapes["qkv"][1]), ("a", q_dim), ("o", hid), ("r", hid), ("gt", mlp), ("up", mlp),
                      ("d", mlp), ("dn", hid)):
        bufs[nm] = [torch.zeros((M, width), dtype=torch.int16, device=dev) for _ in range(n_layers)]
    ops, weights, packed_all = [], [], []
    L, U, SU = ql.QL_OP_LINEAR, ql.QL_OP_UNIT_RMS, ql.QL_OP_SILU_MUL_UNIT_RMS
    for l in range(n_layers):
        lid = l if layer_ids is None else layer_ids[l]
        gen = qsynth.drafter_layer_weights if drafter else qsynth.stack_layer_weights
        w = {nm: gen(lid, nm, g, shapes) for nm in NAMES}
        pk = {nm: pack_on_device(ql, w[nm], zero_none=drafter) for nm in NAMES}   # symmetric: no zero points passed
        weights.append(w)
        packed_all.append(pk)

        def lin(nm, x, y):
            K, N = shapes[nm]
            return dict(kind=L, M=M, K=K, N=N, g=g, ld_in=x.shape[1], ld_out=N, packed=pk[nm], in0=x, out=y)

        def glue(kind, a, b, out, N):
            return dict(kind=kind, M=M, N=N, ld_in=a.shape[1], ld_out=out.shape[1], in0=a, in1=b, out=out)

        B = {k: v[l] for k, v in bufs.items() if k != "h"}
        ops += [lin("qkv", bufs["h"][l], B["qkv"]),
                glue(U, B["qkv"], None, B["a"], q_dim),
                lin("o", B["a"], B["o"]),
                glue(U, B["o"], None, B["r"], hid),
                lin("gate", B["r"], B["gt"]),
                lin("up", B["r"], B["up"]),
                glue(SU, B["gt"], B["up"], B["d"], mlp),
                lin("down", B["d"], B["dn"]),
                glue(U, B["dn"], None, bufs["h"][l + 1], hid)]
    return ops, bufs, weights, packed_all


def check_layer(l, bufs, weights, shapes, g, q_dim):
    B = {k: host_u16(v[l]) for k, v in bufs.items() if k != "h"}
    h_in, h_out = host_u16(bufs["h"][l]), host_u16(bufs["h"][l + 1])
    w = weights[l]

    def lin_check(nm, x_bits, y_bits):
        y64 = orc.qlinear_f64(x_bits, w[nm]["wq"], w[nm]["scale"], w[nm]["zero"], g)
        return check_against_oracle(y_bits, y64, f"layer {l} {nm}")

    def ulp_close(got_bits, want64, what):
        want_bits = orc.f64_to_bf16_bits(want64)
        diff = np.abs(got_bits.astype(np.int32) - want_bits.astype(np.int32))
        # same sign assumed where it matters; allow one unit in the last place (fp32 vs fp64 glue math)
        assert diff.max() <= 1, f"{what}: {diff.max()} ulp"
        assert np.count_nonzero(diff) <= 0.02 * diff.size, f"{what}: {np.count_nonzero(diff)} elements differ"

    lin_check("qkv", h_in, B["qkv"])
    ulp_close(B["a"], orc.unit_rms(orc.bf16_bits_to_f64(B["qkv"][:, :q_dim])), "U(q)")
    lin_check("o", B["a"], B["o"])
    ulp_close(B["r"], orc.unit_rms(orc.bf16_bits_to_f64(B["o"])), "U(o)")
    lin_check("gate", B["r"], B["gt"])
    lin_check("up", B["r"], B["up"])
    ulp_close(B["d"], orc.unit_rms(orc.silu(orc.bf16_bits_to_f64(B["gt"])) * orc.bf16_bits_to_f64(B["up"])), "U(silu*up)")
    lin_check("down", B["d"], B["dn"])
    ulp_close(h_out, orc.unit_rms(orc.bf16_bits_to_f64(B["dn"])), "U(down)")


SMALL = {"qkv": (256, 768), "o": (512, 256), "gate": (256, 1152), "up": (256, 1152), "down": (1152, 256)}


@pytest.mark.parametrize("M,g", [(16, 128), (5, 64)])
def test_small_stack_teacher_forced(ql, M, g):
    n_layers, q_dim = 3, 512
    ops, bufs, weights, _pk = build_stack(ql, n_layers, SMALL, M, g, q_dim)
    bufs["h"][0].copy_(dev_u16(qsynth.stack_h0(M, 256)))
    ws = ql.new_workspace(M, 1152)
    arr = ql.make_ops(ops)
    ql.qlinear_stack_w4a16(arr, ws)
    torch.cuda.synchronize()
    assert ql.ql_device_status(ws) == ql.QL_OK
    for l in range(n_layers):
        check_layer(l, bufs, weights, SMALL, g, q_dim)
    # free-running drift against the oracle's own chain (reported, not gated beyond sanity)
    h = qsynth.stack_h0(M, 256)
    for l in range(n_layers):
        h, _ = orc.stack_layer_free_running(h, weights[l], g, q_dim)
    drift = orc.rel_frobenius(orc.bf16_bits_to_f64(host_u16(bufs["h"][n_layers])), orc.bf16_bits_to_f64(h))
    print(f"free-running drift after {n_layers} layers: {drift:.3e}")
    assert drift < 0.05


def test_full_size_layers_teacher_forced(ql):
    """The benchmark's layer shapes at M=16, g=128: three layers of the 36 (first, middle, last
    seed), chained, every linear checked teacher-forced."""
    M, g = 16, 128
    ops, bufs, weights, _pk = build_stack(ql, 3, qsynth.LAYER_SHAPES, M, g, qsynth.Q_DIM, layer_ids=[0, 17, 35])
    bufs["h"][0].copy_(dev_u16(qsynth.stack_h0(M)))
    ws = ql.new_workspace(M, qsynth.MLP_DIM)
    arr = ql.make_ops(ops)
    ql.qlinear_stack_w4a16(arr, ws)
    torch.cuda.synchronize()
    assert ql.ql_device_status(ws) == ql.QL_OK
    for l in range(3):
        check_layer(l, bufs, weights, qsynth.LAYER_SHAPES, g, qsynth.Q_DIM)


@pytest.mark.parametrize("g", [128, 64])
def test_full_size_layer_under_every_split(ql, g):
    """The split of a chained operation decides which thread blocks share a tile and in which
    order partial rows are added, never what is computed: one full-size layer under the even
    split, the aligned split without and with the owner's extra chunks, and an extra so large
    that it is clipped; every linear teacher-forced against the oracle each time."""
    M = 16
    ops, bufs, weights, _pk = build_stack(ql, 1, qsynth.LAYER_SHAPES, M, g, qsynth.Q_DIM, layer_ids=[3])
    ws = ql.new_workspace(M, qsynth.MLP_DIM)
    arr = ql.make_ops(ops)
    try:
        for extra in (-2, 0, 1, 4, 9, 1000):
            ql.ql_debug_set_owner_extra(extra)
            kt, kg = qsynth.LAYER_SHAPES["down"][1] // 128, qsynth.LAYER_SHAPES["down"][0] // g
            assert ql.ql_plan_chain_split(kt, kg, 148, 0)["aligned"] == (extra >= 0)
            for v in bufs.values():
                for t in v:
                    t.fill_(0x7FC0)                      # NaN: nothing of an earlier run can pass for a result
            bufs["h"][0].copy_(dev_u16(qsynth.stack_h0(M)))
            ql.qlinear_stack_w4a16(arr, ws)
            torch.cuda.synchronize()
            assert ql.ql_device_status(ws) == ql.QL_OK
            check_layer(0, bufs, weights, qsynth.LAYER_SHAPES, g, qsynth.Q_DIM)
    finally:
        ql.ql_debug_set_owner_extra(-1)


def test_nan_rows_propagate_through_split_tiles(ql):
    """Partial rows of split tiles signal themselves by not being the 'empty' bit pattern (an
    all-ones NaN).  Rows of X that are NaN - the canonical one and the all-ones one - must come out
    as NaN rows without stalling the exchange; the other rows still match the oracle."""
    M, g = 16, 128
    K, N = qsynth.LAYER_SHAPES["o"]
    lin = qsynth.make_linear([77, 3], M, K, N, g)
    x = lin["x"].copy()
    x[3, :] = 0x7FC0
    x[9, :] = 0xFFFF
    y = torch.zeros((M, N), dtype=torch.int16, device="cuda")
    ops = ql.make_ops([dict(kind=ql.QL_OP_LINEAR, M=M, K=K, N=N, g=g, ld_in=K, ld_out=N, packed=pack_on_device(ql, lin),
                            in0=dev_u16(x), out=y)])
    ws = ql.new_workspace(M, N)
    assert ql.ql_plan_chain_split(N // 128, K // g, 148, 0)["aligned"]
    for _ in range(2):
        ql.qlinear_stack_w4a16(ops, ws)
        torch.cuda.synchronize()
        assert ql.ql_device_status(ws) == ql.QL_OK
        got = host_u16(y)
        for r in (3, 9):
            assert np.all((got[r] & 0x7F80) == 0x7F80) and np.all((got[r] & 0x007F) != 0), f"row {r} is not NaN throughout"
        keep = [r for r in range(M) if r not in (3, 9)]
        want = orc.qlinear_f64(lin["x"], lin["wq"], lin["scale"], lin["zero"], g)
        check_against_oracle(got[keep], want[keep], "rows beside the NaN rows")


def test_drafter_layers_symmetric_full_size(ql):
    """The second workload: drafter layers (group-wise symmetric INT4, groups of 128, M = 16; paper
    Sections 3.2 and 3.3) through the same launcher, zero == NULL at the boundary.  Two of the five
    layers at full (synthetic) widths, chained, every linear checked teacher-forced."""
    M, g = 16, 128
    ops, bufs, weights, _pk = build_stack(ql, 2, qsynth.LAYER_SHAPES, M, g, qsynth.Q_DIM, layer_ids=[0, 4], drafter=True)
    bufs["h"][0].copy_(dev_u16(qsynth.stack_h0(M)))
    ws = ql.new_workspace(M, qsynth.MLP_DIM)
    arr = ql.make_ops(ops)
    ql.qlinear_stack_w4a16(arr, ws)
    torch.cuda.synchronize()
    assert ql.ql_device_status(ws) == ql.QL_OK
    assert all(np.all(w[nm]["zero"] == 8) for w in weights for nm in NAMES)
    for l in range(2):
        check_layer(l, bufs, weights, qsynth.LAYER_SHAPES, g, qsynth.Q_DIM)


def test_stack_host_entry_matches_device_entry(ql):
    M, g, q_dim = 16, 128, 512
    ops, bufs, weights, _pk = build_stack(ql, 2, SMALL, M, g, q_dim)
    h0 = qsynth.stack_h0(M, 256)
    ws = ql.new_workspace(M, 1152)
    arr = ql.make_ops(ops)
    bufs["h"][0].copy_(dev_u16(h0))
    ql.qlinear_stack_w4a16(arr, ws)
    torch.cuda.synchronize()
    want = host_u16(bufs["h"][2]).copy()
    bufs["h"][0].zero_()
    bufs["h"][2].zero_()
    host_in = torch.from_numpy(h0.view(np.int16).copy()).pin_memory()
    host_out = torch.zeros((M, 256), dtype=torch.int16).pin_memory()
    ql.qlinear_stack_w4a16_host(arr, host_in, bufs["h"][0], bufs["h"][2], host_out, ws)
    assert np.array_equal(host_out.numpy().view(np.uint16), want)


def test_independent_linears_in_one_stack_call(ql):
    """A list of linears that share no buffer may overlap inside the launcher; each result must
    still match the oracle, and a dependent linear placed after them must see their outputs."""
    M, g = 16, 128
    shapes = [(512, 1024), (1024, 512), (512, 1024), (256, 2560), (512, 1024), (1024, 512)]
    lins = [qsynth.make_linear([98, i, K, N], M, K, N, g) for i, (K, N) in enumerate(shapes)]
    packed = [pack_on_device(ql, d) for d in lins]
    xs = [dev_u16(d["x"]) for d in lins]
    ys = [torch.full((M, d["N"]), 0x7FC0, dtype=torch.int16, device="cuda") for d in lins]
    ops = [dict(kind=ql.QL_OP_LINEAR, M=M, K=d["K"], N=d["N"], g=g, ld_in=d["K"], ld_out=d["N"], packed=p, in0=x, out=y)
           for d, p, x, y in zip(lins, packed, xs, ys)]
    # a dependent tail: the last output (512 columns) feeds one more linear
    tail = qsynth.make_linear([98, 99], M, 512, 384, g)
    ptail = pack_on_device(ql, tail)
    ytail = torch.full((M, 384), 0x7FC0, dtype=torch.int16, device="cuda")
    ops.append(dict(kind=ql.QL_OP_LINEAR, M=M, K=512, N=384, g=g, ld_in=512, ld_out=384, packed=ptail, in0=ys[-1], out=ytail))
    ws = ql.new_workspace(M, 2560)
    arr = ql.make_ops(ops)
    for _ in range(2):
        ql.qlinear_stack_w4a16(arr, ws)
    torch.cuda.synchronize()
    assert ql.ql_device_status(ws) == ql.QL_OK
    for d, y in zip(lins, ys):
        y64 = orc.qlinear_f64(d["x"], d["wq"], d["scale"], d["zero"], g)
        check_against_oracle(host_u16(y), y64, f"independent {d['K']}x{d['N']}")
    y64 = orc.qlinear_f64(host_u16(ys[-1]), tail["wq"], tail["scale"], tail["zero"], g)
    check_against_oracle(host_u16(ytail), y64, "dependent tail")


def test_dependency_at_distance_three_over_small_operations(ql):
    """A large linear, two small independent ones that most thread blocks have no chunk of, then
    a linear that reads the first one's output: a thread block that skipped the small operations
    must still not read that output before every tile of it is finished."""
    M, g = 16, 128
    A = qsynth.make_linear([97, 0], M, 2560, 1024, g)          # 160 chunks: every thread block takes part
    B = qsynth.make_linear([97, 1], M, 1024, 1024, g)          # 64 chunks: fewer than thread blocks
    C = qsynth.make_linear([97, 2], M, 1024, 1024, g)
    D = qsynth.make_linear([97, 3], M, 1024, 2560, g)          # reads A's output
    pk = [pack_on_device(ql, d) for d in (A, B, C, D)]
    xa, xb, xc = dev_u16(A["x"]), dev_u16(B["x"]), dev_u16(C["x"])
    ya, yb, yc = (torch.full((M, 1024), 0x7FC0, dtype=torch.int16, device="cuda") for _ in range(3))
    yd = torch.full((M, 2560), 0x7FC0, dtype=torch.int16, device="cuda")
    lin = lambda d, p, x, y: dict(kind=ql.QL_OP_LINEAR, M=M, K=d["K"], N=d["N"], g=g, ld_in=d["K"], ld_out=d["N"], packed=p, in0=x, out=y)
    arr = ql.make_ops([lin(A, pk[0], xa, ya), lin(B, pk[1], xb, yb), lin(C, pk[2], xc, yc), lin(D, pk[3], ya, yd)])
    ws = ql.new_workspace(M, 2560)
    plan = ql.ql_stack_plan(arr, ws.data_ptr(), ws.numel())
    assert plan["stack_launches"] == 1 and plan["batch_launches"] == 0 and plan["independent"] == 0   # a chain: everybody waits
    for rep in range(5):
        ya.fill_(0x7FC0)
        yd.fill_(0x7FC0)
        ql.qlinear_stack_w4a16(arr, ws)
        torch.cuda.synchronize()
        assert ql.ql_device_status(ws) == ql.QL_OK
        y64 = orc.qlinear_f64(host_u16(ya), D["wq"], D["scale"], D["zero"], g)
        check_against_oracle(host_u16(yd), y64, f"D after A, repetition {rep}")
    for d, y in ((A, ya), (B, yb), (C, yc)):
        check_against_oracle(host_u16(y), orc.qlinear_f64(d["x"], d["wq"], d["scale"], d["zero"], g), "A/B/C")


def test_repeated_and_alternating_calls_with_one_workspace(ql):
    """A repeated call may reuse the staged descriptors; a different list in between, a changed
    pointer inside an otherwise equal list, or a re-initialised workspace must all be noticed."""
    M, g = 16, 128
    a = qsynth.make_linear([96, 0], M, 1024, 1536, g)
    b = qsynth.make_linear([96, 1], M, 1024, 1536, g)
    pa, pb = pack_on_device(ql, a), pack_on_device(ql, b)
    xa, xb = dev_u16(a["x"]), dev_u16(b["x"])
    ya, yb, yc = (torch.full((M, 1536), 0x7FC0, dtype=torch.int16, device="cuda") for _ in range(3))
    lin = lambda d, p, x, y: ql.make_ops([dict(kind=ql.QL_OP_LINEAR, M=M, K=1024, N=1536, g=g, ld_in=1024, ld_out=1536, packed=p, in0=x, out=y)])
    ops_a, ops_b, ops_a2 = lin(a, pa, xa, ya), lin(b, pb, xb, yb), lin(a, pa, xa, yc)
    ws = ql.new_workspace(M, 1536)
    want_a = orc.qlinear_f64(a["x"], a["wq"], a["scale"], a["zero"], g)
    want_b = orc.qlinear_f64(b["x"], b["wq"], b["scale"], b["zero"], g)
    n0 = ql.ql_launch_count()
    for ops, y, want in ((ops_a, ya, want_a), (ops_a, ya, want_a), (ops_b, yb, want_b), (ops_a, ya, want_a), (ops_a2, yc, want_a)):
        y.fill_(0x7FC0)
        ql.qlinear_stack_w4a16(ops, ws)
        torch.cuda.synchronize()
        check_against_oracle(host_u16(y), want, "alternating lists")
    ql.ql_workspace_init(ws)
    ya.fill_(0x7FC0)
    ql.qlinear_stack_w4a16(ops_a2, ws)          # same list as the last call, but the workspace was wiped
    ql.qlinear_stack_w4a16(ops_a, ws)
    torch.cuda.synchronize()
    assert ql.ql_device_status(ws) == ql.QL_OK
    check_against_oracle(host_u16(ya), want_a, "after re-initialisation")
    assert ql.ql_launch_count() - n0 == 7


@pytest.mark.parametrize("path_name", ["MMA", "TC5"])
def test_one_workspace_for_stack_and_single_launch_calls(ql, path_name):
    """The stack kernel leaves its (tagged) partial-row flags behind; the tile counters of the
    single-launch kernels must not see them, and the other way round."""
    M, g, K, N = 16, 128, 512, 9728                       # 76 tiles: more tiles than a thread block has flag words
    a = qsynth.make_linear([94, 0], M, K, N, g)
    pa, xa = pack_on_device(ql, a), dev_u16(a["x"])
    want = orc.qlinear_f64(a["x"], a["wq"], a["scale"], a["zero"], g)
    ws = ql.new_workspace(M, N)
    path = getattr(ql, "QL_PATH_" + path_name)
    y = torch.full((M, N), 0x7FC0, dtype=torch.int16, device="cuda")
    ops = ql.make_ops([dict(kind=ql.QL_OP_LINEAR, M=M, K=K, N=N, g=g, ld_in=K, ld_out=N, packed=pa, in0=xa, out=y)])
    for order in ("stack, single", "single, stack", "stack, stack, single"):
        for what in order.split(", "):
            y.fill_(0x7FC0)
            if what == "stack":
                ql.qlinear_stack_w4a16(ops, ws)
            else:
                ql.qlinear_w4a16(pa, xa, y, None, M, K, N, g, ws, path=path)
            torch.cuda.synchronize()
            assert ql.ql_device_status(ws) == ql.QL_OK
            check_against_oracle(host_u16(y), want, f"{what} call in the order [{order}]")


def test_full_verify_step_one_launch_sampled_layers(ql):
    """The benchmark's step at full size and in the launch configuration bench.py times: 36 layers
    + LM head with arg-max in ONE qlinear_stack_w4a16 call (one launch of the persistent kernel).
    Layers 0, 17 and 35 are checked teacher-forced (every linear and glue operation), the LM head
    through its arg-max against the oracle on the input the GPU fed it."""
    M, g = 16, 128
    ops, bufs, weights, _pk = build_stack(ql, qsynth.N_LAYERS, qsynth.LAYER_SHAPES, M, g, qsynth.Q_DIM)
    lm = qsynth.config3()
    lm_packed = pack_on_device(ql, lm)
    tokens = torch.full((M,), -1, dtype=torch.int32, device="cuda")
    ops.append(dict(kind=ql.QL_OP_LINEAR, M=M, K=qsynth.HIDDEN, N=qsynth.VOCAB, g=g, ld_in=qsynth.HIDDEN,
                    ld_out=qsynth.VOCAB, packed=lm_packed, in0=bufs["h"][qsynth.N_LAYERS], out=None, argmax_out=tokens))
    bufs["h"][0].copy_(dev_u16(qsynth.stack_h0(M)))
    ws = ql.new_workspace(M, qsynth.VOCAB)
    arr = ql.make_ops(ops)
    plan = ql.ql_stack_plan(arr, ws.data_ptr(), ws.numel())
    assert plan["stack_launches"] == 1 and plan["fused_ops"] == 4 * qsynth.N_LAYERS + 1 and plan["single_linears"] == 0
    before = ql.ql_launch_count()
    ql.qlinear_stack_w4a16(arr, ws)
    torch.cuda.synchronize()
    assert ql.ql_launch_count() - before == 1
    assert ql.ql_device_status(ws) == ql.QL_OK
    for l in (0, 17, 35):
        check_layer(l, bufs, weights, qsynth.LAYER_SHAPES, g, qsynth.Q_DIM)
    h_last = host_u16(bufs["h"][qsynth.N_LAYERS])
    y64 = orc.qlinear_f64(h_last, lm["wq"], lm["scale"], lm["zero"], g, col_block=8192)
    idx, gap = orc.argmax_rows(y64)
    safe = gap >= 1e-3
    print(f"LM head after 36 layers: {int((~safe).sum())} of {M} rows excluded (fp64 top-2 gap < 1e-3), min gap {gap.min():.3e}")
    assert np.array_equal(tokens.cpu().numpy().astype(np.int64)[safe], idx[safe])
    # a second run of the same step is bit-identical
    first = [host_u16(bufs["h"][qsynth.N_LAYERS]).copy(), tokens.cpu().numpy().copy()]
    ql.qlinear_stack_w4a16(arr, ws)
    torch.cuda.synchronize()
    assert np.array_equal(host_u16(bufs["h"][qsynth.N_LAYERS]), first[0]) and np.array_equal(tokens.cpu().numpy(), first[1])


def test_stack_with_strided_buffers(ql):
    """gate and up write the two halves of one wide buffer (leading dimension 2 x MLP), the glue and
    the down projection read them from there: leading dimensions differ from the logical widths."""
    M, g, hid, mlp = 16, 128, 256, 1152
    wg, wu, wd = (qsynth.make_linear([99, i], 0, K, N, g, with_x=False) for i, (K, N) in enumerate([(hid, mlp), (hid, mlp), (mlp, hid)]))
    pg, pu, pd = (pack_on_device(ql, w) for w in (wg, wu, wd))
    x = dev_u16(qsynth.make_x([99, 7], M, hid))
    gu = torch.zeros((M, 2 * mlp), dtype=torch.int16, device="cuda")
    d = torch.zeros((M, mlp + 64), dtype=torch.int16, device="cuda")          # padded rows
    y = torch.zeros((M, hid), dtype=torch.int16, device="cuda")
    up_ptr = gu.data_ptr() + 2 * mlp
    ops = [dict(kind=ql.QL_OP_LINEAR, M=M, K=hid, N=mlp, g=g, ld_in=hid, ld_out=2 * mlp, packed=pg, in0=x, out=gu),
           dict(kind=ql.QL_OP_LINEAR, M=M, K=hid, N=mlp, g=g, ld_in=hid, ld_out=2 * mlp, packed=pu, in0=x, out=up_ptr),
           dict(kind=ql.QL_OP_SILU_MUL_UNIT_RMS, M=M, N=mlp, ld_in=2 * mlp, ld_out=mlp + 64, in0=gu, in1=up_ptr, out=d),
           dict(kind=ql.QL_OP_LINEAR, M=M, K=mlp, N=hid, g=g, ld_in=mlp + 64, ld_out=hid, packed=pd, in0=d, out=y)]
    ws = ql.new_workspace(M, mlp)
    arr = ql.make_ops(ops)
    plan = ql.ql_stack_plan(arr, ws.data_ptr(), ws.numel())
    assert plan["dual_ops"] == 1 and plan["folded_glue"] == 1 and plan["stack_launches"] == 1
    ql.qlinear_stack_w4a16(arr, ws)
    torch.cuda.synchronize()
    assert ql.ql_device_status(ws) == ql.QL_OK
    xh, guh, dh, yh = host_u16(x), host_u16(gu), host_u16(d)[:, :mlp], host_u16(y)
    check_against_oracle(guh[:, :mlp], orc.qlinear_f64(xh, wg["wq"], wg["scale"], wg["zero"], g), "gate (strided)")
    check_against_oracle(guh[:, mlp:], orc.qlinear_f64(xh, wu["wq"], wu["scale"], wu["zero"], g), "up (strided)")
    want = orc.f64_to_bf16_bits(orc.unit_rms(orc.silu(orc.bf16_bits_to_f64(guh[:, :mlp])) * orc.bf16_bits_to_f64(guh[:, mlp:])))
    diff = np.abs(dh.astype(np.int32) - want.astype(np.int32))
    assert diff.max() <= 1 and np.count_nonzero(diff) <= 0.02 * diff.size
    check_against_oracle(yh, orc.qlinear_f64(dh, wd["wq"], wd["scale"], wd["zero"], g), "down (strided input)")
    assert np.all(host_u16(d)[:, mlp:] == 0)                                    # the padding columns stay untouched
