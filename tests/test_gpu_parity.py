"""GPU parity tests: the CUDA library, called through its C ABI, against the CPU oracle on the
same seeded inputs.  Bars: repack bit-exact; GEMM relative Frobenius error <= 2e-3 and
|err| <= 1e-2 * (|ref| + 1) per element on the bf16 output against the fp64 oracle; arg-max exact
on rows whose fp64 top-2 gap is >= 1e-3."""
import numpy as np
import pytest
import torch

import qsynth
from oracle import w4a16_oracle as orc
from gpu_util import (check_against_oracle, dev_u16, dev_u32, dev_u8, host_u16, pack_on_device, run_linear)

pytestmark = pytest.mark.gpu


# ---- repack: bit exact ------------------------------------------------------------------------

@pytest.mark.parametrize("K,N,g,sym", [(512, 256, 128, False), (256, 384, 64, False), (384, 128, 128, True),
                                        (2560, 1280, 128, False), (1024, 2560, 64, True)])
def test_qpack_bit_exact(ql, K, N, g, sym):
    d = qsynth.make_linear([90, K, N, g], 0, K, N, g, symmetric=sym, with_x=False)
    ref = orc.pack_ref(d["wq"], d["scale"], None if sym else d["zero"], g)
    got = pack_on_device(ql, d, zero_none=sym).cpu().numpy()
    assert got.size == ref.size == ql.ql_packed_bytes(K, N, g)
    assert np.array_equal(got, ref)
    wq, sc, z = orc.unpack_ref(got, K, N, g)
    assert np.array_equal(wq, d["wq"]) and np.array_equal(sc, d["scale"]) and np.array_equal(z, d["zero"])


def test_qpack_explicit_eights_equal_null_zero(ql):
    d = qsynth.make_linear(91, 0, 256, 256, 128, symmetric=True, with_x=False)
    a = pack_on_device(ql, d, zero_none=True).cpu().numpy()
    b = pack_on_device(ql, d, zero_none=False).cpu().numpy()
    assert np.array_equal(a, b)


# ---- GEMM parity ------------------------------------------------------------------------------

PATHS = [pytest.param(2, id="mma"), pytest.param(3, id="tcgen05")]


def _skip_unless_supported(ql, path, M, K, N, g):
    """The tcgen05 kernel needs the X columns a CTA touches to fit in shared memory.  Up to 16 rows
    they always do for these shapes; above, the plan for the forced path says whether they fit."""
    if path != ql.QL_PATH_TC5:
        return
    try:
        ql.ql_linear_plan(M, K, N, g, ql.QL_PATH_TC5)
    except ql.QlError:
        pytest.skip("X does not fit in shared memory for the tcgen05 path at this shape")


def _parity(ql, d, path=0, argmax=False):
    M, K, N, g = d["M"], d["K"], d["N"], d["g"]
    _skip_unless_supported(ql, path, M, K, N, g)
    packed = pack_on_device(ql, d)
    y_bits, am = run_linear(ql, packed, d["x"], M, K, N, g, want_argmax=argmax, path=path)
    y64 = orc.qlinear_f64(d["x"], d["wq"], d["scale"], d["zero"], g, col_block=16384)
    rf, me = check_against_oracle(y_bits, y64, f"M{M} K{K} N{N} g{g}")
    return y_bits, am, y64, rf, me


@pytest.mark.parametrize("path", PATHS)
def test_config0_single_small_linear(ql, path):
    _parity(ql, qsynth.config0(), path)


@pytest.mark.parametrize("M,K,N,g,sym", [
    (16, 512, 1024, 128, False),      # several tiles, one group run per CTA
    (3, 1024, 384, 128, False),       # ragged M, split-K inside tiles
    (5, 640, 2560, 64, False),        # g = 64
    (17, 768, 512, 128, True),        # M just over one 16-row tile, symmetric
    (63, 512, 640, 64, False),        # largest padded M, ragged
    (64, 1280, 256, 128, False),
    (1, 2560, 128, 128, False),       # a single column tile split over many CTAs
    (8, 128, 19456, 128, False),      # one group, many tiles (no split-K at all)
    (16, 4096, 2560, 128, False),     # o-proj shape
    (32, 2560, 6144, 64, True),
])
@pytest.mark.parametrize("path", PATHS)
def test_linear_parity_shapes(ql, M, K, N, g, sym, path):
    d = qsynth.make_linear([92, M, K, N, g, int(sym)], M, K, N, g, symmetric=sym)
    _parity(ql, d, path)


@pytest.mark.parametrize("path", PATHS)
def test_config1_mlp_linears_full_size(ql, path):
    cfg = qsynth.config1()
    for name in ("gate", "up", "down"):
        _, _, _, rf, me = _parity(ql, cfg[name], path)
        print(f"config1 {name}: relF {rf:.3e} max_scaled {me:.3e}")


@pytest.mark.parametrize("path", PATHS)
def test_exact_case_power_of_two_scales_integer_x(ql, path):
    """All partial sums are multiples of 2^-3 below 2^24, so fp32 accumulation is exact in any
    order: the output must be bit-identical to the rounded oracle, and the arg-max identical."""
    M, K, N, g = 16, 1024, 512, 128
    rng = np.random.default_rng(5)
    codes = rng.integers(0, 16, (K, N), dtype=np.uint8)
    zero = rng.integers(0, 16, (K // g, N), dtype=np.uint8)
    xi = rng.integers(-2, 3, (M, K))
    d = dict(wq=qsynth.pack_codes_k8(codes), scale=np.full((K // g, N), 0x3E00, dtype=np.uint16), zero=zero,
             x=qsynth.f32_to_bf16_bits(xi.astype(np.float32)), M=M, K=K, N=N, g=g)
    packed = pack_on_device(ql, d)
    y_bits, am = run_linear(ql, packed, d["x"], M, K, N, g, want_argmax=True, path=path)
    y64 = orc.qlinear_f64(d["x"], d["wq"], d["scale"], d["zero"], g)
    assert np.array_equal(y_bits, orc.f64_to_bf16_bits(y64))
    idx, _ = orc.argmax_rows(y64)
    assert np.array_equal(am.astype(np.int64), idx)


@pytest.mark.parametrize("path", PATHS)
def test_zero_weights_give_exact_zero(ql, path):
    M, K, N, g = 7, 512, 256, 128
    d = qsynth.make_linear(93, M, K, N, g)
    d["wq"] = qsynth.pack_codes_k8(np.repeat(d["zero"], g, axis=0))
    packed = pack_on_device(ql, d)
    y_bits, _ = run_linear(ql, packed, d["x"], M, K, N, g, path=path)
    assert np.all((y_bits & 0x7FFF) == 0)


@pytest.mark.parametrize("path", PATHS)
def test_one_hot_rows_read_back_weights(ql, path):
    """X = e_k selects row k of the dequantised matrix: pins the k order of the packed layout and
    the group a row belongs to, through the GPU path."""
    K, N, g = 512, 256, 128
    d = qsynth.make_linear(94, 0, K, N, g, with_x=False)
    ks = [0, 1, 7, 8, 31, 32, 127, 128, 255, 256, 300, 511, 129, 64, 33, 200]
    x = np.zeros((16, K), dtype=np.uint16)
    for m, k in enumerate(ks):
        x[m, k] = 0x3F80
    packed = pack_on_device(ql, d)
    y_bits, _ = run_linear(ql, packed, x, 16, K, N, g, path=path)
    w = orc.dequant_f32(d["wq"], d["scale"], d["zero"], g).astype(np.float64)
    assert np.array_equal(y_bits, orc.f64_to_bf16_bits(w[ks, :]))


@pytest.mark.parametrize("path", PATHS)
def test_run_to_run_bit_identical(ql, path):
    d = qsynth.make_linear(95, 16, 2560, 1280, 128)
    packed = pack_on_device(ql, d)
    ws = ql.new_workspace(16, 1280)
    a, am_a = run_linear(ql, packed, d["x"], 16, 2560, 1280, 128, ws=ws, want_argmax=True, path=path)
    for _ in range(3):
        b, am_b = run_linear(ql, packed, d["x"], 16, 2560, 1280, 128, ws=ws, want_argmax=True, path=path)
        assert np.array_equal(a, b) and np.array_equal(am_a, am_b)


def test_workspace_reuse_across_shapes(ql):
    """One workspace, calls of different shapes back to back: control words must come back to zero."""
    ws = ql.new_workspace(64, 4096)
    for (M, K, N, g) in [(16, 512, 1024, 128), (64, 256, 4096, 64), (1, 2560, 128, 128), (16, 512, 1024, 128)]:
        d = qsynth.make_linear([96, M, K, N, g], M, K, N, g)
        packed = pack_on_device(ql, d)
        y_bits, am = run_linear(ql, packed, d["x"], M, K, N, g, ws=ws, want_argmax=True)
        y64 = orc.qlinear_f64(d["x"], d["wq"], d["scale"], d["zero"], g)
        check_against_oracle(y_bits, y64)
    assert int(ws[:16640].to(torch.int32).abs().sum().item()) == 0


# ---- LM head: arg-max -------------------------------------------------------------------------

def _check_argmax(am, y64, what):
    idx, gap = orc.argmax_rows(y64)
    safe = gap >= 1e-3
    excluded = int(np.count_nonzero(~safe))
    print(f"{what}: {excluded} of {len(idx)} rows excluded (fp64 top-2 gap < 1e-3), min gap {gap.min():.3e}")
    assert np.array_equal(am.astype(np.int64)[safe], idx[safe])
    assert np.all((am >= 0) & (am < y64.shape[1]))


@pytest.mark.parametrize("path", PATHS)
def test_argmax_small_vocab_and_ties(ql, path):
    M, K, N, g = 16, 512, 128 * 37, 128
    d = qsynth.make_linear(97, M, K, N, g)
    packed = pack_on_device(ql, d)
    y_bits, am = run_linear(ql, packed, d["x"], M, K, N, g, want_argmax=True, path=path)
    y64 = orc.qlinear_f64(d["x"], d["wq"], d["scale"], d["zero"], g)
    _check_argmax(am, y64, "vocab 4736")
    # argmax only (no Y buffer) gives the same tokens
    _, am2 = run_linear(ql, packed, d["x"], M, K, N, g, want_argmax=True, want_y=False, path=path)
    assert np.array_equal(am, am2)
    # exact ties: duplicate the columns of tile 3 into tile 20 -> the lower index must win
    wq, sc, z = d["wq"].copy(), d["scale"].copy(), d["zero"].copy()
    lo, hi = slice(3 * 128, 4 * 128), slice(20 * 128, 21 * 128)
    wq[:, hi], sc[:, hi], z[:, hi] = wq[:, lo], sc[:, lo], z[:, lo]
    sc[:, lo] = sc[:, lo] + np.uint16(0x100)      # x4: make these columns the row maxima (or minima)
    sc[:, hi] = sc[:, lo]
    d2 = dict(d, wq=wq, scale=sc, zero=z)
    packed2 = pack_on_device(ql, d2)
    _, am3 = run_linear(ql, packed2, d["x"], M, K, N, g, want_argmax=True, path=path)
    y64b = orc.qlinear_f64(d["x"], wq, sc, z, g)
    idx, _ = orc.argmax_rows(y64b)
    tied = (idx >= 3 * 128) & (idx < 4 * 128)
    assert tied.any()
    assert np.array_equal(am3.astype(np.int64)[tied], idx[tied])


@pytest.mark.parametrize("path", PATHS)
def test_config3_lm_head_full_size_argmax(ql, path):
    d = qsynth.config3()
    M, K, N, g = d["M"], d["K"], d["N"], d["g"]
    _skip_unless_supported(ql, path, M, K, N, g)
    packed = pack_on_device(ql, d)
    y_bits, am = run_linear(ql, packed, d["x"], M, K, N, g, want_argmax=True, path=path)
    y64 = orc.qlinear_f64(d["x"], d["wq"], d["scale"], d["zero"], g, col_block=8192)
    check_against_oracle(y_bits, y64, "LM head")
    _check_argmax(am, y64, "LM head 151936")
