"""Pins for the CPU oracle: each check compares the oracle with something that is not the
oracle - exact rational brute force, hand-packed words, closed forms, invariants.

Citations are to the paper's sections: the dequantised weight is scale times code (Section 2.1),
groups of 128 along K and symmetric codes (Section 3.3), 16-row verify blocks (Section 3.2),
exact greedy verification (Section 4)."""
from fractions import Fraction

import numpy as np
import pytest

import qsynth
from oracle import w4a16_oracle as orc


def _bf16_fraction(bits: int) -> Fraction:
    """Value of a bf16 bit pattern as an exact rational, from the IEEE field definition."""
    s = (bits >> 15) & 1
    e = (bits >> 7) & 0xFF
    m = bits & 0x7F
    if e == 0:
        v = Fraction(m, 128) * Fraction(2) ** (-126)
    else:
        v = (1 + Fraction(m, 128)) * Fraction(2) ** (e - 127)
    return -v if s else v


def _brute(x_bits, wq, scale_bits, zero, g):
    """Scalar triple loop over exact rationals; every input is a dyadic rational."""
    M, K = x_bits.shape
    N = wq.shape[1]
    out = [[Fraction(0)] * N for _ in range(M)]
    for m in range(M):
        for n in range(N):
            acc = Fraction(0)
            for k in range(K):
                code = (int(wq[k // 8, n]) >> (4 * (k % 8))) & 15
                z = 8 if zero is None else int(zero[k // g, n])
                w = (code - z) * _bf16_fraction(int(scale_bits[k // g, n]))
                acc += _bf16_fraction(int(x_bits[m, k])) * w
            out[m][n] = acc
    return out


@pytest.mark.parametrize("M,K,N,g,sym", [(3, 32, 8, 8, False), (2, 16, 5, 16, False), (1, 32, 4, 16, True),
                                          (2, 64, 3, 32, False)])
def test_brute_force_exact_rationals(M, K, N, g, sym):
    d = qsynth.make_linear([77, M, K, N, g], M, K, N, g, symmetric=sym)
    zero = None if sym else d["zero"]
    y = orc.qlinear_f64(d["x"], d["wq"], d["scale"], zero, g)
    ref = _brute(d["x"], d["wq"], d["scale"], zero, g)
    for m in range(M):
        for n in range(N):
            r = float(ref[m][n])          # correctly rounded conversion of the exact value
            assert abs(y[m, n] - r) <= 4 * np.spacing(abs(r)) + 1e-300, (m, n, y[m, n], r)


def test_symmetric_is_zero_point_eight():
    d = qsynth.make_linear(5, 2, 32, 8, 16, symmetric=True)
    assert np.all(d["zero"] == 8)
    a = orc.qlinear_f64(d["x"], d["wq"], d["scale"], None, 16)
    b = orc.qlinear_f64(d["x"], d["wq"], d["scale"], d["zero"], 16)
    assert np.array_equal(a, b)


def test_nibble_order_hand_packed():
    # word 0x76543210: code j at bits [4j, 4j+4) -> rows 0..7 carry codes 0..7 (low nibble first)
    wq = np.array([[0x76543210, 0xFEDCBA98], [0x00000001, 0xF0000000]], dtype=np.uint32)
    q = orc.unpack_codes(wq)
    assert q.shape == (16, 2)
    assert list(q[:8, 0]) == [0, 1, 2, 3, 4, 5, 6, 7]
    assert list(q[:8, 1]) == [8, 9, 10, 11, 12, 13, 14, 15]
    assert list(q[8:, 0]) == [1, 0, 0, 0, 0, 0, 0, 0]
    assert list(q[8:, 1]) == [0, 0, 0, 0, 0, 0, 0, 15]
    # and the generator's packer is the inverse
    assert np.array_equal(qsynth.pack_codes_k8(q), wq)


def test_one_hot_rows_read_back_dequantised_weights_at_group_boundaries():
    K, N, g = 64, 6, 16
    d = qsynth.make_linear(11, 1, K, N, g)
    for k in (0, g - 1, g, 2 * g - 1, 2 * g, K - 1):
        x = np.zeros((1, K), dtype=np.uint16)
        x[0, k] = 0x3F80                                        # bf16 1.0
        y = orc.qlinear_f64(x, d["wq"], d["scale"], d["zero"], g)
        for n in range(N):
            code = (int(d["wq"][k // 8, n]) >> (4 * (k % 8))) & 15
            want = (code - int(d["zero"][k // g, n])) * float(_bf16_fraction(int(d["scale"][k // g, n])))
            assert y[0, n] == want


def test_power_of_two_scales_integer_activations_exact():
    # scale 2^-3, x in {-2..2}: every product and partial sum is an integer multiple of 2^-3
    M, K, N, g = 4, 256, 16, 128
    rng = np.random.default_rng(3)
    codes = rng.integers(0, 16, (K, N), dtype=np.uint8)
    zero = rng.integers(0, 16, (K // g, N), dtype=np.uint8)
    xi = rng.integers(-2, 3, (M, K))
    scale = np.full((K // g, N), 0x3E00, dtype=np.uint16)       # bf16 0.125
    x = qsynth.f32_to_bf16_bits(xi.astype(np.float32))
    y = orc.qlinear_f64(x, qsynth.pack_codes_k8(codes), scale, zero, g)
    want = xi.astype(np.int64) @ (codes.astype(np.int64) - np.repeat(zero.astype(np.int64), g, axis=0))
    assert np.array_equal(y * 8.0, want.astype(np.float64))


def test_all_ones_x_gives_scaled_integer_column_sums():
    K, N, g = 256, 12, 64
    d = qsynth.make_linear(21, 1, K, N, g)
    x = np.full((3, K), 0x3F80, dtype=np.uint16)
    y = orc.qlinear_f64(x, d["wq"], d["scale"], d["zero"], g)
    for n in range(N):
        tot = Fraction(0)
        for G in range(K // g):
            csum = sum((int(d["wq"][k // 8, n]) >> (4 * (k % 8))) & 15 for k in range(G * g, (G + 1) * g))
            tot += _bf16_fraction(int(d["scale"][G, n])) * (csum - g * int(d["zero"][G, n]))
        assert abs(y[0, n] - float(tot)) <= 8 * np.spacing(abs(float(tot)))
        assert y[1, n] == y[0, n] == y[2, n]


def test_zero_weights_give_zero():
    K, N, g = 128, 8, 32
    d = qsynth.make_linear(31, 2, K, N, g)
    codes = np.repeat(d["zero"], g, axis=0)                      # q == z everywhere
    y = orc.qlinear_f64(d["x"], qsynth.pack_codes_k8(codes), d["scale"], d["zero"], g)
    assert np.all(y == 0.0)


def test_invariants():
    M, K, N, g = 3, 128, 10, 32
    d = qsynth.make_linear(41, M, K, N, g)
    y = orc.qlinear_f64(d["x"], d["wq"], d["scale"], d["zero"], g)
    # doubling every scale (exponent +1) doubles Y exactly
    y2 = orc.qlinear_f64(d["x"], d["wq"], d["scale"] + np.uint16(0x80), d["zero"], g)
    assert np.array_equal(y2, 2.0 * y)
    # permuting columns of (Wq, scale, zero) permutes Y
    perm = np.random.default_rng(0).permutation(N)
    yp = orc.qlinear_f64(d["x"], d["wq"][:, perm], d["scale"][:, perm], d["zero"][:, perm], g)
    assert np.array_equal(yp, y[:, perm])
    # additivity over a split of K at a group boundary
    k1 = 2 * g
    ya = orc.qlinear_f64(d["x"][:, :k1], d["wq"][:k1 // 8], d["scale"][:2], d["zero"][:2], g)
    yb = orc.qlinear_f64(d["x"][:, k1:], d["wq"][k1 // 8:], d["scale"][2:], d["zero"][2:], g)
    assert np.allclose(ya + yb, y, rtol=0, atol=1e-12)
    # adding 1 to every code and zero point of a group (no clamp) leaves Y unchanged
    codes = orc.unpack_codes(d["wq"]).astype(np.int32)
    zero = d["zero"].astype(np.int32)
    codes = np.clip(codes, 0, 14)
    zero = np.clip(zero, 0, 14)
    y0 = orc.qlinear_f64(d["x"], qsynth.pack_codes_k8(codes.astype(np.uint8)), d["scale"], zero.astype(np.uint8), g)
    y1 = orc.qlinear_f64(d["x"], qsynth.pack_codes_k8((codes + 1).astype(np.uint8)), d["scale"],
                         (zero + 1).astype(np.uint8), g)
    assert np.array_equal(y0, y1)
    # linear in X: Y(2x) = 2 Y(x)
    yx2 = orc.qlinear_f64(d["x"] + np.uint16(0x80), d["wq"], d["scale"], d["zero"], g)
    assert np.array_equal(yx2, 2.0 * y)
    # column blocking changes nothing
    yb = orc.qlinear_f64(d["x"], d["wq"], d["scale"], d["zero"], g, col_block=3)
    assert np.array_equal(yb, y)


def test_dequant_matches_scalar_definition():
    K, N, g = 64, 7, 32
    d = qsynth.make_linear(51, 1, K, N, g)
    w = orc.dequant_f32(d["wq"], d["scale"], d["zero"], g)
    assert w.dtype == np.float32 and w.shape == (K, N)
    for k in (0, 1, 7, 8, 31, 32, 63):
        for n in range(N):
            code = (int(d["wq"][k // 8, n]) >> (4 * (k % 8))) & 15
            want = (code - int(d["zero"][k // g, n])) * _bf16_fraction(int(d["scale"][k // g, n]))
            assert Fraction(float(w[k, n])) == want


def test_bf16_rounding_known_values_and_independent_implementation():
    # exact values, ties to even, from the format definition (8 significant bits)
    cases = {1.0: 0x3F80, -2.0: 0xC000, 1.0 + 2.0 ** -8: 0x3F80, 1.0 + 3 * 2.0 ** -8: 0x3F82,
             1.0 + 2.0 ** -8 + 2.0 ** -20: 0x3F81, 0.0: 0x0000, 3.140625: 0x4049, 65280.0: 0x477F}
    for v, bits in cases.items():
        assert int(orc.f64_to_bf16_bits(np.array([v]))[0]) == bits, v
        assert float(orc.bf16_bits_to_f64(np.array([bits], dtype=np.uint16))[0]) == pytest.approx(
            float(_bf16_fraction(bits)), abs=0)
    # against the generator's integer bit-trick rounding on float32-representable values
    a = np.random.default_rng(1).standard_normal(20000).astype(np.float32) * np.float32(37.0)
    assert np.array_equal(orc.f64_to_bf16_bits(a.astype(np.float64)), qsynth.f32_to_bf16_bits(a))
    for bits in (0x0001 << 7, 0x3F80, 0x4049, 0xC2F7):
        assert float(orc.bf16_bits_to_f64(np.array([bits], dtype=np.uint16))[0]) == float(_bf16_fraction(bits))


def test_argmax_lowest_index_and_gap():
    y = np.array([[1.0, 5.0, 5.0, 2.0], [-3.0, -1.0, -2.0, -1.5], [7.0, 1.0, 2.0, 6.5]])
    idx, gap = orc.argmax_rows(y)
    assert list(idx) == [1, 1, 0]
    assert list(gap) == [0.0, 0.5, 0.5]


def test_glue_closed_forms():
    u = orc.unit_rms(np.array([[3.0, 4.0], [1.0, 1.0], [-2.0, 0.0]]))
    assert np.allclose(u[0], [3 / np.sqrt(12.5), 4 / np.sqrt(12.5)], rtol=1e-15)
    assert np.allclose(u[1], [1.0, 1.0]) and np.allclose(u[2], [-np.sqrt(2.0), 0.0])
    assert np.allclose(np.mean(orc.unit_rms(np.random.default_rng(0).standard_normal((4, 100))) ** 2, axis=1), 1.0)
    v = np.linspace(-6, 6, 25)
    assert orc.silu(np.array([0.0]))[0] == 0.0
    assert np.allclose(orc.silu(v) - orc.silu(-v), v, atol=1e-15)         # x*sigmoid(x) - (-x)*sigmoid(-x) = x
    assert abs(orc.silu(np.array([1.0]))[0] - 0.7310585786300049) < 1e-15  # 1/(1+e^-1)


# ---- packed layout reference ---------------------------------------------------------------

def _layout_locate(K, N, g, k, n):
    """Byte offset and nibble (0 = low) of weight (k, n), straight from the layout description."""
    T, nn = divmod(n, 128)
    G, r = divmod(k, g)
    c, r = divmod(r, 32)
    j, i = divmod(r, 8)
    cb = 64 * g + 320
    base = (T * (K // g) + G) * cb
    word = (c * 128 + nn) * 4 + j
    pos = (i >> 1) + 4 * (i & 1)
    return base + 4 * word + pos // 2, pos % 2


@pytest.mark.parametrize("g", [64, 128])
def test_pack_ref_single_code_lands_where_the_layout_says(g):
    K, N = 2 * g, 256
    scale = np.zeros((K // g, N), dtype=np.uint16)
    zero = np.zeros((K // g, N), dtype=np.uint8)
    for (k, n, code) in [(0, 0, 15), (1, 0, 9), (7, 3, 5), (8, 127, 1), (33, 128, 6), (g - 1, 255, 3),
                         (g, 17, 12), (2 * g - 1, 200, 7), (g + 40, 129, 10)]:
        codes = np.zeros((K, N), dtype=np.uint8)
        codes[k, n] = code
        p = orc.pack_ref(qsynth.pack_codes_k8(codes), scale, zero, g)
        assert p.size == orc.packed_bytes(K, N, g) == (N // 128) * (K // g) * (64 * g + 320)
        byte, hi = _layout_locate(K, N, g, k, n)
        nz = np.flatnonzero(p)
        assert list(nz) == [byte], (k, n, nz, byte)
        assert int(p[byte]) == (code << 4 if hi else code)


@pytest.mark.parametrize("g", [64, 128])
def test_pack_ref_scale_and_zero_positions(g):
    K, N = g, 256
    codes = np.zeros((K, N), dtype=np.uint8)
    scale = np.zeros((1, N), dtype=np.uint16)
    zero = np.zeros((1, N), dtype=np.uint8)
    scale[0, 130] = 0xBEEF
    zero[0, 141] = 0xB
    p = orc.pack_ref(qsynth.pack_codes_k8(codes), scale, zero, g)
    cb = 64 * g + 320
    base = 1 * cb                                   # column tile 1, group 0
    assert p[base + 64 * g + 2 * 2] == 0xEF and p[base + 64 * g + 2 * 2 + 1] == 0xBE
    zoff = base + 64 * g + 256 + 4 * (13 >> 3) + (13 & 7) // 2
    assert p[zoff] == (0xB << 4)                    # n & 7 = 5 -> odd nibble
    assert np.count_nonzero(p) == 3


@pytest.mark.parametrize("K,N,g,sym", [(256, 256, 128, False), (192, 128, 64, False), (128, 384, 64, True)])
def test_pack_ref_round_trip(K, N, g, sym):
    d = qsynth.make_linear([61, K, N, g], 0, K, N, g, symmetric=sym, with_x=False)
    p = orc.pack_ref(d["wq"], d["scale"], None if sym else d["zero"], g)
    wq, sc, z = orc.unpack_ref(p, K, N, g)
    assert np.array_equal(wq, d["wq"]) and np.array_equal(sc, d["scale"]) and np.array_equal(z, d["zero"])


# ---- what the tolerances leave room for ----------------------------------------------------

def test_tolerance_floor_of_bf16_output_rounding():
    """A perfect accumulator rounded once to bf16 already uses most of the 2e-3 Frobenius budget;
    the floor must be below the bar on the benchmark's own seeds or no bf16-output kernel can pass."""
    d = qsynth.config0()
    y = orc.qlinear_f64(d["x"], d["wq"], d["scale"], d["zero"], 128)
    f0 = orc.rel_frobenius(orc.round_to_bf16(y), y)
    d1 = qsynth.make_linear([1, 0], 16, 512, 1024, 128)
    y1 = orc.qlinear_f64(d1["x"], d1["wq"], d1["scale"], d1["zero"], 128)
    f1 = orc.rel_frobenius(orc.round_to_bf16(y1), y1)
    print(f"bf16 output-rounding floor: config0 {f0:.3e}, 16x512x1024 {f1:.3e}")
    assert f0 < 2e-3 and f1 < 2e-3
    assert orc.max_scaled_abs_err(orc.round_to_bf16(y1), y1) < 1e-2


# ---- the chained layer of the benchmark stack ---------------------------------------------------

def _fraction_to_bf16_bits(v: Fraction) -> int:
    """Round an exact rational to the nearest bf16 (ties to even), from the format definition
    (normal range only - enough for this test)."""
    if v == 0:
        return 0
    s = 1 if v < 0 else 0
    a = -v if s else v
    e = 0
    while a >= 2 ** (e + 1):
        e += 1
    while a < Fraction(2) ** e:
        e -= 1
    q = a / Fraction(2) ** (e - 7)                # in [128, 256)
    lo = q.numerator // q.denominator
    rem = q - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and (lo & 1)):
        lo += 1
    if lo == 256:
        lo, e = 128, e + 1
    assert 1 <= e + 127 <= 254
    return (s << 15) | ((e + 127) << 7) | (lo - 128)


def test_chained_layer_written_out_by_hand():
    """stack_layer_free_running against the chain spelled out step by step: every linear by the
    exact-rational brute force, every stored activation rounded to bf16 from the format definition,
    the glue with scalar Python math.  A wrong slice, gate and up swapped, or a missing rounding
    between two steps changes the bits."""
    import math
    M, hid, q_dim, kv, mlp, g = 2, 16, 8, 4, 32, 8
    shapes = {"qkv": (hid, q_dim + 2 * kv), "o": (q_dim, hid), "gate": (hid, mlp), "up": (hid, mlp), "down": (mlp, hid)}
    w = {nm: qsynth.stack_layer_weights(3, nm, g, shapes) for nm in shapes}
    h = qsynth.stack_h0(M, hid)

    def lin(x_bits, nm):                           # bf16 bits in, bf16 bits out
        exact = _brute(x_bits, w[nm]["wq"], w[nm]["scale"], w[nm]["zero"], g)
        return np.array([[_fraction_to_bf16_bits(v) for v in row] for row in exact], dtype=np.uint16)

    def unit(rows):                                # list of rows of Python floats -> bf16 bits
        out = []
        for r in rows:
            rms = math.sqrt(sum(v * v for v in r) / len(r))
            out.append([_fraction_to_bf16_bits(Fraction(v / rms)) for v in r])
        return np.array(out, dtype=np.uint16)

    val = lambda bits: [[float(_bf16_fraction(int(b))) for b in row] for row in bits]
    qkv = lin(h, "qkv")
    a = unit([r[:q_dim] for r in val(qkv)])        # the q slice stands in for the attention output
    o = lin(a, "o")
    r_ = unit(val(o))
    gt, up = lin(r_, "gate"), lin(r_, "up")
    prod = [[gv / (1.0 + math.exp(-gv)) * uv for gv, uv in zip(gr, ur)] for gr, ur in zip(val(gt), val(up))]
    d = unit(prod)
    dn = lin(d, "down")
    h_next = unit(val(dn))

    got, ins = orc.stack_layer_free_running(h, w, g, q_dim)
    assert np.array_equal(ins["qkv"], h) and np.array_equal(ins["o"], a)
    assert np.array_equal(ins["gate"], r_) and np.array_equal(ins["up"], r_)
    assert np.array_equal(ins["down"], d)
    assert np.array_equal(got, h_next)
    # the variants a plausible mistake would compute are different results
    swapped = unit([[uv / (1.0 + math.exp(-uv)) * gv for gv, uv in zip(gr, ur)] for gr, ur in zip(val(gt), val(up))])
    assert not np.array_equal(swapped, d)
    assert not np.array_equal(unit([r[q_dim - 4:2 * q_dim - 4] for r in val(qkv)]), a)


# ---- verification tail: accepted prefix and bonus token -------------------------------------------

def test_accept_prefix_planted_prefixes_and_brute_force():
    """Planted agreement prefixes of every length incl. 0, 1, 15 and 16 on a 16-row block; a
    disagreement later in the block must not matter; and all 2^8 agreement patterns of an 8-row
    block against the definition 'count leading ones'."""
    rng = np.random.default_rng(21)
    tokens = rng.integers(0, 151936, 16)
    for a in range(17):
        draft = tokens.copy()
        if a < 16:
            draft[a] = (tokens[a] + 7) % 151936                 # first disagreement at row a
            draft[a + 1:] = rng.integers(0, 151936, 15 - a)     # whatever follows is irrelevant
            if a + 2 < 16:
                draft[a + 2] = tokens[a + 2]                    # an agreement after the break does not count
        got = orc.accept_prefix(tokens, draft)
        assert got == (a, int(tokens[a]) if a < 16 else -1), (a, got)
    tok8 = np.arange(100, 108)
    for pattern in range(256):
        agree = [(pattern >> i) & 1 for i in range(8)]
        draft = [int(t) if ok else -5 for t, ok in zip(tok8, agree)]
        lead = 0
        while lead < 8 and agree[lead]:
            lead += 1
        assert orc.accept_prefix(tok8, draft) == (lead, int(tok8[lead]) if lead < 8 else -1)


def test_accept_prefix_uses_the_lowest_index_on_a_logit_tie():
    """With two equal row maxima the greedy token is the lower index (argmax_rows), and that is the
    token the drafted id has to match."""
    y = np.zeros((3, 6))
    y[0, [2, 4]] = 5.0          # tie -> token 2
    y[1, 3] = 1.0
    y[2, 5] = 2.0
    tokens, _ = orc.argmax_rows(y)
    assert orc.accept_prefix(tokens, [2, 3, 5]) == (3, -1)
    assert orc.accept_prefix(tokens, [4, 3, 5]) == (0, 2)


# ---- grid-preserving re-quantisation ---------------------------------------------------------------

def _fraction_to_f32(v: Fraction) -> Fraction:
    """Exact rational -> nearest IEEE float32 (ties to even), as an exact rational; normal range."""
    if v == 0:
        return Fraction(0)
    s, a, e = (-1 if v < 0 else 1), abs(v), 0
    while a >= 2 ** (e + 1):
        e += 1
    while a < Fraction(2) ** e:
        e -= 1
    q = a / Fraction(2) ** (e - 23)
    lo = q.numerator // q.denominator
    rem = q - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and (lo & 1)):
        lo += 1
    return s * lo * Fraction(2) ** (e - 23)


def _rne_int(v: Fraction) -> int:
    lo = v.numerator // v.denominator               # floor
    rem = v - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and (lo & 1)):
        lo += 1
    return lo


def test_requant_brute_force_exact_rationals():
    """Every element by exact rational arithmetic: the quotient rounded to float32 from its exact
    value, then to the nearest integer with ties to even, shifted by the zero point and clamped."""
    rng = np.random.default_rng(31)
    K, N, g = 32, 6, 16
    scale = qsynth.f32_to_bf16_bits(np.abs(rng.standard_normal((K // g, N), dtype=np.float32)) * np.float32(0.01) + np.float32(1e-3))
    zero = rng.integers(0, 16, (K // g, N), dtype=np.uint8)
    w = qsynth.f32_to_bf16_bits(rng.standard_normal((K, N), dtype=np.float32) * np.float32(0.08))
    for z in (zero, None):
        got = orc.requant_codes(w, scale, z, g)
        for k in range(K):
            for n in range(N):
                quo = _fraction_to_f32(_bf16_fraction(int(w[k, n])) / _bf16_fraction(int(scale[k // g, n])))
                zz = 8 if z is None else int(z[k // g, n])
                want = min(15, max(0, _rne_int(quo) + zz))
                assert int(got[k, n]) == want, (k, n)


def test_requant_hand_made_grid_ties_and_clamps():
    """Scale 2^-3, zero point 5: weights placed exactly on the grid come back as their codes; exact
    halves go to the even neighbour; values beyond the grid clamp to 0 and 15."""
    g = 8
    s = np.full((1, 1), 0x3E00, dtype=np.uint16)                # 2^-3
    z = np.full((1, 1), 5, dtype=np.uint8)
    vals = [(c - 5) / 8 for c in range(8)]                      # on the grid: codes 0..7
    w = qsynth.f32_to_bf16_bits(np.array(vals, dtype=np.float32).reshape(8, 1))
    assert orc.requant_codes(w, s, z, g)[:, 0].tolist() == list(range(8))
    halves = [0.5 / 8, 1.5 / 8, 2.5 / 8, -0.5 / 8, -1.5 / 8, 100.0, -100.0, 9.5 / 8]
    w = qsynth.f32_to_bf16_bits(np.array(halves, dtype=np.float32).reshape(8, 1))
    #            0.5->0   1.5->2   2.5->2   -0.5->-0  -1.5->-2  clamp  clamp  9.5->10
    assert orc.requant_codes(w, s, z, g)[:, 0].tolist() == [5, 7, 7, 5, 3, 15, 0, 15]


def test_requant_round_trip_of_dequantised_weights_with_power_of_two_scales():
    """With power-of-two scales the dequantised weights are exact in bf16, so re-quantising them
    returns the codes they came from (the grid is preserved)."""
    rng = np.random.default_rng(32)
    K, N, g = 64, 16, 32
    codes = rng.integers(0, 16, (K, N), dtype=np.uint8)
    zero = rng.integers(0, 16, (K // g, N), dtype=np.uint8)
    scale = np.full((K // g, N), 0x3D00, dtype=np.uint16)       # 2^-5
    w = orc.dequant_f32(qsynth.pack_codes_k8(codes), scale, zero, g)
    assert np.array_equal(orc.requant_codes(qsynth.f32_to_bf16_bits(w), scale, zero, g), codes)
