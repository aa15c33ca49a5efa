"""CPU oracle for the W4A16 group-quantised linear layer.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain definition that the CUDA library is checked against.  Only the
tests, the smoke check and the benchmark's cpu-baseline leg may import it; the product path never
does, and this file imports nothing from the product (it shares no code, table or constant with
the CUDA sources).

What it computes.  The paper's quantised target stores every linear layer as INT4 codes W_q under
frozen per-group scales s and runs it as activations times the dequantised weights s (.) W_q
(Section 2.1: the dequantised weights are the element-wise product of s and W_q, the per-group
scales are symmetric and frozen, the model is served as W4A16; Section 3.3: group-wise INT4 with
group size 128; Section 3.2: block size 16, i.e. M = 16 rows per verify step; Section 4: the
speculative step does not change the output, so the arg-max of the verify logits must be
reproduced exactly).  The paper gives no equation for
the layer beyond that, so the definition below is the plain one:

    q[k,n]   = (wq[k div 8, n] >> 4*(k mod 8)) & 15                (8 codes per word, low nibble first)
    w[k,n]   = float32(q[k,n] - z[k div g, n]) * float32(s[k div g, n])     (exact in fp32)
    Y[m,n]   = sum_k  float64(x[m,k]) * float64(w[k,n])            (fp64)

with bf16 x and s.  The symmetric case of the paper is z == 8; a free zero point 0..15 is the
generalisation the benchmark configurations use.  All floating point is fp64 except the fp32
dequantisation product, which is exact (|q-z| <= 15 needs 4 bits, a bf16 significand 8 bits).

Every function is pinned by tests/test_oracle_pins.py to something other than itself: a brute
force over exact rationals, hand-packed words, closed forms and invariants.  No function here is
"parity unpinned".
"""
from __future__ import annotations

import numpy as np

# --------------------------------------------------------------------------------------------
# number formats


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """bf16 bit pattern -> float64 of the same value (bf16 is the top half of an IEEE float32)."""
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def f64_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float64 -> bf16 bit pattern, one rounding, to nearest, ties to even (finite, normal range)."""
    a = np.asarray(a, dtype=np.float64)
    m, e = np.frexp(a)                       # a = m * 2**e, 0.5 <= |m| < 1
    m8 = np.rint(m * 256.0) / 256.0          # 8 significant bits; rint rounds half to even
    r = np.ldexp(m8, e).astype(np.float32)   # representable in bf16, hence exactly in float32
    return (r.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """float64 -> the nearest bf16 value, returned as float64."""
    return bf16_bits_to_f64(f64_to_bf16_bits(a))


# --------------------------------------------------------------------------------------------
# the linear layer (Section 2.1: s ⊙ W_q; Section 3.3: groups of g along K)


def unpack_codes(wq: np.ndarray) -> np.ndarray:
    """uint32 [K/8, N] -> uint8 codes [K, N]; code of row k sits at bits [4*(k%8), +4) of word k//8."""
    R, N = wq.shape
    q = np.empty((R, 8, N), dtype=np.uint8)
    for j in range(8):
        q[:, j, :] = (wq >> np.uint32(4 * j)) & np.uint32(0xF)
    return q.reshape(R * 8, N)


def dequant_f32(wq: np.ndarray, scale_bits: np.ndarray, zero: np.ndarray | None, g: int) -> np.ndarray:
    """Dequantised weights w[k,n] = (q - z) * s in float32 (Section 2.1).  zero=None means z == 8."""
    q = unpack_codes(wq).astype(np.int32)
    K, N = q.shape
    assert K % g == 0 and scale_bits.shape == (K // g, N)
    z = np.full((K // g, N), 8, dtype=np.int32) if zero is None else zero.astype(np.int32)
    assert z.shape == (K // g, N)
    d = q - np.repeat(z, g, axis=0)                                  # integers in [-15, 15]
    s64 = np.repeat(bf16_bits_to_f64(scale_bits), g, axis=0)
    w32 = d.astype(np.float32) * s64.astype(np.float32)
    # the fp32 product is exact; checked rather than assumed
    assert np.array_equal(w32.astype(np.float64), d.astype(np.float64) * s64)
    return w32


def qlinear_f64(x_bits: np.ndarray, wq: np.ndarray, scale_bits: np.ndarray, zero: np.ndarray | None,
                g: int, col_block: int | None = None) -> np.ndarray:
    """Y = X · dequant(Wq) in float64, [M, N].  `col_block` only bounds memory: output columns are
    independent, so computing them a block at a time changes no arithmetic."""
    x = bf16_bits_to_f64(x_bits)
    N = wq.shape[1]
    if col_block is None or col_block >= N:
        return x @ dequant_f32(wq, scale_bits, zero, g).astype(np.float64)
    y = np.empty((x.shape[0], N), dtype=np.float64)
    for c0 in range(0, N, col_block):
        c1 = min(N, c0 + col_block)
        zc = None if zero is None else zero[:, c0:c1]
        w = dequant_f32(np.ascontiguousarray(wq[:, c0:c1]), scale_bits[:, c0:c1], zc, g)
        y[:, c0:c1] = x @ w.astype(np.float64)
    return y


def argmax_rows(y: np.ndarray):
    """Greedy token per row (Section 4: lossless verification): lowest index of the row maximum,
    and the gap between the two largest entries of the row."""
    idx = np.argmax(y, axis=1)                       # numpy returns the first maximum
    top1 = y[np.arange(y.shape[0]), idx]
    rest = y.copy()
    rest[np.arange(y.shape[0]), idx] = -np.inf
    top2 = rest.max(axis=1) if y.shape[1] > 1 else np.full(y.shape[0], -np.inf)
    return idx.astype(np.int64), top1 - top2


def requant_codes(w_bits: np.ndarray, scale_bits: np.ndarray, zero: np.ndarray | None, g: int) -> np.ndarray:
    """Grid-preserving re-quantisation (Section 2.1: after distillation the updated BF16 weights are
    rounded back onto the same quantisation grid, which gives new INT4 codes under the original
    frozen scales).  For bf16 weights w[K,N], the frozen bf16 scales s[K/g,N] and zero points z
    (None: the symmetric grid, z = 8):
        code[k,n] = clamp( rne( float32(w[k,n]) / float32(s[k div g, n]) ) + z[k div g, n], 0, 15 )
    The quotient is the IEEE float32 division (correctly rounded), rne is round-half-to-even to an
    integer: the paper fixes neither, this is the precision the decision is taken in on both sides.
    Returns uint8 codes [K, N]."""
    w = bf16_bits_to_f64(w_bits).astype(np.float32)           # exact widening
    s = bf16_bits_to_f64(scale_bits).astype(np.float32)
    K, N = w.shape
    ng = K // g
    z = np.full((ng, N), 8, dtype=np.int64) if zero is None else zero.astype(np.int64)
    q = np.empty((K, N), dtype=np.uint8)
    for G in range(ng):
        quo = w[G * g:(G + 1) * g, :] / s[G:G + 1, :]           # float32 / float32 -> float32
        r = np.rint(quo).astype(np.int64)                        # half to even
        q[G * g:(G + 1) * g, :] = np.clip(r + z[G:G + 1, :], 0, 15).astype(np.uint8)
    return q


def accept_prefix(tokens, draft_ids):
    """Verification of a drafted block (Section 2.2: the target scores the whole block in one pass
    and keeps the longest prefix of drafted tokens it agrees with; Section 4: under greedy decoding
    this changes nothing in the output).  tokens[i] is the target's greedy token of row i,
    draft_ids[i] the drafted token that row i is to confirm.  Returns (a, bonus): a = number of
    leading rows with tokens[i] == draft_ids[i]; bonus = the target's own token of the first row that
    disagrees, tokens[a], or -1 if every row agrees (there is no row left to take it from).
    The paper states the rule in words only; which row confirms which drafted token is the
    caller's business (it builds draft_ids)."""
    a = 0
    for t, d in zip(tokens, draft_ids):
        if int(t) != int(d):
            break
        a += 1
    bonus = int(tokens[a]) if a < len(tokens) else -1
    return a, bonus


# --------------------------------------------------------------------------------------------
# the glue that chains linears in the 36-layer benchmark stack (not from the paper: the
# benchmark's stand-in for normalisation / attention / activation between projections)


def unit_rms(v: np.ndarray) -> np.ndarray:
    """Row-wise v / sqrt(mean(v^2)), float64."""
    v = np.asarray(v, dtype=np.float64)
    return v / np.sqrt(np.mean(v * v, axis=1, keepdims=True))


def silu(v: np.ndarray) -> np.ndarray:
    v = np.asarray(v, dtype=np.float64)
    return v / (1.0 + np.exp(-v))


def stack_layer_free_running(h_bits: np.ndarray, weights: dict, g: int = 128, q_dim: int = 4096):
    """One decoder layer of the benchmark stack, every activation rounded to bf16 where the
    library stores bf16:
        qkv = L(h); a = U(qkv[:, :q_dim]); o = L(a); r = U(o);
        gt = L(r); up = L(r); d = U(silu(gt) * up); dn = L(d); h' = U(dn)
    L = quantised linear with bf16 output, U = unit-RMS rescale with bf16 output (input: the
    bf16 values as stored).  Returns h' (bf16 bits) and the bf16 input of each linear."""
    def L(xb, name):
        w = weights[name]
        return f64_to_bf16_bits(qlinear_f64(xb, w["wq"], w["scale"], w["zero"], g))

    def U(v64):
        return f64_to_bf16_bits(unit_rms(v64))

    ins = {"qkv": h_bits}
    qkv = L(h_bits, "qkv")
    a = U(bf16_bits_to_f64(qkv[:, :q_dim]))
    ins["o"] = a
    o = L(a, "o")
    r = U(bf16_bits_to_f64(o))
    ins["gate"] = r
    ins["up"] = r
    gt = L(r, "gate")
    up = L(r, "up")
    d = U(silu(bf16_bits_to_f64(gt)) * bf16_bits_to_f64(up))
    ins["down"] = d
    dn = L(d, "down")
    return U(bf16_bits_to_f64(dn)), ins


# --------------------------------------------------------------------------------------------
# reference of the packed tile layout (written from the layout description, independently of
# the CUDA repack kernel).
#
# The packed buffer is a sequence of chunks, one per (column tile T of 128 columns, group G of g
# rows), ordered T-major: chunk (T, G) starts at byte (T*(K/g) + G) * CB, CB = 64*g + 320.
# Inside a chunk:
#   [0, 64*g)            weight words.  32-bit little-endian word number (c*128 + n)*4 + j,
#                        c in [0, g/32), n in [0,128), j in [0,4), holds the 8 codes of column
#                        128*T+n, rows k = g*G + 32*c + 8*j + i, i = 0..7; code i sits in nibble
#                        position (i >> 1) + 4*(i & 1)  (even i in the low half-word).
#   [64*g, 64*g+256)     128 bf16 scales of (G, 128*T+n), n ascending.
#   [64*g+256, +64)      128 zero points, 4 bits each: 32-bit word n >> 3, nibble n & 7.
#                        (symmetric weights store the constant 8 here.)
# There is no padding: the buffer has (N/128)*(K/g)*CB bytes.

TILE_N = 128


def chunk_bytes(g: int) -> int:
    return 64 * g + 320


def packed_bytes(K: int, N: int, g: int) -> int:
    return (N // TILE_N) * (K // g) * chunk_bytes(g)


def pack_ref(wq: np.ndarray, scale_bits: np.ndarray, zero: np.ndarray | None, g: int) -> np.ndarray:
    """Boundary tensors -> packed buffer (uint8), by the layout description above."""
    q = unpack_codes(wq)
    K, N = q.shape
    assert N % TILE_N == 0 and K % g == 0 and g % 32 == 0
    nt, ng, cb = N // TILE_N, K // g, chunk_bytes(g)
    z = np.full((ng, N), 8, dtype=np.uint8) if zero is None else zero
    out = np.zeros(nt * ng * cb, dtype=np.uint8)
    nib_pos = [(i >> 1) + 4 * (i & 1) for i in range(8)]
    for T in range(nt):
        for G in range(ng):
            base = (T * ng + G) * cb
            blk = q[G * g:(G + 1) * g, T * TILE_N:(T + 1) * TILE_N]       # [g, 128]
            # blk[32c + 8j + i, n]  ->  word (c, n, j), nibble nib_pos[i]
            b = blk.reshape(g // 32, 4, 8, TILE_N).astype(np.uint32)       # [c, j, i, n]
            words = np.zeros((g // 32, TILE_N, 4), dtype=np.uint32)       # [c, n, j]
            for i in range(8):
                words |= np.transpose(b[:, :, i, :], (0, 2, 1)) << np.uint32(4 * nib_pos[i])
            out[base:base + 64 * g] = words.reshape(-1).view(np.uint8)
            sc = np.ascontiguousarray(scale_bits[G, T * TILE_N:(T + 1) * TILE_N], dtype=np.uint16)
            out[base + 64 * g: base + 64 * g + 256] = sc.view(np.uint8)
            zz = z[G, T * TILE_N:(T + 1) * TILE_N].astype(np.uint32).reshape(16, 8)
            zw = np.zeros(16, dtype=np.uint32)
            for i in range(8):
                zw |= zz[:, i] << np.uint32(4 * i)
            out[base + 64 * g + 256: base + cb] = zw.view(np.uint8)
    return out


def unpack_ref(packed: np.ndarray, K: int, N: int, g: int):
    """Packed buffer -> (wq uint32 [K/8,N], scale bits [K/g,N], zero uint8 [K/g,N]); inverse of pack_ref."""
    nt, ng, cb = N // TILE_N, K // g, chunk_bytes(g)
    assert packed.dtype == np.uint8 and packed.size == nt * ng * cb
    q = np.zeros((K, N), dtype=np.uint8)
    scale = np.zeros((ng, N), dtype=np.uint16)
    zero = np.zeros((ng, N), dtype=np.uint8)
    for T in range(nt):
        for G in range(ng):
            base = (T * ng + G) * cb
            words = packed[base:base + 64 * g].view(np.uint32).reshape(g // 32, TILE_N, 4)
            for c in range(g // 32):
                for j in range(4):
                    for i in range(8):
                        pos = (i >> 1) + 4 * (i & 1)
                        q[G * g + 32 * c + 8 * j + i, T * TILE_N:(T + 1) * TILE_N] = \
                            (words[c, :, j] >> np.uint32(4 * pos)) & np.uint32(0xF)
            scale[G, T * TILE_N:(T + 1) * TILE_N] = packed[base + 64 * g: base + 64 * g + 256].view(np.uint16)
            zw = packed[base + 64 * g + 256: base + cb].view(np.uint32)
            for n in range(TILE_N):
                zero[G, T * TILE_N + n] = (zw[n >> 3] >> np.uint32(4 * (n & 7))) & np.uint32(0xF)
    # re-pack codes into the boundary word format: code of row k at bits [4*(k%8), +4) of word k//8
    wq = np.zeros((K // 8, N), dtype=np.uint32)
    qq = q.reshape(K // 8, 8, N).astype(np.uint32)
    for j in range(8):
        wq |= qq[:, j, :] << np.uint32(4 * j)
    return wq, scale, zero


# --------------------------------------------------------------------------------------------
# comparison metrics used by the parity tests (the tolerances themselves are written in the tests)


def rel_frobenius(y_test: np.ndarray, y_ref: np.ndarray) -> float:
    den = float(np.linalg.norm(y_ref))
    num = float(np.linalg.norm(np.asarray(y_test, dtype=np.float64) - y_ref))
    return num / den if den > 0 else (0.0 if num == 0 else float("inf"))


def max_scaled_abs_err(y_test: np.ndarray, y_ref: np.ndarray) -> float:
    """max over elements of |test - ref| / (|ref| + 1)."""
    return float(np.max(np.abs(np.asarray(y_test, dtype=np.float64) - y_ref) / (np.abs(y_ref) + 1.0)))
