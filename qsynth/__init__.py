"""Seeded synthetic inputs for the W4A16 linear (shared by the oracle side and the CUDA side).

This module only *draws and formats* inputs: random int4 codes, bf16 scales, int4 zero points and
bf16 activations, in the boundary formats of the library.  It holds none of the method's
arithmetic (no unpacking, no dequantisation, no matmul): the oracle and the CUDA path each
implement those on their own.

Formats (the library boundary):
  wq     uint32 [K/8, N]  row-major; word (r, n) holds the codes of k = 8r+j, column n,
                          at bits [4j, 4j+4)  (8 per word along K, low nibble first)
  scale  uint16 [K/g, N]  bf16 bit patterns
  zero   uint8  [K/g, N]  one code 0..15 per byte (constant 8 in the symmetric variant)
  x      uint16 [M, K]    bf16 bit patterns

Recipe per linear, one numpy PCG64 stream seeded with SeedSequence(entropy), draw order
codes -> scales -> zeros -> X:
  codes = integers(0, 16, (K, N))            uniform int4
  scale = bf16(|N(0,1)| * 0.01 + 1e-3)       float32 draw, rounded to nearest-even bf16
  zero  = integers(0, 16, (K/g, N))          (drawn even when symmetric, then replaced by 8,
                                              so X is the same for both zero modes)
  x     = bf16(N(0,1))                       float32 draw
These stand in for the trained checkpoint and prompts of the paper's experiments, which are
not available; the cost of the linear depends only on the shapes.
"""
from __future__ import annotations

import numpy as np

# "4B-class" decoder shapes used by every benchmark configuration.
HIDDEN = 2560
Q_DIM, KV_DIM = 4096, 1024
QKV_DIM = Q_DIM + 2 * KV_DIM  # 6144
MLP_DIM = 9728
VOCAB = 151936
N_LAYERS = 36
LINEAR_IDX = {"qkv": 0, "o": 1, "gate": 2, "up": 3, "down": 4}
LAYER_SHAPES = {  # name -> (K, N)
    "qkv": (HIDDEN, QKV_DIM),
    "o": (Q_DIM, HIDDEN),
    "gate": (HIDDEN, MLP_DIM),
    "up": (HIDDEN, MLP_DIM),
    "down": (MLP_DIM, HIDDEN),
}


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit pattern, round to nearest even (finite inputs)."""
    b = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = (b + 0x7FFF + ((b >> 16) & 1)) >> 16
    return r.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """bf16 bit pattern -> the float32 with the same value (format widening, exact)."""
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def pack_codes_k8(codes: np.ndarray) -> np.ndarray:
    """uint8 codes [K, N] (values 0..15) -> uint32 [K/8, N], 8 codes per word along K, low nibble first."""
    K, N = codes.shape
    assert K % 8 == 0
    c = codes.reshape(K // 8, 8, N).astype(np.uint32)
    w = np.zeros((K // 8, N), dtype=np.uint32)
    for j in range(8):
        w |= c[:, j, :] << np.uint32(4 * j)
    return w


def make_linear(entropy, M: int, K: int, N: int, g: int = 128, symmetric: bool = False,
                with_x: bool = True) -> dict:
    """Draw one linear's inputs.  `entropy` is an int or a sequence of ints (SeedSequence entropy)."""
    assert K % g == 0 and K % 8 == 0
    rng = np.random.default_rng(np.random.SeedSequence(entropy))
    codes = rng.integers(0, 16, size=(K, N), dtype=np.uint8)
    wq = pack_codes_k8(codes)
    del codes
    sc = np.abs(rng.standard_normal((K // g, N), dtype=np.float32)) * np.float32(0.01) + np.float32(1e-3)
    scale = f32_to_bf16_bits(sc)
    zero = rng.integers(0, 16, size=(K // g, N), dtype=np.uint8)
    if symmetric:
        zero = np.full_like(zero, 8)
    out = dict(wq=wq, scale=scale, zero=zero, M=M, K=K, N=N, g=g, symmetric=symmetric)
    if with_x:
        out["x"] = f32_to_bf16_bits(rng.standard_normal((M, K), dtype=np.float32))
    return out


def make_x(entropy, M: int, K: int) -> np.ndarray:
    rng = np.random.default_rng(np.random.SeedSequence(entropy))
    return f32_to_bf16_bits(rng.standard_normal((M, K), dtype=np.float32))


# ---- the five benchmark configurations -------------------------------------------------------

def config0() -> dict:
    """Single linear, M=1, K=512, N=256, g=128, seed 0."""
    return make_linear(0, 1, 512, 256, 128)


def config1() -> dict:
    """Verify-step MLP at M=16, seed 1: gate, up (2560->9728) and down (9728->2560), each an
    independent linear with its own bf16 N(0,1) input."""
    return {
        "gate": make_linear([1, 0], 16, HIDDEN, MLP_DIM),
        "up": make_linear([1, 1], 16, HIDDEN, MLP_DIM),
        "down": make_linear([1, 2], 16, MLP_DIM, HIDDEN),
    }


def stack_layer_weights(layer: int, name: str, g: int = 128, shapes: dict | None = None) -> dict:
    """Weights of one projection of one layer of the 36-layer stack: entropy [layer, linear_idx]."""
    K, N = (shapes or LAYER_SHAPES)[name]
    return make_linear([layer, LINEAR_IDX[name]], 0, K, N, g, with_x=False)


# Second workload: the drafter.  The paper gives its depth (5 layers), hidden size (2560), block
# size (16) and quantisation (group-wise symmetric INT4, groups of 128) but not its projection
# widths; the widths used here are the target's (SYNTHETIC: 5 x 100.9 M = 505 M parameters, close to
# the ~537 M the paper states for the whole drafter).
DRAFTER_LAYERS = 5


def drafter_layer_weights(layer: int, name: str, g: int = 128, shapes: dict | None = None) -> dict:
    """Weights of one projection of one drafter layer: symmetric codes (zero point 8), entropy [5, layer, linear_idx]."""
    K, N = (shapes or LAYER_SHAPES)[name]
    return make_linear([5, layer, LINEAR_IDX[name]], 0, K, N, g, symmetric=True, with_x=False)


def stack_h0(M: int = 16, hidden: int = HIDDEN) -> np.ndarray:
    """Input of layer 0 of the stack: bf16 N(0,1) [M, hidden], entropy [2, 0xACE]."""
    return make_x([2, 0xACE], M, hidden)


def config3(N: int = VOCAB, M: int = 16, K: int = HIDDEN) -> dict:
    """LM head, seed 3."""
    return make_linear(3, M, K, N, 128)


SWEEP_SHAPES = [(HIDDEN, MLP_DIM), (MLP_DIM, HIDDEN), (HIDDEN, QKV_DIM)]
SWEEP_M = [1, 2, 4, 8, 16, 32, 64]


def config4_point(shape_idx: int, M: int, g: int, symmetric: bool) -> dict:
    """One point of the M-sweep; entropy [4, shape_idx, g, symmetric] so that the weights of a
    (shape, g, zero mode) are the same for every M (X differs per M through its own stream)."""
    K, N = SWEEP_SHAPES[shape_idx]
    d = make_linear([4, shape_idx, g, int(symmetric)], 0, K, N, g, symmetric, with_x=False)
    d["x"] = make_x([4, shape_idx, g, int(symmetric), M], M, K)
    d["M"] = M
    return d


# --------------------------------------------------------------------------------------------
# drafter attention (synthetic stand-ins for the drafter's queries and its key/value cache)

ATTN_HEADS, ATTN_KV_HEADS, ATTN_HEAD_DIM = 32, 8, 128     # the target's synthetic geometry (4096 = 32 x 128, 1024 = 8 x 128)
SWA_CONTEXTS = (64, 2048, 8192)                          # input lengths of the paper's three latency settings
SWA_WINDOWS = (1024, 2048)


def attention_inputs(entropy, n_q: int, T: int, Hq: int, Hkv: int, d: int = ATTN_HEAD_DIM):
    """bf16 bit patterns: q [n_q, Hq, d], k and v [T, Hkv, d], all N(0,1); draw order q, k, v."""
    rng = np.random.Generator(np.random.PCG64(np.random.SeedSequence([0x5A, int(entropy)])))
    q = f32_to_bf16_bits(rng.standard_normal((n_q, Hq, d), dtype=np.float32))
    k = f32_to_bf16_bits(rng.standard_normal((T, Hkv, d), dtype=np.float32))
    v = f32_to_bf16_bits(rng.standard_normal((T, Hkv, d), dtype=np.float32))
    return q, k, v
