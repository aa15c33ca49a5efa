"""qrequant_pack_w4 on the GPU against the oracle, byte for byte: bf16 weights near the frozen grid
(dequantised codes plus a perturbation, as after a few distillation steps), with exact half-way
cases and out-of-grid values planted, re-quantised and packed in one kernel."""
import numpy as np
import pytest
import torch

import qsynth
from oracle import w4a16_oracle as orc
from gpu_util import dev_u16, dev_u8

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("K,N,g,sym", [(512, 256, 128, False), (256, 384, 64, False), (2560, 1280, 128, True), (1024, 2560, 64, False)])
def test_requant_pack_bit_exact(ql, K, N, g, sym):
    d = qsynth.make_linear([66, K, N, g], 0, K, N, g, symmetric=sym, with_x=False)
    rng = np.random.default_rng(K + N)
    w32 = orc.dequant_f32(d["wq"], d["scale"], d["zero"], g)                       # on the grid
    s32 = np.repeat(qsynth.bf16_bits_to_f32(d["scale"]), g, axis=0)
    w32 = w32 + s32 * rng.uniform(-0.8, 0.8, (K, N)).astype(np.float32)            # drifted off it
    w32[::7, ::5] = (s32 * (rng.integers(-9, 9, (K, N)) + 0.5))[::7, ::5]           # exact halves (where representable)
    w32[3::11, 1::3] *= 40.0                                                       # far outside: clamps
    w = qsynth.f32_to_bf16_bits(w32)
    zero = None if sym else d["zero"]
    want_codes = orc.requant_codes(w, d["scale"], zero, g)
    want = orc.pack_ref(qsynth.pack_codes_k8(want_codes), d["scale"], zero, g)
    got = ql.qrequant_pack_w4(dev_u16(w), dev_u16(d["scale"]), None if sym else dev_u8(d["zero"]), K, N, g).cpu().numpy()
    assert got.size == want.size == ql.ql_packed_bytes(K, N, g)
    assert np.array_equal(got, want)
    hist = np.bincount(want_codes.reshape(-1), minlength=16)
    assert hist[0] > 0 and hist[15] > 0 and hist[1:15].min() > 0                   # every code, both clamps exercised


def test_requant_of_dequantised_weights_reproduces_the_packed_buffer(ql):
    """Power-of-two scales: the dequantised weights are exact in bf16, so re-quantising them must
    give the very bytes qpack_w4_g128 produces from the original codes."""
    K, N, g = 512, 384, 128
    rng = np.random.default_rng(3)
    codes = rng.integers(0, 16, (K, N), dtype=np.uint8)
    zero = rng.integers(0, 16, (K // g, N), dtype=np.uint8)
    scale = np.full((K // g, N), 0x3D00, dtype=np.uint16)
    wq = qsynth.pack_codes_k8(codes)
    w = qsynth.f32_to_bf16_bits(orc.dequant_f32(wq, scale, zero, g))
    a = ql.qrequant_pack_w4(dev_u16(w), dev_u16(scale), dev_u8(zero), K, N, g).cpu().numpy()
    b = ql.qpack_w4_g128(torch.from_numpy(wq.view(np.int32)).cuda(), dev_u16(scale), dev_u8(zero), K, N, g).cpu().numpy()
    assert np.array_equal(a, b) and np.array_equal(a, orc.pack_ref(wq, scale, zero, g))
