// qpack_w4_g128: boundary format -> packed tile layout.  One CTA per chunk (column tile T,
// group G); pure integer permutation, so the output is bit-exact by construction.
// qrequant_pack_w4: the same layout written from bf16 weights re-quantised onto the frozen grid.
#include "ql_device.cuh"

namespace ql {

// Moves code i (bits [4i,4i+4)) of an input word to nibble (i>>1) + 4*(i&1): even rows of the
// 8-row run go to the low half-word, odd rows to the high half-word, so that one masked
// extraction (w >> 4s) & 0x000f000f yields rows (2s, 2s+1) as a bf16x2 operand pair.
__device__ __forceinline__ uint32_t interleave_codes(uint32_t w) {
  uint32_t even = w & 0x0F0F0F0Fu;           // codes 0,2,4,6 at bits 0,8,16,24
  uint32_t odd = (w >> 4) & 0x0F0F0F0Fu;     // codes 1,3,5,7
  even = (even | (even >> 4)) & 0x00FF00FFu; // codes (0,2) at bits 0..7, (4,6) at bits 16..23
  even = (even | (even >> 8)) & 0x0000FFFFu;
  odd = (odd | (odd >> 4)) & 0x00FF00FFu;
  odd = (odd | (odd >> 8)) & 0x0000FFFFu;
  return even | (odd << 16);
}

template <int G>
__global__ void __launch_bounds__(128) qpack_kernel(const uint32_t* __restrict__ wq, const uint16_t* __restrict__ scale,
                                                    const uint8_t* __restrict__ zero, int N, int n_groups,
                                                    uint8_t* __restrict__ packed) {
  const int Gi = blockIdx.x, T = blockIdx.y, n = threadIdx.x;
  const size_t col = (size_t)T * kTileN + n;
  uint8_t* chunk = packed + ((size_t)T * n_groups + Gi) * chunk_bytes(G);
  uint4* wout = reinterpret_cast<uint4*>(chunk);
  const size_t row0 = (size_t)Gi * (G / 8);                     // first input word row of the group
#pragma unroll
  for (int c = 0; c < G / 32; ++c) {
    uint4 o;
    o.x = interleave_codes(wq[(row0 + 4 * c + 0) * N + col]);
    o.y = interleave_codes(wq[(row0 + 4 * c + 1) * N + col]);
    o.z = interleave_codes(wq[(row0 + 4 * c + 2) * N + col]);
    o.w = interleave_codes(wq[(row0 + 4 * c + 3) * N + col]);
    wout[c * kTileN + n] = o;                                   // word (c, n, j = 0..3)
  }
  reinterpret_cast<uint16_t*>(chunk + 64 * G)[n] = scale[(size_t)Gi * N + col];
  // zero points: 8 lanes combine their nibbles into one word
  uint32_t z = (zero != nullptr) ? (uint32_t)(zero[(size_t)Gi * N + col] & 0xF) : 8u;
  z <<= 4 * (n & 7);
  z |= __shfl_xor_sync(0xffffffffu, z, 1);
  z |= __shfl_xor_sync(0xffffffffu, z, 2);
  z |= __shfl_xor_sync(0xffffffffu, z, 4);
  if ((n & 7) == 0) reinterpret_cast<uint32_t*>(chunk + 64 * G + 256)[n >> 3] = z;
}

// qrequant_pack_w4: bf16 weights + frozen scales (+ zero points) -> new codes on the same grid,
// written straight into the packed tile layout (the codes never exist in the boundary format).
// code = clamp(rne(w / s) + z, 0, 15): IEEE float32 division, round-half-to-even - integer
// decisions, so both are spelled out (no fast-math substitutes).
template <int G>
__global__ void __launch_bounds__(128) qrequant_kernel(const uint16_t* __restrict__ w, const uint16_t* __restrict__ scale,
                                                       const uint8_t* __restrict__ zero, int N, int n_groups,
                                                       uint8_t* __restrict__ packed) {
  const int Gi = blockIdx.x, T = blockIdx.y, n = threadIdx.x;
  const size_t col = (size_t)T * kTileN + n;
  uint8_t* chunk = packed + ((size_t)T * n_groups + Gi) * chunk_bytes(G);
  uint4* wout = reinterpret_cast<uint4*>(chunk);
  const uint16_t sbits = scale[(size_t)Gi * N + col];
  const float s = __uint_as_float((uint32_t)sbits << 16);
  const int z = (zero != nullptr) ? (int)(zero[(size_t)Gi * N + col] & 0xF) : 8;
  const size_t row0 = (size_t)Gi * G;
#pragma unroll
  for (int c = 0; c < G / 32; ++c) {
    uint32_t words[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      uint32_t word = 0;
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const float v = __uint_as_float((uint32_t)w[(row0 + 32 * c + 8 * j + i) * N + col] << 16);
        int q = (int)rintf(__fdiv_rn(v, s)) + z;
        q = q < 0 ? 0 : (q > 15 ? 15 : q);
        word |= (uint32_t)q << (4 * ((i >> 1) + 4 * (i & 1)));     // row i of the run -> nibble (i>>1) + 4*(i&1)
      }
      words[j] = word;
    }
    wout[c * kTileN + n] = make_uint4(words[0], words[1], words[2], words[3]);
  }
  reinterpret_cast<uint16_t*>(chunk + 64 * G)[n] = sbits;
  uint32_t zz = (uint32_t)z << (4 * (n & 7));
  zz |= __shfl_xor_sync(0xffffffffu, zz, 1);
  zz |= __shfl_xor_sync(0xffffffffu, zz, 2);
  zz |= __shfl_xor_sync(0xffffffffu, zz, 4);
  if ((n & 7) == 0) reinterpret_cast<uint32_t*>(chunk + 64 * G + 256)[n >> 3] = zz;
}

cudaError_t launch_qrequant(const uint16_t* w, const uint16_t* scale, const uint8_t* zero, int K, int N, int g,
                            uint8_t* packed, cudaStream_t stream) {
  dim3 grid(K / g, N / kTileN);
  if (g == 128)
    qrequant_kernel<128><<<grid, 128, 0, stream>>>(w, scale, zero, N, K / g, packed);
  else
    qrequant_kernel<64><<<grid, 128, 0, stream>>>(w, scale, zero, N, K / g, packed);
  return cudaGetLastError();
}

cudaError_t launch_qpack(const uint32_t* wq, const uint16_t* scale, const uint8_t* zero, int K, int N, int g,
                         uint8_t* packed, cudaStream_t stream) {
  dim3 grid(K / g, N / kTileN);
  if (g == 128)
    qpack_kernel<128><<<grid, 128, 0, stream>>>(wq, scale, zero, N, K / g, packed);
  else
    qpack_kernel<64><<<grid, 128, 0, stream>>>(wq, scale, zero, N, K / g, packed);
  return cudaGetLastError();
}

}  // namespace ql
