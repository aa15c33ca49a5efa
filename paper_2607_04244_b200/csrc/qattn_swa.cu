// Symmetric sliding-window attention of the drafter's block (paper Section 3.3, "Drafter SWA"): the
// n_q <= 16 mask-token queries of a drafted block attend bidirectionally to a complete key/value
// cache, every query restricted to a window that is symmetric around its own position; sequences
// that fit into the window are attended in full.  Nothing is evicted or rotated: the window exists
// only here, in the attention computation.
//
//   visible(p) = { k : |k - p| <= W div 2 } ∩ [0, T)          (all of [0, T) when T <= W)
//   out[i, h, :] = sum_k softmax_k(q[i,h,:] . key[k, h div G, :] / sqrt(d)) value[k, h div G, :]
//
// Work split (flash-decoding style, one launch).  The union of the queries' windows is a key range
// of at most W + n_q keys; it is cut into pieces of whole 64-key sub-blocks so that about one CTA
// per SM exists: CTA (piece b, key/value head h).  Two warps of a CTA own query head h G + w: their
// 16 rows are the 16 queries.  Per sub-block each of the two forms S = Q K^T with
// mma.sync.m16n8k16 (bf16 operands, fp32 accumulate; K fragments by ldmatrix from shared memory),
// masks S per row with that row's window, keeps a running maximum and sum (online softmax, base 2),
// and accumulates its half of the 128 output columns of O += P V, with P split into two bf16 terms
// (P = hi + lo, so that the probabilities enter with 16 significant bits; V fragments by
// ldmatrix.trans).  S is computed twice, which costs less than handing it over.  A piece leaves
// (max, sum, O) per row in the workspace; the CTA that arrives last at the head's counter merges
// the pieces in piece order (deterministic, nobody waits) and stores the bf16 rows.
//
// The path is bound by the bytes of K and V inside the window (2 x span x Hkv x 256 B, 8.5 MB for a
// window of 2,048) and, at these sizes, by launch and pipeline latency; tensor cores are used
// because S and O are real contractions (64 rows x 128 x span per head), not to reach their peak.
#include <atomic>

#include "ql_params.h"

namespace ql {

constexpr int kAttnD = 128;                      // head dimension
constexpr int kAttnSub = 64;                     // keys per sub-block
constexpr int kAttnRow = kAttnD * 2 + 16;        // bytes of one key (or value) row in shared memory: +16 spreads the banks for ldmatrix
constexpr int kAttnPartStride = kAttnD + 4;      // floats per row of a partial: O[128], max, sum, 2 unused (16-byte multiple)

__device__ __forceinline__ void ldmatrix_x4(uint32_t (&r)[4], const void* smem_row) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(smem_row)));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t (&r)[4], const void* smem_row) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(smem_u32(smem_row)));
}

// keys a query at position p sees
__device__ __forceinline__ void attn_key_range(int p, int T, int window, int& lo, int& hi) {
  if (T <= window) { lo = 0; hi = T; return; }
  const int half = window >> 1;
  lo = max(0, p - half);
  hi = min(T, p + half + 1);
}

template <int G>
__global__ void __launch_bounds__(64 * G) qattn_swa_kernel(const __grid_constant__ AttnParams p) {
  extern __shared__ __align__(128) uint8_t attn_smem[];   // two stages of (keys, values) of one sub-block
  __shared__ int s_last;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g8 = lane >> 2, t = lane & 3;
  constexpr int nthreads = 64 * G;
  const int piece = blockIdx.x, hk = blockIdx.y;
  const int hq = hk * G + (warp >> 1);                  // two warps per query head
  const int half = warp & 1;                            // which 64 of the 128 output columns this warp accumulates
  const int k_begin = p.key_lo + piece * p.sub_per_piece * kAttnSub;
  const int k_end = min(p.key_hi, k_begin + p.sub_per_piece * kAttnSub);

  // Q fragments of this warp's head: a[s] covers d = 16 s .. 16 s + 15, rows g8 and g8 + 8
  uint32_t qa[kAttnD / 16][4];
  {
    const uint16_t* q0 = p.Q + (size_t)g8 * p.ld_q + (size_t)hq * kAttnD;
    const uint16_t* q1 = q0 + (size_t)8 * p.ld_q;
    const bool live0 = g8 < p.n_q, live1 = g8 + 8 < p.n_q;
#pragma unroll
    for (int s = 0; s < kAttnD / 16; ++s) {
      qa[s][0] = live0 ? __ldg(reinterpret_cast<const uint32_t*>(q0 + 16 * s + 2 * t)) : 0u;
      qa[s][1] = live1 ? __ldg(reinterpret_cast<const uint32_t*>(q1 + 16 * s + 2 * t)) : 0u;
      qa[s][2] = live0 ? __ldg(reinterpret_cast<const uint32_t*>(q0 + 16 * s + 8 + 2 * t)) : 0u;
      qa[s][3] = live1 ? __ldg(reinterpret_cast<const uint32_t*>(q1 + 16 * s + 8 + 2 * t)) : 0u;
    }
  }
  int lo0, hi0, lo1, hi1;                               // windows of the thread's two rows
  attn_key_range(p.p0 + g8, p.T, p.window, lo0, hi0);
  attn_key_range(p.p0 + g8 + 8, p.T, p.window, lo1, hi1);
  if (g8 >= p.n_q) { lo0 = 0; hi0 = 0; }
  if (g8 + 8 >= p.n_q) { lo1 = 0; hi1 = 0; }

  constexpr int NB = kAttnD / 16;                       // 8-column blocks of this warp's half
  float o[NB][4];
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.f;
  float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;   // running maxima (base-2 scores) and this thread's share of the sums

  // keys and values of one sub-block into a stage of shared memory (rows beyond the piece are zero)
  auto load_sub = [&](int kb, int stage) {
    uint8_t* Kd = attn_smem + (size_t)stage * 2 * kAttnSub * kAttnRow;
    uint8_t* Vd = Kd + kAttnSub * kAttnRow;
    for (int u = tid; u < kAttnSub * (kAttnD / 8); u += nthreads) {
      const int r = u / (kAttnD / 8), c = u % (kAttnD / 8);
      const int key = kb + r;
      const bool live = key < k_end;
      const size_t src = (size_t)(live ? key : 0) * p.ld_kv + (size_t)hk * kAttnD + 8 * c;
      cp_async16(Kd + r * kAttnRow + 16 * c, p.K + src, live ? 16u : 0u);
      cp_async16(Vd + r * kAttnRow + 16 * c, p.V + src, live ? 16u : 0u);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  load_sub(k_begin, 0);
  int it = 0;
  for (int kb = k_begin; kb < k_end; kb += kAttnSub, ++it) {
    // the next sub-block is fetched while this one is used
    if (kb + kAttnSub < k_end) {
      load_sub(kb + kAttnSub, (it & 1) ^ 1);
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();
    const uint8_t* Ks = attn_smem + (size_t)(it & 1) * 2 * kAttnSub * kAttnRow;
    const uint8_t* Vs = Ks + kAttnSub * kAttnRow;

    // ---- S = Q K^T: 16 rows x 64 keys per warp ----
    float s[kAttnSub / 8][4];
#pragma unroll
    for (int j = 0; j < kAttnSub / 8; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
    {
      const int mi = lane >> 3, r = lane & 7;           // ldmatrix: lane -> (matrix, row)
#pragma unroll
      for (int ks = 0; ks < kAttnD / 16; ++ks) {
#pragma unroll
        for (int jp = 0; jp < kAttnSub / 16; ++jp) {
          // matrices: (keys 16jp.., d 16ks..), (same keys, d 16ks+8..), (keys 16jp+8.., d 16ks..), (keys 16jp+8.., d 16ks+8..)
          uint32_t b[4];
          ldmatrix_x4(b, Ks + (16 * jp + 8 * (mi >> 1) + r) * kAttnRow + (16 * ks + 8 * (mi & 1)) * 2);
          mma_bf16_16816(s[2 * jp], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b[0], b[1]);
          mma_bf16_16816(s[2 * jp + 1], qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3], b[2], b[3]);
        }
      }
    }
    // ---- scale, mask with each row's window, online softmax ----
    float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
    for (int j = 0; j < kAttnSub / 8; ++j) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int key = kb + 8 * j + 2 * t + (e & 1);
        const bool vis = (e < 2) ? (key >= lo0 && key < hi0) : (key >= lo1 && key < hi1);
        const float v = (vis && key < k_end) ? s[j][e] * p.scale_log2 : -INFINITY;
        s[j][e] = v;
        if (e < 2) mx0 = fmaxf(mx0, v); else mx1 = fmaxf(mx1, v);
      }
    }
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
    const float n0 = fmaxf(m0, mx0), n1 = fmaxf(m1, mx1);
    const float u0 = (n0 == -INFINITY) ? 0.f : n0, u1 = (n1 == -INFINITY) ? 0.f : n1;   // no visible key so far: every p is 0
    const float al0 = exp2f(m0 - u0), al1 = exp2f(m1 - u1);                              // exp2(-inf) = 0
    m0 = n0; m1 = n1;
    l0 *= al0; l1 *= al1;
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) { o[nb][0] *= al0; o[nb][1] *= al0; o[nb][2] *= al1; o[nb][3] *= al1; }
#pragma unroll
    for (int j = 0; j < kAttnSub / 8; ++j) {
      s[j][0] = exp2f(s[j][0] - u0); s[j][1] = exp2f(s[j][1] - u0);
      s[j][2] = exp2f(s[j][2] - u1); s[j][3] = exp2f(s[j][3] - u1);
      l0 += s[j][0] + s[j][1];
      l1 += s[j][2] + s[j][3];
    }
    // ---- O += P V, P = hi + lo (two bf16 terms) ----
    {
      const int mi = lane >> 3, r = lane & 7;
#pragma unroll
      for (int jj = 0; jj < kAttnSub / 16; ++jj) {
        uint32_t ph[4], pl[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          // A fragment q: rows g8 (q even) / g8 + 8 (q odd), keys 16jj + 8 (q div 2) + 2t, +1
          const float x = s[2 * jj + (q >> 1)][2 * (q & 1)], y = s[2 * jj + (q >> 1)][2 * (q & 1) + 1];
          ph[q] = pack_bf16x2_rn(x, y);
          pl[q] = pack_bf16x2_rn(x - bf16lo_to_f32(ph[q]), y - bf16hi_to_f32(ph[q]));
        }
#pragma unroll
        for (int np = 0; np < NB / 2; ++np) {
          // matrices: (keys 16jj.., d c..), (keys 16jj+8.., d c..), (keys 16jj.., d c+8..), (keys 16jj+8.., d c+8..), c = 64 half + 16 np
          uint32_t b[4];
          ldmatrix_x4_trans(b, Vs + (16 * jj + 8 * (mi & 1) + r) * kAttnRow + (64 * half + 16 * np + 8 * (mi >> 1)) * 2);
          mma_bf16_16816(o[2 * np], ph[0], ph[1], ph[2], ph[3], b[0], b[1]);
          mma_bf16_16816(o[2 * np], pl[0], pl[1], pl[2], pl[3], b[0], b[1]);
          mma_bf16_16816(o[2 * np + 1], ph[0], ph[1], ph[2], ph[3], b[2], b[3]);
          mma_bf16_16816(o[2 * np + 1], pl[0], pl[1], pl[2], pl[3], b[2], b[3]);
        }
      }
    }
    __syncthreads();                                    // this stage is refilled by the next iteration's fetch
  }
  l0 += __shfl_xor_sync(0xffffffffu, l0, 1);
  l0 += __shfl_xor_sync(0xffffffffu, l0, 2);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 1);
  l1 += __shfl_xor_sync(0xffffffffu, l1, 2);

  if (p.n_pieces == 1) {
    // the only piece of its head: the rows are complete, no hand-over through the workspace
    const float i0 = l0 > 0.f ? 1.f / l0 : 0.f, i1 = l1 > 0.f ? 1.f / l1 : 0.f;
    uint16_t* y0 = p.out + (size_t)g8 * p.ld_out + (size_t)hq * kAttnD + 64 * half + 2 * t;
    uint16_t* y1 = y0 + (size_t)8 * p.ld_out;
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
      if (g8 < p.n_q) *reinterpret_cast<uint32_t*>(y0 + 8 * nb) = pack_bf16x2_rn(o[nb][0] * i0, o[nb][1] * i0);
      if (g8 + 8 < p.n_q) *reinterpret_cast<uint32_t*>(y1 + 8 * nb) = pack_bf16x2_rn(o[nb][2] * i1, o[nb][3] * i1);
    }
    return;
  }
  // ---- the piece's partial rows (each warp its 64 columns; the first of a head also maximum and sum) ----
  float* my = p.part + ((((size_t)hk * p.n_pieces + piece) * G + (warp >> 1)) * 16) * kAttnPartStride;
#pragma unroll
  for (int nb = 0; nb < NB; ++nb) {
    __stcg(reinterpret_cast<float2*>(my + (size_t)g8 * kAttnPartStride + 64 * half + 8 * nb + 2 * t), make_float2(o[nb][0], o[nb][1]));
    __stcg(reinterpret_cast<float2*>(my + (size_t)(g8 + 8) * kAttnPartStride + 64 * half + 8 * nb + 2 * t), make_float2(o[nb][2], o[nb][3]));
  }
  if (t == 0 && half == 0) {
    __stcg(reinterpret_cast<float2*>(my + (size_t)g8 * kAttnPartStride + kAttnD), make_float2(m0, l0));
    __stcg(reinterpret_cast<float2*>(my + (size_t)(g8 + 8) * kAttnPartStride + kAttnD), make_float2(m1, l1));
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const int old = atomicAdd(&p.counters[hk], 1);
    s_last = (old == p.n_pieces - 1);
    if (s_last) p.counters[hk] = 0;                      // ready for the next call
  }
  __syncthreads();
  if (!s_last) return;
  __threadfence();

  // ---- the last CTA of the head merges the pieces, in piece order.  A warp merges its half of the
  //      columns of its head: lane l keeps columns 2l, 2l+1 of all 16 rows, so that the loads of
  //      four pieces are in flight together; lane l also looks after the maximum and the sum of
  //      row l mod 16 ----
  const float* base = p.part + (((size_t)hk * p.n_pieces) * G + (warp >> 1)) * 16 * kAttnPartStride;
  const size_t piece_stride = (size_t)G * 16 * kAttnPartStride;
  const int myrow = lane & 15;
  float M = -INFINITY;                                  // running maximum of row myrow over the pieces merged so far
  float2 acc[16];
#pragma unroll
  for (int r = 0; r < 16; ++r) acc[r] = make_float2(0.f, 0.f);
  float L = 0.f;
  for (int b0 = 0; b0 < p.n_pieces; b0 += 4) {
    float2 ml[4], v[4][16];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int b = min(b0 + q, p.n_pieces - 1);
      const float* pb = base + b * piece_stride;
      ml[q] = __ldcg(reinterpret_cast<const float2*>(pb + (size_t)myrow * kAttnPartStride + kAttnD));
#pragma unroll
      for (int r = 0; r < 16; ++r) v[q][r] = __ldcg(reinterpret_cast<const float2*>(pb + (size_t)r * kAttnPartStride + 64 * half) + lane);
    }
    // new maximum over these four pieces, then what is already summed is rescaled once
    float Mn = M;
#pragma unroll
    for (int q = 0; q < 4; ++q)
      if (b0 + q < p.n_pieces) Mn = fmaxf(Mn, ml[q].x);
    const float Mu = (Mn == -INFINITY) ? 0.f : Mn;
    const float resc = exp2f(M - Mu);                    // exp2(-inf) = 0 on the first round: nothing summed yet
    M = Mn;
    L *= resc;
#pragma unroll
    for (int r = 0; r < 16; ++r) {
      const float w = __shfl_sync(0xffffffffu, resc, r);
      acc[r].x *= w;
      acc[r].y *= w;
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      // a piece without a visible key of the row weighs nothing; so does a repeated last piece
      const float wm = (b0 + q >= p.n_pieces || ml[q].x == -INFINITY) ? 0.f : exp2f(ml[q].x - Mu);
      L = fmaf(wm, ml[q].y, L);
#pragma unroll
      for (int r = 0; r < 16; ++r) {
        const float w = __shfl_sync(0xffffffffu, wm, r);
        acc[r].x = fmaf(w, v[q][r].x, acc[r].x);
        acc[r].y = fmaf(w, v[q][r].y, acc[r].y);
      }
    }
  }
  const float inv_mine = L > 0.f ? 1.f / L : 0.f;
#pragma unroll
  for (int r = 0; r < 16; ++r) {
    const float inv = __shfl_sync(0xffffffffu, inv_mine, r);
    if (r < p.n_q)
      *reinterpret_cast<uint32_t*>(p.out + (size_t)r * p.ld_out + (size_t)hq * kAttnD + 64 * half + 2 * lane) =
          pack_bf16x2_rn(acc[r].x * inv, acc[r].y * inv);
  }
}

// ---- host side ---------------------------------------------------------------------------------

// Fills the split fields of `p` (key range, pieces) for `sms` SMs; returns the floats of partials needed.
size_t attn_plan(AttnParams& p, int sms) {
  int lo = p.T, hi = 0;
  for (int i = 0; i < p.n_q; ++i) {
    int a, b;
    const int pos = p.p0 + i;
    if (p.T <= p.window) { a = 0; b = p.T; }
    else { const int half = p.window >> 1; a = pos - half < 0 ? 0 : pos - half; b = pos + half + 1 > p.T ? p.T : pos + half + 1; }
    if (a < lo) lo = a;
    if (b > hi) hi = b;
  }
  if (hi < lo) hi = lo;
  p.key_lo = lo;
  p.key_hi = hi;
  const int n_sub = (hi - lo + kAttnSub - 1) / kAttnSub > 0 ? (hi - lo + kAttnSub - 1) / kAttnSub : 1;
  int max_pieces = sms / p.Hkv;
  if (max_pieces < 1) max_pieces = 1;
  p.sub_per_piece = (n_sub + max_pieces - 1) / max_pieces;
  if (n_sub <= 2) p.sub_per_piece = n_sub;               // a hand-over through the workspace costs more than a second sub-block
  p.n_pieces = (n_sub + p.sub_per_piece - 1) / p.sub_per_piece;
  return (size_t)p.Hkv * p.n_pieces * p.G * 16 * kAttnPartStride;
}

template <int G>
static cudaError_t attn_launch_g(const AttnParams& p, cudaStream_t stream) {
  constexpr int smem = 2 * 2 * kAttnSub * kAttnRow;      // 69,632 bytes
  static std::atomic<unsigned> attr_set{0};              // bit per device
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 32 && !(attr_set.load(std::memory_order_acquire) & (1u << dev))) {
    cudaError_t e = cudaFuncSetAttribute(qattn_swa_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    attr_set.fetch_or(1u << dev, std::memory_order_release);
  }
  qattn_swa_kernel<G><<<dim3(p.n_pieces, p.Hkv), dim3(64 * G), smem, stream>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_attn_swa(const AttnParams& p, cudaStream_t stream) {
  switch (p.G) {
    case 1: return attn_launch_g<1>(p, stream);
    case 2: return attn_launch_g<2>(p, stream);
    case 4: return attn_launch_g<4>(p, stream);
    case 8: return attn_launch_g<8>(p, stream);
    default: return cudaErrorInvalidConfiguration;
  }
}

}  // namespace ql
