// Warp-level tensor-core path of qlinear_w4a16 (ql_path QL_PATH_MMA).
//
// One persistent CTA per SM.  CTA i owns a contiguous run of packed chunks (a chunk is one
// 128-column tile x one quantisation group), i.e. a contiguous byte range of the packed buffer,
// so HBM traffic is balanced to within one chunk whatever the shape (stream-K split).
//
//   warp 8      producer: one elected lane issues one bulk copy (TMA engine, no tensor map) per
//               packed chunk into a ring of shared memory stages; completion is counted on one
//               mbarrier per stage.  X is not streamed: the consumers load, once per CTA, the
//               X columns of every group the CTA's chunks touch (cp.async from all 256 threads)
//               while the first weight chunks are in flight.
//   warps 0..7  consumers: warp = (kg, wn); the two k-groups kg take alternate chunks, warp wn
//               owns columns [32wn, 32wn+32) of the tile.  Codes are expanded to the exact bf16
//               integers q - z in registers, multiplied with X by mma.sync m16n8k16 into a
//               per-group fp32 partial, and the bf16 scale is applied once per group in fp32.
//
// A run of chunks that ends inside a tile leaves a partial tile: it is written to a workspace
// slot and the CTA that arrives last at the tile's counter adds all slots in CTA order (fixed
// order -> deterministic, no floating-point atomics, nobody ever waits for another CTA).
#include "ql_params.h"

namespace ql {

__host__ __device__ constexpr int mma_kgroups(int mt) { return mt == 1 ? 4 : 2; }   // k-groups (sets of 4 consumer warps taking alternate chunks)
constexpr int kMaxStages = 32;
constexpr uint32_t kSmemBudget = 232448u;   // 227 KB of dynamic shared memory per CTA

__host__ __device__ inline uint32_t mma_stage_bytes(int g) { return align128(chunk_bytes(g)); }
__host__ __device__ inline uint32_t mma_xslot_bytes(int g, int m_pad) { return (uint32_t)m_pad * 2u * g; }
__host__ __device__ inline uint32_t mma_fixed_smem(int mt) { return 8192u * mt * (mma_kgroups(mt) - 1) + kMaxStages * 16u + 2048u + 64u; }

// k-permutation used inside a 32-row block c of a group (it only has to be the same for X and W):
// lane t = lane & 3 owns rows 32c + 8t + i, i = 0..7; the first MMA of the pair contracts
// i = 0..3, the second i = 4..7.  The packed nibble order puts (i, i+1) for even i into one
// masked extraction, low half-word = even i.
template <int MT, int G>
__device__ __forceinline__ void compute_chunk(const uint8_t* __restrict__ st, const uint8_t* __restrict__ xs, int wn,
                                              int g8, int t, float (&acc)[4][MT][4]) {
  constexpr int NC = G / 32;
  const uint32_t* W = reinterpret_cast<const uint32_t*>(st);
  const uint32_t* S32 = reinterpret_cast<const uint32_t*>(st + 64 * G);
  const uint32_t* Z = reinterpret_cast<const uint32_t*>(st + 64 * G + 256);
  const int n0 = wn * 32;

  uint32_t zb[4];
  float s0[4], s1[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const uint32_t z = (Z[wn * 4 + j] >> (4 * g8)) & 0xFu;        // zero point of B-fragment column n0+8j+g8
    zb[j] = 0x43004300u | z | (z << 16);                           // bf16x2 of 128 + z
    const uint32_t sp = S32[(n0 + 8 * j + 2 * t) >> 1];            // scales of accumulator columns 2t, 2t+1
    s0[j] = bf16lo_to_f32(sp);
    s1[j] = bf16hi_to_f32(sp);
  }

  float P[4][MT][4];
#pragma unroll
  for (int j = 0; j < 4; ++j)
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int e = 0; e < 4; ++e) P[j][mt][e] = 0.f;

#pragma unroll
  for (int c = 0; c < NC; ++c) {
    uint4 xa[MT], xb[MT];
    const int unit = (4 * c + t) ^ ((g8 & 1) << 2);
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      const int r0 = mt * 16 + g8;
      xa[mt] = *reinterpret_cast<const uint4*>(xs + r0 * (2 * G) + unit * 16);
      xb[mt] = *reinterpret_cast<const uint4*>(xs + (r0 + 8) * (2 * G) + unit * 16);
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint32_t w = W[(c * 128 + n0 + 8 * j + g8) * 4 + t];
      uint32_t b0, b1, b2, b3;
      unpack_word(w, zb[j], b0, b1, b2, b3);
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        mma_bf16_16816(P[j][mt], xa[mt].x, xb[mt].x, xa[mt].y, xb[mt].y, b0, b1);
        mma_bf16_16816(P[j][mt], xa[mt].z, xb[mt].z, xa[mt].w, xb[mt].w, b2, b3);
      }
    }
  }
#pragma unroll
  for (int j = 0; j < 4; ++j)
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      acc[j][mt][0] = fmaf(s0[j], P[j][mt][0], acc[j][mt][0]);
      acc[j][mt][1] = fmaf(s1[j], P[j][mt][1], acc[j][mt][1]);
      acc[j][mt][2] = fmaf(s0[j], P[j][mt][2], acc[j][mt][2]);
      acc[j][mt][3] = fmaf(s1[j], P[j][mt][3], acc[j][mt][3]);
    }
}

// (value, index) comparison of the arg-max: larger value wins, lower index on equal values.
__device__ __forceinline__ void amax_merge(float& bv, int& bi, float v, int i) {
  if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
}

template <int MT, int G>
__global__ void __launch_bounds__(mma_kgroups(MT) * 128 + 32, 1) qlinear_mma_kernel(const __grid_constant__ LinearParams p) {
  constexpr int KG = mma_kgroups(MT);
  constexpr int NCONS = KG * 128;                        // consumer threads
  extern __shared__ __align__(1024) uint8_t smem[];
  const int NS = p.n_stages;
  const uint32_t stage = p.stage_bytes;
  uint8_t* ring = smem;
  uint8_t* xbuf = smem + (size_t)NS * stage;                          // [n_x][m_pad][2G bytes], 16-byte units swizzled
  const uint32_t xslot = mma_xslot_bytes(G, p.m_pad);
  uint8_t* after_x = xbuf + (size_t)p.n_x * xslot;
  float4* red4 = reinterpret_cast<float4*>(after_x);
  uint64_t* full = reinterpret_cast<uint64_t*>(after_x + 8192u * MT * (KG - 1));
  uint64_t* empty = full + kMaxStages;
  float2* s_amax = reinterpret_cast<float2*>(empty + kMaxStages);      // [4][64]
  int* s_flag = reinterpret_cast<int*>(s_amax + 4 * 64);                // [0..3] flags, [8] abort
  volatile int* s_abort = s_flag + 8;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t Gn = p.n_groups;
  const uint32_t total = p.total_chunks;
  const uint32_t start = cta_first_chunk(blockIdx.x, total, p.ncta);
  const uint32_t end = cta_first_chunk(blockIdx.x + 1, total, p.ncta);

  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(&full[s], 1);     // the producer's arrive.expect_tx; the bulk copy completes the bytes
      mbar_init(&empty[s], 4);    // the 4 warps of the k-group that consumed the stage
    }
    *s_abort = 0;
    fence_mbar_init();
  }
  __syncthreads();

  // Programmatic dependent launch: the next kernel of the stream may be scheduled as soon as every CTA of
  // this one has got here (its CTAs start where SMs become free, and their set-up overlaps this
  // kernel's tail).  Nothing a kernel does before its own griddepcontrol.wait may depend on the
  // kernels before it: here that is the barrier set-up only.
  grid_dep_launch();

  if (warp == KG * 4) {
    // ------------------------------------------------------------------ producer
    uint32_t it = 0;
    if (lane == 0) {
      grid_dep_wait();                                   // the packed weights may be the previous kernel's output
      const uint64_t pol = policy_evict_first();
      const uint32_t cb = chunk_bytes(G);
      const uint8_t* src = p.packed + (size_t)start * cb;
      uint32_t s = 0, ph = 0;
      for (uint32_t c = start; c < end; ++c, ++it, src += cb) {
        if (it >= (uint32_t)NS) mbar_wait(&empty[s], ph ^ 1, s_abort, p.ws.status);
        mbar_arrive_expect_tx(&full[s], cb);
        bulk_g2s_hint(ring + (size_t)s * stage, src, cb, &full[s], pol);
        if (++s == (uint32_t)NS) { s = 0; ph ^= 1; }
      }
    }
    it = __shfl_sync(0xffffffffu, it, 0);
    if (*s_abort) {
      // a wait gave up somewhere: let this CTA's own copies land before the CTA exits
      if (lane == 0) {
        const uint32_t n = it < (uint32_t)NS ? it : (uint32_t)NS;
        for (uint32_t k = 0; k < n; ++k) {
          const uint32_t i2 = it - 1 - k;
          const uint64_t t0 = globaltimer_ns();
          while (!mbar_try_wait(&full[i2 % NS], (i2 / NS) & 1) && globaltimer_ns() - t0 < 20000000ull) {}
        }
      }
    }
    return;
  }

  // -------------------------------------------------------------------- consumers
  const int kg = warp >> 2, wn = warp & 3, g8 = lane >> 2, t = lane & 3;
  // X, the workspace and Y belong to the kernels before this one until they have completed
  grid_dep_wait();
  const size_t slot_f4 = ws_slot_floats(p.m_pad) / 4;
  const uint32_t g_first = start % Gn;
  // X staging: slot k of xbuf receives the X columns of the group of the CTA's chunk number
  // first_it + k (groups advance cyclically with the chunk number), rows >= M are zero-filled.
  // Resident mode (x_phase == 0): all groups the CTA touches are loaded once, up front.
  // Phased mode (x_phase == P): X of the next P chunks is reloaded every P chunks (large M only).
  const uint32_t my_chunks = end - start;
  const uint32_t XP = (uint32_t)p.x_phase;
  auto load_x_slots = [&](uint32_t first_it, uint32_t count) {
    constexpr int UPR = G / 8;                           // 16-byte units per row of one group
    const uint32_t per_slot = (uint32_t)p.m_pad * UPR;
    for (uint32_t q = tid; q < count * per_slot; q += NCONS) {
      const uint32_t k = q / per_slot, rem = q - k * per_slot;
      const uint32_t r = rem / UPR, u = rem % UPR;
      const uint32_t Gi = (g_first + first_it + k) % Gn;
      const bool live = (int)r < p.M;
      const uint16_t* src = live ? (p.X + (size_t)r * p.ldx + (size_t)Gi * G + u * 8) : p.X;
      cp_async16(xbuf + (size_t)k * xslot + r * (2 * G) + ((u ^ ((r & 1) << 2)) * 16), src, live ? 16u : 0u);
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
    named_bar_sync(1, NCONS);
  };
  if (XP == 0) load_x_slots(0, min(my_chunks, Gn));
  float acc[4][MT][4];
  uint32_t it = 0, pos = start;
  int seg = 0;
  while (pos < end) {
    const uint32_t T = pos / Gn;
    const uint32_t g0 = pos - T * Gn;
    const uint32_t nch = min(Gn - g0, end - pos);
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[j][mt][e] = 0.f;

    if (MT <= 2 && XP == 0) {
      // resident X (kernels for up to 32 rows): the k-group walks its own chunks (every KG-th) with ring stage, phase and X slot
      // carried along - no division and no skipped iteration per chunk
      uint32_t ci = ((uint32_t)kg + KG - (it % KG)) % KG;
      const uint32_t itk = it + ci;
      uint32_t s = itk % NS, ph = (itk / NS) & 1;
      uint32_t xk = (g0 + ci + Gn - g_first) % Gn;
      const uint8_t* stp = ring + (size_t)s * stage;
      const uint8_t* xp = xbuf + (size_t)xk * xslot;
      for (; ci < nch; ci += KG) {
        mbar_wait(&full[s], ph, s_abort, p.ws.status);
        if (!(p.ablate & 1)) compute_chunk<MT, G>(stp, xp, wn, g8, t, acc);
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[s]);
        s += KG; stp += (size_t)KG * stage;
        while (s >= (uint32_t)NS) { s -= NS; ph ^= 1; stp -= (size_t)NS * stage; }
        xk += KG; xp += (size_t)KG * xslot;
        while (xk >= Gn) { xk -= Gn; xp -= (size_t)Gn * xslot; }
      }
      it += nch;
    } else
    for (uint32_t ci = 0; ci < nch; ++ci, ++it) {
      if (XP != 0 && it % XP == 0) {
        named_bar_sync(1, NCONS);                          // every consumer is done with the previous phase's X
        load_x_slots(it, min(XP, my_chunks - it));
      }
      if ((int)(it % KG) != kg) continue;
      const int s = it % NS;
      mbar_wait(&full[s], (it / NS) & 1, s_abort, p.ws.status);
      uint32_t xk;
      if (XP != 0) {
        xk = it % XP;
      } else {
        xk = g0 + ci + Gn - g_first;
        if (xk >= Gn) xk -= Gn;
      }
      if (!(p.ablate & 1)) compute_chunk<MT, G>(ring + (size_t)s * stage, xbuf + (size_t)xk * xslot, wn, g8, t, acc);
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[s]);
    }

    // ---- end of a tile segment: add the k-groups (fixed order: kg0 + kg1 + ...) -------------
    if (kg != 0) {
#pragma unroll
      for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
          red4[(((kg - 1) * 16 + wn * 4 + j) * MT + mt) * 32 + lane] = make_float4(acc[j][mt][0], acc[j][mt][1], acc[j][mt][2], acc[j][mt][3]);
    }
    named_bar_sync(1, NCONS);
    if (kg == 0) {
#pragma unroll
      for (int k2 = 0; k2 < KG - 1; ++k2)
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            const float4 v = red4[((k2 * 16 + wn * 4 + j) * MT + mt) * 32 + lane];
            acc[j][mt][0] += v.x; acc[j][mt][1] += v.y; acc[j][mt][2] += v.z; acc[j][mt][3] += v.w;
          }
    }
    named_bar_sync(1, NCONS);
    const bool whole = (g0 == 0 && nch == Gn);
    pos += nch;
    const int my_seg = seg++;
    if (kg != 0) continue;

    // ---- k-group 0 (128 threads) finishes the segment ------------------------------------
    if (!whole) {
      float4* my = reinterpret_cast<float4*>(p.ws.slots) + ((size_t)blockIdx.x * 2 + (my_seg == 0 ? 0 : 1)) * slot_f4;
#pragma unroll
      for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
          __stcg(&my[((wn * 4 + j) * MT + mt) * 32 + lane], make_float4(acc[j][mt][0], acc[j][mt][1], acc[j][mt][2], acc[j][mt][3]));
      __threadfence();
      named_bar_sync(2, 128);
      if (tid == 0) {
        const uint32_t first = chunk_owner(T * Gn, total, p.ncta);
        const uint32_t last = chunk_owner(T * Gn + Gn - 1, total, p.ncta);
        const int old = atomicAdd(&p.ws.tile_cnt[T], 1);
        const int is_last = (old == (int)(last - first));
        if (is_last) p.ws.tile_cnt[T] = 0;           // leave the counter ready for the next call
        s_flag[0] = is_last; s_flag[1] = (int)first; s_flag[2] = (int)last;
      }
      named_bar_sync(2, 128);
      if (!s_flag[0]) continue;
      __threadfence();
      const uint32_t first = (uint32_t)s_flag[1], last = (uint32_t)s_flag[2];
#pragma unroll
      for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[j][mt][e] = 0.f;
      for (uint32_t i = first; i <= last; ++i) {
        const int sl = (cta_first_chunk(i, total, p.ncta) / Gn == T) ? 0 : 1;
        const float4* src = reinterpret_cast<const float4*>(p.ws.slots) + ((size_t)i * 2 + sl) * slot_f4;
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            const float4 v = __ldcg(&src[((wn * 4 + j) * MT + mt) * 32 + lane]);
            acc[j][mt][0] += v.x; acc[j][mt][1] += v.y; acc[j][mt][2] += v.z; acc[j][mt][3] += v.w;
          }
      }
    }

    // ---- epilogue: bf16 store, arg-max candidates ------------------------------------------
    const int col0 = (int)T * kTileN + wn * 32;
    if (p.Y != nullptr) {
#pragma unroll
      for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
          const int r0 = mt * 16 + g8, c = col0 + 8 * j + 2 * t;
          if (r0 < p.M) *reinterpret_cast<uint32_t*>(p.Y + (size_t)r0 * p.ldy + c) = pack_bf16x2_rn(acc[j][mt][0], acc[j][mt][1]);
          if (r0 + 8 < p.M) *reinterpret_cast<uint32_t*>(p.Y + (size_t)(r0 + 8) * p.ldy + c) = pack_bf16x2_rn(acc[j][mt][2], acc[j][mt][3]);
        }
    }
    if (p.argmax_out != nullptr) {
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          float bv = -INFINITY;
          int bi = col0 + 2 * t;
#pragma unroll
          for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int e = 0; e < 2; ++e) amax_merge(bv, bi, acc[j][mt][2 * h + e], col0 + 8 * j + 2 * t + e);
#pragma unroll
          for (int off = 1; off <= 2; off <<= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
            amax_merge(bv, bi, ov, oi);
          }
          if (t == 0) s_amax[wn * 64 + mt * 16 + 8 * h + g8] = make_float2(bv, __int_as_float(bi));
        }
      named_bar_sync(2, 128);
      if (tid < p.m_pad) {
        float bv = -INFINITY;
        int bi = 0x7fffffff;
        for (int w = 0; w < 4; ++w) {
          const float2 c = s_amax[w * 64 + tid];
          amax_merge(bv, bi, c.x, __float_as_int(c.y));
        }
        __stcg(&p.ws.cand[(size_t)tid * p.n_tiles + T], make_float2(bv, __int_as_float(bi)));   // [row][tile]
      }
      __threadfence();
      named_bar_sync(2, 128);
      if (tid == 0) {
        const int old = atomicAdd(p.ws.amax_done, 1);
        const int is_last = (old == p.n_tiles - 1);
        if (is_last) *p.ws.amax_done = 0;
        s_flag[3] = is_last;
      }
      named_bar_sync(2, 128);
      if (s_flag[3]) {
        __threadfence();
        for (int row = warp; row < p.M; row += 4) {
          float bv = -INFINITY;
          int bi = 0x7fffffff;
          for (int t0 = lane; t0 < p.n_tiles; t0 += 32 * 8) {        // eight candidates per lane in flight
            float2 c[8];
#pragma unroll
            for (int q = 0; q < 8; ++q)
              c[q] = (t0 + 32 * q < p.n_tiles) ? __ldcg(&p.ws.cand[(size_t)row * p.n_tiles + t0 + 32 * q]) : make_float2(-INFINITY, __int_as_float(0x7fffffff));
#pragma unroll
            for (int q = 0; q < 8; ++q) amax_merge(bv, bi, c[q].x, __float_as_int(c[q].y));
          }
#pragma unroll
          for (int off = 16; off >= 1; off >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
            amax_merge(bv, bi, ov, oi);
          }
          if (lane == 0) p.argmax_out[row] = bi;
        }
      }
    }
  }
}

// ---- host side ---------------------------------------------------------------------------------
template <int MT, int G>
static cudaError_t launch_one(const LinearParams& p, size_t smem, cudaStream_t stream) {
  static bool attr_set[16] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 16 && !attr_set[dev]) {
    cudaError_t e = cudaFuncSetAttribute(qlinear_mma_kernel<MT, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBudget);
    if (e != cudaSuccess) return e;
    attr_set[dev] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.ncta);
  cfg.blockDim = dim3(mma_kgroups(MT) * 128 + 32);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see grid_dep_launch / grid_dep_wait in the kernel
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, qlinear_mma_kernel<MT, G>, p);
}

// Fills the path-specific fields of `p` (ring depth, X slots, resident or phased X); returns the
// dynamic shared memory the launch needs, 0 if the shape cannot run.
size_t plan_linear_mma(LinearParams& p) {
  const int mt = p.m_pad / 16;
  const int mtt = mt <= 1 ? 1 : (mt == 2 ? 2 : 4);           // kernels exist for 16, 32 and 64 padded rows
  p.m_pad = mtt * 16;
  p.stage_bytes = mma_stage_bytes(p.g);
  const uint32_t fixed = mma_fixed_smem(mtt);
  const uint32_t per_cta = (p.total_chunks + p.ncta - 1) / p.ncta;
  const uint32_t xslot = mma_xslot_bytes(p.g, p.m_pad);
  p.n_x = (int)(per_cta < (uint32_t)p.n_groups ? per_cta : (uint32_t)p.n_groups);
  p.x_phase = 0;
  const uint32_t min_ring = 6 * p.stage_bytes;
  if (fixed + (uint32_t)p.n_x * xslot + min_ring > kSmemBudget) {
    // X of all the CTA's groups does not fit beside a useful ring: reload it every x_phase chunks
    const int fit = (int)((kSmemBudget - fixed - min_ring) / xslot);
    if (fit < 1) return 0;
    p.n_x = fit;
    p.x_phase = fit;
  }
  const uint32_t xbytes = (uint32_t)p.n_x * xslot;
  int ns = (int)((kSmemBudget - fixed - xbytes) / p.stage_bytes);
  if (ns > kMaxStages) ns = kMaxStages;
  if ((uint32_t)ns > per_cta) ns = (int)per_cta;
  if (ns < 2) ns = 2;
  p.n_stages = ns;
  return (size_t)ns * p.stage_bytes + xbytes + fixed;
}

// Fills the path-specific fields of `p` and launches.  Returns a cudaError_t.
cudaError_t launch_linear_mma(LinearParams p, cudaStream_t stream) {
  const size_t smem = plan_linear_mma(p);
  if (smem == 0) return cudaErrorInvalidConfiguration;
  const int mtt = p.m_pad / 16;
  if (p.g == 128) {
    if (mtt == 1) return launch_one<1, 128>(p, smem, stream);
    if (mtt == 2) return launch_one<2, 128>(p, smem, stream);
    return launch_one<4, 128>(p, smem, stream);
  } else {
    if (mtt == 1) return launch_one<1, 64>(p, smem, stream);
    if (mtt == 2) return launch_one<2, 64>(p, smem, stream);
    return launch_one<4, 64>(p, smem, stream);
  }
}

}  // namespace ql
