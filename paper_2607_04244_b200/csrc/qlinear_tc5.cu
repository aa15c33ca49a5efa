// tcgen05 path of qlinear_w4a16 (ql_path QL_PATH_TC5): the 5th-generation tensor core does the
// contraction, with the weight tile as the 128-row A operand in tensor memory.
//
//     D^T[n, m] (128 x MPAD, fp32, TMEM)  =  sum_k  (q - z)[k, n] (A: TMEM, bf16)  *  X[m, k] (B: SMEM, K-major)
//
// per quantisation group; the per-group bf16 scale multiplies D in registers (one scalar per
// thread, because a thread owns one column n = one TMEM lane).
//
// CTA = 11 warps, persistent over a contiguous run of packed chunks (stream-K split, as in the
// warp-MMA path); two CTAs share an SM when M <= 16, so that with programmatic dependent launch
// the next linear streams its first weights while the current one drains.
//   warp 8  producer: one bulk copy per packed chunk into a ring of shared-memory stages
//   warps 9, 10  one thread each issues the tcgen05.mma of the chunks of one unpack group (G/16
//           instructions of K = 16 per chunk) and commits them to mbarriers; warp 9 also owns
//           the tensor-memory allocation
//   warps 0-7  two groups of 4 warps (128 threads = 128 columns) that take alternate chunks:
//           16-byte shared loads of the column's codes -> exact bf16 (q - z) pairs -> tcgen05.st
//           into an A buffer, half a chunk at a time (two A buffers per group, so unpacking the
//           next half overlaps the MMAs of the previous one); after the MMAs, tcgen05.ld of the
//           column's MPAD partial sums (two D buffers per group) and acc[m] += s * D[m], done
//           one chunk late so that it never waits for the tensor core.
// X (all groups the CTA touches) is loaded once into shared memory in the operand's canonical
// no-swizzle K-major layout [k/8][m][16 bytes].
// Split-K partial tiles, the last-arriver reduction and the arg-max are as in the warp-MMA path.
#include <cstdio>
#include <cstdlib>

#include "ql_params.h"

namespace ql {

constexpr int kTcThreads = 352;
constexpr int kTcMaxStages = 32;
constexpr uint32_t kTcSmemTwoPerSm = 114000u;   // two CTAs of this size (+1 KB each reserved) fit one SM
constexpr uint32_t kTcSmemBudget = 232448u;

__host__ __device__ inline uint32_t tc_stage_bytes(int g) { return align128(chunk_bytes(g)); }
__host__ __device__ inline uint32_t tc_xslot_bytes(int g, int m_pad) { return (uint32_t)m_pad * 2u * g; }
__host__ __device__ inline uint32_t tc_fixed_smem(int m_pad) { return 512u * m_pad + 2u * kTcMaxStages * 8u + 128u + 2048u + 64u; }

__device__ __forceinline__ void tc_amax_merge(float& bv, int& bi, float v, int i) {
  if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
}

template <int MPAD, int G>
__global__ void __launch_bounds__(kTcThreads, (MPAD == 16 ? 2 : 1)) qlinear_tc5_kernel(const __grid_constant__ LinearParams p) {
  extern __shared__ __align__(1024) uint8_t smem[];
  constexpr uint32_t STAGE = align128(chunk_bytes(G));
  constexpr uint32_t XSLOT = (uint32_t)MPAD * 2u * G;
  constexpr int NK = G / 16;                           // tcgen05.mma instructions per chunk
  constexpr int NC = G / 32;                           // 16-byte code words per column per chunk
  constexpr uint32_t TMEM_COLS = (G + 4 * MPAD <= 256) ? 256u : 512u;
  // tensor-memory columns: A buffer (group w, half h) at (2w+h)*(G/4), G/4 columns of bf16 pairs;
  //                        D buffer (group w, parity b) at G + (2w+b)*MPAD, MPAD fp32 columns
  const int NS = p.n_stages;
  uint8_t* ring = smem;
  uint8_t* xbuf = smem + (size_t)NS * STAGE;
  float* red = reinterpret_cast<float*>(xbuf + (size_t)p.n_x * XSLOT);            // [MPAD][128]
  uint64_t* full = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(red) + 512u * MPAD);
  uint64_t* empty = full + kTcMaxStages;
  uint64_t* a_full = empty + kTcMaxStages;             // [2][2] codes of half a chunk are in tensor memory
  uint64_t* a_empty = a_full + 4;                      // [2][2] the MMAs reading that A buffer have completed
  uint64_t* d_full = a_empty + 4;                      // [2][2] all MMAs of a chunk have completed
  uint64_t* x_full = d_full + 4;                       // X is in shared memory
  float2* s_amax = reinterpret_cast<float2*>(x_full + 4);                           // [4][64]
  int* s_flag = reinterpret_cast<int*>(s_amax + 4 * 64);
  volatile int* s_abort = s_flag + 8;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_flag + 9);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t Gn = p.n_groups;
  const uint32_t total = p.total_chunks;
  const uint32_t start = cta_first_chunk(blockIdx.x, total, p.ncta);
  const uint32_t end = cta_first_chunk(blockIdx.x + 1, total, p.ncta);
  const uint32_t my_chunks = end - start;

  grid_dep_launch();                                   // the next kernel in the stream may start its prologue
  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 4);
    }
    for (int i = 0; i < 4; ++i) {
      mbar_init(&a_full[i], 4);                        // one elected lane of each of the group's 4 warps
      mbar_init(&a_empty[i], 1);                       // tcgen05.commit
      mbar_init(&d_full[i], 1);                        // tcgen05.commit
    }
    mbar_init(x_full, 8);
    *s_abort = 0;
    fence_mbar_init();
  }
  if (warp == 9) {
    tmem_alloc(s_tmem, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = *s_tmem;

  if (warp == 8) {
    // ------------------------------------------------------------------ producer
    if (lane == 0) {
      const uint64_t pol = policy_evict_first();
      const uint32_t cb = chunk_bytes(G);
      const uint8_t* src = p.packed + (size_t)start * cb;
      uint32_t s = 0, ph = 0;
      for (uint32_t it = 0; it < my_chunks; ++it, src += cb) {
        if (it >= (uint32_t)NS) mbar_wait(&empty[s], ph ^ 1, s_abort, p.ws.status, 1);
        mbar_arrive_expect_tx(&full[s], cb);
        bulk_g2s_hint(ring + (size_t)s * STAGE, src, cb, &full[s], pol);
        if (++s == (uint32_t)NS) { s = 0; ph ^= 1; }
      }
      if (*s_abort) {
        // a wait gave up somewhere: let this CTA's own copies land before the CTA exits
        const uint32_t n = my_chunks < (uint32_t)NS ? my_chunks : (uint32_t)NS;
        for (uint32_t k = 0; k < n; ++k) {
          const uint32_t i2 = my_chunks - 1 - k;
          const uint64_t t0 = globaltimer_ns();
          while (!mbar_try_wait(&full[i2 % NS], (i2 / NS) & 1) && globaltimer_ns() - t0 < 20000000ull) {}
        }
      }
    }
  } else if (warp >= 9) {
    // ------------------------------------------------------------------ MMA issue for group w = warp - 9
    if (lane == 0) {
      constexpr uint32_t idesc = tc_idesc_bf16_m128(MPAD);
      const uint32_t w = warp - 9;
      mbar_wait(x_full, 0, s_abort, p.ws.status, 2);
      tc_fence_after_sync();
      // descriptor of X slot 0, k-step 0; slot and k-step only move the 16-byte-granular start address
      const uint64_t desc0 = tc_smem_desc_kmajor(smem_u32(xbuf), MPAD * 16u, 128u);
      constexpr uint32_t KSTEP = (2u * MPAD * 16u) >> 4;      // two 8-column core matrices per k-step
      constexpr uint32_t SLOT = XSLOT >> 4;
      uint32_t xk = w;                                      // chunk i uses X slot i mod Gn
      if (xk >= Gn) xk -= Gn;
      const uint32_t a_base = tmem + 2 * w * (G / 4);
      for (uint32_t i = w, k = 0; i < my_chunks; i += 2, ++k) {
        const uint32_t d_tmem = tmem + G + (2 * w + (k & 1)) * MPAD;
        const uint64_t xdesc = desc0 + (uint64_t)(xk * SLOT);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          mbar_wait(&a_full[2 * w + h], k & 1, s_abort, p.ws.status, 3);
          tc_fence_after_sync();
#pragma unroll
          for (int jj = 0; jj < NK / 2; ++jj) {
            const int j = h * (NK / 2) + jj;
            tc_mma_ts_f16(d_tmem, a_base + h * (G / 4) + 8 * jj, xdesc + (uint64_t)(j * KSTEP), idesc, j > 0 ? 1u : 0u);
          }
          tc_commit(&a_empty[2 * w + h]);
        }
        tc_commit(&d_full[2 * w + (k & 1)]);
        xk += 2;
        if (xk >= Gn) xk -= Gn;
        if (xk >= Gn) xk -= Gn;                             // Gn == 1: 2 steps wrap twice
      }
    }
  } else {
    // ------------------------------------------------------------------ unpack / scale / epilogue
    const int w = warp >> 2;                           // chunk parity this group of 4 warps takes
    const int n = (warp & 3) * 32 + lane;              // column inside the 128-column tile = TMEM lane
    const uint32_t tlane = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t a_addr = tlane + 2 * w * (G / 4);       // + h*(G/4)
    const uint32_t d_addr = tlane + G + 2 * w * MPAD;       // + b*MPAD
    const size_t slot_f = ws_slot_floats(p.m_pad);
    const uint32_t g_first = start % Gn;

    grid_dep_wait();                                   // X and the workspace belong to earlier kernels until here
    {
      // X prologue: slot k = group (g_first + k) mod Gn, layout [k/8][m][16 bytes], rows >= M zero.
      // The copies are only waited for just before this warp's first MMA hand-off.
      constexpr uint32_t UPS = (uint32_t)MPAD * (G / 8);   // 16-byte units per slot (power of two)
      const uint32_t n_x = min(my_chunks, Gn);
      for (uint32_t u = tid; u < UPS; u += 256) {          // unit u = (k-octet ku, row m), the same for every slot
        const uint32_t ku = u / MPAD, m = u % MPAD;
        const bool live = (int)m < p.M;
        const uint16_t* row = p.X + (size_t)m * p.ldx + ku * 8;
        uint8_t* dst = xbuf + (size_t)u * 16;
        uint32_t Gi = g_first;
        for (uint32_t k = 0; k < n_x; ++k, dst += XSLOT) {
          cp_async16(dst, live ? (row + (size_t)Gi * G) : p.X, live ? 16u : 0u);
          if (++Gi == Gn) Gi = 0;
        }
      }
    }
    bool x_pending = true;
    auto publish_x = [&]() {
      asm volatile("cp.async.wait_all;" ::: "memory");
      fence_proxy_async();                             // generic-proxy writes -> visible to the tensor core
      __syncwarp();
      if (lane == 0) mbar_arrive(x_full);
      x_pending = false;
    };
    if (my_chunks <= (uint32_t)w) publish_x();         // this group has no chunk at all

    float acc[MPAD];
    uint32_t it = 0, pos = start, stg = 0, sph = 0;     // stg/sph: ring stage and phase of chunk `it`
    uint32_t kloc = 0;                                  // chunks this group has handed to the tensor core
    int seg = 0;

    // acc[m] += s * D[m] for the chunk number kq of this group (waits for its MMAs)
    auto drain = [&](uint32_t kq, float s_q) {
      const uint32_t b = kq & 1;
      mbar_wait(&d_full[2 * w + b], (kq >> 1) & 1, s_abort, p.ws.status, 4);
      tc_fence_after_sync();
#pragma unroll
      for (int mb = 0; mb < MPAD / 16; ++mb) {
        float d[16];
        tmem_ld16(d_addr + b * MPAD + 16 * mb, d);
        tmem_wait_ld();
#pragma unroll
        for (int m = 0; m < 16; ++m) acc[16 * mb + m] = fmaf(s_q, d[m], acc[16 * mb + m]);
      }
    };

    while (pos < end) {
      const uint32_t T = pos / Gn;
      const uint32_t g0 = pos - T * Gn;
      const uint32_t nch = min(Gn - g0, end - pos);
#pragma unroll
      for (int m = 0; m < MPAD; ++m) acc[m] = 0.f;
      bool has_prev = false;
      float s_prev = 0.f;

      for (uint32_t ci = 0; ci < nch; ++ci, ++it) {
        const uint32_t my_stage = stg, my_phase = sph;
        if (++stg == (uint32_t)NS) { stg = 0; sph ^= 1; }
        if ((int)(it & 1) != w) continue;
        const uint8_t* st = ring + (size_t)my_stage * STAGE;
        mbar_wait(&full[my_stage], my_phase, s_abort, p.ws.status, 5);
        const float sc = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(st + 64 * G)[n] << 16);
        const uint32_t z = (reinterpret_cast<const uint32_t*>(st + 64 * G + 256)[n >> 3] >> (4 * (n & 7))) & 0xFu;
        const uint32_t zb = 0x43004300u | z | (z << 16);
        const uint4* wst = reinterpret_cast<const uint4*>(st);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          if (kloc > 0) {
            // the MMAs of this group's previous chunk have finished reading A buffer h
            mbar_wait(&a_empty[2 * w + h], (kloc - 1) & 1, s_abort, p.ws.status, 6);
            tc_fence_after_sync();
          }
#pragma unroll
          for (int cc = 0; cc < NC / 2; ++cc) {
            uint32_t v[16];

            unpack_codes32(wst[(h * (NC / 2) + cc) * kTileN + n], zb, v);
            tmem_st16(a_addr + h * (G / 4) + 16 * cc, v);
          }
          if (x_pending) publish_x();
          tmem_wait_st();
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) {
            mbar_arrive(&a_full[2 * w + h]);
            if (h == 1) mbar_arrive(&empty[my_stage]);
          }
        }
        if (has_prev) drain(kloc - 1, s_prev);
        has_prev = true;
        s_prev = sc;
        ++kloc;
      }
      if (has_prev) {
        drain(kloc - 1, s_prev);
        tc_fence_before_sync();
      }

      // ---- end of a tile segment: add the two groups (fixed order: group 0 + group 1) -------
      if (x_pending) publish_x();                      // never enter a CTA-wide barrier with X unpublished:
                                                       // the other group's MMAs (hence its drain) wait for it
      if (w == 1) {
#pragma unroll
        for (int m = 0; m < MPAD; ++m) red[m * kTileN + n] = acc[m];
      }
      named_bar_sync(1, 256);
      if (w == 0) {
#pragma unroll
        for (int m = 0; m < MPAD; ++m) acc[m] += red[m * kTileN + n];
      }
      named_bar_sync(1, 256);
      const bool whole = (g0 == 0 && nch == Gn);
      pos += nch;
      const int my_seg = seg++;
      if (w == 1) continue;

      // ---- group 0 (threads 0..127) finishes the segment ------------------------------------
      if (!whole) {
        float* my = p.ws.slots + ((size_t)blockIdx.x * 2 + (my_seg == 0 ? 0 : 1)) * slot_f;
#pragma unroll
        for (int m = 0; m < MPAD; ++m) __stcg(&my[m * kTileN + n], acc[m]);
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
        for (int m = 0; m < MPAD; ++m) acc[m] = 0.f;
        constexpr int QB = 64 / MPAD;                    // contributors per round (register budget)
        for (uint32_t i0 = first; i0 <= last; i0 += QB) {
          // QB contributors per round: their loads are all in flight together; the adds keep CTA order
          const float* src[QB];
#pragma unroll
          for (int q = 0; q < QB; ++q) {
            const uint32_t i = min(i0 + q, last);
            const int sl = (cta_first_chunk(i, total, p.ncta) / Gn == T) ? 0 : 1;
            src[q] = p.ws.slots + ((size_t)i * 2 + sl) * slot_f;
          }
          float v[QB][MPAD];
#pragma unroll
          for (int q = 0; q < QB; ++q)
#pragma unroll
            for (int m = 0; m < MPAD; ++m) v[q][m] = __ldcg(&src[q][m * kTileN + n]);
#pragma unroll
          for (int q = 0; q < QB; ++q)
            if (i0 + q <= last) {
#pragma unroll
              for (int m = 0; m < MPAD; ++m) acc[m] += v[q][m];
            }
        }
      }

      const int col = (int)T * kTileN + n;
      if (p.Y != nullptr) {
#pragma unroll
        for (int m = 0; m < MPAD; ++m)
          if (m < p.M) reinterpret_cast<__nv_bfloat16*>(p.Y)[(size_t)m * p.ldy + col] = __float2bfloat16_rn(acc[m]);
      }
      if (p.argmax_out != nullptr) {
#pragma unroll
        for (int m = 0; m < MPAD; ++m) {
          float bv = acc[m];
          int bi = col;
#pragma unroll
          for (int off = 16; off >= 1; off >>= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
            const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
            tc_amax_merge(bv, bi, ov, oi);
          }
          if (lane == 0) s_amax[(warp & 3) * 64 + m] = make_float2(bv, __int_as_float(bi));
        }
        named_bar_sync(2, 128);
        if (tid < p.m_pad) {
          float bv = -INFINITY;
          int bi = 0x7fffffff;
          for (int q = 0; q < 4; ++q) {
            const float2 c = s_amax[q * 64 + tid];
            tc_amax_merge(bv, bi, c.x, __float_as_int(c.y));
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
            for (int t0 = lane; t0 < p.n_tiles; t0 += 32 * 8) {      // eight candidates per lane in flight
              float2 c[8];
#pragma unroll
              for (int q = 0; q < 8; ++q)
                c[q] = (t0 + 32 * q < p.n_tiles) ? __ldcg(&p.ws.cand[(size_t)row * p.n_tiles + t0 + 32 * q]) : make_float2(-INFINITY, __int_as_float(0x7fffffff));
#pragma unroll
              for (int q = 0; q < 8; ++q) tc_amax_merge(bv, bi, c[q].x, __float_as_int(c[q].y));
            }
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) {
              const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
              const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
              tc_amax_merge(bv, bi, ov, oi);
            }
            if (lane == 0) p.argmax_out[row] = bi;
          }
        }
      }
    }
  }

  // every tensor-memory access of the CTA is complete past this barrier
  tc_fence_before_sync();
  __syncthreads();
  if (warp == 9) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, TMEM_COLS);
  }
}

// ---- host side ---------------------------------------------------------------------------------
template <int MPAD, int G>
static cudaError_t tc_launch_one(const LinearParams& p, size_t smem, cudaStream_t stream, bool pdl) {
  static bool attr_set[16] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (dev < 16 && !attr_set[dev]) {
    cudaError_t e = cudaFuncSetAttribute(qlinear_tc5_kernel<MPAD, G>, cudaFuncAttributeMaxDynamicSharedMemorySize, kTcSmemBudget);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(qlinear_tc5_kernel<MPAD, G>, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
    if (e != cudaSuccess) return e;
    attr_set[dev] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(p.ncta);
  cfg.blockDim = dim3(kTcThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, qlinear_tc5_kernel<MPAD, G>, p);
}

// CTA count and shared-memory plan of the tcgen05 path.
struct TcPlan {
  int ncta, n_x, n_stages;
  size_t smem;
  bool ok;
};

// Tries two CTAs per SM first (M <= 16: more warps in flight hide the unpack latencies, and with
// programmatic dependent launch two consecutive linears overlap), then one CTA per SM.
static TcPlan tc_plan(const LinearParams& p, int sms) {
  const uint32_t stage = tc_stage_bytes(p.g), fixed = tc_fixed_smem(p.m_pad), xslot = tc_xslot_bytes(p.g, p.m_pad);
  TcPlan r = {};
  for (int per_sm = (p.m_pad == 16 ? 2 : 1); per_sm >= 1; --per_sm) {
    int ncta = sms * per_sm;
    if (ncta > kMaxCtas) ncta = kMaxCtas;
    if ((uint32_t)ncta > p.total_chunks) ncta = (int)p.total_chunks;
    const uint32_t per_cta = (p.total_chunks + ncta - 1) / ncta;
    const uint32_t n_x = per_cta < (uint32_t)p.n_groups ? per_cta : (uint32_t)p.n_groups;
    const uint32_t budget = per_sm == 2 ? kTcSmemTwoPerSm : kTcSmemBudget;
    const uint32_t min_ring = (per_sm == 2 ? 4u : 2u) * stage;
    if (fixed + n_x * xslot + min_ring > budget) continue;
    int ns = (int)((budget - fixed - n_x * xslot) / stage);
    if (ns > kTcMaxStages) ns = kTcMaxStages;
    if ((uint32_t)ns > per_cta) ns = (int)per_cta;
    if (ns < 2) ns = 2;
    r.ncta = ncta; r.n_x = (int)n_x; r.n_stages = ns;
    r.smem = (size_t)ns * stage + (size_t)n_x * xslot + fixed;
    r.ok = true;
    return r;
  }
  return r;
}

// True if the tcgen05 path can run the shape: X of every group a CTA touches must fit in shared
// memory beside a ring of at least two stages.
bool tc5_supported(const LinearParams& p, int sms) { return tc_plan(p, sms).ok; }

cudaError_t launch_linear_tc5(LinearParams p, int sms, cudaStream_t stream, bool pdl) {
  const TcPlan plan = tc_plan(p, sms);
  if (!plan.ok) return cudaErrorInvalidConfiguration;
  p.ncta = plan.ncta;
  p.n_x = plan.n_x;
  p.x_phase = 0;
  p.stage_bytes = tc_stage_bytes(p.g);
  p.n_stages = plan.n_stages;
  const size_t smem = plan.smem;
  if (p.g == 128) {
    if (p.m_pad == 16) return tc_launch_one<16, 128>(p, smem, stream, pdl);
    if (p.m_pad == 32) return tc_launch_one<32, 128>(p, smem, stream, pdl);
    return tc_launch_one<64, 128>(p, smem, stream, pdl);
  } else {
    if (p.m_pad == 16) return tc_launch_one<16, 64>(p, smem, stream, pdl);
    if (p.m_pad == 32) return tc_launch_one<32, 64>(p, smem, stream, pdl);
    return tc_launch_one<64, 64>(p, smem, stream, pdl);
  }
}

}  // namespace ql
