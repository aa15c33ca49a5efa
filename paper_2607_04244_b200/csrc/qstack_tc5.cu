// Persistent stack kernel: one cooperative launch runs a whole list of fused operations (the
// projections of many decoder layers and the LM head) with one CTA of 22 warps per SM, so that
// nothing of the hot path crosses a kernel boundary.
//
// Warps
//   0-15   four unpack groups of 128 threads (thread n of a group = column n of a 128-column tile =
//          tensor-memory lane n).  A group takes every fourth sub-chunk: it expands the int4 codes to
//          the exact bf16 integers q - z, stores them into tensor memory as the A operand, later
//          reads the 16 partial sums of its column back and adds them, scaled, to its accumulators.
//          The same 512 threads build the X operand of an operation and finish its tiles.
//   16     producer: one bulk copy (TMA engine, no tensor map, no multicast) per packed chunk into a
//          ring of shared-memory stages; it runs ahead over operation boundaries, so the weights of
//          operation j+1 are on chip while operation j is still being reduced.
//   17-20  one MMA issuer per unpack group (a tcgen05.mma costs its issuing thread ~50-150 cycles).
//   21     watcher: polls the counter of the previous operation, so that the other warps can work
//          while they wait, and computes the row scales 1/rms from the per-tile sums of squares.
//
// What keeps a chain of dependent operations short (each one needs every output of the one before):
//   * a group owns three half-chunk A buffers in tensor memory and unpacks the first one and a
//     half chunks of operation j+1 BEFORE its X exists (the A operand depends on weights only);
//     the issuers hold the MMAs back until X has been published;
//   * waiting is done with relaxed loads (no fence per poll); the one acquire fence follows the
//     successful poll;
//   * split tiles: a contributor writes its partial sums as (value, tag) pairs and then sets a
//     flag without a fence in between; the owner of the tile polls the flag, loads the pairs and
//     checks every tag (a pair is one 8-byte store, so a matching tag proves the value), adding them
//     in CTA order - deterministic, no floating-point atomics;
//   * the glue between linears is folded in: a finished tile also leaves the row sums of squares
//     of what the next operation normalises, and that operation builds its X operand as
//     bf16(in * rsqrt(mean square)) (optionally of silu(gate) * up) while it loads it;
//   * gate and up (two linears with one input) run as one dual operation: even groups take the gate
//     chunks, odd groups the up chunks of the same (tile, group) positions, they share X.
// Every wait is bounded: on expiry the CTA records QL_ERR_DEVICE_TIMEOUT, raises its abort flag
// (every later wait then falls through), lets its copies land, frees its tensor memory and exits.
// M <= 16 only.
#include "ql_params.h"

namespace ql {

constexpr int NWG = 4;                                  // unpack groups per CTA
constexpr int AH = 3;                                   // half-chunk A buffers per group
constexpr int MP = 16;                                  // padded rows
constexpr int kUnpackThreads = NWG * 128;               // 512
constexpr int kWarpProducer = NWG * 4, kWarpIssuer0 = NWG * 4 + 1, kWarpWatcher = NWG * 4 + 1 + NWG;
constexpr int kStThreads = (kWarpWatcher + 1) * 32;     // 704
constexpr int kStMaxStages = 24;
constexpr uint32_t kStSmemBudget = 232448u;
constexpr uint32_t kXLbo = 16u * MP + 16u;              // bytes between K-adjacent 8x16-byte core matrices (+16: bank spread)
__host__ __device__ constexpr uint32_t st_xslot_bytes(int g) { return (uint32_t)(g / 8) * kXLbo; }
__host__ __device__ constexpr uint32_t st_fixed_smem() { return NWG * MP * 128u * 4u + 1024u; }
constexpr uint32_t kSlotWords = 2u * MP * 128u;         // (value, tag) pairs of one CTA's partial tile, two matrices

__device__ __forceinline__ float st_silu(float v) { return v / (1.f + __expf(-v)); }
__device__ __forceinline__ void st_amax_merge(float& bv, int& bi, float v, int i) {
  if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
}
__device__ __forceinline__ int ld_relaxed(const int* p) {
  int v;
  asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_relaxed(int* p, int v) {
  asm volatile("st.relaxed.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void red_relaxed_add(int* p, int v) {
  asm volatile("red.relaxed.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void fence_gpu() { asm volatile("fence.acq_rel.gpu;" ::: "memory"); }
__device__ __forceinline__ void ld_pairs(const uint64_t* p, uint64_t& a, uint64_t& b) {
  asm volatile("ld.relaxed.gpu.global.v2.b64 {%0,%1}, [%2];" : "=l"(a), "=l"(b) : "l"(p) : "memory");
}
__device__ __forceinline__ void st_pairs(uint64_t* p, uint64_t a, uint64_t b) {
  asm volatile("st.relaxed.gpu.global.v2.b64 [%0], {%1,%2};" ::"l"(p), "l"(a), "l"(b) : "memory");
}
__device__ __forceinline__ uint64_t tagged(float v, uint32_t tag) { return ((uint64_t)tag << 32) | (uint64_t)__float_as_uint(v); }

struct WaitCtx {
  volatile int* s_abort;
  int* status;
  uint64_t budget;
};
__device__ __forceinline__ void wait_fail(const WaitCtx& w, int site) {
  *w.s_abort = 1;
  atomicCAS(w.status, 0, kStatusTimeout | (site << 8) | ((int)blockIdx.x << 16));
}
// Bounded wait on an mbarrier phase (see mbar_wait; the budget is a launch parameter here).
__device__ __forceinline__ void st_mbar_wait(uint64_t* bar, uint32_t parity, const WaitCtx& w, int site) {
  if (mbar_try_wait(bar, parity)) return;
  if (*w.s_abort) return;
  const uint64_t t0 = globaltimer_ns();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 63u) == 0) {
      if (*w.s_abort) return;
      if (globaltimer_ns() - t0 > w.budget) { wait_fail(w, site); return; }
    }
  }
}
// Bounded wait until a global word written by another CTA satisfies `*p >= target` (geq) or `*p == target`.
template <bool GEQ>
__device__ __forceinline__ void wait_global(const int* p, int target, const WaitCtx& w, int site) {
  int v = ld_relaxed(p);
  if (GEQ ? v >= target : v == target) return;
  if (*w.s_abort) return;
  const uint64_t t0 = globaltimer_ns();
  uint32_t spins = 0;
  for (;;) {
    v = ld_relaxed(p);
    if (GEQ ? v >= target : v == target) return;
    if ((++spins & 15u) == 0) {
      if (*w.s_abort) return;
      if (globaltimer_ns() - t0 > w.budget) { wait_fail(w, site); return; }
    }
  }
}
// Bounded wait until a shared-memory word of this CTA exceeds `seen`.
__device__ __forceinline__ void wait_shared_gt(volatile int* p, int seen, const WaitCtx& w, int site) {
  if (*p > seen) return;
  if (*w.s_abort) return;
  const uint64_t t0 = globaltimer_ns();
  uint32_t spins = 0;
  while (*p <= seen) {
    if ((++spins & 63u) == 0) {
      if (*w.s_abort) return;
      if (globaltimer_ns() - t0 > w.budget) { wait_fail(w, site); return; }
    }
  }
}

// The fields of a descriptor that every role needs at every operation (two 16-byte loads through
// the read-only path: the descriptors do not change while the kernel runs).
struct OpHead {
  uint32_t nc, cq, cr, cat_base, total_chunks;
  int n_groups, n_tiles, flags;
};
__device__ __forceinline__ OpHead load_head(const MegaOp* op) {
  const uint4 a = __ldg(reinterpret_cast<const uint4*>(op));
  const uint4 b = __ldg(reinterpret_cast<const uint4*>(op) + 1);
  OpHead h;
  h.nc = a.x; h.cq = a.y; h.cr = a.z; h.cat_base = a.w;
  h.total_chunks = b.x; h.n_groups = (int)b.y; h.n_tiles = (int)b.z; h.flags = (int)b.w;
  return h;
}
template <typename T>
__device__ __forceinline__ T* ldg_ptr(T* const* p) {
  return reinterpret_cast<T*>(__ldg(reinterpret_cast<const unsigned long long*>(p)));
}

template <int G>
__global__ void __launch_bounds__(kStThreads, 1) qstack_tc5_kernel(const __grid_constant__ StackParams sp) {
  extern __shared__ __align__(1024) uint8_t smem[];
  constexpr uint32_t STAGE = align128(chunk_bytes(G));
  constexpr uint32_t XSLOT = st_xslot_bytes(G);
  constexpr int NK = G / 16;                            // MMAs per chunk
  constexpr int NC = G / 32;                            // 16-byte code groups per column per chunk
  constexpr uint32_t AHC = G / 4;                       // tensor-memory columns of one half-chunk A buffer
  constexpr uint32_t TMEM_COLS = 512;
  constexpr uint32_t D_COL0 = NWG * AH * AHC;           // first accumulator column
  static_assert(D_COL0 + NWG * 2 * MP <= TMEM_COLS, "tensor memory layout");
  // tensor-memory columns: A buffer (group w, slot s) at (w*AH + s)*AHC; D buffer (group w, parity b) at D_COL0 + (2w+b)*MP
  const int NS = sp.n_stages;
  uint8_t* ring = smem;
  uint8_t* xbuf = smem + (size_t)NS * STAGE;
  float* red = reinterpret_cast<float*>(xbuf + (size_t)sp.n_x * XSLOT);                 // [NWG][MP][128]
  uint64_t* full = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(red) + NWG * MP * 128u * 4u);
  uint64_t* empty = full + kStMaxStages;
  uint64_t* a_full = empty + kStMaxStages;              // [NWG][AH]
  uint64_t* a_empty = a_full + NWG * AH;                // [NWG][AH]
  uint64_t* d_full = a_empty + NWG * AH;                // [NWG][2]
  uint64_t* x_full = d_full + NWG * 2;                  // [1]
  float* s_inv = reinterpret_cast<float*>(x_full + 2);  // [16] 1/rms per row of the operation being prepared
  int* s_flag = reinterpret_cast<int*>(s_inv + 16);     // [0..7]
  volatile int* s_abort = s_flag + 8;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_flag + 9);
  volatile int* s_dep = s_flag + 10;                    // operations whose predecessor is known to be complete
  volatile int* s_invrdy = s_flag + 11;                 // operations whose 1/rms values are in s_inv

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const MegaOp* __restrict__ ops = sp.ops;
  const WaitCtx wc = {s_abort, sp.ws.status, sp.wait_ns};
  const uint32_t cta = blockIdx.x;

  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(&full[s], 1);
      mbar_init(&empty[s], 4);
    }
    for (int i = 0; i < NWG * AH; ++i) {
      mbar_init(&a_full[i], 4);
      mbar_init(&a_empty[i], 1);
    }
    for (int i = 0; i < NWG * 2; ++i) mbar_init(&d_full[i], 1);
    mbar_init(x_full, NWG * 4);
    *s_abort = 0;
    *s_dep = 0;
    *s_invrdy = 0;
    fence_mbar_init();
  }
  if (warp == kWarpIssuer0) {
    tmem_alloc(s_tmem, TMEM_COLS);
    tmem_relinquish();
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem = *s_tmem;

  if (warp == kWarpProducer) {
    // ------------------------------------------------------------------ producer: runs ahead over all operations
    if (lane == 0) {
      const uint64_t pol = policy_evict_first();
      const uint32_t cb = chunk_bytes(G);
      uint32_t s = 0, ph = 0, gs = 0;
      for (int j = 0; j < sp.n_ops; ++j) {
        const OpHead h = load_head(ops + j);
        uint32_t start, end;
        op_local_range(h.nc, h.cq, h.cr, h.cat_base, h.total_chunks, cta, start, end);
        if (start >= end) continue;
        const uint8_t* p0 = ldg_ptr(&ops[j].packed0);
        const uint8_t* p1 = ldg_ptr(&ops[j].packed1);
        const int nmat = (h.flags & kOpDual) ? 2 : 1;
        for (uint32_t c = start; c < end; ++c) {
          for (int mt = 0; mt < nmat; ++mt, ++gs) {
            if (gs >= (uint32_t)NS) st_mbar_wait(&empty[s], ph ^ 1, wc, 1);
            if (*s_abort) goto producer_done;            // never arm a stage that may still be in use
            mbar_arrive_expect_tx(&full[s], cb);
            bulk_g2s_hint(ring + (size_t)s * STAGE, (mt ? p1 : p0) + (size_t)c * cb, cb, &full[s], pol);
            if (++s == (uint32_t)NS) { s = 0; ph ^= 1; }
          }
        }
      }
    producer_done:
      if (*s_abort) {
        // a wait gave up somewhere: let this CTA's own copies land before it exits
        const uint32_t n = gs < (uint32_t)NS ? gs : (uint32_t)NS;
        for (uint32_t k = 0; k < n; ++k) {
          const uint32_t i2 = gs - 1 - k;
          const uint64_t t0 = globaltimer_ns();
          while (!mbar_try_wait(&full[i2 % NS], (i2 / NS) & 1) && globaltimer_ns() - t0 < 20000000ull) {}
        }
      }
    }
  } else if (warp == kWarpWatcher) {
    // ------------------------------------------------------------------ watcher: dependencies and row scales
    for (int j = 0; j < sp.n_ops; ++j) {
      const OpHead h = load_head(ops + j);
      if (j > 0 && (h.flags & kOpWait)) {
        if (lane == 0) {
          const int need = __ldg(&ops[j - 1].n_tiles);
          wait_global<true>(&sp.ws.op_done[j - 1], need, wc, 7);
        }
        __syncwarp();
        fence_gpu();                                     // acquire: everything the finishers published
      }
      if (lane == 0) {
        __threadfence_block();
        *s_dep = j + 1;
      }
      const int prologue = __ldg(&ops[j].prologue);
      uint32_t start, end;
      op_local_range(h.nc, h.cq, h.cr, h.cat_base, h.total_chunks, cta, start, end);
      if (prologue != 0 && start < end) {
        // 1/rms of every row from the per-tile sums of squares the producer operation left
        // (fixed order: tiles of one parity ascending, then even + odd)
        const int src_tiles = __ldg(&ops[j].src_tiles);
        const float* ssq = sp.ws.ssq + (size_t)((j - 1) & 1) * sp.ws.n_tiles * 16;
        const int row = lane & 15, half = lane >> 4;
        float sum = 0.f;
        for (int t0 = half; t0 < src_tiles; t0 += 16) {
          float v[8];
#pragma unroll
          for (int q = 0; q < 8; ++q) v[q] = (t0 + 2 * q < src_tiles) ? __ldcg(&ssq[(size_t)(t0 + 2 * q) * 16 + row]) : 0.f;
#pragma unroll
          for (int q = 0; q < 8; ++q) sum += v[q];
        }
        const float other = __shfl_xor_sync(0xffffffffu, sum, 16);
        const float tot = half == 0 ? sum + other : other + sum;
        if (lane < 16) s_inv[row] = rsqrtf(tot / (float)(src_tiles * kTileN));
        __syncwarp();
        if (lane == 0) {
          __threadfence_block();
          *s_invrdy = j + 1;
        }
      }
      if (*s_abort) break;
    }
  } else if (warp >= kWarpIssuer0) {
    // ------------------------------------------------------------------ MMA issue for unpack group w
    if (lane == 0) {
      constexpr uint32_t idesc = tc_idesc_bf16_m128(MP);
      const uint32_t w = warp - kWarpIssuer0;
      const uint64_t desc0 = tc_smem_desc_kmajor(smem_u32(xbuf), kXLbo, 128u);
      constexpr uint32_t KSTEP = (2u * kXLbo) >> 4;     // one MMA contracts 16 rows of K = two core matrices
      constexpr uint32_t SLOT = XSLOT >> 4;
      const uint32_t a_base = tmem + w * AH * AHC;
      uint32_t k = 0;                                  // chunks this group has handed over so far
      uint32_t hs = 0;                                 // half-chunks
      uint32_t xops = 0;                               // operations this CTA took part in so far
      for (int j = 0; j < sp.n_ops; ++j) {
        const OpHead h = load_head(ops + j);
        uint32_t start, end;
        op_local_range(h.nc, h.cq, h.cr, h.cat_base, h.total_chunks, cta, start, end);
        if (start >= end) continue;
        const bool dual = (h.flags & kOpDual) != 0;
        const uint32_t Gn = (uint32_t)h.n_groups;
        const uint32_t n_sub = (end - start) * (dual ? 2u : 1u);
        ++xops;
        bool first = true;
        for (uint32_t e = w; e < n_sub; e += NWG, ++k) {
          uint32_t xk = dual ? (e >> 1) : e;           // X slot = chunk number within the CTA, modulo the group count
          xk = xk % Gn;
          const uint32_t d_tmem = tmem + D_COL0 + (2 * w + (k & 1)) * MP;
          const uint64_t xdesc = desc0 + (uint64_t)(xk * SLOT);
#pragma unroll
          for (int hh = 0; hh < 2; ++hh, ++hs) {
            const uint32_t slot = hs % AH;
            st_mbar_wait(&a_full[w * AH + slot], (hs / AH) & 1, wc, 3);
            if (first) {
              st_mbar_wait(x_full, (xops - 1) & 1, wc, 2);   // X of this operation is in shared memory
              first = false;
            }
            tc_fence_after_sync();
#pragma unroll
            for (int jj = 0; jj < NK / 2; ++jj) {
              const int jk = hh * (NK / 2) + jj;
              tc_mma_ts_f16(d_tmem, a_base + slot * AHC + 8 * jj, xdesc + (uint64_t)(jk * KSTEP), idesc, jk > 0 ? 1u : 0u);
            }
            tc_commit(&a_empty[w * AH + slot]);
          }
          tc_commit(&d_full[2 * w + (k & 1)]);
        }
      }
    }
  } else {
    // ------------------------------------------------------------------ unpack groups
    const int w = warp >> 2;
    const int wq = warp & 3;
    const int n = wq * 32 + lane;                      // column inside the tile = TMEM lane
    const uint32_t tlane = tmem + ((uint32_t)(wq * 32) << 16);
    const uint32_t a_addr = tlane + w * AH * AHC;
    const uint32_t d_addr = tlane + D_COL0 + 2 * w * MP;
    uint64_t* my_slot = reinterpret_cast<uint64_t*>(sp.ws.slots) + (size_t)cta * kSlotWords;
    uint32_t stg = 0, sph = 0;                          // ring stage / phase of the next sub-chunk (any group's)
    uint32_t kloc = 0;                                  // chunks this group has handed to the tensor core
    uint32_t hs = 0;                                    // half-chunks this group has stored
    float acc[MP];

    auto drain = [&](uint32_t kq, float s_q) {
      const uint32_t b = kq & 1;
      st_mbar_wait(&d_full[2 * w + b], (kq >> 1) & 1, wc, 4);
      tc_fence_after_sync();
      float d[16];
      tmem_ld16(d_addr + b * MP, d);
      tmem_wait_ld();
#pragma unroll
      for (int m = 0; m < 16; ++m) acc[m] = fmaf(s_q, d[m], acc[m]);
    };

    for (int j = 0; j < sp.n_ops; ++j) {
      const OpHead h = load_head(ops + j);
      uint32_t start, end;
      op_local_range(h.nc, h.cq, h.cr, h.cat_base, h.total_chunks, cta, start, end);
      if (start >= end) continue;
      const MegaOp* op = ops + j;
      const bool dual = (h.flags & kOpDual) != 0;
      const uint32_t Gn = (uint32_t)h.n_groups;
      const uint32_t my_chunks = end - start;
      const uint32_t tag = (sp.epoch << 9) | (uint32_t)(j + 1);
      bool x_done = false;
      uint32_t pre = 0;                                 // half-chunks of this operation stored before its X exists

      // -------- X duty (all 512 threads): wait for the previous operation, build the X operand --------
      auto x_duty = [&]() {
        constexpr uint32_t UPG = (uint32_t)MP * (G / 8);   // 16-byte units per group
        const uint32_t n_x = min(my_chunks, Gn);
        const uint32_t g_first = start % Gn;
        const uint32_t n_units = n_x * UPG;
        const int prologue = __ldg(&op->prologue);
        const int ld_in = __ldg(&op->ld_in);
        const uint16_t* in0 = ldg_ptr(&op->in0);
        // unit idx: slot k = idx / UPG, row m = (idx / (G/8)) % MP, k-unit ku = idx % (G/8): lanes run along K
        auto unit_addr = [&](uint32_t k, uint32_t m, uint32_t ku) -> uint8_t* {
          return xbuf + (size_t)k * XSLOT + ku * kXLbo + (m >> 3) * 128u + (m & 7u) * 16u;
        };
        wait_shared_gt(s_dep, j, wc, 8);
        __threadfence_block();
        if (prologue == 0) {
          for (uint32_t idx = tid; idx < n_units; idx += kUnpackThreads) {
            const uint32_t k = idx / UPG, r = idx % UPG;
            const uint32_t m = r / (G / 8), ku = r % (G / 8);
            uint32_t Gi = g_first + k;
            if (Gi >= Gn) Gi -= Gn;
            const bool live = (int)m < sp.M;
            cp_async16(unit_addr(k, m, ku), live ? (in0 + (size_t)m * ld_in + (size_t)Gi * G + ku * 8) : in0, live ? 16u : 0u);
          }
          asm volatile("cp.async.wait_all;" ::: "memory");
        } else {
          // X = bf16(v * 1/rms): v is the producer's bf16 output (prologue 1) or the fp32 product
          // silu(gate) * up it left in the workspace (prologue 2).  The loads of a batch are all
          // issued before any is used; 1/rms arrives from the watcher meanwhile.
          constexpr int XB = 4;
          const bool from_act = (prologue == 2);
          const float* act = sp.ws.act;
          const int K = __ldg(&op->K);
          uint16_t* xout = ldg_ptr(&op->xout);
          const int ld_xout = __ldg(&op->ld_xout);
          bool have_inv = false;
          for (uint32_t base = tid; base < n_units; base += kUnpackThreads * XB) {
            uint4 ra[XB], rb[XB];
            uint32_t kk[XB], mm[XB], uu[XB], gg[XB];
#pragma unroll
            for (int q = 0; q < XB; ++q) {
              const uint32_t idx = base + q * kUnpackThreads;
              const bool in_range = idx < n_units;
              const uint32_t k = in_range ? idx / UPG : 0, r = idx % UPG;
              const uint32_t m = r / (G / 8), ku = r % (G / 8);
              uint32_t Gi = g_first + k;
              if (Gi >= Gn) Gi -= Gn;
              kk[q] = k; mm[q] = m; uu[q] = ku; gg[q] = Gi;
              ra[q] = make_uint4(0u, 0u, 0u, 0u); rb[q] = ra[q];
              if (in_range && (int)m < sp.M) {
                const size_t col0 = (size_t)Gi * G + ku * 8;
                if (from_act) {
                  const uint4* p = reinterpret_cast<const uint4*>(act + (size_t)m * K + col0);
                  ra[q] = __ldcg(p);
                  rb[q] = __ldcg(p + 1);
                } else {
                  ra[q] = __ldcg(reinterpret_cast<const uint4*>(in0 + (size_t)m * ld_in + col0));
                }
              }
            }
            if (!have_inv) {
              wait_shared_gt(s_invrdy, j, wc, 9);
              __threadfence_block();
              have_inv = true;
            }
#pragma unroll
            for (int q = 0; q < XB; ++q) {
              const uint32_t idx = base + q * kUnpackThreads;
              if (idx >= n_units) continue;
              uint4 o = make_uint4(0u, 0u, 0u, 0u);
              if ((int)mm[q] < sp.M) {
                const float inv = s_inv[mm[q]];
                if (!from_act) {
                  o.x = pack_bf16x2_rn(bf16lo_to_f32(ra[q].x) * inv, bf16hi_to_f32(ra[q].x) * inv);
                  o.y = pack_bf16x2_rn(bf16lo_to_f32(ra[q].y) * inv, bf16hi_to_f32(ra[q].y) * inv);
                  o.z = pack_bf16x2_rn(bf16lo_to_f32(ra[q].z) * inv, bf16hi_to_f32(ra[q].z) * inv);
                  o.w = pack_bf16x2_rn(bf16lo_to_f32(ra[q].w) * inv, bf16hi_to_f32(ra[q].w) * inv);
                } else {
                  o.x = pack_bf16x2_rn(__uint_as_float(ra[q].x) * inv, __uint_as_float(ra[q].y) * inv);
                  o.y = pack_bf16x2_rn(__uint_as_float(ra[q].z) * inv, __uint_as_float(ra[q].w) * inv);
                  o.z = pack_bf16x2_rn(__uint_as_float(rb[q].x) * inv, __uint_as_float(rb[q].y) * inv);
                  o.w = pack_bf16x2_rn(__uint_as_float(rb[q].z) * inv, __uint_as_float(rb[q].w) * inv);
                }
                // the CTA that owns (tile 0, group Gi) writes the normalised X out for the record
                if (xout != nullptr && start + kk[q] < Gn)
                  *reinterpret_cast<uint4*>(xout + (size_t)mm[q] * ld_xout + (size_t)gg[q] * G + uu[q] * 8) = o;
              }
              *reinterpret_cast<uint4*>(unit_addr(kk[q], mm[q], uu[q])) = o;
            }
          }
        }
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) mbar_arrive(x_full);
        x_done = true;
      };

      // -------- chunks of this operation --------
      uint32_t pos = start, e = 0;                      // e: sub-chunk counter of the operation (this CTA)
      while (pos < end) {
        const uint32_t T = pos / Gn;
        const uint32_t g0 = pos - T * Gn;
        const uint32_t nch = min(Gn - g0, end - pos);
#pragma unroll
        for (int m = 0; m < MP; ++m) acc[m] = 0.f;
        // scale-and-accumulate lags the unpack by two chunks (two D buffers per group) and is done
        // before this chunk's tensor-memory stores are issued: a tcgen05.ld queued behind them waits
        int n_pend = 0;
        float s_p1 = 0.f, s_p2 = 0.f;
        const uint32_t n_sub = nch * (dual ? 2u : 1u);
        for (uint32_t si = 0; si < n_sub; ++si, ++e) {
          const uint32_t my_stage = stg, my_phase = sph;
          if (++stg == (uint32_t)NS) { stg = 0; sph ^= 1; }
          if ((int)(e % NWG) != w) continue;
          const uint8_t* st = ring + (size_t)my_stage * STAGE;
          st_mbar_wait(&full[my_stage], my_phase, wc, 5);
          const float sc = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(st + 64 * G)[n] << 16);
          const uint32_t z = (reinterpret_cast<const uint32_t*>(st + 64 * G + 256)[n >> 3] >> (4 * (n & 7))) & 0xFu;
          const uint32_t zb = 0x43004300u | z | (z << 16);
          const uint4* wst = reinterpret_cast<const uint4*>(st);
          if (n_pend == 2) { drain(kloc - 2, s_p2); n_pend = 1; }
#pragma unroll
          for (int hh = 0; hh < 2; ++hh, ++hs) {
            // the A buffers hold AH half-chunks: whatever fits is unpacked before X exists, then
            // the group turns to the X operand, whose MMAs free the buffers again
            if (!x_done && pre == AH) x_duty();
            ++pre;
            const uint32_t slot = hs % AH;
            if (hs >= AH) {
              st_mbar_wait(&a_empty[w * AH + slot], ((hs / AH) - 1) & 1, wc, 6);
              tc_fence_after_sync();
            }
#pragma unroll
            for (int cc = 0; cc < NC / 2; ++cc) {
              uint32_t v[16];
              unpack_codes32(wst[(hh * (NC / 2) + cc) * kTileN + n], zb, v);
              tmem_st16(a_addr + slot * AHC + 16 * cc, v);
            }
            tmem_wait_st();
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) {
              mbar_arrive(&a_full[w * AH + slot]);
              if (hh == 1) mbar_arrive(&empty[my_stage]);
            }
          }
          s_p2 = s_p1;
          s_p1 = sc;
          ++n_pend;
          ++kloc;
        }
        if (!x_done) x_duty();                           // fewer than AH half-chunks before the segment's end
        if (n_pend == 2) drain(kloc - 2, s_p2);
        if (n_pend >= 1) drain(kloc - 1, s_p1);
        tc_fence_before_sync();

        // ---- end of a tile segment: the four groups' accumulators meet in shared memory; from here
        //      on warp r owns row r of the tile and lane l its columns 4l..4l+3 ----
#pragma unroll
        for (int m = 0; m < MP; ++m) red[(w * MP + m) * kTileN + n] = acc[m];
        named_bar_sync(1, kUnpackThreads);
        const int rw = warp;
        float f0[4], f1[4] = {0.f, 0.f, 0.f, 0.f};
        {
          const float4* r4 = reinterpret_cast<const float4*>(red);
          const float4 v0 = r4[(0 * MP + rw) * 32 + lane], v1 = r4[(1 * MP + rw) * 32 + lane];
          const float4 v2 = r4[(2 * MP + rw) * 32 + lane], v3 = r4[(3 * MP + rw) * 32 + lane];
          if (dual) {                                    // even groups hold matrix 0, odd groups matrix 1
            f0[0] = v0.x + v2.x; f0[1] = v0.y + v2.y; f0[2] = v0.z + v2.z; f0[3] = v0.w + v2.w;
            f1[0] = v1.x + v3.x; f1[1] = v1.y + v3.y; f1[2] = v1.z + v3.z; f1[3] = v1.w + v3.w;
          } else {
            f0[0] = ((v0.x + v1.x) + v2.x) + v3.x; f0[1] = ((v0.y + v1.y) + v2.y) + v3.y;
            f0[2] = ((v0.z + v1.z) + v2.z) + v3.z; f0[3] = ((v0.w + v1.w) + v2.w) + v3.w;
          }
        }
        const bool whole = (g0 == 0 && nch == Gn);
        const bool finish = (g0 == 0);                   // my run contains the tile's first chunk
        pos += nch;
        const int nmat = dual ? 2 : 1;

        if (!whole && !finish) {
          // ---- contributor: (value, tag) pairs, then the flag; no fence in between - the owner
          //      checks every tag.  (A run that does not begin its tile meets it in its first
          //      segment, so one slot per CTA is enough.) ----
          for (int mt = 0; mt < nmat; ++mt) {
            const float* f = mt ? f1 : f0;
            uint64_t* dst = my_slot + (size_t)(mt * MP + rw) * kTileN + 4 * lane;
            st_pairs(dst, tagged(f[0], tag), tagged(f[1], tag));
            st_pairs(dst + 2, tagged(f[2], tag), tagged(f[3], tag));
          }
          named_bar_sync(1, kUnpackThreads);             // red is free; everybody's pairs are on their way
          if (tid == 0) st_relaxed(&sp.ws.tile_cnt[cta], (int)tag);
          continue;
        }
        if (!whole) {
          // ---- owner of a split tile: its own partial stays in registers; the others' are added in
          //      CTA order once their flags are up ----
          if (tid == 0) s_flag[1] = (int)run_chunk_owner(h.nc, h.cq, h.cr, h.cat_base + T * Gn + Gn - 1);
          named_bar_sync(1, kUnpackThreads);
          const uint32_t last = (uint32_t)s_flag[1];
          for (uint32_t i = cta + 1 + tid; i <= last; i += kUnpackThreads)
            wait_global<false>(&sp.ws.tile_cnt[i], (int)tag, wc, 10);
          named_bar_sync(1, kUnpackThreads);
          const uint64_t* slots64 = reinterpret_cast<const uint64_t*>(sp.ws.slots);
          for (int mt = 0; mt < nmat; ++mt) {
            float* f = mt ? f1 : f0;
            for (uint32_t i0 = cta + 1; i0 <= last; i0 += 2) {
              uint64_t v[2][4];
#pragma unroll
              for (int q = 0; q < 2; ++q) {
                const uint32_t i = min(i0 + q, last);
                const uint64_t* src = slots64 + (size_t)i * kSlotWords + (size_t)(mt * MP + rw) * kTileN + 4 * lane;
                ld_pairs(src, v[q][0], v[q][1]);
                ld_pairs(src + 2, v[q][2], v[q][3]);
              }
#pragma unroll
              for (int q = 0; q < 2; ++q) {
                if (i0 + q > last) continue;
                bool ok = (uint32_t)(v[q][0] >> 32) == tag && (uint32_t)(v[q][1] >> 32) == tag &&
                          (uint32_t)(v[q][2] >> 32) == tag && (uint32_t)(v[q][3] >> 32) == tag;
                if (!ok && !*s_abort) {
                  // the flag overtook some of the pairs: reload until every tag matches (bounded)
                  const uint64_t* src = slots64 + (size_t)(i0 + q) * kSlotWords + (size_t)(mt * MP + rw) * kTileN + 4 * lane;
                  const uint64_t t0 = globaltimer_ns();
                  while (!ok) {
                    ld_pairs(src, v[q][0], v[q][1]);
                    ld_pairs(src + 2, v[q][2], v[q][3]);
                    ok = (uint32_t)(v[q][0] >> 32) == tag && (uint32_t)(v[q][1] >> 32) == tag &&
                         (uint32_t)(v[q][2] >> 32) == tag && (uint32_t)(v[q][3] >> 32) == tag;
                    if (!ok && (*s_abort || globaltimer_ns() - t0 > wc.budget)) { wait_fail(wc, 11); break; }
                  }
                }
#pragma unroll
                for (int r = 0; r < 4; ++r) f[r] += __uint_as_float((uint32_t)v[q][r]);
              }
            }
          }
        }

        // ---- tile epilogue: bf16 stores, sums of squares for the next operation, arg-max ----
        {
          uint16_t* out0 = ldg_ptr(&op->out0);
          uint16_t* out1 = ldg_ptr(&op->out1);
          int32_t* argmax_out = ldg_ptr(&op->argmax_out);
          const int emit_ssq = __ldg(&op->emit_ssq);
          const int ld_out = __ldg(&op->ld_out);
          const int col = (int)T * kTileN + 4 * lane;
          const bool live = rw < sp.M;
          float a[4];
          uint2 y0;
          y0.x = pack_bf16x2_rn(f0[0], f0[1]);
          y0.y = pack_bf16x2_rn(f0[2], f0[3]);
          if (out0 != nullptr && live) *reinterpret_cast<uint2*>(out0 + (size_t)rw * ld_out + col) = y0;
          a[0] = bf16lo_to_f32(y0.x); a[1] = bf16hi_to_f32(y0.x); a[2] = bf16lo_to_f32(y0.y); a[3] = bf16hi_to_f32(y0.y);
          if (dual) {
            uint2 y1;
            y1.x = pack_bf16x2_rn(f1[0], f1[1]);
            y1.y = pack_bf16x2_rn(f1[2], f1[3]);
            if (live) *reinterpret_cast<uint2*>(out1 + (size_t)rw * ld_out + col) = y1;
            if (emit_ssq == 2) {
              a[0] = st_silu(a[0]) * bf16lo_to_f32(y1.x); a[1] = st_silu(a[1]) * bf16hi_to_f32(y1.x);
              a[2] = st_silu(a[2]) * bf16lo_to_f32(y1.y); a[3] = st_silu(a[3]) * bf16hi_to_f32(y1.y);
              // the fp32 product [M][N], for the operation that consumes it
              if (live) __stcg(reinterpret_cast<float4*>(sp.ws.act + (size_t)rw * __ldg(&op->N) + col), make_float4(a[0], a[1], a[2], a[3]));
            }
          }
          if (emit_ssq != 0) {
            float sq = ((a[0] * a[0] + a[1] * a[1]) + a[2] * a[2]) + a[3] * a[3];
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, off);
            if (lane == 0) __stcg(&sp.ws.ssq[((size_t)(j & 1) * sp.ws.n_tiles + T) * 16 + rw], sq);
          }
          if (argmax_out != nullptr) {
            float bv = f0[0];
            int bi = col;
#pragma unroll
            for (int r = 1; r < 4; ++r) st_amax_merge(bv, bi, f0[r], col + r);
#pragma unroll
            for (int off = 16; off >= 1; off >>= 1) {
              const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
              const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
              st_amax_merge(bv, bi, ov, oi);
            }
            if (lane == 0) __stcg(&sp.ws.cand[(size_t)T * MP + rw], make_float2(bv, __int_as_float(bi)));
          }
          named_bar_sync(1, kUnpackThreads);             // all stores of the tile issued; red is free again
          if (argmax_out != nullptr) {
            // the CTA that finishes the operation's last tile reduces the per-tile candidates
            if (tid == 0) {
              int old;
              asm volatile("atom.add.acq_rel.gpu.global.s32 %0, [%1], 1;" : "=r"(old) : "l"(sp.ws.amax_done) : "memory");
              const int is_last = (old == h.n_tiles - 1);
              if (is_last) *sp.ws.amax_done = 0;
              s_flag[3] = is_last;
            }
            named_bar_sync(1, kUnpackThreads);
            if (s_flag[3]) {
              for (int row = warp; row < sp.M; row += NWG * 4) {
                float bv = -INFINITY;
                int bi = 0x7fffffff;
                for (int tt = lane; tt < h.n_tiles; tt += 32) {
                  const float2 c = __ldcg(&sp.ws.cand[(size_t)tt * MP + row]);
                  st_amax_merge(bv, bi, c.x, __float_as_int(c.y));
                }
#pragma unroll
                for (int off = 16; off >= 1; off >>= 1) {
                  const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
                  const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
                  st_amax_merge(bv, bi, ov, oi);
                }
                if (lane == 0) argmax_out[row] = bi;
              }
            }
            named_bar_sync(1, kUnpackThreads);
          }
          // the tile is complete: publish it to the operation's counter (one fence after everybody's stores)
          if (tid == 0 && !(h.flags & kOpNoRelease)) {
            fence_gpu();
            red_relaxed_add(&sp.ws.op_done[j], 1);
          }
        }
      }
    }
  }

  // every tensor-memory access of the CTA is complete past this barrier
  tc_fence_before_sync();
  __syncthreads();
  if (warp == kWarpIssuer0) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, TMEM_COLS);
  }
  if (tid == 0) {
    // the last CTA to leave restores the operation counters for the next launch
    __threadfence();
    const int old = atomicAdd(sp.ws.exit_cnt, 1);
    if (old == (int)gridDim.x - 1) {
      for (int j = 0; j < sp.n_ops; ++j) sp.ws.op_done[j] = 0;
      *sp.ws.amax_done = 0;
      *sp.ws.exit_cnt = 0;
    }
  }
}

// ---- host side ---------------------------------------------------------------------------------

// Shared-memory plan for a list of operations with common M <= 16 and g whose split fields are
// set; ok = false if some operation's X does not fit beside a ring of at least 6 stages.
struct StackPlan {
  int ncta, n_x, n_stages;
  size_t smem;
  bool ok;
};

int stack_ncta(int sms) { return sms < kMaxCtas / 2 ? sms : kMaxCtas / 2; }   // one 32 KB partial slot per CTA

StackPlan stack_plan(const MegaOp* ops, int n_ops, int g, int sms) {
  StackPlan r = {};
  const int ncta = stack_ncta(sms);
  uint32_t n_x = 1;
  for (int j = 0; j < n_ops; ++j) {
    // the longest piece of this operation that one CTA owns
    uint32_t longest = 0;
    const uint32_t nc = ops[j].nc;
    for (uint32_t i = 0; i < nc; ++i) {
      uint32_t lo, hi;
      op_local_range(ops[j].nc, ops[j].cq, ops[j].cr, ops[j].cat_base, ops[j].total_chunks, i, lo, hi);
      if (hi - lo > longest) longest = hi - lo;
    }
    const uint32_t need = longest < (uint32_t)ops[j].n_groups ? longest : (uint32_t)ops[j].n_groups;
    if (need > n_x) n_x = need;
  }
  const uint32_t stage = align128(chunk_bytes(g)), xslot = st_xslot_bytes(g);
  const uint32_t fixed = st_fixed_smem();
  if (fixed + n_x * xslot + 6 * stage > kStSmemBudget) return r;
  int ns = (int)((kStSmemBudget - fixed - n_x * xslot) / stage);
  if (ns > kStMaxStages) ns = kStMaxStages;
  r.ncta = ncta; r.n_x = (int)n_x; r.n_stages = ns;
  r.smem = (size_t)ns * stage + (size_t)n_x * xslot + fixed;
  r.ok = true;
  return r;
}

template <int G>
static cudaError_t stack_launch_g(const StackParams& sp, size_t smem, cudaStream_t stream) {
  // all CTAs wait on one another's progress: they must be co-resident (the cooperative launch checks it)
  cudaError_t e = cudaFuncSetAttribute(qstack_tc5_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStSmemBudget);
  if (e != cudaSuccess) return e;
  void* args[] = {const_cast<StackParams*>(&sp)};
  return cudaLaunchCooperativeKernel(reinterpret_cast<void*>(qstack_tc5_kernel<G>), dim3(sp.ncta), dim3(kStThreads), args, smem, stream);
}

cudaError_t launch_stack_tc5(const StackParams& sp, int g, size_t smem, cudaStream_t stream) {
  return g == 128 ? stack_launch_g<128>(sp, smem, stream) : stack_launch_g<64>(sp, smem, stream);
}

}  // namespace ql
