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
//   17-20  one MMA-issuing thread per unpack group (a tcgen05.mma with N = 16 costs its issuing thread
//          ~100 cycles while tensor-memory stores are running, and a chunk needs 8); in the variant
//          for chains two of them share a warp (lanes 0 and 16), so that 20 warps leave 96 registers
//          per thread; the watcher and the X loader follow the issuer warps.
//   21     watcher: polls the counter of the previous operation, so that the other warps can work
//          while they wait, and computes the row scales 1/rms from the per-tile sums of squares.
//   22     X loader, only for one stream of independent linears: copies the X columns of every chunk
//          into a ring of X slots ahead of the MMAs (cp.async, completion on an mbarrier per slot),
//          so that an operation boundary costs the unpack groups nothing and K may be of any length.
//
// What keeps a chain of dependent operations short (each one needs every output of the one before):
//   * a group owns three half-chunk A buffers in tensor memory and unpacks the first one and a
//     half chunks of operation j+1 BEFORE its X exists (the A operand depends on weights only);
//     the issuers hold the MMAs back until X has been published;
//   * waiting is done with relaxed loads (no fence per poll); one acquire load per counter follows
//     the successful poll;
//   * the end of a tile is handled row by row: after one exchange through shared memory warp r owns
//     row r, and from there on the 16 warps never meet again - a contributor's warp stores its row
//     of the partial tile into its slot, whose words are an "empty" bit pattern until a value lands;
//     the owner's warp r polls the contributors' slots until no word is empty, adds the rows in CTA
//     order, puts the empty pattern back (deterministic, no floating-point atomics), stores the bf16 row and the
//     row's sum of squares and publishes the row to a per-row counter of the operation;
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
constexpr int kWarpProducer = NWG * 4, kWarpIssuer0 = NWG * 4 + 1;
// One issuing thread per unpack group.  PAIRED (chains): two of them share a warp (lanes 0 and 16), the CTA has
// 20 warps and 96 registers per thread - in a chain the issuers mostly wait, and the unpack loop gains more
// from the registers than it loses from the shared issue slot.  Streams keep one warp per issuer (80 registers).
__host__ __device__ constexpr int st_issuer_warps(bool paired) { return paired ? NWG / 2 : NWG; }
__host__ __device__ constexpr int st_warp_watcher(bool paired) { return kWarpIssuer0 + st_issuer_warps(paired); }
__host__ __device__ constexpr int st_threads(bool ring, bool paired) { return (st_warp_watcher(paired) + 1 + (ring ? 1 : 0)) * 32; }   // the X loader follows the watcher
constexpr int kXRingSlots = 16;                         // X slots of the ring (one stream of independent linears)
constexpr int kStMaxStages = 24;
constexpr uint32_t kStSmemBudget = 232448u;
constexpr uint32_t kXLbo = 16u * MP + 16u;              // bytes between K-adjacent 8x16-byte core matrices (+16: bank spread)
__host__ __device__ constexpr uint32_t st_xslot_bytes(int g) { return (uint32_t)(g / 8) * kXLbo; }
// accumulator exchange buffer + barriers, flags and the two descriptor slots (656 + 64 + 128 + 320 bytes);
// the table of descriptor heads (32 bytes per operation) follows
__host__ __device__ constexpr uint32_t st_fixed_smem() { return NWG * MP * 128u * 4u + 2048u; }
constexpr uint32_t kSlotWords = 2u * MP * 128u;         // floats of one CTA's partial tile, two matrices

__device__ __forceinline__ float st_silu(float v) { return __fdividef(v, 1.f + __expf(-v)); }
__device__ __forceinline__ void st_amax_merge(float& bv, int& bi, float v, int i) {
  if (v > bv || (v == bv && i < bi)) { bv = v; bi = i; }
}
__device__ __forceinline__ int ld_relaxed(const int* p) {
  int v;
  asm volatile("ld.relaxed.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_relaxed(int* p, int v) {
  asm volatile("st.relaxed.gpu.global.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void red_relaxed_add(int* p, int v) {
  asm volatile("red.relaxed.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ void fence_gpu() { asm volatile("fence.acq_rel.gpu;" ::: "memory"); }
// Partial rows travel between CTAs as plain fp32 words that signal themselves: a word of the slot is
// kPartEmpty until the contributor's value lands (32-bit accesses are single-copy atomic), and the
// owner puts kPartEmpty back once it has added the row - no fence after the stores, no flag, no fence
// before the loads.  The put-back is ordered before the slot's next use (two operations later, or
// the next launch) by the owner's own publish fence and the chain of waits behind it.
__device__ __forceinline__ void st_part(float* p, float a, float b, float c, float d) {
  uint32_t u0 = __float_as_uint(a), u1 = __float_as_uint(b), u2 = __float_as_uint(c), u3 = __float_as_uint(d);
  u0 = u0 == kPartEmpty ? 0x7FFFFFFFu : u0; u1 = u1 == kPartEmpty ? 0x7FFFFFFFu : u1;   // (a NaN stays a NaN)
  u2 = u2 == kPartEmpty ? 0x7FFFFFFFu : u2; u3 = u3 == kPartEmpty ? 0x7FFFFFFFu : u3;
  asm volatile("st.relaxed.gpu.global.v4.b32 [%0], {%1, %2, %3, %4};" ::"l"(p), "r"(u0), "r"(u1), "r"(u2), "r"(u3) : "memory");
}
__device__ __forceinline__ void ld_part(const float* p, uint32_t (&u)[4]) {
  asm volatile("ld.relaxed.gpu.global.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]) : "l"(p) : "memory");
}
__device__ __forceinline__ void clear_part(float* p) {
  asm volatile("st.relaxed.gpu.global.v4.b32 [%0], {%1, %1, %1, %1};" ::"l"(p), "r"(kPartEmpty) : "memory");
}

// In-kernel timeline (builds with -DQL_TIMELINE): thread 0 of a CTA stamps the phases of every
// operation, the watcher's lane 0 the moment it saw the previous operation complete.
// slots: 0 operation entered, 1 first chunk unpacked (before X), 2 dependency seen, 3 X built,
//        4 last chunk of the first segment drained, 5 its accumulators exchanged, 6 its tile published / partial sent,
//        7 watcher saw the predecessor complete; of the LAST segment: 8 drained, 9 exchanged, 10 contributors' flags
//        seen, 11 partials added, 12 epilogue stores issued, 13 barrier passed, 14 published / partial sent
#ifdef QL_TIMELINE
// (stamps are SM cycle counts, comparable within a thread block; slots 7 and 15 also exist as globaltimer
//  nanoseconds, 256 ns resolution, in a second array for comparisons between thread blocks)
#define QL_STAMP(slot) do { if (sp.timeline != nullptr && tid == 0) { sp.timeline[((size_t)cta * sp.n_ops + j) * 16 + (slot)] = (uint64_t)clock64(); \
    if ((slot) == 14) sp.timeline[((size_t)cta * sp.n_ops + j) * 16 + 15] = globaltimer_ns(); } } while (0)
#define QL_STAMP_W(slot) do { if (sp.timeline != nullptr && lane == 0) { sp.timeline[((size_t)cta * sp.n_ops + j) * 16 + (slot)] = (uint64_t)clock64(); \
    sp.timeline[(size_t)160 * sp.n_ops * 16 + (size_t)2 * 160 * NWG * 8 + (size_t)cta * sp.n_ops + j] = globaltimer_ns(); } } while (0)
// cycle accounting of the unpack loop (lane 0 of the first warp of every group):
// 0 wait for the ring stage, 1 wait for a free A buffer, 2 unpack + tensor-memory stores issued, 3 wait::st,
// 4 wait for the MMAs of the chunk two back, 5 tensor-memory load + scale-accumulate, 6 chunks
#define QL_CYC_DECL long long cyc_[8] = {0, 0, 0, 0, 0, 0, 0, 0}; long long cyc_te_ = 0; (void)cyc_te_; long long cyc_t_ = clock64(); (void)cyc_t_
#define QL_CYC_BEGIN() do { const long long now_ = clock64(); cyc_[7] += now_ - cyc_t_; cyc_t_ = now_; } while (0)   /* slot 7: everything else */
#define QL_CYC_END(i) do { const long long now_ = clock64(); cyc_[i] += now_ - cyc_t_; cyc_t_ = now_; } while (0)
#define QL_CYC_ADD(i, v) do { cyc_[i] += (v); } while (0)
#define QL_CYC_FLUSH() do { if (sp.timeline != nullptr && wq == 0 && lane == 0) { \
    uint64_t* dst_ = sp.timeline + (size_t)160 * sp.n_ops * 16 + ((size_t)cta * NWG + w) * 8; \
    for (int i_ = 0; i_ < 8; ++i_) dst_[i_] = (uint64_t)cyc_[i_]; \
    sp.timeline[(size_t)160 * sp.n_ops * 16 + (size_t)2 * 160 * NWG * 8 + (size_t)160 * sp.n_ops + (size_t)cta * NWG + w] = (uint64_t)cyc_te_; } } while (0)
#define QL_CYC_FLUSH_I() do { if (sp.timeline != nullptr) { \
    uint64_t* dst_ = sp.timeline + (size_t)160 * sp.n_ops * 16 + (size_t)160 * NWG * 8 + ((size_t)cta * NWG + w) * 8; \
    for (int i_ = 0; i_ < 8; ++i_) dst_[i_] = (uint64_t)cyc_[i_]; } } while (0)
#else
#define QL_CYC_FLUSH_I() do {} while (0)
#define QL_STAMP(slot) do {} while (0)
#define QL_STAMP_W(slot) do {} while (0)
#define QL_CYC_DECL do {} while (0)
#define QL_CYC_BEGIN() do {} while (0)
#define QL_CYC_END(i) do {} while (0)
#define QL_CYC_ADD(i, v) do {} while (0)
#define QL_CYC_FLUSH() do {} while (0)
#endif

// Ablation switches for timing experiments (sp.ablate; the results are garbage when any is set):
// 1 no weight copies, unpacking or MMAs, 2 X operand not loaded or converted, 4 1/rms not awaited,
// 8 split tiles not exchanged, 16 rows published without the fence, 32 no accumulator exchange,
// 64 no row epilogue (publish only), 256 watcher without its acquire fence
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
// (SUSPEND: the single-thread roles that wait most of the time let the hardware suspend them)
template <bool SUSPEND = false>
__device__ __forceinline__ void st_mbar_wait(uint64_t* bar, uint32_t parity, const WaitCtx& w, int site) {
  if (mbar_try_wait(bar, parity)) return;
  if (*w.s_abort) return;
  const uint64_t t0 = globaltimer_ns();
  uint32_t spins = 0;
  while (!(SUSPEND ? mbar_try_wait_hint(bar, parity, 2000u) : mbar_try_wait(bar, parity))) {
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
    __nanosleep(32);                                     // leave the issue slots to the warps that work
    if ((++spins & 63u) == 0) {
      if (*w.s_abort) return;
      if (globaltimer_ns() - t0 > w.budget) { wait_fail(w, site); return; }
    }
  }
}

// The fields of a descriptor that every role needs at every operation (two 16-byte loads through
// the read-only path: the descriptors do not change while the kernel runs).
struct OpHead {
  uint32_t start, end;     // this CTA's chunks of the operation (per matrix); start >= end: none
  uint32_t last;           // the last CTA that works on the tile of chunk end - 1
  uint32_t total_chunks;
  int n_groups, n_tiles, flags;
};
// (when it starts, the kernel resolves the split of every operation for its own CTA and keeps the
// result in shared memory: no role repeats the split's divisions at every operation)
__device__ __forceinline__ OpHead load_head(const uint4* s_heads, int j) {
  const uint4 a = s_heads[2 * j];
  const uint4 b = s_heads[2 * j + 1];
  OpHead h;
  h.start = a.x; h.end = a.y; h.last = a.z;
  h.total_chunks = b.x; h.n_groups = (int)b.y; h.n_tiles = (int)b.z; h.flags = (int)b.w;
  return h;
}
__device__ __forceinline__ void resolve_head(const StackParams& sp, int j, uint32_t cta, uint4* s_heads) {
  const uint4 a = __ldg(reinterpret_cast<const uint4*>(sp.ops + j));
  const uint4 b = __ldg(reinterpret_cast<const uint4*>(sp.ops + j) + 1);
  const uint32_t Gn = b.y;
  uint32_t lo = 0, hi = 0, last = 0;
  op_local_range(a.x, a.y, a.z, a.w, b.x, cta, lo, hi);
  if (lo < hi) last = op_last_cta(a.x, a.y, a.z, a.w, Gn, (hi - 1) / Gn);
  s_heads[2 * j] = make_uint4(lo, hi, last, 0u);
  s_heads[2 * j + 1] = b;
}
template <typename T>
__device__ __forceinline__ T* ldg_ptr(T* const* p) {
  return reinterpret_cast<T*>(__ldg(reinterpret_cast<const unsigned long long*>(p)));
}

// X duty of one operation (all 512 unpack threads, no barrier among them): waits until the watcher
// has seen the previous operation complete, then builds the CTA's share of the X operand in shared
// memory - 16-byte units (8 consecutive k of one row) in the K-major core-matrix layout the MMA
// reads, slot k holding the group of the CTA's chunk number k.  `d` is the operation's descriptor
// in shared memory.  All loads of a thread are issued before the first is used.
template <int G>
__device__ __forceinline__ void build_x(const StackParams& sp, const MegaOp& d, int j, uint8_t* xbuf, const float* s_inv,
                                     volatile int* s_dep, volatile int* s_invrdy, uint64_t* x_full, const WaitCtx& wc,
                                     uint32_t start, uint32_t my_chunks, uint32_t Gn) {
  constexpr uint32_t XSLOT = st_xslot_bytes(G);
  constexpr uint32_t UPR = G / 8;                       // 16-byte units per row of one group
  constexpr uint32_t UPG = (uint32_t)MP * UPR;          // per group
  const int tid = threadIdx.x, lane = tid & 31;
  const uint32_t cta = blockIdx.x;
  (void)cta;
  const uint32_t n_x = min(my_chunks, Gn);
  const uint32_t g_first = start % Gn;
  const uint32_t n_units = n_x * UPG;
  const int prologue = d.prologue;
  const int rows = d.rows;
  const int ld_in = d.ld_in;
  const uint16_t* in0 = d.in0;
  // unit idx: slot k = idx / UPG, row m = (idx / UPR) % MP, k-unit ku = idx % UPR: lanes run along K
  auto unit_addr = [&](uint32_t idx) -> uint8_t* {
    const uint32_t k = idx / UPG, r = idx % UPG, m = r / UPR, ku = r % UPR;
    return xbuf + (size_t)k * XSLOT + ku * kXLbo + (m >> 3) * 128u + (m & 7u) * 16u;
  };
  auto unit_col = [&](uint32_t idx) -> size_t {          // first column (k index) of the unit in the source row
    const uint32_t k = idx / UPG, ku = idx % UPR;
    uint32_t Gi = g_first + k;
    if (Gi >= Gn) Gi -= Gn;
    return (size_t)Gi * G + ku * 8;
  };
  auto unit_row = [&](uint32_t idx) -> uint32_t { return (idx % UPG) / UPR; };
  wait_shared_gt(s_dep, j, wc, 8);
  __threadfence_block();
  QL_STAMP(2);
  if (sp.ablate & 2) {
    if (prologue != 0 && !(sp.ablate & 4)) { wait_shared_gt(s_invrdy, j, wc, 9); }
  } else if (prologue == 0) {
    for (uint32_t idx = tid; idx < n_units; idx += kUnpackThreads) {
      const uint32_t m = unit_row(idx);
      const bool live = (int)m < rows;
      cp_async16(unit_addr(idx), live ? (in0 + (size_t)m * ld_in + unit_col(idx)) : in0, live ? 16u : 0u);
    }
    asm volatile("cp.async.wait_all;" ::: "memory");
  } else {
    // X = bf16(v * 1/rms): v is the producer's bf16 output (prologue 1) or the fp32 product
    // silu(gate) * up it left in the workspace (prologue 2); 1/rms arrives from the watcher meanwhile.
    uint16_t* xout = d.xout;
    const int ld_xout = d.ld_xout;
    auto emit = [&](uint32_t idx, uint4 o) {
      const uint32_t m = unit_row(idx);
      // the CTA that owns (tile 0, group Gi) writes the normalised X out for the record
      if (xout != nullptr && (int)m < rows && start + idx / UPG < Gn)
        *reinterpret_cast<uint4*>(xout + (size_t)m * ld_xout + unit_col(idx)) = o;
      *reinterpret_cast<uint4*>(unit_addr(idx)) = o;
    };
    bool have_inv = false;
    auto need_inv = [&]() {
      if (!have_inv && !(sp.ablate & 4)) {
        wait_shared_gt(s_invrdy, j, wc, 9);
        __threadfence_block();
        have_inv = true;
      }
    };
    if (prologue == 1) {
      constexpr int XB = 10;                             // 10 units per thread cover 20 groups
      for (uint32_t base = tid; base < n_units; base += kUnpackThreads * XB) {
        uint4 ra[XB];
#pragma unroll
        for (int q = 0; q < XB; ++q) {
          const uint32_t idx = base + q * kUnpackThreads;
          ra[q] = make_uint4(0u, 0u, 0u, 0u);
          if (idx < n_units && (int)unit_row(idx) < rows)
            ra[q] = __ldcg(reinterpret_cast<const uint4*>(in0 + (size_t)unit_row(idx) * ld_in + unit_col(idx)));
        }
        need_inv();
#pragma unroll
        for (int q = 0; q < XB; ++q) {
          const uint32_t idx = base + q * kUnpackThreads;
          if (idx >= n_units) continue;
          const float inv = (int)unit_row(idx) < rows ? s_inv[unit_row(idx)] : 0.f;
          uint4 o;
          o.x = pack_bf16x2_rn(bf16lo_to_f32(ra[q].x) * inv, bf16hi_to_f32(ra[q].x) * inv);
          o.y = pack_bf16x2_rn(bf16lo_to_f32(ra[q].y) * inv, bf16hi_to_f32(ra[q].y) * inv);
          o.z = pack_bf16x2_rn(bf16lo_to_f32(ra[q].z) * inv, bf16hi_to_f32(ra[q].z) * inv);
          o.w = pack_bf16x2_rn(bf16lo_to_f32(ra[q].w) * inv, bf16hi_to_f32(ra[q].w) * inv);
          emit(idx, o);
        }
      }
    } else {
      constexpr int XB = 6;                              // 6 units per thread cover 12 groups
      const float* act = sp.ws.act;
      const int K = d.K;
      for (uint32_t base = tid; base < n_units; base += kUnpackThreads * XB) {
        uint4 ra[XB], rb[XB];
#pragma unroll
        for (int q = 0; q < XB; ++q) {
          const uint32_t idx = base + q * kUnpackThreads;
          ra[q] = make_uint4(0u, 0u, 0u, 0u); rb[q] = ra[q];
          if (idx < n_units && (int)unit_row(idx) < rows) {
            const uint4* p = reinterpret_cast<const uint4*>(act + (size_t)unit_row(idx) * K + unit_col(idx));
            ra[q] = __ldcg(p);
            rb[q] = __ldcg(p + 1);
          }
        }
        need_inv();
#pragma unroll
        for (int q = 0; q < XB; ++q) {
          const uint32_t idx = base + q * kUnpackThreads;
          if (idx >= n_units) continue;
          const float inv = (int)unit_row(idx) < rows ? s_inv[unit_row(idx)] : 0.f;
          uint4 o;
          o.x = pack_bf16x2_rn(__uint_as_float(ra[q].x) * inv, __uint_as_float(ra[q].y) * inv);
          o.y = pack_bf16x2_rn(__uint_as_float(ra[q].z) * inv, __uint_as_float(ra[q].w) * inv);
          o.z = pack_bf16x2_rn(__uint_as_float(rb[q].x) * inv, __uint_as_float(rb[q].y) * inv);
          o.w = pack_bf16x2_rn(__uint_as_float(rb[q].z) * inv, __uint_as_float(rb[q].w) * inv);
          emit(idx, o);
        }
      }
    }
  }
  fence_proxy_async();
  __syncwarp();
  if (lane == 0) mbar_arrive(x_full);
}

// RING: variant for one stream of independent linears whose X does not fit per operation (one more
// warp, the X loader; the issuers take X slot by slot).  The other variant has none of that code.
template <int G, bool RING, bool PAIRED>
__global__ void __launch_bounds__(st_threads(RING, PAIRED), 1) qstack_tc5_kernel(const __grid_constant__ StackParams sp) {
  constexpr int kWarpWatcher = st_warp_watcher(PAIRED);
  constexpr int kWarpXLoader = kWarpWatcher + 1;
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
  uint64_t* xr_full = x_full + 2;                       // [kXRingSlots] X ring: the slot's columns have landed
  uint64_t* xr_empty = xr_full + kXRingSlots;           // [kXRingSlots] the MMAs that read the slot are complete
  float* s_inv = reinterpret_cast<float*>(xr_empty + kXRingSlots);  // [16] 1/rms per row of the operation being prepared
  int* s_flag = reinterpret_cast<int*>(s_inv + 16);     // [0..7]
  volatile int* s_abort = s_flag + 8;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(s_flag + 9);
  volatile int* s_dep = s_flag + 10;                    // operations whose predecessor is known to be complete
  volatile int* s_invrdy = s_flag + 11;                 // operations whose 1/rms values are in s_inv
  volatile int* s_descrdy = s_flag + 12;                // operations whose descriptor is in s_desc
  volatile int* s_prog = s_flag + 16;                   // [16] operations (of those this CTA takes part in) each unpack warp has left behind
  MegaOp* s_desc = reinterpret_cast<MegaOp*>(s_flag + 32);   // [2] descriptors of the operations this CTA takes part in, filled by the watcher
  uint4* s_heads = reinterpret_cast<uint4*>(s_desc + 2);     // [n_ops][2] first 32 bytes of every descriptor

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
    for (int i = 0; i < kXRingSlots; ++i) {
      mbar_init(&xr_full[i], 32);                        // the loader's 32 lanes, each when its copies have landed
      mbar_init(&xr_empty[i], 1);
    }
    // a status word that is still set means an earlier launch gave up on this workspace and nobody has
    // initialised it again: its counters and partial-tile slots cannot be trusted, so this launch
    // does not wait for anything either (it runs through, and the status keeps saying why)
    *s_abort = ld_relaxed(sp.ws.status) != 0 ? 1 : 0;
    *s_dep = 0;
    *s_invrdy = 0;
    *s_descrdy = 0;
    for (int i = 0; i < 16; ++i) s_prog[i] = 0;
    fence_mbar_init();
  }
  if (warp == kWarpIssuer0) {
    tmem_alloc(s_tmem, TMEM_COLS);
    tmem_relinquish();
  }
  for (int i = tid; i < sp.n_ops; i += st_threads(RING, PAIRED)) resolve_head(sp, i, cta, s_heads);
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
        const OpHead h = load_head(s_heads, j);
        uint32_t start, end;
        start = h.start; end = h.end;
        if (start >= end) continue;
        if (sp.ablate & 1) continue;
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
    // ------------------------------------------------------------------ watcher: descriptors, dependencies, row scales
    int pcount = 0;                                      // operations this CTA took part in so far
    for (int j = 0; j < sp.n_ops; ++j) {
      const OpHead h = load_head(s_heads, j);
      {
        // operations this CTA has no chunk of need nothing from it: a later operation it takes part in
        // waits for its own predecessor, which cannot be complete before everything ahead of it is
        uint32_t lo, hi;
        lo = h.start; hi = h.end;
        if (lo >= hi) continue;
      }
      // the unpack warps read the descriptor from shared memory (two slots, alternating); a slot is
      // free once every unpack warp has left the operation that used it behind
      if (pcount >= 2) {
        const uint64_t t0 = globaltimer_ns();
        for (;;) {
          int p = lane < 16 ? s_prog[lane] : 0x7fffffff;
#pragma unroll
          for (int off = 8; off >= 1; off >>= 1) p = min(p, __shfl_xor_sync(0xffffffffu, p, off));
          p = __shfl_sync(0xffffffffu, p, 0);
          if (p >= pcount - 1 || *s_abort) break;
          if (globaltimer_ns() - t0 > wc.budget) { if (lane == 0) wait_fail(wc, 12); break; }
          __nanosleep(64);
        }
      }
      if (lane < (int)(sizeof(MegaOp) / 16)) reinterpret_cast<uint4*>(&s_desc[pcount & 1])[lane] = __ldg(reinterpret_cast<const uint4*>(ops + j) + lane);
      __syncwarp();
      if (lane == 0) {
        __threadfence_block();
        *s_descrdy = j + 1;
      }
      ++pcount;
      // an operation waits for the one before it (it consumes its output), or only for the one two
      // back (independent operations: the partial-tile slots and flags alternate between two sets)
      const int dep = (h.flags & kOpWait) ? j - 1 : -1;
      // (read before the wait: after it, every load is on the path to the next operation's X)
      const int prologue = __ldg(&ops[j].prologue);
      const int src_tiles = __ldg(&ops[j].src_tiles);
      if (dep >= 0) {
        // every tile is published row by row; lane r polls the counter of row r (one line per counter)
        if (lane < 16) {
          const int need = load_head(s_heads, dep).n_tiles;
          wait_global<true>(&sp.ws.op_done[((size_t)dep * 16 + lane) * kOpDoneStride], need, wc, 7);
        }
        // acquire: everything the finishers published.  One acquire load of the complete counter per
        // polling lane instead of a fence after the relaxed polls (the fence cost 0.9 us per operation)
        if (lane < 16 && !(sp.ablate & 256)) ld_acquire(&sp.ws.op_done[((size_t)dep * 16 + lane) * kOpDoneStride]);
        __syncwarp();
      }
      QL_STAMP_W(7);
      if (lane == 0) {
        __threadfence_block();
        *s_dep = j + 1;
      }
      uint32_t start, end;
      start = h.start; end = h.end;
      if (prologue != 0 && start < end) {
        // 1/rms of every row from the per-tile sums of squares the producer operation left
        // (fixed order: tiles of one parity ascending, then even + odd)
        const float* ssq = sp.ws.ssq + (size_t)((j - 1) & 1) * sp.ws.n_tiles * 16;
        const int row = lane & 15, half = lane >> 4;
        float sum = 0.f;
        for (int t0 = half; t0 < src_tiles; t0 += 80) {   // 40 loads in flight per lane: one round trip up to 80 tiles
          float v[40];
#pragma unroll
          for (int q = 0; q < 40; ++q) v[q] = (t0 + 2 * q < src_tiles) ? __ldcg(&ssq[(size_t)(t0 + 2 * q) * 16 + row]) : 0.f;
#pragma unroll
          for (int q = 0; q < 40; ++q) sum += v[q];
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
    if (lane == 0 && *s_abort) { *s_descrdy = 0x7ffffff0; *s_dep = 0x7ffffff0; *s_invrdy = 0x7ffffff0; }
  } else if (RING && warp == kWarpXLoader) {
    // ------------------------------------------------------------------ X loader (one stream of independent linears)
    if (sp.x_ring > 0 && !(sp.ablate & 1)) {
      constexpr uint32_t UPR = G / 8;                     // 16-byte units per row of one group
      const uint32_t P = (uint32_t)sp.x_ring;
      uint32_t r = 0;                                    // ring position = chunks of this CTA so far
      for (int j = 0; j < sp.n_ops; ++j) {
        const OpHead h = load_head(s_heads, j);
        uint32_t start, end;
        start = h.start; end = h.end;
        if (start >= end) continue;
        const uint16_t* in0 = ldg_ptr(&ops[j].in0);
        const int ld_in = __ldg(&ops[j].ld_in);
        const int rows = __ldg(&ops[j].rows);
        const uint32_t Gn = (uint32_t)h.n_groups;
        for (uint32_t c = start; c < end; ++c, ++r) {
          const uint32_t slot = r % P;
          if (r >= P) {
            if (lane == 0) st_mbar_wait(&xr_empty[slot], ((r / P) - 1) & 1, wc, 18);
            __syncwarp();
          }
          if (*s_abort) break;
          const uint32_t Gi = c % Gn;                    // the chunk's group
          uint8_t* dst = xbuf + (size_t)slot * XSLOT;
          // unit (row m, k-unit ku): lanes run along K, two rows per pass
#pragma unroll
          for (uint32_t u = (uint32_t)lane; u < (uint32_t)MP * UPR; u += 32) {
            const uint32_t m = u / UPR, ku = u % UPR;
            const bool live = (int)m < rows;
            cp_async16(dst + ku * kXLbo + (m >> 3) * 128u + (m & 7u) * 16u,
                       live ? (in0 + (size_t)m * ld_in + (size_t)Gi * G + ku * 8) : in0, live ? 16u : 0u);
          }
          cp_async_arrive_noinc(&xr_full[slot]);
        }
        if (*s_abort) break;
      }
      asm volatile("cp.async.wait_all;" ::: "memory");   // nothing of this warp is in flight when the CTA exits
    }
  } else if (warp >= kWarpIssuer0) {
    // ------------------------------------------------------------------ MMA issue for unpack group w
    if (PAIRED ? (lane & 15) == 0 : lane == 0) {
      constexpr uint32_t idesc = tc_idesc_bf16_m128(MP);
      const uint32_t w = PAIRED ? 2 * (warp - kWarpIssuer0) + (lane >> 4) : warp - kWarpIssuer0;   // unpack group served
      const uint64_t desc0 = tc_smem_desc_kmajor(smem_u32(xbuf), kXLbo, 128u);
      constexpr uint32_t KSTEP = (2u * kXLbo) >> 4;     // one MMA contracts 16 rows of K = two core matrices
      constexpr uint32_t SLOT = XSLOT >> 4;
      const uint32_t a_base = tmem + w * AH * AHC;
      uint32_t k = 0;                                  // chunks this group has handed over so far
      uint32_t hs = 0;                                 // half-chunks
      uint32_t xops = 0;                               // operations this CTA took part in so far whose X the unpack threads built
      uint32_t rbase = 0;                              // X ring: chunks of this CTA before the current operation
      const uint32_t P = RING ? (uint32_t)sp.x_ring : 1u;
      QL_CYC_DECL;
      for (int j = 0; j < sp.n_ops; ++j) {
        const OpHead h = load_head(s_heads, j);
        uint32_t start, end;
        start = h.start; end = h.end;
        if (start >= end) continue;
        const bool dual = (h.flags & kOpDual) != 0;
        const uint32_t Gn = (uint32_t)h.n_groups;
        const uint32_t n_sub = (end - start) * (dual ? 2u : 1u);
        constexpr bool ring = RING;                    // X comes chunk by chunk from the loader warp (never with dual operations)
        if (!ring) ++xops;
        if (sp.ablate & 1) { rbase += end - start; continue; }
        bool first = !ring;
        for (uint32_t e = w; e < n_sub; e += NWG, ++k) {
          uint32_t xk = dual ? (e >> 1) : e;           // X slot = chunk number within the CTA, modulo the group count
          if (ring) {
            const uint32_t r = rbase + e;
            xk = r % P;
            st_mbar_wait(&xr_full[xk], (r / P) & 1, wc, 17);
            fence_proxy_async();                         // the copies were generic-proxy writes; the MMAs read through the async proxy
          } else {
            xk = xk % Gn;
          }
          const uint32_t d_tmem = tmem + D_COL0 + (2 * w + (k & 1)) * MP;
          const uint64_t xdesc = desc0 + (uint64_t)(xk * SLOT);
#pragma unroll
          for (int hh = 0; hh < 2; ++hh, ++hs) {
            const uint32_t slot = hs % AH;
            QL_CYC_BEGIN();
            // in a chain the issuer waits most of the time (for X, for the predecessor): suspended it leaves
            // the issue slots to the unpack warps; on a stream its wake-up would cost more than its polling
            if (h.flags & kOpWait) st_mbar_wait<true>(&a_full[w * AH + slot], (hs / AH) & 1, wc, 3);
            else st_mbar_wait(&a_full[w * AH + slot], (hs / AH) & 1, wc, 3);
            QL_CYC_END(0);
            if (first) {
              st_mbar_wait(x_full, (xops - 1) & 1, wc, 2);   // X of this operation is in shared memory
              first = false;
            }
            QL_CYC_END(1);
            tc_fence_after_sync();
#pragma unroll
            for (int jj = 0; jj < NK / 2; ++jj) {
              const int jk = hh * (NK / 2) + jj;
              tc_mma_ts_f16(d_tmem, a_base + slot * AHC + 8 * jj, xdesc + (uint64_t)(jk * KSTEP), idesc, jk > 0 ? 1u : 0u);
            }
            tc_commit(&a_empty[w * AH + slot]);
            QL_CYC_END(2);
            QL_CYC_ADD(3, 1);
          }
          tc_commit(&d_full[2 * w + (k & 1)]);
          if (ring) tc_commit(&xr_empty[xk]);            // the slot may be refilled once this chunk's MMAs are complete
        }
        rbase += end - start;
      }
      QL_CYC_FLUSH_I();
    }
  } else {
    // ------------------------------------------------------------------ unpack groups
    const int w = warp >> 2;
    const int wq = warp & 3;
    const int n = wq * 32 + lane;                      // column inside the tile = TMEM lane
    const uint32_t tlane = tmem + ((uint32_t)(wq * 32) << 16);
    const uint32_t a_addr = tlane + w * AH * AHC;
    const uint32_t d_addr = tlane + D_COL0 + 2 * w * MP;
    constexpr uint32_t kSetCtas = kMaxCtas / 2;          // partial-tile slots and row flags: two sets of 160
    // per-row arg-max counters (rows 0..15) and the verification-tail counter (16), one 128-byte line each:
    // every CTA adds to them at about the same moment, and atomics on one line are served one after the other
    int* const amax_cnt = sp.ws.tile_cnt + kMaxTiles + kStackFlagWords;
    uint32_t stg = 0, sph = 0;                          // ring stage / phase of the next sub-chunk (any group's)
    uint32_t kloc = 0;                                  // chunks this group has handed to the tensor core
    uint32_t hs = 0;                                    // half-chunks this group has stored
    float acc[MP];
    QL_CYC_DECL;

    auto drain = [&](uint32_t kq, float s_q) {
      const uint32_t b = kq & 1;
      QL_CYC_BEGIN();
      st_mbar_wait(&d_full[2 * w + b], (kq >> 1) & 1, wc, 4);
      QL_CYC_END(4);
      tc_fence_after_sync();
      float d[16];
      tmem_ld16(d_addr + b * MP, d);
      tmem_wait_ld();
#pragma unroll
      for (int m = 0; m < 16; ++m) acc[m] = fmaf(s_q, d[m], acc[m]);
      QL_CYC_END(5);
    };

    int pcount = 0;                                      // operations this CTA took part in so far
    for (int j = 0; j < sp.n_ops; ++j) {
      const OpHead h = load_head(s_heads, j);
      uint32_t start, end;
      start = h.start; end = h.end;
      if (start >= end) continue;
      // the watcher has put the descriptor into shared memory (normally long before)
      if (lane == 0) wait_shared_gt(s_descrdy, j, wc, 13);
      __syncwarp();
      __threadfence_block();
      const MegaOp& dsc = s_desc[pcount & 1];
      ++pcount;
      const bool dual = (h.flags & kOpDual) != 0;
      const uint32_t Gn = (uint32_t)h.n_groups;
      const uint32_t my_chunks = end - start;
      const uint32_t n_sub_total = my_chunks * (dual ? 2u : 1u);
      QL_STAMP(0);

      // Expands one packed chunk (ring stage s) into two half-chunk A buffers of this group and
      // hands them to the issuer; returns the column's scale.
      auto unpack_subchunk = [&](uint32_t s, uint32_t ph) -> float {
        const uint8_t* st = ring + (size_t)s * STAGE;
        QL_CYC_BEGIN();
        st_mbar_wait(&full[s], ph, wc, 5);
        QL_CYC_END(0);
        QL_CYC_ADD(6, 1);
        const float sc = __uint_as_float((uint32_t)reinterpret_cast<const uint16_t*>(st + 64 * G)[n] << 16);
        const uint32_t z = (reinterpret_cast<const uint32_t*>(st + 64 * G + 256)[n >> 3] >> (4 * (n & 7))) & 0xFu;
        const uint32_t zb = 0x43004300u | z | (z << 16);
        const uint4* wst = reinterpret_cast<const uint4*>(st);
#pragma unroll
        for (int hh = 0; hh < 2; ++hh, ++hs) {
          const uint32_t slot = hs % AH;
          if (hs >= AH) {
            st_mbar_wait(&a_empty[w * AH + slot], ((hs / AH) - 1) & 1, wc, 6);
            tc_fence_after_sync();
          }
          QL_CYC_END(1);
#pragma unroll
          for (int cc = 0; cc < NC / 2; ++cc) {
            uint32_t v[16];
            unpack_codes32(wst[(hh * (NC / 2) + cc) * kTileN + n], zb, v);
            tmem_st16(a_addr + slot * AHC + 16 * cc, v);
          }
          QL_CYC_END(2);
          tmem_wait_st();
          QL_CYC_END(3);
          tc_fence_before_sync();
          __syncwarp();
          if (lane == 0) {
            mbar_arrive(&a_full[w * AH + slot]);
            if (hh == 1) mbar_arrive(&empty[s]);
          }
        }
        return sc;
      };

      // -------- the group's first chunk of the operation is unpacked BEFORE its X exists (the A
      //          operand depends on weights only; the issuer holds the MMAs back) --------
      // this group's sub-chunks of the operation are e = w, w + 4, ...; (s_own, ph_own) is the ring
      // stage and phase of the next one
      uint32_t e_own = (uint32_t)w, s_own = stg + (uint32_t)w, ph_own = sph;
      if (s_own >= (uint32_t)NS) { s_own -= (uint32_t)NS; ph_own ^= 1; }
      auto advance_own = [&]() {
        e_own += NWG;
        s_own += NWG;
        if (s_own >= (uint32_t)NS) { s_own -= (uint32_t)NS; ph_own ^= 1; }
      };
      float pre_sc = 0.f;
      bool pre_done = false;                            // sub-chunk e_own is already unpacked
      if (e_own < n_sub_total && !(sp.ablate & 1)) {
        pre_sc = unpack_subchunk(s_own, ph_own);
        pre_done = true;
      }
      QL_STAMP(1);
      // -------- X duty (all 512 threads): wait for the previous operation, build the X operand --------
      if (!RING) build_x<G>(sp, dsc, j, xbuf, s_inv, s_dep, s_invrdy, x_full, wc, start, my_chunks, Gn);
      QL_STAMP(3);

      // -------- chunks of this operation --------
      uint32_t pos = start, e_seg_end = 0;              // sub-chunks of the operation up to the end of the current segment
      int am_tiles = 0;                                  // tiles of this operation the CTA has finished (arg-max bookkeeping)
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
        e_seg_end += nch * (dual ? 2u : 1u);
        while (e_own < e_seg_end) {
          float sc;
          if (sp.ablate & 1) {
            sc = 0.f;
          } else if (pre_done) {
            sc = pre_sc;                                 // unpacked ahead (before X duty, or before the previous tile end)
            pre_done = false;
          } else {
            if (n_pend == 2) { drain(kloc - 2, s_p2); n_pend = 1; }
            sc = unpack_subchunk(s_own, ph_own);
          }
          if (sp.ablate & 1) n_pend = 0;
          s_p2 = s_p1;
          s_p1 = sc;
          ++n_pend;
          ++kloc;
          advance_own();
        }
        if (!(sp.ablate & 1)) {
          if (n_pend == 2) drain(kloc - 2, s_p2);
          // a segment that is not the piece's last: the group's first chunk of the NEXT segment is
          // unpacked before this segment's tile end, so that its MMAs run while the rows are finished
          // (the tile of a segment in the middle of a piece is a whole one, or one whose owner gathers
          // the partial rows at the end of ITS piece: nobody waits for it yet) - and before the last
          // chunk of this segment is read back: its MMAs were handed over a moment ago, and the
          // accumulator buffer the new chunk will use is the one just drained
          if (e_own < n_sub_total && !pre_done) {
            pre_sc = unpack_subchunk(s_own, ph_own);
            pre_done = true;
          }
          if (n_pend >= 1) drain(kloc - 1, s_p1);
        }
        tc_fence_before_sync();
#ifdef QL_TIMELINE
        const long long te0_ = clock64();
#endif
        if (pos == start) QL_STAMP(4);
        if (pos + nch == end) QL_STAMP(8);

        // ---- end of a tile segment: the four groups' accumulators meet in shared memory.  From the
        //      second barrier on, every warp works alone: warp r owns row r of the tile (lane l its
        //      columns 4l..4l+3), exchanges row r of split tiles, stores it and publishes it. ----
        if (!(sp.ablate & 32)) {
        named_bar_sync(1, kUnpackThreads);               // every warp is done reading the previous segment's sums
#pragma unroll
        for (int m = 0; m < MP; ++m) red[(w * MP + m) * kTileN + n] = acc[m];
        named_bar_sync(1, kUnpackThreads);
        }
        if (pos == start) QL_STAMP(5);
        if (pos + nch == end) QL_STAMP(9);
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
        bool finish = (g0 == 0);                         // my run contains the tile's first chunk
        if ((sp.ablate & 8) && !whole && !finish) { pos += nch; continue; }
        pos += nch;
        const int nmat = dual ? 2 : 1;
        // partial rows of split tiles: [set j & 1][CTA][matrix][row][column]
        float* set_parts = sp.ws.parts + (size_t)(j & 1) * kSetCtas * kSlotWords;
        const size_t row_off = (size_t)rw * kTileN + 4 * lane;

        if (!whole && !finish) {
          // ---- contributor: row r of its partial tile; nothing else to do.  (A run that does not
          //      begin its tile meets it in its first segment, so one slot per CTA is enough.) ----
          for (int mt = 0; mt < nmat; ++mt) {
            const float* f = mt ? f1 : f0;
            st_part(set_parts + (size_t)cta * kSlotWords + (size_t)mt * MP * kTileN + row_off, f[0], f[1], f[2], f[3]);
          }
          if (pos - nch == start) QL_STAMP(6);
          if (pos == end) QL_STAMP(14);
          continue;
        }
        if (!whole && !(sp.ablate & 8)) {
          // ---- owner of a split tile: its own partial stays in registers; the others' rows are
          //      polled until no word is empty any more, added in CTA order, and their slots emptied ----
          const uint32_t last = h.last;                  // (a split tile that a piece begins is the piece's last tile)
          if (pos == end) QL_STAMP(10);
          // items = (contributor, matrix) in CTA order, the two matrices of a dual operation side by
          // side: in chains eight items are in flight together (one round of loads covers every tile of
          // the verify step: at most 7 contributors of a plain linear, 2 or 3 of a gate/up pair)
          constexpr int GB = PAIRED ? 8 : 4;             // (the variants for streams have 80 registers and few contributors)
          const uint32_t items = (last - cta) * (uint32_t)nmat;
          for (uint32_t k0 = 0; k0 < items; k0 += GB) {
            uint32_t u[GB][4];
            uint64_t t0 = 0;
            uint32_t spins = 0;
            for (;;) {
#pragma unroll
              for (int q = 0; q < GB; ++q) {
                const uint32_t k = min(k0 + q, items - 1);
                const uint32_t i = cta + 1 + (dual ? (k >> 1) : k);
                const uint32_t mt = dual ? (k & 1u) : 0u;
                ld_part(set_parts + (size_t)i * kSlotWords + (size_t)mt * MP * kTileN + row_off, u[q]);
              }
              bool ok = true;
#pragma unroll
              for (int q = 0; q < GB; ++q)
#pragma unroll
                for (int e = 0; e < 4; ++e) ok = ok && (u[q][e] != kPartEmpty);
              if (ok) break;
              if (spins == 0) {
                if (*wc.s_abort) break;
                t0 = globaltimer_ns();
              }
              if ((++spins & 15u) == 0) {
                if (*wc.s_abort) break;
                if (globaltimer_ns() - t0 > wc.budget) { wait_fail(wc, 10); break; }
              }
            }
#pragma unroll
            for (int q = 0; q < GB; ++q) {
              if (k0 + q >= items) continue;
              const float a0 = __uint_as_float(u[q][0]), a1 = __uint_as_float(u[q][1]);
              const float a2 = __uint_as_float(u[q][2]), a3 = __uint_as_float(u[q][3]);
              if (dual && (q & 1)) { f1[0] += a0; f1[1] += a1; f1[2] += a2; f1[3] += a3; }   // (k0 is even: item parity = q parity)
              else { f0[0] += a0; f0[1] += a1; f0[2] += a2; f0[3] += a3; }
              const uint32_t k = k0 + q;
              const uint32_t i = cta + 1 + (dual ? (k >> 1) : k);
              const uint32_t mt = dual ? (k & 1u) : 0u;
              clear_part(set_parts + (size_t)i * kSlotWords + (size_t)mt * MP * kTileN + row_off);
            }
          }
          __syncwarp();
        }

        if (pos == end) QL_STAMP(11);
        // ---- row epilogue: bf16 stores, sum of squares for the next operation, arg-max ----
        if (sp.ablate & 64) {
          __syncwarp();
          if (lane == 0) red_relaxed_add(&sp.ws.op_done[((size_t)j * 16 + rw) * kOpDoneStride], 1);
        } else {
          uint16_t* out0 = dsc.out0;
          int32_t* argmax_out = dsc.argmax_out;
          const int emit_ssq = dsc.emit_ssq;
          const int ld_out = dsc.ld_out;
          const int col = (int)T * kTileN + 4 * lane;
          const int op_rows = dsc.rows;
          const bool live = rw < op_rows;
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
            if (live) *reinterpret_cast<uint2*>(dsc.out1 + (size_t)rw * ld_out + col) = y1;
            if (emit_ssq == 2) {
              a[0] = st_silu(a[0]) * bf16lo_to_f32(y1.x); a[1] = st_silu(a[1]) * bf16hi_to_f32(y1.x);
              a[2] = st_silu(a[2]) * bf16lo_to_f32(y1.y); a[3] = st_silu(a[3]) * bf16hi_to_f32(y1.y);
              // the fp32 product [M][N], for the operation that consumes it
              if (live) __stcg(reinterpret_cast<float4*>(sp.ws.act + (size_t)rw * dsc.N + col), make_float4(a[0], a[1], a[2], a[3]));
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
            // Every finished tile leaves the row's candidate; the row's counter is raised once per
            // CTA, by the number of tiles it finished, at its last tile of the operation (the last
            // segment of a run always finishes its tile: atomics on one line from every tile of a
            // 150,000-column head cost more than the tiles).  The warp whose addition completes
            // the count reduces the candidates of all tiles.
            int is_last = 0;
            ++am_tiles;
            if (lane == 0) {
              __stcg(&sp.ws.cand[(size_t)rw * h.n_tiles + T], make_float2(bv, __int_as_float(bi)));   // [row][tile]: the final reduction reads a row contiguously
              if (pos == end) {
                // release with a fence of its own, then a RELAXED atomic: 148 acquire-release atomics on one
                // address are served one after the other at ~0.1 us each
                int old;
                fence_gpu();
                asm volatile("atom.add.relaxed.gpu.global.s32 %0, [%1], %2;" : "=r"(old) : "l"(amax_cnt + rw * 32), "r"(am_tiles) : "memory");
                is_last = (old + am_tiles == h.n_tiles);
                if (is_last) {
                  fence_gpu();                           // acquire: the other CTAs' candidates
                  amax_cnt[rw * 32] = 0;
                }
              }
            }
            is_last = __shfl_sync(0xffffffffu, is_last, 0);
            if (is_last && live) {
              bv = -INFINITY;
              bi = 0x7fffffff;
              for (int t0 = lane; t0 < h.n_tiles; t0 += 32 * 8) {      // eight candidates per lane in flight: a round trip per 256 tiles
                float2 c[8];
#pragma unroll
                for (int q = 0; q < 8; ++q)
                  c[q] = (t0 + 32 * q < h.n_tiles) ? __ldcg(&sp.ws.cand[(size_t)rw * h.n_tiles + t0 + 32 * q]) : make_float2(-INFINITY, __int_as_float(0x7fffffff));
#pragma unroll
                for (int q = 0; q < 8; ++q) st_amax_merge(bv, bi, c[q].x, __float_as_int(c[q].y));
              }
#pragma unroll
              for (int off = 16; off >= 1; off >>= 1) {
                const float ov = __shfl_xor_sync(0xffffffffu, bv, off);
                const int oi = __shfl_xor_sync(0xffffffffu, bi, off);
                st_amax_merge(bv, bi, ov, oi);
              }
              if (lane == 0) argmax_out[rw] = bi;
              // Verification tail: the warp that settles the LAST row's greedy token compares the
              // block with the drafted tokens - length of the agreeing prefix, and the target's
              // own token at the first disagreement.
              if (dsc.draft_ids != nullptr) {
                int rows_done = 0;
                if (lane == 0) {
                  fence_gpu();                           // release: this row's token
                  asm volatile("atom.add.relaxed.gpu.global.s32 %0, [%1], 1;" : "=r"(rows_done) : "l"(amax_cnt + 16 * 32) : "memory");
                  if (rows_done == op_rows - 1) fence_gpu();   // acquire: the other rows' tokens
                }
                rows_done = __shfl_sync(0xffffffffu, rows_done, 0);
                if (rows_done == op_rows - 1) {
                  const int tok = lane < op_rows ? (lane == rw ? bi : __ldcg(&argmax_out[lane])) : -1;
                  const int drf = lane < op_rows ? __ldg(&dsc.draft_ids[lane]) : -2;
                  const unsigned agree = __ballot_sync(0xffffffffu, lane < op_rows && tok == drf);
                  const int a = __ffs(~agree) - 1;            // first row that disagrees (rows >= M never agree)
                  const int bonus = __shfl_sync(0xffffffffu, tok, a < op_rows ? a : 0);
                  if (lane == 0) {
                    dsc.accept_out[0] = a;
                    dsc.accept_out[1] = a < op_rows ? bonus : -1;
                    amax_cnt[16 * 32] = 0;
                  }
                }
              }
            }
          }
          if (pos == end) QL_STAMP(12);
          // the row of the tile is complete: publish it (one fence after the warp's stores)
          __syncwarp();
          if (lane == 0 && !(h.flags & (kOpNoRelease | kOpLazy))) {
            if (!(sp.ablate & 16)) fence_gpu();
            red_relaxed_add(&sp.ws.op_done[((size_t)j * 16 + rw) * kOpDoneStride], 1);
          }
          if (pos - nch == start) QL_STAMP(6);
          if (pos == end) QL_STAMP(14);
        }
#ifdef QL_TIMELINE
        cyc_te_ += clock64() - te0_;
#endif
      }
      {
        const uint32_t t = stg + n_sub_total;             // ring position after this operation's sub-chunks
        sph ^= (t / (uint32_t)NS) & 1u;
        stg = t % (uint32_t)NS;
      }
      __syncwarp();
      if (lane == 0) s_prog[warp] = pcount;
    }
    QL_CYC_FLUSH();
  }

  // every tensor-memory access of the CTA is complete past this barrier
  tc_fence_before_sync();
  __syncthreads();
  if (warp == kWarpIssuer0) {
    tc_fence_after_sync();
    tmem_dealloc(tmem, TMEM_COLS);
  }
  if (warp == 0) {
    // the last CTA to leave restores the counters for the next launch
    int old = 0;
    if (lane == 0) {
      __threadfence();
      old = atomicAdd(sp.ws.exit_cnt, 1);
    }
    old = __shfl_sync(0xffffffffu, old, 0);
    if (old == (int)gridDim.x - 1) {
      for (int i = lane; i < sp.n_ops * 16; i += 32) sp.ws.op_done[(size_t)i * kOpDoneStride] = 0;
      if (lane <= 16) sp.ws.tile_cnt[kMaxTiles + kStackFlagWords + lane * 32] = 0;   // per-row arg-max counters, verification-tail row counter
      if (lane == 0) { *sp.ws.amax_done = 0; *sp.ws.exit_cnt = 0; }
    }
  }
}

// ---- host side ---------------------------------------------------------------------------------

// Shared-memory plan for a list of operations with common M <= 16 and g whose split fields are
// set; ok = false if some operation's X does not fit beside a ring of at least 6 stages.
struct StackPlan {
  int ncta, n_x, n_stages, x_ring;
  size_t smem;
  bool ok;
};

int stack_ncta(int sms) { return sms < kMaxCtas / 2 ? sms : kMaxCtas / 2; }   // one 32 KB partial slot per CTA

// x_ring: the operations are independent plain linears laid end to end whose X does not fit per operation;
// it comes through a ring of kXRingSlots slots filled by the loader warp, whatever K is.
StackPlan stack_plan(const MegaOp* ops, int n_ops, int g, int sms, bool one_stream) {
  StackPlan r = {};
  const int ncta = stack_ncta(sms);
  uint32_t n_x = 1;
  for (int j = 0; j < n_ops && !one_stream; ++j) {
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
  if (one_stream) n_x = kXRingSlots;
  const uint32_t stage = align128(chunk_bytes(g)), xslot = st_xslot_bytes(g);
  const uint32_t fixed = st_fixed_smem() + 32u * (uint32_t)n_ops;   // + the head table
  if (fixed + n_x * xslot + 6 * stage > kStSmemBudget) return r;
  int ns = (int)((kStSmemBudget - fixed - n_x * xslot) / stage);
  if (ns > kStMaxStages) ns = kStMaxStages;
  r.ncta = ncta; r.n_x = (int)n_x; r.n_stages = ns; r.x_ring = one_stream ? kXRingSlots : 0;
  r.smem = (size_t)ns * stage + (size_t)n_x * xslot + fixed;
  r.ok = true;
  return r;
}

template <int G, bool RING, bool PAIRED>
static cudaError_t stack_launch_g(const StackParams& sp, size_t smem, cudaStream_t stream) {
  // all CTAs wait on one another's progress: they must be co-resident (the cooperative launch checks it)
  cudaError_t e = cudaFuncSetAttribute(qstack_tc5_kernel<G, RING, PAIRED>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kStSmemBudget);
  if (e != cudaSuccess) return e;
  void* args[] = {const_cast<StackParams*>(&sp)};
  return cudaLaunchCooperativeKernel(reinterpret_cast<void*>(qstack_tc5_kernel<G, RING, PAIRED>), dim3(sp.ncta),
                                     dim3(st_threads(RING, PAIRED)), args, smem, stream);
}

// Three variants: chains (paired issuers), one stream with X resident per operation, one stream with the X ring.
cudaError_t launch_stack_tc5(const StackParams& sp, int g, size_t smem, cudaStream_t stream) {
  if (sp.x_ring > 0) return g == 128 ? stack_launch_g<128, true, false>(sp, smem, stream) : stack_launch_g<64, true, false>(sp, smem, stream);
  if (sp.one_stream) return g == 128 ? stack_launch_g<128, false, false>(sp, smem, stream) : stack_launch_g<64, false, false>(sp, smem, stream);
  return g == 128 ? stack_launch_g<128, false, true>(sp, smem, stream) : stack_launch_g<64, false, true>(sp, smem, stream);
}

}  // namespace ql
