// Device-side helpers shared by the qlinear kernels: packed-layout constants, mbarrier /
// bulk-copy / cp.async wrappers with bounded waits, the bf16 tensor-core MMA, nibble unpacking.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace ql {

// ---- packed layout (see the header of qpack_w4_g128) ----------------------------------------
constexpr int kTileN = 128;                       // columns per chunk
__host__ __device__ constexpr uint32_t chunk_bytes(int g) { return 64u * g + 320u; }
__host__ __device__ constexpr uint32_t chunk_w_bytes(int g) { return 64u * g; }
__host__ __device__ constexpr uint32_t align128(uint32_t x) { return (x + 127u) & ~127u; }

// ---- workspace layout -----------------------------------------------------------------------
// [0, 256)        control header: word 0 status, word 1 finished-tile counter (arg-max),
//                 word 2 finished-CTA counter of the stack kernel
// then            per-tile arrival counters (split-K) of the single-linear kernels [kMaxTiles], a reserved
//                 block [2][160][16], the stack kernel's per-row arg-max counters and its verification-tail
//                 counter on lines of their own                    [kFlagWords in all]
// then            per-operation, per-row finished-tile counters of the stack kernel, one 128-byte line each
//                                                                [kMaxOps][16][32]
// -- everything above is zero between calls (ql_workspace_init zeroes it once, kernels restore it) --
// then            operation descriptors of the stack kernel      [kMaxOps * kOpDescBytes]
// then            partial tiles of the stack kernel (self-signalling values)   [kWsPartBytes]
// then            row sums of squares per tile, two buffers      [2][tiles][16] fp32
// then            fp32 product silu(gate)*up of a dual operation, dense [16][N]   [16][tiles*128]
// then            arg-max candidates                             [m_pad][tiles] (value, index)
// then            split-K partial tiles  [kMaxCtas][2 segments][2 matrices][m_pad*128] fp32
constexpr int kMaxCtas = 320;                     // up to two CTAs per SM
constexpr int kMaxTiles = 4096;                   // N <= 128 * 4096
constexpr int kStackFlagWords = 2 * 160 * 16;      // reserved (row flags of an earlier exchange scheme; the words stay zero)
constexpr int kFlagWords = kMaxTiles + kStackFlagWords + 1024;   // tile counters [kMaxTiles], the reserved block, then the stack kernel's 16 per-row arg-max counters and its verification-tail counter on lines of their own
constexpr int kMaxOps = 256;                      // fused operations per stack-kernel launch
constexpr int kOpDoneStride = 32;                 // ints between the counters of two rows (one line each: they are polled)
constexpr int kOpDescBytes = 160;
constexpr int kWsHeaderBytes = 256;
constexpr size_t kWsControlBytes = kWsHeaderBytes + (size_t)kFlagWords * 4 + (size_t)kMaxOps * 16 * kOpDoneStride * 4;
constexpr size_t kWsDescBytes = (size_t)kMaxOps * kOpDescBytes;
// Partial tiles of the stack kernel, fp32 [2 sets][160 CTAs][2 matrices][16 rows][128].  A word is either
// kPartEmpty (ql_workspace_init fills the region with it, and the CTA that has added a partial row puts
// it back) or a value a contributor stored: the value is its own signal, no flag and no fence travel
// with it.  The region is written by that kernel only and sits at a fixed offset.
constexpr uint32_t kPartEmpty = 0xFFFFFFFFu;         // a NaN no arithmetic produces (stores replace it by the canonical NaN)
constexpr size_t kWsPartBytes = (size_t)kMaxCtas * 2 * 16 * 128 * 4;

struct Workspace {
  int* status;
  int* amax_done;
  int* exit_cnt;
  int* tile_cnt;
  int* op_done;
  uint8_t* desc;
  float* ssq;        // [2][n_tiles][16]
  float* act;        // [16][N] of the dual operation that wrote it, dense (capacity 16 * n_tiles * 128)
  float2* cand;      // .x = value, .y = index bits
  float* slots;
  float* parts;      // partial tiles of the stack kernel (kPartEmpty where nothing is waiting)
  int n_tiles;       // tile capacity the regions were carved for
};

// m rounded up to the row counts the kernels are built for
__host__ __device__ inline int pad_rows(int m) { return m <= 16 ? 16 : (m <= 32 ? 32 : 64); }
__host__ __device__ inline size_t ws_ssq_bytes(int n_tiles) { return (size_t)2 * n_tiles * 16 * 4; }
__host__ __device__ inline size_t ws_cand_bytes(int n_tiles, int m_pad) { return ((size_t)n_tiles * m_pad * 8 + 255) & ~(size_t)255; }
__host__ __device__ inline size_t ws_slot_floats(int m_pad) { return (size_t)2 * m_pad * kTileN; }   // two matrices
__host__ __device__ inline size_t ws_act_bytes(int n_tiles) { return (size_t)16 * n_tiles * kTileN * 4; }
__host__ __device__ inline size_t ws_total_bytes(int n_tiles, int m_pad) {
  return kWsControlBytes + kWsDescBytes + kWsPartBytes + ws_ssq_bytes(n_tiles) + ws_act_bytes(n_tiles) + ws_cand_bytes(n_tiles, m_pad) +
         (size_t)kMaxCtas * 2 * ws_slot_floats(m_pad) * 4;
}
// Carves the regions for a tile capacity and row padding.  Within one workspace every call must
// use the same (n_tiles, m_pad) carve only for regions it shares with concurrently running
// kernels; kernels of one stream run one after the other, so each call may carve for itself.
__host__ __device__ inline Workspace ws_carve(void* base, int n_tiles, int m_pad) {
  char* p = (char*)base;
  Workspace w;
  w.status = (int*)p;
  w.amax_done = (int*)p + 1;
  w.exit_cnt = (int*)p + 2;
  w.tile_cnt = (int*)(p + kWsHeaderBytes);
  w.op_done = w.tile_cnt + kFlagWords;
  w.desc = (uint8_t*)(p + kWsControlBytes);
  w.parts = (float*)(p + kWsControlBytes + kWsDescBytes);
  p += kWsControlBytes + kWsDescBytes + kWsPartBytes;
  w.ssq = (float*)p;
  p += ws_ssq_bytes(n_tiles);
  w.act = (float*)p;
  p += ws_act_bytes(n_tiles);
  w.cand = (float2*)p;
  p += ws_cand_bytes(n_tiles, m_pad);
  w.slots = (float*)p;
  w.n_tiles = n_tiles;
  return w;
}

#ifdef __CUDACC__
// ---- small PTX wrappers ---------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ uint64_t globaltimer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}

// The same with a suspend-time hint: a thread that finds the phase incomplete may be suspended by the
// hardware for up to `hint_ns` (it is resumed when the phase completes), instead of spinning on
// the instruction and taking issue slots from the warps that work.
__device__ __forceinline__ bool mbar_try_wait_hint(uint64_t* bar, uint32_t parity, uint32_t hint_ns) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity), "r"(hint_ns)
      : "memory");
  return ok != 0;
}

// Bounded wait on an mbarrier phase.  Gives up after kWaitBudgetNs: records QL_ERR_DEVICE_TIMEOUT
// in the status word, raises the CTA-wide abort flag and returns, so that every later wait of
// the CTA falls through at once and the kernel runs to its end (with garbage results, which the
// status word reports) instead of hanging.
constexpr uint64_t kWaitBudgetNs = 2000000000ull;   // 2 s
constexpr int kStatusTimeout = 7;                   // QL_ERR_DEVICE_TIMEOUT

// `site` identifies the wait in the timeout report: status word = 7 | site << 8 | blockIdx.x << 16.
__device__ __forceinline__ void mbar_wait(uint64_t* bar, uint32_t parity, volatile int* s_abort, int* status,
                                          int site = 0) {
  if (mbar_try_wait(bar, parity)) return;
  if (*s_abort) return;
  const uint64_t t0 = globaltimer_ns();
  uint32_t spins = 0;
  while (!mbar_try_wait(bar, parity)) {
    if ((++spins & 255u) == 0) {
      if (*s_abort) return;
      if (globaltimer_ns() - t0 > kWaitBudgetNs) {
        *s_abort = 1;
        atomicCAS(status, 0, kStatusTimeout | (site << 8) | ((int)blockIdx.x << 16));
        return;
      }
    }
  }
}

// Contiguous global -> shared bulk copy (TMA engine, no tensor map), completion on an mbarrier.
// dst, src 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_g2s(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   smem_u32(dst_smem)),
               "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void bulk_g2s_hint(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar,
                                              uint64_t policy) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
          smem_u32(dst_smem)),
      "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar)), "l"(policy)
      : "memory");
}

// 16-byte asynchronous copy global -> shared; src_bytes = 0 writes zeros instead.
__device__ __forceinline__ void cp_async16(void* dst_smem, const void* src_gmem, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst_smem)), "l"(src_gmem), "r"(src_bytes)
               : "memory");
}
// Makes `bar` receive one (pre-counted) arrival once all cp.async of this thread have landed.
__device__ __forceinline__ void cp_async_arrive_noinc(uint64_t* bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}

__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Two int4 codes (bits [3:0] of each half-word of `v`, already masked) -> bf16x2 of (code - z),
// exact: 0x4300 | code is the bf16 128 + code, and (128 + code) - (128 + z) has at most 5 bits.
__device__ __forceinline__ uint32_t codes_minus_zero(uint32_t masked, uint32_t zbias) {
  uint32_t e = masked | 0x43004300u;
  __nv_bfloat162 r = __hsub2(*reinterpret_cast<__nv_bfloat162*>(&e), *reinterpret_cast<__nv_bfloat162*>(&zbias));
  return *reinterpret_cast<uint32_t*>(&r);
}

// One 32-bit word of the packed layout (8 codes: extraction s takes the nibbles at bits 4s and
// 16 + 4s) -> four bf16x2 registers of the exact integers code - z.  Written in PTX so that the
// instruction sequence is the intended one (3 shifts, 4 and-or LOP3s, 4 packed subtractions); the
// compiler's own selection for the C++ form was 15 % slower in the mma.sync kernel's chunk loop.
__device__ __forceinline__ void unpack_word(uint32_t w, uint32_t zbias, uint32_t& b0, uint32_t& b1, uint32_t& b2, uint32_t& b3) {
  asm("{\n\t"
      ".reg .b32 w1, w2, w3;\n\t"
      "shr.u32 w1, %4, 4;\n\t"
      "shr.u32 w2, %4, 8;\n\t"
      "shr.u32 w3, %4, 12;\n\t"
      "lop3.b32 %0, %4, 0x000f000f, 0x43004300, 0xea;\n\t"
      "lop3.b32 %1, w1, 0x000f000f, 0x43004300, 0xea;\n\t"
      "lop3.b32 %2, w2, 0x000f000f, 0x43004300, 0xea;\n\t"
      "lop3.b32 %3, w3, 0x000f000f, 0x43004300, 0xea;\n\t"
      "sub.bf16x2 %0, %0, %5;\n\t"
      "sub.bf16x2 %1, %1, %5;\n\t"
      "sub.bf16x2 %2, %2, %5;\n\t"
      "sub.bf16x2 %3, %3, %5;\n\t"
      "}"
      : "=&r"(b0), "=&r"(b1), "=&r"(b2), "=&r"(b3)
      : "r"(w), "r"(zbias));
}

// ---- tcgen05 (5th-generation tensor core, tensor memory) ----------------------------------------
// Tensor-memory addresses are (lane << 16) | column.  A warp may touch only lanes
// [32*(warp%4), 32*(warp%4)+32).
__device__ __forceinline__ void tmem_alloc(uint32_t* smem_result, uint32_t ncols) {   // one full warp
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(smem_result)), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t addr, uint32_t ncols) {         // the allocating warp
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(addr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// Arrives once on `bar` when every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// D(tmem, 128 x N fp32) (+)= A(tmem, 128 x 16 bf16) * B(smem descriptor, N x 16 bf16, K-major)
__device__ __forceinline__ void tc_mma_ts_f16(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                              uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}
// 16 consecutive 32-bit columns of this thread's lane: registers -> tensor memory, and back.
__device__ __forceinline__ void tmem_st16(uint32_t addr, const uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(addr),
      "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]),
      "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t addr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(addr)
      : "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
// Shared-memory operand descriptor, K-major, no swizzle: 8-row x 16-byte core matrices;
// lbo = bytes between core matrices adjacent in K, sbo = bytes between 8-row blocks.
__device__ __forceinline__ uint64_t tc_smem_desc_kmajor(uint32_t smem_addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((smem_addr >> 4) & 0x3FFFu) | ((uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32) | (1ull << 46);
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__host__ __device__ constexpr uint32_t tc_idesc_bf16_m128(uint32_t n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | ((128u >> 4) << 24);
}

// One 16-byte word group of the packed layout (32 codes of one column, rows 8j + 2s + {0,1} in
// word j, extraction s) -> 16 bf16x2 registers of the exact integers q - z, in row order: register
// 4j + s holds rows (8j + 2s, 8j + 2s + 1), the order of a K-major operand in tensor memory.
__device__ __forceinline__ void unpack_codes32(const uint4 w4, uint32_t zbias, uint32_t (&v)[16]) {
  const uint32_t ww[4] = {w4.x, w4.y, w4.z, w4.w};
#pragma unroll
  for (int j = 0; j < 4; ++j) unpack_word(ww[j], zbias, v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
}

__device__ __forceinline__ float bf16lo_to_f32(uint32_t pair) { return __uint_as_float(pair << 16); }
__device__ __forceinline__ float bf16hi_to_f32(uint32_t pair) { return __uint_as_float(pair & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16x2_rn(float lo, float hi) {
  __nv_bfloat162 r = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&r);
}
#endif  // __CUDACC__

}  // namespace ql
