// Kernel parameter block of one quantised linear (host fills it, kernels read it).
#pragma once
#include <stdint.h>

#include "ql_device.cuh"

namespace ql {

struct LinearParams {
  const uint8_t* packed;   // packed weights, chunk (T, G) at (T*n_groups + G) * chunk_bytes
  const uint16_t* X;       // bf16 [M, ldx]
  uint16_t* Y;             // bf16 [M, ldy] or nullptr
  int32_t* argmax_out;     // [M] or nullptr
  int M, K, N, g;
  int ldx, ldy;
  int n_tiles;             // N / 128
  int n_groups;            // K / g
  uint32_t total_chunks;   // n_tiles * n_groups
  int ncta;                // CTAs launched; CTA i owns chunks [i*total/ncta, (i+1)*total/ncta)
  int m_pad;               // M rounded up to 16
  int n_stages;            // depth of the shared-memory ring
  int n_x;                 // X slots (groups) in shared memory per CTA
  int x_phase;             // 0: X resident; P > 0: X of the next P chunks reloaded every P chunks
  uint32_t stage_bytes;    // bytes of one ring stage (weights chunk + X slice)
  int ablate;              // timing experiments (1: chunks are received but not computed)
  Workspace ws;
};

// One fused operation of the stack kernel: a linear (or two linears that share their input, e.g.
// gate and up), with the element-wise glue in front of it folded into how it loads X.
//
// Work split.  Operations are grouped into runs; the chunks of a run's operations, laid end to end,
// are shared out in contiguous pieces among the first nc CTAs.  A run is either one operation
// (chained operations: every CTA takes its share of every operation) or a list of independent
// plain linears (each CTA then works through one long piece that touches one or two of them).
// The first 32 bytes hold what every role reads at every operation.
constexpr int kOpDual = 1;        // two matrices (packed0, packed1) share X
constexpr int kOpWait = 2;        // X may be read only after operation j-1 has finished every tile
constexpr int kOpLazy = 16;       // nothing in the launch waits for this operation's tiles (independent linears of one stream, the
                                  // last operation of a chain): they need not be published
constexpr int kOpNoRelease = 4;   // test hook: finished tiles are not published (the next operation's wait runs out)
struct MegaOp {
  uint32_t nc, cq, cr;     // CTA i owns run positions [i*cq + i*cr/nc, (i+1)*cq + (i+1)*cr/nc), i < nc; or, with
                           // cr = kSplitAligned | n_tiles and cq = the owner's extra chunks, the aligned split
  uint32_t cat_base;       // run position of this operation's chunk 0
  uint32_t total_chunks;   // n_tiles * n_groups (per matrix)
  int n_groups, n_tiles;
  int flags;               // kOp* bits
  const uint8_t* packed0;  // packed weights
  const uint8_t* packed1;  // second matrix of a dual operation (same K, N, g), else nullptr
  const uint16_t* in0;     // X source, bf16 [M, ld_in]
  const uint16_t* in1;     // second X source (silu(in0) * in1), else nullptr
  uint16_t* out0;          // Y of matrix 0, bf16 [M, ld_out] (may be nullptr when only arg-max is wanted)
  uint16_t* out1;          // Y of matrix 1 (dual)
  uint16_t* xout;          // where the normalised X is written for the record (prologue != 0), else nullptr
  int32_t* argmax_out;     // [M] or nullptr
  int K, N, ld_in, ld_out;
  int ld_xout;
  int prologue;            // 0: X = in0;  1: X = unit_rms(in0);  2: X = unit_rms(silu(in0) * in1)
  int src_tiles;           // column tiles of the producer that make up a normalised row (prologue != 0)
  int emit_ssq;            // 0: none; 1: per-tile row sums of bf16(Y)^2; 2: of (silu(bf16 Y0) * bf16 Y1)^2
  const int32_t* draft_ids;  // [M] drafted tokens the greedy tokens are compared with (verification tail), else nullptr
  int32_t* accept_out;       // [2] accepted-prefix length, bonus token
  int rows;                  // rows of X and Y this operation works on (1..16)
  int pad0_;
  uint64_t pad_;
};
static_assert(sizeof(MegaOp) == kOpDescBytes, "operation descriptor layout");

struct StackParams {
  const MegaOp* ops;       // device copy of the descriptors (in the workspace)
  int n_ops;
  int M;                   // (host bookkeeping; the kernel takes the row count of every operation from its descriptor)
  int ncta;
  int n_stages;            // ring depth
  int n_x;                 // X slots (groups) in shared memory
  int x_ring;              // 0: X of an operation is built once, by the unpack threads; P > 0 (one stream of independent
                           // linears): the X slots are a ring of P chunks filled by a loader warp, chunk by chunk
  int one_stream;          // the operations are independent plain linears laid end to end (selects the kernel variant)
  int ablate;              // timing experiments only (see the stack kernel); 0 in production
  uint32_t epoch;          // launch number (kept for diagnostics; nothing in the kernel depends on it)
  uint64_t wait_ns;        // budget of every bounded wait
  uint64_t* timeline;      // builds with -DQL_TIMELINE only: [ncta][n_ops][8] globaltimer stamps, else nullptr
  Workspace ws;
};

// Run position of the first chunk of CTA i (32-bit arithmetic only; i*cr < 2^18).
__host__ __device__ inline uint32_t run_first_chunk(uint32_t nc, uint32_t cq, uint32_t cr, uint32_t i) {
  return i * cq + (i * cr) / nc;
}
// Aligned split of a chained operation with at most nc / 2 tiles (cr = kSplitAligned | n_tiles, cq = the
// owner's extra chunks e): tile T belongs to the CTAs [T nc / n_tiles, (T + 1) nc / n_tiles) alone, so no CTA
// works on two tiles and nobody ends a tile segment in the middle of its piece.  The first CTA of a tile
// (its owner: it adds the others' partial rows and finishes the tile) takes e chunks more than an even
// share of the rest: that is the time the others' partial rows need to reach it.
constexpr uint32_t kSplitAligned = 0x80000000u;
__host__ __device__ inline void aligned_tile_ctas(uint32_t nc, uint32_t nt, uint32_t T, uint32_t& c0, uint32_t& c1) {
  c0 = (T * nc) / nt;
  c1 = ((T + 1) * nc) / nt;
}
__host__ __device__ inline void aligned_range(uint32_t nc, uint32_t extra, uint32_t nt, uint32_t total, uint32_t i,
                                              uint32_t& lo, uint32_t& hi) {
  const uint32_t Gn = total / nt;
  const uint32_t T = ((i + 1) * nt + nc - 1) / nc - 1;   // the largest T with T nc / nt <= i
  uint32_t c0, c1;
  aligned_tile_ctas(nc, nt, T, c0, c1);
  const uint32_t n = c1 - c0, r = i - c0, rest = Gn - extra;
  lo = T * Gn + (r == 0 ? 0u : extra + (r * rest) / n);
  hi = T * Gn + extra + ((r + 1) * rest) / n;
}
// Chunks [lo, hi) of operation `op` (per matrix) that CTA i owns; lo == hi if none.
__host__ __device__ inline void op_local_range(uint32_t nc, uint32_t cq, uint32_t cr, uint32_t cat_base, uint32_t total,
                                               uint32_t i, uint32_t& lo, uint32_t& hi) {
  lo = hi = 0;
  if (i >= nc) return;
  if (cr & kSplitAligned) { aligned_range(nc, cq, cr & ~kSplitAligned, total, i, lo, hi); return; }
  uint32_t a = run_first_chunk(nc, cq, cr, i), b = run_first_chunk(nc, cq, cr, i + 1);
  const uint32_t top = cat_base + total;
  if (a < cat_base) a = cat_base;
  if (b > top) b = top;
  if (a < b) { lo = a - cat_base; hi = b - cat_base; }
}
// The CTA that owns run position p: the largest i with run_first_chunk(i) <= p (float guess, exact correction).
__host__ __device__ inline uint32_t run_chunk_owner(uint32_t nc, uint32_t cq, uint32_t cr, uint32_t p) {
  const float total = (float)(nc * cq + cr);
  uint32_t i = (uint32_t)(((float)p + 0.5f) * ((float)nc / total));
  if (i >= nc) i = nc - 1;
  while (i > 0 && run_first_chunk(nc, cq, cr, i) > p) --i;
  while (i + 1 < nc && run_first_chunk(nc, cq, cr, i + 1) <= p) ++i;
  return i;
}
// The last CTA that works on tile T of an operation with n_groups chunks per tile.
__host__ __device__ inline uint32_t op_last_cta(uint32_t nc, uint32_t cq, uint32_t cr, uint32_t cat_base, uint32_t n_groups, uint32_t T) {
  if (cr & kSplitAligned) {
    uint32_t c0, c1;
    aligned_tile_ctas(nc, cr & ~kSplitAligned, T, c0, c1);
    return c1 - 1;
  }
  return run_chunk_owner(nc, cq, cr, cat_base + T * n_groups + n_groups - 1);
}
// Host: split a run of `run_total` chunks among ncta CTAs.
inline void run_split(uint32_t run_total, uint32_t ncta, uint32_t& nc, uint32_t& cq, uint32_t& cr) {
  nc = ncta < run_total ? ncta : run_total;
  cq = run_total / nc;
  cr = run_total % nc;
}

// First chunk of CTA i (64-bit product: total_chunks * ncta can exceed 2^32).
__host__ __device__ inline uint32_t cta_first_chunk(uint32_t i, uint32_t total, uint32_t ncta) {
  return (uint32_t)(((uint64_t)i * total) / ncta);
}
// The CTA that owns chunk c: the largest i with cta_first_chunk(i) <= c.
__host__ __device__ inline uint32_t chunk_owner(uint32_t c, uint32_t total, uint32_t ncta) {
  return (uint32_t)((((uint64_t)c + 1) * ncta + total - 1) / total) - 1;
}

// Sliding-window attention of a drafted block (qattn_swa.cu).
struct AttnParams {
  const uint16_t* Q;
  const uint16_t* K;
  const uint16_t* V;
  uint16_t* out;
  float* part;            // [Hkv][n_pieces][G][16][kAttnPartStride]
  int* counters;          // [Hkv], zero between calls
  int n_q, T, Hq, Hkv, G;
  int p0, window;
  int ld_q, ld_kv, ld_out;   // elements between consecutive queries / tokens / output rows
  int key_lo, key_hi;        // union of the visible keys of all queries
  int sub_per_piece, n_pieces;
  float scale_log2;          // log2(e) / sqrt(d)
};

}  // namespace ql
