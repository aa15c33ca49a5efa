// Host side of the C-ABI: argument checks, path selection, launches.  No allocation, no
// synchronisation except where the header says so.
#include <atomic>
#include <cstring>
#include <vector>

#include "../../include/qlinear_w4a16.h"
#include "ql_params.h"

namespace ql {
cudaError_t launch_qpack(const uint32_t*, const uint16_t*, const uint8_t*, int, int, int, uint8_t*, cudaStream_t);
cudaError_t launch_qrequant(const uint16_t*, const uint16_t*, const uint8_t*, int, int, int, uint8_t*, cudaStream_t);
cudaError_t launch_linear_mma(LinearParams, cudaStream_t);
size_t attn_plan(AttnParams&, int sms);
cudaError_t launch_attn_swa(const AttnParams&, cudaStream_t);
size_t plan_linear_mma(LinearParams&);
cudaError_t launch_linear_tc5(LinearParams, int sms, cudaStream_t, bool pdl);
bool tc5_supported(const LinearParams&, int sms);
struct StackPlan { int ncta, n_x, n_stages, x_ring; size_t smem; bool ok; };
int stack_ncta(int sms);
StackPlan stack_plan(const MegaOp* ops, int n_ops, int g, int sms, bool one_stream = false);
cudaError_t launch_stack_tc5(const StackParams& sp, int g, size_t smem, cudaStream_t stream);
cudaError_t launch_unit_rms(const uint16_t*, const uint16_t*, uint16_t*, int, int, int, int, bool, cudaStream_t);

static std::atomic<uint64_t> g_launches{0};
static std::atomic<uint32_t> g_epoch{0};                  // stack-kernel launches so far
static std::atomic<uint64_t> g_wait_ns{kWaitBudgetNs};    // budget of the stack kernel's bounded waits
// Bumped whenever operation descriptors are staged into any workspace, a workspace is re-initialised or a
// debug hook changes: a remembered plan is valid only while nothing of that happened since it was staged.
static std::atomic<uint64_t> g_desc_gen{1};
static std::atomic<int> g_no_release_op{-1};              // test hook: fused operation that does not publish its tiles
constexpr int kOwnerExtraChunks = 0;                      // aligned split: chunks the owner of a tile takes beyond an even share
static std::atomic<int> g_owner_extra{kOwnerExtraChunks}; // (measurement hook ql_debug_set_owner_extra; negative: even split everywhere)
static std::atomic<int> g_ablate{0};                      // timing experiments: phases of the stack kernel switched off
static std::atomic<uint64_t*> g_timeline{nullptr};        // device buffer for the in-kernel timeline (QL_TIMELINE builds)

void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

static bool shape_ok(int M, int K, int N, int g) {
  if (M < 1 || M > 64) return false;
  if (g != 64 && g != 128) return false;
  if (K <= 0 || N <= 0 || K % g != 0 || N % kTileN != 0) return false;
  if (N / kTileN > kMaxTiles) return false;
  if ((int64_t)(N / kTileN) * (K / g) > 0x7fffffffLL) return false;
  return true;
}
static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int num_sms() {
  static int cached[16] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return -1;
  if (dev < 16 && cached[dev] > 0) return cached[dev];
  int n = 0;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return -1;
  if (dev < 16) cached[dev] = n;
  return n;
}

// Pure argument validation of one linear (no device query, nothing launched).
static int validate_linear(const void* packed, const uint16_t* X, int ldx, const uint16_t* Y, int ldy,
                           const int32_t* argmax_out, int M, int K, int N, int g, const void* workspace,
                           size_t workspace_bytes) {
  if (packed == nullptr || X == nullptr || workspace == nullptr) return QL_ERR_NULL;
  if (Y == nullptr && argmax_out == nullptr) return QL_ERR_NULL;
  if (!shape_ok(M, K, N, g)) return QL_ERR_SHAPE;
  if (ldx < K || (Y != nullptr && ldy < N)) return QL_ERR_SHAPE;
  if (!aligned16(packed) || !aligned16(X) || !aligned16(workspace) || (Y != nullptr && !aligned16(Y))) return QL_ERR_ALIGN;
  if (ldx % 8 != 0 || (Y != nullptr && ldy % 8 != 0)) return QL_ERR_ALIGN;
  if (argmax_out != nullptr && (reinterpret_cast<uintptr_t>(argmax_out) & 3u)) return QL_ERR_ALIGN;
  if (workspace_bytes < ws_total_bytes(N / kTileN, pad_rows(M))) return QL_ERR_WORKSPACE;
  return QL_OK;
}

// Validates one linear and fills the path-independent parameters.
static int prepare_linear(LinearParams& p, const void* packed, const uint16_t* X, int ldx, uint16_t* Y, int ldy,
                          int32_t* argmax_out, int M, int K, int N, int g, void* workspace, size_t workspace_bytes) {
  const int st = validate_linear(packed, X, ldx, Y, ldy, argmax_out, M, K, N, g, workspace, workspace_bytes);
  if (st != QL_OK) return st;
  const int n_tiles = N / kTileN, m_pad = pad_rows(M);
  const int sms = num_sms();
  if (sms <= 0) return QL_ERR_CUDA;
  p.packed = static_cast<const uint8_t*>(packed);
  p.X = X; p.Y = Y; p.argmax_out = argmax_out;
  p.M = M; p.K = K; p.N = N; p.g = g; p.ldx = ldx; p.ldy = ldy;
  p.n_tiles = n_tiles; p.n_groups = K / g;
  p.total_chunks = (uint32_t)n_tiles * (uint32_t)(K / g);
  int ncta = sms < kMaxCtas ? sms : kMaxCtas;           // one CTA per SM; a path may choose otherwise
  if ((uint32_t)ncta > p.total_chunks) ncta = (int)p.total_chunks;
  p.ncta = ncta;
  p.m_pad = m_pad;
  p.n_stages = 0; p.stage_bytes = 0; p.n_x = 0; p.x_phase = 0;
  p.ablate = g_ablate.load(std::memory_order_relaxed);
  p.ws = ws_carve(workspace, n_tiles, m_pad);
  return QL_OK;
}

// Path choice for a linear launched on its own (measured with `bench.py --paths`, 24 cold weight
// sets, one launch per linear): up to 32 rows the warp-level mma.sync kernel is faster than the
// tcgen05 kernel (11.5-16 us against 17-26 us up to 16 rows, 15.8-21.6 against 18.8-23 at 32 rows:
// both are latency-bound, the tcgen05 kernel pays for the tensor-memory allocation and a second
// barrier hop per chunk, and the mma.sync kernel's launches overlap their set-up with the
// predecessor's tail); at 64 rows tcgen05 wins where its X operand fits in shared memory.  (The
// persistent stack kernel, which the stack launcher uses for M <= 16, is a tcgen05 kernel.)
static int select_path(const LinearParams& p, int sms) {
  if (p.M <= 32) return QL_PATH_MMA;
  return tc5_supported(p, sms) ? QL_PATH_TC5 : QL_PATH_MMA;
}

static int run_linear(const LinearParams& p, int path, cudaStream_t stream, bool pdl = false) {
  const int sms = num_sms();
  if (sms <= 0) return QL_ERR_CUDA;
  if (path == QL_PATH_AUTO) path = select_path(p, sms);
  cudaError_t e;
  switch (path) {
    case QL_PATH_MMA: e = launch_linear_mma(p, stream); break;
    case QL_PATH_TC5:
      if (!tc5_supported(p, sms)) return QL_ERR_UNSUPPORTED;
      e = launch_linear_tc5(p, sms, stream, pdl);
      break;
    default: return QL_ERR_UNSUPPORTED;
  }
  if (e != cudaSuccess) return QL_ERR_CUDA;
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return QL_OK;
}

static int validate_glue(const ql_op& o) {
  if (o.in0 == nullptr || o.out == nullptr) return QL_ERR_NULL;
  if (o.kind == QL_OP_SILU_MUL_UNIT_RMS && o.in1 == nullptr) return QL_ERR_NULL;
  if (o.M < 1 || o.M > 64 || o.N <= 0 || o.N % 8 != 0 || o.ld_in < o.N || o.ld_out < o.N) return QL_ERR_SHAPE;
  if (o.ld_in % 8 != 0 || o.ld_out % 8 != 0 || !aligned16(o.in0) || !aligned16(o.out)) return QL_ERR_ALIGN;
  if (o.in1 != nullptr && !aligned16(o.in1)) return QL_ERR_ALIGN;
  return QL_OK;
}

// ---- stack execution ------------------------------------------------------------------------------
// The operation list is cut into runs that the persistent stack kernel can execute in one launch
// (M <= 16, one group size, every operation's X fits in shared memory).  Inside a run, a glue
// operation that sits between the linear that produces its input and the linear that consumes its
// output is folded into those two, and a gate/up pair followed by its SILU_MUL_UNIT_RMS becomes one
// dual operation.  Whatever does not fit a run is launched on its own, in order.

static int launch_linear_op(const ql_op& o, void* workspace, size_t workspace_bytes, cudaStream_t s, bool pdl) {
  LinearParams p;
  int st = prepare_linear(p, o.packed, o.in0, o.ld_in, o.out, o.ld_out, o.argmax_out, o.M, o.K, o.N, o.g, workspace,
                          workspace_bytes);
  if (st != QL_OK) return st;
  return run_linear(p, QL_PATH_AUTO, s, pdl);
}

static int launch_glue_op(const ql_op& o, cudaStream_t s) {
  if (launch_unit_rms(o.in0, o.in1, o.out, o.M, o.N, o.ld_in, o.ld_out, o.kind == QL_OP_SILU_MUL_UNIT_RMS, s) != cudaSuccess)
    return QL_ERR_CUDA;
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return QL_OK;
}

static MegaOp make_mega(const ql_op& o, const ql_op* second) {
  MegaOp m = {};
  m.packed0 = static_cast<const uint8_t*>(o.packed);
  m.packed1 = second ? static_cast<const uint8_t*>(second->packed) : nullptr;
  m.in0 = o.in0; m.in1 = nullptr;
  m.out0 = o.out; m.out1 = second ? second->out : nullptr;
  m.xout = nullptr; m.argmax_out = o.argmax_out;
  m.draft_ids = o.draft_ids; m.accept_out = o.accept_out;
  m.K = o.K; m.N = o.N; m.ld_in = o.ld_in; m.ld_out = o.ld_out; m.ld_xout = 0;
  m.rows = o.M;
  m.n_tiles = o.N / kTileN; m.n_groups = o.K / o.g;
  m.total_chunks = (uint32_t)m.n_tiles * (uint32_t)m.n_groups;
  m.flags = second ? kOpDual : 0;
  m.prologue = 0; m.src_tiles = 0; m.emit_ssq = 0;
  m.cat_base = 0;
  run_split(m.total_chunks, 1, m.nc, m.cq, m.cr);
  return m;
}

// Byte ranges [lo, hi) of the buffers an operation reads and writes, for the independence test.
struct Span { uintptr_t lo, hi; };
static Span span_of(const void* p, int M, int ld, int n, int elt) {
  if (p == nullptr) return {0, 0};
  const uintptr_t lo = reinterpret_cast<uintptr_t>(p);
  return {lo, lo + ((size_t)(M - 1) * ld + n) * elt};
}
static bool overlap(Span a, Span b) { return a.lo < b.hi && b.lo < a.hi; }

// True if `cur` neither reads nor overwrites anything `prev` writes, nor overwrites what it reads.
static bool independent_ops(const MegaOp& prev, const MegaOp& cur) {
  if (cur.prologue != 0 || prev.argmax_out != nullptr || cur.argmax_out != nullptr) return false;
  const Span pw[3] = {span_of(prev.out0, prev.rows, prev.ld_out, prev.N, 2), span_of(prev.out1, prev.rows, prev.ld_out, prev.N, 2),
                      span_of(prev.xout, prev.rows, prev.ld_xout, prev.K, 2)};
  const Span pr[2] = {span_of(prev.in0, prev.rows, prev.ld_in, prev.K, 2), span_of(prev.in1, prev.rows, prev.ld_in, prev.K, 2)};
  const Span cw[2] = {span_of(cur.out0, cur.rows, cur.ld_out, cur.N, 2), span_of(cur.out1, cur.rows, cur.ld_out, cur.N, 2)};
  const Span cr[1] = {span_of(cur.in0, cur.rows, cur.ld_in, cur.K, 2)};
  for (const Span& a : cw) {
    for (const Span& b : pw) if (overlap(a, b)) return false;
    for (const Span& b : pr) if (overlap(a, b)) return false;
  }
  for (const Span& a : cr)
    for (const Span& b : pw) if (overlap(a, b)) return false;
  return true;
}

// True if the run is a list of plain linears no two of which share a buffer other than inputs
// that both only read: nothing in it has to wait for a result.
static bool independent_run(const std::vector<MegaOp>& mega) {
  if (mega.size() < 2) return false;
  for (const MegaOp& m : mega)
    if (m.packed1 != nullptr || m.prologue != 0 || m.emit_ssq != 0 || m.argmax_out != nullptr || m.out0 == nullptr) return false;
  for (size_t a = 0; a < mega.size(); ++a)
    for (size_t b = a + 1; b < mega.size(); ++b)
      if (!independent_ops(mega[a], mega[b]) || !independent_ops(mega[b], mega[a])) return false;
  return true;
}

// An independent run is laid end to end and cut into one contiguous piece per CTA.
static void split_one_stream(std::vector<MegaOp>& mega, int ncta) {
  uint32_t total = 0;
  for (MegaOp& m : mega) { m.cat_base = total; total += m.total_chunks; }
  for (MegaOp& m : mega) run_split(total, (uint32_t)ncta, m.nc, m.cq, m.cr);
}

// Split of a chained operation.  Where every tile can have at least two CTAs of its own and two
// chunks for each of them (the fused qkv, attention-output and MLP-down projections of a verify
// step: 48 or 20 tiles on 148 CTAs), the aligned split is taken: no CTA meets two tiles.  The
// first CTA of a tile - its owner, which adds the others' partial rows and finishes the tile - can
// be given g_owner_extra chunks more than an even share of the rest; that paid while the rows
// travelled behind a fence and a flag (4 chunks) and no longer does (0: the rows signal themselves
// and arrive while the owner passes its own tile end).  Otherwise (gate/up pairs: 76 double tiles;
// the LM head) the chunks are shared out evenly and pieces cross tile boundaries.
static void chain_split(MegaOp& m, int ncta) {
  m.cat_base = 0;
  const uint32_t nt = (uint32_t)m.n_tiles, Gn = (uint32_t)m.n_groups, nc = (uint32_t)ncta;
  const uint32_t most = (nc + nt - 1) / nt;                  // CTAs of the best-served tile
  const int extra_want = g_owner_extra.load(std::memory_order_relaxed);
  if (extra_want >= 0 && 2 * nt <= nc && Gn >= 2 * most) {
    const uint32_t extra = (uint32_t)extra_want < Gn - most ? (uint32_t)extra_want : Gn - most;   // everyone keeps at least one chunk
    m.nc = nc; m.cq = extra; m.cr = kSplitAligned | nt;
    return;
  }
  run_split(m.total_chunks, nc, m.nc, m.cq, m.cr);
}

static bool is_dual(const ql_op* ops, int i, int n_ops) {
  if (i + 2 >= n_ops) return false;
  const ql_op &a = ops[i], &b = ops[i + 1], &c = ops[i + 2];
  if (b.kind != QL_OP_LINEAR || c.kind != QL_OP_SILU_MUL_UNIT_RMS) return false;
  if (a.in0 != b.in0 || a.K != b.K || a.N != b.N || a.g != b.g || a.M != b.M || a.ld_in != b.ld_in || a.ld_out != b.ld_out) return false;
  if (a.out == nullptr || b.out == nullptr || a.argmax_out != nullptr || b.argmax_out != nullptr) return false;
  if (c.in0 != a.out || c.in1 != b.out || c.N != a.N || c.ld_in != a.ld_out || c.M != a.M) return false;
  return true;
}

// Operations per stack-kernel launch (the partial-tile tags keep 9 bits for the operation number).
constexpr int kStackRunOps = kMaxOps;

// What the planner made of an operation list (ql_stack_plan reports it without launching).
struct StackCounts {
  int stack_launches = 0;   // launches of the persistent stack kernel
  int fused_ops = 0;        // fused operations inside them
  int dual_ops = 0;         // of which gate/up pairs
  int folded_glue = 0;      // glue operations folded into their neighbours
  int independent = 0;      // fused operations that need not wait for their predecessor
  int single_linears = 0;   // linears launched on their own
  int single_glue = 0;      // glue operations launched on their own
  int batch_launches = 0;   // of the stack launches, those that took the batch kernel (independent linears)
};

// A call that turned out to be exactly one launch of the stack kernel, remembered so that the same
// call again (same operation list, workspace and stream, nothing staged in between) only launches:
// the descriptors are still in the workspace.
struct KeptLaunch {
  StackParams sp;
  int g = 0;
  size_t smem = 0;
  uint64_t gen = 0;          // g_desc_gen right after the descriptors were staged
};

static int run_stack(const ql_op* ops, int n_ops, void* workspace, size_t workspace_bytes, cudaStream_t s,
                     StackCounts* dry = nullptr, KeptLaunch* keep = nullptr, StackCounts* counts_out = nullptr) {
  int sms = num_sms();
  if (sms <= 0) {
    if (dry == nullptr) return QL_ERR_CUDA;
    sms = 148;                                          // planning without a device: answer for a B200
  }
  StackCounts cnt;
  static thread_local std::vector<MegaOp> mega;
  mega.clear();
  const ql_op* pend = nullptr;        // glue operation waiting for the linear that consumes its output
  int run_M = 0, run_g = 0;
  bool first_launch = true;

  auto flush = [&]() -> int {
    if (!mega.empty()) {
      const int ncta = stack_ncta(sms);
      // Independent plain linears form ONE run: their chunks are laid end to end and every CTA
      // takes one contiguous piece.  Anything else is a chain: every operation is its own run and
      // waits for the one before it.
      const bool indep = independent_run(mega);
      const bool batch = indep;
      bool x_ring = false;
      if (batch) {
        split_one_stream(mega, ncta);
        for (MegaOp& m : mega) m.flags |= kOpLazy;
        // X resident per operation where it fits (faster: no per-chunk hand-over), else through the ring
        x_ring = !stack_plan(mega.data(), (int)mega.size(), run_g, sms, false).ok;
      } else {
        for (size_t j = 0; j < mega.size(); ++j) {
          MegaOp& m = mega[j];
          chain_split(m, ncta);
          if (j > 0) m.flags |= kOpWait;
        }
        mega.back().flags |= kOpLazy;   // nothing in the launch waits for the last operation: its rows need not be published

      }
      const int hook = g_no_release_op.load(std::memory_order_relaxed);
      if (hook >= 0 && hook < (int)mega.size()) mega[hook].flags |= kOpNoRelease;
      StackPlan plan = stack_plan(mega.data(), (int)mega.size(), run_g, sms, x_ring);
      if (!plan.ok) return QL_ERR_UNSUPPORTED;   // cannot happen: every operation was checked when it was added
      int n_tiles_cap = 1;
      for (const MegaOp& m : mega) n_tiles_cap = m.n_tiles > n_tiles_cap ? m.n_tiles : n_tiles_cap;
      StackParams sp = {};
      sp.ws = ws_carve(workspace, n_tiles_cap, 16);
      sp.ops = reinterpret_cast<const MegaOp*>(sp.ws.desc);
      sp.n_ops = (int)mega.size(); sp.M = run_M; sp.ncta = plan.ncta; sp.n_stages = plan.n_stages; sp.n_x = plan.n_x; sp.x_ring = plan.x_ring; sp.one_stream = batch ? 1 : 0;
      sp.wait_ns = g_wait_ns.load(std::memory_order_relaxed);
      sp.ablate = g_ablate.load(std::memory_order_relaxed);
      sp.timeline = g_timeline.load(std::memory_order_relaxed);
      cnt.stack_launches += 1;
      cnt.batch_launches += batch ? 1 : 0;
      cnt.fused_ops += (int)mega.size();
      for (size_t j = 0; j < mega.size(); ++j) {
        const MegaOp& m = mega[j];
        cnt.dual_ops += (m.flags & kOpDual) != 0;
        cnt.folded_glue += m.prologue != 0;
        cnt.independent += (j > 0 && !(m.flags & kOpWait)) ? 1 : 0;
      }
      if (dry == nullptr) {
        sp.epoch = g_epoch.fetch_add(1, std::memory_order_relaxed) + 1;
        if (cudaMemcpyAsync(sp.ws.desc, mega.data(), mega.size() * sizeof(MegaOp), cudaMemcpyHostToDevice, s) != cudaSuccess)
          return QL_ERR_CUDA;
        const uint64_t gen = g_desc_gen.fetch_add(1, std::memory_order_relaxed) + 1;
        if (launch_stack_tc5(sp, run_g, plan.smem, s) != cudaSuccess) return QL_ERR_CUDA;
        g_launches.fetch_add(1, std::memory_order_relaxed);
        if (keep != nullptr) { keep->sp = sp; keep->g = run_g; keep->smem = plan.smem; keep->gen = gen; }
      }
      mega.clear();
      first_launch = false;
    }
    if (pend != nullptr) {
      cnt.single_glue += 1;
      if (dry == nullptr) {
        const int st = launch_glue_op(*pend, s);
        if (st != QL_OK) return st;
      }
      pend = nullptr;
      first_launch = false;
    }
    return QL_OK;
  };

  // A list of plain linears with one common row count above 16: every linear becomes ceil(M / 16)
  // operations of at most 16 rows each (the persistent kernel's row count), which write disjoint rows
  // and therefore form one stream together with the other linears' slabs.  The weights are then
  // unpacked once per slab, but cross HBM about once: the slabs of a linear are neighbours in the
  // stream, so thread blocks work on them at the same time and meet in L2.
  bool slabs = n_ops > 0;
  for (int i = 0; i < n_ops && slabs; ++i) {
    const ql_op& o = ops[i];
    slabs = o.kind == QL_OP_LINEAR && o.M > 16 && o.M == ops[0].M && o.g == ops[0].g && o.argmax_out == nullptr &&
            o.out != nullptr && o.draft_ids == nullptr && ws_total_bytes(o.N / kTileN, 16) <= workspace_bytes;
    if (slabs) {
      ql_op probe_op = o;
      probe_op.M = 16;
      MegaOp probe = make_mega(probe_op, nullptr);
      run_split(probe.total_chunks, (uint32_t)stack_ncta(sms), probe.nc, probe.cq, probe.cr);
      slabs = stack_plan(&probe, 1, o.g, sms).ok;
    }
  }
  if (slabs) {
    static thread_local std::vector<MegaOp> all;
    all.clear();
    for (int i = 0; i < n_ops; ++i) {
      for (int r0 = 0; r0 < ops[i].M; r0 += 16) {
        ql_op so = ops[i];
        so.M = ops[i].M - r0 < 16 ? ops[i].M - r0 : 16;
        so.in0 = ops[i].in0 + (size_t)r0 * ops[i].ld_in;
        so.out = ops[i].out + (size_t)r0 * ops[i].ld_out;
        all.push_back(make_mega(so, nullptr));
      }
    }
    // only a stream of independent operations gains from this; linears that depend on one another
    // keep their one launch each
    if (independent_run(all)) {
      run_M = 16;
      run_g = ops[0].g;
      for (const MegaOp& m : all) {
        if ((int)mega.size() >= kStackRunOps) {
          const int st = flush();
          if (st != QL_OK) return st;
        }
        mega.push_back(m);
      }
      const int st = flush();
      if (dry != nullptr) *dry = cnt;
      if (counts_out != nullptr) *counts_out = cnt;
      return st;
    }
  }

  for (int i = 0; i < n_ops; ++i) {
    const ql_op& o = ops[i];
    if (o.kind == QL_OP_LINEAR) {
      const bool dual = is_dual(ops, i, n_ops);
      MegaOp m = make_mega(o, dual ? &ops[i + 1] : nullptr);
      if ((int)mega.size() >= kStackRunOps) {           // a launch is full: start the next one
        const int st = flush();
        if (st != QL_OK) return st;
      }
      bool fits = o.M <= 16 && ws_total_bytes(m.n_tiles, 16) <= workspace_bytes;
      if (fits) {
        MegaOp probe = m;                               // would it fit as a chained operation?
        chain_split(probe, stack_ncta(sms));
        fits = stack_plan(&probe, 1, o.g, sms).ok;
      }
      if (fits && !mega.empty() && (o.M != run_M || o.g != run_g)) {
        const int st = flush();
        if (st != QL_OK) return st;
      }
      if (!fits) {
        if (o.draft_ids != nullptr) return QL_ERR_UNSUPPORTED;   // the verification tail lives in the persistent kernel
        int st = flush();
        if (st != QL_OK) return st;
        cnt.single_linears += 1;
        if (dry == nullptr) {
          st = launch_linear_op(o, workspace, workspace_bytes, s, !first_launch);
          if (st != QL_OK) return st;
        }
        first_launch = false;
        continue;
      }
      if (pend != nullptr) {
        // (a gate/up pair that consumes a silu-mul product is not folded: its tiles would overwrite the
        // fp32 product in the workspace while other CTAs still build their X from it)
        const bool fuse = !mega.empty() && pend->out == o.in0 && o.ld_in == pend->ld_out && o.K == pend->N && o.M == run_M &&
                          o.g == run_g && !(dual && pend->kind == QL_OP_SILU_MUL_UNIT_RMS);
        if (fuse) {
          const int kind = pend->kind == QL_OP_SILU_MUL_UNIT_RMS ? 2 : 1;
          m.prologue = kind;
          m.in0 = pend->in0; m.in1 = pend->in1; m.ld_in = pend->ld_in;
          m.xout = pend->out; m.ld_xout = pend->ld_out;
          m.src_tiles = pend->N / kTileN;
          mega.back().emit_ssq = kind;
          pend = nullptr;
        } else {
          const int st = flush();
          if (st != QL_OK) return st;
        }
      }
      if (mega.empty()) { run_M = o.M; run_g = o.g; }
      mega.push_back(m);
      if (dual) ++i;                                  // the second linear of the pair is part of this operation
    } else {
      if (pend != nullptr) {
        const int st = flush();
        if (st != QL_OK) return st;
      }
      bool attach = !mega.empty() && o.M == run_M;
      if (attach) {
        const MegaOp& prod = mega.back();
        if (o.kind == QL_OP_UNIT_RMS)
          attach = !(prod.flags & kOpDual) && prod.out0 != nullptr && o.in0 == prod.out0 && o.ld_in == prod.ld_out &&
                   o.N % kTileN == 0 && o.N <= prod.N;
        else
          attach = (prod.flags & kOpDual) && o.in0 == prod.out0 && o.in1 == prod.out1 && o.N == prod.N && o.ld_in == prod.ld_out;
      }
      if (attach) {
        pend = &o;
      } else {
        int st = flush();
        if (st != QL_OK) return st;
        cnt.single_glue += 1;
        if (dry == nullptr) {
          st = launch_glue_op(o, s);
          if (st != QL_OK) return st;
        }
        first_launch = false;
      }
    }
  }
  const int st = flush();
  if (dry != nullptr) *dry = cnt;
  if (counts_out != nullptr) *counts_out = cnt;
  return st;
}

struct PlanMemo {
  std::vector<ql_op> ops;
  void* workspace = nullptr;
  size_t workspace_bytes = 0;
  cudaStream_t stream = nullptr;
  int device = -1;
  uint64_t gen = 0;          // 0: nothing remembered
  KeptLaunch launch;
};
static thread_local PlanMemo t_memo;
}  // namespace ql

using namespace ql;

extern "C" {

const char* ql_status_str(int s) {
  switch (s) {
    case QL_OK: return "ok";
    case QL_ERR_NULL: return "null pointer";
    case QL_ERR_SHAPE: return "unsupported shape";
    case QL_ERR_ALIGN: return "misaligned pointer or leading dimension";
    case QL_ERR_UNSUPPORTED: return "path not available for this shape or device";
    case QL_ERR_WORKSPACE: return "buffer too small";
    case QL_ERR_CUDA: return "CUDA runtime error";
    case QL_ERR_DEVICE_TIMEOUT: return "bounded wait inside a kernel ran out";
    default: return "unknown status";
  }
}

size_t ql_packed_bytes(int K, int N, int g) {
  if (!shape_ok(1, K, N, g)) return 0;
  return (size_t)(N / kTileN) * (size_t)(K / g) * chunk_bytes(g);
}

size_t ql_workspace_bytes(int M_max, int N_max) {
  if (M_max < 1 || M_max > 64 || N_max <= 0 || N_max % kTileN != 0 || N_max / kTileN > kMaxTiles) return 0;
  return ws_total_bytes(N_max / kTileN, pad_rows(M_max));
}

int ql_workspace_init(void* workspace, size_t workspace_bytes, void* stream) {
  if (workspace == nullptr) return QL_ERR_NULL;
  if (workspace_bytes < kWsControlBytes) return QL_ERR_WORKSPACE;
  if (!aligned16(workspace)) return QL_ERR_ALIGN;
  g_desc_gen.fetch_add(1, std::memory_order_relaxed);     // staged descriptors are gone
  // everything, not only the control words; the stack kernel's partial-tile region holds "nothing waiting" (all ones)
  if (cudaMemsetAsync(workspace, 0, workspace_bytes, static_cast<cudaStream_t>(stream)) != cudaSuccess) return QL_ERR_CUDA;
  const size_t parts_at = kWsControlBytes + kWsDescBytes;
  if (workspace_bytes >= parts_at + kWsPartBytes &&
      cudaMemsetAsync(static_cast<char*>(workspace) + parts_at, 0xFF, kWsPartBytes, static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return QL_ERR_CUDA;
  return QL_OK;
}

int ql_device_status(const void* workspace, int* host_out, void* stream) {
  if (workspace == nullptr || host_out == nullptr) return QL_ERR_NULL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(host_out, workspace, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return QL_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return QL_ERR_CUDA;
  *host_out &= 0xFF;                                   // the upper bits say where a wait gave up
  return QL_OK;
}

int ql_device_status_raw(const void* workspace, int* host_out, void* stream) {
  if (workspace == nullptr || host_out == nullptr) return QL_ERR_NULL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(host_out, workspace, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return QL_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return QL_ERR_CUDA;
  return QL_OK;
}

int qpack_w4_g128(const uint32_t* wq, const uint16_t* scale, const uint8_t* zero, int K, int N, int g, void* packed,
                  size_t packed_bytes, void* stream) {
  if (wq == nullptr || scale == nullptr || packed == nullptr) return QL_ERR_NULL;
  if (!shape_ok(1, K, N, g)) return QL_ERR_SHAPE;
  if (!aligned16(wq) || !aligned16(scale) || !aligned16(packed)) return QL_ERR_ALIGN;
  if (packed_bytes < ql_packed_bytes(K, N, g)) return QL_ERR_WORKSPACE;
  if (launch_qpack(wq, scale, zero, K, N, g, static_cast<uint8_t*>(packed), static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return QL_ERR_CUDA;
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return QL_OK;
}

int qrequant_pack_w4(const uint16_t* w, const uint16_t* scale, const uint8_t* zero, int K, int N, int g, void* packed,
                     size_t packed_bytes, void* stream) {
  if (w == nullptr || scale == nullptr || packed == nullptr) return QL_ERR_NULL;
  if (!shape_ok(1, K, N, g)) return QL_ERR_SHAPE;
  if (!aligned16(w) || !aligned16(scale) || !aligned16(packed)) return QL_ERR_ALIGN;
  if (packed_bytes < ql_packed_bytes(K, N, g)) return QL_ERR_WORKSPACE;
  if (launch_qrequant(w, scale, zero, K, N, g, static_cast<uint8_t*>(packed), static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return QL_ERR_CUDA;
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return QL_OK;
}

// ---- drafter attention ----------------------------------------------------------------------
constexpr size_t kAttnCounterBytes = 256;                // one counter per key/value head, zero between calls

static int attn_fill(AttnParams& p, int n_q, int T, int Hq, int Hkv, int d, int p0, int window, int ld_q, int ld_kv, int ld_out) {
  if (d != 128) return QL_ERR_UNSUPPORTED;
  if (n_q < 1 || n_q > 16 || T < 1 || Hq < 1 || Hkv < 1 || Hq % Hkv != 0 || Hkv > 64 || window < 0) return QL_ERR_SHAPE;
  const int G = Hq / Hkv;
  if (G != 1 && G != 2 && G != 4 && G != 8) return QL_ERR_UNSUPPORTED;
  if (p0 < 0 || p0 + n_q > T) return QL_ERR_SHAPE;        // every query stands on a position of the cache
  if (ld_q < Hq * d || ld_out < Hq * d || ld_kv < Hkv * d) return QL_ERR_SHAPE;
  if (ld_q % 8 != 0 || ld_kv % 8 != 0 || ld_out % 8 != 0) return QL_ERR_ALIGN;
  p.n_q = n_q; p.T = T; p.Hq = Hq; p.Hkv = Hkv; p.G = G; p.p0 = p0; p.window = window;
  p.ld_q = ld_q; p.ld_kv = ld_kv; p.ld_out = ld_out;
  p.scale_log2 = 1.4426950408889634f / sqrtf((float)d);
  return QL_OK;
}

size_t ql_attn_workspace_bytes(int Hq, int Hkv) {
  if (Hq < 1 || Hkv < 1 || Hq % Hkv != 0) return 0;
  int sms = num_sms();
  if (sms <= 0) sms = 148;                              // no device: answer for a B200
  int pieces = sms / Hkv;
  if (pieces < 1) pieces = 1;
  const size_t need = kAttnCounterBytes + (size_t)Hq * pieces * 16 * 132 * sizeof(float);
  return need < kWsControlBytes ? kWsControlBytes : need;   // ql_workspace_init zeroes it: not smaller than what that call accepts
}

int qattn_swa_bf16(const uint16_t* Q, const uint16_t* K, const uint16_t* V, uint16_t* out, int n_q, int T, int Hq, int Hkv,
                   int d, int p0, int window, int ld_q, int ld_kv, int ld_out, void* workspace, size_t workspace_bytes,
                   void* stream) {
  if (Q == nullptr || K == nullptr || V == nullptr || out == nullptr || workspace == nullptr) return QL_ERR_NULL;
  AttnParams p = {};
  const int st = attn_fill(p, n_q, T, Hq, Hkv, d, p0, window, ld_q, ld_kv, ld_out);
  if (st != QL_OK) return st;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(out) || !aligned16(workspace)) return QL_ERR_ALIGN;
  const int sms = num_sms();
  if (sms <= 0) return QL_ERR_CUDA;
  const size_t floats = attn_plan(p, sms);
  if (workspace_bytes < kAttnCounterBytes + floats * sizeof(float)) return QL_ERR_WORKSPACE;
  p.Q = Q; p.K = K; p.V = V; p.out = out;
  p.counters = static_cast<int*>(workspace);
  p.part = reinterpret_cast<float*>(static_cast<char*>(workspace) + kAttnCounterBytes);
  g_desc_gen.fetch_add(1, std::memory_order_relaxed);     // the memory may once have held a stack call's descriptors
  if (launch_attn_swa(p, static_cast<cudaStream_t>(stream)) != cudaSuccess) return QL_ERR_CUDA;
  g_launches.fetch_add(1, std::memory_order_relaxed);
  return QL_OK;
}

int ql_attn_plan(int n_q, int T, int Hq, int Hkv, int d, int p0, int window, int out[4]) {
  if (out == nullptr) return QL_ERR_NULL;
  AttnParams p = {};
  const int st = attn_fill(p, n_q, T, Hq, Hkv, d, p0, window, Hq * d, Hkv * d, Hq * d);
  if (st != QL_OK) return st;
  int sms = num_sms();
  if (sms <= 0) sms = 148;                              // no device: answer for a B200
  attn_plan(p, sms);
  out[0] = p.key_lo; out[1] = p.key_hi; out[2] = p.n_pieces; out[3] = p.sub_per_piece;
  return QL_OK;
}

int ql_select_path(int M, int K, int N, int g) {
  if (!shape_ok(M, K, N, g)) return -QL_ERR_SHAPE;
  LinearParams p = {};
  p.M = M; p.K = K; p.N = N; p.g = g;
  p.n_tiles = N / kTileN; p.n_groups = K / g;
  p.total_chunks = (uint32_t)p.n_tiles * (uint32_t)p.n_groups;
  int sms = num_sms();
  if (sms <= 0) sms = 148;                              // no device: answer for a B200
  int ncta = sms < kMaxCtas ? sms : kMaxCtas;
  if ((uint32_t)ncta > p.total_chunks) ncta = (int)p.total_chunks;
  p.ncta = ncta;
  p.m_pad = pad_rows(M);
  return select_path(p, sms);
}

int ql_linear_plan(int M, int K, int N, int g, int path, int out[4]) {
  if (out == nullptr) return QL_ERR_NULL;
  if (!shape_ok(M, K, N, g)) return QL_ERR_SHAPE;
  if (path != QL_PATH_AUTO && path != QL_PATH_MMA && path != QL_PATH_TC5) return QL_ERR_UNSUPPORTED;
  LinearParams p = {};
  p.M = M; p.K = K; p.N = N; p.g = g;
  p.n_tiles = N / kTileN; p.n_groups = K / g;
  p.total_chunks = (uint32_t)p.n_tiles * (uint32_t)p.n_groups;
  int sms = num_sms();
  if (sms <= 0) sms = 148;                              // no device: answer for a B200
  int ncta = sms < kMaxCtas ? sms : kMaxCtas;
  if ((uint32_t)ncta > p.total_chunks) ncta = (int)p.total_chunks;
  p.ncta = ncta;
  p.m_pad = pad_rows(M);
  if (path == QL_PATH_AUTO) path = select_path(p, sms);
  if (path == QL_PATH_TC5 && !tc5_supported(p, sms)) return QL_ERR_UNSUPPORTED;
  out[0] = path; out[1] = 0; out[2] = 0; out[3] = 0;
  if (path == QL_PATH_MMA) {
    if (plan_linear_mma(p) == 0) return QL_ERR_UNSUPPORTED;
    out[1] = p.n_stages; out[2] = p.n_x; out[3] = p.x_phase;
  }
  return QL_OK;
}

int qlinear_w4a16_path(const void* packed, const uint16_t* X, uint16_t* Y, int32_t* argmax_out, int M, int K, int N,
                       int g, void* workspace, size_t workspace_bytes, void* stream, int path) {
  LinearParams p;
  int st = validate_linear(packed, X, K, Y, N, argmax_out, M, K, N, g, workspace, workspace_bytes);
  if (st != QL_OK) return st;
  if (path != QL_PATH_AUTO && path != QL_PATH_MMA && path != QL_PATH_TC5) return QL_ERR_UNSUPPORTED;
  st = prepare_linear(p, packed, X, K, Y, N, argmax_out, M, K, N, g, workspace, workspace_bytes);
  if (st != QL_OK) return st;
  return run_linear(p, path, static_cast<cudaStream_t>(stream));
}

int qlinear_w4a16(const void* packed, const uint16_t* X, uint16_t* Y, int32_t* argmax_out, int M, int K, int N, int g,
                  void* workspace, size_t workspace_bytes, void* stream) {
  return qlinear_w4a16_path(packed, X, Y, argmax_out, M, K, N, g, workspace, workspace_bytes, stream, QL_PATH_AUTO);
}

static int validate_stack(const ql_op* ops, int n_ops, const void* workspace, size_t workspace_bytes) {
  if (ops == nullptr || workspace == nullptr) return QL_ERR_NULL;
  if (n_ops < 0) return QL_ERR_SHAPE;
  for (int i = 0; i < n_ops; ++i) {
    const ql_op& o = ops[i];
    if (o.reserved != 0) return QL_ERR_SHAPE;
    if (o.kind == QL_OP_LINEAR) {
      const int st = validate_linear(o.packed, o.in0, o.ld_in, o.out, o.ld_out, o.argmax_out, o.M, o.K, o.N, o.g,
                                     workspace, workspace_bytes);
      if (st != QL_OK) return st;
      if (o.draft_ids != nullptr || o.accept_out != nullptr) {       // verification tail
        if (o.draft_ids == nullptr || o.accept_out == nullptr || o.argmax_out == nullptr) return QL_ERR_NULL;
        if ((reinterpret_cast<uintptr_t>(o.draft_ids) & 3u) || (reinterpret_cast<uintptr_t>(o.accept_out) & 3u)) return QL_ERR_ALIGN;
        if (o.M > 16) return QL_ERR_UNSUPPORTED;
      }
    } else if (o.kind == QL_OP_UNIT_RMS || o.kind == QL_OP_SILU_MUL_UNIT_RMS) {
      const int st = validate_glue(o);
      if (st != QL_OK) return st;
      if (o.draft_ids != nullptr || o.accept_out != nullptr) return QL_ERR_UNSUPPORTED;
    } else {
      return QL_ERR_UNSUPPORTED;
    }
  }
  return QL_OK;
}

int qlinear_stack_w4a16(const ql_op* ops, int n_ops, void* workspace, size_t workspace_bytes, void* stream) {
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  PlanMemo& memo = t_memo;
  int dev = -1;
  // the same call as the last one of this thread, with its descriptors still staged: launch only
  if (ops != nullptr && n_ops > 0 && memo.gen != 0 && memo.gen == g_desc_gen.load(std::memory_order_relaxed) &&
      (size_t)n_ops == memo.ops.size() && workspace == memo.workspace && workspace_bytes == memo.workspace_bytes &&
      s == memo.stream && cudaGetDevice(&dev) == cudaSuccess && dev == memo.device &&
      std::memcmp(ops, memo.ops.data(), sizeof(ql_op) * (size_t)n_ops) == 0) {
    StackParams sp = memo.launch.sp;
    sp.epoch = g_epoch.fetch_add(1, std::memory_order_relaxed) + 1;
    if (launch_stack_tc5(sp, memo.launch.g, memo.launch.smem, s) != cudaSuccess) return QL_ERR_CUDA;
    g_launches.fetch_add(1, std::memory_order_relaxed);
    return QL_OK;
  }
  // validate everything before anything is launched
  const int vst = validate_stack(ops, n_ops, workspace, workspace_bytes);
  if (vst != QL_OK) return vst;
  memo.gen = 0;
  KeptLaunch kept;
  StackCounts cnt;
  const int st = run_stack(ops, n_ops, workspace, workspace_bytes, s, nullptr, &kept, &cnt);
  if (st == QL_OK && cnt.stack_launches == 1 && cnt.single_linears == 0 && cnt.single_glue == 0 &&
      cudaGetDevice(&dev) == cudaSuccess) {
    memo.ops.assign(ops, ops + n_ops);
    memo.workspace = workspace; memo.workspace_bytes = workspace_bytes; memo.stream = s; memo.device = dev;
    memo.launch = kept;
    memo.gen = kept.gen;     // valid while g_desc_gen still has this value: nothing was staged anywhere since
  }
  return st;
}

int qlinear_stack_w4a16_host(const ql_op* ops, int n_ops, const void* host_in, void* dev_in, size_t in_bytes,
                             const void* dev_out, void* host_out, size_t out_bytes, void* workspace,
                             size_t workspace_bytes, void* stream) {
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (in_bytes > 0) {
    if (host_in == nullptr || dev_in == nullptr) return QL_ERR_NULL;
    if (cudaMemcpyAsync(dev_in, host_in, in_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return QL_ERR_CUDA;
  }
  const int st = qlinear_stack_w4a16(ops, n_ops, workspace, workspace_bytes, stream);
  if (st != QL_OK) return st;
  if (out_bytes > 0) {
    if (host_out == nullptr || dev_out == nullptr) return QL_ERR_NULL;
    if (cudaMemcpyAsync(host_out, dev_out, out_bytes, cudaMemcpyDeviceToHost, s) != cudaSuccess) return QL_ERR_CUDA;
  }
  if (cudaStreamSynchronize(s) != cudaSuccess) return QL_ERR_CUDA;
  return QL_OK;
}

int ql_stack_plan(const ql_op* ops, int n_ops, void* workspace, size_t workspace_bytes, int counts[8]) {
  if (counts == nullptr) return QL_ERR_NULL;
  const int vst = validate_stack(ops, n_ops, workspace, workspace_bytes);
  if (vst != QL_OK) return vst;
  StackCounts c;
  const int st = run_stack(ops, n_ops, workspace, workspace_bytes, nullptr, &c);
  counts[0] = c.stack_launches; counts[1] = c.fused_ops; counts[2] = c.dual_ops; counts[3] = c.folded_glue;
  counts[4] = c.independent; counts[5] = c.single_linears; counts[6] = c.single_glue; counts[7] = c.batch_launches;
  return st;
}

uint32_t ql_plan_first_chunk(uint32_t total_chunks, uint32_t ncta, uint32_t cta) {
  if (total_chunks == 0 || ncta == 0) return 0;
  uint32_t nc, cq, cr;
  run_split(total_chunks, ncta, nc, cq, cr);
  return run_first_chunk(nc, cq, cr, cta < nc ? cta : nc);
}

uint32_t ql_plan_chunk_owner(uint32_t total_chunks, uint32_t ncta, uint32_t chunk) {
  if (total_chunks == 0 || ncta == 0 || chunk >= total_chunks) return 0;
  uint32_t nc, cq, cr;
  run_split(total_chunks, ncta, nc, cq, cr);
  return run_chunk_owner(nc, cq, cr, chunk);
}

int ql_plan_chain_split(int n_tiles, int n_groups, int ncta, int cta, uint32_t range[4]) {
  if (range == nullptr) return QL_ERR_NULL;
  if (n_tiles < 1 || n_groups < 1 || ncta < 1 || ncta > kMaxCtas / 2 || cta < 0 || cta >= ncta) return QL_ERR_SHAPE;
  MegaOp m = {};
  m.n_tiles = n_tiles; m.n_groups = n_groups;
  m.total_chunks = (uint32_t)n_tiles * (uint32_t)n_groups;
  chain_split(m, ncta);
  op_local_range(m.nc, m.cq, m.cr, 0, m.total_chunks, (uint32_t)cta, range[0], range[1]);
  range[2] = (m.cr & kSplitAligned) ? 1u : 0u;
  range[3] = range[0] < range[1] ? op_last_cta(m.nc, m.cq, m.cr, 0, (uint32_t)n_groups, (range[1] - 1) / (uint32_t)n_groups) : 0u;
  return QL_OK;
}

void ql_debug_set_wait_budget_ns(uint64_t ns) { g_desc_gen.fetch_add(1, std::memory_order_relaxed); g_wait_ns.store(ns == 0 ? kWaitBudgetNs : ns, std::memory_order_relaxed); }
void ql_debug_set_timeline(void* device_buffer) { g_desc_gen.fetch_add(1, std::memory_order_relaxed); g_timeline.store(static_cast<uint64_t*>(device_buffer), std::memory_order_relaxed); }
int ql_debug_timeline_enabled(void) {
#ifdef QL_TIMELINE
  return 1;
#else
  return 0;
#endif
}
void ql_debug_set_ablate(int mask) { g_desc_gen.fetch_add(1, std::memory_order_relaxed); g_ablate.store(mask, std::memory_order_relaxed); }
void ql_debug_set_owner_extra(int chunks) {
  g_desc_gen.fetch_add(1, std::memory_order_relaxed);
  g_owner_extra.store(chunks == -1 ? kOwnerExtraChunks : chunks, std::memory_order_relaxed);
}
void ql_debug_no_release(int fused_op) { g_desc_gen.fetch_add(1, std::memory_order_relaxed); g_no_release_op.store(fused_op, std::memory_order_relaxed); }

uint64_t ql_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

}  // extern "C"
