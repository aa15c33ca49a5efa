// qlinear_w4a16_static: the single-linear GEMM with its scratch memory (split-K partial tiles,
// tile counters, arg-max candidates, status word) in a static device array of this library
// instead of a caller-provided workspace.  Nothing is allocated, by this code or by any library
// it calls.  The kernel is the warp-level MMA kernel of qlinear_w4a16 (QL_PATH_MMA), unchanged.
#include <atomic>

#include "../../include/qlinear_w4a16.h"
#include "ql_params.h"

namespace ql {
cudaError_t launch_linear_mma(LinearParams, cudaStream_t);
void count_launch();

// Limits of the static variant (stated in the header): M <= 16 rows, N <= 16384 columns.
constexpr int kStaticMaxM = 16;
constexpr int kStaticMaxTiles = 128;                          // N <= 128 * 128
constexpr int kStaticMaxCtas = 160;                           // one CTA per SM
constexpr size_t kStaticCandBytes = (size_t)kStaticMaxTiles * 16 * 8;
constexpr size_t kStaticSlotBytes = (size_t)kStaticMaxCtas * 2 * 2 * 16 * kTileN * 4;   // ws_slot_floats(16) floats per slot
constexpr size_t kStaticBytes = kWsControlBytes + kStaticCandBytes + kStaticSlotBytes;    // about 5.8 MB

// Every GPU that loads the library holds this array until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticBytes];

// Device address of the array, resolved once per device.  In host code `g_static_scratch` is only
// a handle for the runtime, not an address a kernel could use.
static unsigned char* static_scratch_ptr() {
  static std::atomic<unsigned char*> ptr[16] = {};     // two threads may make the first call at once
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 16) return nullptr;
  unsigned char* cur = ptr[dev].load(std::memory_order_acquire);
  if (cur == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess) return nullptr;
    cur = static_cast<unsigned char*>(p);
    ptr[dev].store(cur, std::memory_order_release);
  }
  return cur;
}
}  // namespace ql

using namespace ql;

extern "C" int qlinear_w4a16_static(const void* packed, const uint16_t* X, uint16_t* Y, int32_t* argmax_out, int M,
                                    int K, int N, int g, void* stream) {
  if (packed == nullptr || X == nullptr) return QL_ERR_NULL;
  if (Y == nullptr && argmax_out == nullptr) return QL_ERR_NULL;
  if (M < 1 || (g != 64 && g != 128) || K <= 0 || N <= 0 || K % g != 0 || N % kTileN != 0) return QL_ERR_SHAPE;
  if (M > kStaticMaxM || N / kTileN > kStaticMaxTiles) return QL_ERR_WORKSPACE;   // beyond the static scratch
  if ((int64_t)(N / kTileN) * (K / g) > 0x7fffffffLL) return QL_ERR_SHAPE;
  auto mis16 = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) != 0; };
  if (mis16(packed) || mis16(X) || (Y != nullptr && mis16(Y)) || K % 8 != 0) return QL_ERR_ALIGN;
  if (argmax_out != nullptr && (reinterpret_cast<uintptr_t>(argmax_out) & 3u)) return QL_ERR_ALIGN;

  unsigned char* scratch = static_scratch_ptr();       // first call on a device resolves the address
  if (scratch == nullptr) return QL_ERR_CUDA;
  int dev = 0, sms = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return QL_ERR_CUDA;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) return QL_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  // every call shares the array and it keeps the last call's contents: the control words
  // (status, counters) must start at zero, the rest is overwritten before it is read
  if (cudaMemsetAsync(scratch, 0, kWsControlBytes, s) != cudaSuccess) return QL_ERR_CUDA;

  LinearParams p = {};
  p.packed = static_cast<const uint8_t*>(packed);
  p.X = X; p.Y = Y; p.argmax_out = argmax_out;
  p.M = M; p.K = K; p.N = N; p.g = g; p.ldx = K; p.ldy = N;
  p.n_tiles = N / kTileN; p.n_groups = K / g;
  p.total_chunks = (uint32_t)p.n_tiles * (uint32_t)p.n_groups;
  int ncta = sms < kStaticMaxCtas ? sms : kStaticMaxCtas;
  if ((uint32_t)ncta > p.total_chunks) ncta = (int)p.total_chunks;
  p.ncta = ncta;
  p.m_pad = 16;
  Workspace w = {};
  w.status = reinterpret_cast<int*>(scratch);
  w.amax_done = w.status + 1;
  w.exit_cnt = w.status + 2;
  w.tile_cnt = reinterpret_cast<int*>(scratch + kWsHeaderBytes);
  w.op_done = w.tile_cnt + kFlagWords;
  w.cand = reinterpret_cast<float2*>(scratch + kWsControlBytes);
  w.slots = reinterpret_cast<float*>(scratch + kWsControlBytes + kStaticCandBytes);
  w.n_tiles = kStaticMaxTiles;
  p.ws = w;
  if (launch_linear_mma(p, s) != cudaSuccess) return QL_ERR_CUDA;
  count_launch();
  return QL_OK;
}

extern "C" int ql_static_status(int* host_out, void* stream) {
  if (host_out == nullptr) return QL_ERR_NULL;
  unsigned char* scratch = static_scratch_ptr();
  if (scratch == nullptr) return QL_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaMemcpyAsync(host_out, scratch, sizeof(int), cudaMemcpyDeviceToHost, s) != cudaSuccess) return QL_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return QL_ERR_CUDA;
  *host_out &= 0xFF;
  return QL_OK;
}
