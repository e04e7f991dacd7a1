// rom_route_noalloc: the router / top-K / permutation step for callers that cannot allocate
// device memory.  Some hosts hand this library a fixed set of buffers and forbid cudaMalloc at run
// time (a memory pool owned by another component, an allocator that is locked during steady-state
// serving, a real-time loop where an allocation's latency and possible failure are unacceptable).
// rom_route needs about 2 MiB of scratch beyond its inputs and outputs; here that scratch is a
// fixed array in the library's own device image, so the caller passes inputs and outputs only.
//
// The array exists once per GPU that loads the library and lives until the process exits.  Every
// call on a GPU shares it: two calls that overlap on that GPU (different streams, different host
// threads) race on it.  It keeps the previous call's contents; each call rewrites every table it
// reads, and the one table that must start cleared (row -> assignment, -1 in padding rows) is
// cleared by the launch sequence on the caller's stream.
#include <mutex>

#include "rom_internal.cuh"

namespace rom {
namespace {

constexpr int kNoAllocMaxTokens = 65536;          // B * L
constexpr int kNoAllocMaxAssign = 131072;         // B * L * K
constexpr size_t kNoAllocBytes = (size_t)3 << 20; // 3 MiB: the tables below at the maxima, E = 64

static __device__ __align__(256) unsigned char g_route_scratch[kNoAllocBytes];

// Only the tables the routing kernels touch, packed; the remaining fields stay 0 and unused.
WsLayout make_route_only_layout(const rom_config& c) {
  WsLayout l{};
  l.esz = c.dtype == ROM_BF16 ? 2 : 4;
  l.T = (int64_t)c.B * c.L;
  l.A = l.T * c.K;
  l.rows_max = (int64_t)align_up((size_t)l.A, kTileM) + (int64_t)c.E * kTileM;
  l.max_m_tiles = l.rows_max / kTileM;
  l.n_chunks = (l.T + kChunkTokens - 1) / kChunkTokens;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
  l.status = take(sizeof(int32_t) * kStatusInts);      // only its blocks-done counter is used: zero at load, left zero by every call
  l.counts = take(sizeof(int32_t) * c.E);
  l.offsets = take(sizeof(int32_t) * (c.E + 1));
  l.pad_offsets = take(sizeof(int32_t) * (c.E + 1));
  l.num_m_tiles = take(sizeof(int32_t) * 4);
  l.tile_expert = take(sizeof(int32_t) * l.max_m_tiles);
  l.chunk_counts = take(sizeof(int32_t) * l.n_chunks * c.E);
  l.topk_idx = take(sizeof(int32_t) * l.A);
  l.row_of_assign = take(sizeof(int32_t) * l.A);
  l.assign_of_row = take(sizeof(int32_t) * l.rows_max);
  l.total = o;
  return l;
}

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char* g_scratch_addr[kMaxDevices] = {};   // device address of g_route_scratch, per device ordinal

// The array's name is only a host-side handle in host code; the kernels need its device address,
// which differs per GPU.  Looked up once per device, with that device current.
int scratch_for_current_device(unsigned char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return ROM_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return ROM_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_route_scratch) != cudaSuccess || !p) return ROM_ERR_CUDA;
    g_scratch_addr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_addr[dev];
  return ROM_OK;
}

}  // namespace
}  // namespace rom

using namespace rom;

extern "C" int rom_route_noalloc(const rom_config* cfg, const void* x, const void* W_r, const float* b_r,
                                 int32_t* topk_idx, float* gates, int32_t* counts, int32_t* offsets,
                                 int32_t* perm, int32_t* inv_perm, void* stream) {
  if (!cfg || !x || !W_r) return ROM_ERR_INVALID_ARG;
  const int cfg_rc = check_config(cfg, 1);      // the same argument rules as rom_route
  if (cfg_rc != ROM_OK) return cfg_rc;
  const rom_config& c = *cfg;
  if ((reinterpret_cast<uintptr_t>(x) & 15u) || (reinterpret_cast<uintptr_t>(W_r) & 15u)) return ROM_ERR_INVALID_ARG;
  // the built-in scratch has a fixed size: larger problems must use rom_route with a caller workspace
  if ((int64_t)c.B * c.L > kNoAllocMaxTokens || (int64_t)c.B * c.L * c.K > kNoAllocMaxAssign) return ROM_ERR_STATIC_SCRATCH;
  const WsLayout lay = make_route_only_layout(c);
  if (lay.total > kNoAllocBytes) return ROM_ERR_STATIC_SCRATCH;
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return ROM_ERR_CUDA;
  if (major != 10) return ROM_ERR_ARCH;
  unsigned char* scratch = nullptr;
  const int rc = scratch_for_current_device(&scratch);
  if (rc != ROM_OK) return rc;
  LaunchCounter::count = 0;
  if (launch_route(c, x, W_r, b_r, topk_idx, gates, counts, offsets, perm, inv_perm, reinterpret_cast<char*>(scratch), lay,
                   static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return ROM_ERR_CUDA;
  return ROM_OK;
}
