// Feed-forward SwiGLU mixture of experts that reuses the routing decision of the preceding RoM layer
// (Appendix A.2, the hybrid "RoM + FFN-MoE" model):
//   Y_t = sum_i R_i * 1[i in TopK] * f_i(X_t),   f_i(x) = W_down,i ( SiLU(W_gate,i x) * (W_up,i x) ),
// with the selected experts and their gates R_i handed over from that layer's router.
// Launch sequence: permutation tables from the given indices -> gather tokens by expert -> grouped
// [gate | up] projection with the SwiGLU product as its output op -> grouped down projection ->
// gate-weighted sum over the K slots (fused into the down projection's output op when K = 1).
#include "rom_internal.cuh"

namespace rom {
namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Workspace of rom_ffn_moe_forward: the routing tables and three row buffers in expert order.
WsLayout make_ffn_layout(const rom_config& c, int d_ff) {
  WsLayout l{};
  l.esz = c.dtype == ROM_BF16 ? 2 : 4;
  l.T = (int64_t)c.B * c.L;
  l.A = l.T * c.K;
  l.rows_max = (int64_t)align_up((size_t)l.A, kTileM) + (int64_t)c.E * kTileM;
  l.max_m_tiles = l.rows_max / kTileM;
  l.n_chunks = (l.T + kChunkTokens - 1) / kChunkTokens;
  const bool tc = c.dtype == ROM_BF16 && !(c.flags & ROM_FLAG_SIMT_GEMM);
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
  l.status = take(sizeof(int32_t) * kStatusInts);
  l.counts = take(sizeof(int32_t) * c.E);
  l.offsets = take(sizeof(int32_t) * (c.E + 1));
  l.pad_offsets = take(sizeof(int32_t) * (c.E + 1));
  l.num_m_tiles = take(sizeof(int32_t) * 4);
  l.tile_expert = take(sizeof(int32_t) * l.max_m_tiles);
  l.chunk_counts = take(sizeof(int32_t) * l.n_chunks * c.E);
  l.topk_idx = take(sizeof(int32_t) * l.A);
  l.row_of_assign = take(sizeof(int32_t) * l.A);
  l.assign_of_row = take(sizeof(int32_t) * l.rows_max);
  l.x_perm = take(l.esz * (size_t)l.rows_max * c.d_model);
  l.XZp = take(tc ? 0 : l.esz * (size_t)l.rows_max * 2 * d_ff);     // [gate | up] rows: only the plain-FMA path stores them
  l.Ygp = take(l.esz * (size_t)l.rows_max * d_ff);                  // hidden rows SiLU(gate) * up
  l.Op = take((tc && c.K == 1) ? 0 : l.esz * (size_t)l.rows_max * c.d_model);
  l.total = o;
  return l;
}

int check_ffn(const rom_config* c, int d_ff) {
  if (!c) return ROM_ERR_INVALID_ARG;
  if (c->dtype != ROM_F32 && c->dtype != ROM_BF16) return ROM_ERR_INVALID_ARG;
  if (c->B < 1 || c->L < 1 || c->E < 1 || c->K < 1 || c->K > c->E) return ROM_ERR_INVALID_ARG;
  if ((c->flags & ~ROM_FLAG_SIMT_GEMM) != 0) return ROM_ERR_INVALID_ARG;
  if (c->E > kMaxE || c->K > kMaxK) return ROM_ERR_UNSUPPORTED;
  if (c->d_model < 64 || c->d_model % 64 != 0) return ROM_ERR_INVALID_ARG;
  if (d_ff < 128 || d_ff % 128 != 0) return d_ff < 1 ? ROM_ERR_INVALID_ARG : ROM_ERR_UNSUPPORTED;
  if ((int64_t)c->B * c->L * c->K >= (int64_t)1 << 30) return ROM_ERR_UNSUPPORTED;
  return ROM_OK;
}

// Plain-FMA path only: H[r, j] = SiLU(GU[r, j]) * GU[r, d_ff + j] over the valid rows.
template <typename T>
__global__ void __launch_bounds__(256)
swiglu_rows(const T* __restrict__ GU, T* __restrict__ H, const int32_t* __restrict__ pad_offsets, int E, int d_ff, long long total) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total) return;
  const long long r = i / d_ff;
  if (r >= pad_offsets[E]) return;
  const int j = (int)(i % d_ff);
  const float g = to_f32(GU[r * 2 * d_ff + j]), u = to_f32(GU[r * 2 * d_ff + d_ff + j]);
  H[i] = from_f32<T>(silu_f(g) * u);
}

#define ROM_CUDA(expr)                            \
  do {                                            \
    cudaError_t e__ = (expr);                     \
    if (e__ != cudaSuccess) return ROM_ERR_CUDA;  \
  } while (0)

}  // namespace
}  // namespace rom

using namespace rom;

extern "C" {

int rom_ffn_moe_workspace_size(const rom_config* cfg, int32_t d_ff, size_t* bytes) {
  if (!bytes) return ROM_ERR_INVALID_ARG;
  const int rc = check_ffn(cfg, d_ff);
  if (rc != ROM_OK) return rc;
  *bytes = make_ffn_layout(*cfg, d_ff).total;
  return ROM_OK;
}

int rom_ffn_moe_forward(const rom_config* cfg, int32_t d_ff, const void* W_gu, const void* W_down, const void* x,
                        const int32_t* topk_idx, const float* gates, void* out, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_ffn(cfg, d_ff);
  if (rc != ROM_OK) return rc;
  if (!W_gu || !W_down || !x || !topk_idx || !gates || !out || !ws) return ROM_ERR_INVALID_ARG;
  const void* ptrs[] = {W_gu, W_down, x, topk_idx, gates, out, ws};
  for (const void* p : ptrs)
    if (!aligned16(p)) return ROM_ERR_INVALID_ARG;
  const rom_config& c = *cfg;
  const WsLayout lay = make_ffn_layout(c, d_ff);
  if (ws_bytes < lay.total) return ROM_ERR_WORKSPACE;
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return ROM_ERR_CUDA;
  if (major != 10) return ROM_ERR_ARCH;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* W = static_cast<char*>(ws);
  LaunchCounter::count = 0;

  const int Dm = c.d_model;
  const bool tc = c.dtype == ROM_BF16 && !(c.flags & ROM_FLAG_SIMT_GEMM);
  int32_t* status = reinterpret_cast<int32_t*>(W + lay.status);
  const int32_t* tile_expert = reinterpret_cast<const int32_t*>(W + lay.tile_expert);
  const int32_t* num_m_tiles = reinterpret_cast<const int32_t*>(W + lay.num_m_tiles);
  const int32_t* row_of_assign = reinterpret_cast<const int32_t*>(W + lay.row_of_assign);
  const int32_t* assign_of_row = reinterpret_cast<const int32_t*>(W + lay.assign_of_row);

  ROM_CUDA(cudaMemsetAsync(status, 0, sizeof(int32_t) * kStatusInts, st));
  // the shared routing decision -> this call's own permutation tables
  ROM_CUDA(launch_perm_from_idx(c, topk_idx, nullptr, nullptr, nullptr, nullptr, W, lay, st));
  ROM_CUDA(launch_gather_rows(c, x, W, lay, st));
  if (tc) {
    // [gate | up] projection; the output op forms SiLU(gate) * up from the accumulator, nothing wider is stored
    Epilogue e_up{EPI_SWIGLU, W + lay.Ygp, d_ff, nullptr, nullptr, nullptr, d_ff, 0, nullptr, nullptr};
    ROM_CUDA(launch_gemm_tc(W + lay.x_perm, Dm, W_gu, Dm, c.E, (int)lay.rows_max, d_ff, Dm, tile_expert, num_m_tiles, e_up, status, st));
    if (c.K == 1) {
      // down projection: rows scaled by their gate and written at their token's position
      Epilogue e_dn{EPI_OUTPROJ, out, Dm, nullptr, nullptr, nullptr, 0, 0, assign_of_row, gates};
      ROM_CUDA(launch_gemm_tc(W + lay.Ygp, d_ff, W_down, d_ff, c.E, (int)lay.rows_max, Dm, d_ff, tile_expert, num_m_tiles, e_dn, status, st));
      return ROM_OK;
    }
    Epilogue e_dn{EPI_STORE, W + lay.Op, Dm, nullptr, nullptr, nullptr, 0, 0, nullptr, nullptr};
    ROM_CUDA(launch_gemm_tc(W + lay.Ygp, d_ff, W_down, d_ff, c.E, (int)lay.rows_max, Dm, d_ff, tile_expert, num_m_tiles, e_dn, status, st));
  } else {
    Epilogue e_up{EPI_STORE, W + lay.XZp, 2 * d_ff, nullptr, nullptr, nullptr, 0, 0, nullptr, nullptr};
    ROM_CUDA(launch_gemm_simt(c.dtype, W + lay.x_perm, Dm, W_gu, Dm, (int64_t)2 * d_ff * Dm, (int)lay.rows_max, 2 * d_ff, Dm,
                              tile_expert, num_m_tiles, e_up, st));
    const long long total = (long long)lay.rows_max * d_ff;
    const unsigned blocks = (unsigned)((total + 255) / 256);
    const int32_t* pad_offsets = reinterpret_cast<const int32_t*>(W + lay.pad_offsets);
    if (c.dtype == ROM_BF16)
      swiglu_rows<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)(W + lay.XZp), (__nv_bfloat16*)(W + lay.Ygp), pad_offsets, c.E, d_ff, total);
    else
      swiglu_rows<float><<<blocks, 256, 0, st>>>((const float*)(W + lay.XZp), (float*)(W + lay.Ygp), pad_offsets, c.E, d_ff, total);
    count_launch();
    ROM_CUDA(cudaGetLastError());
    Epilogue e_dn{EPI_STORE, W + lay.Op, Dm, nullptr, nullptr, nullptr, 0, 0, nullptr, nullptr};
    ROM_CUDA(launch_gemm_simt(c.dtype, W + lay.Ygp, d_ff, W_down, d_ff, (int64_t)Dm * d_ff, (int)lay.rows_max, Dm, d_ff, tile_expert,
                              num_m_tiles, e_dn, st));
  }
  ROM_CUDA(launch_combine(c, W + lay.Op, row_of_assign, gates, out, st));
  return ROM_OK;
}

}  // extern "C"
