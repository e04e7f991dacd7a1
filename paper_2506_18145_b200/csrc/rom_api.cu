// C ABI of the RoM layer forward: argument checks, workspace carving, launch sequence.
#include <cstring>

#include "rom_internal.cuh"

namespace rom {

thread_local int LaunchCounter::count = 0;

WsLayout make_layout(const rom_config& c) {
  WsLayout l{};
  l.esz = c.dtype == ROM_BF16 ? 2 : 4;
  l.T = (int64_t)c.B * c.L;
  l.A = l.T * c.K;
  // every expert segment is padded to a multiple of kTileM rows: at most kTileM-1 extra rows each
  l.rows_max = (int64_t)align_up((size_t)l.A, kTileM) + (int64_t)c.E * kTileM;
  l.max_m_tiles = l.rows_max / kTileM;
  l.n_chunks = (l.T + kChunkTokens - 1) / kChunkTokens;
  const int R = c.dt_rank, N = c.d_state;
  size_t o = 0;
  const bool canaries = (c.flags & ROM_FLAG_DEBUG_CHECKS) != 0;
  auto take = [&](size_t bytes) {
    size_t at = o;
    o = align_up(o + bytes, 256);
    if (canaries && l.n_canary < kMaxCanaries) { l.canary[l.n_canary++] = o; o += kCanaryBytes; }
    return at;
  };
  l.status = take(sizeof(int32_t) * kStatusInts);
  l.counts = take(sizeof(int32_t) * c.E);
  l.offsets = take(sizeof(int32_t) * (c.E + 1));
  l.pad_offsets = take(sizeof(int32_t) * (c.E + 1));
  l.num_m_tiles = take(sizeof(int32_t) * 4);
  l.tile_expert = take(sizeof(int32_t) * l.max_m_tiles);
  l.chunk_counts = take(sizeof(int32_t) * l.n_chunks * c.E);
  l.chunk_prob = take(sizeof(double) * l.n_chunks * c.E);      // per-chunk softmax sums (rom_route_balance)
  l.topk_idx = take(sizeof(int32_t) * l.A);
  l.gates = take(sizeof(float) * l.A);
  l.perm = take(sizeof(int32_t) * l.A);
  l.inv_perm = take(sizeof(int32_t) * l.A);
  l.row_of_assign = take(sizeof(int32_t) * l.A);
  l.assign_of_row = take(sizeof(int32_t) * l.rows_max);
  l.x_perm = take(l.esz * (size_t)l.rows_max * c.d_model);
  l.XZp = take(l.esz * (size_t)l.rows_max * 2 * c.d_inner);
  l.U = take(l.esz * (size_t)l.T * c.d_inner);
  l.Zs = take(c.K > 1 ? l.esz * (size_t)l.T * c.d_inner : 0);   // gate rows summed over the K slots
  l.delta_r = take(l.esz * (size_t)l.T * R);
  l.Bm = take(sizeof(float) * (size_t)l.T * N);
  l.Cm = take(sizeof(float) * (size_t)l.T * N);
  l.Delta = take(l.esz * (size_t)l.T * c.d_inner);
  l.Ygp = take(l.esz * (size_t)l.rows_max * c.d_inner);
  l.Op = take(l.esz * (size_t)l.rows_max * c.d_model);
  l.scan_ws = take(sizeof(float) * scan_ws_floats(c.B, c.d_inner, c.L));
  // per-expert x Proj / dt Proj: their outputs in expert order, summed over the K slots afterwards
  const bool routed_small = c.small_proj_experts > 1;
  l.delta_rp = take(routed_small ? l.esz * (size_t)l.rows_max * R : 0);
  l.Bp = take(routed_small ? sizeof(float) * (size_t)l.rows_max * N : 0);
  l.Cp = take(routed_small ? sizeof(float) * (size_t)l.rows_max * N : 0);
  l.Dpre = take(routed_small ? sizeof(float) * (size_t)l.rows_max * c.d_inner : 0);
  l.total = o;
  return l;
}

cudaError_t current_device_sm_count(int* n) {
  constexpr int kMaxDev = 64;
  static int cache[kMaxDev] = {};      // 0 = not looked up yet; every writer stores the same value for a device
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < kMaxDev && cache[dev] > 0) { *n = cache[dev]; return cudaSuccess; }
  int v = 0;
  e = cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  if (dev >= 0 && dev < kMaxDev) cache[dev] = v;
  *n = v;
  return cudaSuccess;
}

// which == 0: full layer; 1: route only; 2: scan only
int check_config(const rom_config* c, int which) {
  if (!c) return ROM_ERR_INVALID_ARG;
  if (c->dtype != ROM_F32 && c->dtype != ROM_BF16) return ROM_ERR_INVALID_ARG;
  if (c->B < 1 || c->L < 1) return ROM_ERR_INVALID_ARG;
  if ((c->flags & ~(ROM_FLAG_SIMT_GEMM | ROM_FLAG_DEBUG_CHECKS | ROM_FLAG_TEST_STALL | ROM_FLAG_FUSED_SMALL)) != 0) return ROM_ERR_INVALID_ARG;
  if (which != 2) {
    if (c->E < 1 || c->K < 1 || c->K > c->E) return ROM_ERR_INVALID_ARG;
    if (c->E > kMaxE || c->K > kMaxK) return ROM_ERR_UNSUPPORTED;
    if (c->gate_mode != 0 && c->gate_mode != 1) return ROM_ERR_INVALID_ARG;
    if (c->d_model < 64 || c->d_model % 64 != 0) return ROM_ERR_INVALID_ARG;
    if ((int64_t)c->B * c->L * c->K >= (int64_t)1 << 30) return ROM_ERR_UNSUPPORTED;
    if (c->small_proj_experts != 0 && c->small_proj_experts != 1 && c->small_proj_experts != c->E) return ROM_ERR_INVALID_ARG;
  } else if (c->small_proj_experts < 0) {
    return ROM_ERR_INVALID_ARG;
  }
  if (which != 1) {
    if (c->d_inner < 64 || c->d_inner % 64 != 0) return ROM_ERR_INVALID_ARG;
    if (c->d_state < 1) return ROM_ERR_INVALID_ARG;
    if (c->d_state != 16) return ROM_ERR_UNSUPPORTED;
    if (c->disc_mode != 0 && c->disc_mode != 1) return ROM_ERR_INVALID_ARG;
    if ((int64_t)c->B * c->L >= (int64_t)1 << 30) return ROM_ERR_UNSUPPORTED;
    if (c->B > 65535) return ROM_ERR_UNSUPPORTED;
  }
  if (which == 0) {
    if (c->d_conv < 2 || c->d_conv > 4) return c->d_conv < 1 ? ROM_ERR_INVALID_ARG : ROM_ERR_UNSUPPORTED;
    if (c->dt_rank < 1) return ROM_ERR_INVALID_ARG;
    if (c->dtype == ROM_BF16 && c->dt_rank % 16 != 0) return ROM_ERR_UNSUPPORTED;
    if (c->dtype == ROM_F32 && c->dt_rank % 4 != 0) return ROM_ERR_UNSUPPORTED;
  }
  return ROM_OK;
}

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

int check_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return ROM_ERR_CUDA;
  int major = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return ROM_ERR_CUDA;
  return major == 10 ? ROM_OK : ROM_ERR_ARCH;
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

int rom_workspace_size(const rom_config* cfg, size_t* bytes) {
  if (!bytes) return ROM_ERR_INVALID_ARG;
  // the layout is a function of the sizes only; fields a partial entry point ignores may be 0
  if (!cfg || cfg->B < 1 || cfg->L < 1 || cfg->E < 1 || cfg->K < 1 || cfg->d_model < 0 || cfg->d_inner < 0 ||
      cfg->dt_rank < 0 || cfg->d_state < 0 || (cfg->dtype != ROM_F32 && cfg->dtype != ROM_BF16))
    return ROM_ERR_INVALID_ARG;
  *bytes = make_layout(*cfg).total;
  return ROM_OK;
}

int rom_scan_workspace_size(const rom_config* cfg, size_t* bytes) {
  if (!bytes) return ROM_ERR_INVALID_ARG;
  const int rc = check_config(cfg, 2);
  if (rc != ROM_OK) return rc;
  *bytes = align_up(sizeof(float) * scan_ws_floats(cfg->B, cfg->d_inner, cfg->L), 256);
  return ROM_OK;
}

int rom_workspace_find(const rom_config* cfg, const char* name, size_t* offset, size_t* bytes) {
  if (!cfg || !name || !offset || !bytes) return ROM_ERR_INVALID_ARG;
  const WsLayout l = make_layout(*cfg);
  struct Item { const char* n; size_t off, sz; };
  const Item items[] = {
      {"U", l.U, l.esz * (size_t)l.T * cfg->d_inner},
      {"delta_r", l.delta_r, l.esz * (size_t)l.T * cfg->dt_rank},
      {"Bm", l.Bm, sizeof(float) * (size_t)l.T * cfg->d_state},
      {"Cm", l.Cm, sizeof(float) * (size_t)l.T * cfg->d_state},
      {"Delta", l.Delta, l.esz * (size_t)l.T * cfg->d_inner},
      {"row_of_assign", l.row_of_assign, sizeof(int32_t) * (size_t)l.A},
      {"XZp", l.XZp, l.esz * (size_t)l.rows_max * 2 * cfg->d_inner},
      {"Ygp", l.Ygp, l.esz * (size_t)l.rows_max * cfg->d_inner},
      {"pad_offsets", l.pad_offsets, sizeof(int32_t) * (size_t)(cfg->E + 1)},
  };
  for (const Item& it : items)
    if (std::strcmp(it.n, name) == 0) { *offset = it.off; *bytes = it.sz; return ROM_OK; }
  return ROM_ERR_INVALID_ARG;
}

int rom_route(const rom_config* cfg, const void* x, const void* W_r, const float* b_r, int32_t* topk_idx, float* gates,
              int32_t* counts, int32_t* offsets, int32_t* perm, int32_t* inv_perm, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_config(cfg, 1);
  if (rc != ROM_OK) return rc;
  if (!x || !W_r || !ws) return ROM_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(W_r) || !aligned16(ws)) return ROM_ERR_INVALID_ARG;
  const WsLayout lay = make_layout(*cfg);
  if (ws_bytes < lay.total) return ROM_ERR_WORKSPACE;
  if ((rc = check_device()) != ROM_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  LaunchCounter::count = 0;
  ROM_CUDA(cudaMemsetAsync(static_cast<char*>(ws) + lay.status, 0, sizeof(int32_t) * kStatusInts, st));
  ROM_CUDA(launch_route(*cfg, x, W_r, b_r, topk_idx, gates, counts, offsets, perm, inv_perm, static_cast<char*>(ws), lay, st));
  return ROM_OK;
}

int rom_route_balance(const rom_config* cfg, const void* x, const void* W_r, const float* b_r, float alpha, float* F, float* Pbar,
                      float* loss, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_config(cfg, 1);
  if (rc != ROM_OK) return rc;
  if (!x || !W_r || !ws) return ROM_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(W_r) || !aligned16(ws)) return ROM_ERR_INVALID_ARG;
  const WsLayout lay = make_layout(*cfg);
  if (ws_bytes < lay.total) return ROM_ERR_WORKSPACE;
  if ((rc = check_device()) != ROM_OK) return rc;
  LaunchCounter::count = 0;
  ROM_CUDA(cudaMemsetAsync(static_cast<char*>(ws) + lay.status, 0, sizeof(int32_t) * kStatusInts, static_cast<cudaStream_t>(stream)));
  ROM_CUDA(launch_balance(*cfg, x, W_r, b_r, alpha, F, Pbar, loss, static_cast<char*>(ws), lay, static_cast<cudaStream_t>(stream)));
  return ROM_OK;
}

int rom_scan(const rom_config* cfg, const void* u, const float* delta, const float* A, const float* Bm, const float* Cm,
             const float* D, const void* z, const float* h0, void* y, float* h_last, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_config(cfg, 2);
  if (rc != ROM_OK) return rc;
  if (!u || !delta || !A || !Bm || !Cm || !y) return ROM_ERR_INVALID_ARG;
  if (!aligned16(u) || !aligned16(delta) || !aligned16(A) || !aligned16(Bm) || !aligned16(Cm) || !aligned16(y) ||
      (z && !aligned16(z)))
    return ROM_ERR_INVALID_ARG;
  if ((rc = check_device()) != ROM_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  LaunchCounter::count = 0;
  // with a workspace of rom_scan_workspace_size bytes a long sequence is scanned in parallel chunks; without one, in one pass
  float* chunk_ws = nullptr;
  if (ws != nullptr) {
    if (!aligned16(ws)) return ROM_ERR_INVALID_ARG;
    if (ws_bytes < sizeof(float) * scan_ws_floats(cfg->B, cfg->d_inner, cfg->L)) return ROM_ERR_WORKSPACE;
    chunk_ws = static_cast<float*>(ws);
  }
  ROM_CUDA(launch_scan(*cfg, u, delta, true, A, Bm, Cm, D, z, cfg->d_inner, nullptr, h0, y, h_last, nullptr, 1, chunk_ws, false, st));
  return ROM_OK;
}

int rom_scan_backward_workspace_size(const rom_config* cfg, size_t* bytes) {
  if (!bytes) return ROM_ERR_INVALID_ARG;
  const int rc = check_config(cfg, 2);
  if (rc != ROM_OK) return rc;
  *bytes = scan_bwd_ws_bytes(cfg->B, cfg->d_inner, cfg->L);
  return ROM_OK;
}

int rom_scan_backward(const rom_config* cfg, const void* dy, const void* u, const float* delta, const float* A, const float* Bm,
                      const float* Cm, const float* D, const void* z, const float* h0, const float* dh_last, void* du,
                      float* ddelta, float* dA, float* dBm, float* dCm, float* dD, void* dz, float* dh0, void* ws, size_t ws_bytes,
                      void* stream) {
  int rc = check_config(cfg, 2);
  if (rc != ROM_OK) return rc;
  if (!dy || !u || !delta || !A || !Bm || !Cm || !du || !ddelta || !dA || !dBm || !dCm || !ws) return ROM_ERR_INVALID_ARG;
  if ((D == nullptr) != (dD == nullptr) || (z == nullptr) != (dz == nullptr)) return ROM_ERR_INVALID_ARG;
  const void* ptrs[] = {dy, u, delta, A, Bm, Cm, du, ddelta, dA, dBm, dCm, ws, z, dz, h0, dh_last, dh0};
  for (const void* p : ptrs)
    if (p && !aligned16(p)) return ROM_ERR_INVALID_ARG;
  if (ws_bytes < scan_bwd_ws_bytes(cfg->B, cfg->d_inner, cfg->L)) return ROM_ERR_WORKSPACE;
  if ((rc = check_device()) != ROM_OK) return rc;
  LaunchCounter::count = 0;
  ROM_CUDA(launch_scan_backward(*cfg, dy, u, delta, A, Bm, Cm, D, z, h0, dh_last, du, ddelta, dA, dBm, dCm, dD, dz, dh0,
                                static_cast<float*>(ws), cfg->d_inner, static_cast<cudaStream_t>(stream)));
  return ROM_OK;
}

}  // extern "C"

namespace rom {
namespace {

constexpr int kNumStages = 9;
const char* const kStageNames[kNumStages] = {"route", "gather", "in_proj", "conv", "x_proj", "dt_proj", "scan", "out_proj", "combine"};

// ev == nullptr: plain launch sequence.  Otherwise ev[0] is recorded before the first stage and
// ev[i+1] after stage i (kNumStages + 1 events).
// conv_state / ssm_state (both or neither): single-token step, L == 1, states read and advanced in place.
int layer_forward_impl(const rom_config* cfg, const rom_weights* w, const void* x, void* out, int32_t* topk_idx_out,
                       float* gates_out, int32_t* counts_out, void* ws, size_t ws_bytes, void* stream, cudaEvent_t* ev,
                       float* conv_state = nullptr, float* ssm_state = nullptr) {
  int rc = check_config(cfg, 0);
  if (rc != ROM_OK) return rc;
  if ((conv_state == nullptr) != (ssm_state == nullptr)) return ROM_ERR_INVALID_ARG;
  if (conv_state && (cfg->L != 1 || !aligned16(conv_state) || !aligned16(ssm_state))) return ROM_ERR_INVALID_ARG;
  if (!w || !x || !out || !ws) return ROM_ERR_INVALID_ARG;
  if (!w->W_r || !w->W_inz || !w->w_conv || !w->W_x || !w->W_dt || !w->A || !w->W_out) return ROM_ERR_INVALID_ARG;
  const void* ptrs[] = {x, out, ws, w->W_r, w->W_inz, w->w_conv, w->W_x, w->W_dt, w->A, w->W_out};
  for (const void* p : ptrs)
    if (!aligned16(p)) return ROM_ERR_INVALID_ARG;
  const rom_config& c = *cfg;
  const WsLayout lay = make_layout(c);
  if (ws_bytes < lay.total) return ROM_ERR_WORKSPACE;
  if ((rc = check_device()) != ROM_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* W = static_cast<char*>(ws);
  LaunchCounter::count = 0;

  const int T = (int)lay.T, De = c.d_inner, Dm = c.d_model, R = c.dt_rank, N = c.d_state;
  const bool tc = c.dtype == ROM_BF16 && !(c.flags & ROM_FLAG_SIMT_GEMM);
  int32_t* status = reinterpret_cast<int32_t*>(W + lay.status);
  int32_t* tile_expert = reinterpret_cast<int32_t*>(W + lay.tile_expert);
  int32_t* num_m_tiles = reinterpret_cast<int32_t*>(W + lay.num_m_tiles);
  int32_t* row_of_assign = reinterpret_cast<int32_t*>(W + lay.row_of_assign);
  float* gates = gates_out ? gates_out : reinterpret_cast<float*>(W + lay.gates);

  int stage = 0;
#define ROM_STAGE_DONE()                                       \
  do {                                                         \
    if (ev) ROM_CUDA(cudaEventRecord(ev[++stage], st));        \
  } while (0)
  if (ev) ROM_CUDA(cudaEventRecord(ev[0], st));
  ROM_CUDA(cudaMemsetAsync(status, 0, sizeof(int32_t) * kStatusInts, st));
  const bool debug_checks = (c.flags & ROM_FLAG_DEBUG_CHECKS) != 0;
  if (debug_checks) ROM_CUDA(launch_canaries(W, lay, false, st));
  // S1 + S2: router, top-K, permutation tables
  // ... and the token rows gathered into padded expert order (the second of the two launches copies them)
  ROM_CUDA(launch_route_gather(c, x, w->W_r, w->b_r, topk_idx_out, gates, counts_out, W, lay, st));
  if (debug_checks) ROM_CUDA(launch_check_tables(c, W, lay, st));
  ROM_STAGE_DONE();
  ROM_STAGE_DONE();      // "gather": fused into the routing launches

  auto gemm = [&](const void* A_, int lda, const void* B_, int ldb, int n_experts, int64_t bstride, int M_max, int Nn, int Kd,
                  const int32_t* te, const int32_t* nmt, const Epilogue& ep) -> cudaError_t {
    // a handful of rows against a long K (the x Proj of a single-token step): one 128-row tensor tile would be walked by a
    // single CTA; the lane-split kernel spreads it over the GPU
    if (!te && M_max <= 128 && Kd >= 1024 && Kd % 2048 == 0 && ep.mode == EPI_XPROJ)
      return launch_gemm_skinny(c.dtype, A_, lda, B_, ldb, M_max, Nn, Kd, ep, st);
    if (tc) return launch_gemm_tc(A_, lda, B_, ldb, n_experts, M_max, Nn, Kd, te, nmt, ep, status, st,
                                  (c.flags & ROM_FLAG_TEST_STALL) != 0 && (ep.mode == EPI_INPROJ || (ep.mode == EPI_STORE && Nn == 2 * De)));
    return launch_gemm_simt(c.dtype, A_, lda, B_, ldb, bstride, M_max, Nn, Kd, te, nmt, ep, st);
  };

  // S3: grouped [Conv Proj | Gate Proj]
  // K = 1: the Gate Proj half is stored activated (SiLU); K > 1: raw, the activation follows the sum over slots in S4
  // Tensor path with one expert per token: the epilogue also puts every row back at its token's position, so the
  // conv and the scan read H and the gate without indirection.
  const bool in_token_order = tc && c.K == 1;
  Epilogue e_in{c.K == 1 ? EPI_INPROJ : EPI_STORE, W + lay.XZp, 2 * De, nullptr, nullptr, nullptr, De, 0,
                in_token_order ? reinterpret_cast<const int32_t*>(W + lay.assign_of_row) : nullptr, nullptr};
  ROM_CUDA(gemm(W + lay.x_perm, Dm, w->W_inz, Dm, c.E, (int64_t)2 * De * Dm, (int)lay.rows_max, 2 * De, Dm, tile_expert, num_m_tiles, e_in));
  ROM_STAGE_DONE();
  // S4 + S5 + S6 as one kernel (opt-in): tensor path, top-1 (rows already in token order), shared x Proj / dt Proj
  const bool fused_small = in_token_order && !conv_state && c.small_proj_experts <= 1 && (c.flags & ROM_FLAG_FUSED_SMALL) &&
                           fused_conv_xdt_supported(c);
  if (fused_small) {
    ROM_CUDA(launch_fused_conv_xdt(c, W + lay.XZp, 2 * De, w->w_conv, w->b_conv, w->W_x, w->W_dt, w->b_dt, W + lay.U, W + lay.delta_r,
                                   reinterpret_cast<float*>(W + lay.Bm), reinterpret_cast<float*>(W + lay.Cm), W + lay.Delta, status, st));
    ROM_STAGE_DONE();      // "conv": the fused kernel's time is reported here
    ROM_STAGE_DONE();      // "x_proj"
    ROM_STAGE_DONE();      // "dt_proj"
  } else {
  // S4: un-permute + sum over selected experts + conv + SiLU
  if (conv_state)
    ROM_CUDA(launch_conv_step(c, W + lay.XZp, in_token_order ? nullptr : row_of_assign, w->w_conv, w->b_conv, conv_state, W + lay.U,
                              c.K > 1 ? W + lay.Zs : nullptr, st));
  else
    ROM_CUDA(launch_conv(c, W + lay.XZp, in_token_order ? nullptr : row_of_assign, w->w_conv, w->b_conv, W + lay.U, c.K > 1 ? W + lay.Zs : nullptr, st));
  ROM_STAGE_DONE();
  if (c.small_proj_experts <= 1) {
    // S5: x Proj -> delta_r | B | C  (shared by all experts)
    Epilogue e_x{EPI_XPROJ, W + lay.delta_r, R, reinterpret_cast<float*>(W + lay.Bm), reinterpret_cast<float*>(W + lay.Cm), nullptr, R, N, nullptr, nullptr};
    ROM_CUDA(gemm(W + lay.U, De, w->W_x, De, 1, 0, T, R + 2 * N, De, nullptr, nullptr, e_x));
    ROM_STAGE_DONE();
    // S6: dt Proj + softplus
    Epilogue e_dt{EPI_SOFTPLUS, W + lay.Delta, De, nullptr, nullptr, w->b_dt, 0, 0, nullptr, nullptr};
    ROM_CUDA(gemm(W + lay.delta_r, R, w->W_dt, R, 1, 0, T, De, R, nullptr, nullptr, e_dt));
    ROM_STAGE_DONE();
  } else {
    // Per-expert x Proj / dt Proj under the same routing: U rows gathered into expert order (in the buffer the
    // scan fills later), two more grouped GEMMs over the existing row tiles, then the sum over the K slots.
    ROM_CUDA(launch_gather_rows_to(c, W + lay.U, W + lay.Ygp, De, W, lay, st));
    if (tc && c.K == 1) {
      // one expert per token on the tensor path: nothing to sum over slots, so the output ops put B, C and Delta
      // (bias + softplus applied) straight at the token's row; only delta_r stays in expert order for the dt Proj
      const int32_t* row_token = reinterpret_cast<const int32_t*>(W + lay.assign_of_row);
      Epilogue e_x{EPI_XPROJ, W + lay.delta_rp, R, reinterpret_cast<float*>(W + lay.Bm), reinterpret_cast<float*>(W + lay.Cm), nullptr, R, N, row_token, nullptr};
      ROM_CUDA(gemm(W + lay.Ygp, De, w->W_x, De, c.E, (int64_t)(R + 2 * N) * De, (int)lay.rows_max, R + 2 * N, De, tile_expert, num_m_tiles, e_x));
      ROM_STAGE_DONE();
      Epilogue e_dt{EPI_SOFTPLUS_ROWS, W + lay.Delta, De, nullptr, nullptr, w->b_dt, 0, 0, row_token, nullptr};
      ROM_CUDA(gemm(W + lay.delta_rp, R, w->W_dt, R, c.E, (int64_t)De * R, (int)lay.rows_max, De, R, tile_expert, num_m_tiles, e_dt));
      ROM_STAGE_DONE();
    } else {
      Epilogue e_x{EPI_XPROJ, W + lay.delta_rp, R, reinterpret_cast<float*>(W + lay.Bp), reinterpret_cast<float*>(W + lay.Cp), nullptr, R, N, nullptr, nullptr};
      ROM_CUDA(gemm(W + lay.Ygp, De, w->W_x, De, c.E, (int64_t)(R + 2 * N) * De, (int)lay.rows_max, R + 2 * N, De, tile_expert, num_m_tiles, e_x));
      ROM_STAGE_DONE();
      Epilogue e_dt{EPI_F32, W + lay.Dpre, De, nullptr, nullptr, nullptr, 0, 0, nullptr, nullptr};
      ROM_CUDA(gemm(W + lay.delta_rp, R, w->W_dt, R, c.E, (int64_t)De * R, (int)lay.rows_max, De, R, tile_expert, num_m_tiles, e_dt));
      ROM_CUDA(launch_small_combine(c, reinterpret_cast<float*>(W + lay.Bp), reinterpret_cast<float*>(W + lay.Cp),
                                    reinterpret_cast<float*>(W + lay.Dpre), row_of_assign, w->b_dt, reinterpret_cast<float*>(W + lay.Bm),
                                    reinterpret_cast<float*>(W + lay.Cm), W + lay.Delta, st));
      ROM_STAGE_DONE();
    }
  }
  }      // !fused_small
  // S7 + S8 + S9: scan, gate, re-permute
  // K = 1: the gate row of a token is its Gate Proj row in expert order; K > 1: the summed rows from S4
  const char* zbase = c.K == 1 ? W + lay.XZp + (size_t)De * lay.esz : W + lay.Zs;
  ROM_CUDA(launch_scan(c, W + lay.U, W + lay.Delta, false, w->A, reinterpret_cast<float*>(W + lay.Bm),
                       reinterpret_cast<float*>(W + lay.Cm), w->D, zbase, c.K == 1 ? 2 * De : De, (c.K == 1 && !in_token_order) ? row_of_assign : nullptr,
                       ssm_state, W + lay.Ygp, ssm_state, row_of_assign, c.K, reinterpret_cast<float*>(W + lay.scan_ws), true, st));
  ROM_STAGE_DONE();
  // S10 + S11.  Tensor path with one expert per token: the epilogue of the grouped Out Proj scales each row by
  // its gate and writes it at its token's position (no intermediate rows, no combine pass).  Otherwise: grouped
  // Out Proj into expert-order rows, then the gate-weighted sum over the K slots.
  const bool fused_out = tc && c.K == 1;
  if (fused_out) {
    Epilogue e_out{EPI_OUTPROJ, out, Dm, nullptr, nullptr, nullptr, 0, 0, reinterpret_cast<const int32_t*>(W + lay.assign_of_row), gates};
    ROM_CUDA(gemm(W + lay.Ygp, De, w->W_out, De, c.E, (int64_t)Dm * De, (int)lay.rows_max, Dm, De, tile_expert, num_m_tiles, e_out));
    ROM_STAGE_DONE();
    ROM_STAGE_DONE();
  } else {
    Epilogue e_out{EPI_STORE, W + lay.Op, Dm, nullptr, nullptr, nullptr, 0, 0, nullptr, nullptr};
    ROM_CUDA(gemm(W + lay.Ygp, De, w->W_out, De, c.E, (int64_t)Dm * De, (int)lay.rows_max, Dm, De, tile_expert, num_m_tiles, e_out));
    ROM_STAGE_DONE();
    ROM_CUDA(launch_combine(c, W + lay.Op, row_of_assign, gates, out, st));
    ROM_STAGE_DONE();
  }
#undef ROM_STAGE_DONE
  if (debug_checks) ROM_CUDA(launch_canaries(W, lay, true, st));
  return ROM_OK;
}

}  // namespace
}  // namespace rom

namespace rom {
namespace {

// Scratch of rom_layer_backward: the forward workspace (routing tables and recomputed activations) followed by the
// gradient buffers and the transposed weights.
struct BwdLayout {
  size_t HZs, D32, dOp, dYgu, dYg, rowscale, dgate, dU1, ddelta, dBm, dCm, dpre, dxdbl, dU2, dHZs, dHZp, dxp, dlogit;
  size_t WoT, WiT, WdtT, WxT, ckpt, Xt, Yt, total;
};
BwdLayout make_bwd_layout(const rom_config& c, const WsLayout& l) {
  BwdLayout b{};
  size_t o = align_up(l.total, 256);
  auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
  const size_t T = (size_t)l.T, rows = (size_t)l.rows_max, De = c.d_inner, Dm = c.d_model, N = c.d_state, R = c.dt_rank, esz = l.esz;
  b.HZs = take(esz * T * 2 * De);
  b.D32 = take(4 * T * De);
  b.dOp = take(esz * rows * Dm);
  b.dYgu = take(esz * rows * De);
  b.dYg = take(esz * T * De);
  b.rowscale = take(4 * rows);
  b.dgate = take(4 * T * c.K);
  b.dU1 = take(esz * T * De);
  b.ddelta = take(4 * T * De);
  b.dBm = take(4 * T * N);
  b.dCm = take(4 * T * N);
  b.dpre = take(esz * T * De);
  b.dxdbl = take(esz * T * (R + 2 * N));
  b.dU2 = take(esz * T * De);
  b.dHZs = take(esz * T * 2 * De);
  b.dHZp = take(esz * rows * 2 * De);
  b.dxp = take(esz * rows * Dm);
  b.dlogit = take(4 * T * c.E);
  b.WoT = take(esz * (size_t)c.E * De * Dm);
  b.WiT = take(esz * (size_t)c.E * Dm * 2 * De);
  b.WdtT = take(esz * R * De);
  b.WxT = take(esz * De * (R + 2 * N));
  b.ckpt = take(scan_bwd_ws_bytes(c.B, c.d_inner, c.L));
  // tensor path: the activations of the two grouped weight gradients, transposed (token rows contiguous)
  const bool tcw = c.dtype == ROM_BF16 && !(c.flags & ROM_FLAG_SIMT_GEMM);
  b.Xt = take(tcw ? esz * 2 * De * rows : 0);
  b.Yt = take(tcw ? esz * (De > Dm ? De : Dm) * rows : 0);
  b.total = o;
  return b;
}

}  // namespace
}  // namespace rom

extern "C" {

int rom_layer_backward_workspace_size(const rom_config* cfg, size_t* bytes) {
  if (!bytes) return ROM_ERR_INVALID_ARG;
  const int rc = check_config(cfg, 0);
  if (rc != ROM_OK) return rc;
  *bytes = make_bwd_layout(*cfg, make_layout(*cfg)).total;
  return ROM_OK;
}

int rom_layer_backward(const rom_config* cfg, const rom_weights* w, const void* x, const void* dout, void* dx, const rom_grads* g,
                       void* ws, size_t ws_bytes, void* stream) {
  int rc = check_config(cfg, 0);
  if (rc != ROM_OK) return rc;
  if (cfg->small_proj_experts > 1) return ROM_ERR_UNSUPPORTED;      // only the shared x Proj / dt Proj wiring is differentiated
  if (!w || !x || !dout || !dx || !g || !ws) return ROM_ERR_INVALID_ARG;
  if (!w->W_r || !w->W_inz || !w->w_conv || !w->W_x || !w->W_dt || !w->A || !w->W_out) return ROM_ERR_INVALID_ARG;
  if (!g->dW_r || !g->dW_inz || !g->dw_conv || !g->db_conv || !g->dW_x || !g->dW_dt || !g->db_dt || !g->dA || !g->dW_out) return ROM_ERR_INVALID_ARG;
  if ((w->D == nullptr) != (g->dD == nullptr)) return ROM_ERR_INVALID_ARG;
  const void* ptrs[] = {x, dout, dx, ws, w->W_r, w->W_inz, w->w_conv, w->W_x, w->W_dt, w->A, w->W_out, g->dW_r, g->dW_inz, g->dw_conv,
                        g->db_conv, g->dW_x, g->dW_dt, g->db_dt, g->dA, g->dW_out};
  for (const void* p : ptrs)
    if (!aligned16(p)) return ROM_ERR_INVALID_ARG;
  const rom_config& c = *cfg;
  const WsLayout lay = make_layout(c);
  const BwdLayout bl = make_bwd_layout(c, lay);
  if (ws_bytes < bl.total) return ROM_ERR_WORKSPACE;
  if ((rc = check_device()) != ROM_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* W = static_cast<char*>(ws);
  LaunchCounter::count = 0;

  const int T = (int)lay.T, De = c.d_inner, Dm = c.d_model, R = c.dt_rank, N = c.d_state, rows = (int)lay.rows_max;
  const size_t esz = lay.esz;
  const bool tc = c.dtype == ROM_BF16 && !(c.flags & ROM_FLAG_SIMT_GEMM);
  int32_t* status = reinterpret_cast<int32_t*>(W + lay.status);
  const int32_t* tile_expert = reinterpret_cast<int32_t*>(W + lay.tile_expert);
  const int32_t* num_m_tiles = reinterpret_cast<int32_t*>(W + lay.num_m_tiles);
  const int32_t* row_of_assign = reinterpret_cast<int32_t*>(W + lay.row_of_assign);
  const int32_t* pad_offsets = reinterpret_cast<int32_t*>(W + lay.pad_offsets);
  float* gates = reinterpret_cast<float*>(W + lay.gates);
  float* Bm = reinterpret_cast<float*>(W + lay.Bm);
  float* Cm = reinterpret_cast<float*>(W + lay.Cm);
  auto gemm = [&](const void* A_, int lda, const void* B_, int ldb, int n_experts, int64_t bstride, int M_max, int Nn, int Kd,
                  const int32_t* te, const int32_t* nmt, const Epilogue& ep) -> cudaError_t {
    if (tc) return launch_gemm_tc(A_, lda, B_, ldb, n_experts, M_max, Nn, Kd, te, nmt, ep, status, st);
    return launch_gemm_simt(c.dtype, A_, lda, B_, ldb, bstride, M_max, Nn, Kd, te, nmt, ep, st);
  };
  auto store_to = [&](void* C_, int ldc) { return Epilogue{EPI_STORE, C_, ldc, nullptr, nullptr, nullptr, 0, 0, nullptr, nullptr}; };

  // ---- forward, recomputed with the raw Gate Proj rows kept (the forward proper stores them activated at top-1)
  ROM_CUDA(cudaMemsetAsync(status, 0, sizeof(int32_t) * kStatusInts, st));
  ROM_CUDA(launch_route_gather(c, x, w->W_r, w->b_r, nullptr, gates, nullptr, W, lay, st));
  ROM_CUDA(gemm(W + lay.x_perm, Dm, w->W_inz, Dm, c.E, (int64_t)2 * De * Dm, rows, 2 * De, Dm, tile_expert, num_m_tiles, store_to(W + lay.XZp, 2 * De)));
  ROM_CUDA(launch_slot_sum(c.dtype, W + lay.XZp, row_of_assign, W + bl.HZs, T, 2 * De, c.K, st));       // H_t, Z_t: sums over the selected experts
  rom_config c1 = c;
  c1.K = 1;
  ROM_CUDA(launch_conv(c1, W + bl.HZs, nullptr, w->w_conv, w->b_conv, W + lay.U, nullptr, st));
  Epilogue e_x{EPI_XPROJ, W + lay.delta_r, R, Bm, Cm, nullptr, R, N, nullptr, nullptr};
  ROM_CUDA(gemm(W + lay.U, De, w->W_x, De, 1, 0, T, R + 2 * N, De, nullptr, nullptr, e_x));
  Epilogue e_dt{EPI_SOFTPLUS, W + lay.Delta, De, nullptr, nullptr, w->b_dt, 0, 0, nullptr, nullptr};
  ROM_CUDA(gemm(W + lay.delta_r, R, w->W_dt, R, 1, 0, T, De, R, nullptr, nullptr, e_dt));
  float* D32 = reinterpret_cast<float*>(W + bl.D32);
  ROM_CUDA(launch_cast_f32(c.dtype, W + lay.Delta, D32, (long long)T * De, st));
  // gated scan output in expert order (operand of the Out Proj weight gradient); padding rows must be zero
  ROM_CUDA(cudaMemsetAsync(W + lay.Ygp, 0, esz * (size_t)rows * De, st));
  const char* zraw = W + bl.HZs + (size_t)De * esz;
  ROM_CUDA(launch_scan(c, W + lay.U, W + lay.Delta, false, w->A, Bm, Cm, w->D, zraw, 2 * De, nullptr, nullptr, W + lay.Ygp, nullptr,
                       row_of_assign, c.K, reinterpret_cast<float*>(W + lay.scan_ws), false, st));

  // ---- Out Proj and combine, reversed: back_k = dO_t W_out,k; dYg, dgate; dW_out
  ROM_CUDA(launch_gather_rows_to(c, dout, W + bl.dOp, Dm, W, lay, st));
  ROM_CUDA(launch_transpose(c.dtype, w->W_out, W + bl.WoT, c.E, Dm, De, st));
  ROM_CUDA(gemm(W + bl.dOp, Dm, W + bl.WoT, Dm, c.E, (int64_t)De * Dm, rows, De, Dm, tile_expert, num_m_tiles, store_to(W + bl.dYgu, De)));
  float* rowscale = reinterpret_cast<float*>(W + bl.rowscale);
  float* dgate = reinterpret_cast<float*>(W + bl.dgate);
  ROM_CUDA(cudaMemsetAsync(rowscale, 0, sizeof(float) * rows, st));
  ROM_CUDA(launch_combine_bwd(c.dtype, W + bl.dYgu, W + lay.Ygp, row_of_assign, gates, W + bl.dYg, dgate, rowscale, T, De, c.K, st));
  // grouped weight gradient (a sum over each expert's row segment): tensor path = the grouped GEMM over transposed
  // activations with per-expert K ranges; otherwise the plain fp32-FMA kernel
  auto grouped_wgrad = [&](const void* X, int P, const void* Y, int Q, const float* scale, float* C) -> cudaError_t {
    if (!tc) return launch_wgrad(c.dtype, X, P, Y, Q, scale, pad_offsets, c.E, rows, P, Q, C, st);
    cudaError_t e = launch_transpose_scaled(c.dtype, X, W + bl.Xt, rows, P, rows, scale, st);
    if (e == cudaSuccess) e = launch_transpose_scaled(c.dtype, Y, W + bl.Yt, rows, Q, rows, nullptr, st);
    if (e == cudaSuccess) e = launch_gemm_tc_wgrad(W + bl.Xt, W + bl.Yt, rows, pad_offsets, c.E, P, Q, C, status, st);
    return e;
  };
  ROM_CUDA(grouped_wgrad(W + bl.dOp, Dm, W + lay.Ygp, De, rowscale, g->dW_out));

  // ---- gate and scan, reversed
  float* ddelta = reinterpret_cast<float*>(W + bl.ddelta);
  float* dBm = reinterpret_cast<float*>(W + bl.dBm);
  float* dCm = reinterpret_cast<float*>(W + bl.dCm);
  ROM_CUDA(launch_scan_backward(c, W + bl.dYg, W + lay.U, D32, w->A, Bm, Cm, w->D, zraw, nullptr, nullptr, W + bl.dU1, ddelta, g->dA, dBm, dCm,
                                g->dD, W + bl.dHZs + (size_t)De * esz, nullptr, reinterpret_cast<float*>(W + bl.ckpt), 2 * De, st));

  // ---- dt Proj and x Proj, reversed
  ROM_CUDA(cudaMemsetAsync(g->db_dt, 0, sizeof(float) * De, st));
  ROM_CUDA(launch_softplus_bwd(c.dtype, ddelta, D32, W + bl.dpre, g->db_dt, T, De, st));
  ROM_CUDA(launch_transpose(c.dtype, w->W_dt, W + bl.WdtT, 1, De, R, st));
  ROM_CUDA(gemm(W + bl.dpre, De, W + bl.WdtT, De, 1, 0, T, R, De, nullptr, nullptr, store_to(W + bl.dxdbl, R + 2 * N)));      // d(delta) into columns [0, R)
  // weight gradient of a shared projection (a sum over all tokens): tensor path = the plain GEMM over transposed
  // activations (row pitch padded to 64 tokens; the tail of the last K block is filled with zeros by the tensor map)
  const int Tp = (int)align_up((size_t)T, 64);
  auto shared_wgrad = [&](const void* X, int P, const void* Y, int Q, float* C) -> cudaError_t {
    if (!tc) return launch_wgrad(c.dtype, X, P, Y, Q, nullptr, nullptr, 1, T, P, Q, C, st);
    cudaError_t e = launch_transpose_scaled(c.dtype, X, W + bl.Xt, T, P, Tp, nullptr, st);
    if (e == cudaSuccess) e = launch_transpose_scaled(c.dtype, Y, W + bl.Yt, T, Q, Tp, nullptr, st);
    if (e == cudaSuccess) e = launch_gemm_tc(W + bl.Xt, Tp, W + bl.Yt, Tp, 1, P, Q, T, nullptr, nullptr,
                                             Epilogue{EPI_F32, C, Q, nullptr, nullptr, nullptr, 0, 0, nullptr, nullptr}, status, st);
    return e;
  };
  ROM_CUDA(shared_wgrad(W + bl.dpre, De, W + lay.delta_r, R, g->dW_dt));
  ROM_CUDA(launch_pack_bc(c.dtype, dBm, dCm, W + bl.dxdbl, T, R, N, st));
  ROM_CUDA(launch_transpose(c.dtype, w->W_x, W + bl.WxT, 1, R + 2 * N, De, st));
  ROM_CUDA(gemm(W + bl.dxdbl, R + 2 * N, W + bl.WxT, R + 2 * N, 1, 0, T, De, R + 2 * N, nullptr, nullptr, store_to(W + bl.dU2, De)));
  ROM_CUDA(shared_wgrad(W + bl.dxdbl, R + 2 * N, W + lay.U, De, g->dW_x));

  // ---- conv, reversed (dU = scan part + x Proj part)
  ROM_CUDA(cudaMemsetAsync(g->dw_conv, 0, sizeof(float) * (size_t)c.d_conv * De, st));
  ROM_CUDA(cudaMemsetAsync(g->db_conv, 0, sizeof(float) * De, st));
  ROM_CUDA(launch_conv_bwd(c, W + bl.HZs, w->w_conv, w->b_conv, W + bl.dU1, W + bl.dU2, W + bl.dHZs, g->dw_conv, g->db_conv, st));

  // ---- Conv Proj | Gate Proj, reversed: every selected expert of a token receives the token's (dH, dZ)
  ROM_CUDA(launch_gather_rows_to(c, W + bl.dHZs, W + bl.dHZp, 2 * De, W, lay, st));
  ROM_CUDA(launch_transpose(c.dtype, w->W_inz, W + bl.WiT, c.E, 2 * De, Dm, st));
  ROM_CUDA(gemm(W + bl.dHZp, 2 * De, W + bl.WiT, 2 * De, c.E, (int64_t)Dm * 2 * De, rows, Dm, 2 * De, tile_expert, num_m_tiles, store_to(W + bl.dxp, Dm)));
  ROM_CUDA(grouped_wgrad(W + bl.dHZp, 2 * De, W + lay.x_perm, Dm, nullptr, g->dW_inz));

  // ---- router, reversed (through the gate values only), and dx
  float* dlogit = reinterpret_cast<float*>(W + bl.dlogit);
  ROM_CUDA(cudaMemsetAsync(g->dW_r, 0, sizeof(float) * (size_t)c.E * Dm, st));
  if (g->db_r) ROM_CUDA(cudaMemsetAsync(g->db_r, 0, sizeof(float) * c.E, st));
  ROM_CUDA(launch_router_bwd(c, x, w->W_r, w->b_r, reinterpret_cast<const int32_t*>(W + lay.topk_idx), gates, dgate, dlogit, g->db_r, g->dW_r, st));
  ROM_CUDA(launch_dx(c, W + bl.dxp, row_of_assign, dlogit, w->W_r, dx, st));
  return ROM_OK;
}

int rom_layer_forward(const rom_config* cfg, const rom_weights* w, const void* x, void* out, int32_t* topk_idx_out,
                      float* gates_out, int32_t* counts_out, void* ws, size_t ws_bytes, void* stream) {
  return layer_forward_impl(cfg, w, x, out, topk_idx_out, gates_out, counts_out, ws, ws_bytes, stream, nullptr);
}

int rom_layer_forward_host(const rom_config* cfg, const rom_weights* w, const void* x_host, void* out_host, void* x_dev,
                           void* out_dev, void* ws, size_t ws_bytes, void* stream) {
  if (!cfg || !x_host || !out_host || !x_dev || !out_dev) return ROM_ERR_INVALID_ARG;
  int rc = check_config(cfg, 0);
  if (rc != ROM_OK) return rc;
  if (!ws || ws_bytes < make_layout(*cfg).total) return ws ? ROM_ERR_WORKSPACE : ROM_ERR_INVALID_ARG;
  const size_t bytes = (size_t)cfg->B * cfg->L * cfg->d_model * (cfg->dtype == ROM_BF16 ? 2 : 4);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ROM_CUDA(cudaMemcpyAsync(x_dev, x_host, bytes, cudaMemcpyHostToDevice, st));
  rc = layer_forward_impl(cfg, w, x_dev, out_dev, nullptr, nullptr, nullptr, ws, ws_bytes, stream, nullptr);
  if (rc != ROM_OK) return rc;
  ROM_CUDA(cudaMemcpyAsync(out_host, out_dev, bytes, cudaMemcpyDeviceToHost, st));
  return ROM_OK;
}

int rom_layer_step(const rom_config* cfg, const rom_weights* w, const void* x, float* conv_state, float* ssm_state, void* out,
                   int32_t* topk_idx_out, float* gates_out, void* ws, size_t ws_bytes, void* stream) {
  if (!conv_state || !ssm_state) return ROM_ERR_INVALID_ARG;
  return layer_forward_impl(cfg, w, x, out, topk_idx_out, gates_out, nullptr, ws, ws_bytes, stream, nullptr, conv_state, ssm_state);
}

int rom_layer_forward_profile(const rom_config* cfg, const rom_weights* w, const void* x, void* out, void* ws, size_t ws_bytes,
                              void* stream, float* stage_ms, int n_stage_ms) {
  if (!stage_ms || n_stage_ms < kNumStages) return ROM_ERR_INVALID_ARG;
  cudaEvent_t ev[kNumStages + 1];
  int made = 0;
  int rc = ROM_OK;
  for (; made <= kNumStages; ++made)
    if (cudaEventCreate(&ev[made]) != cudaSuccess) { rc = ROM_ERR_CUDA; break; }
  if (rc == ROM_OK) rc = layer_forward_impl(cfg, w, x, out, nullptr, nullptr, nullptr, ws, ws_bytes, stream, ev);
  if (rc == ROM_OK && cudaStreamSynchronize(static_cast<cudaStream_t>(stream)) != cudaSuccess) rc = ROM_ERR_CUDA;
  if (rc == ROM_OK)
    for (int i = 0; i < kNumStages; ++i)
      if (cudaEventElapsedTime(&stage_ms[i], ev[i], ev[i + 1]) != cudaSuccess) rc = ROM_ERR_CUDA;
  for (int i = 0; i < made; ++i) cudaEventDestroy(ev[i]);
  return rc;
}

int rom_debug_check(const rom_config* cfg, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_config(cfg, 0);
  if (rc != ROM_OK) return rc;
  if (!(cfg->flags & ROM_FLAG_DEBUG_CHECKS)) return ROM_ERR_INVALID_ARG;
  if (!ws || !aligned16(ws)) return ROM_ERR_INVALID_ARG;
  const WsLayout lay = make_layout(*cfg);
  if (ws_bytes < lay.total) return ROM_ERR_WORKSPACE;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  ROM_CUDA(launch_check_tables(*cfg, static_cast<char*>(ws), lay, st));
  ROM_CUDA(launch_canaries(static_cast<char*>(ws), lay, true, st));
  return ROM_OK;
}

int rom_num_stages(void) { return kNumStages; }

const char* rom_stage_name(int i) { return (i >= 0 && i < kNumStages) ? kStageNames[i] : ""; }

int rom_get_status(void* ws, void* stream, int32_t* host_code) {
  if (!ws || !host_code) return ROM_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int32_t v[2] = {0, 0};
  ROM_CUDA(cudaMemcpyAsync(v, ws, sizeof(v), cudaMemcpyDeviceToHost, st));
  ROM_CUDA(cudaStreamSynchronize(st));
  ROM_CUDA(cudaMemsetAsync(ws, 0, sizeof(int32_t) * kStatusInts, st));
  *host_code = v[kStatCode];      // 0, or the rom_status a kernel latched
  return ROM_OK;
}

const char* rom_status_string(int code) {
  switch (code) {
    case ROM_OK: return "ok";
    case ROM_ERR_INVALID_ARG: return "invalid argument";
    case ROM_ERR_UNSUPPORTED: return "unsupported configuration";
    case ROM_ERR_WORKSPACE: return "workspace too small";
    case ROM_ERR_CUDA: return "CUDA call failed";
    case ROM_ERR_ARCH: return "device is not sm_100";
    case ROM_ERR_DEVICE_TIMEOUT: return "a bounded device-side wait expired";
    case ROM_ERR_STATIC_SCRATCH: return "problem exceeds the built-in scratch of rom_route_noalloc";
    case ROM_ERR_DEBUG_CHECK: return "a debug check failed (routing-table index out of range or workspace canary overwritten)";
    default: return "unknown status";
  }
}

int rom_last_launch_count(void) { return LaunchCounter::count; }

}  // extern "C"
