// Internal declarations shared by the CUDA translation units of the RoM forward library.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "rom.h"

namespace rom {

constexpr int kTileM = 128;        // expert segments are padded to this many rows (GEMM M tile)
constexpr int kChunkTokens = 32;   // tokens per routing chunk (one warp)
constexpr int kMaxE = 64;
constexpr int kMaxK = 8;
constexpr int kStatusInts = 64;    // status block at the head of the workspace

// status word slots
constexpr int kStatCode = 0;       // 0 or the rom_status a kernel latched (a wait that expired, an index out of range)
constexpr int kStatWhere = 1;      // which wait gave up / which debug check failed (debug aid)
constexpr int kStatIndex = 2;      // debug checks: the offending index
constexpr int kStatTicket = 8;     // router: blocks-done counter (zero between calls)
constexpr int kMaxCanaries = 40;   // sub-buffers of the workspace (debug checks put a canary after each)
constexpr int kCanaryBytes = 256;

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Chunks per sequence of the selective scan: 1 when batch x channels already gives the GPU about 2048 warps at
// 8 states per thread; else the chunk count n (at most 24, each chunk at least 256 steps) for which the n - 1
// chunks of each of the two launches best fill whole waves of two 256-thread blocks per SM (148 SMs assumed
// for sizing).  A function of the problem sizes only, so that workspace sizing and the launch agree.
inline int scan_chunks(int B, int De, int L) {
  const long long blocks1 = (long long)B * ((De + 127) / 128);
  if (blocks1 * 8 >= 2048) return 1;
  const long long cap = 2 * 148;
  int best = 1;
  double best_fill = 0.0;
  for (int n = 2; n <= 24 && (L + n - 1) / n >= 256; ++n) {
    const long long blocks = blocks1 * (n - 1);
    if (blocks * 8 < 2048 && n < 24 && (L + n) / (n + 1) >= 256) continue;      // still too few warps: keep growing
    const double fill = (double)blocks / (double)(((blocks + cap - 1) / cap) * cap);
    if (fill > best_fill + 1e-9) { best_fill = fill; best = n; }
  }
  return best;
}
inline size_t scan_ws_floats(int B, int De, int L) {
  const int nch = scan_chunks(B, De, L);
  return nch == 1 ? 0 : (size_t)B * nch * De * (2 * 16 + 1);
}

// Workspace carving, identical for every entry point (host arithmetic only).
struct WsLayout {
  size_t status, counts, offsets, pad_offsets, num_m_tiles, tile_expert, chunk_counts, chunk_prob;
  size_t topk_idx, gates, perm, inv_perm, row_of_assign, assign_of_row;
  size_t x_perm, XZp, U, Zs, delta_r, Bm, Cm, Delta, Ygp, Op, scan_ws;
  size_t delta_rp, Bp, Cp, Dpre;      // per-expert x Proj / dt Proj only
  size_t total;
  int64_t T, A, rows_max, max_m_tiles, n_chunks;
  size_t esz;
  size_t canary[kMaxCanaries];        // ROM_FLAG_DEBUG_CHECKS: offset of the canary after each sub-buffer
  int n_canary;
};
WsLayout make_layout(const rom_config& c);

// Host-side checks of a rom_config shared by every entry point.  which == 0: full layer; 1: route only; 2: scan only.
int check_config(const rom_config* c, int which);

// Number of SMs of the current device (looked up per device ordinal; nothing is assumed about other devices).
cudaError_t current_device_sm_count(int* n);

// ROM_FLAG_DEBUG_CHECKS: validate the routing tables in the workspace (latches ROM_ERR_DEBUG_CHECK in the status word);
// write (check == false) or compare (check == true) the canary words between the workspace sub-buffers.
cudaError_t launch_check_tables(const rom_config& c, char* ws, const WsLayout& lay, cudaStream_t st);
cudaError_t launch_canaries(char* ws, const WsLayout& lay, bool check, cudaStream_t st);

struct LaunchCounter { static thread_local int count; };
inline void count_launch() { LaunchCounter::count++; }

// ---------------------------------------------------------------- epilogues shared by both GEMM paths
enum EpiMode : int {
  EPI_STORE = 0,      // C[m, n] = acc                          (dtype)
  EPI_XPROJ = 1,      // n < R: delta_r[m, n] (dtype); then Bm[m, n-R], Cm[m, n-R-N] (fp32)
  EPI_SOFTPLUS = 2,   // Delta[m, n] = softplus(acc + bias[n])  (dtype)
  EPI_INPROJ = 3,     // C[m, n] = acc for n < R (Conv Proj), SiLU(acc) for n >= R (Gate Proj)   (dtype); with row_token
                      // (tensor path, top-1) row m is written at row row_token[m], i.e. back in token order
  EPI_OUTPROJ = 4,    // top-1 combine fused: C[row_token[m], n] = row_scale[row_token[m]] * acc; rows with
                      // row_token[m] < 0 (segment padding) are skipped   (dtype; tensor path only)
  EPI_F32 = 5,        // C[m, n] = acc                          (fp32)
  EPI_SWIGLU = 6,     // C[m, j] = SiLU(acc[m, j]) * acc[m, N + j], j < N: B holds, per expert, N "gate" rows then N "up"
                      // rows; N % 128 == 0   (dtype; tensor path only)
  EPI_SOFTPLUS_ROWS = 7  // EPI_SOFTPLUS with row m written at row row_token[m] (skipped when negative)   (tensor path only)
};
struct Epilogue {
  int mode;
  void* C;            // EPI_STORE, EPI_SOFTPLUS: [M, ldc] dtype;  EPI_XPROJ: delta_r [M, R] dtype;  EPI_F32: float [M, ldc]
  int ldc;
  float* Bm;          // EPI_XPROJ
  float* Cm;
  const float* bias;  // EPI_SOFTPLUS (may be null)
  int R, N;
  const int32_t* row_token;   // EPI_OUTPROJ, EPI_INPROJ: token of each (padded) row, -1 in padding
  const float* row_scale;     // EPI_OUTPROJ: gate of each token
};

// ---------------------------------------------------------------- launchers (each returns a cudaError_t)
cudaError_t launch_route(const rom_config& c, const void* x, const void* W_r, const float* b_r,
                         int32_t* topk_idx, float* gates, int32_t* counts, int32_t* offsets,
                         int32_t* perm, int32_t* inv_perm, char* ws, const WsLayout& lay, cudaStream_t st);

// launch_route with the per-chunk sums of the router softmax as an extra output (chunk_prob [n_chunks, E] fp64, or nullptr);
// gather_x: also fill x_perm (the token rows in padded expert order, zero rows in the padding).
// The status block of the workspace (its blocks-done counter) must be zero on entry; it is left zero.
cudaError_t launch_route_stats(const rom_config& c, const void* x, const void* W_r, const float* b_r,
                               int32_t* topk_idx, float* gates, int32_t* counts, int32_t* offsets,
                               int32_t* perm, int32_t* inv_perm, char* ws, const WsLayout& lay, double* chunk_prob, cudaStream_t st,
                               bool gather_x);
// Router + tables + x_perm in two launches (the layer's path).
cudaError_t launch_route_gather(const rom_config& c, const void* x, const void* W_r, const float* b_r,
                                int32_t* topk_idx, float* gates, int32_t* counts, char* ws, const WsLayout& lay, cudaStream_t st);
// Router + load-balance statistic: F[E], Pbar[E], loss[1] (device fp32, each may be null).
cudaError_t launch_balance(const rom_config& c, const void* x, const void* W_r, const float* b_r, float alpha,
                           float* F, float* Pbar, float* loss, char* ws, const WsLayout& lay, cudaStream_t st);

// Permutation tables from a routing decision made elsewhere: topk_idx [T, K] (device) -> the same tables launch_route
// leaves in the workspace (counts, offsets, padded offsets, row tiles, row <-> assignment maps).
cudaError_t launch_perm_from_idx(const rom_config& c, const int32_t* topk_idx, int32_t* counts, int32_t* offsets, int32_t* perm,
                                 int32_t* inv_perm, char* ws, const WsLayout& lay, cudaStream_t st);

cudaError_t launch_gather_rows(const rom_config& c, const void* x, char* ws, const WsLayout& lay, cudaStream_t st);
// dst[row, :] = src[token of row, :] for rows of `width` dtype elements (zero rows in the padding); dst has rows_max rows.
cudaError_t launch_gather_rows_to(const rom_config& c, const void* src, void* dst, int width, char* ws, const WsLayout& lay,
                                  cudaStream_t st);
// Per-expert x Proj / dt Proj: sums over the K slots of a token, in ascending slot order (fp32):
//   Bm[t, :] = sum_k Bp[row(t,k), :],  Cm likewise,  Delta[t, c] = softplus(b_dt[c] + sum_k Dpre[row(t,k), c]).
cudaError_t launch_small_combine(const rom_config& c, const float* Bp, const float* Cp, const float* Dpre,
                                 const int32_t* row_of_assign, const float* b_dt, float* Bm, float* Cm, void* Delta /*dtype*/,
                                 cudaStream_t st);

// C[M,N] = A[M,Kd] * B[e][N,Kd]^T, A and B K-contiguous.  Grouped when tile_expert != nullptr: row tile
// i (kTileM rows) uses expert tile_expert[i]; the number of valid row tiles is *num_m_tiles_dev.
cudaError_t launch_gemm_simt(int dtype, const void* A, int lda, const void* Bw, int ldb, int64_t b_expert_stride,
                             int M_max, int N, int Kd, const int32_t* tile_expert, const int32_t* num_m_tiles_dev,
                             const Epilogue& epi, cudaStream_t st);

// Ungrouped GEMM for a few rows and a long K (M <= 128, Kd a multiple of 2048 for bf16 / 1024 for fp32): K split over
// the threads of a block.
cudaError_t launch_gemm_skinny(int dtype, const void* A, int lda, const void* Bw, int ldb, int M, int N, int Kd,
                               const Epilogue& epi, cudaStream_t st);

cudaError_t launch_gemm_tc(const void* A, int lda, const void* Bw, int ldb, int n_experts,
                           int M_max, int N, int Kd, const int32_t* tile_expert, const int32_t* num_m_tiles_dev,
                           const Epilogue& epi, int32_t* status, cudaStream_t st, bool test_stall = false);

// Grouped weight gradient on the tensor cores (bf16): C[s][P, Q] fp32 = sum over rows r of segment s of Xt[p, r] Yt[q, r];
// Xt [P, ld], Yt [Q, ld] bf16 (activations transposed); seg: n_seg + 1 device row offsets, multiples of 64.
cudaError_t launch_gemm_tc_wgrad(const void* Xt, const void* Yt, int ld, const int32_t* seg, int n_seg, int P, int Q, float* C,
                                 int32_t* status, cudaStream_t st);
// out[c][r] = scale[r] * in[r][c] for in [R, C] (scale may be nullptr); out has row pitch ldo >= R.
cudaError_t launch_transpose_scaled(int dtype, const void* in, void* out, int R, int C, int ldo, const float* scale, cudaStream_t st);

// Conv + SiLU, x Proj and dt Proj + softplus as one tcgen05 kernel (bf16, rows of HZ in token order, shared small layers):
// U, delta_r, Bm, Cm, Delta as the three separate launches leave them.  fused_conv_xdt_supported says whether the sizes fit.
bool fused_conv_xdt_supported(const rom_config& c);
cudaError_t launch_fused_conv_xdt(const rom_config& c, const void* HZ, int ldh, const void* w_conv, const float* b_conv, const void* W_x,
                                  const void* W_dt, const float* b_dt, void* U, void* delta_r, float* Bm, float* Cm, void* Delta,
                                  int32_t* status, cudaStream_t st);

// row_of_assign == nullptr (top-1, rows already in token order): row t of XZp belongs to token t.
// Zs (K > 1 only): [T, d_inner], SiLU of the Gate Proj rows summed over the K slots.
cudaError_t launch_conv(const rom_config& c, const void* XZp, const int32_t* row_of_assign, const void* w_conv,
                        const float* b_conv, void* U, void* Zs, cudaStream_t st);
// One token per sequence (L == 1): conv_state [B, d_conv-1, d_inner] fp32 holds H of the previous tokens (oldest first)
// and is advanced by one token.
cudaError_t launch_conv_step(const rom_config& c, const void* XZp, const int32_t* row_of_assign, const void* w_conv,
                             const float* b_conv, float* conv_state, void* U, void* Zs, cudaStream_t st);

// Scan.  z is a [rows, ldz] matrix; the gate row of token t is z_row[t] (z_row == nullptr: row t).
// y_rows == nullptr: y is [T, d_inner]; otherwise the output row of token t is written K times, to rows
// y_rows[t*K + k].
// gate_activated: z already holds SiLU of the gate pre-activation (the producer applied it).
// chunk_ws == nullptr: one pass per sequence.  Otherwise a long sequence with too few channels to fill the GPU
// is cut into scan_chunks() chunks scanned in parallel (two passes); chunk_ws holds scan_ws_floats() floats.
// delta: [B, L, d_inner], fp32 when delta_fp32, else in the storage dtype.
cudaError_t launch_scan(const rom_config& c, const void* u, const void* delta, bool delta_fp32, const float* A, const float* Bm,
                        const float* Cm, const float* D, const void* z, int ldz, const int32_t* z_row, const float* h0,
                        void* y, float* h_last, const int32_t* y_rows, int K, float* chunk_ws, bool gate_activated, cudaStream_t st,
                        bool scalar_A = false /* A[c, :] constant per channel and disc_mode 1: one exponential per channel and step */);

// One-pass scan for few long sequences (rom_scan_seq.cu): every exponential evaluated once, no workspace.  bf16 storage only.
bool scan_seq_applicable(const rom_config& c, const void* u, const void* delta, bool delta_fp32, const float* Bm, const float* Cm,
                         const void* z, int ldz, const int32_t* z_row, const int32_t* y_rows, bool gate_activated, int num_sms);
cudaError_t launch_scan_seq(const rom_config& c, const void* u, const void* delta, bool delta_fp32, const float* A, const float* Bm,
                            const float* Cm, const float* D, const void* z, int ldz, const float* h0, void* y, float* h_last,
                            const int32_t* y_rows, int K, bool gate_activated, cudaStream_t st);

// State recurrence alone over uniform chunks (rom_scan.cu; used by the backward pass): see the definition.
cudaError_t launch_scan_states(const rom_config& c, const void* u, const float* delta, const float* A, const float* Bm, int Lc, int ncc,
                               const float* h_in, float* h_end, float* sum_delta, float* ckpt, int nck, cudaStream_t st);

// Backward of the scan (gradients of every input); ckpt: scan_bwd_ws_bytes() bytes of scratch.  dA, dBm, dCm, dD are
// zeroed here and accumulated with atomics.  z / dz, h0, dh_last, dD, dh0 may be null.
size_t scan_bwd_ws_bytes(int B, int De, int L);
cudaError_t launch_scan_backward(const rom_config& c, const void* dy, const void* u, const float* delta, const float* A,
                                 const float* Bm, const float* Cm, const float* D, const void* z, const float* h0,
                                 const float* dh_last, void* du, float* ddelta, float* dA, float* dBm, float* dCm, float* dD,
                                 void* dz, float* dh0, float* ckpt, int ldz /* row pitch of z and dz */, cudaStream_t st);

// Pieces of the layer's backward pass (rom_backward.cu); dtype tensors per the config, sums in fp32.
cudaError_t launch_transpose(int dtype, const void* in, void* out, int batch, int R, int C, cudaStream_t st);      // out[b][c][r] = in[b][r][c]
cudaError_t launch_slot_sum(int dtype, const void* src, const int32_t* row_of_assign, void* dst, long long Tn, int width, int K, cudaStream_t st);
cudaError_t launch_cast_f32(int dtype, const void* in, float* out, long long n, cudaStream_t st);
cudaError_t launch_combine_bwd(int dtype, const void* dYgu, const void* Ygp, const int32_t* row_of_assign, const float* gates, void* dYg,
                               float* dgate, float* rowscale, long long Tn, int De, int K, cudaStream_t st);
cudaError_t launch_softplus_bwd(int dtype, const float* ddelta, const float* Delta32, void* dpre, float* db_dt, long long Tn, int De, cudaStream_t st);
cudaError_t launch_pack_bc(int dtype, const float* dBm, const float* dCm, void* dxdbl, long long Tn, int R, int N, cudaStream_t st);
cudaError_t launch_conv_bwd(const rom_config& c, const void* HZ, const void* w_conv, const float* b_conv, const void* dU1, const void* dU2,
                            void* dHZ, float* dw, float* db, cudaStream_t st);
cudaError_t launch_router_bwd(const rom_config& c, const void* x, const void* W_r, const float* b_r, const int32_t* idx, const float* gates,
                              const float* dgate, float* dlogit, float* db_r, float* dW_r, cudaStream_t st);
cudaError_t launch_dx(const rom_config& c, const void* dxp, const int32_t* row_of_assign, const float* dlogit, const void* W_r, void* dx,
                      cudaStream_t st);
// C[s][P, Q] = sum over rows r of segment s of scale[r] X[r, :P]^T Y[r, :Q]; seg: n_seg + 1 row offsets (device) or nullptr = one
// segment of rows_total rows; scale may be nullptr.
cudaError_t launch_wgrad(int dtype, const void* X, int ldx, const void* Y, int ldy, const float* scale, const int32_t* seg, int n_seg,
                         int rows_total, int P, int Q, float* C, cudaStream_t st);

cudaError_t launch_combine(const rom_config& c, const void* Op, const int32_t* row_of_assign, const float* gates,
                           void* out, cudaStream_t st);

// ---------------------------------------------------------------- device helpers
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

__device__ __forceinline__ float silu_f(float v) { return v / (1.0f + __expf(-v)); }
// Fast forms for the bf16 path (results are rounded to bf16 or feed a 2e-2 tolerance): the special-function
// unit's approximate exp2 / log2 / reciprocal with flush-to-zero, relative error ~1e-6, no range fix-ups.
__device__ __forceinline__ float ex2_ftz(float x) { float y; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ float lg2_ftz(float x) { float y; asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ float rcp_ftz(float x) { float y; asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x)); return y; }
__device__ __forceinline__ float silu_fast(float v) { return v * rcp_ftz(1.0f + ex2_ftz(-1.4426950408889634f * v)); }

// 16 bytes of consecutive elements as floats
template <typename T> struct V16;
template <> struct V16<__nv_bfloat16> {
  static constexpr int N = 8;
  uint4 q;
  __device__ __forceinline__ void load(const __nv_bfloat16* p) { q = __ldg(reinterpret_cast<const uint4*>(p)); }
  __device__ __forceinline__ void zero() { q = make_uint4(0, 0, 0, 0); }
  __device__ __forceinline__ void get(float (&v)[8]) const {
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) { v[2 * i] = __uint_as_float(w[i] << 16); v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u); }
  }
  static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&v)[8]) {
    uint4 o;
    uint32_t* w = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
    for (int i = 0; i < 4; ++i) { const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]); w[i] = *reinterpret_cast<const uint32_t*>(&h); }
    *reinterpret_cast<uint4*>(p) = o;
  }
};
template <> struct V16<float> {
  static constexpr int N = 4;
  float4 q;
  __device__ __forceinline__ void load(const float* p) { q = __ldg(reinterpret_cast<const float4*>(p)); }
  __device__ __forceinline__ void zero() { q = make_float4(0.0f, 0.0f, 0.0f, 0.0f); }
  __device__ __forceinline__ void get(float (&v)[4]) const { v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w; }
  static __device__ __forceinline__ void store(float* p, const float (&v)[4]) { *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]); }
};

// softplus for results that are rounded to bf16: max(v,0) + log1p(e), e = exp(-|v|) in (0, 1], with
// log1p(e) = e * q(e), q a degree-4 polynomial fitted to log1p(e)/e on [0, 1] (relative error 6.3e-5, a
// sixtieth of a bf16 rounding step): one special-function operation per value instead of two.
__device__ __forceinline__ float softplus_bf16(float v) {
  const float e = ex2_ftz(-1.4426950408889634f * fabsf(v));
  float q = fmaf(0.04066344f, e, -0.15602953f);
  q = fmaf(q, e, 0.30539998f);
  q = fmaf(q, e, -0.49678875f);
  q = fmaf(q, e, 0.99993682f);
  return fmaf(e, q, fmaxf(v, 0.0f));
}
__device__ __forceinline__ float softplus_fast(float v) {
  // max(v,0) + log(1 + e), e = exp(-|v|) in (0, 1].  For tiny e, 1 + e loses e's low bits: use log1p(e) ~ e.
  const float e = ex2_ftz(-1.4426950408889634f * fabsf(v));
  const float l = e < 2.44140625e-4f ? e : 0.6931471805599453f * lg2_ftz(1.0f + e);
  return fmaxf(v, 0.0f) + l;
}
__device__ __forceinline__ float softplus_f(float v) {
  // max(v,0) + log1p(exp(-|v|)); log1pf keeps relative accuracy when exp(-|v|) is tiny
  return fmaxf(v, 0.0f) + log1pf(__expf(-fabsf(v)));
}

}  // namespace rom
