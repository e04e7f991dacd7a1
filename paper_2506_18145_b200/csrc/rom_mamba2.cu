// Routing Mamba on a Mamba2-style block (Section 5.2 "RoM on other linear recurrent architectures", Section 5.4 first
// insight, Appendix A.2): every major projection of the block -- the fused input projection [z | x | B | C | dt] and
// the output projection -- is a set of experts under the layer's one routing decision; the depthwise conv, the
// per-head scalars A, D, the dt bias and the gated RMS norm's weight are shared.  The paper prints no equations for
// this variant; the block is the published Mamba2 block with one B/C group:
//   [z|x|B|C|dt]_t = sum_i 1_i X_t W_in,i;  (x,B,C) <- SiLU(conv(x,B,C));  dt = softplus(dt + dt_bias);
//   per head h:  H_t = exp(dt A_h) H_{t-1} + dt x_t (x) B_t,  y_t = C_t H_t + D_h x_t;
//   y^ = RMSNorm(y * SiLU(z)) * w_norm;  O_t = sum_i R_i y^_t W_out,i.
// Launch sequence: the RoM layer's router / permutation / gather, the grouped GEMM (rows back in token order at top-1 on
// the tensor path, otherwise a sum over the slots), a conv over the x|B|C slab, a per-head dt expansion, the selective-scan kernel (the scalar-per-head recurrence is its special case
// A[c, n] = A_head(c), Delta[t, c] = dt[t, head(c)], B-bar = Delta B), a row-wise gated RMS norm that writes the rows in
// expert order, the grouped output GEMM and the gate-weighted combine.
#include "rom_internal.cuh"

namespace rom {
namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

struct M2Layout {
  WsLayout t;          // routing tables + x_perm (the fields launch_route_gather and the GEMMs use)
  size_t ZXp, ZXs, xc, Bm, Cm, D32, A_exp, D_exp, Yt, Ygp, Op, scan_ws, total;
  int W;               // width of the fused input projection
};

M2Layout make_m2_layout(const rom_config& c, int headdim) {
  M2Layout m{};
  WsLayout& l = m.t;
  l.esz = c.dtype == ROM_BF16 ? 2 : 4;
  l.T = (int64_t)c.B * c.L;
  l.A = l.T * c.K;
  l.rows_max = (int64_t)align_up((size_t)l.A, kTileM) + (int64_t)c.E * kTileM;
  l.max_m_tiles = l.rows_max / kTileM;
  l.n_chunks = (l.T + kChunkTokens - 1) / kChunkTokens;
  const size_t De = c.d_inner, N = c.d_state, T = (size_t)l.T, rows = (size_t)l.rows_max, esz = l.esz;
  m.W = (int)(2 * De + 2 * N + De / headdim);
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
  l.gates = take(sizeof(float) * l.A);
  l.row_of_assign = take(sizeof(int32_t) * l.A);
  l.assign_of_row = take(sizeof(int32_t) * l.rows_max);
  l.x_perm = take(esz * rows * c.d_model);
  m.ZXp = take(esz * rows * m.W);
  m.ZXs = take(esz * T * m.W);
  m.xc = take(esz * T * De);
  m.Bm = take(4 * T * N);
  m.Cm = take(4 * T * N);
  m.D32 = take(4 * T * De);
  m.A_exp = take(4 * De * N);
  m.D_exp = take(4 * De);
  m.Yt = take(esz * T * De);
  m.Ygp = take(esz * rows * De);
  m.Op = take(esz * rows * c.d_model);
  m.scan_ws = take(sizeof(float) * scan_ws_floats(c.B, c.d_inner, c.L));
  m.total = o;
  l.total = o;
  return m;
}

int check_m2(const rom_config* c, int headdim) {
  int rc = check_config(c, 1);
  if (rc != ROM_OK) return rc;
  if (c->d_inner < 64 || c->d_inner % 64 != 0) return ROM_ERR_INVALID_ARG;
  if (c->d_state != 16) return c->d_state < 1 ? ROM_ERR_INVALID_ARG : ROM_ERR_UNSUPPORTED;
  if (c->d_conv < 2 || c->d_conv > 4) return c->d_conv < 1 ? ROM_ERR_INVALID_ARG : ROM_ERR_UNSUPPORTED;
  if (headdim < 8 || c->d_inner % headdim != 0 || (c->d_inner / headdim) % 8 != 0) return ROM_ERR_UNSUPPORTED;
  if (c->B > 65535) return ROM_ERR_UNSUPPORTED;
  return ROM_OK;
}

constexpr int M2_TCH = 16;      // tokens per thread of the conv kernel

// SiLU(conv) over the x | B | C slab of the token-order projection rows.  A thread owns one 16-byte group of channels
// and M2_TCH consecutive tokens of one sequence: the M2_TCH + 3 rows it needs are requested at once.
//   ZXs [T, W]: columns [De, 2De + 2N) are the slab; x part -> xc [T, De] (dtype), B, C parts -> Bm, Cm [T, N] (fp32).
template <typename T>
__global__ void __launch_bounds__(128)
m2_conv_kernel(const T* __restrict__ ZXs, const T* __restrict__ w_conv, const float* __restrict__ b_conv, T* __restrict__ xc,
               float* __restrict__ Bm, float* __restrict__ Cm, int L, int De, int N, int W, int k) {
  constexpr int V = V16<T>::N;
  const int Cs = De + 2 * N;
  const int c0 = (blockIdx.x * blockDim.x + threadIdx.x) * V;
  if (c0 >= Cs) return;
  const int tb = blockIdx.y * M2_TCH;
  const size_t tok0 = (size_t)blockIdx.z * L;
  constexpr int NR = M2_TCH + 3;
  V16<T> raw[NR];
#pragma unroll
  for (int r = 0; r < NR; ++r) {
    const int t = tb - 3 + r;
    if (t >= 0 && t < L) raw[r].load(ZXs + (tok0 + t) * W + De + c0);
    else raw[r].zero();
  }
  // taps right-aligned into 4 slots: slot 3 multiplies the current token
  float w[4][V], bias[V];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int src = j - (4 - k);
    if (src >= 0) { V16<T> t; t.load(w_conv + (size_t)src * Cs + c0); t.get(w[j]); }
    else {
#pragma unroll
      for (int i = 0; i < V; ++i) w[j][i] = 0.0f;
    }
  }
#pragma unroll
  for (int i = 0; i < V; ++i) bias[i] = b_conv ? b_conv[c0 + i] : 0.0f;
#pragma unroll
  for (int r = 0; r < M2_TCH; ++r) {
    const int t = tb + r;
    if (t >= L) break;
    float acc[V];
#pragma unroll
    for (int i = 0; i < V; ++i) acc[i] = bias[i];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float hv[V];
      raw[r + j].get(hv);
#pragma unroll
      for (int i = 0; i < V; ++i) acc[i] = fmaf(w[j][i], hv[i], acc[i]);
    }
#pragma unroll
    for (int i = 0; i < V; ++i) acc[i] = sizeof(T) == 4 ? acc[i] / (1.0f + expf(-acc[i])) : silu_fast(acc[i]);
    const size_t tok = tok0 + t;
    if (c0 < De) {
      V16<T>::store(xc + tok * De + c0, acc);
    } else {
      float* dst = c0 < De + N ? Bm + tok * N + (c0 - De) : Cm + tok * N + (c0 - De - N);
#pragma unroll
      for (int i = 0; i < V; i += 4) *reinterpret_cast<float4*>(dst + i) = make_float4(acc[i], acc[i + 1], acc[i + 2], acc[i + 3]);
    }
  }
}

// Delta[t, c] = softplus(dt_raw[t, head(c)] + dt_bias[head(c)]) expanded over the head's channels (fp32), four channels
// per thread; the first threads also expand A_h, D_h to the per-(channel, state) / per-channel arrays the scan kernel reads.
template <typename T>
__global__ void __launch_bounds__(256)
m2_dt_kernel(const T* __restrict__ ZXs, const float* __restrict__ dt_bias, const float* __restrict__ A, const float* __restrict__ D,
             float* __restrict__ D32, float* __restrict__ A_exp, float* __restrict__ D_exp, int De, int N, int W, int headdim, long long Tn) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < (long long)De) {
    const int h = (int)i / headdim;
    for (int n = 0; n < N; ++n) A_exp[i * N + n] = A[h];
    D_exp[i] = D ? D[h] : 0.0f;
  }
  const int q4 = De / 4;
  if (i >= Tn * q4) return;
  const long long tok = i / q4;
  const int c = (int)(i % q4) * 4, h = c / headdim;       // headdim is a multiple of 8: the four channels share a head
  const float v = softplus_f(to_f32(ZXs[tok * W + 2 * De + 2 * N + h]) + (dt_bias ? dt_bias[h] : 0.0f));
  *reinterpret_cast<float4*>(D32 + tok * De + c) = make_float4(v, v, v, v);
}

// y^ = g / sqrt(mean g^2 + eps) * w_norm with g = the gated scan output of the token (one block per token, 16-byte
// accesses), written to the K expert-order rows of the token.
template <typename T>
__global__ void __launch_bounds__(256)
m2_norm_kernel(const T* __restrict__ Yt, const float* __restrict__ w_norm, const int32_t* __restrict__ row_of_assign, T* __restrict__ Ygp,
               int De, int K, float eps) {
  constexpr int V = V16<T>::N;
  __shared__ float red[8];
  const size_t t = blockIdx.x;
  const int nvec = De / V;
  float ss = 0.0f;
  for (int i = threadIdx.x; i < nvec; i += blockDim.x) {
    V16<T> q; q.load(Yt + t * De + (size_t)i * V);
    float v[V]; q.get(v);
#pragma unroll
    for (int j = 0; j < V; ++j) ss = fmaf(v[j], v[j], ss);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.0f;
#pragma unroll
  for (int i = 0; i < 8; ++i) tot += red[i];
  const float r = rsqrtf(tot / (float)De + eps);
  for (int i = threadIdx.x; i < nvec; i += blockDim.x) {
    V16<T> q; q.load(Yt + t * De + (size_t)i * V);
    float v[V]; q.get(v);
#pragma unroll
    for (int j = 0; j < V; ++j) v[j] = to_f32(from_f32<T>(v[j] * r * w_norm[(size_t)i * V + j]));
    for (int k = 0; k < K; ++k) V16<T>::store(Ygp + (size_t)row_of_assign[t * K + k] * De + (size_t)i * V, v);
  }
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

int rom_mamba2_workspace_size(const rom_config* cfg, int32_t headdim, size_t* bytes) {
  if (!bytes) return ROM_ERR_INVALID_ARG;
  const int rc = check_m2(cfg, headdim);
  if (rc != ROM_OK) return rc;
  *bytes = make_m2_layout(*cfg, headdim).total;
  return ROM_OK;
}

int rom_mamba2_layer_forward(const rom_config* cfg, int32_t headdim, const rom_mamba2_weights* w, const void* x, void* out,
                             int32_t* topk_idx_out, float* gates_out, int32_t* counts_out, void* ws, size_t ws_bytes, void* stream) {
  int rc = check_m2(cfg, headdim);
  if (rc != ROM_OK) return rc;
  if (!w || !x || !out || !ws) return ROM_ERR_INVALID_ARG;
  if (!w->W_r || !w->W_in || !w->w_conv || !w->A || !w->w_norm || !w->W_out) return ROM_ERR_INVALID_ARG;
  const void* ptrs[] = {x, out, ws, w->W_r, w->W_in, w->w_conv, w->A, w->w_norm, w->W_out};
  for (const void* p : ptrs)
    if (!aligned16(p)) return ROM_ERR_INVALID_ARG;
  const rom_config& c = *cfg;
  const M2Layout m = make_m2_layout(c, headdim);
  const WsLayout& lay = m.t;
  if (ws_bytes < m.total) return ROM_ERR_WORKSPACE;
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return ROM_ERR_CUDA;
  if (major != 10) return ROM_ERR_ARCH;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* W = static_cast<char*>(ws);
  LaunchCounter::count = 0;

  const int T = (int)lay.T, De = c.d_inner, Dm = c.d_model, N = c.d_state, rows = (int)lay.rows_max, Wd = m.W;
  const bool tc = c.dtype == ROM_BF16 && !(c.flags & ROM_FLAG_SIMT_GEMM);
  const bool bf = c.dtype == ROM_BF16;
  int32_t* status = reinterpret_cast<int32_t*>(W + lay.status);
  const int32_t* tile_expert = reinterpret_cast<const int32_t*>(W + lay.tile_expert);
  const int32_t* num_m_tiles = reinterpret_cast<const int32_t*>(W + lay.num_m_tiles);
  const int32_t* row_of_assign = reinterpret_cast<const int32_t*>(W + lay.row_of_assign);
  float* gates = gates_out ? gates_out : reinterpret_cast<float*>(W + lay.gates);
  auto gemm = [&](const void* A_, int lda, const void* B_, int ldb, int64_t bstride, int Nn, int Kd, const Epilogue& ep) -> cudaError_t {
    if (tc) return launch_gemm_tc(A_, lda, B_, ldb, c.E, rows, Nn, Kd, tile_expert, num_m_tiles, ep, status, st);
    return launch_gemm_simt(c.dtype, A_, lda, B_, ldb, bstride, rows, Nn, Kd, tile_expert, num_m_tiles, ep, st);
  };

  ROM_CUDA(cudaMemsetAsync(status, 0, sizeof(int32_t) * kStatusInts, st));
  ROM_CUDA(launch_route_gather(c, x, w->W_r, w->b_r, topk_idx_out, gates, counts_out, W, lay, st));
  // fused input projection of the selected experts, then the sum over a token's slots (indicator only)
  if (tc && c.K == 1) {
    // one expert per token: the output op writes every row straight to its token's position (no activation: R = width)
    Epilogue e_in{EPI_INPROJ, W + m.ZXs, Wd, nullptr, nullptr, nullptr, Wd, 0, reinterpret_cast<const int32_t*>(W + lay.assign_of_row), nullptr};
    ROM_CUDA(gemm(W + lay.x_perm, Dm, w->W_in, Dm, (int64_t)Wd * Dm, Wd, Dm, e_in));
  } else {
    Epilogue e_in{EPI_STORE, W + m.ZXp, Wd, nullptr, nullptr, nullptr, 0, 0, nullptr, nullptr};
    ROM_CUDA(gemm(W + lay.x_perm, Dm, w->W_in, Dm, (int64_t)Wd * Dm, Wd, Dm, e_in));
    ROM_CUDA(launch_slot_sum(c.dtype, W + m.ZXp, row_of_assign, W + m.ZXs, T, Wd, c.K, st));
  }
  // shared conv + SiLU over x | B | C; dt per head
  {
    const int Cs = De + 2 * N;
    const int vec = bf ? 8 : 4;
    dim3 cgrid((Cs / vec + 127) / 128, (c.L + M2_TCH - 1) / M2_TCH, c.B);
    float* Bm = reinterpret_cast<float*>(W + m.Bm);
    float* Cm = reinterpret_cast<float*>(W + m.Cm);
    if (bf) m2_conv_kernel<__nv_bfloat16><<<cgrid, 128, 0, st>>>((const __nv_bfloat16*)(W + m.ZXs), (const __nv_bfloat16*)w->w_conv, w->b_conv,
                                                                (__nv_bfloat16*)(W + m.xc), Bm, Cm, c.L, De, N, Wd, c.d_conv);
    else m2_conv_kernel<float><<<cgrid, 128, 0, st>>>((const float*)(W + m.ZXs), (const float*)w->w_conv, w->b_conv, (float*)(W + m.xc), Bm, Cm,
                                                    c.L, De, N, Wd, c.d_conv);
    count_launch();
    ROM_CUDA(cudaGetLastError());
    const long long total2 = max((long long)T * (De / 4), (long long)De);
    const unsigned blocks2 = (unsigned)((total2 + 255) / 256);
    float* D32 = reinterpret_cast<float*>(W + m.D32);
    float* A_exp = reinterpret_cast<float*>(W + m.A_exp);
    float* D_exp = reinterpret_cast<float*>(W + m.D_exp);
    if (bf) m2_dt_kernel<__nv_bfloat16><<<blocks2, 256, 0, st>>>((const __nv_bfloat16*)(W + m.ZXs), w->dt_bias, w->A, w->D, D32, A_exp, D_exp, De, N, Wd,
                                                                headdim, T);
    else m2_dt_kernel<float><<<blocks2, 256, 0, st>>>((const float*)(W + m.ZXs), w->dt_bias, w->A, w->D, D32, A_exp, D_exp, De, N, Wd, headdim, T);
    count_launch();
    ROM_CUDA(cudaGetLastError());
    // the scalar-per-head recurrence as a special case of the selective scan (B-bar = Delta B), gate SiLU(z) applied there
    rom_config cs = c;
    cs.disc_mode = 1;
    ROM_CUDA(launch_scan(cs, W + m.xc, D32, true, A_exp, Bm, Cm, w->D ? D_exp : nullptr, W + m.ZXs, Wd, nullptr, nullptr, W + m.Yt, nullptr,
                         nullptr, 1, reinterpret_cast<float*>(W + m.scan_ws), false, st, true));
  }
  // gated RMS norm, rows written in expert order
  if (bf) m2_norm_kernel<__nv_bfloat16><<<T, 256, 0, st>>>((const __nv_bfloat16*)(W + m.Yt), w->w_norm, row_of_assign, (__nv_bfloat16*)(W + m.Ygp), De, c.K, 1e-5f);
  else m2_norm_kernel<float><<<T, 256, 0, st>>>((const float*)(W + m.Yt), w->w_norm, row_of_assign, (float*)(W + m.Ygp), De, c.K, 1e-5f);
  count_launch();
  ROM_CUDA(cudaGetLastError());
  // output projection of the selected experts and the gate-weighted sum
  if (tc && c.K == 1) {
    Epilogue e_out{EPI_OUTPROJ, out, Dm, nullptr, nullptr, nullptr, 0, 0, reinterpret_cast<const int32_t*>(W + lay.assign_of_row), gates};
    ROM_CUDA(gemm(W + m.Ygp, De, w->W_out, De, (int64_t)Dm * De, Dm, De, e_out));
    return ROM_OK;
  }
  Epilogue e_out{EPI_STORE, W + m.Op, Dm, nullptr, nullptr, nullptr, 0, 0, nullptr, nullptr};
  ROM_CUDA(gemm(W + m.Ygp, De, w->W_out, De, (int64_t)Dm * De, Dm, De, e_out));
  ROM_CUDA(launch_combine(c, W + m.Op, row_of_assign, gates, out, st));
  return ROM_OK;
}

}  // extern "C"
