// Un-permute + sum over the selected experts (indicator only, Section 4.2 equation for H_t), then the
// causal depthwise short convolution with SiLU (Section 3.1, U = SiLU(DWConv(H, W_conv))).
// Also the gate-weighted combine of the Out Proj rows (Section 4.2 equation for O_t).
//
// Both are HBM-bound streaming kernels: one 16-byte vector of channels per thread, consecutive
// threads on consecutive vectors, a sliding window of the previous k-1 rows kept in registers.
#include "rom_internal.cuh"

namespace rom {
namespace {

template <typename T> struct Vec;
template <> struct Vec<__nv_bfloat16> { static constexpr int N = 8; };
template <> struct Vec<float> { static constexpr int N = 4; };

__device__ __forceinline__ void load_vec(const __nv_bfloat16* p, float (&v)[8]) {
  const uint4 q = __ldg(reinterpret_cast<const uint4*>(p));
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    v[2 * i] = __uint_as_float(w[i] << 16);
    v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ void load_vec(const float* p, float (&v)[4]) {
  const float4 q = __ldg(reinterpret_cast<const float4*>(p));
  v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
}
__device__ __forceinline__ void store_vec(__nv_bfloat16* p, const float (&v)[8]) {
  uint4 q;
  uint32_t* w = reinterpret_cast<uint32_t*>(&q);
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
    w[i] = *reinterpret_cast<uint32_t*>(&h);
  }
  *reinterpret_cast<uint4*>(p) = q;
}
__device__ __forceinline__ void store_vec(float* p, const float (&v)[4]) {
  *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
}

// One 16-byte vector kept as loaded; converted to fp32 only when used.
template <typename T> struct RawVec;
template <> struct RawVec<__nv_bfloat16> {
  uint4 q;
  __device__ __forceinline__ void load(const __nv_bfloat16* p) { q = __ldg(reinterpret_cast<const uint4*>(p)); }
  __device__ __forceinline__ void zero() { q = make_uint4(0, 0, 0, 0); }
  __device__ __forceinline__ void get(float (&v)[8]) const {
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
};
template <> struct RawVec<float> {
  float4 q;
  __device__ __forceinline__ void load(const float* p) { q = __ldg(reinterpret_cast<const float4*>(p)); }
  __device__ __forceinline__ void zero() { q = make_float4(0.0f, 0.0f, 0.0f, 0.0f); }
  __device__ __forceinline__ void get(float (&v)[4]) const { v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w; }
};

// Sum over the K slots of a token of one 16-byte vector of a [rows, ld] matrix (fp32 accumulation).
template <typename T, int V, int KT>
__device__ __forceinline__ void load_sum(const T* M, int ld, const int32_t* row_of_assign, int K, size_t t, int c0, float (&h)[V]) {
  if constexpr (KT == 1) {
    load_vec(M + (size_t)__ldg(row_of_assign + t) * ld + c0, h);
  } else {
    const int kk = KT > 0 ? KT : K;
#pragma unroll
    for (int i = 0; i < V; ++i) h[i] = 0.0f;
#pragma unroll
    for (int k = 0; k < kk; ++k) {
      float v[V];
      load_vec(M + (size_t)__ldg(row_of_assign + t * kk + k) * ld + c0, v);
#pragma unroll
      for (int i = 0; i < V; ++i) h[i] += v[i];
    }
  }
}

// One thread: one 16-byte vector of channels, TCH consecutive time steps of one sequence.  All rows it
// needs (TCH + 3 of H, TCH of Z when Zs != nullptr) are loaded before anything is consumed, so the
// memory system sees TCH + 3 independent requests per thread.  KT > 0 fixes K at compile time.
constexpr int TCH = 8;

template <typename T, int KT>
__global__ void __launch_bounds__(128)
conv_silu_kernel(const T* __restrict__ XZp, const int32_t* __restrict__ row_of_assign, const T* __restrict__ w_conv,
                 const float* __restrict__ b_conv, T* __restrict__ U, T* __restrict__ Zs, int L, int De, int K, int dconv) {
  constexpr int V = Vec<T>::N;
  const int c0 = (blockIdx.x * blockDim.x + threadIdx.x) * V;
  if (c0 >= De) return;
  const int b = blockIdx.z;
  const int tb = blockIdx.y * TCH;
  const int ld = 2 * De;
  const size_t tok0 = (size_t)b * L;

  // rows tb-3 .. tb+TCH-1 of H.  K = 1, 2: kept as raw 16-byte words (row indices first, then all rows in
  // flight at once), converted and summed over the slots on use; other K: summed over the slots as they arrive.
  constexpr int NR = TCH + 3;
  constexpr bool RAWP = KT == 1 || KT == 2;
  constexpr int KS = RAWP ? KT : 1;
  RawVec<T> raw[RAWP ? NR : 1][KS];
  int32_t rix[RAWP ? NR : 1][KS];
  float hsum[RAWP ? 1 : NR][V];
  if constexpr (RAWP) {
#pragma unroll
    for (int r = 0; r < NR; ++r) {
      const int t = tb - 3 + r;
#pragma unroll
      for (int k = 0; k < KS; ++k)
        rix[r][k] = (t >= 0 && t < L) ? (row_of_assign ? __ldg(row_of_assign + (tok0 + t) * KS + k) : (int32_t)(tok0 + t)) : -1;
    }
#pragma unroll
    for (int r = 0; r < NR; ++r) {
#pragma unroll
      for (int k = 0; k < KS; ++k) {
        if (rix[r][k] >= 0) raw[r][k].load(XZp + (size_t)rix[r][k] * ld + c0);
        else raw[r][k].zero();
      }
    }
  } else {
#pragma unroll
    for (int r = 0; r < NR; ++r) {
      const int t = tb - 3 + r;
      if (t >= 0 && t < L) load_sum<T, V, KT>(XZp, ld, row_of_assign, K, tok0 + t, c0, hsum[r]);
      else {
#pragma unroll
        for (int i = 0; i < V; ++i) hsum[r][i] = 0.0f;
      }
    }
  }
  auto hrow = [&](int r, float (&out)[V]) {
    if constexpr (RAWP) {
      raw[r][0].get(out);
      if constexpr (KS == 2) {
        float v2[V];
        raw[r][1].get(v2);
#pragma unroll
        for (int i = 0; i < V; ++i) out[i] += v2[i];
      }
    } else {
#pragma unroll
      for (int i = 0; i < V; ++i) out[i] = hsum[r][i];
    }
  };
  // taps right-aligned into 4 slots: slot 3 multiplies the current token
  float w[4][V];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int src = j - (4 - dconv);
    if (src >= 0) load_vec(w_conv + (size_t)src * De + c0, w[j]);
    else {
#pragma unroll
      for (int i = 0; i < V; ++i) w[j][i] = 0.0f;
    }
  }
  float bias[V];
#pragma unroll
  for (int i = 0; i < V; ++i) bias[i] = b_conv ? b_conv[c0 + i] : 0.0f;

#pragma unroll
  for (int r = 0; r < TCH; ++r) {
    const int t = tb + r;
    if (t >= L) break;
    float u[V], h0[V], h1[V], h2[V], h3[V];
    hrow(r, h0); hrow(r + 1, h1); hrow(r + 2, h2); hrow(r + 3, h3);
#pragma unroll
    for (int i = 0; i < V; ++i) {
      float pre = bias[i];
      pre = fmaf(w[0][i], h0[i], pre);
      pre = fmaf(w[1][i], h1[i], pre);
      pre = fmaf(w[2][i], h2[i], pre);
      pre = fmaf(w[3][i], h3[i], pre);
      u[i] = sizeof(T) == 2 ? silu_fast(pre) : silu_f(pre);
    }
    store_vec(U + (tok0 + t) * De + c0, u);
  }
  if (Zs != nullptr) {
    // G = SiLU(sum over the selected experts of the Gate Proj rows) (indicator only), one row per token
    if constexpr (KS == 2) {
      // the Gate rows of the TCH tokens: same row indices as H, all requested before any is used
#pragma unroll
      for (int r = 0; r < TCH; ++r) {
#pragma unroll
        for (int k = 0; k < KS; ++k) {
          if (rix[r + 3][k] >= 0) raw[r][k].load(XZp + De + (size_t)rix[r + 3][k] * ld + c0);
          else raw[r][k].zero();
        }
      }
#pragma unroll
      for (int r = 0; r < TCH; ++r) {
        const int t = tb + r;
        if (t >= L) break;
        float zsum[V];
        hrow(r, zsum);
#pragma unroll
        for (int i = 0; i < V; ++i) zsum[i] = sizeof(T) == 2 ? silu_fast(zsum[i]) : silu_f(zsum[i]);
        store_vec(Zs + (tok0 + t) * De + c0, zsum);
      }
    } else {
#pragma unroll
      for (int r = 0; r < TCH; ++r) {
        const int t = tb + r;
        if (t >= L) break;
        float zsum[V];
        load_sum<T, V, KT>(XZp + De, ld, row_of_assign, K, tok0 + t, c0, zsum);
#pragma unroll
        for (int i = 0; i < V; ++i) zsum[i] = sizeof(T) == 2 ? silu_fast(zsum[i]) : silu_f(zsum[i]);
        store_vec(Zs + (tok0 + t) * De + c0, zsum);
      }
    }
  }
}

// Single-token step of the short convolution: one thread = one 16-byte vector of channels of one sequence.
// conv_state [B, dconv-1, De] fp32 holds H of the previous dconv-1 tokens, oldest first; it is shifted by one and
// the new H appended.  Taps are applied in the same order as in conv_silu_kernel (right-aligned into 4 slots).
template <typename T>
__global__ void __launch_bounds__(128)
conv_step_kernel(const T* __restrict__ XZp, const int32_t* __restrict__ row_of_assign, const T* __restrict__ w_conv,
                 const float* __restrict__ b_conv, float* __restrict__ conv_state, T* __restrict__ U, T* __restrict__ Zs,
                 int De, int K, int dconv) {
  constexpr int V = Vec<T>::N;
  const int c0 = (blockIdx.x * blockDim.x + threadIdx.x) * V;
  if (c0 >= De) return;
  const size_t b = blockIdx.y;
  const int ld = 2 * De;
  float win[4][V];                       // slot 3 = the current token, slots 4-dconv .. 2 = the state rows
  if (row_of_assign) load_sum<T, V, 0>(XZp, ld, row_of_assign, K, b, c0, win[3]);
  else load_vec(XZp + b * ld + c0, win[3]);
  float* st = conv_state + b * (size_t)(dconv - 1) * De + c0;
#pragma unroll
  for (int j = 0; j < 3; ++j) {
    const int src = j - (4 - dconv);     // state row feeding slot j
#pragma unroll
    for (int i = 0; i < V; ++i) win[j][i] = src >= 0 ? st[(size_t)src * De + i] : 0.0f;
  }
  float u[V];
#pragma unroll
  for (int i = 0; i < V; ++i) u[i] = b_conv ? b_conv[c0 + i] : 0.0f;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int src = j - (4 - dconv);
    if (src < 0) continue;
    float w[V];
    load_vec(w_conv + (size_t)src * De + c0, w);
#pragma unroll
    for (int i = 0; i < V; ++i) u[i] = fmaf(w[i], win[j][i], u[i]);
  }
#pragma unroll
  for (int i = 0; i < V; ++i) u[i] = sizeof(T) == 2 ? silu_fast(u[i]) : silu_f(u[i]);
  store_vec(U + b * De + c0, u);
  // new state: drop the oldest row, append the current H
#pragma unroll
  for (int j = 0; j < 3; ++j) {
    const int dst = j - (4 - dconv);
    if (dst < 0) continue;
#pragma unroll
    for (int i = 0; i < V; ++i) st[(size_t)dst * De + i] = win[j + 1][i];
  }
  if (Zs != nullptr) {
    float zsum[V];
    load_sum<T, V, 0>(XZp + De, ld, row_of_assign, K, b, c0, zsum);
#pragma unroll
    for (int i = 0; i < V; ++i) zsum[i] = sizeof(T) == 2 ? silu_fast(zsum[i]) : silu_f(zsum[i]);
    store_vec(Zs + b * De + c0, zsum);
  }
}

// out[t, :] = sum_k gates[t,k] * Op[row_of_assign[t*K+k], :], slots added in ascending k.
template <typename T>
__global__ void __launch_bounds__(256)
combine_kernel(const T* __restrict__ Op, const int32_t* __restrict__ row_of_assign, const float* __restrict__ gates,
               T* __restrict__ out, int Dm, int K, long long total_vec) {
  constexpr int V = Vec<T>::N;
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total_vec) return;
  const int vpr = Dm / V;
  const long long t = i / vpr;
  const int c0 = (int)(i % vpr) * V;
  float acc[V];
#pragma unroll
  for (int j = 0; j < V; ++j) acc[j] = 0.0f;
  for (int k = 0; k < K; ++k) {
    const int row = __ldg(row_of_assign + t * K + k);
    const float g = __ldg(gates + t * K + k);
    float v[V];
    load_vec(Op + (size_t)row * Dm + c0, v);
#pragma unroll
    for (int j = 0; j < V; ++j) acc[j] = fmaf(g, v[j], acc[j]);
  }
  store_vec(out + t * Dm + c0, acc);
}

// Per-expert x Proj / dt Proj: one thread per float4 of a token's [Delta | B | C] row; the K slots are added in
// ascending order, then (Delta only) the shared bias and the softplus.
template <typename T>
__global__ void __launch_bounds__(256)
small_combine_kernel(const float* __restrict__ Bp, const float* __restrict__ Cp, const float* __restrict__ Dpre,
                     const int32_t* __restrict__ row_of_assign, const float* __restrict__ b_dt, float* __restrict__ Bm,
                     float* __restrict__ Cm, T* __restrict__ Delta, int De, int N, int K, long long total_vec) {
  constexpr bool PRECISE = sizeof(T) == 4;
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total_vec) return;
  const int vpr = (De + 2 * N) / 4;
  const long long t = i / vpr;
  const int c0 = (int)(i % vpr) * 4;
  const float* src; float* dst = nullptr; int ld, col;
  if (c0 < De) { src = Dpre; ld = De; col = c0; }
  else if (c0 < De + N) { src = Bp; dst = Bm; ld = N; col = c0 - De; }
  else { src = Cp; dst = Cm; ld = N; col = c0 - De - N; }
  float4 acc = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
  for (int k = 0; k < K; ++k) {
    const int row = __ldg(row_of_assign + t * K + k);
    const float4 v = __ldg(reinterpret_cast<const float4*>(src + (size_t)row * ld + col));
    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
  }
  if (c0 < De) {
    const float4 b = b_dt ? __ldg(reinterpret_cast<const float4*>(b_dt + col)) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    if (PRECISE) acc = make_float4(softplus_f(acc.x + b.x), softplus_f(acc.y + b.y), softplus_f(acc.z + b.z), softplus_f(acc.w + b.w));
    else acc = make_float4(softplus_fast(acc.x + b.x), softplus_fast(acc.y + b.y), softplus_fast(acc.z + b.z), softplus_fast(acc.w + b.w));
    T* d = Delta + (size_t)t * ld + col;
    d[0] = from_f32<T>(acc.x); d[1] = from_f32<T>(acc.y); d[2] = from_f32<T>(acc.z); d[3] = from_f32<T>(acc.w);
    return;
  }
  *reinterpret_cast<float4*>(dst + (size_t)t * ld + col) = acc;
}

}  // namespace

template <typename T>
cudaError_t launch_conv_t(const rom_config& c, const void* XZp, const int32_t* row_of_assign, const void* w_conv,
                          const float* b_conv, void* U, void* Zs, cudaStream_t st) {
  constexpr int V = Vec<T>::N;
  const int threads = 128;
  dim3 grid((c.d_inner / V + threads - 1) / threads, (c.L + TCH - 1) / TCH, c.B);
  auto args = [&](auto kern) {
    kern<<<grid, threads, 0, st>>>((const T*)XZp, row_of_assign, (const T*)w_conv, b_conv, (T*)U, (T*)Zs, c.L, c.d_inner, c.K, c.d_conv);
  };
  if (c.K == 1) args(conv_silu_kernel<T, 1>);
  else if (c.K == 2) args(conv_silu_kernel<T, 2>);
  else args(conv_silu_kernel<T, 0>);
  count_launch();
  return cudaGetLastError();
}

// Zs: [T, d_inner] sum over the K slots of the Gate Proj rows, or nullptr (not produced).
cudaError_t launch_conv(const rom_config& c, const void* XZp, const int32_t* row_of_assign, const void* w_conv,
                        const float* b_conv, void* U, void* Zs, cudaStream_t st) {
  if (c.B > 65535 || (c.L + TCH - 1) / TCH > 65535) return cudaErrorInvalidConfiguration;
  return c.dtype == ROM_BF16 ? launch_conv_t<__nv_bfloat16>(c, XZp, row_of_assign, w_conv, b_conv, U, Zs, st)
                             : launch_conv_t<float>(c, XZp, row_of_assign, w_conv, b_conv, U, Zs, st);
}

cudaError_t launch_combine(const rom_config& c, const void* Op, const int32_t* row_of_assign, const float* gates,
                           void* out, cudaStream_t st) {
  const bool bf = c.dtype == ROM_BF16;
  const int V = bf ? 8 : 4;
  const long long total = (long long)c.B * c.L * (c.d_model / V);
  const int threads = 256;
  const unsigned blocks = (unsigned)((total + threads - 1) / threads);
  if (bf)
    combine_kernel<__nv_bfloat16><<<blocks, threads, 0, st>>>((const __nv_bfloat16*)Op, row_of_assign, gates, (__nv_bfloat16*)out,
                                                             c.d_model, c.K, total);
  else
    combine_kernel<float><<<blocks, threads, 0, st>>>((const float*)Op, row_of_assign, gates, (float*)out, c.d_model, c.K, total);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_small_combine(const rom_config& c, const float* Bp, const float* Cp, const float* Dpre,
                                 const int32_t* row_of_assign, const float* b_dt, float* Bm, float* Cm, void* Delta,
                                 cudaStream_t st) {
  const long long total = (long long)c.B * c.L * ((c.d_inner + 2 * c.d_state) / 4);
  const unsigned blocks = (unsigned)((total + 255) / 256);
  if (c.dtype == ROM_F32)
    small_combine_kernel<float><<<blocks, 256, 0, st>>>(Bp, Cp, Dpre, row_of_assign, b_dt, Bm, Cm, (float*)Delta, c.d_inner, c.d_state, c.K, total);
  else
    small_combine_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(Bp, Cp, Dpre, row_of_assign, b_dt, Bm, Cm, (__nv_bfloat16*)Delta, c.d_inner, c.d_state, c.K, total);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_conv_step(const rom_config& c, const void* XZp, const int32_t* row_of_assign, const void* w_conv,
                             const float* b_conv, float* conv_state, void* U, void* Zs, cudaStream_t st) {
  const bool bf = c.dtype == ROM_BF16;
  const int V = bf ? 8 : 4;
  const int threads = 128;
  dim3 grid((c.d_inner / V + threads - 1) / threads, c.B);
  if (bf)
    conv_step_kernel<__nv_bfloat16><<<grid, threads, 0, st>>>((const __nv_bfloat16*)XZp, row_of_assign, (const __nv_bfloat16*)w_conv, b_conv,
                                                            conv_state, (__nv_bfloat16*)U, (__nv_bfloat16*)Zs, c.d_inner, c.K, c.d_conv);
  else
    conv_step_kernel<float><<<grid, threads, 0, st>>>((const float*)XZp, row_of_assign, (const float*)w_conv, b_conv, conv_state,
                                                     (float*)U, (float*)Zs, c.d_inner, c.K, c.d_conv);
  count_launch();
  return cudaGetLastError();
}

}  // namespace rom
