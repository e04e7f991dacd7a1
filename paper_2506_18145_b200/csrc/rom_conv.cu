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

// H row of token t (global token index) = sum over its K slots of the first D_e columns of XZp.
template <typename T, int V>
__device__ __forceinline__ void load_h(const T* XZp, int ld, const int32_t* row_of_assign, int K, int t, int c0, float (&h)[V]) {
#pragma unroll
  for (int i = 0; i < V; ++i) h[i] = 0.0f;
  for (int k = 0; k < K; ++k) {
    const int row = __ldg(row_of_assign + (size_t)t * K + k);
    float v[V];
    load_vec(XZp + (size_t)row * ld + c0, v);
#pragma unroll
    for (int i = 0; i < V; ++i) h[i] += v[i];
  }
}

template <typename T>
__global__ void __launch_bounds__(128)
conv_silu_kernel(const T* __restrict__ XZp, const int32_t* __restrict__ row_of_assign, const T* __restrict__ w_conv,
                 const float* __restrict__ b_conv, T* __restrict__ U, int L, int De, int K, int dconv, int tchunk) {
  constexpr int V = Vec<T>::N;
  const int c0 = (blockIdx.x * blockDim.x + threadIdx.x) * V;
  if (c0 >= De) return;
  const int b = blockIdx.z;
  const int tb = blockIdx.y * tchunk;
  const int te = min(L, tb + tchunk);
  const int ld = 2 * De;
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
  float h1[V], h2[V], h3[V];     // rows t-1, t-2, t-3
  const size_t tok0 = (size_t)b * L;
  if (tb - 1 >= 0) load_h<T, V>(XZp, ld, row_of_assign, K, (int)(tok0 + tb - 1), c0, h1);
  else {
#pragma unroll
    for (int i = 0; i < V; ++i) h1[i] = 0.0f;
  }
  if (tb - 2 >= 0) load_h<T, V>(XZp, ld, row_of_assign, K, (int)(tok0 + tb - 2), c0, h2);
  else {
#pragma unroll
    for (int i = 0; i < V; ++i) h2[i] = 0.0f;
  }
  if (tb - 3 >= 0) load_h<T, V>(XZp, ld, row_of_assign, K, (int)(tok0 + tb - 3), c0, h3);
  else {
#pragma unroll
    for (int i = 0; i < V; ++i) h3[i] = 0.0f;
  }
  for (int t = tb; t < te; ++t) {
    float h0[V], u[V];
    load_h<T, V>(XZp, ld, row_of_assign, K, (int)(tok0 + t), c0, h0);
#pragma unroll
    for (int i = 0; i < V; ++i) {
      float pre = bias[i];
      pre = fmaf(w[0][i], h3[i], pre);
      pre = fmaf(w[1][i], h2[i], pre);
      pre = fmaf(w[2][i], h1[i], pre);
      pre = fmaf(w[3][i], h0[i], pre);
      u[i] = silu_f(pre);
      h3[i] = h2[i]; h2[i] = h1[i]; h1[i] = h0[i];
    }
    store_vec(U + (tok0 + t) * De + c0, u);
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

}  // namespace

cudaError_t launch_conv(const rom_config& c, const void* XZp, const int32_t* row_of_assign, const void* w_conv,
                        const float* b_conv, void* U, cudaStream_t st) {
  const int tchunk = 64;
  const bool bf = c.dtype == ROM_BF16;
  const int V = bf ? 8 : 4;
  const int threads = 128;
  dim3 grid((c.d_inner / V + threads - 1) / threads, (c.L + tchunk - 1) / tchunk, c.B);
  if (bf)
    conv_silu_kernel<__nv_bfloat16><<<grid, threads, 0, st>>>((const __nv_bfloat16*)XZp, row_of_assign, (const __nv_bfloat16*)w_conv,
                                                             b_conv, (__nv_bfloat16*)U, c.L, c.d_inner, c.K, c.d_conv, tchunk);
  else
    conv_silu_kernel<float><<<grid, threads, 0, st>>>((const float*)XZp, row_of_assign, (const float*)w_conv, b_conv, (float*)U,
                                                     c.L, c.d_inner, c.K, c.d_conv, tchunk);
  count_launch();
  return cudaGetLastError();
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

}  // namespace rom
