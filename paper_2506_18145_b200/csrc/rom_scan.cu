// Selective scan (Section 3.1): h_t = exp(Delta_t A) h_{t-1} + B-bar_t U_t, Y_t = C_t h_t (+ D U_t),
// fused with the output gate y * SiLU(z) and with the re-permutation of the gated rows into expert
// order (the routing decision of the Gate/Conv projections is reused for Out Proj, Section 4.2).
//
// State and arithmetic are fp32.  One thread owns one channel and keeps its d_state = 16 states in
// registers; consecutive lanes own consecutive channels, so every load and store of u, Delta, z, y
// is coalesced.  B_t / C_t are staged through shared memory per block of time steps.
#include "rom_internal.cuh"

namespace rom {
namespace {

constexpr int NST = 16;        // d_state
constexpr int TS = 64;         // time steps of B/C staged per shared-memory tile
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// PRECISE: libm-accurate exp / expm1 (fp32 configuration, 1e-4 tolerance).
// otherwise: one MUFU ex2 per state update; expm1 taken as a - 1 (bf16 configurations).
template <typename T, bool PRECISE>
__global__ void __launch_bounds__(128)
scan_kernel(const T* __restrict__ u, const float* __restrict__ delta, const float* __restrict__ A,
            const float* __restrict__ Bm, const float* __restrict__ Cm, const float* __restrict__ D,
            const T* __restrict__ z, int ldz, const float* __restrict__ h0, T* __restrict__ y,
            float* __restrict__ h_last, const int32_t* __restrict__ row_map, int K, int L, int De, int disc_mode) {
  __shared__ float Bs[TS][NST];
  __shared__ float Cs[TS][NST];
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  const int b = blockIdx.y;
  const bool active = c < De;
  const int cc = active ? c : De - 1;

  float a_n[NST], inv_a[NST], h[NST];
#pragma unroll
  for (int n = 0; n < NST; ++n) {
    const float av = A[(size_t)cc * NST + n];
    a_n[n] = PRECISE ? av : av * kLog2e;
    inv_a[n] = 1.0f / av;
    h[n] = h0 ? h0[((size_t)b * De + cc) * NST + n] : 0.0f;
  }
  const float dskip = D ? D[cc] : 0.0f;
  const size_t tok0 = (size_t)b * L;

  for (int t0 = 0; t0 < L; t0 += TS) {
    const int nt = min(TS, L - t0);
    __syncthreads();
    for (int i = threadIdx.x; i < nt * NST; i += blockDim.x) {
      (&Bs[0][0])[i] = Bm[(tok0 + t0) * NST + i];
      (&Cs[0][0])[i] = Cm[(tok0 + t0) * NST + i];
    }
    __syncthreads();
    for (int tt = 0; tt < nt; ++tt) {
      const size_t tok = tok0 + t0 + tt;
      const float dl = delta[tok * De + cc];
      const float uu = to_f32(u[tok * De + cc]);
      float acc = 0.0f;
#pragma unroll
      for (int n = 0; n < NST; ++n) {
        float a, bbar;
        if (PRECISE) {
          const float dA = dl * a_n[n];
          a = expf(dA);
          bbar = (disc_mode == 0) ? expm1f(dA) * inv_a[n] * Bs[tt][n] : dl * Bs[tt][n];
        } else {
          a = ex2_approx(dl * a_n[n]);
          bbar = (disc_mode == 0) ? (a - 1.0f) * inv_a[n] * Bs[tt][n] : dl * Bs[tt][n];
        }
        h[n] = fmaf(a, h[n], bbar * uu);
        acc = fmaf(Cs[tt][n], h[n], acc);
      }
      acc = fmaf(dskip, uu, acc);
      if (row_map == nullptr) {
        if (z) acc *= silu_f(to_f32(z[tok * ldz + cc]));
        if (active) y[tok * De + cc] = from_f32<T>(acc);
      } else {
        float zs = 0.0f;
        for (int k = 0; k < K; ++k) zs += to_f32(z[(size_t)row_map[tok * K + k] * ldz + cc]);
        acc *= silu_f(zs);
        if (active)
          for (int k = 0; k < K; ++k) y[(size_t)row_map[tok * K + k] * De + cc] = from_f32<T>(acc);
      }
    }
  }
  if (h_last && active) {
#pragma unroll
    for (int n = 0; n < NST; ++n) h_last[((size_t)b * De + c) * NST + n] = h[n];
  }
}

}  // namespace

cudaError_t launch_scan(const rom_config& c, const void* u, const float* delta, const float* A, const float* Bm,
                        const float* Cm, const float* D, const void* z, int ldz, const float* h0, void* y,
                        float* h_last, const int32_t* row_map, int K, cudaStream_t st) {
  const int threads = 64;
  dim3 grid((c.d_inner + threads - 1) / threads, c.B);
  if (c.dtype == ROM_BF16)
    scan_kernel<__nv_bfloat16, false><<<grid, threads, 0, st>>>((const __nv_bfloat16*)u, delta, A, Bm, Cm, D, (const __nv_bfloat16*)z, ldz,
                                                               h0, (__nv_bfloat16*)y, h_last, row_map, K, c.L, c.d_inner, c.disc_mode);
  else
    scan_kernel<float, true><<<grid, threads, 0, st>>>((const float*)u, delta, A, Bm, Cm, D, (const float*)z, ldz, h0, (float*)y,
                                                      h_last, row_map, K, c.L, c.d_inner, c.disc_mode);
  count_launch();
  return cudaGetLastError();
}

}  // namespace rom
