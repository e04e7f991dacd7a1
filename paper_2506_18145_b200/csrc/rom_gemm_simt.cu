// Plain fp32-FMA tiled GEMM, C[M,N] = A[M,Kd] * B[e][N,Kd]^T with fp32 accumulation.
// It is the projection path of the fp32 configuration (a tf32 tensor path would not hold the 1e-4
// tolerance) and, under ROM_FLAG_SIMT_GEMM, a bisecting aid for the bf16 tensor path.
#include "rom_internal.cuh"

namespace rom {
namespace {

constexpr int BM = 64, BN = 64, BK = 16;

template <typename T>
__device__ __forceinline__ void epi_store_scalar(const Epilogue& ep, int m, int n, float v) {
  switch (ep.mode) {
    case EPI_STORE:
      reinterpret_cast<T*>(ep.C)[(size_t)m * ep.ldc + n] = from_f32<T>(v);
      break;
    case EPI_INPROJ:
      reinterpret_cast<T*>(ep.C)[(size_t)m * ep.ldc + n] = from_f32<T>(n >= ep.R ? silu_f(v) : v);
      break;
    case EPI_XPROJ:
      if (n < ep.R) reinterpret_cast<T*>(ep.C)[(size_t)m * ep.R + n] = from_f32<T>(v);
      else if (n < ep.R + ep.N) ep.Bm[(size_t)m * ep.N + (n - ep.R)] = v;
      else ep.Cm[(size_t)m * ep.N + (n - ep.R - ep.N)] = v;
      break;
    case EPI_F32:
      reinterpret_cast<float*>(ep.C)[(size_t)m * ep.ldc + n] = v;
      break;
    default:
      reinterpret_cast<T*>(ep.C)[(size_t)m * ep.ldc + n] = from_f32<T>(softplus_f(v + (ep.bias ? ep.bias[n] : 0.0f)));
      break;
  }
}

template <typename T>
__global__ void __launch_bounds__(256)
gemm_simt(const T* __restrict__ A, int lda, const T* __restrict__ Bw, int ldb, int64_t b_expert_stride,
          int M_max, int N, int Kd, const int32_t* __restrict__ tile_expert, const int32_t* __restrict__ num_m_tiles_dev,
          Epilogue ep) {
  __shared__ float As[BK][BM + 1];
  __shared__ float Bs[BK][BN + 1];
  const int m0 = blockIdx.x * BM, n0 = blockIdx.y * BN;
  int M = M_max;
  if (num_m_tiles_dev) M = min(M_max, *num_m_tiles_dev * kTileM);
  if (m0 >= M) return;
  const T* Bp = Bw;
  if (tile_expert) {
    const int e = tile_expert[m0 / kTileM];
    if (e < 0) return;
    Bp = Bw + (size_t)e * b_expert_stride;
  }
  const int tid = threadIdx.x;
  const int ty = tid / 16, tx = tid % 16;
  float acc[4][4] = {};
  // each thread brings 4 elements of the A tile and 4 of the B tile per K block; the next block's elements are
  // requested before the current block is multiplied, so the global-memory latency overlaps the arithmetic
  float pa[4], pb[4];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int i = tid + 256 * j;
      const int r = i / BK, k = i % BK;
      const int m = m0 + r, n = n0 + r, kk = k0 + k;
      pa[j] = (m < M && kk < Kd) ? to_f32(A[(size_t)m * lda + kk]) : 0.0f;
      pb[j] = (n < N && kk < Kd) ? to_f32(Bp[(size_t)n * ldb + kk]) : 0.0f;
    }
  };
  fetch(0);
  for (int k0 = 0; k0 < Kd; k0 += BK) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int i = tid + 256 * j;
      As[i % BK][i / BK] = pa[j];
      Bs[i % BK][i / BK] = pb[j];
    }
    __syncthreads();
    if (k0 + BK < Kd) fetch(k0 + BK);
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[k][ty * 4 + i]; b[i] = Bs[k][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n < N) epi_store_scalar<T>(ep, m, n, acc[i][j]);
    }
  }
}

}  // namespace

cudaError_t launch_gemm_simt(int dtype, const void* A, int lda, const void* Bw, int ldb, int64_t b_expert_stride,
                             int M_max, int N, int Kd, const int32_t* tile_expert, const int32_t* num_m_tiles_dev,
                             const Epilogue& epi, cudaStream_t st) {
  dim3 grid((M_max + BM - 1) / BM, (N + BN - 1) / BN);
  if (dtype == ROM_BF16)
    gemm_simt<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)A, lda, (const __nv_bfloat16*)Bw, ldb, b_expert_stride,
                                                  M_max, N, Kd, tile_expert, num_m_tiles_dev, epi);
  else
    gemm_simt<float><<<grid, 256, 0, st>>>((const float*)A, lda, (const float*)Bw, ldb, b_expert_stride, M_max, N, Kd,
                                          tile_expert, num_m_tiles_dev, epi);
  count_launch();
  return cudaGetLastError();
}

}  // namespace rom
