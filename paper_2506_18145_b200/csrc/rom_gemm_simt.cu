// Plain fp32-FMA tiled GEMM, C[M,N] = A[M,Kd] * B[e][N,Kd]^T with fp32 accumulation.
// It is the projection path of the fp32 configuration (a tf32 tensor path would not hold the 1e-4
// tolerance) and, under ROM_FLAG_SIMT_GEMM, a bisecting aid for the bf16 tensor path.
#include "rom_internal.cuh"

namespace rom {
namespace {

constexpr int BM = 64, BN = 64, BK = 16;

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

// Few rows, long K (the x Proj of a single-token step): C[M,N] = A[M,Kd] * B[N,Kd]^T with the K dimension split over
// all 256 threads of a block.  A block owns 2 rows x 4 columns, so a handful of rows still spreads over
// (M/2) x (N/4) blocks and every thread has only Kd / (256 V) rounds of loads in flight behind one another
// (V = 16 bytes of T; Kd % (256 V) == 0).  Partial sums: lanes by shuffles, then the 8 warps in warp order.
template <typename T>
__global__ void __launch_bounds__(256)
gemm_skinny(const T* __restrict__ A, int lda, const T* __restrict__ Bw, int ldb, int M, int N, int Kd, Epilogue ep) {
  constexpr int V = 16 / sizeof(T);
  __shared__ float part[8][8];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int n0 = blockIdx.x * 4;
  const int r0 = blockIdx.y * 2;
  const bool row1 = r0 + 1 < M;
  float acc[2][4] = {};
  for (int k = threadIdx.x * V; k < Kd; k += 256 * V) {
    float a0[V], a1[V];
    load_vec(A + (size_t)r0 * lda + k, a0);
    if (row1) load_vec(A + (size_t)(r0 + 1) * lda + k, a1);
    else {
#pragma unroll
      for (int i = 0; i < V; ++i) a1[i] = 0.0f;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float w[V];
      load_vec(Bw + (size_t)min(n0 + j, N - 1) * ldb + k, w);
#pragma unroll
      for (int i = 0; i < V; ++i) {
        acc[0][j] = fmaf(a0[i], w[i], acc[0][j]);
        acc[1][j] = fmaf(a1[i], w[i], acc[1][j]);
      }
    }
  }
#pragma unroll
  for (int r = 0; r < 2; ++r)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float v = acc[r][j];
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0) part[warp][r * 4 + j] = v;
    }
  __syncthreads();
  if (threadIdx.x < 8) {
    const int r = threadIdx.x >> 2, j = threadIdx.x & 3;
    float v = 0.0f;
#pragma unroll
    for (int w = 0; w < 8; ++w) v += part[w][threadIdx.x];
    if (r0 + r < M && n0 + j < N) epi_store_scalar<T>(ep, r0 + r, n0 + j, v);
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

cudaError_t launch_gemm_skinny(int dtype, const void* A, int lda, const void* Bw, int ldb, int M, int N, int Kd,
                               const Epilogue& epi, cudaStream_t st) {
  dim3 grid((N + 3) / 4, (M + 1) / 2);
  if (dtype == ROM_BF16)
    gemm_skinny<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)A, lda, (const __nv_bfloat16*)Bw, ldb, M, N, Kd, epi);
  else
    gemm_skinny<float><<<grid, 256, 0, st>>>((const float*)A, lda, (const float*)Bw, ldb, M, N, Kd, epi);
  count_launch();
  return cudaGetLastError();
}

}  // namespace rom
