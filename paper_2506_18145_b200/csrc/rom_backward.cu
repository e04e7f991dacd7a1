// Kernels of the layer's backward pass other than the scan's (rom_scan_bwd.cu) and the projections' data gradients
// (the forward grouped GEMMs run on transposed weights): transposes, the sum over a token's slots, the reverse of the
// gate-weighted combine, softplus / conv / router reverses and the weight gradients (sums over tokens).
//
// Section 5.1 trains the layer end to end and Appendix A.3 trains the router through the gate values; the equations
// differentiated are those of Sections 3.1 and 4.2 (forward: rom_api.cu).  This is the first, plain version: every
// kernel is a straightforward fp32-accumulating loop, weight gradients leave in fp32, and sums that cross thread
// blocks use floating-point atomics (their last bits vary from run to run).
#include "rom_internal.cuh"

namespace rom {
namespace {

template <typename T> struct VecN { static constexpr int N = 16 / sizeof(T); };

__device__ __forceinline__ void ldv(const __nv_bfloat16* p, float (&v)[8]) {
  const uint4 q = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) { v[2 * i] = __uint_as_float(w[i] << 16); v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u); }
}
__device__ __forceinline__ void ldv(const float* p, float (&v)[4]) {
  const float4 q = *reinterpret_cast<const float4*>(p);
  v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
}
__device__ __forceinline__ void stv(__nv_bfloat16* p, const float (&v)[8]) {
  uint4 q;
  uint32_t* w = reinterpret_cast<uint32_t*>(&q);
#pragma unroll
  for (int i = 0; i < 4; ++i) { const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]); w[i] = *reinterpret_cast<const uint32_t*>(&h); }
  *reinterpret_cast<uint4*>(p) = q;
}
__device__ __forceinline__ void stv(float* p, const float (&v)[4]) { *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]); }

// out[b][c][r] = in[b][r][c]
template <typename T>
__global__ void __launch_bounds__(256)
transpose_kernel(const T* __restrict__ in, T* __restrict__ out, int R, int C) {
  __shared__ T tile[32][33];
  const size_t base = (size_t)blockIdx.z * R * C;
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  for (int i = threadIdx.y; i < 32; i += 8) {
    const int r = r0 + i, c = c0 + threadIdx.x;
    if (r < R && c < C) tile[i][threadIdx.x] = in[base + (size_t)r * C + c];
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += 8) {
    const int c = c0 + i, r = r0 + threadIdx.x;
    if (r < R && c < C) out[base + (size_t)c * R + r] = tile[threadIdx.x][i];
  }
}

// out[c][r] = scale[r] * in[r][c] (activations transposed for the tensor-core weight gradient; scale = the row's gate)
template <typename T>
__global__ void __launch_bounds__(256)
transpose_scaled_kernel(const T* __restrict__ in, T* __restrict__ out, int R, int C, int ldo, const float* __restrict__ scale) {
  __shared__ float tile[32][33];
  const int c0 = blockIdx.x * 32, r0 = blockIdx.y * 32;
  for (int i = threadIdx.y; i < 32; i += 8) {
    const int r = r0 + i, c = c0 + threadIdx.x;
    if (r < R && c < C) tile[i][threadIdx.x] = to_f32(in[(size_t)r * C + c]) * (scale ? scale[r] : 1.0f);
  }
  __syncthreads();
  for (int i = threadIdx.y; i < 32; i += 8) {
    const int c = c0 + i, r = r0 + threadIdx.x;
    if (r < R && c < C) out[(size_t)c * ldo + r] = from_f32<T>(tile[threadIdx.x][i]);
  }
}

// dst[t, :] = sum_k src[row_of_assign[t*K + k], :]  (ascending k, fp32 accumulation), rows `width` wide
template <typename T>
__global__ void __launch_bounds__(256)
slot_sum_kernel(const T* __restrict__ src, const int32_t* __restrict__ row_of_assign, T* __restrict__ dst, int width, int K, long long total_vec) {
  constexpr int V = VecN<T>::N;
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total_vec) return;
  const int vpr = width / V;
  const long long t = i / vpr;
  const int c0 = (int)(i % vpr) * V;
  float acc[V];
#pragma unroll
  for (int j = 0; j < V; ++j) acc[j] = 0.0f;
  for (int k = 0; k < K; ++k) {
    float v[V];
    ldv(src + (size_t)row_of_assign[t * K + k] * width + c0, v);
#pragma unroll
    for (int j = 0; j < V; ++j) acc[j] += v[j];
  }
  stv(dst + t * width + c0, acc);
}

template <typename T>
__global__ void __launch_bounds__(256)
cast_f32_kernel(const T* __restrict__ in, float* __restrict__ out, long long n) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = to_f32(in[i]);
}

// Reverse of O_t = sum_k gate_k * (Yg_t W_out,k): with back_k = dO_t W_out,k (rows of dYgu, expert order),
//   dYg_t = sum_k gate_k back_k,  dgate_k = <back_k, Yg_t>;  also the gate of every padded row (scale of the weight gradient).
template <typename T>
__global__ void __launch_bounds__(128)
combine_bwd_kernel(const T* __restrict__ dYgu, const T* __restrict__ Ygp, const int32_t* __restrict__ row_of_assign,
                   const float* __restrict__ gates, T* __restrict__ dYg, float* __restrict__ dgate, float* __restrict__ rowscale,
                   int De, int K) {
  __shared__ float red[kMaxK][4];
  const size_t t = blockIdx.x;
  int rows[kMaxK]; float g[kMaxK], part[kMaxK];
  for (int k = 0; k < K; ++k) { rows[k] = row_of_assign[t * K + k]; g[k] = gates[t * K + k]; part[k] = 0.0f; }
  const T* yg = Ygp + (size_t)rows[0] * De;          // the K rows of a token hold the same gated scan output
  constexpr int V = V16<T>::N;
  if (De % V == 0) {                                   // 16-byte accesses
    for (int i = threadIdx.x; i < De / V; i += blockDim.x) {
      V16<T> q;
      float y[V], acc[V];
      q.load(yg + (size_t)i * V); q.get(y);
#pragma unroll
      for (int j = 0; j < V; ++j) acc[j] = 0.0f;
      for (int k = 0; k < K; ++k) {
        float bv[V];
        q.load(dYgu + (size_t)rows[k] * De + (size_t)i * V); q.get(bv);
#pragma unroll
        for (int j = 0; j < V; ++j) { acc[j] = fmaf(g[k], bv[j], acc[j]); part[k] = fmaf(bv[j], y[j], part[k]); }
      }
      V16<T>::store(dYg + t * De + (size_t)i * V, acc);
    }
  } else {
    for (int c = threadIdx.x; c < De; c += blockDim.x) {
      const float y = to_f32(yg[c]);
      float acc = 0.0f;
      for (int k = 0; k < K; ++k) {
        const float b = to_f32(dYgu[(size_t)rows[k] * De + c]);
        acc = fmaf(g[k], b, acc);
        part[k] = fmaf(b, y, part[k]);
      }
      dYg[t * De + c] = from_f32<T>(acc);
    }
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int k = 0; k < K; ++k) {
    float v = part[k];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (lane == 0) red[k][warp] = v;
  }
  __syncthreads();
  if (threadIdx.x < K) {
    const int k = threadIdx.x;
    dgate[t * K + k] = (red[k][0] + red[k][1]) + (red[k][2] + red[k][3]);
    rowscale[rows[k]] = g[k];
  }
}

// Reverse of Delta = softplus(pre): dpre = dDelta * sigmoid(pre) = dDelta * (1 - exp(-Delta)); db_dt[c] = sum_t dpre.
template <typename T>
__global__ void __launch_bounds__(256)
softplus_bwd_kernel(const float* __restrict__ ddelta, const float* __restrict__ Delta32, T* __restrict__ dpre, float* __restrict__ db_dt,
                    long long Tn, int De) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= De) return;
  const long long t0 = (long long)blockIdx.y * 64, t1 = min(t0 + 64, Tn);
  float s = 0.0f;
  for (long long t = t0; t < t1; ++t) {
    const float v = ddelta[t * De + c] * (-expm1f(-Delta32[t * De + c]));
    dpre[t * De + c] = from_f32<T>(v);
    s += v;
  }
  atomicAdd(db_dt + c, s);
}

// dxdbl[t, R + j] = dB[t, j] (j < N) or dC[t, j - N]: the B | C part of the gradient of (delta, B, C) = U W_x
template <typename T>
__global__ void __launch_bounds__(256)
pack_bc_kernel(const float* __restrict__ dBm, const float* __restrict__ dCm, T* __restrict__ dxdbl, long long Tn, int R, int N) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= Tn * 2 * N) return;
  const long long t = i / (2 * N);
  const int j = (int)(i % (2 * N));
  dxdbl[t * (R + 2 * N) + R + j] = from_f32<T>(j < N ? dBm[t * N + j] : dCm[t * N + (j - N)]);
}

// Reverse of U = SiLU(b + sum_j w[j] H[t - (k-1-j)]) for a segment of 64 steps of one channel per thread:
//   g_t = dU_t SiLU'(pre_t);  dH_tau = sum_j w[j] g_{tau + (k-1-j)};  dw[j] = sum_t g_t H[t - (k-1-j)];  db = sum_t g_t.
// H is the left half of HZ ([T, 2 De]); dU = dU1 + dU2 (scan part + x Proj part); dH goes to the left half of dHZ.
constexpr int CSEG = 64;
template <typename T>
__global__ void __launch_bounds__(128)
conv_bwd_kernel(const T* __restrict__ HZ, const T* __restrict__ w_conv, const float* __restrict__ b_conv, const T* __restrict__ dU1,
                const T* __restrict__ dU2, T* __restrict__ dHZ, float* __restrict__ dw, float* __restrict__ db, int L, int De, int k) {
  const int c = blockIdx.x * blockDim.x + threadIdx.x;
  if (c >= De) return;
  const size_t tok0 = (size_t)blockIdx.z * L;
  const int t0 = blockIdx.y * CSEG, t1 = min(t0 + CSEG, L), t_end = min(t1 + k - 1, L);
  const int ld = 2 * De;
  float w[4] = {0.0f, 0.0f, 0.0f, 0.0f}, hw[4] = {0.0f, 0.0f, 0.0f, 0.0f}, dacc[4] = {0.0f, 0.0f, 0.0f, 0.0f}, dwl[4] = {0.0f, 0.0f, 0.0f, 0.0f};
  for (int j = 0; j < k; ++j) w[j] = to_f32(w_conv[(size_t)j * De + c]);
  const float bias = b_conv ? b_conv[c] : 0.0f;
  float dbl = 0.0f;
  // hw[j] = H[t - (k-1-j)]: before step t0 the window holds H[t0-k+1 .. t0-1] in hw[1 .. k-1]
  for (int j = 1; j < k; ++j) {
    const int t = t0 - k + j;
    hw[j] = t >= 0 ? to_f32(HZ[(tok0 + t) * ld + c]) : 0.0f;
  }
  constexpr int G = 8;                      // steps whose loads are in flight together
  for (int tg = t0; tg < t_end; tg += G) {
    float hz[G], d1[G], d2[G];
#pragma unroll
    for (int i = 0; i < G; ++i) {
      const int t = min(tg + i, t_end - 1);
      hz[i] = to_f32(HZ[(tok0 + t) * ld + c]);
      d1[i] = to_f32(dU1[(tok0 + t) * De + c]);
      d2[i] = to_f32(dU2[(tok0 + t) * De + c]);
    }
#pragma unroll
    for (int i = 0; i < G; ++i) {
      const int t = tg + i;
      if (t >= t_end) break;
      for (int j = 0; j + 1 < k; ++j) hw[j] = hw[j + 1];
      hw[k - 1] = hz[i];
      float pre = bias;
      for (int j = 0; j < k; ++j) pre = fmaf(w[j], hw[j], pre);
      const float sg = 1.0f / (1.0f + expf(-pre));
      const float g = (d1[i] + d2[i]) * sg * (1.0f + pre * (1.0f - sg));
      if (t < t1) {
        dbl += g;
        for (int j = 0; j < k; ++j) dwl[j] = fmaf(g, hw[j], dwl[j]);
      }
      // dacc[i] collects dH of step t - (k-1) + i; after this step's terms, index 0 is complete
      for (int j = 0; j < k; ++j) dacc[j] = fmaf(w[j], g, dacc[j]);
      const int tau = t - (k - 1);
      if (tau >= t0) dHZ[(tok0 + tau) * ld + c] = from_f32<T>(dacc[0]);
      for (int j = 0; j + 1 < k; ++j) dacc[j] = dacc[j + 1];
      dacc[k - 1] = 0.0f;
    }
  }
  // steps whose later neighbours do not exist (end of the sequence): what has been collected is final
  for (int i = 0; i + 1 < k; ++i) {
    const int tau = t_end - (k - 1) + i;
    if (tau >= t0 && tau < t1) dHZ[(tok0 + tau) * ld + c] = from_f32<T>(dacc[i]);
  }
  for (int j = 0; j < k; ++j) atomicAdd(dw + (size_t)j * De + c, dwl[j]);
  atomicAdd(db + c, dbl);
}

// Reverse of the gate values with the selected set held fixed (one warp per token): logits and softmax are recomputed,
// dP[idx_k] = dgate_k (gate_mode 0) or (dgate_k - sum_j dgate_j gate_j) / sum_j P[idx_j] (gate_mode 1),
// dlogit = P (dP - sum_e dP_e P_e).  Writes dlogit [T, E] (fp32) and adds db_r.
template <typename T>
__global__ void __launch_bounds__(256)
router_bwd_kernel(const T* __restrict__ x, const T* __restrict__ W_r, const float* __restrict__ b_r, const int32_t* __restrict__ idx,
                  const float* __restrict__ gates, const float* __restrict__ dgate, float* __restrict__ dlogit, float* __restrict__ db_r,
                  long long Tn, int Dm, int E, int K, int gate_mode) {
  const int lane = threadIdx.x & 31;
  const long long t = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (t >= Tn) return;
  float lg[2] = {0.0f, 0.0f};              // lane e & 31 holds logit[e] in lg[e >> 5]
  for (int e = 0; e < E; ++e) {
    float s = 0.0f;
    for (int d = lane; d < Dm; d += 32) s = fmaf(to_f32(x[t * Dm + d]), to_f32(W_r[(size_t)e * Dm + d]), s);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    s += b_r ? b_r[e] : 0.0f;
    if ((e & 31) == lane) lg[e >> 5] = s;
  }
  // softmax over E (two values per lane at most)
  float m = -INFINITY;
  for (int h = 0; h < 2; ++h) if (lane + 32 * h < E) m = fmaxf(m, lg[h]);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  float p[2] = {0.0f, 0.0f}, den = 0.0f;
  for (int h = 0; h < 2; ++h) if (lane + 32 * h < E) { p[h] = expf(lg[h] - m); den += p[h]; }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) den += __shfl_xor_sync(0xffffffffu, den, o);
  p[0] /= den; p[1] /= den;
  // dP on the selected experts
  float S = 1.0f, dot = 0.0f;
  if (gate_mode == 1) {
    S = 0.0f;
    for (int k = 0; k < K; ++k) {
      const int e = idx[t * K + k];
      S += __shfl_sync(0xffffffffu, p[e >> 5], e & 31);
      dot = fmaf(dgate[t * K + k], gates[t * K + k], dot);
    }
  }
  float dP[2] = {0.0f, 0.0f};
  for (int k = 0; k < K; ++k) {
    const int e = idx[t * K + k];
    const float ds = gate_mode == 1 ? (dgate[t * K + k] - dot) / S : dgate[t * K + k];
    if ((e & 31) == lane) dP[e >> 5] += ds;
  }
  float mean = dP[0] * p[0] + dP[1] * p[1];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) mean += __shfl_xor_sync(0xffffffffu, mean, o);
  for (int h = 0; h < 2; ++h) {
    const int e = lane + 32 * h;
    if (e < E) {
      const float dl = p[h] * (dP[h] - mean);
      dlogit[t * E + e] = dl;
      if (db_r) atomicAdd(db_r + e, dl);
    }
  }
}

// dx[t, :] = sum_k dxp[row(t,k), :] + sum_e dlogit[t, e] W_r[e, :]
template <typename T>
__global__ void __launch_bounds__(256)
dx_kernel(const T* __restrict__ dxp, const int32_t* __restrict__ row_of_assign, const float* __restrict__ dlogit, const T* __restrict__ W_r,
          T* __restrict__ dx, int Dm, int E, int K, long long total_vec) {
  constexpr int V = VecN<T>::N;
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= total_vec) return;
  const int vpr = Dm / V;
  const long long t = i / vpr;
  const int c0 = (int)(i % vpr) * V;
  float acc[V];
#pragma unroll
  for (int j = 0; j < V; ++j) acc[j] = 0.0f;
  for (int k = 0; k < K; ++k) {
    float v[V];
    ldv(dxp + (size_t)row_of_assign[t * K + k] * Dm + c0, v);
#pragma unroll
    for (int j = 0; j < V; ++j) acc[j] += v[j];
  }
  for (int e = 0; e < E; ++e) {
    const float dl = dlogit[t * E + e];
    float v[V];
    ldv(W_r + (size_t)e * Dm + c0, v);
#pragma unroll
    for (int j = 0; j < V; ++j) acc[j] = fmaf(dl, v[j], acc[j]);
  }
  stv(dx + t * Dm + c0, acc);
}

// dW_r[e, d] = sum_t dlogit[t, e] x[t, d]: the tokens are cut into slabs of 1024, one atomic per slab and element
template <typename T>
__global__ void __launch_bounds__(128)
router_wgrad_kernel(const float* __restrict__ dlogit, const T* __restrict__ x, float* __restrict__ dW_r, long long Tn, int Dm, int E) {
  const int d = blockIdx.x * blockDim.x + threadIdx.x;
  if (d >= Dm) return;
  const int e = blockIdx.y;
  const long long t0 = (long long)blockIdx.z * 1024, t1 = min(t0 + 1024, Tn);
  float s = 0.0f;
  for (long long t = t0; t < t1; ++t) s = fmaf(dlogit[t * E + e], to_f32(x[t * Dm + d]), s);
  atomicAdd(dW_r + (size_t)e * Dm + d, s);
}

// Weight gradient of a (grouped) projection: C[s][p, q] = sum over the rows r of segment s of scale[r] X[r, p] Y[r, q]
// (X, Y row-major with the contracted index, the token row, outermost).  64 x 64 outputs per block, 4 x 4 per thread,
// 16 rows per step through shared memory; fp32 accumulation and output.  seg == nullptr: one segment [0, rows_total).
template <typename T>
__global__ void __launch_bounds__(256)
wgrad_kernel(const T* __restrict__ X, int ldx, const T* __restrict__ Y, int ldy, const float* __restrict__ scale,
             const int32_t* __restrict__ seg, int rows_total, int P, int Q, float* __restrict__ C) {
  __shared__ float Xs[16][64 + 4];
  __shared__ float Ys[16][64 + 4];
  const int s = blockIdx.z;
  const int r0 = seg ? seg[s] : 0, r1 = seg ? seg[s + 1] : rows_total;
  const int p0 = blockIdx.y * 64, q0 = blockIdx.x * 64;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  const int lr = threadIdx.x >> 4, lc = (threadIdx.x & 15) * 4;       // loader: row lr of the step, 4 consecutive columns from lc
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;
  for (int r = r0; r < r1; r += 16) {
    const int row = r + lr;
    const bool in = row < r1;
    const float sc = (in && scale) ? scale[row] : 1.0f;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int p = p0 + lc + j, q = q0 + lc + j;
      Xs[lr][lc + j] = (in && p < P) ? sc * to_f32(X[(size_t)row * ldx + p]) : 0.0f;
      Ys[lr][lc + j] = (in && q < Q) ? to_f32(Y[(size_t)row * ldy + q]) : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      float xa[4], yb[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { xa[i] = Xs[kk][ty * 4 + i]; yb[i] = Ys[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(xa[i], yb[j], acc[i][j]);
    }
    __syncthreads();
  }
  float* Cs = C + (size_t)s * P * Q;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int p = p0 + ty * 4 + i, q = q0 + tx * 4 + j;
      if (p < P && q < Q) Cs[(size_t)p * Q + q] = acc[i][j];
    }
}

}  // namespace

cudaError_t launch_transpose(int dtype, const void* in, void* out, int batch, int R, int C, cudaStream_t st) {
  const dim3 grid((C + 31) / 32, (R + 31) / 32, batch), block(32, 8);
  if (dtype == ROM_BF16) transpose_kernel<__nv_bfloat16><<<grid, block, 0, st>>>((const __nv_bfloat16*)in, (__nv_bfloat16*)out, R, C);
  else transpose_kernel<float><<<grid, block, 0, st>>>((const float*)in, (float*)out, R, C);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_transpose_scaled(int dtype, const void* in, void* out, int R, int C, int ldo, const float* scale, cudaStream_t st) {
  const dim3 grid((C + 31) / 32, (R + 31) / 32), block(32, 8);
  if (dtype == ROM_BF16) transpose_scaled_kernel<__nv_bfloat16><<<grid, block, 0, st>>>((const __nv_bfloat16*)in, (__nv_bfloat16*)out, R, C, ldo, scale);
  else transpose_scaled_kernel<float><<<grid, block, 0, st>>>((const float*)in, (float*)out, R, C, ldo, scale);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_slot_sum(int dtype, const void* src, const int32_t* row_of_assign, void* dst, long long Tn, int width, int K, cudaStream_t st) {
  const long long total = Tn * (width / (dtype == ROM_BF16 ? 8 : 4));
  const unsigned blocks = (unsigned)((total + 255) / 256);
  if (dtype == ROM_BF16) slot_sum_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)src, row_of_assign, (__nv_bfloat16*)dst, width, K, total);
  else slot_sum_kernel<float><<<blocks, 256, 0, st>>>((const float*)src, row_of_assign, (float*)dst, width, K, total);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_cast_f32(int dtype, const void* in, float* out, long long n, cudaStream_t st) {
  const unsigned blocks = (unsigned)((n + 255) / 256);
  if (dtype == ROM_BF16) cast_f32_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)in, out, n);
  else cast_f32_kernel<float><<<blocks, 256, 0, st>>>((const float*)in, out, n);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_combine_bwd(int dtype, const void* dYgu, const void* Ygp, const int32_t* row_of_assign, const float* gates, void* dYg,
                               float* dgate, float* rowscale, long long Tn, int De, int K, cudaStream_t st) {
  if (dtype == ROM_BF16)
    combine_bwd_kernel<__nv_bfloat16><<<(unsigned)Tn, 128, 0, st>>>((const __nv_bfloat16*)dYgu, (const __nv_bfloat16*)Ygp, row_of_assign, gates,
                                                                  (__nv_bfloat16*)dYg, dgate, rowscale, De, K);
  else
    combine_bwd_kernel<float><<<(unsigned)Tn, 128, 0, st>>>((const float*)dYgu, (const float*)Ygp, row_of_assign, gates, (float*)dYg, dgate,
                                                          rowscale, De, K);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_softplus_bwd(int dtype, const float* ddelta, const float* Delta32, void* dpre, float* db_dt, long long Tn, int De, cudaStream_t st) {
  const dim3 grid((De + 255) / 256, (unsigned)((Tn + 63) / 64));
  if (dtype == ROM_BF16) softplus_bwd_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(ddelta, Delta32, (__nv_bfloat16*)dpre, db_dt, Tn, De);
  else softplus_bwd_kernel<float><<<grid, 256, 0, st>>>(ddelta, Delta32, (float*)dpre, db_dt, Tn, De);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_pack_bc(int dtype, const float* dBm, const float* dCm, void* dxdbl, long long Tn, int R, int N, cudaStream_t st) {
  const unsigned blocks = (unsigned)((Tn * 2 * N + 255) / 256);
  if (dtype == ROM_BF16) pack_bc_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(dBm, dCm, (__nv_bfloat16*)dxdbl, Tn, R, N);
  else pack_bc_kernel<float><<<blocks, 256, 0, st>>>(dBm, dCm, (float*)dxdbl, Tn, R, N);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_conv_bwd(const rom_config& c, const void* HZ, const void* w_conv, const float* b_conv, const void* dU1, const void* dU2,
                            void* dHZ, float* dw, float* db, cudaStream_t st) {
  const dim3 grid((c.d_inner + 127) / 128, (c.L + CSEG - 1) / CSEG, c.B);
  if (c.dtype == ROM_BF16)
    conv_bwd_kernel<__nv_bfloat16><<<grid, 128, 0, st>>>((const __nv_bfloat16*)HZ, (const __nv_bfloat16*)w_conv, b_conv, (const __nv_bfloat16*)dU1,
                                                       (const __nv_bfloat16*)dU2, (__nv_bfloat16*)dHZ, dw, db, c.L, c.d_inner, c.d_conv);
  else
    conv_bwd_kernel<float><<<grid, 128, 0, st>>>((const float*)HZ, (const float*)w_conv, b_conv, (const float*)dU1, (const float*)dU2, (float*)dHZ,
                                               dw, db, c.L, c.d_inner, c.d_conv);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_router_bwd(const rom_config& c, const void* x, const void* W_r, const float* b_r, const int32_t* idx, const float* gates,
                              const float* dgate, float* dlogit, float* db_r, float* dW_r, cudaStream_t st) {
  const long long Tn = (long long)c.B * c.L;
  const unsigned blocks = (unsigned)((Tn + 7) / 8);
  const dim3 wgrid((c.d_model + 127) / 128, c.E, (unsigned)((Tn + 1023) / 1024));
  if (c.dtype == ROM_BF16) {
    router_bwd_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)x, (const __nv_bfloat16*)W_r, b_r, idx, gates, dgate, dlogit, db_r,
                                                           Tn, c.d_model, c.E, c.K, c.gate_mode);
    count_launch();
    router_wgrad_kernel<__nv_bfloat16><<<wgrid, 128, 0, st>>>(dlogit, (const __nv_bfloat16*)x, dW_r, Tn, c.d_model, c.E);
  } else {
    router_bwd_kernel<float><<<blocks, 256, 0, st>>>((const float*)x, (const float*)W_r, b_r, idx, gates, dgate, dlogit, db_r, Tn, c.d_model, c.E,
                                                   c.K, c.gate_mode);
    count_launch();
    router_wgrad_kernel<float><<<wgrid, 128, 0, st>>>(dlogit, (const float*)x, dW_r, Tn, c.d_model, c.E);
  }
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_dx(const rom_config& c, const void* dxp, const int32_t* row_of_assign, const float* dlogit, const void* W_r, void* dx,
                      cudaStream_t st) {
  const long long total = (long long)c.B * c.L * (c.d_model / (c.dtype == ROM_BF16 ? 8 : 4));
  const unsigned blocks = (unsigned)((total + 255) / 256);
  if (c.dtype == ROM_BF16)
    dx_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>((const __nv_bfloat16*)dxp, row_of_assign, dlogit, (const __nv_bfloat16*)W_r, (__nv_bfloat16*)dx,
                                                   c.d_model, c.E, c.K, total);
  else
    dx_kernel<float><<<blocks, 256, 0, st>>>((const float*)dxp, row_of_assign, dlogit, (const float*)W_r, (float*)dx, c.d_model, c.E, c.K, total);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_wgrad(int dtype, const void* X, int ldx, const void* Y, int ldy, const float* scale, const int32_t* seg, int n_seg,
                         int rows_total, int P, int Q, float* C, cudaStream_t st) {
  const dim3 grid((Q + 63) / 64, (P + 63) / 64, n_seg);
  if (dtype == ROM_BF16)
    wgrad_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)X, ldx, (const __nv_bfloat16*)Y, ldy, scale, seg, rows_total, P, Q, C);
  else
    wgrad_kernel<float><<<grid, 256, 0, st>>>((const float*)X, ldx, (const float*)Y, ldy, scale, seg, rows_total, P, Q, C);
  count_launch();
  return cudaGetLastError();
}

}  // namespace rom
