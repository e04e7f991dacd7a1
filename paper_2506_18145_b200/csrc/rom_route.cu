// Router, top-K and dropless permutation (Section 4.2 routing equation; Section 5.1: no capacity
// factor and no token dropping), plus the row gather that feeds the grouped Conv/Gate projection.
//
// Kernels
//   route_weights_f64 : W_r in fp64, experts padded to a multiple of 8, once per call.
//   route_logits_topk : logits in fp64 on the tensor cores (products of bf16 or fp32 inputs are exact in
//                       fp64; every expert's sum is taken in the same order, so ties stay ties), softmax,
//                       top-K with ties to the lowest expert id, per-chunk histogram.
//   route_offsets     : per-expert exclusive scan of the chunk histograms (warp shuffles), expert
//                       offsets, offsets padded to the GEMM row tile, row-tile -> expert map.
//   route_scatter     : stable rank of every assignment inside its chunk by warp ballots; writes
//                       perm / inv_perm and the padded-row tables.
//   gather_rows       : x_perm[row] = x[token of row] (zero rows in the padding).
#include "rom_internal.cuh"

namespace rom {
namespace {

constexpr int RT = kChunkTokens;   // tokens per block of route_logits_topk = one routing chunk
constexpr int NT8 = 8;             // experts per warp (one fp64 MMA column tile)

// Wd[e][d] = (double) W_r[e][d], experts padded with zero rows to a multiple of 8: the router weights in the
// precision and layout the MMA fragments are loaded in (four consecutive d of one expert = 32 bytes).
template <typename T>
__global__ void __launch_bounds__(256)
route_weights_f64(const T* __restrict__ W_r, double* __restrict__ Wd, int Dm, int E, int Epad) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= Dm * Epad) return;
  const int e = i / Dm;
  Wd[i] = e < E ? (double)to_f32(W_r[i]) : 0.0;
}

// D (8x8) += A (8x4, row) * B (4x8, col), all fp64, on the tensor cores.  Lane l holds A[l/4][l%4], B[l%4][l/4]
// and D[l/4][2*(l%4) + {0,1}].
__device__ __forceinline__ void dmma_m8n8k4(double (&d)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0, %1}, {%2}, {%3}, {%0, %1};"
               : "+d"(d[0]), "+d"(d[1]) : "d"(a), "d"(b));
}
// four consecutive elements of a row, kept as loaded and widened to fp64 when used
template <typename T> struct RawX4;
template <> struct RawX4<__nv_bfloat16> {
  uint2 v;
  __device__ __forceinline__ void load(const __nv_bfloat16* p) { v = __ldg(reinterpret_cast<const uint2*>(p)); }
  __device__ __forceinline__ void get(double (&xd)[4]) const {
    xd[0] = (double)__uint_as_float(v.x << 16); xd[1] = (double)__uint_as_float(v.x & 0xffff0000u);
    xd[2] = (double)__uint_as_float(v.y << 16); xd[3] = (double)__uint_as_float(v.y & 0xffff0000u);
  }
};
template <> struct RawX4<float> {
  float4 v;
  __device__ __forceinline__ void load(const float* p) { v = __ldg(reinterpret_cast<const float4*>(p)); }
  __device__ __forceinline__ void get(double (&xd)[4]) const { xd[0] = v.x; xd[1] = v.y; xd[2] = v.z; xd[3] = v.w; }
};

// One block = 32 tokens (one routing chunk); warp w computes the logits of experts [8w, 8w+8) for them with
// fp64 tensor-core MMAs (products of bf16/fp32 inputs are exact in fp64; every expert column is accumulated
// in the same order, so equal weight rows give bit-equal logits and ties stay ties).  Per 16 elements of
// d_model a lane reads 4 consecutive elements of one token row per 8-token tile (32-byte sectors, straight
// from global memory) and 4 consecutive fp64 weights of one expert (L1/L2-resident copy); MMA j of the step
// contracts elements {j, 4+j, 8+j, 12+j} of the 16.  No shared memory until the logits meet for the top-K.
template <typename T>
__global__ void __launch_bounds__(512)
route_logits_topk(const T* __restrict__ x, const double* __restrict__ Wd, const float* __restrict__ b_r,
                  int T_tokens, int Dm, int E, int K, int gate_mode,
                  int32_t* __restrict__ topk_idx, float* __restrict__ gates,
                  int32_t* __restrict__ chunk_counts, double* __restrict__ chunk_prob) {
  extern __shared__ __align__(16) unsigned char smem[];
  const int Epad = (E + NT8 - 1) / NT8 * NT8;
  const int n_wtiles = Epad / NT8;
  const int dsplit = (blockDim.x >> 5) / n_wtiles;                 // warps that share one expert tile, each on its own d range
  double* lg = reinterpret_cast<double*>(smem);                    // [dsplit][RT][Epad] partial logits; [0] becomes the sum
  int32_t* idx_s = reinterpret_cast<int32_t*>(lg + dsplit * RT * Epad);   // [RT][K]

  const int tid = threadIdx.x;
  const int lane = tid & 31, wq = tid >> 5;
  const int w = wq / dsplit, dq = wq % dsplit;                     // expert tile, d range [dq, dq+1) * Dm / dsplit
  const int d_lo = (Dm / 16 * dq / dsplit) * 16, d_hi = (Dm / 16 * (dq + 1) / dsplit) * 16;
  const int gq = lane >> 2, t4 = lane & 3;                        // fragment row / column group of this lane
  const int t0 = blockIdx.x * RT;

  // accumulators: 4 tiles of 8 tokens x this warp's 8 experts; lane holds (token 8*mt + gq, experts 2*t4, 2*t4+1)
  double acc[4][2];
#pragma unroll
  for (int mt = 0; mt < 4; ++mt) {
#pragma unroll
    for (int i = 0; i < 2; ++i) {
      const int ee = w * NT8 + 2 * t4 + i;
      acc[mt][i] = (b_r != nullptr && ee < E && dq == 0) ? (double)b_r[ee] : 0.0;
    }
  }
  const T* xrow[4];
#pragma unroll
  for (int mt = 0; mt < 4; ++mt) xrow[mt] = x + (size_t)min(t0 + 8 * mt + gq, T_tokens - 1) * Dm + 4 * t4;   // rows past the end repeat the last token
  const double* wrow = Wd + (size_t)(w * NT8 + gq) * Dm + 4 * t4;

  // operands of the next PF-1 steps are in flight (raw, unconverted) while one step is contracted
  // (d_model is a multiple of 64, so there are at least PF steps)
  constexpr int PF = 4;
  RawX4<T> rx[PF][4];
  double2 rw[PF][2];
  auto fetch = [&](int d, RawX4<T> (&xo)[4], double2 (&wo)[2]) {
#pragma unroll
    for (int mt = 0; mt < 4; ++mt) xo[mt].load(xrow[mt] + d);
    wo[0] = __ldg(reinterpret_cast<const double2*>(wrow + d));
    wo[1] = __ldg(reinterpret_cast<const double2*>(wrow + d) + 1);
  };
#pragma unroll
  for (int i = 0; i < PF - 1; ++i)
    if (d_lo + 16 * i < d_hi) fetch(d_lo + 16 * i, rx[i], rw[i]);
  for (int d0 = d_lo; d0 < d_hi; d0 += 16 * PF) {
#pragma unroll
    for (int i = 0; i < PF; ++i) {
      if (d0 + 16 * i >= d_hi) break;
      const int dn = d0 + 16 * (i + PF - 1);                              // step that enters the ring now
      if (dn < d_hi) fetch(dn, rx[(i + PF - 1) % PF], rw[(i + PF - 1) % PF]);
      const double wb[4] = {rw[i][0].x, rw[i][0].y, rw[i][1].x, rw[i][1].y};
      double xa[4][4];
#pragma unroll
      for (int mt = 0; mt < 4; ++mt) rx[i][mt].get(xa[mt]);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
#pragma unroll
        for (int mt = 0; mt < 4; ++mt) dmma_m8n8k4(acc[mt], xa[mt][j], wb[j]);
      }
    }
  }
#pragma unroll
  for (int mt = 0; mt < 4; ++mt) {
    lg[(dq * RT + 8 * mt + gq) * Epad + w * NT8 + 2 * t4] = acc[mt][0];
    lg[(dq * RT + 8 * mt + gq) * Epad + w * NT8 + 2 * t4 + 1] = acc[mt][1];
  }
  __syncthreads();

  // the d ranges are added in a fixed order, the same for every expert
  for (int i = tid; i < RT * Epad; i += blockDim.x) {
    double v = lg[i];
    for (int q = 1; q < dsplit; ++q) v += lg[q * RT * Epad + i];
    lg[i] = v;
  }
  __syncthreads();

  if (tid < RT) {
    const int t = t0 + tid;
    const double* l = lg + tid * Epad;
    double m = -INFINITY, denom = 1.0;
    if (t < T_tokens) {
      for (int e = 0; e < E; ++e) { double v = l[e]; if (v > m) m = v; }   // NaN never raises m
      denom = 0.0;
      for (int e = 0; e < E; ++e) denom += exp(l[e] - m);
      unsigned long long taken = 0ull;
      double gsel[kMaxK];
      int isel[kMaxK];
      double gsum = 0.0;
      for (int k = 0; k < K; ++k) {
        int best = -1; double bestv = -INFINITY;
        for (int e = 0; e < E; ++e) {
          if ((taken >> e) & 1ull) continue;
          double v = l[e];
          if (v != v) v = -INFINITY;
          if (best < 0 || v > bestv) { best = e; bestv = v; }
        }
        taken |= 1ull << best;
        isel[k] = best;
        gsel[k] = exp(l[best] - m) / denom;
        gsum += gsel[k];
      }
      for (int k = 0; k < K; ++k) {
        const double gk = (gate_mode == 1) ? gsel[k] / gsum : gsel[k];
        idx_s[tid * K + k] = isel[k];
        if (topk_idx) topk_idx[(size_t)t * K + k] = isel[k];
        if (gates) gates[(size_t)t * K + k] = (float)gk;
      }
    } else {
      for (int k = 0; k < K; ++k) idx_s[tid * K + k] = -1;
    }
    // optional: sum over the chunk's tokens of Softmax(X W_r), per expert (Appendix A.3 statistic); the lanes are
    // added in a fixed shuffle order, so the result does not depend on scheduling
    if (chunk_prob != nullptr) {
      for (int e = 0; e < E; ++e) {
        double pe = t < T_tokens ? exp(l[e] - m) / denom : 0.0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) pe += __shfl_down_sync(0xffffffffu, pe, o);
        if (tid == 0) chunk_prob[(size_t)blockIdx.x * E + e] = pe;
      }
    }
    // histogram of this chunk by warp ballots (warp 0 holds all 32 tokens)
    for (int e = 0; e < E; ++e) {
      int c = 0;
      for (int k = 0; k < K; ++k) c += __popc(__ballot_sync(0xffffffffu, idx_s[tid * K + k] == e));
      if (tid == 0) chunk_counts[(size_t)blockIdx.x * E + e] = c;
    }
  }
}

// One block.  Warp w scans the chunk histogram of experts w, w+32, ... over all chunks.
__global__ void __launch_bounds__(1024)
route_offsets(int32_t* __restrict__ chunk_counts, int n_chunks, int E,
              int32_t* __restrict__ counts_ws, int32_t* __restrict__ offsets_ws, int32_t* __restrict__ pad_offsets,
              int32_t* __restrict__ num_m_tiles, int32_t* __restrict__ tile_expert, int max_m_tiles,
              int32_t* __restrict__ counts_out, int32_t* __restrict__ offsets_out) {
  __shared__ int32_t cnt[kMaxE];
  __shared__ int32_t off[kMaxE + 1];
  __shared__ int32_t poff[kMaxE + 1];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
  for (int e = warp; e < E; e += nwarps) {
    int carry = 0;
    constexpr int UB = 8;                         // chunks-of-32 whose loads are issued together
    for (int cb = 0; cb < n_chunks; cb += 32 * UB) {
      int vv[UB];
#pragma unroll
      for (int i = 0; i < UB; ++i) {
        const int c = cb + 32 * i + lane;
        vv[i] = (c < n_chunks) ? chunk_counts[(size_t)c * E + e] : 0;
      }
#pragma unroll
      for (int i = 0; i < UB; ++i) {
        const int c = cb + 32 * i + lane;
        const int v = vv[i];
        int inc = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          int n = __shfl_up_sync(0xffffffffu, inc, o);
          if (lane >= o) inc += n;
        }
        if (c < n_chunks) chunk_counts[(size_t)c * E + e] = carry + inc - v;    // exclusive base
        carry += __shfl_sync(0xffffffffu, inc, 31);
      }
    }
    if (lane == 0) cnt[e] = carry;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int o = 0, p = 0;
    for (int e = 0; e < E; ++e) {
      off[e] = o; poff[e] = p;
      o += cnt[e];
      p += (cnt[e] + kTileM - 1) / kTileM * kTileM;
    }
    off[E] = o; poff[E] = p;
    *num_m_tiles = p / kTileM;
  }
  __syncthreads();
  for (int e = threadIdx.x; e <= E; e += blockDim.x) {
    offsets_ws[e] = off[e];
    pad_offsets[e] = poff[e];
    if (offsets_out) offsets_out[e] = off[e];
    if (e < E) {
      counts_ws[e] = cnt[e];
      if (counts_out) counts_out[e] = cnt[e];
    }
  }
  const int ntiles = poff[E] / kTileM;
  for (int i = threadIdx.x; i < max_m_tiles; i += blockDim.x) {
    int ex = -1;
    if (i < ntiles) {
      const int row = i * kTileM;
      for (int e = 0; e < E; ++e)
        if (row >= poff[e] && row < poff[e + 1]) ex = e;
    }
    tile_expert[i] = ex;
  }
}

// One warp per chunk of 32 tokens.
__global__ void __launch_bounds__(256)
route_scatter(const int32_t* __restrict__ topk_idx, const int32_t* __restrict__ chunk_base,
              const int32_t* __restrict__ offsets, const int32_t* __restrict__ pad_offsets,
              int T_tokens, int E, int K, int n_chunks,
              int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm,
              int32_t* __restrict__ row_of_assign, int32_t* __restrict__ assign_of_row) {
  const int lane = threadIdx.x & 31;
  const int chunk = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (chunk >= n_chunks) return;
  const int t = chunk * kChunkTokens + lane;
  int my_e[kMaxK], my_rank[kMaxK];
  for (int k = 0; k < K; ++k) {
    my_e[k] = (t < T_tokens) ? topk_idx[(size_t)t * K + k] : -1;
    my_rank[k] = 0;
  }
  const unsigned lt = (1u << lane) - 1u;
  for (int e = 0; e < E; ++e) {
    int before = 0;      // assignments of expert e held by lower tokens of this chunk
    for (int k = 0; k < K; ++k) before += __popc(__ballot_sync(0xffffffffu, my_e[k] == e) & lt);
    for (int k = 0; k < K; ++k)
      if (my_e[k] == e) my_rank[k] = before;    // a token's K experts are distinct
  }
  if (t >= T_tokens) return;
  for (int k = 0; k < K; ++k) {
    const int e = my_e[k];
    const int a = t * K + k;
    const int within = chunk_base[(size_t)chunk * E + e] + my_rank[k];
    const int r = offsets[e] + within;
    const int pr = pad_offsets[e] + within;
    if (perm) perm[r] = a;
    if (inv_perm) inv_perm[a] = r;
    row_of_assign[a] = pr;
    assign_of_row[pr] = a;
  }
}

// Routing decision given from outside (a later layer that reuses it): one warp per chunk of 32 tokens counts the
// chunk's assignments per expert.  Indices outside [0, E) are clamped into range in the working copy idx_ws
// (so every later table stays in bounds) and reported through the status word.
__global__ void __launch_bounds__(256)
idx_chunk_histogram(const int32_t* __restrict__ topk_idx, int32_t* __restrict__ idx_ws, int T_tokens, int E, int K, int n_chunks,
                    int32_t* __restrict__ chunk_counts, int32_t* __restrict__ status) {
  const int lane = threadIdx.x & 31;
  const int chunk = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (chunk >= n_chunks) return;
  const int t = chunk * kChunkTokens + lane;
  int my_e[kMaxK];
  bool bad = false;
  for (int k = 0; k < K; ++k) {
    int e = -1;
    if (t < T_tokens) {
      e = topk_idx[(size_t)t * K + k];
      if (e < 0 || e >= E) { bad = true; e = min(max(e, 0), E - 1); }
      idx_ws[(size_t)t * K + k] = e;
    }
    my_e[k] = e;
  }
  if (bad) atomicExch(status + kStatCode, ROM_ERR_INVALID_ARG);
  for (int e = 0; e < E; ++e) {
    int c = 0;
    for (int k = 0; k < K; ++k) c += __popc(__ballot_sync(0xffffffffu, my_e[k] == e));
    if (lane == 0) chunk_counts[(size_t)chunk * E + e] = c;
  }
}

// One warp per padded row: x_perm[row, :] = x[token(row), :], zeros in padding rows.
__global__ void __launch_bounds__(256)
gather_rows(const uint4* __restrict__ x, uint4* __restrict__ x_perm, const int32_t* __restrict__ assign_of_row,
            const int32_t* __restrict__ pad_offsets, int E, int K, int vec_per_row, int rows_max) {
  const int lane = threadIdx.x & 31;
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= rows_max || row >= pad_offsets[E]) return;
  const int a = assign_of_row[row];
  uint4* dst = x_perm + (size_t)row * vec_per_row;
  if (a < 0) {
    for (int v = lane; v < vec_per_row; v += 32) dst[v] = make_uint4(0, 0, 0, 0);
  } else {
    const uint4* src = x + (size_t)(a / K) * vec_per_row;
    for (int v = lane; v < vec_per_row; v += 32) dst[v] = __ldg(src + v);
  }
}

}  // namespace

cudaError_t launch_route(const rom_config& c, const void* x, const void* W_r, const float* b_r,
                         int32_t* topk_idx, float* gates, int32_t* counts, int32_t* offsets,
                         int32_t* perm, int32_t* inv_perm, char* ws, const WsLayout& lay, cudaStream_t st) {
  return launch_route_stats(c, x, W_r, b_r, topk_idx, gates, counts, offsets, perm, inv_perm, ws, lay, nullptr, st);
}

// Load-balance statistic (Appendix A.3): F_i = assignments of expert i / tokens, Pbar_i = mean over tokens of
// Softmax(X W_r)_i, loss = alpha * E * sum_i F_i * Pbar_i.  One block; chunk sums are added in chunk order.
__global__ void __launch_bounds__(64)
balance_finish(const double* __restrict__ chunk_prob, const int32_t* __restrict__ counts, int n_chunks, int E, int T_tokens,
               float alpha, float* __restrict__ F, float* __restrict__ Pbar, float* __restrict__ loss) {
  __shared__ double term[kMaxE];
  const int e = threadIdx.x;
  if (e < E) {
    double ps = 0.0;
    for (int c = 0; c < n_chunks; ++c) ps += chunk_prob[(size_t)c * E + e];
    const double f = (double)counts[e] / (double)T_tokens, pb = ps / (double)T_tokens;
    if (F) F[e] = (float)f;
    if (Pbar) Pbar[e] = (float)pb;
    term[e] = f * pb;
  }
  __syncthreads();
  if (threadIdx.x == 0 && loss) {
    double sum = 0.0;
    for (int i = 0; i < E; ++i) sum += term[i];
    *loss = (float)((double)alpha * E * sum);
  }
}

cudaError_t launch_balance(const rom_config& c, const void* x, const void* W_r, const float* b_r, float alpha,
                           float* F, float* Pbar, float* loss, char* ws, const WsLayout& lay, cudaStream_t st) {
  double* chunk_prob = reinterpret_cast<double*>(ws + lay.chunk_prob);
  cudaError_t err = launch_route_stats(c, x, W_r, b_r, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, ws, lay, chunk_prob, st);
  if (err != cudaSuccess) return err;
  balance_finish<<<1, 64, 0, st>>>(chunk_prob, reinterpret_cast<const int32_t*>(ws + lay.counts), (int)lay.n_chunks, c.E, (int)lay.T,
                                  alpha, F, Pbar, loss);
  count_launch();
  return cudaGetLastError();
}

static cudaError_t launch_perm_tables(const rom_config& c, const int32_t* idx_ws, int32_t* counts, int32_t* offsets, int32_t* perm,
                                      int32_t* inv_perm, char* ws, const WsLayout& lay, cudaStream_t st);

cudaError_t launch_route_stats(const rom_config& c, const void* x, const void* W_r, const float* b_r,
                               int32_t* topk_idx, float* gates, int32_t* counts, int32_t* offsets,
                               int32_t* perm, int32_t* inv_perm, char* ws, const WsLayout& lay, double* chunk_prob, cudaStream_t st) {
  const int T = (int)lay.T;
  int32_t* idx_ws = topk_idx ? topk_idx : reinterpret_cast<int32_t*>(ws + lay.topk_idx);
  int32_t* chunk_counts = reinterpret_cast<int32_t*>(ws + lay.chunk_counts);
  int32_t* assign_of_row = reinterpret_cast<int32_t*>(ws + lay.assign_of_row);
  cudaError_t err = cudaMemsetAsync(assign_of_row, 0xff, sizeof(int32_t) * lay.rows_max, st);
  if (err != cudaSuccess) return err;

  const int n_wtiles = (c.E + NT8 - 1) / NT8;
  const int Epad8 = n_wtiles * NT8;
  // warps per chunk: one per 8-expert tile, times a split of d_model that puts more loads in flight: up to 4 ranges,
  // up to 16 when there are too few chunks to fill the GPU (a handful of tokens: latency is all that matters)
  const int blocks = (T + RT - 1) / RT;
  int dsplit = blocks < 148 ? 16 : 4;
  while (dsplit > 1 && (n_wtiles * dsplit > 16 || c.d_model / 16 < 4 * dsplit)) dsplit >>= 1;
  const int threads = 32 * n_wtiles * dsplit;
  const bool bf = c.dtype == ROM_BF16;
  double* Wd = reinterpret_cast<double*>(ws + lay.wr_f64);
  const int nW = c.d_model * Epad8;
  if (bf) route_weights_f64<__nv_bfloat16><<<(nW + 255) / 256, 256, 0, st>>>((const __nv_bfloat16*)W_r, Wd, c.d_model, c.E, Epad8);
  else route_weights_f64<float><<<(nW + 255) / 256, 256, 0, st>>>((const float*)W_r, Wd, c.d_model, c.E, Epad8);
  count_launch();
  const size_t smem = sizeof(double) * (size_t)dsplit * RT * Epad8 + sizeof(int32_t) * RT * c.K;
  if (bf)
    route_logits_topk<__nv_bfloat16><<<blocks, threads, smem, st>>>(
        (const __nv_bfloat16*)x, Wd, b_r, T, c.d_model, c.E, c.K, c.gate_mode, idx_ws, gates, chunk_counts, chunk_prob);
  else
    route_logits_topk<float><<<blocks, threads, smem, st>>>(
        (const float*)x, Wd, b_r, T, c.d_model, c.E, c.K, c.gate_mode, idx_ws, gates, chunk_counts, chunk_prob);
  count_launch();
  return launch_perm_tables(c, idx_ws, counts, offsets, perm, inv_perm, ws, lay, st);
}

// offsets, padded offsets, row tiles and the permutation from the per-chunk histogram and the indices
static cudaError_t launch_perm_tables(const rom_config& c, const int32_t* idx_ws, int32_t* counts, int32_t* offsets, int32_t* perm,
                                      int32_t* inv_perm, char* ws, const WsLayout& lay, cudaStream_t st) {
  const int T = (int)lay.T;
  int32_t* chunk_counts = reinterpret_cast<int32_t*>(ws + lay.chunk_counts);
  int32_t* assign_of_row = reinterpret_cast<int32_t*>(ws + lay.assign_of_row);
  route_offsets<<<1, 1024, 0, st>>>(chunk_counts, (int)lay.n_chunks, c.E,
                                   reinterpret_cast<int32_t*>(ws + lay.counts), reinterpret_cast<int32_t*>(ws + lay.offsets),
                                   reinterpret_cast<int32_t*>(ws + lay.pad_offsets), reinterpret_cast<int32_t*>(ws + lay.num_m_tiles),
                                   reinterpret_cast<int32_t*>(ws + lay.tile_expert), (int)lay.max_m_tiles, counts, offsets);
  count_launch();
  const int wpb = 8;
  route_scatter<<<((int)lay.n_chunks + wpb - 1) / wpb, wpb * 32, 0, st>>>(
      idx_ws, chunk_counts, reinterpret_cast<int32_t*>(ws + lay.offsets), reinterpret_cast<int32_t*>(ws + lay.pad_offsets),
      T, c.E, c.K, (int)lay.n_chunks, perm, inv_perm, reinterpret_cast<int32_t*>(ws + lay.row_of_assign), assign_of_row);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_gather_rows(const rom_config& c, const void* x, char* ws, const WsLayout& lay, cudaStream_t st) {
  return launch_gather_rows_to(c, x, ws + lay.x_perm, c.d_model, ws, lay, st);
}

cudaError_t launch_gather_rows_to(const rom_config& c, const void* src, void* dst, int width, char* ws, const WsLayout& lay,
                                  cudaStream_t st) {
  const int vec_per_row = (int)((size_t)width * lay.esz / 16);
  const int wpb = 8;
  const int blocks = (int)((lay.rows_max + wpb - 1) / wpb);
  gather_rows<<<blocks, wpb * 32, 0, st>>>(reinterpret_cast<const uint4*>(src), reinterpret_cast<uint4*>(dst),
                                          reinterpret_cast<const int32_t*>(ws + lay.assign_of_row),
                                          reinterpret_cast<const int32_t*>(ws + lay.pad_offsets), c.E, c.K, vec_per_row,
                                          (int)lay.rows_max);
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_perm_from_idx(const rom_config& c, const int32_t* topk_idx, int32_t* counts, int32_t* offsets, int32_t* perm,
                                 int32_t* inv_perm, char* ws, const WsLayout& lay, cudaStream_t st) {
  int32_t* idx_ws = reinterpret_cast<int32_t*>(ws + lay.topk_idx);
  cudaError_t err = cudaMemsetAsync(ws + lay.assign_of_row, 0xff, sizeof(int32_t) * lay.rows_max, st);
  if (err != cudaSuccess) return err;
  const int wpb = 8;
  idx_chunk_histogram<<<((int)lay.n_chunks + wpb - 1) / wpb, wpb * 32, 0, st>>>(
      topk_idx, idx_ws, (int)lay.T, c.E, c.K, (int)lay.n_chunks, reinterpret_cast<int32_t*>(ws + lay.chunk_counts),
      reinterpret_cast<int32_t*>(ws + lay.status));
  count_launch();
  return launch_perm_tables(c, idx_ws, counts, offsets, perm, inv_perm, ws, lay, st);
}

}  // namespace rom
