// Router, top-K and dropless permutation (Section 4.2 routing equation; Section 5.1: no capacity
// factor and no token dropping), plus the row gather that feeds the grouped Conv/Gate projection.
//
// Kernels
//   route_logits_topk : logits in fp64 (products of bf16 or fp32 inputs are exact in fp64 and the sum
//                       runs strictly in ascending d, so the logits equal a left-to-right fp64 sum bit
//                       for bit), softmax, top-K with ties to the lowest expert id, per-chunk histogram.
//   route_offsets     : per-expert exclusive scan of the chunk histograms (warp shuffles), expert
//                       offsets, offsets padded to the GEMM row tile, row-tile -> expert map.
//   route_scatter     : stable rank of every assignment inside its chunk by warp ballots; writes
//                       perm / inv_perm and the padded-row tables.
//   gather_rows       : x_perm[row] = x[token of row] (zero rows in the padding).
#include "rom_internal.cuh"

namespace rom {
namespace {

constexpr int RT = kChunkTokens;   // tokens per block of route_logits_topk = one routing chunk (lanes of a warp)
constexpr int EG = 4;              // experts accumulated per thread (one warp = 32 tokens x EG experts)
constexpr int DC = 64;             // d_model elements staged per step

template <typename T> struct XRow;
template <> struct XRow<__nv_bfloat16> { static constexpr int kStrideBytes = DC * 2 + 16; };
template <> struct XRow<float> { static constexpr int kStrideBytes = DC * 4 + 16; };

__device__ __forceinline__ void load8(const __nv_bfloat16* p, double (&xd)[8]) {
  uint4 v = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    xd[2 * i] = (double)__uint_as_float(w[i] << 16);
    xd[2 * i + 1] = (double)__uint_as_float(w[i] & 0xffff0000u);
  }
}
__device__ __forceinline__ void load8(const float* p, double (&xd)[8]) {
  float4 a = *reinterpret_cast<const float4*>(p);
  float4 b = *reinterpret_cast<const float4*>(p + 4);
  xd[0] = a.x; xd[1] = a.y; xd[2] = a.z; xd[3] = a.w;
  xd[4] = b.x; xd[5] = b.y; xd[6] = b.z; xd[7] = b.w;
}

// One block = 32 tokens (one routing chunk).  Warp g accumulates experts [4g, 4g+4) for the 32 tokens
// (lane = token): per element of d_model one x value from the lane's staged row and four router
// weights broadcast from shared memory, four independent fp64 FMA chains, strictly ascending d.
template <typename T>
__global__ void __launch_bounds__(512)
route_logits_topk(const T* __restrict__ x, const T* __restrict__ W_r, const float* __restrict__ b_r,
                  int T_tokens, int Dm, int E, int K, int gate_mode,
                  int32_t* __restrict__ topk_idx, float* __restrict__ gates,
                  int32_t* __restrict__ chunk_counts, double* __restrict__ chunk_prob) {
  extern __shared__ __align__(16) unsigned char smem[];
  const int groups = (E + EG - 1) / EG;
  const int Epad = groups * EG;
  constexpr int XS = XRow<T>::kStrideBytes;
  unsigned char* xs = smem;                                        // [2][RT][XS]   (double-buffered)
  double* wsd = reinterpret_cast<double*>(smem + 2 * RT * XS);     // [2][groups][DC][EG]: a warp's four experts of one d are adjacent
  double* lg = wsd + 2 * DC * Epad;                                // [RT][Epad]
  int32_t* idx_s = reinterpret_cast<int32_t*>(lg + RT * Epad);     // [RT][K]

  const int tid = threadIdx.x;
  const int tok = tid & 31;
  const int g = tid >> 5;
  const int t0 = blockIdx.x * RT;
  const int nthr = blockDim.x;

  double acc[EG];
#pragma unroll
  for (int e = 0; e < EG; ++e) {
    const int ee = g * EG + e;
    acc[e] = (b_r != nullptr && ee < E) ? (double)b_r[ee] : 0.0;
  }

  // Chunk i+1 of x goes global -> shared with 16-byte asynchronous copies (rows past the end are
  // zero-filled) and chunk i+1 of W_r is held in registers while chunk i is accumulated.
  constexpr int VPR = DC * (int)sizeof(T) / 16;      // 16-byte vectors per row
  constexpr int WPT = EG * DC / 32;                  // router weights per thread per chunk (Epad*DC / nthr)
  auto copy_x = [&](int d0, int buf) {
    for (int v = tid; v < RT * VPR; v += nthr) {
      const int r = v / VPR, cv = v % VPR;
      const bool in = t0 + r < T_tokens;
      const unsigned char* src = reinterpret_cast<const unsigned char*>(x + (size_t)(in ? t0 + r : 0) * Dm + d0) + cv * 16;
      const uint32_t dst = (uint32_t)__cvta_generic_to_shared(xs + (buf * RT + r) * XS + cv * 16);
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(in ? 16 : 0) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  float wpre[WPT];
  auto fetch_w = [&](int d0) {
#pragma unroll
    for (int i = 0; i < WPT; ++i) {
      const int v = tid + i * nthr, e = v / DC, d = v % DC;
      wpre[i] = (e < E) ? to_f32(W_r[(size_t)e * Dm + d0 + d]) : 0.0f;
    }
  };
  auto stash_w = [&](int buf) {
#pragma unroll
    for (int i = 0; i < WPT; ++i) {
      const int v = tid + i * nthr, e = v / DC, d = v % DC;
      wsd[((buf * groups + e / EG) * DC + d) * EG + (e % EG)] = (double)wpre[i];
    }
  };

  copy_x(0, 0);
  fetch_w(0);
  stash_w(0);
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();

  int buf = 0;
  for (int d0 = 0; d0 < Dm; d0 += DC, buf ^= 1) {
    const bool more = d0 + DC < Dm;
    if (more) { copy_x(d0 + DC, buf ^ 1); fetch_w(d0 + DC); }
    const T* xrow = reinterpret_cast<const T*>(xs + (buf * RT + tok) * XS);
    const double* wg = wsd + (buf * groups + g) * DC * EG;
#pragma unroll 2
    for (int d8 = 0; d8 < DC; d8 += 8) {
      double xd[8];
      load8(xrow + d8, xd);
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const double2 w01 = *reinterpret_cast<const double2*>(wg + (d8 + j) * EG);
        const double2 w23 = *reinterpret_cast<const double2*>(wg + (d8 + j) * EG + 2);
        acc[0] = fma(xd[j], w01.x, acc[0]);
        acc[1] = fma(xd[j], w01.y, acc[1]);
        acc[2] = fma(xd[j], w23.x, acc[2]);
        acc[3] = fma(xd[j], w23.y, acc[3]);
      }
    }
    if (more) stash_w(buf ^ 1);
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
  }
  __syncthreads();
#pragma unroll
  for (int e = 0; e < EG; ++e) lg[tok * Epad + g * EG + e] = acc[e];
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
    for (int c0 = 0; c0 < n_chunks; c0 += 32) {
      const int c = c0 + lane;
      const int v = (c < n_chunks) ? chunk_counts[(size_t)c * E + e] : 0;
      int inc = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        int n = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += n;
      }
      if (c < n_chunks) chunk_counts[(size_t)c * E + e] = carry + inc - v;    // exclusive base
      carry += __shfl_sync(0xffffffffu, inc, 31);
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

cudaError_t launch_route_stats(const rom_config& c, const void* x, const void* W_r, const float* b_r,
                               int32_t* topk_idx, float* gates, int32_t* counts, int32_t* offsets,
                               int32_t* perm, int32_t* inv_perm, char* ws, const WsLayout& lay, double* chunk_prob, cudaStream_t st) {
  const int T = (int)lay.T;
  const int groups = (c.E + EG - 1) / EG;
  const int Epad = groups * EG;
  int32_t* idx_ws = topk_idx ? topk_idx : reinterpret_cast<int32_t*>(ws + lay.topk_idx);
  int32_t* chunk_counts = reinterpret_cast<int32_t*>(ws + lay.chunk_counts);
  int32_t* assign_of_row = reinterpret_cast<int32_t*>(ws + lay.assign_of_row);
  cudaError_t err = cudaMemsetAsync(assign_of_row, 0xff, sizeof(int32_t) * lay.rows_max, st);
  if (err != cudaSuccess) return err;

  const int threads = RT * groups;
  const int blocks = (T + RT - 1) / RT;
  const bool bf = c.dtype == ROM_BF16;
  const size_t xs_bytes = (size_t)RT * (bf ? XRow<__nv_bfloat16>::kStrideBytes : XRow<float>::kStrideBytes);
  const size_t smem = 2 * xs_bytes + sizeof(double) * (2 * (size_t)Epad * DC + (size_t)RT * Epad) + sizeof(int32_t) * RT * c.K;
  if (bf) {
    err = cudaFuncSetAttribute(route_logits_topk<__nv_bfloat16>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    route_logits_topk<__nv_bfloat16><<<blocks, threads, smem, st>>>(
        (const __nv_bfloat16*)x, (const __nv_bfloat16*)W_r, b_r, T, c.d_model, c.E, c.K, c.gate_mode, idx_ws, gates, chunk_counts, chunk_prob);
  } else {
    err = cudaFuncSetAttribute(route_logits_topk<float>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (err != cudaSuccess) return err;
    route_logits_topk<float><<<blocks, threads, smem, st>>>(
        (const float*)x, (const float*)W_r, b_r, T, c.d_model, c.E, c.K, c.gate_mode, idx_ws, gates, chunk_counts, chunk_prob);
  }
  count_launch();
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
  const int vec_per_row = (int)((size_t)c.d_model * lay.esz / 16);
  const int wpb = 8;
  const int blocks = (int)((lay.rows_max + wpb - 1) / wpb);
  gather_rows<<<blocks, wpb * 32, 0, st>>>(reinterpret_cast<const uint4*>(x), reinterpret_cast<uint4*>(ws + lay.x_perm),
                                          reinterpret_cast<const int32_t*>(ws + lay.assign_of_row),
                                          reinterpret_cast<const int32_t*>(ws + lay.pad_offsets), c.E, c.K, vec_per_row,
                                          (int)lay.rows_max);
  count_launch();
  return cudaGetLastError();
}

}  // namespace rom
