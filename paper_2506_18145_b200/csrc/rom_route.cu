// Router, top-K and dropless permutation (Section 4.2 routing equation; Section 5.1: no capacity
// factor and no token dropping), plus the row gather that feeds the grouped Conv/Gate projection.
//
// Kernels (two launches on the layer's path)
//   route_logits_topk : logits in fp64 on the tensor cores (products of bf16 or fp32 inputs are exact in
//                       fp64; every expert's sum is taken in the same order, so ties stay ties), softmax,
//                       top-K with ties to the lowest expert id, per-chunk histogram; clears the
//                       row -> assignment table; the block that finishes last (an atomic ticket, no
//                       waiting) turns the chunk histograms into expert offsets, offsets padded to the
//                       GEMM row tile and the row-tile -> expert map.
//   route_scatter     : stable rank of every assignment inside its chunk by warp ballots; writes
//                       perm / inv_perm and the padded-row tables and, when asked, copies each token's
//                       row to its padded row (x_perm, zero rows in the padding) while x is still in L2.
//   route_offsets, idx_chunk_histogram, gather_rows : the same steps as separate kernels, for tables
//                       built from a routing decision made elsewhere and for other row gathers.
#include "rom_internal.cuh"

namespace rom {
namespace {

constexpr int RT = kChunkTokens;   // tokens per block of route_logits_topk = one routing chunk
constexpr int NT8 = 8;             // experts per warp (one fp64 MMA column tile)

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

// Run by one block: warp w scans the chunk histogram of experts w, w + nwarps, ... over all chunks (exclusive bases
// written back in place), then expert offsets, offsets padded to the row tile, tile count and row-tile -> expert map.
__device__ void offsets_from_histograms(int32_t* __restrict__ chunk_counts, int n_chunks, int E,
                                        int32_t* __restrict__ counts_ws, int32_t* __restrict__ offsets_ws, int32_t* __restrict__ pad_offsets,
                                        int32_t* __restrict__ num_m_tiles, int32_t* __restrict__ tile_expert, int max_m_tiles,
                                        int32_t* __restrict__ counts_out, int32_t* __restrict__ offsets_out,
                                        int32_t* cnt, int32_t* off, int32_t* poff /* shared: kMaxE, kMaxE+1, kMaxE+1 */) {
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

struct OffsetsArgs {
  int32_t* counts_ws; int32_t* offsets_ws; int32_t* pad_offsets; int32_t* num_m_tiles; int32_t* tile_expert; int max_m_tiles;
  int32_t* counts_out; int32_t* offsets_out;
  int32_t* assign_of_row; int rows_max;      // cleared to -1 by the grid
  int32_t* ticket;                           // zero on entry; left zero on exit
};

__global__ void __launch_bounds__(1024)
route_offsets(int32_t* __restrict__ chunk_counts, int n_chunks, int E, const OffsetsArgs o) {
  __shared__ int32_t cnt[kMaxE];
  __shared__ int32_t off[kMaxE + 1];
  __shared__ int32_t poff[kMaxE + 1];
  offsets_from_histograms(chunk_counts, n_chunks, E, o.counts_ws, o.offsets_ws, o.pad_offsets, o.num_m_tiles, o.tile_expert,
                          o.max_m_tiles, o.counts_out, o.offsets_out, cnt, off, poff);
}

// One block = 32 tokens (one routing chunk); warp w computes the logits of experts [8w, 8w+8) for them with
// fp64 tensor-core MMAs (products of bf16/fp32 inputs are exact in fp64; every expert column is accumulated
// in the same order, so equal weight rows give bit-equal logits and ties stay ties).  Per 16 elements of
// d_model a lane reads 4 consecutive elements of one token row per 8-token tile (32-byte sectors, straight
// from global memory) and 4 consecutive fp64 weights of one expert (L1/L2-resident copy); MMA j of the step
// contracts elements {j, 4+j, 8+j, 12+j} of the 16.  No shared memory until the logits meet for the top-K.
template <typename T>
__global__ void __launch_bounds__(512)
route_logits_topk(const T* __restrict__ x, const T* __restrict__ W_r, const float* __restrict__ b_r,
                  int T_tokens, int Dm, int E, int K, int gate_mode,
                  int32_t* __restrict__ topk_idx, float* __restrict__ gates,
                  int32_t* __restrict__ chunk_counts, double* __restrict__ chunk_prob, int n_chunks, const OffsetsArgs oa) {
  extern __shared__ __align__(16) unsigned char smem[];
  const int Epad = (E + NT8 - 1) / NT8 * NT8;
  const int n_wtiles = Epad / NT8;
  const int dsplit = (blockDim.x >> 5) / n_wtiles;                 // warps that share one expert tile, each on its own d range
  double* lg = reinterpret_cast<double*>(smem);                    // [dsplit][RT][Epad] partial logits; [0] becomes the sum
  int32_t* idx_s = reinterpret_cast<int32_t*>(lg + max(dsplit, 2) * RT * Epad);   // [RT][K] (later: scratch of the offsets scan)

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
  // weights: 4 consecutive d of expert 8w + gq, read in the storage type and widened on use (exact); experts beyond E
  // (padding of the 8-expert tile) read expert E-1 and are zeroed
  const bool w_ok = w * NT8 + gq < E;
  const T* wrow = W_r + (size_t)min(w * NT8 + gq, E - 1) * Dm + 4 * t4;

  // the row -> assignment table starts at -1 everywhere (padding rows keep it); the whole grid clears it
  for (int i = blockIdx.x * blockDim.x + tid; i < oa.rows_max; i += gridDim.x * blockDim.x) oa.assign_of_row[i] = -1;

  // operands of the next PF-1 steps are in flight (raw, unconverted) while one step is contracted
  // (d_model is a multiple of 64, so there are at least PF steps)
  constexpr int PF = 4;
  RawX4<T> rx[PF][4];
  RawX4<T> rw[PF];
  auto fetch = [&](int d, RawX4<T> (&xo)[4], RawX4<T>& wo) {
#pragma unroll
    for (int mt = 0; mt < 4; ++mt) xo[mt].load(xrow[mt] + d);
    wo.load(wrow + d);
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
      double wb[4];
      rw[i].get(wb);
      if (!w_ok) { wb[0] = 0.0; wb[1] = 0.0; wb[2] = 0.0; wb[3] = 0.0; }
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

  // softmax numerators, one (token, expert) pair per thread: pr[t][e] = exp(l[t][e] - max_e l[t][e])
  double* pr = lg + RT * Epad;                                     // second partial-sum slab (dsplit >= 2) or the extra slab
  for (int i = tid; i < RT * E; i += blockDim.x) {
    const int tt = i / E, e = i - tt * E;
    const double* l = lg + tt * Epad;
    double m = -INFINITY;
    for (int j = 0; j < E; ++j) { const double v = l[j]; if (v > m) m = v; }   // NaN never raises m
    pr[tt * Epad + e] = exp(l[e] - m);
  }
  __syncthreads();

  if (tid < RT) {
    const int t = t0 + tid;
    const double* l = lg + tid * Epad;
    const double* pe_row = pr + tid * Epad;
    double denom = 1.0;
    if (t < T_tokens) {
      denom = 0.0;
      for (int e = 0; e < E; ++e) denom += pe_row[e];
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
        gsel[k] = pe_row[best] / denom;
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
        double pe = t < T_tokens ? pe_row[e] / denom : 0.0;
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

  // The block that finishes last builds the offsets from all the histograms: every block publishes its writes
  // (histogram, cleared table slice) and takes a ticket; nobody waits for anybody.
  if (oa.ticket == nullptr) return;
  __shared__ int s_last;
  __threadfence();
  __syncthreads();
  if (tid == 0) s_last = (atomicAdd(oa.ticket, 1) == (int)gridDim.x - 1);
  __syncthreads();
  if (!s_last) return;
  __threadfence();
  if (tid == 0) *oa.ticket = 0;                  // ready for the next call on this workspace
  int32_t* cnt = idx_s;                          // the top-K scratch is free now: kMaxE + 2 (kMaxE + 1) ints (sized by the launcher)
  offsets_from_histograms(chunk_counts, n_chunks, E, oa.counts_ws, oa.offsets_ws, oa.pad_offsets, oa.num_m_tiles, oa.tile_expert,
                          oa.max_m_tiles, oa.counts_out, oa.offsets_out, cnt, cnt + kMaxE, cnt + 2 * kMaxE + 1);
}

// Stable rank of the chunk's assignments by warp ballots, then the table entries; called by one full warp.
// my_row[k] receives the padded row of (token, slot k), -1 past the end.
__device__ __forceinline__ void scatter_chunk(const int32_t* __restrict__ topk_idx, const int32_t* __restrict__ chunk_base,
                                              const int32_t* __restrict__ offsets, const int32_t* __restrict__ pad_offsets,
                                              int T_tokens, int E, int K, int chunk, int lane,
                                              int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm,
                                              int32_t* __restrict__ row_of_assign, int32_t* __restrict__ assign_of_row,
                                              int (&my_row)[kMaxK]) {
  const int t = chunk * kChunkTokens + lane;
  int my_e[kMaxK], my_rank[kMaxK];
  for (int k = 0; k < K; ++k) {
    my_e[k] = (t < T_tokens) ? topk_idx[(size_t)t * K + k] : -1;
    my_rank[k] = 0;
    my_row[k] = -1;
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
    my_row[k] = pr;
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
  int my_row[kMaxK];
  scatter_chunk(topk_idx, chunk_base, offsets, pad_offsets, T_tokens, E, K, chunk, lane, perm, inv_perm, row_of_assign, assign_of_row, my_row);
}

// One block of 8 warps per chunk of 32 tokens: warp 0 builds the chunk's table entries, then every warp copies the rows
// of four of the chunk's tokens to their padded rows (x_perm, the operand of the grouped Conv/Gate projection; x was read
// by the router a moment ago and is still in L2), and the grid zero-fills the padding rows of every expert segment.
__global__ void __launch_bounds__(256)
route_scatter_gather(const int32_t* __restrict__ topk_idx, const int32_t* __restrict__ chunk_base,
                     const int32_t* __restrict__ offsets, const int32_t* __restrict__ pad_offsets,
                     int T_tokens, int E, int K, int n_chunks,
                     int32_t* __restrict__ perm, int32_t* __restrict__ inv_perm,
                     int32_t* __restrict__ row_of_assign, int32_t* __restrict__ assign_of_row,
                     const uint4* __restrict__ x, uint4* __restrict__ x_perm, int vec_per_row) {
  __shared__ int32_t rows_s[kChunkTokens * kMaxK];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int chunk = blockIdx.x;
  // blocks beyond the last chunk (the grid never drops below one block per SM) only help with the padding rows
  if (chunk < n_chunks && warp == 0) {
    int my_row[kMaxK];
    scatter_chunk(topk_idx, chunk_base, offsets, pad_offsets, T_tokens, E, K, chunk, lane, perm, inv_perm, row_of_assign, assign_of_row, my_row);
    for (int k = 0; k < K; ++k) rows_s[lane * K + k] = my_row[k];
  }
  __syncthreads();
  const int n_tok = chunk < n_chunks ? min(kChunkTokens, T_tokens - chunk * kChunkTokens) : 0;
  for (int j = warp; j < n_tok; j += 8) {
    const uint4* src = x + (size_t)(chunk * kChunkTokens + j) * vec_per_row;
    for (int v0 = 0; v0 < vec_per_row; v0 += 32 * 8) {
      uint4 buf[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        const int v = v0 + 32 * i + lane;
        if (v < vec_per_row) buf[i] = __ldg(src + v);
      }
      for (int k = 0; k < K; ++k) {
        uint4* dst = x_perm + (size_t)rows_s[j * K + k] * vec_per_row;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const int v = v0 + 32 * i + lane;
          if (v < vec_per_row) dst[v] = buf[i];
        }
      }
    }
  }
  const int n_warps = gridDim.x * 8, gw = blockIdx.x * 8 + warp;
  for (int e = 0; e < E; ++e) {
    const int first = pad_offsets[e] + (offsets[e + 1] - offsets[e]), last = pad_offsets[e + 1];
    for (int r = first + gw; r < last; r += n_warps) {
      uint4* dst = x_perm + (size_t)r * vec_per_row;
      for (int v = lane; v < vec_per_row; v += 32) dst[v] = make_uint4(0, 0, 0, 0);
    }
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
  return launch_route_stats(c, x, W_r, b_r, topk_idx, gates, counts, offsets, perm, inv_perm, ws, lay, nullptr, st, false);
}

cudaError_t launch_route_gather(const rom_config& c, const void* x, const void* W_r, const float* b_r,
                                int32_t* topk_idx, float* gates, int32_t* counts, char* ws, const WsLayout& lay, cudaStream_t st) {
  return launch_route_stats(c, x, W_r, b_r, topk_idx, gates, counts, nullptr, nullptr, nullptr, ws, lay, nullptr, st, true);
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
  cudaError_t err = launch_route_stats(c, x, W_r, b_r, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, ws, lay, chunk_prob, st, false);
  if (err != cudaSuccess) return err;
  balance_finish<<<1, 64, 0, st>>>(chunk_prob, reinterpret_cast<const int32_t*>(ws + lay.counts), (int)lay.n_chunks, c.E, (int)lay.T,
                                  alpha, F, Pbar, loss);
  count_launch();
  return cudaGetLastError();
}

static cudaError_t launch_perm_tables(const rom_config& c, const int32_t* idx_ws, int32_t* counts, int32_t* offsets, int32_t* perm,
                                      int32_t* inv_perm, char* ws, const WsLayout& lay, cudaStream_t st);
static cudaError_t launch_scatter(const rom_config& c, const int32_t* idx_ws, int32_t* perm, int32_t* inv_perm, char* ws,
                                  const WsLayout& lay, const void* x, cudaStream_t st);

cudaError_t launch_route_stats(const rom_config& c, const void* x, const void* W_r, const float* b_r,
                               int32_t* topk_idx, float* gates, int32_t* counts, int32_t* offsets,
                               int32_t* perm, int32_t* inv_perm, char* ws, const WsLayout& lay, double* chunk_prob, cudaStream_t st,
                               bool gather_x) {
  const int T = (int)lay.T;
  int32_t* idx_ws = topk_idx ? topk_idx : reinterpret_cast<int32_t*>(ws + lay.topk_idx);
  int32_t* chunk_counts = reinterpret_cast<int32_t*>(ws + lay.chunk_counts);
  int32_t* assign_of_row = reinterpret_cast<int32_t*>(ws + lay.assign_of_row);

  const int n_wtiles = (c.E + NT8 - 1) / NT8;
  const int Epad8 = n_wtiles * NT8;
  // warps per chunk: one per 8-expert tile, times a split of d_model that puts more loads in flight: up to 4 ranges,
  // up to 16 when there are too few chunks to fill the GPU (a handful of tokens: latency is all that matters)
  const int blocks = (T + RT - 1) / RT;
  int dsplit = blocks < 148 ? 16 : 4;
  while (dsplit > 1 && (n_wtiles * dsplit > 16 || c.d_model / 16 < 4 * dsplit)) dsplit >>= 1;
  const int threads = 32 * n_wtiles * dsplit;
  const bool bf = c.dtype == ROM_BF16;
  const OffsetsArgs oa{reinterpret_cast<int32_t*>(ws + lay.counts), reinterpret_cast<int32_t*>(ws + lay.offsets),
                       reinterpret_cast<int32_t*>(ws + lay.pad_offsets), reinterpret_cast<int32_t*>(ws + lay.num_m_tiles),
                       reinterpret_cast<int32_t*>(ws + lay.tile_expert), (int)lay.max_m_tiles, counts, offsets,
                       assign_of_row, (int)lay.rows_max, reinterpret_cast<int32_t*>(ws + lay.status) + kStatTicket};
  const int idx_ints = RT * c.K > 3 * kMaxE + 2 ? RT * c.K : 3 * kMaxE + 2;
  const size_t smem = sizeof(double) * (size_t)(dsplit > 2 ? dsplit : 2) * RT * Epad8 + sizeof(int32_t) * idx_ints;
  if (bf)
    route_logits_topk<__nv_bfloat16><<<blocks, threads, smem, st>>>(
        (const __nv_bfloat16*)x, (const __nv_bfloat16*)W_r, b_r, T, c.d_model, c.E, c.K, c.gate_mode, idx_ws, gates, chunk_counts,
        chunk_prob, (int)lay.n_chunks, oa);
  else
    route_logits_topk<float><<<blocks, threads, smem, st>>>(
        (const float*)x, (const float*)W_r, b_r, T, c.d_model, c.E, c.K, c.gate_mode, idx_ws, gates, chunk_counts, chunk_prob,
        (int)lay.n_chunks, oa);
  count_launch();
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  return launch_scatter(c, idx_ws, perm, inv_perm, ws, lay, gather_x ? x : nullptr, st);
}

// the permutation (and, with x, the gathered rows) from the indices, the per-chunk bases and the offsets
static cudaError_t launch_scatter(const rom_config& c, const int32_t* idx_ws, int32_t* perm, int32_t* inv_perm, char* ws,
                                  const WsLayout& lay, const void* x, cudaStream_t st) {
  const int32_t* chunk_base = reinterpret_cast<int32_t*>(ws + lay.chunk_counts);
  const int32_t* offs = reinterpret_cast<int32_t*>(ws + lay.offsets);
  const int32_t* poffs = reinterpret_cast<int32_t*>(ws + lay.pad_offsets);
  int32_t* roa = reinterpret_cast<int32_t*>(ws + lay.row_of_assign);
  int32_t* aor = reinterpret_cast<int32_t*>(ws + lay.assign_of_row);
  if (x != nullptr) {
    int num_sms = 0;
    const cudaError_t e = current_device_sm_count(&num_sms);
    if (e != cudaSuccess) return e;
    const int grid = (int)lay.n_chunks > num_sms ? (int)lay.n_chunks : num_sms;
    route_scatter_gather<<<grid, 256, 0, st>>>(idx_ws, chunk_base, offs, poffs, (int)lay.T, c.E, c.K, (int)lay.n_chunks, perm, inv_perm, roa, aor,
                                                           reinterpret_cast<const uint4*>(x), reinterpret_cast<uint4*>(ws + lay.x_perm),
                                                           (int)((size_t)c.d_model * lay.esz / 16));
  } else {
    const int wpb = 8;
    route_scatter<<<((int)lay.n_chunks + wpb - 1) / wpb, wpb * 32, 0, st>>>(idx_ws, chunk_base, offs, poffs, (int)lay.T, c.E, c.K,
                                                                          (int)lay.n_chunks, perm, inv_perm, roa, aor);
  }
  count_launch();
  return cudaGetLastError();
}

// offsets, padded offsets, row tiles and the permutation from the per-chunk histogram and the indices (separate launches)
static cudaError_t launch_perm_tables(const rom_config& c, const int32_t* idx_ws, int32_t* counts, int32_t* offsets, int32_t* perm,
                                      int32_t* inv_perm, char* ws, const WsLayout& lay, cudaStream_t st) {
  const OffsetsArgs oa{reinterpret_cast<int32_t*>(ws + lay.counts), reinterpret_cast<int32_t*>(ws + lay.offsets),
                       reinterpret_cast<int32_t*>(ws + lay.pad_offsets), reinterpret_cast<int32_t*>(ws + lay.num_m_tiles),
                       reinterpret_cast<int32_t*>(ws + lay.tile_expert), (int)lay.max_m_tiles, counts, offsets, nullptr, 0, nullptr};
  route_offsets<<<1, 1024, 0, st>>>(reinterpret_cast<int32_t*>(ws + lay.chunk_counts), (int)lay.n_chunks, c.E, oa);
  count_launch();
  return launch_scatter(c, idx_ws, perm, inv_perm, ws, lay, nullptr, st);
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
