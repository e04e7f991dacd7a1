// Backward of the selective scan (Section 3.1 recurrence; Section 5.1 trains the layer end to end).
//
// Forward:  h_t = a_t h_{t-1} + b_t u_t,  y_t = sum_n C_t,n h_t,n + D u_t,  out_t = y_t * SiLU(z_t)   (gate optional)
//           a = exp(Delta A);  b = expm1(Delta A)/A * B (zero-order hold)  or  Delta B.
// Reverse, with g = dLoss/dh_t carried from later steps and e_t = dout_t * SiLU(z_t):
//           g += C_t e_t;  dC_t = sum_c e_t h_t;  dA-bar = g h_{t-1};  db = g u_t;  du_t = sum_n g b + D e_t;  g <- a_t g.
//
// The reverse sweep needs h_{t-1} and h_t at every step.  First the forward scan kernel runs the recurrence in its
// state-only mode and keeps the state at the start of every chunk of 16 steps (checkpoints in the workspace).  The second kernel walks the chunks
// backwards: it recomputes the chunk's states from its checkpoint into shared memory, then sweeps the chunk in
// reverse.  A thread owns 4 of the 16 states of one channel of one sequence (4 adjacent lanes per channel): sums over
// the states (dDelta, du, the forward y for the gate's derivative) are shuffles over those lanes; sums over channels
// (dB, dC) are shuffles over the 8 channels of a warp, shared-memory atomics over the block and one global atomic per
// (step, state) and block; dA and dD accumulate in registers over the sequence and leave with one atomic per thread.
// A long sequence with few channels is cut into coarse chunks that run in parallel, as in the forward scan: both
// recurrences are linear, the states' forward in time and the state gradients' backward in time.  A pre-pass runs, per
// coarse chunk, the state recurrence from a zero state (end state, sum of Delta) and the gradient recurrence from a
// zero gradient (the gradient leaving the chunk's start); a chain kernel composes them into the true state at the start
// and the true gradient at the end of every coarse chunk; the two kernels above then run once per coarse chunk.
// All arithmetic is fp32; the fp32 configuration uses the accurate exp / expm1, the bf16 one a single ex2.approx per state
// and step (exp(x) - 1 by subtraction: with Delta A down to -5e-4 that is still good to a few 1e-4 relative).
#include "rom_internal.cuh"

namespace rom {
namespace {

constexpr int NST = 16;
constexpr int CK = 16;            // steps per chunk (16: four blocks fit an SM's shared memory)
constexpr int BCH = 32;           // channels per block
constexpr int BT = BCH * 4;       // threads per block
constexpr size_t BWD_SMEM = sizeof(float4) * CK * BT + sizeof(float) * CK * (8 * BCH + 4 * NST);

struct BwdArgs {
  const void* dy; const void* u; const float* delta; const float* A; const float* Bm; const float* Cm; const float* D;
  const void* z; const float* h0; const float* dh_last;
  void* du; float* ddelta; float* dA; float* dBm; float* dCm; float* dD; void* dz; float* dh0;
  float* ckpt;        // [B, nck, De, 16]
  int L, De, nck;
  int ldz;            // row pitch (elements) of z and dz
  // coarse chunks (blockIdx.z): chunk j covers steps [j Lc, (j+1) Lc); Lc is a multiple of CK.  ncc == 1: the whole sequence.
  int Lc, ncc;
  const float* h_in;  // [B, ncc, De, 16] state at the start of every coarse chunk (ncc > 1)
  const float* g_in;  // [B, ncc, De, 16] state gradient at the end of every coarse chunk (ncc > 1)
  float* h_end; float* q_start; float* sum_delta;     // pre-pass outputs: [B, ncc, De, 16] x 2 and [B, ncc, De]
};

__device__ __forceinline__ float sigmoid_f(float v) { return 1.0f / (1.0f + expf(-v)); }

// exp(x) and exp(x) - 1
template <bool PRECISE>
__device__ __forceinline__ void exp_and_expm1(float x, float& ex, float& em1) {
  if (PRECISE) { ex = expf(x); em1 = expm1f(x); }
  else { ex = ex2_ftz(1.4426950408889634f * x); em1 = ex - 1.0f; }
}
template <bool PRECISE>
__device__ __forceinline__ float exp_only(float x) { return PRECISE ? expf(x) : ex2_ftz(1.4426950408889634f * x); }

template <typename T, bool ZOH>
__global__ void __launch_bounds__(BT)
scan_bwd_kernel(const BwdArgs p) {
  extern __shared__ __align__(16) unsigned char bwd_smem[];
  float4 (*hbuf)[BT] = reinterpret_cast<float4 (*)[BT]>(bwd_smem);                    // states after each step of the chunk (this thread's 4)
  float (*s_dl)[BCH] = reinterpret_cast<float (*)[BCH]>(bwd_smem + sizeof(float4) * CK * BT);
  float (*s_u)[BCH] = s_dl + CK;
  float (*s_e)[BCH] = s_u + CK;
  float (*s_z)[BCH] = s_e + CK;
  float (*s_dy)[BCH] = s_z + CK;
  float (*s_dd)[BCH] = s_dy + CK;
  float (*s_du)[BCH] = s_dd + CK;
  float (*s_y)[BCH] = s_du + CK;
  float (*s_B)[NST] = reinterpret_cast<float (*)[NST]>(s_y + CK);
  float (*s_C)[NST] = s_B + CK;
  float (*s_dB)[NST] = s_C + CK;
  float (*s_dC)[NST] = s_dB + CK;

  const int tid = threadIdx.x, cl = tid >> 2, q = tid & 3, lane = tid & 31;
  const int c_base = blockIdx.x * BCH;
  const int c = c_base + cl;
  const bool c_ok = c < p.De;
  const int cc = c_ok ? c : p.De - 1;
  const size_t b = blockIdx.y;
  const T* __restrict__ u = static_cast<const T*>(p.u);
  const T* __restrict__ dy = static_cast<const T*>(p.dy);
  const T* __restrict__ z = static_cast<const T*>(p.z);
  T* __restrict__ du = static_cast<T*>(p.du);
  T* __restrict__ dz = static_cast<T*>(p.dz);

  const int cj = blockIdx.z;
  const int k_lo = cj * (p.Lc / CK), k_hi = min(k_lo + p.Lc / CK, p.nck);
  float a[4], g[4], dAacc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    a[i] = p.A[(size_t)cc * NST + 4 * q + i];
    if (p.ncc > 1) g[i] = p.g_in[((b * p.ncc + cj) * p.De + cc) * NST + 4 * q + i];
    else g[i] = p.dh_last ? p.dh_last[(b * p.De + cc) * NST + 4 * q + i] : 0.0f;
  }
  const float Dc = p.D ? p.D[cc] : 0.0f;
  float dDacc = 0.0f;
  constexpr bool PRECISE = sizeof(T) == 4;
  float ia[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) ia[i] = 1.0f / a[i];

  for (int k = k_hi - 1; k >= k_lo; --k) {
    const int t0 = k * CK;
    const int nt = min(CK, p.L - t0);
    // ---- stage the chunk's inputs; e = dout * SiLU(z) is the gradient arriving at y
    for (int i = tid; i < CK * BCH; i += BT) {
      const int r = i / BCH, j = i % BCH;
      float dl = 0.0f, uu = 0.0f, dyv = 0.0f, zz = 0.0f;
      if (r < nt && c_base + j < p.De) {
        const size_t e = (b * p.L + t0 + r) * p.De + c_base + j;
        dl = p.delta[e]; uu = to_f32(u[e]); dyv = to_f32(dy[e]);
        if (z) zz = to_f32(z[(b * p.L + t0 + r) * p.ldz + c_base + j]);
      }
      s_dl[r][j] = dl; s_u[r][j] = uu; s_dy[r][j] = dyv; s_z[r][j] = zz;
      s_e[r][j] = z ? dyv * zz * sigmoid_f(zz) : dyv;
    }
    for (int i = tid; i < CK * NST; i += BT) {
      const int r = i / NST, n = i % NST;
      const bool in = r < nt;
      s_B[r][n] = in ? p.Bm[(b * p.L + t0 + r) * NST + n] : 0.0f;
      s_C[r][n] = in ? p.Cm[(b * p.L + t0 + r) * NST + n] : 0.0f;
      s_dB[r][n] = 0.0f; s_dC[r][n] = 0.0f;
    }
    __syncthreads();

    // ---- recompute the chunk's states from its checkpoint
    const float4 h4 = *reinterpret_cast<const float4*>(p.ckpt + ((b * p.nck + k) * p.De + cc) * NST + 4 * q);
    const float hstart[4] = {h4.x, h4.y, h4.z, h4.w};
    float h[4] = {h4.x, h4.y, h4.z, h4.w};
    for (int r = 0; r < nt; ++r) {
      const float dl = s_dl[r][cl], uu = s_u[r][cl];
      float ys = 0.0f;
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        float ex, em1;
        exp_and_expm1<PRECISE>(dl * a[i], ex, em1);
        const float bb = ZOH ? em1 * ia[i] * s_B[r][4 * q + i] : dl * s_B[r][4 * q + i];
        h[i] = fmaf(ex, h[i], bb * uu);
        ys = fmaf(s_C[r][4 * q + i], h[i], ys);
      }
      hbuf[r][tid] = make_float4(h[0], h[1], h[2], h[3]);
      if (z) {                                     // forward y (before the gate) for the gate's derivative
        ys += __shfl_xor_sync(0xffffffffu, ys, 1);
        ys += __shfl_xor_sync(0xffffffffu, ys, 2);
        if (q == 0) s_y[r][cl] = fmaf(Dc, uu, ys);
      }
    }

    // ---- reverse sweep over the chunk
    for (int r = nt - 1; r >= 0; --r) {
      const float dl = s_dl[r][cl], uu = s_u[r][cl], ev = c_ok ? s_e[r][cl] : 0.0f;
      const float4 hc4 = hbuf[r][tid];
      const float hc[4] = {hc4.x, hc4.y, hc4.z, hc4.w};
      float hp[4];
      if (r > 0) { const float4 v = hbuf[r - 1][tid]; hp[0] = v.x; hp[1] = v.y; hp[2] = v.z; hp[3] = v.w; }
      else { hp[0] = hstart[0]; hp[1] = hstart[1]; hp[2] = hstart[2]; hp[3] = hstart[3]; }
      float dd = 0.0f, duv = 0.0f, dBp[4], dCp[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float Bv = s_B[r][4 * q + i], Cv = s_C[r][4 * q + i];
        g[i] = fmaf(Cv, ev, g[i]);
        dCp[i] = ev * hc[i];
        float ex, em1;
        exp_and_expm1<PRECISE>(dl * a[i], ex, em1);
        float dx = g[i] * hp[i] * ex;              // through A-bar = exp(x)
        if (ZOH) {
          const float gub = g[i] * uu * Bv * ia[i], ge = g[i] * em1 * ia[i];
          dx = fmaf(gub, ex, dx);                  // through expm1(x)
          dAacc[i] = fmaf(gub, -em1 * ia[i], dAacc[i]);
          dBp[i] = ge * uu;
          duv = fmaf(ge, Bv, duv);
          dd = fmaf(dx, a[i], dd);
        } else {
          dBp[i] = g[i] * uu * dl;
          duv = fmaf(g[i] * dl, Bv, duv);
          dd = fmaf(dx, a[i], dd);
          dd = fmaf(g[i] * uu, Bv, dd);
        }
        dAacc[i] = fmaf(dx, dl, dAacc[i]);
        g[i] *= ex;
      }
      // sums over the 16 states: the 4 lanes of the channel
      dd += __shfl_xor_sync(0xffffffffu, dd, 1);  dd += __shfl_xor_sync(0xffffffffu, dd, 2);
      duv += __shfl_xor_sync(0xffffffffu, duv, 1); duv += __shfl_xor_sync(0xffffffffu, duv, 2);
      if (q == 0) {
        s_dd[r][cl] = dd;
        s_du[r][cl] = fmaf(Dc, ev, duv);
        dDacc = fmaf(ev, uu, dDacc);
      }
      // sums over channels: the 8 channels of a warp hold 8 values each (4 dB, 4 dC of the lane's states); three exchange
      // steps halve the values a lane keeps while adding its partner's, so every lane ends with ONE fully reduced value
      // (7 shuffles instead of 24), then the block's warps meet in shared-memory atomics
      {
        float v[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) { v[i] = c_ok ? dBp[i] : 0.0f; v[4 + i] = dCp[i]; }
        const bool b2 = lane & 4, b3 = lane & 8, b4 = lane & 16;
        float w4[4], w2[2];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float send = b2 ? v[i] : v[4 + i], keep = b2 ? v[4 + i] : v[i];
          w4[i] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const float send = b3 ? w4[i] : w4[2 + i], keep = b3 ? w4[2 + i] : w4[i];
          w2[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
        }
        const float send = b4 ? w2[0] : w2[1], keep = b4 ? w2[1] : w2[0];
        const float tot = keep + __shfl_xor_sync(0xffffffffu, send, 16);
        const int idx = (b2 ? 4 : 0) + (b3 ? 2 : 0) + (b4 ? 1 : 0);      // which of the 8 values this lane ended with
        float* dst = idx < 4 ? &s_dB[r][4 * q + idx] : &s_dC[r][4 * q + (idx - 4)];
        atomicAdd(dst, tot);
      }
    }
    __syncthreads();

    // ---- write the chunk's outputs
    for (int i = tid; i < CK * BCH; i += BT) {
      const int r = i / BCH, j = i % BCH;
      if (r < nt && c_base + j < p.De) {
        const size_t e = (b * p.L + t0 + r) * p.De + c_base + j;
        p.ddelta[e] = s_dd[r][j];
        du[e] = from_f32<T>(s_du[r][j]);
        if (z) {
          const float zz = s_z[r][j], sg = sigmoid_f(zz);
          dz[(b * p.L + t0 + r) * p.ldz + c_base + j] = from_f32<T>(s_dy[r][j] * s_y[r][j] * sg * (1.0f + zz * (1.0f - sg)));
        }
      }
    }
    for (int i = tid; i < CK * NST; i += BT) {
      const int r = i / NST, n = i % NST;
      if (r < nt) {
        atomicAdd(p.dBm + (b * p.L + t0 + r) * NST + n, s_dB[r][n]);
        atomicAdd(p.dCm + (b * p.L + t0 + r) * NST + n, s_dC[r][n]);
      }
    }
    __syncthreads();
  }

  if (c_ok) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      atomicAdd(p.dA + (size_t)c * NST + 4 * q + i, dAacc[i]);
      if (p.dh0 && cj == 0) p.dh0[(b * p.De + c) * NST + 4 * q + i] = g[i];
    }
    if (q == 0 && p.dD) atomicAdd(p.dD + c, dDacc);
  }
}


// Pre-pass of the chunk-parallel form, one coarse chunk per blockIdx.z: from a zero gradient, the gradient that leaves the
// chunk's start (g <- a_t (g + C_t e_t), t descending).  (The chunk's end state and sum of Delta from a zero state come
// from the forward scan kernel's state-only mode.)
template <typename T>
__global__ void __launch_bounds__(BT)
scan_bwd_prepass_kernel(const BwdArgs p) {
  const int tid = threadIdx.x, cl = tid >> 2, q = tid & 3;
  const int c = blockIdx.x * BCH + cl;
  const size_t b = blockIdx.y;
  if (c >= p.De) return;
  const int cj = blockIdx.z;
  const int t_lo = cj * p.Lc, t_hi = min(t_lo + p.Lc, p.L);
  const T* __restrict__ dy = static_cast<const T*>(p.dy);
  const T* __restrict__ z = static_cast<const T*>(p.z);
  float a[4], g[4] = {0.0f, 0.0f, 0.0f, 0.0f};
#pragma unroll
  for (int i = 0; i < 4; ++i) a[i] = p.A[(size_t)c * NST + 4 * q + i];
  constexpr bool PRECISE = sizeof(T) == 4;
  constexpr int G = 8;                            // steps whose loads are in flight together
  for (int t4 = t_hi - 1; t4 >= t_lo; t4 -= G) {
    float dl[G], ev[G], zz[G];
    float4 C4[G];
#pragma unroll
    for (int j = 0; j < G; ++j) {
      const int t = max(t4 - j, t_lo);
      const size_t e = (b * p.L + t) * p.De + c;
      dl[j] = p.delta[e];
      ev[j] = to_f32(dy[e]);
      zz[j] = z ? to_f32(z[(b * p.L + t) * p.ldz + c]) : 0.0f;
      C4[j] = *reinterpret_cast<const float4*>(p.Cm + (b * p.L + t) * NST + 4 * q);
    }
#pragma unroll
    for (int j = 0; j < G; ++j) {
      if (t4 - j < t_lo) break;
      if (z) ev[j] *= zz[j] * sigmoid_f(zz[j]);
      const float cv[4] = {C4[j].x, C4[j].y, C4[j].z, C4[j].w};
#pragma unroll
      for (int i = 0; i < 4; ++i) g[i] = fmaf(cv[i], ev[j], g[i]) * exp_only<PRECISE>(dl[j] * a[i]);
    }
  }
  const size_t o = ((b * p.ncc + cj) * p.De + c) * NST + 4 * q;
  *reinterpret_cast<float4*>(p.q_start + o) = make_float4(g[0], g[1], g[2], g[3]);
}

// Composes the coarse chunks (both recurrences are linear): with P_j = exp(A sum_delta_j),
//   h_in[0] = h0,  h_in[j+1] = P_j h_in[j] + h_end[j];   g_in[ncc-1] = dh_last,  g_in[j-1] = P_j g_in[j] + q_start[j].
__global__ void __launch_bounds__(256)
scan_bwd_chain_kernel(const float* __restrict__ A, const float* __restrict__ h0, const float* __restrict__ dh_last,
                      const float* __restrict__ h_end, const float* __restrict__ q_start, const float* __restrict__ sum_delta,
                      float* __restrict__ h_in, float* __restrict__ g_in, int B, int De, int ncc) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (long long)B * De * NST) return;
  const int n = (int)(i % NST);
  const int c = (int)((i / NST) % De);
  const size_t b = (size_t)(i / ((long long)NST * De));
  const float a = A[(size_t)c * NST + n];
  float h = h0 ? h0[i] : 0.0f;
  for (int j = 0; j < ncc; ++j) {
    const size_t sq = b * ncc + j;
    h_in[(sq * De + c) * NST + n] = h;
    h = fmaf(expf(a * sum_delta[sq * De + c]), h, h_end[(sq * De + c) * NST + n]);
  }
  float g = dh_last ? dh_last[i] : 0.0f;
  for (int j = ncc - 1; j >= 0; --j) {
    const size_t sq = b * ncc + j;
    g_in[(sq * De + c) * NST + n] = g;
    g = fmaf(expf(a * sum_delta[sq * De + c]), g, q_start[(sq * De + c) * NST + n]);
  }
}

// Coarse chunks per sequence: 1 when batch x channels already give about 2048 blocks' worth of work, else enough chunks
// (each a multiple of CK steps, at least 4 CK) to get there.  A function of the sizes only (workspace sizing = launch).
int coarse_chunks(int B, int De, int L, int* Lc_out) {
  const long long blocks1 = (long long)B * ((De + BCH - 1) / BCH);
  int ncc = 1;
  if (blocks1 < 1024) {
    ncc = (int)((2048 + blocks1 - 1) / blocks1);
    const int max_ncc = (L + 4 * CK - 1) / (4 * CK);
    if (ncc > max_ncc) ncc = max_ncc;
    if (ncc < 1) ncc = 1;
  }
  int Lc = (L + ncc - 1) / ncc;
  Lc = (Lc + CK - 1) / CK * CK;
  ncc = (L + Lc - 1) / Lc;
  *Lc_out = Lc;
  return ncc;
}

}  // namespace

size_t scan_bwd_ws_bytes(int B, int De, int L) {
  const size_t nck = (size_t)(L + CK - 1) / CK;
  int Lc = 0;
  const int ncc = coarse_chunks(B, De, L, &Lc);
  size_t floats = (size_t)B * nck * De * NST;
  if (ncc > 1) floats += (size_t)B * ncc * De * (4 * NST + 1);
  return align_up(sizeof(float) * floats, 256);
}

cudaError_t launch_scan_backward(const rom_config& c, const void* dy, const void* u, const float* delta, const float* A,
                                 const float* Bm, const float* Cm, const float* D, const void* z, const float* h0,
                                 const float* dh_last, void* du, float* ddelta, float* dA, float* dBm, float* dCm, float* dD,
                                 void* dz, float* dh0, float* ckpt, int ldz, cudaStream_t st) {
  const int nck = (c.L + CK - 1) / CK;
  int Lc = 0;
  const int ncc = coarse_chunks(c.B, c.d_inner, c.L, &Lc);
  const size_t n_fine = (size_t)c.B * nck * c.d_inner * NST, n_coarse = (size_t)c.B * ncc * c.d_inner * NST;
  float* h_end = ckpt + n_fine;
  float* q_start = h_end + n_coarse;
  float* h_in = q_start + n_coarse;
  float* g_in = h_in + n_coarse;
  float* sum_delta = g_in + n_coarse;
  const BwdArgs a{dy, u, delta, A, Bm, Cm, D, z, h0, dh_last, du, ddelta, dA, dBm, dCm, dD, dz, dh0, ckpt, c.L, c.d_inner, nck, ldz,
                  Lc, ncc, h_in, g_in, h_end, q_start, sum_delta};
  cudaError_t e = cudaMemsetAsync(dA, 0, sizeof(float) * (size_t)c.d_inner * NST, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(dBm, 0, sizeof(float) * (size_t)c.B * c.L * NST, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(dCm, 0, sizeof(float) * (size_t)c.B * c.L * NST, st);
  if (e == cudaSuccess && dD) e = cudaMemsetAsync(dD, 0, sizeof(float) * (size_t)c.d_inner, st);
  if (e != cudaSuccess) return e;
  const dim3 grid((c.d_inner + BCH - 1) / BCH, c.B, ncc);
  const bool zoh = c.disc_mode == 0, bf = c.dtype == ROM_BF16;
  if (ncc > 1) {
    // chunk end states and sums of Delta from a zero state (forward scan kernel, state-only), chunk-start gradients from zero
    if ((e = launch_scan_states(c, u, delta, A, Bm, Lc, ncc, nullptr, h_end, sum_delta, nullptr, 0, st)) != cudaSuccess) return e;
    if (bf) scan_bwd_prepass_kernel<__nv_bfloat16><<<grid, BT, 0, st>>>(a); else scan_bwd_prepass_kernel<float><<<grid, BT, 0, st>>>(a);
    count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    const long long n_thr = (long long)c.B * c.d_inner * NST;
    scan_bwd_chain_kernel<<<(unsigned)((n_thr + 255) / 256), 256, 0, st>>>(A, h0, dh_last, h_end, q_start, sum_delta, h_in, g_in, c.B, c.d_inner, ncc);
    count_launch();
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
  }
  // the state at the start of every 16 steps, from the true chunk-start states (forward scan kernel, state-only)
  if ((e = launch_scan_states(c, u, delta, A, Bm, Lc, ncc, ncc > 1 ? h_in : h0, nullptr, nullptr, ckpt, nck, st)) != cudaSuccess) return e;
  auto kern = bf ? (zoh ? scan_bwd_kernel<__nv_bfloat16, true> : scan_bwd_kernel<__nv_bfloat16, false>)
                 : (zoh ? scan_bwd_kernel<float, true> : scan_bwd_kernel<float, false>);
  if ((e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)BWD_SMEM)) != cudaSuccess) return e;
  kern<<<grid, BT, BWD_SMEM, st>>>(a);
  count_launch();
  return cudaGetLastError();
}

}  // namespace rom
