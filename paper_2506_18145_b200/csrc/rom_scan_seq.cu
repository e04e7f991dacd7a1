// Selective scan (Section 3.1) of FEW long sequences in ONE pass: h_t = exp(Delta_t A) h_{t-1} + B-bar_t U_t,
// Y_t = C_t h_t + D U_t, times the gate.  bf16 storage, fp32 state and arithmetic, one ex2.approx per state update.
//
// With one or two sequences there are only B * D_e * 16 independent recurrences, too few to fill the GPU in the
// shape of the general kernel (rom_scan.cu), which then needs a workspace to cut the sequence into chunks (and
// evaluates most exponentials twice).  This kernel needs no workspace: it runs at very low occupancy, one warp per
// SM sub-partition, and covers latency with independent work of the same warp.
//
//   * a warp owns 8 channels; lane = 4 * channel + g owns states [4g, 4g + 4) of its channel (two packed pairs);
//     a block is 4 independent warps (32 channels of one sequence); nothing is shared between warps;
//   * each warp streams its own operands with 16-byte cp.async copies into a private ring of tiles of 32 steps
//     (Delta, u, z: its 8 channels; B, C: all 16 states; the output rows when they are scattered): no block-wide
//     barrier, no spin-wait (cp.async.wait_group + __syncwarp only), copies stay inside the sequence;
//   * per step and thread: 4 shared-memory loads (all lanes of a channel read the same Delta / u word, all
//     channels the same B / C quad), 4 exponentials, 14 packed fp32 operations;
//   * the sum over states of C h is finished four steps at a time by a transposing exchange (3 shuffles): lane g
//     ends up with the sum of step g of the group, adds D u, applies the gate, rounds and stores that one value;
//   * the loop is software-pipelined by hand over groups of four steps (six stages, see the kernel).
// Measured on one 16384-step sequence of 4096 channels (fp32 Delta, raw gate): 0.74 ms (the general kernel without a
// workspace: 1.04 ms; with a workspace, chunked: 0.67 ms).  What binds is not the special-function unit: with every shared-memory load,
// exponential and shuffle taken out the remaining fp32 / integer stream alone needs 0.48 ms, and two sequences take
// 1.8 x the time of one, i.e. the fp32 pipes are the limit (a packed fp32 operation occupies them for two cycles:
// 128 lanes per clock per SM, packed or not, as measured).
#include <cuda_bf16.h>

#include <type_traits>

#include "rom_internal.cuh"

namespace rom {
namespace {

constexpr int NST = 16;          // d_state
constexpr int Q_WARPS = 4;       // warps per block
constexpr int Q_CH = 8;          // channels per warp
constexpr int Q_TT = 32;         // steps per tile
constexpr int Q_STAGES = 4;      // tiles in the ring of a warp
constexpr float kLog2e = 1.4426950408889634f;

template <typename TD>
struct __align__(16) SeqStage {
  TD delta[Q_TT][Q_CH];
  __nv_bfloat16 u[Q_TT][Q_CH];
  __nv_bfloat16 z[Q_TT][Q_CH];
  float Bm[Q_TT][NST];
  float Cm[Q_TT][NST];
  int32_t rows[Q_TT];              // output row of each step (only when the caller scatters the rows)
};

struct SeqArgs {
  const void* u; const void* delta; const float* A; const float* Bm; const float* Cm; const float* D;
  const void* z; int ldz; const float* h0; void* y; float* h_last; const int32_t* y_rows;
  int K, L, De, gate_activated;
};

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void cp_async16(void* dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async4(void* dst, const void* src) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ float raw_f32(float v) { return v; }
__device__ __forceinline__ float raw_f32(__nv_bfloat16 v) { return __bfloat162float(v); }

// GATE: 0 no gate, 1 z holds SiLU(gate) already, 2 z holds the raw gate.  ROWS: outputs go to the rows listed in y_rows.
template <typename TD, bool ZOH, int GATE, bool ROWS>
__global__ void __launch_bounds__(Q_WARPS * 32, 1)
scan_seq_kernel(const SeqArgs p) {
  using Stage = SeqStage<TD>;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  Stage* stages = reinterpret_cast<Stage*>(smem_raw) + warp * Q_STAGES;
  const int c0 = (blockIdx.x * Q_WARPS + warp) * Q_CH;        // first channel of this warp
  if (c0 >= p.De) return;                                      // whole warp (D_e is a multiple of 8)
  const int b = blockIdx.y;
  const int L = p.L, De = p.De;
  const int ch = lane >> 2, g = lane & 3;
  const int c = c0 + ch;
  const size_t tok0 = (size_t)b * L;

  const TD* __restrict__ gd = static_cast<const TD*>(p.delta) + tok0 * De + c0;
  const __nv_bfloat16* __restrict__ gu = static_cast<const __nv_bfloat16*>(p.u) + tok0 * De + c0;
  const __nv_bfloat16* __restrict__ gz = GATE ? static_cast<const __nv_bfloat16*>(p.z) + tok0 * p.ldz + c0 : nullptr;
  const float* __restrict__ gB = p.Bm + tok0 * NST;
  const float* __restrict__ gC = p.Cm + tok0 * NST;
  __nv_bfloat16* __restrict__ y = static_cast<__nv_bfloat16*>(p.y);

  // copies of one tile: lane i brings row i of Delta, u, z and four 16-byte pieces of B and of C
  auto issue = [&](int tile) {
    Stage& s = stages[tile % Q_STAGES];
    const int t = tile * Q_TT + lane;
    if (t < L) {
      const char* src = reinterpret_cast<const char*>(gd + (size_t)t * De);
#pragma unroll
      for (int k = 0; k < (int)(sizeof(TD) * Q_CH / 16); ++k) cp_async16(reinterpret_cast<char*>(&s.delta[lane][0]) + 16 * k, src + 16 * k);
      cp_async16(&s.u[lane][0], gu + (size_t)t * De);
      if (GATE) cp_async16(&s.z[lane][0], gz + (size_t)t * p.ldz);
      if (ROWS) cp_async4(&s.rows[lane], p.y_rows + tok0 + t);
    }
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int piece = lane + 32 * k;                  // 16-byte piece of the [32][16] fp32 tile
      const int tr = tile * Q_TT + (piece >> 2);
      if (tr < L) {
        cp_async16(reinterpret_cast<char*>(&s.Bm[0][0]) + 16 * piece, reinterpret_cast<const char*>(gB + (size_t)tile * Q_TT * NST) + 16 * piece);
        cp_async16(reinterpret_cast<char*>(&s.Cm[0][0]) + 16 * piece, reinterpret_cast<const char*>(gC + (size_t)tile * Q_TT * NST) + 16 * piece);
      }
    }
  };

  // per-thread constants and state
  float2 a2[2], kin[2], h[2];
#pragma unroll
  for (int q = 0; q < 2; ++q) {
    const int n = 4 * g + 2 * q;
    const float a0 = p.A[(size_t)c * NST + n], a1 = p.A[(size_t)c * NST + n + 1];
    a2[q] = make_float2(a0 * kLog2e, a1 * kLog2e);
    kin[q] = make_float2(-1.0f / a0, -1.0f / a1);
    h[q] = p.h0 ? make_float2(p.h0[((size_t)b * De + c) * NST + n], p.h0[((size_t)b * De + c) * NST + n + 1]) : make_float2(0.0f, 0.0f);
  }
  const float Dc = p.D ? p.D[c] : 0.0f;
  const bool odd1 = (g & 1) != 0, odd2 = (g & 2) != 0;

  // One warp per scheduler: every latency has to be covered by independent work of the same warp.  The work of a group
  // of four steps is therefore cut into six stages that hand their results on in registers, and iteration k of the loop
  // runs stage 1 of group k+2, stage 2 of group k+1, ... stage 6 of group k-3: every producer of a long-latency result
  // (shared-memory load, exponential, shuffle) is a whole iteration ahead of its consumer.
  //   S1 raw operand loads;  S2 conversions, exponentials, input terms w;  S3 the recurrence and the partial sums C h;
  //   S4, S5 the two steps of the exchange that finishes the sums;  S6 skip term, gate, rounding, store.
  struct Raw {
    TD d[4];
    __nv_bfloat16 u[4];
    float4 B4[4], C4[4];
    __nv_bfloat16 ue, ze;    // u and gate of the step this lane finishes (step g of the group)
    int row;                 // its output row
  };
  struct Ops {
    float2 a[4][2], w[4][2];
    float4 C4[4];
  };
  struct Meta { float ue, ze; int row; };
  struct X1 { float k0, k1, r0, r1; Meta m; };       // kept partial sums and what the partner sent (first exchange)
  struct X2 { float k, r; Meta m; };                 // the same for the second exchange

  auto S1 = [&](int grp, Raw& o) {
    const Stage& s = stages[(grp >> 3) % Q_STAGES];
    const int r0 = (grp & 7) * 4;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      o.d[j] = s.delta[r0 + j][ch];
      o.u[j] = s.u[r0 + j][ch];
      o.B4[j] = *reinterpret_cast<const float4*>(&s.Bm[r0 + j][4 * g]);
      o.C4[j] = *reinterpret_cast<const float4*>(&s.Cm[r0 + j][4 * g]);
    }
    o.ue = s.u[r0 + g][ch];
    if (GATE) o.ze = s.z[r0 + g][ch];
    if (ROWS) o.row = s.rows[r0 + g];
  };
  auto S2 = [&](const Raw& in, Ops& o, Meta& m) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float dl = raw_f32(in.d[j]);
      const float uu = raw_f32(in.u[j]);
      const float vv = ZOH ? uu : dl * uu;
      const float2 dl2 = make_float2(dl, dl), vv2 = make_float2(vv, vv);
      o.C4[j] = in.C4[j];
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        const float2 Bv = q ? make_float2(in.B4[j].z, in.B4[j].w) : make_float2(in.B4[j].x, in.B4[j].y);
        const float2 x = __fmul2_rn(dl2, a2[q]);
        o.a[j][q] = make_float2(ex2_approx(x.x), ex2_approx(x.y));
        // zero-order hold: w = -B u / A (h <- a (h - w) + w); otherwise w = (Delta u) B (h <- a h + w)
        o.w[j][q] = ZOH ? __fmul2_rn(__fmul2_rn(vv2, kin[q]), Bv) : __fmul2_rn(vv2, Bv);
      }
    }
    m.ue = raw_f32(in.ue);
    m.ze = GATE ? raw_f32(in.ze) : 1.0f;
    m.row = ROWS ? in.row : 0;
  };
  auto S3 = [&](const Ops& o, float (&part)[4], auto fast_tag, int nvalid) {
    constexpr bool FAST = decltype(fast_tag)::value;      // every step of the group is inside the sequence
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      float2 hn[2];
#pragma unroll
      for (int q = 0; q < 2; ++q) {
        if (ZOH) {
          const float2 sdiff = __ffma2_rn(o.w[j][q], make_float2(-1.0f, -1.0f), h[q]);
          hn[q] = __ffma2_rn(o.a[j][q], sdiff, o.w[j][q]);
        } else {
          hn[q] = __ffma2_rn(o.a[j][q], h[q], o.w[j][q]);
        }
      }
      if (FAST || j < nvalid) { h[0] = hn[0]; h[1] = hn[1]; }
      const float2 acc = __ffma2_rn(make_float2(o.C4[j].z, o.C4[j].w), hn[1], __fmul2_rn(make_float2(o.C4[j].x, o.C4[j].y), hn[0]));
      part[j] = acc.x + acc.y;
    }
  };
  // transposing exchange over the 4 lanes of the channel: lane g ends with the full sum of step g of the group
  auto S4 = [&](const float (&part)[4], const Meta& m, X1& x) {
    x.k0 = odd1 ? part[1] : part[0];                                               // step (g & 1)
    x.k1 = odd1 ? part[3] : part[2];                                               // step 2 + (g & 1)
    x.r0 = __shfl_xor_sync(0xffffffffu, odd1 ? part[0] : part[1], 1);
    x.r1 = __shfl_xor_sync(0xffffffffu, odd1 ? part[2] : part[3], 1);
    x.m = m;
  };
  auto S5 = [&](const X1& in, X2& x) {
    const float k0 = in.k0 + in.r0, k1 = in.k1 + in.r1;
    x.k = odd2 ? k1 : k0;                                                          // step g
    x.r = __shfl_xor_sync(0xffffffffu, odd2 ? k0 : k1, 2);
    x.m = in.m;
  };
  auto S6 = [&](int grp, const X2& in, auto fast_tag) {
    constexpr bool FAST = decltype(fast_tag)::value;
    const int t = grp * 4 + g;
    if (FAST || (grp >= 0 && t < L)) {
      float o = fmaf(Dc, in.m.ue, in.k + in.r);
      if (GATE == 1) o *= in.m.ze;
      if (GATE == 2) o *= silu_fast(in.m.ze);
      const size_t orow = ROWS ? (size_t)in.m.row : tok0 + (size_t)t;
      y[orow * De + c] = __float2bfloat16_rn(o);
    }
  };

  const int ntiles = (L + Q_TT - 1) / Q_TT;
  const int ngroups = (L + 3) / 4;                   // the last one may be partial
  const int nfull = L / 4;
  const int niter = ngroups + 3;                     // three more iterations drain the last groups through S4..S6
#pragma unroll
  for (int k = 0; k < Q_STAGES - 1; ++k) {
    if (k < ntiles) issue(k);
    cp_async_commit();
  }
  cp_async_wait<Q_STAGES - 2>();                     // tile 0 has landed
  __syncwarp();
  Raw rc, rn;
  Ops ops, opn;
  Meta mc, mn;
  float part[4] = {0.0f, 0.0f, 0.0f, 0.0f};
  X1 x1{};
  X2 x2{};
  S1(0, rc);
  S2(rc, ops, mc);
  S1(1, rc);
  Meta mprev = mc;                                   // meta of the group whose partial sums are in part[]
  for (int i = 0; 8 * i < niter; ++i) {
    __syncwarp();                                    // every lane has taken what it needs from tile i - 1 (S1 runs two groups ahead)
    if (i + Q_STAGES - 1 < ntiles) issue(i + Q_STAGES - 1);      // refills the stage of tile i - 1
    cp_async_commit();
    cp_async_wait<Q_STAGES - 2>();                   // tiles <= i + 1 have landed (this thread's copies) ...
    __syncwarp();                                    // ... and the other lanes'
    if (i > 0 && 8 * i + 8 <= nfull) {
      // a tile in the middle of the sequence: no step to skip, no group index to check: straight-line code
#pragma unroll
      for (int gg = 0; gg < 8; ++gg) {
        const int k = 8 * i + gg;
        X2 x2n; X1 x1n;
        S6(k - 3, x2, std::true_type{});
        S5(x1, x2n);
        S4(part, mprev, x1n);
        S3(ops, part, std::true_type{}, 4);
        mprev = mc;
        S2(rc, opn, mn);
        S1(k + 2, rn);
        rc = rn; ops = opn; mc = mn; x1 = x1n; x2 = x2n;
      }
    } else {
      const int kend = min(8 * i + 8, niter);
      for (int k = 8 * i; k < kend; ++k) {
        X2 x2n; X1 x1n;
        S6(k - 3, x2, std::false_type{});
        S5(x1, x2n);
        S4(part, mprev, x1n);
        S3(ops, part, std::false_type{}, k < nfull ? 4 : max(0, L - 4 * k));
        mprev = mc;
        S2(rc, opn, mn);
        S1(k + 2, rn);
        rc = rn; ops = opn; mc = mn; x1 = x1n; x2 = x2n;
      }
    }
  }

  if (p.h_last) {
    float4* dst = reinterpret_cast<float4*>(p.h_last + ((size_t)b * De + c) * NST + 4 * g);
    *dst = make_float4(h[0].x, h[0].y, h[1].x, h[1].y);
  }
}

template <typename TD, bool ZOH, int GATE, bool ROWS>
cudaError_t launch_seq_k(const SeqArgs& a, int B, cudaStream_t st) {
  const size_t smem = sizeof(SeqStage<TD>) * Q_STAGES * Q_WARPS;
  auto kern = scan_seq_kernel<TD, ZOH, GATE, ROWS>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid((a.De + Q_WARPS * Q_CH - 1) / (Q_WARPS * Q_CH), B);
  kern<<<grid, Q_WARPS * 32, smem, st>>>(a);
  count_launch();
  return cudaGetLastError();
}
template <typename TD, bool ZOH>
cudaError_t launch_seq_t(const SeqArgs& a, int B, cudaStream_t st) {
  // the entry point that reaches this kernel passes the raw gate (or none) and writes rows in token order
  return a.z == nullptr ? launch_seq_k<TD, ZOH, 0, false>(a, B, st) : launch_seq_k<TD, ZOH, 2, false>(a, B, st);
}

bool aligned16p(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

bool scan_seq_applicable(const rom_config& c, const void* u, const void* delta, bool delta_fp32, const float* Bm, const float* Cm,
                         const void* z, int ldz, const int32_t* z_row, const int32_t* y_rows, bool gate_activated, int num_sms) {
  if (y_rows != nullptr || (z != nullptr && gate_activated)) return false;      // only the plain forms are instantiated
  if (c.dtype != ROM_BF16 || c.d_state != NST || c.L < 2 || z_row != nullptr) return false;
  if (c.d_inner % Q_CH != 0 || (z && ldz % Q_CH != 0)) return false;
  if (!aligned16p(u) || !aligned16p(delta) || !aligned16p(Bm) || !aligned16p(Cm) || (z && !aligned16p(z))) return false;
  (void)delta_fp32;
  // few independent recurrences: at most two warps of this kernel per SM sub-partition
  const long long warps = (long long)c.B * ((c.d_inner + Q_CH - 1) / Q_CH);
  return warps <= 2LL * 4 * num_sms;
}

cudaError_t launch_scan_seq(const rom_config& c, const void* u, const void* delta, bool delta_fp32, const float* A, const float* Bm,
                            const float* Cm, const float* D, const void* z, int ldz, const float* h0, void* y, float* h_last,
                            const int32_t* y_rows, int K, bool gate_activated, cudaStream_t st) {
  const SeqArgs a{u, delta, A, Bm, Cm, D, z, ldz, h0, y, h_last, y_rows, K, c.L, c.d_inner, gate_activated ? 1 : 0};
  const bool zoh = c.disc_mode == 0;
  if (delta_fp32) return zoh ? launch_seq_t<float, true>(a, c.B, st) : launch_seq_t<float, false>(a, c.B, st);
  return zoh ? launch_seq_t<__nv_bfloat16, true>(a, c.B, st) : launch_seq_t<__nv_bfloat16, false>(a, c.B, st);
}

}  // namespace rom
