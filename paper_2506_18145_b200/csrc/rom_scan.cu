// Selective scan (Section 3.1): h_t = exp(Delta_t A) h_{t-1} + B-bar_t U_t, Y_t = C_t h_t (+ D U_t),
// fused with the output gate y * SiLU(z) and with the re-permutation of the gated rows into expert
// order (the routing decision of the Gate/Conv projections is reused for Out Proj, Section 4.2).
//
// State and arithmetic are fp32.  The recurrence is sequential in t, so the parallelism is
// (sequence, channel, state).  One thread owns NS of the 16 states of NC adjacent channels
// (registers, packed pairs); the S = 16/NS lanes of a channel group are adjacent.  Per state and step
// the work is one exponential on the special-function unit (16 per clock per SM: the binding limit),
// about six fp32 multiply/FMA lanes, and the shared-memory words for (Delta, u) and (B, C).  The
// launcher picks the largest work per thread that still fills the GPU (small NS only for a single
// long sequence).
//
// A single long sequence does not have enough (channel, state) lanes for the efficient shapes, so
// the sequence is then cut into chunks that run in parallel, in two passes: pass 1 scans every chunk
// from a zero state and keeps only its final state and sum of Delta; a small kernel chains the
// chunk states (h_in[j+1] = exp(A sum_j Delta) h_in[j] + h_end[j], exact because the recurrence is
// linear in h); pass 2 is the full scan of every chunk from its true initial state.  The
// exponentials are evaluated twice; in exchange every SM runs the shape that keeps its pipes busy.
//
// A block of 256 threads owns CH = NC*256/S channels of one sequence and walks the sequence in tiles
// of TS = 2048/CH steps, so every thread also owns one (row, 8 channels) piece of each tile: it
// fetches that piece of tile i+1 (Delta, u, z) from global memory into registers -- raw,
// unconverted, so nothing waits on the loads -- while tile i is computed from shared memory, then
// converts and stores it to the other shared buffer.  The scan proper leaves sum_n C h in shared
// memory; the skip term, the gate, the rounding and the 16-byte row stores are done by the thread
// that loaded that piece, which still holds u and z in registers.  One __syncthreads per tile.  The
// per-channel operands are stored once, (Delta, v), and duplicated into packed pairs in registers: the
// path that returns shared-memory data to the register file (128 bytes per clock per SM, one copy per
// lane whatever the sharing) is as busy as the special-function unit in this kernel, so every byte
// counts; the channel pairs of an 8-channel group are rotated so that loader stores and compute loads
// are both bank-conflict free.
#include <type_traits>

#include <cmath>

#include "rom_internal.cuh"

namespace rom {
namespace {

constexpr int NST = 16;            // d_state
constexpr int BLOCK = 256;
constexpr int TILE_ELEMS = 2048;   // (time steps) x (channels) per tile = 8 per thread
constexpr float kLog2e = 1.4426950408889634f;

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// 8 consecutive elements of a row, kept raw (16-byte words) until consumed.
template <typename T> struct Raw8;
template <> struct Raw8<__nv_bfloat16> {
  uint4 q;
  __device__ __forceinline__ void load(const __nv_bfloat16* p) { q = __ldg(reinterpret_cast<const uint4*>(p)); }
  __device__ __forceinline__ void zero() { q = make_uint4(0, 0, 0, 0); }
  __device__ __forceinline__ void get(float (&v)[8]) const {
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&v)[8]) {
    uint4 o;
    uint32_t* w = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 hh = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
      w[i] = *reinterpret_cast<const uint32_t*>(&hh);
    }
    *reinterpret_cast<uint4*>(p) = o;
  }
};
template <> struct Raw8<float> {
  float4 a, b;
  __device__ __forceinline__ void load(const float* p) {
    a = __ldg(reinterpret_cast<const float4*>(p));
    b = __ldg(reinterpret_cast<const float4*>(p) + 1);
  }
  __device__ __forceinline__ void zero() { a = make_float4(0.0f, 0.0f, 0.0f, 0.0f); b = a; }
  __device__ __forceinline__ void get(float (&v)[8]) const {
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
  }
  static __device__ __forceinline__ void store(float* p, const float (&v)[8]) {
    reinterpret_cast<float4*>(p)[0] = make_float4(v[0], v[1], v[2], v[3]);
    reinterpret_cast<float4*>(p)[1] = make_float4(v[4], v[5], v[6], v[7]);
  }
};

template <int NC, int NS>
struct Geo {
  static constexpr int S = NST / NS;                    // lanes per channel group
  static constexpr int NP = NS / 2;                     // packed state pairs per channel per thread
  static constexpr int CH = BLOCK / S * NC;             // channels per block
  static constexpr int TS = TILE_ELEMS / CH;            // time steps per tile
  static constexpr int CG = CH / 8;                     // 8-channel groups (= loader threads) per row
  static constexpr int SLOT = 32 + 32 / S;              // words per time slot of the partial-sum strip (padded)
  static constexpr int STRIP = S > 4 ? S * SLOT : 0;    // words per warp (only the 8-lane split uses the strip)
  static constexpr int YP = CH + (S > 4 ? 4 : 0);       // row pitch (words) of the staged sums
  static constexpr int NBC = TS * 32 / BLOCK;           // B/C words fetched per thread per tile
  static_assert(NS % 2 == 0 && S >= 1 && S <= 8 && TS % S == 0 && CG * TS == BLOCK && (NC == 1 || S <= 4), "unsupported split");
};

// position of channel c inside its tile row: the 8 channels of a group are permuted by the group index
// (the four channel pairs of a group are rotated by half the group index: a loader thread's four 16-byte stores then
// fall into different banks than its neighbours')
__device__ __forceinline__ int swz(int c) { return (c & ~7) | ((((c >> 1) + (c >> 4)) & 3) << 1) | (c & 1); }

// Shared-memory image of one input tile.
template <int NC, int NS>
struct Tile {
  float2 dv[Geo<NC, NS>::TS][Geo<NC, NS>::CH];   // (Delta, v) at [t][swz(c)]: v = u (zero-order hold) or Delta*u
  float4 bc[Geo<NC, NS>::TS][NST / 2];           // (B_n, B_n+1, C_n, C_n+1) per state pair
};

struct ScanArgs {
  const void* u; const void* delta; const float* A; const float* Bm; const float* Cm; const float* D;
  const void* z; int ldz; const int32_t* z_row; const float* h0; void* y; float* h_last; const int32_t* y_rows;
  int K, L, De;
  int Lc, nch;          // chunk length and chunks per sequence (nch == 1: Lc == L); blockIdx.z = chunk
  int L0;               // length of chunk 0; chunk j >= 1 covers steps [L0 + (j-1) Lc, L0 + j Lc)
  float* sum_delta;     // state-only blocks: [B*nch, De] sum of Delta over the chunk
  int gate_activated;   // z already holds SiLU(gate pre-activation): multiply only
  int chunk_off;        // chunk of blockIdx.z == 0
  float* ckpt;          // MODE 3: [B, nck, De, 16] state at the start of every 16 steps (nck per sequence)
  int nck;
  int scalar_a;         // A[c, :] is one value per channel (scalar-per-head decay of a Mamba2-style block): one exponential
                        // per channel and step instead of one per state (only with B-bar = Delta B)
};
// TD: type Delta is stored in: float (the rom_scan entry point, the fp32 layer) or the storage type (bf16 layer).

// PRECISE: libm-accurate exp / expm1 (fp32 configuration, 1e-4 tolerance); otherwise one ex2.approx per
// state update (bf16 configurations, 2e-2 tolerance).
// ZOH: zero-order-hold B-bar (disc_mode 0); otherwise B-bar = Delta B.
// MODE 0: full scan.  MODE 1: state only (no outputs, only h_last and sum_delta of every chunk).  MODE 3: state only
// from the given chunk-start states, storing the state at the start of every 16 steps (backward pass).  MODE 2: first
// launch of the chunked scan: chunk 0 runs the full scan from the caller's initial state (h0 indexed by
// sequence), the other chunks run state-only from a zero state.
template <typename T, typename TD, int NC, int NS, bool PRECISE, bool ZOH, int MODE>
__global__ void __launch_bounds__(BLOCK, NS >= 8 ? 2 : 1)
scan_kernel(const ScanArgs p) {
  using G = Geo<NC, NS>;
  using TileT = Tile<NC, NS>;
  constexpr int S = G::S, NP = G::NP, CH = G::CH, TS = G::TS, YP = G::YP;
  extern __shared__ __align__(16) unsigned char smem_raw[];
  TileT* tiles = reinterpret_cast<TileT*>(smem_raw);                                        // [2]
  float* ysum = reinterpret_cast<float*>(smem_raw + 2 * sizeof(TileT));                     // [2][TS][YP]
  float* ps_all = ysum + 2 * TS * YP;                                                       // [8 warps][STRIP]

  const T* __restrict__ u = static_cast<const T*>(p.u);

  T* __restrict__ y = static_cast<T*>(p.y);
  const int De = p.De, K = p.K;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int chunk = blockIdx.z + p.chunk_off;
  const bool so = MODE == 1 || MODE == 3 || (MODE == 2 && chunk != 0);  // this block only produces states
  const T* __restrict__ z = so ? nullptr : static_cast<const T*>(p.z);
  const int t_first = chunk == 0 ? 0 : p.L0 + (chunk - 1) * p.Lc;
  const int L = min(chunk == 0 ? p.L0 : p.Lc, p.L - t_first);   // steps of this chunk (<= 0: an empty chunk)
  const int b = blockIdx.y * p.nch + chunk;               // index of the (sequence, chunk) state
  const int c_base = blockIdx.x * CH;
  const size_t tok0 = (size_t)blockIdx.y * p.L + (size_t)t_first;

  // ---- compute role: NC adjacent channels from block-local channel cl, states [g*NS, g*NS+NS)
  const int cl = (tid / S) * NC, g = tid % S;
  float2 a2[NC][NP], kin[NC][NP], h[NC][NP];
  int cl_sw[NC];
#pragma unroll
  for (int i = 0; i < NC; ++i) {
    const int c = min(c_base + cl + i, De - 1);
    cl_sw[i] = swz(cl + i);
#pragma unroll
    for (int q = 0; q < NP; ++q) {
      const int n = g * NS + 2 * q;
      const float a0 = p.A[(size_t)c * NST + n], a1 = p.A[(size_t)c * NST + n + 1];
      a2[i][q] = PRECISE ? make_float2(a0, a1) : make_float2(a0 * kLog2e, a1 * kLog2e);
      kin[i][q] = make_float2(-1.0f / a0, -1.0f / a1);
      const size_t hb = MODE == 2 ? (size_t)blockIdx.y : (size_t)b;
      h[i][q] = (p.h0 && !(MODE == 2 && so)) ? make_float2(p.h0[(hb * De + c) * NST + n], p.h0[(hb * De + c) * NST + n + 1])
                                             : make_float2(0.0f, 0.0f);
    }
  }
  float* ps = ps_all + warp * G::STRIP;
  float sdel[NC];
#pragma unroll
  for (int i = 0; i < NC; ++i) sdel[i] = 0.0f;

  // ---- loader / finisher role: row lr of every tile, channels [lc, lc + 8)
  const int lr = tid / G::CG, lc = (tid % G::CG) * 8;
  const bool lc_ok = c_base + lc < De;
  const int lc_eff = lc_ok ? c_base + lc : 0;
  float dsk[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) dsk[i] = p.D ? p.D[lc_eff + i] : 0.0f;
  // running pointers to this thread's piece of the next tile to fetch
  const TD* dptr = static_cast<const TD*>(p.delta) + (tok0 + lr) * De + lc_eff;
  const T* uptr = u + (tok0 + lr) * De + lc_eff;
  const size_t row_step = (size_t)TS * De;
  // B/C: word i of this thread is element (r = warp + 8 i, j = lane) of the [TS][32] tile (B | C)
  const float* bcptr = (lane < NST ? p.Bm : p.Cm) + (tok0 + warp) * NST + (lane & 15);
  const int bc_dst = ((lane & 15) >> 1) * 4 + ((lane >> 4) << 1) + (lane & 1);

  Raw8<TD> pre_d;
  Raw8<T> pre_u, pre_z, cur_u, cur_z;
  float pre_bc[G::NBC];

  auto fetch = [&](int t0) {        // global -> registers, no conversion
    const int t = t0 + lr;
    pre_d.zero(); pre_u.zero(); pre_z.zero();
    if (lc_ok && t < L) {
      pre_d.load(dptr);
      pre_u.load(uptr);
      if (z) {
        const size_t zrow = p.z_row ? (size_t)__ldg(p.z_row + tok0 + t) : tok0 + t;
        pre_z.load(z + zrow * p.ldz + lc_eff);
      }
    }
    dptr += row_step; uptr += row_step;
#pragma unroll
    for (int i = 0; i < G::NBC; ++i) pre_bc[i] = (t0 + warp + 8 * i < L) ? __ldg(bcptr + i * 8 * NST) : 0.0f;
    bcptr += TS * NST;
  };
  auto stash = [&](TileT& tl) {     // registers -> shared, converting
    float d[8], uu[8];
    pre_d.get(d); pre_u.get(uu);
    float4* row = reinterpret_cast<float4*>(&tl.dv[lr][lc]);       // the group's four channel pairs
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float v0 = ZOH ? uu[2 * i] : d[2 * i] * uu[2 * i], v1 = ZOH ? uu[2 * i + 1] : d[2 * i + 1] * uu[2 * i + 1];
      row[(i + (lc >> 4)) & 3] = make_float4(d[2 * i], v0, d[2 * i + 1], v1);
    }
#pragma unroll
    for (int i = 0; i < G::NBC; ++i) reinterpret_cast<float*>(&tl.bc[warp + 8 * i][0])[bc_dst] = pre_bc[i];
  };
  // y = (sum_n C h + D u) * SiLU(z), rounded, written to the K output rows of the token
  auto flush = [&](int t0, const float* ys) {
    const int t = t0 + lr;
    if (!lc_ok || t >= L) return;
    float uu[8], o[8];
    cur_u.get(uu);
    const float4 s0 = *reinterpret_cast<const float4*>(ys + lr * YP + lc), s1 = *reinterpret_cast<const float4*>(ys + lr * YP + lc + 4);
    const float sv[8] = {s0.x, s0.y, s0.z, s0.w, s1.x, s1.y, s1.z, s1.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) o[i] = fmaf(dsk[i], uu[i], sv[i]);
    if (z) {
      float zz[8];
      cur_z.get(zz);
      if (p.gate_activated) {
#pragma unroll
        for (int i = 0; i < 8; ++i) o[i] *= zz[i];
      } else {
#pragma unroll
        for (int i = 0; i < 8; ++i)
          o[i] *= PRECISE ? zz[i] / (1.0f + expf(-zz[i])) : silu_fast(zz[i]);
      }
    }
    const size_t tok = tok0 + t;
    if (p.y_rows == nullptr) {
      Raw8<T>::store(y + tok * De + lc_eff, o);
    } else {
      for (int kk = 0; kk < K; ++kk) Raw8<T>::store(y + (size_t)__ldg(p.y_rows + tok * K + kk) * De + lc_eff, o);
    }
  };

  fetch(0);
  stash(tiles[0]);
  cur_u = pre_u; cur_z = pre_z;
  __syncthreads();

  int buf = 0;
  for (int t0 = 0; t0 < L; t0 += TS, buf ^= 1) {
    const bool more = t0 + TS < L;
    if (more) fetch(t0 + TS);
    if constexpr (MODE == 3) {
      static_assert(MODE != 3 || (TS == 16 && NC == 1), "one checkpoint per tile");
      const int c = c_base + cl;
      if (c < De) {
        float* dst = p.ckpt + (((size_t)blockIdx.y * p.nck + (size_t)((t_first + t0) >> 4)) * De + c) * NST + g * NS;
#pragma unroll
        for (int q = 0; q < NP; q += 2)
          *reinterpret_cast<float4*>(dst + 2 * q) = make_float4(h[0][q].x, h[0][q].y, h[0][q + 1].x, h[0][q + 1].y);
      }
    }
    const TileT& tl = tiles[buf];
    float* ys = ysum + buf * TS * YP;

    // Plain loop over the steps of the tile: loads, exponentials and the recurrence of one step in
    // program order, unrolled a few steps so the scheduler can overlap them.  The restrict-qualified
    // views tell the compiler that the stores of the sums never alias the tile it reads.
    const float2* __restrict__ dvp = &tl.dv[0][0];
    const float4* __restrict__ bcp = &tl.bc[0][g * NP];
    float* __restrict__ ysp = ys + cl;
    float* __restrict__ psp = ps;
    constexpr int UF = S > 4 ? S : (NC * NS >= 16 ? 2 : 4);
    float held = 0.0f;      // the even step's partial sum, kept for the paired exchange (S == 2)
    float pend_keep = 0.0f, pend_recv = 0.0f;   // the exchange of the previous pair, finished one pair later (S == 2)
    auto tile_steps = [&](auto so_tag, auto sc_tag) {
    constexpr bool STATE_ONLY = decltype(so_tag)::value;
    constexpr bool SCALAR_A = decltype(sc_tag)::value && !ZOH;
#pragma unroll UF
    for (int tt = 0; tt < TS; ++tt) {
      float4 bc[NP];
#pragma unroll
      for (int q = 0; q < NP; ++q) bc[q] = bcp[tt * (NST / 2) + q];
      float part[NC];
#pragma unroll
      for (int i = 0; i < NC; ++i) {
        const float2 dv = dvp[tt * CH + cl_sw[i]];
        const float2 dl2 = make_float2(dv.x, dv.x), vv2 = make_float2(dv.y, dv.y);
        if (STATE_ONLY) sdel[i] += dv.x;
        float2 acc0 = make_float2(0.0f, 0.0f), acc1 = make_float2(0.0f, 0.0f);
        float a_all = 0.0f;
        if (SCALAR_A) a_all = PRECISE ? expf(dl2.x * a2[i][0].x) : ex2_approx(dl2.x * a2[i][0].x);
#pragma unroll
        for (int q = 0; q < NP; ++q) {
          const float2 Bv = make_float2(bc[q].x, bc[q].y), Cv = make_float2(bc[q].z, bc[q].w);
          if (SCALAR_A) {
            h[i][q] = __ffma2_rn(make_float2(a_all, a_all), h[i][q], __fmul2_rn(vv2, Bv));      // w = (Delta u) B
            if (!STATE_ONLY) {
              float2& acc = (q & 1) ? acc1 : acc0;
              acc = q < 2 ? __fmul2_rn(Cv, h[i][q]) : __ffma2_rn(Cv, h[i][q], acc);
            }
          } else if (PRECISE) {
            const float dA0 = dl2.x * a2[i][q].x, dA1 = dl2.x * a2[i][q].y;
            // B-bar u: zero-order hold expm1(dA)/A * B * u, or (Delta u) * B
            const float w0 = ZOH ? -expm1f(dA0) * kin[i][q].x * Bv.x * vv2.x : Bv.x * vv2.x;
            const float w1 = ZOH ? -expm1f(dA1) * kin[i][q].y * Bv.y * vv2.x : Bv.y * vv2.x;
            h[i][q].x = fmaf(expf(dA0), h[i][q].x, w0);
            h[i][q].y = fmaf(expf(dA1), h[i][q].y, w1);
            if (!STATE_ONLY) {
              acc0.x = fmaf(Cv.x, h[i][q].x, acc0.x);
              acc0.y = fmaf(Cv.y, h[i][q].y, acc0.y);
            }
          } else {
            const float2 x = __fmul2_rn(dl2, a2[i][q]);
            const float2 a = make_float2(ex2_approx(x.x), ex2_approx(x.y));
            if (ZOH) {
              // zero-order hold: w = -B u / A, h <- a (h - w) + w = a h + (a - 1) B u / A
              const float2 w = __fmul2_rn(__fmul2_rn(vv2, kin[i][q]), Bv);
              const float2 sdiff = __ffma2_rn(w, make_float2(-1.0f, -1.0f), h[i][q]);
              h[i][q] = __ffma2_rn(a, sdiff, w);
            } else {
              h[i][q] = __ffma2_rn(a, h[i][q], __fmul2_rn(vv2, Bv));      // w = (Delta u) B
            }
            if (!STATE_ONLY) {
              float2& acc = (q & 1) ? acc1 : acc0;
              acc = q < 2 ? __fmul2_rn(Cv, h[i][q]) : __ffma2_rn(Cv, h[i][q], acc);
            }
          }
        }
        if (NP > 1 && (!PRECISE || SCALAR_A)) acc0 = __fadd2_rn(acc0, acc1);
        part[i] = acc0.x + acc0.y;
      }
      if (STATE_ONLY) {
        // nothing to store: only the state and the sum of Delta leave this pass
      } else if (S == 1) {
#pragma unroll
        for (int i = 0; i < NC; ++i) ysp[tt * YP + i] = part[i];
      } else if (S == 2 && NC == 1) {
        // steps are finished in pairs with one exchange: lane 0 completes the even step (it needs the partner's
        // even partial), lane 1 the odd step (it needs the partner's odd partial)
        if ((tt & 1) == 0) {
          held = part[0];
        } else {
          // the sum of the previous pair is stored only now: its shuffle has had two steps to complete
          if (tt > 1) ysp[(tt - 3 + g) * YP] = pend_keep + pend_recv;
          pend_recv = __shfl_xor_sync(0xffffffffu, g ? held : part[0], 1);
          pend_keep = g ? part[0] : held;
        }
      } else if (S <= 4) {
        // all S lanes of the channel get the sum; lane g stores the steps with tt % S == g
#pragma unroll
        for (int i = 0; i < NC; ++i) {
#pragma unroll
          for (int o = 1; o < S; o <<= 1) part[i] += __shfl_xor_sync(0xffffffffu, part[i], o);
        }
        if ((tt % S) == g) {
#pragma unroll
          for (int i = 0; i < NC; ++i) ysp[tt * YP + i] = part[i];
        }
      } else {
        psp[(tt % S) * G::SLOT + lane] = part[0];
        if ((tt % S) == S - 1) {
          __syncwarp();
          // lane g of the channel adds up the S partial sums of time step tt - (S-1) + g
          const float* src = psp + g * G::SLOT + (lane / S) * S;
          float sum = 0.0f;
#pragma unroll
          for (int j = 0; j < S; j += 4) {
            const float4 v4 = *reinterpret_cast<const float4*>(src + j);
            sum += (v4.x + v4.y) + (v4.z + v4.w);
          }
          ysp[(tt - (S - 1) + g) * YP] = sum;
          __syncwarp();
        }
      }
    }

    };
    if (MODE == 1 || MODE == 3) {
      tile_steps(std::true_type{}, std::false_type{});
    } else if (p.scalar_a) {
      if (MODE == 2 && so) tile_steps(std::true_type{}, std::true_type{});
      else tile_steps(std::false_type{}, std::true_type{});
    } else {
      if (MODE == 2 && so) tile_steps(std::true_type{}, std::false_type{});
      else tile_steps(std::false_type{}, std::false_type{});
    }

    if (S == 2 && NC == 1 && !so) ysp[(TS - 2 + g) * YP] = pend_keep + pend_recv;      // the tile's last pair
    if (more) stash(tiles[buf ^ 1]);
    __syncthreads();
    if (!so) {
      flush(t0, ys);
      if (more) { cur_u = pre_u; cur_z = pre_z; }
    }
  }

  if (p.h_last) {
#pragma unroll
    for (int i = 0; i < NC; ++i) {
      const int c = c_base + cl + i;
      if (c >= De) continue;
#pragma unroll
      for (int q = 0; q < NP; ++q) {
        const int n = g * NS + 2 * q;
        p.h_last[((size_t)b * De + c) * NST + n] = h[i][q].x;
        p.h_last[((size_t)b * De + c) * NST + n + 1] = h[i][q].y;
      }
      if (so && g == 0 && p.sum_delta) p.sum_delta[(size_t)b * De + c] = sdel[i];
    }
  }
}

// One step per sequence (L == 1, recurrent inference): a thread owns all 16 states of one channel of one
// sequence; the state is read and written once (64 contiguous bytes per thread), B and C of the sequence are the
// same for every thread of the block.  Same arithmetic as scan_kernel (per PRECISE / ZOH).
template <typename T, typename TD, bool PRECISE, bool ZOH>
__global__ void __launch_bounds__(BLOCK)
scan_step_kernel(const ScanArgs p) {
  const int c = blockIdx.x * BLOCK + threadIdx.x;
  const size_t b = blockIdx.y;
  if (c >= p.De) return;
  const T* __restrict__ u = static_cast<const T*>(p.u);
  const float dl = to_f32(static_cast<const TD*>(p.delta)[b * p.De + c]);
  const float uu = to_f32(u[b * p.De + c]);
  const float4* Bq = reinterpret_cast<const float4*>(p.Bm + b * NST);
  const float4* Cq = reinterpret_cast<const float4*>(p.Cm + b * NST);
  const float4* Aq = reinterpret_cast<const float4*>(p.A + (size_t)c * NST);
  const float4* Hq = p.h0 ? reinterpret_cast<const float4*>(p.h0 + (b * p.De + c) * NST) : nullptr;
  float4* Ho = p.h_last ? reinterpret_cast<float4*>(p.h_last + (b * p.De + c) * NST) : nullptr;
  float y = 0.0f;
#pragma unroll
  for (int q = 0; q < NST / 4; ++q) {
    const float4 a4 = __ldg(Aq + q), b4 = __ldg(Bq + q), c4 = __ldg(Cq + q);
    const float4 h4 = Hq ? Hq[q] : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
    const float av[4] = {a4.x, a4.y, a4.z, a4.w}, bv[4] = {b4.x, b4.y, b4.z, b4.w}, cv[4] = {c4.x, c4.y, c4.z, c4.w};
    float hv[4] = {h4.x, h4.y, h4.z, h4.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      if (PRECISE) {
        const float dA = dl * av[i];
        const float w = ZOH ? -expm1f(dA) * (-1.0f / av[i]) * bv[i] * uu : bv[i] * (dl * uu);
        hv[i] = fmaf(expf(dA), hv[i], w);
      } else {
        const float a = ex2_approx(dl * (av[i] * kLog2e));
        if (ZOH) {
          const float w = (uu * (-1.0f / av[i])) * bv[i];
          hv[i] = fmaf(a, hv[i] - w, w);
        } else {
          hv[i] = fmaf(a, hv[i], (dl * uu) * bv[i]);
        }
      }
      y = fmaf(cv[i], hv[i], y);
    }
    if (Ho) Ho[q] = make_float4(hv[0], hv[1], hv[2], hv[3]);
  }
  if (p.D) y = fmaf(p.D[c], uu, y);
  if (p.z) {
    const T* __restrict__ z = static_cast<const T*>(p.z);
    const size_t zrow = p.z_row ? (size_t)__ldg(p.z_row + b) : b;
    const float zz = to_f32(z[zrow * p.ldz + c]);
    y *= p.gate_activated ? zz : (PRECISE ? zz / (1.0f + expf(-zz)) : silu_fast(zz));
  }
  T* __restrict__ yo = static_cast<T*>(p.y);
  if (p.y_rows == nullptr) {
    yo[b * p.De + c] = from_f32<T>(y);
  } else {
    for (int kk = 0; kk < p.K; ++kk) yo[(size_t)__ldg(p.y_rows + b * p.K + kk) * p.De + c] = from_f32<T>(y);
  }
}

// Initial state of every chunk after the first.  h_end[0] is the true state after chunk 0 (it ran from the
// caller's h0); for j >= 1, h_end[j] is chunk j's end state from a zero start.  In chunk order, per
// (sequence, channel, state):  h = h_end[0];  h_in[j] = h;  h = exp(A * sum_delta[j]) * h + h_end[j].
__global__ void __launch_bounds__(256)
chain_chunk_states(const float* __restrict__ A, const float* __restrict__ h_end, const float* __restrict__ sum_delta,
                   float* __restrict__ h_in, float* __restrict__ h_last, int B, int De, int nch, int n_end) {
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= (long long)B * De * NST) return;
  const int n = (int)(i % NST);
  const int c = (int)((i / NST) % De);
  const int b = (int)(i / ((long long)NST * De));
  const float a = A[(size_t)c * NST + n];
  float h = h_end[(((size_t)b * nch) * De + c) * NST + n];
  for (int j = 1; j < nch; ++j) {
    const size_t sq = (size_t)b * nch + j;
    h_in[(sq * De + c) * NST + n] = h;
    if (j < n_end) h = fmaf(expf(a * sum_delta[sq * De + c]), h, h_end[(sq * De + c) * NST + n]);
  }
  if (h_last) h_last[i] = h;
}

template <typename T, typename TD, int NC, int NS, bool PRECISE, bool ZOH, int MODE>
cudaError_t launch_one(const ScanArgs& a, int B, int grid_z, cudaStream_t st) {
  using G = Geo<NC, NS>;
  const size_t smem = 2 * sizeof(Tile<NC, NS>) + (2 * (size_t)G::TS * G::YP + (BLOCK / 32) * G::STRIP) * sizeof(float);
  cudaError_t e = cudaFuncSetAttribute(scan_kernel<T, TD, NC, NS, PRECISE, ZOH, MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid((a.De + G::CH - 1) / G::CH, B, grid_z);
  scan_kernel<T, TD, NC, NS, PRECISE, ZOH, MODE><<<grid, BLOCK, smem, st>>>(a);
  count_launch();
  return cudaGetLastError();
}

// Work per thread, NC channels x NS states, as NC * 100 + NS: the largest of 1x8, 1x4, 1x2 that still
// gives every SM sub-partition about two warps.
constexpr double kFirstChunkRatio = 0.7;

int pick_thread_shape(int B, int De, int num_sms) {
  const long long want_warps = 2LL * 4 * num_sms;
  const int shapes[2][2] = {{1, 8}, {1, 4}};
  for (const auto& sh : shapes) {
    const int ch = BLOCK / (NST / sh[1]) * sh[0];
    const long long warps = (long long)B * ((De + ch - 1) / ch) * (BLOCK / 32);
    if (warps >= want_warps) return sh[0] * 100 + sh[1];
  }
  return 102;
}

template <typename T, typename TD, bool PRECISE, bool ZOH>
cudaError_t launch_shape(int shape, const ScanArgs& a, int B, cudaStream_t st) {
  switch (shape) {
    case 108: return launch_one<T, TD, 1, 8, PRECISE, ZOH, 0>(a, B, a.nch, st);
    case 104: return launch_one<T, TD, 1, 4, PRECISE, ZOH, 0>(a, B, a.nch, st);
    case 102: return launch_one<T, TD, 1, 2, PRECISE, ZOH, 0>(a, B, a.nch, st);
    default: return cudaErrorInvalidValue;
  }
}

template <typename T, typename TD, bool PRECISE>
cudaError_t launch_scan_t(const rom_config& c, ScanArgs a, const float* A, const float* h0, float* h_last,
                          float* chunk_ws, int num_sms, cudaStream_t st) {
  const bool zoh = c.disc_mode == 0;
  if (c.L == 1) {
    a.h0 = h0; a.h_last = h_last;
    dim3 grid((c.d_inner + BLOCK - 1) / BLOCK, c.B);
    if (zoh) scan_step_kernel<T, TD, PRECISE, true><<<grid, BLOCK, 0, st>>>(a);
    else scan_step_kernel<T, TD, PRECISE, false><<<grid, BLOCK, 0, st>>>(a);
    count_launch();
    return cudaGetLastError();
  }
  const int nch = chunk_ws ? scan_chunks(c.B, c.d_inner, c.L) : 1;
  if (nch == 1) {
    a.Lc = c.L; a.L0 = c.L; a.nch = 1;
    const int shape = pick_thread_shape(c.B, c.d_inner, num_sms);
    return zoh ? launch_shape<T, TD, PRECISE, true>(shape, a, c.B, st) : launch_shape<T, TD, PRECISE, false>(shape, a, c.B, st);
  }
  // chunked, two launches, 8 states per thread.  Launch A: chunk 0 in full from the caller's state, chunks
  // 1..n_end-1 state-only from zero; chain; launch B: chunks 1..nch-1 in full from their true initial states.
  const size_t n_state = (size_t)c.B * nch * c.d_inner * NST;
  float* h_end = chunk_ws;
  float* h_in = chunk_ws + n_state;
  float* sum_delta = chunk_ws + 2 * n_state;
  // Chunk 0 runs in full inside the first launch, next to state-only chunks that cost less per step: it is made
  // shorter by kFirstChunkRatio so that its blocks do not outlast the others.
  const double x = (double)c.L / ((double)(nch - 1) + kFirstChunkRatio);
  a.Lc = (int)align_up((size_t)ceil(x), 64);
  a.L0 = (int)align_up((size_t)ceil(kFirstChunkRatio * x), 64);
  a.nch = nch;
  const int n_end = h_last ? nch : nch - 1;       // the last chunk's end state is only needed for h_last
  ScanArgs pa = a;
  pa.h_last = h_end; pa.sum_delta = sum_delta; pa.chunk_off = 0;
  cudaError_t e = zoh ? launch_one<T, TD, 1, 8, PRECISE, true, 2>(pa, c.B, n_end, st) : launch_one<T, TD, 1, 8, PRECISE, false, 2>(pa, c.B, n_end, st);
  if (e != cudaSuccess) return e;
  const long long n_thr = (long long)c.B * c.d_inner * NST;
  chain_chunk_states<<<(unsigned)((n_thr + 255) / 256), 256, 0, st>>>(A, h_end, sum_delta, h_in, h_last, c.B, c.d_inner, nch, n_end);
  count_launch();
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  a.h0 = h_in; a.h_last = nullptr; a.chunk_off = 1;
  return zoh ? launch_one<T, TD, 1, 8, PRECISE, true, 0>(a, c.B, nch - 1, st) : launch_one<T, TD, 1, 8, PRECISE, false, 0>(a, c.B, nch - 1, st);
}

}  // namespace

cudaError_t launch_scan(const rom_config& c, const void* u, const void* delta, bool delta_fp32, const float* A, const float* Bm,
                        const float* Cm, const float* D, const void* z, int ldz, const int32_t* z_row, const float* h0,
                        void* y, float* h_last, const int32_t* y_rows, int K, float* chunk_ws, bool gate_activated, cudaStream_t st,
                        bool scalar_A) {
  int num_sms = 0;
  const cudaError_t e = current_device_sm_count(&num_sms);
  if (e != cudaSuccess) return e;
  // Few long sequences and no workspace for the chunked scan: the one-pass low-occupancy kernel (every exponential once;
  // 0.74 ms against 1.04 ms for one 16384-step sequence of 4096 channels).  With a workspace the two chunked launches
  // below are faster (0.67 ms), so they stay the path of the layer.
  if (chunk_ws == nullptr && !scalar_A && scan_seq_applicable(c, u, delta, delta_fp32, Bm, Cm, z, ldz, z_row, y_rows, gate_activated, num_sms))
    return launch_scan_seq(c, u, delta, delta_fp32, A, Bm, Cm, D, z, ldz, h0, y, h_last, y_rows, K, gate_activated, st);
  const ScanArgs a{u, delta, A, Bm, Cm, D, z, ldz, z_row, h0, y, h_last, y_rows, K, c.L, c.d_inner, c.L, 1, c.L, nullptr, gate_activated ? 1 : 0, 0, nullptr, 0, (scalar_A && c.disc_mode == 1) ? 1 : 0};
  if (c.dtype != ROM_BF16) return launch_scan_t<float, float, true>(c, a, A, h0, h_last, chunk_ws, num_sms, st);
  return delta_fp32 ? launch_scan_t<__nv_bfloat16, float, false>(c, a, A, h0, h_last, chunk_ws, num_sms, st)
                    : launch_scan_t<__nv_bfloat16, __nv_bfloat16, false>(c, a, A, h0, h_last, chunk_ws, num_sms, st);
}

// State recurrence alone over uniform chunks of Lc steps (Lc a multiple of 16; ncc chunks per sequence), for the backward pass.
// ckpt == nullptr: every chunk from a zero state; h_end [B, ncc, De, 16] and sum_delta [B, ncc, De] leave.
// ckpt != nullptr: every chunk from its true start state h_in [B, ncc, De, 16] (null: zero); the state at the start of every
// 16 steps is stored to ckpt [B, nck, De, 16].
cudaError_t launch_scan_states(const rom_config& c, const void* u, const float* delta, const float* A, const float* Bm, int Lc, int ncc,
                               const float* h_in, float* h_end, float* sum_delta, float* ckpt, int nck, cudaStream_t st) {
  ScanArgs a{u, delta, A, Bm, /* C is fetched with B but not used */ Bm, nullptr, nullptr, 0, nullptr, h_in, nullptr, h_end, nullptr, 1, c.L, c.d_inner, Lc, ncc, Lc, sum_delta,
             0, 0, ckpt, nck, 0};
  const bool zoh = c.disc_mode == 0;
  if (ckpt == nullptr) {
    a.h0 = nullptr;
    if (c.dtype != ROM_BF16) return zoh ? launch_one<float, float, 1, 8, true, true, 1>(a, c.B, ncc, st) : launch_one<float, float, 1, 8, true, false, 1>(a, c.B, ncc, st);
    return zoh ? launch_one<__nv_bfloat16, float, 1, 8, false, true, 1>(a, c.B, ncc, st) : launch_one<__nv_bfloat16, float, 1, 8, false, false, 1>(a, c.B, ncc, st);
  }
  a.h_last = nullptr;
  if (c.dtype != ROM_BF16) return zoh ? launch_one<float, float, 1, 8, true, true, 3>(a, c.B, ncc, st) : launch_one<float, float, 1, 8, true, false, 3>(a, c.B, ncc, st);
  return zoh ? launch_one<__nv_bfloat16, float, 1, 8, false, true, 3>(a, c.B, ncc, st) : launch_one<__nv_bfloat16, float, 1, 8, false, false, 3>(a, c.B, ncc, st);
}

}  // namespace rom
