// Fused short conv + x Proj + dt Proj + softplus (Section 3.1: U = SiLU(DWConv(H)); Section 4.3: the x Proj / dt Proj
// layers shared by all experts), one kernel on the bf16 tensor path at top-1, where H is already in token order:
//   U = SiLU(conv(H) + b_conv),  (delta | B | C) = U W_x^T,  Delta = softplus(delta W_dt^T + b_dt).
// U is written to HBM once and never read back by these steps, delta never leaves the SM.
//
// One CTA owns a tile of up to 128 tokens (the token count is spread evenly over the SMs) and all D_e channels.  576 threads: a TMA producer warp, an MMA-issuing warp
// (tcgen05, accumulators in tensor memory) and 16 worker warps that change role with the phase:
//   phase 1  per block of 64 channels the producer brings the 131 x 64 block of H (the tile's rows and the three
//            before them) and the matching 64 columns of W_x by TMA, three blocks ahead; the workers compute conv +
//            SiLU from shared memory (8 channels of two consecutive tokens per thread), write it to U and, as bf16 in the
//            128-byte-swizzled K-major layout the tensor core expects, into an operand stage; the MMA thread
//            accumulates the 128 x (d_r + 2 D_s) x Proj tile over all channel blocks.
//   phase 2  workers read that tile from tensor memory: B, C go to HBM in fp32, delta is rounded to bf16 and laid
//            out in shared memory as the A operand of the dt Proj.
//   phase 3  for every block of 256 channels the producer brings the W_dt rows, the MMA thread forms
//            delta W_dt^T (double-buffered accumulators) and the workers apply bias + softplus and write Delta as
//            whole 128-byte row segments (the output op of the stand-alone dt Proj GEMM).
// Shared-memory writes by the workers are made visible to the tensor core with fence.proxy.async before the
// mbarrier arrive.  Every wait is bounded; on expiry the CTA latches an error in the status word, waits (bounded)
// for its copies and MMAs in flight, frees its tensor memory and returns.  Plain single-CTA TMA loads only.
#include "rom_tc_ptx.cuh"

namespace rom {
namespace {

constexpr int FW = 16;                          // worker warps
constexpr int F_THREADS = 64 + 32 * FW;         // 576
constexpr int F_STAGES = 3;
constexpr int FA_BYTES = BLOCK_M * BLOCK_K * 2; // 16 KB: one 128 x 64 bf16 operand block
constexpr int F_MAX_N1 = 160;                   // widest x Proj tile (d_r + 2 D_s) this kernel takes
constexpr int FB1_BYTES = F_MAX_N1 * BLOCK_K * 2;   // 20 KB
constexpr int FB3_BYTES = 256 * BLOCK_K * 2;        // 32 KB: 256 rows of W_dt, one K block
constexpr int F_HALO = 3;                       // rows before the tile that the conv reads (d_conv <= 4)
constexpr int FH_ROWS = BLOCK_M + F_HALO;       // 131 rows of H per block
constexpr int FH_BYTES = 17 * 1024;             // 131 x 128 bytes, rounded up to the 1024-byte alignment of swizzled tiles
constexpr int F_STAGE1 = FA_BYTES + FB1_BYTES + FH_BYTES;            // 53 KB per phase 1 stage
constexpr int F_OUT_BYTES = FW * 32 * 32 * 4;   // 64 KB: staging of the softplus output op (phase 3 only)
constexpr int F_STAGE_REGION = F_STAGES * F_STAGE1 > F_STAGES * FB3_BYTES + F_OUT_BYTES ? F_STAGES * F_STAGE1 : F_STAGES * FB3_BYTES + F_OUT_BYTES;
                                                // 160 KB: phase 1 stages; phase 3 reuses it for its 3 x 32 KB stages + the output staging
constexpr int F_A2_BYTES = 2 * FA_BYTES;        // delta as the dt Proj's A operand: up to two K blocks (d_r <= 128)
constexpr int F_NUM_BARS = 3 * F_STAGES + 2 + 2 * F_STAGES + 4 + 1;
constexpr int F_SMEM = 1024 + F_STAGE_REGION + F_A2_BYTES + 256;
static_assert(F_STAGE1 % 1024 == 0 && FH_ROWS * 128 <= FH_BYTES, "stage layout");
static_assert(8 * F_NUM_BARS + 16 <= 256, "barrier block");

struct FusedArgs {
  const __nv_bfloat16* HZ;      // [T, ldh]: conv input in token order (the Conv Proj half of the in_proj output)
  int ldh;
  const __nv_bfloat16* w_conv;  // [k, De]
  const float* b_conv;          // [De] or null
  const float* b_dt;            // [De] or null
  __nv_bfloat16* U;             // [T, De]
  __nv_bfloat16* delta_r;       // [T, R]
  float* Bm; float* Cm;         // [T, N]
  __nv_bfloat16* Delta;         // [T, De]
  int T, L, De, R, N, k;
  int block_n1;                 // x Proj tile width: R + 2N rounded up to 32
  int block_n3;                 // dt Proj tile width: min(256, De rounded up to 32)
  int rows_cta;                 // tokens per CTA (<= 128, a multiple of 8): chosen so that every SM gets the same share
};

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void unpack8(const uint4& q, float (&v)[8]) {
  const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) { v[2 * i] = __uint_as_float(w[i] << 16); v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u); }
}
__device__ __forceinline__ uint4 pack8(const float (&v)[8]) {
  uint4 q;
  uint32_t* w = reinterpret_cast<uint32_t*>(&q);
#pragma unroll
  for (int i = 0; i < 4; ++i) { const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]); w[i] = *reinterpret_cast<const uint32_t*>(&h); }
  return q;
}

template <int KCONV>
__global__ void __launch_bounds__(F_THREADS, 1)
fused_conv_xdt_kernel(const __grid_constant__ CUtensorMap tmap_h, const __grid_constant__ CUtensorMap tmap_wx,
                      const __grid_constant__ CUtensorMap tmap_wdt, const FusedArgs p, uint32_t idesc1, uint32_t idesc3, int32_t* __restrict__ status, uint32_t wait_limit) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;               // 128B-swizzled tiles need 1024-byte alignment
  unsigned char* smem = smem_raw + (base - raw);
  // [stage region][delta operand][output staging][barriers]
  const uint32_t a2_base = base + F_STAGE_REGION;
  unsigned char* a2_ptr = smem + F_STAGE_REGION;
  float* out_stage = reinterpret_cast<float*>(smem + F_STAGES * FB3_BYTES);      // inside the stage region, behind the phase 3 stages
  const uint32_t bars = base + F_STAGE_REGION + F_A2_BYTES;
  auto fullA = [&](int s) { return bars + 8u * s; };
  auto fullB = [&](int s) { return bars + 8u * (F_STAGES + s); };
  auto empty1 = [&](int s) { return bars + 8u * (2 * F_STAGES + s); };
  constexpr int BB = 3 * F_STAGES;
  const uint32_t d1_full = bars + 8u * BB;
  const uint32_t a2_ready = bars + 8u * (BB + 1);
  auto full3 = [&](int s) { return bars + 8u * (BB + 2 + s); };
  auto empty3 = [&](int s) { return bars + 8u * (BB + 2 + F_STAGES + s); };
  auto tfull = [&](int a) { return bars + 8u * (BB + 2 + 2 * F_STAGES + a); };
  auto tempty = [&](int a) { return bars + 8u * (BB + 4 + 2 * F_STAGES + a); };
  const uint32_t drain_bar = bars + 8u * (BB + 6 + 2 * F_STAGES);
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + F_STAGE_REGION + F_A2_BYTES + 8 * F_NUM_BARS);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m0 = blockIdx.x * p.rows_cta;
  const int nkc = p.De / BLOCK_K;                              // channel blocks of the x Proj contraction
  const int kb3 = (p.R + BLOCK_K - 1) / BLOCK_K;               // K blocks of the dt Proj
  const int nt3 = (p.De + p.block_n3 - 1) / p.block_n3;        // channel tiles of the dt Proj
  const int N1 = p.R + 2 * p.N;

  if (threadIdx.x == 0) {
    for (int s = 0; s < F_STAGES; ++s) {
      mbar_init(fullA(s), FW); mbar_init(fullB(s), 1); mbar_init(empty1(s), 1);
      mbar_init(full3(s), 1); mbar_init(empty3(s), 1);
    }
    mbar_init(d1_full, 1); mbar_init(a2_ready, FW); mbar_init(drain_bar, 1);
    for (int a = 0; a < 2; ++a) { mbar_init(tfull(a), 1); mbar_init(tempty(a), FW); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (warp >= 2) {     // the delta operand starts as zeros: columns at or beyond d_r of its last K block stay zero
    uint4* z = reinterpret_cast<uint4*>(a2_ptr);
    for (int i = threadIdx.x - 64; i < F_A2_BYTES / 16; i += 32 * FW) z[i] = make_uint4(0, 0, 0, 0);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer: H and W_x blocks, then W_dt blocks
    if (lane == 0) {
      uint32_t last_bar[F_STAGES] = {}, last_par[F_STAGES] = {};
      int n_last = 0;
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int kc = 0; kc < nkc && ok; ++kc) {
        if (!mbar_wait(empty1(stage), phase ^ 1u, abort_flag, wait_limit)) { ok = false; break; }
        mbar_expect_tx(fullB(stage), (uint32_t)(p.block_n1 + FH_ROWS) * BLOCK_K * 2);
        const uint32_t ss = base + stage * F_STAGE1;
        tma_load_2d(ss + FA_BYTES + FB1_BYTES, &tmap_h, fullB(stage), kc * BLOCK_K, m0 - F_HALO);   // rows before token 0 and past the end read as zeros
        tma_load_2d(ss + FA_BYTES, &tmap_wx, fullB(stage), kc * BLOCK_K, 0);
        last_bar[n_last % F_STAGES] = fullB(stage); last_par[n_last % F_STAGES] = phase; ++n_last;
        if (++stage == F_STAGES) { stage = 0; phase ^= 1u; }
      }
      // the dt Proj stages reuse the phase 1 region: wait until the last x Proj MMA has read it (the workers are done with H by then)
      if (ok && !mbar_wait(d1_full, 0, abort_flag, wait_limit)) ok = false;
      stage = 0; phase = 0;
      for (int nt = 0; nt < nt3 && ok; ++nt) {
        for (int kb = 0; kb < kb3; ++kb) {
          if (!mbar_wait(empty3(stage), phase ^ 1u, abort_flag, wait_limit)) { ok = false; break; }
          mbar_expect_tx(full3(stage), (uint32_t)p.block_n3 * BLOCK_K * 2);
          tma_load_2d(base + stage * FB3_BYTES, &tmap_wdt, full3(stage), kb * BLOCK_K, nt * p.block_n3);
          last_bar[n_last % F_STAGES] = full3(stage); last_par[n_last % F_STAGES] = phase; ++n_last;
          if (++stage == F_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        if (!*abort_flag) { atomicExch(status + kStatCode, ROM_ERR_DEVICE_TIMEOUT); atomicExch(status + kStatWhere, 21); }
        *abort_flag = 1;
      }
      if (*abort_flag) {      // give this CTA's copies still in flight a bounded time to land before the CTA exits
        for (int i = 0; i < (n_last < F_STAGES ? n_last : F_STAGES); ++i)
          for (uint32_t it = 0; it < (wait_limit >> 2); ++it)
            if (mbar_try_wait(last_bar[i], last_par[i])) break;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      bool ok = true, issued_any = false;
      int stage = 0; uint32_t phase = 0;
      for (int kc = 0; kc < nkc && ok; ++kc) {
        if (!mbar_wait(fullA(stage), phase, abort_flag, wait_limit) || !mbar_wait(fullB(stage), phase, abort_flag, wait_limit)) { ok = false; break; }
        tc_fence_after();
        const uint32_t sa = base + stage * F_STAGE1;
        const uint64_t adesc = make_smem_desc(sa), bdesc = make_smem_desc(sa + FA_BYTES);
#pragma unroll
        for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
          umma_bf16(tmem_base, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc1, (kc | k) != 0 ? 1u : 0u);
        umma_commit(empty1(stage));
        issued_any = true;
        if (++stage == F_STAGES) { stage = 0; phase ^= 1u; }
      }
      if (ok) umma_commit(d1_full);
      // dt Proj: A = delta (written by the workers), B = W_dt blocks
      if (ok && !mbar_wait(a2_ready, 0, abort_flag, wait_limit)) ok = false;
      tc_fence_after();
      stage = 0; phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      for (int nt = 0; nt < nt3 && ok; ++nt) {
        if (!mbar_wait(tempty(acc), acc_phase ^ 1u, abort_flag, wait_limit)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)acc * 256u;
        for (int kb = 0; kb < kb3; ++kb) {
          if (!mbar_wait(full3(stage), phase, abort_flag, wait_limit)) { ok = false; break; }
          tc_fence_after();
          const uint64_t adesc = make_smem_desc(a2_base + kb * FA_BYTES), bdesc = make_smem_desc(base + stage * FB3_BYTES);
#pragma unroll
          for (int k = 0; k < BLOCK_K / UMMA_K; ++k)
            umma_bf16(tmem_d, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc3, (kb | k) != 0 ? 1u : 0u);
          umma_commit(empty3(stage));
          if (++stage == F_STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(tfull(acc));
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
      if (!ok) {
        if (!*abort_flag) { atomicExch(status + kStatCode, ROM_ERR_DEVICE_TIMEOUT); atomicExch(status + kStatWhere, 22); }
        *abort_flag = 1;
      }
      if (*abort_flag && issued_any) {     // MMAs already issued may still read shared memory and write tensor memory
        umma_commit(drain_bar);
        for (uint32_t it = 0; it < (wait_limit >> 2); ++it)
          if (mbar_try_wait(drain_bar, 0)) break;
      }
    }
  } else {
    // ------------------------------------------------------------------ workers (warps 2..17)
    const int w = warp - 2;
    const int wt = w * 32 + lane;                 // 0..511
    bool ok = true;

    // ---- phase 1: conv + SiLU of the tile, one 64-channel block after the other.  A thread owns 8 channels of two
    // consecutive tokens: the five rows of H it needs are unpacked once and serve both tokens.
    {
      const int cg = wt & 7, r0 = (wt >> 3) * 2;  // 16-byte channel group of the block; first of the thread's two rows
      bool valid[2];
      int tpos[2];
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int tok = m0 + r0 + i;
        valid[i] = r0 + i < p.rows_cta && tok < p.T;
        tpos[i] = valid[i] ? tok % p.L : 0;       // position inside its sequence (the conv does not cross sequences)
      }
      __nv_bfloat16* urow = p.U + (size_t)(m0 + r0) * p.De + 8 * cg;
      int stage = 0; uint32_t phase = 0;
      for (int kc = 0; kc < nkc; ++kc) {
        const int c0 = kc * BLOCK_K + 8 * cg;     // first channel of this thread in the layer
        // taps and bias of these 8 channels (L1-resident), requested before the wait for the H block
        float wv[KCONV][8];
#pragma unroll
        for (int j = 0; j < KCONV; ++j) unpack8(__ldg(reinterpret_cast<const uint4*>(p.w_conv + (size_t)j * p.De + c0)), wv[j]);
        float acc[2][8];
        if (p.b_conv) {
          const float4 b0 = __ldg(reinterpret_cast<const float4*>(p.b_conv + c0)), b1 = __ldg(reinterpret_cast<const float4*>(p.b_conv + c0) + 1);
          const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
          for (int i = 0; i < 8; ++i) { acc[0][i] = bb[i]; acc[1][i] = bb[i]; }
        } else {
#pragma unroll
          for (int i = 0; i < 8; ++i) { acc[0][i] = 0.0f; acc[1][i] = 0.0f; }
        }
        // the H block of this stage has landed (the producer reused the stage only after its MMAs were done)
        if (!__all_sync(0xffffffffu, mbar_wait(fullB(stage), phase, abort_flag, wait_limit))) { ok = false; break; }
        unsigned char* sa = smem + stage * F_STAGE1;
        const unsigned char* hs = sa + FA_BYTES + FB1_BYTES;      // row i of the block = token m0 - 3 + i
        // block rows r0 + i, i = 0..4, are tokens r0 - 3 + i: row i is tap i + KCONV - 4 of token r0 and tap i + KCONV - 5 of token r0 + 1
#pragma unroll
        for (int i = 0; i < 5; ++i) {
          constexpr int K4 = KCONV - 4, K5 = KCONV - 5;
          if (i + K4 < 0 && i + K5 < 0) continue;
          const int hr = r0 + i;
          float hv[8];
          unpack8(*reinterpret_cast<const uint4*>(hs + hr * 128 + ((cg ^ (hr & 7)) << 4)), hv);
          if (i + K4 >= 0 && i + K4 < KCONV && valid[0] && tpos[0] - (3 - i) >= 0) {
#pragma unroll
            for (int c = 0; c < 8; ++c) acc[0][c] = fmaf(wv[(i + K4) < 0 ? 0 : (i + K4) >= KCONV ? 0 : (i + K4)][c], hv[c], acc[0][c]);
          }
          if (i + K5 >= 0 && i + K5 < KCONV && valid[1] && tpos[1] - (4 - i) >= 0) {
#pragma unroll
            for (int c = 0; c < 8; ++c) acc[1][c] = fmaf(wv[(i + K5) < 0 ? 0 : (i + K5) >= KCONV ? 0 : (i + K5)][c], hv[c], acc[1][c]);
          }
        }
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          float o[8];
#pragma unroll
          for (int c = 0; c < 8; ++c) o[c] = valid[i] ? silu_fast(acc[i][c]) : 0.0f;
          const uint4 q = pack8(o);
          if (valid[i]) *reinterpret_cast<uint4*>(urow + (size_t)i * p.De + (size_t)kc * BLOCK_K) = q;
          const int r = r0 + i;
          *reinterpret_cast<uint4*>(sa + r * 128 + ((cg ^ (r & 7)) << 4)) = q;
        }
        fence_async_smem();                      // generic-proxy writes -> visible to the tensor core's reads
        __syncwarp();
        if (lane == 0) mbar_arrive(fullA(stage));
        if (++stage == F_STAGES) { stage = 0; phase ^= 1u; }
      }
    }

    // ---- phase 2: the x Proj tile leaves tensor memory: delta -> dt Proj operand (+ HBM), B and C -> HBM
    const int quarter = warp & 3;                // tensor-memory lanes [32 quarter, 32 quarter + 32) belong to this warp
    const int part = w >> 2;                     // 0..3: which of the four warps of the quarter
    if (ok && !__all_sync(0xffffffffu, mbar_wait(d1_full, 0, abort_flag, wait_limit))) ok = false;
    if (ok) {
      tc_fence_after();
      const int row = quarter * 32 + lane;
      const int tok = m0 + row;
      const bool valid = row < p.rows_cta && tok < p.T;
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16);
      for (int ch = part; ch * 32 < p.block_n1; ch += 4) {
        uint32_t ra[32];
        tmem_ld32_issue(taddr + ch * 32, ra);
        tmem_ld_wait(ra);
#pragma unroll
        for (int j = 0; j < 32; j += 8) {
          const int n = ch * 32 + j;
          if (n >= N1) break;
          float v[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(ra[j + i]);
          if (n < p.R) {
            const uint4 q = pack8(v);
            const int kb = n >> 6, c16 = (n & 63) >> 3;
            *reinterpret_cast<uint4*>(a2_ptr + kb * FA_BYTES + row * 128 + ((c16 ^ (row & 7)) << 4)) = valid ? q : make_uint4(0, 0, 0, 0);
            if (valid) *reinterpret_cast<uint4*>(p.delta_r + (size_t)tok * p.R + n) = q;
          } else if (valid) {
            float* dst = (n < p.R + p.N) ? p.Bm + (size_t)tok * p.N + (n - p.R) : p.Cm + (size_t)tok * p.N + (n - p.R - p.N);
            *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
            *reinterpret_cast<float4*>(dst + 4) = make_float4(v[4], v[5], v[6], v[7]);
          }
        }
      }
      fence_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(a2_ready);
    }

    // ---- phase 3: bias + softplus on the dt Proj tiles, rows written as whole 128-byte segments
    if (ok) {
      const Epilogue ep{EPI_SOFTPLUS, p.Delta, p.De, nullptr, nullptr, p.b_dt, 0, 0, nullptr, nullptr};
      uint4* stage_out = reinterpret_cast<uint4*>(out_stage + w * 1024);
      const int n_chunks3 = p.block_n3 >> 5;
      const int c0 = 2 * part;                   // this warp's 32-column chunks of the tile: c0 and c0 + 1
      int acc = 0; uint32_t acc_phase = 0;
      for (int nt = 0; nt < nt3; ++nt) {
        if (!__all_sync(0xffffffffu, mbar_wait(tfull(acc), acc_phase, abort_flag, wait_limit))) { ok = false; break; }
        tc_fence_after();
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)acc * 256u;
        const int n_base = nt * p.block_n3;
        int n_pieces = 0;
        for (int cc = 0; cc < 2 && c0 + cc < n_chunks3; ++cc) {
          uint32_t ra[32];
          float4 bq[8];
          tmem_ld32_issue(taddr + (c0 + cc) * 32, ra);
          const int nb = n_base + (c0 + cc) * 32;
#pragma unroll
          for (int i = 0; i < 8; ++i)
            bq[i] = (p.b_dt && nb + 4 * i < p.De) ? __ldg(reinterpret_cast<const float4*>(p.b_dt + nb) + i) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
          tmem_ld_wait(ra);
          softplus_stage_bf16(stage_out, 4 * cc, ra, bq, lane);
          n_pieces += 4;
        }
        if (n_pieces > 0) {
          __syncwarp();
          softplus_flush_bf16<EPI_SOFTPLUS>(ep, stage_out, m0 + quarter * 32, min(p.T, m0 + p.rows_cta), n_base + c0 * 32, p.De, n_pieces, lane);
          __syncwarp();
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tempty(acc));
        if (++acc == 2) { acc = 0; acc_phase ^= 1u; }
      }
    }
    if (!ok && lane == 0) {
      if (!*abort_flag) { atomicExch(status + kStatCode, ROM_ERR_DEVICE_TIMEOUT); atomicExch(status + kStatWhere, 23); }
      *abort_flag = 1;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

}  // namespace

bool fused_conv_xdt_supported(const rom_config& c) {
  return c.dtype == ROM_BF16 && c.d_state == 16 && c.dt_rank % 16 == 0 && c.dt_rank <= 128 && c.dt_rank + 2 * c.d_state <= F_MAX_N1 &&
         c.d_inner % 64 == 0 && c.d_conv >= 2 && c.d_conv <= 4 && c.L > 1;
}

cudaError_t launch_fused_conv_xdt(const rom_config& c, const void* HZ, int ldh, const void* w_conv, const float* b_conv, const void* W_x,
                                  const void* W_dt, const float* b_dt, void* U, void* delta_r, float* Bm, float* Cm, void* Delta,
                                  int32_t* status, cudaStream_t st) {
  const int T = c.B * c.L, De = c.d_inner, R = c.dt_rank, N = c.d_state;
  const int N1 = R + 2 * N;
  const int block_n1 = (N1 + 31) / 32 * 32;
  const int block_n3 = De >= 256 ? 256 : (De + 31) / 32 * 32;
  CUtensorMap th, twx, twdt;
  if (!make_tmap(&th, HZ, (uint64_t)T, (uint64_t)De, (uint64_t)ldh, (uint32_t)FH_ROWS)) return cudaErrorInvalidValue;
  if (!make_tmap(&twx, W_x, (uint64_t)N1, (uint64_t)De, (uint64_t)De, (uint32_t)block_n1)) return cudaErrorInvalidValue;
  if (!make_tmap(&twdt, W_dt, (uint64_t)De, (uint64_t)R, (uint64_t)R, (uint32_t)block_n3)) return cudaErrorInvalidValue;
  // instruction descriptors: D = f32, A = B = bf16, both K-major, N >> 3 at bit 17, M >> 4 at bit 24
  auto idesc = [](int n) { return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(BLOCK_M >> 4) << 24); };
  // tokens per CTA: the fewest waves of 128-token tiles, then the rows spread evenly over the SMs of those waves
  int num_sms = 0;
  cudaError_t e = current_device_sm_count(&num_sms);
  if (e != cudaSuccess) return e;
  const long long waves = ((long long)T + (long long)BLOCK_M * num_sms - 1) / ((long long)BLOCK_M * num_sms);
  int rows_cta = (int)((T + waves * num_sms - 1) / (waves * num_sms));
  rows_cta = (rows_cta + 7) / 8 * 8;
  if (rows_cta > BLOCK_M) rows_cta = BLOCK_M;
  const FusedArgs a{static_cast<const __nv_bfloat16*>(HZ), ldh, static_cast<const __nv_bfloat16*>(w_conv), b_conv, b_dt,
                    static_cast<__nv_bfloat16*>(U), static_cast<__nv_bfloat16*>(delta_r), Bm, Cm, static_cast<__nv_bfloat16*>(Delta),
                    T, c.L, De, R, N, c.d_conv, block_n1, block_n3, rows_cta};
  auto kern = c.d_conv == 4 ? fused_conv_xdt_kernel<4> : c.d_conv == 3 ? fused_conv_xdt_kernel<3> : fused_conv_xdt_kernel<2>;
  e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, F_SMEM);
  if (e != cudaSuccess) return e;
  kern<<<(T + rows_cta - 1) / rows_cta, F_THREADS, F_SMEM, st>>>(th, twx, twdt, a, idesc(block_n1), idesc(block_n3), status, WAIT_LIMIT);
  count_launch();
  return cudaGetLastError();
}

}  // namespace rom
