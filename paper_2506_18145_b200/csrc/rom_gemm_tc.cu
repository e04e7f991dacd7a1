// bf16 grouped GEMM on the 5th-generation tensor cores (tcgen05 + TMEM), operands staged by TMA.
//
//   C[M, N] = A[M, Kd] * B[e(m)][N, Kd]^T,  fp32 accumulation in tensor memory.
//
// A holds token rows grouped by expert, every expert segment padded to a multiple of the 128-row
// tile, so a row tile never straddles two experts and a device-built table gives the expert of each
// row tile; the number of row tiles is read from device memory (no host synchronisation).  This is
// the per-expert Conv/Gate projection and Out projection of Section 4.2 (dropless, Section 5.1); with
// one "expert" it also serves the shared x Proj / dt Proj.
//
// One persistent CTA per SM, 320 threads:
//   warp 0      TMA producer: A tile 128x64 and B tile block_n x 64 per stage, 128-byte swizzle
//   warp 1      allocates TMEM, issues tcgen05.mma (one thread), commits to mbarriers
//   warps 2..9  epilogue: tcgen05.ld of the 128 x block_n fp32 accumulator, fused output op, stores;
//               two warps share each 32-lane quarter of tensor memory and take alternate 32-column
//               chunks, and the load of the next chunk is in flight while one chunk is processed
// The accumulator is double-buffered in TMEM (2 x 256 columns) so the epilogue of tile i overlaps
// the MMAs of tile i+1.  Every mbarrier wait is bounded; on expiry the CTA latches an error code in
// the status word, waits (bounded) for its own copies and for the MMAs it already issued, frees its
// TMEM and returns.
//
// Every TMA load here is a plain single-CTA load (no thread-block clusters).
#include "rom_tc_ptx.cuh"

namespace rom {
namespace {

constexpr int NUM_EPI_WARPS_C = 8;
constexpr int MAX_BLOCK_N = 256;
constexpr int MAX_STAGES = 4;
constexpr int A_STAGE_BYTES = BLOCK_M * BLOCK_K * 2;          // 16 KB
constexpr int B_STAGE_BYTES = MAX_BLOCK_N * BLOCK_K * 2;      // 32 KB
constexpr int STAGE_BYTES = A_STAGE_BYTES + B_STAGE_BYTES;
constexpr int ACC_STAGES = 2;
constexpr int TMEM_COLS = 512;
constexpr int NUM_EPI_WARPS = NUM_EPI_WARPS_C;
constexpr int NUM_THREADS = 64 + 32 * NUM_EPI_WARPS;
// The dt Proj (softplus output ops) has two K blocks per tile and about ten instructions plus two special-function
// operations per output element: its time is its epilogue's, so it runs sixteen epilogue warps instead of eight.
__host__ __device__ constexpr int epi_warps_of(int mode) { return (mode == EPI_SOFTPLUS || mode == EPI_SOFTPLUS_ROWS) ? 16 : NUM_EPI_WARPS_C; }
__host__ __device__ constexpr int threads_of(int mode) { return 64 + 32 * epi_warps_of(mode); }
// Operand stages and epilogue staging per output op.  The softplus epilogue (dt Proj: only two K blocks per tile,
// and the one GEMM here whose time is its fp32 output) gives up one operand stage for a 32 x 32 fp32 staging
// square per epilogue warp, through which its stores become whole 128-byte row segments.
__host__ __device__ constexpr bool f32_out(int mode) { return mode == EPI_SOFTPLUS || mode == EPI_F32 || mode == EPI_SOFTPLUS_ROWS; }
// The x Proj (a narrow B tile, one wave of row tiles, time set by how many bytes of A are in flight) runs six
// smaller stages: its B tile is at most XPROJ_BLOCK_N rows.
constexpr int XPROJ_BLOCK_N = 160;
__host__ __device__ constexpr int stage_bytes_of(int mode) {
  return mode == EPI_XPROJ ? A_STAGE_BYTES + XPROJ_BLOCK_N * BLOCK_K * 2 : STAGE_BYTES;
}
__host__ __device__ constexpr int stages_of(int mode) { return f32_out(mode) ? 3 : mode == EPI_XPROJ ? 6 : MAX_STAGES; }
__host__ __device__ constexpr int out_stage_bytes_of(int mode) { return f32_out(mode) ? epi_warps_of(mode) * 32 * 32 * 4 : 0; }
__host__ __device__ constexpr int smem_bytes_of(int mode) {
  return stages_of(mode) * stage_bytes_of(mode) + 1024 /*alignment slack*/ + 256 /*barriers*/ + out_stage_bytes_of(mode);
}

// Bias of the 32 columns [n0, n0+32) (EPI_SOFTPLUS only), requested before the accumulator chunk is waited for.
template <int MODE>
__device__ __forceinline__ void load_bias(const Epilogue& ep, int n0, int N, float4 (&bq)[8]) {
  if constexpr (MODE == EPI_SOFTPLUS || MODE == EPI_SOFTPLUS_ROWS) {
#pragma unroll
    for (int i = 0; i < 8; ++i)
      bq[i] = (ep.bias && n0 + 4 * i < N) ? __ldg(reinterpret_cast<const float4*>(ep.bias + n0) + i) : make_float4(0.0f, 0.0f, 0.0f, 0.0f);
  }
}

// Fused output op on 32 consecutive accumulator columns [n0, n0+32) of row m (n0 % 32 == 0); columns at
// or beyond N are skipped in groups of 8 (N % 8 == 0).
// m: output row; m_tok (EPI_XPROJ with row_token only): row of the B / C parts, the token of this expert-order row.
template <int MODE>
__device__ __forceinline__ void epi_store32(const Epilogue& ep, size_t m, size_t m_tok, int n0, int N, const uint32_t (&r)[32],
                                            float scale, const float4 (&bq)[8]) {
#pragma unroll
  for (int j = 0; j < 32; j += 8) {
    const int n = n0 + j;
    if (n >= N) break;
    float v[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __uint_as_float(r[j + i]);
    if (MODE == EPI_INPROJ && n >= ep.R) {
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] = silu_fast(v[i]);
    }
    if (MODE == EPI_OUTPROJ) {
#pragma unroll
      for (int i = 0; i < 8; ++i) v[i] *= scale;
    }
    if (MODE == EPI_STORE || MODE == EPI_INPROJ || MODE == EPI_OUTPROJ || (MODE == EPI_XPROJ && n < ep.R)) {
      const int ld = MODE == EPI_XPROJ ? ep.R : ep.ldc;
      uint4 q;
      uint32_t* w = reinterpret_cast<uint32_t*>(&q);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
        w[i] = *reinterpret_cast<uint32_t*>(&h);
      }
      *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(ep.C) + m * ld + n) = q;
    } else if (MODE == EPI_XPROJ) {
      float* dst = (n < ep.R + ep.N) ? ep.Bm + m_tok * ep.N + (n - ep.R) : ep.Cm + m_tok * ep.N + (n - ep.R - ep.N);
      *reinterpret_cast<float4*>(dst) = make_float4(v[0], v[1], v[2], v[3]);
      *reinterpret_cast<float4*>(dst + 4) = make_float4(v[4], v[5], v[6], v[7]);
    } else {
      // (softplus and plain-fp32 output go through epi_softplus32; nothing reaches this branch)
    }
  }
}

// Softplus output op on a 32 (rows of this warp) x 32 (columns) accumulator square: every lane activates its row,
// the square goes through a swizzled shared-memory staging area, and is written as whole 128-byte row segments
// (8 lanes per row, 4 rows per store instruction) instead of 32 scattered 16-byte pieces.
template <int MODE>
__device__ __forceinline__ void epi_softplus32(const Epilogue& ep, float* sw, int row0, int M_valid, int n0, int N,
                                               const uint32_t (&r)[32], const float4 (&bq)[8], int lane) {
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    float4 o;
    if constexpr (MODE == EPI_F32) {      // plain fp32 rows, no bias, no activation
      o = make_float4(__uint_as_float(r[4 * c]), __uint_as_float(r[4 * c + 1]), __uint_as_float(r[4 * c + 2]), __uint_as_float(r[4 * c + 3]));
    } else {
      const float4 b = bq[c];
      o = make_float4(softplus_bf16(__uint_as_float(r[4 * c]) + b.x), softplus_bf16(__uint_as_float(r[4 * c + 1]) + b.y),
                      softplus_bf16(__uint_as_float(r[4 * c + 2]) + b.z), softplus_bf16(__uint_as_float(r[4 * c + 3]) + b.w));
    }
    *reinterpret_cast<float4*>(sw + lane * 32 + ((c ^ (lane & 7)) << 2)) = o;
  }
  __syncwarp();
  if constexpr (MODE == EPI_F32) {
    const int c = lane & 7;
    const int n = n0 + 4 * c;
#pragma unroll
    for (int r4 = 0; r4 < 8; ++r4) {
      const int R = r4 * 4 + (lane >> 3);
      const float4 v = *reinterpret_cast<const float4*>(sw + R * 32 + ((c ^ (R & 7)) << 2));
      if (row0 + R < M_valid && n < N) *reinterpret_cast<float4*>(reinterpret_cast<float*>(ep.C) + (size_t)(row0 + R) * ep.ldc + n) = v;
    }
  } else {
    // rounded to bf16: a lane takes 8 columns (two staged float4), 4 lanes one 64-byte row segment, 8 rows per store
    const int c8 = lane & 3;
    const int n = n0 + 8 * c8;
#pragma unroll
    for (int r8 = 0; r8 < 4; ++r8) {
      const int R = r8 * 8 + (lane >> 2);
      const float4 v0 = *reinterpret_cast<const float4*>(sw + R * 32 + (((2 * c8) ^ (R & 7)) << 2));
      const float4 v1 = *reinterpret_cast<const float4*>(sw + R * 32 + (((2 * c8 + 1) ^ (R & 7)) << 2));
      uint4 q;
      __nv_bfloat162 h0 = __floats2bfloat162_rn(v0.x, v0.y), h1 = __floats2bfloat162_rn(v0.z, v0.w);
      __nv_bfloat162 h2 = __floats2bfloat162_rn(v1.x, v1.y), h3 = __floats2bfloat162_rn(v1.z, v1.w);
      q.x = *reinterpret_cast<uint32_t*>(&h0); q.y = *reinterpret_cast<uint32_t*>(&h1);
      q.z = *reinterpret_cast<uint32_t*>(&h2); q.w = *reinterpret_cast<uint32_t*>(&h3);
      if (row0 + R < M_valid && n < N) {
        // per-expert dt Proj at top-1: the row goes to its token's position (padding rows are skipped)
        const int orow = MODE == EPI_SOFTPLUS_ROWS ? __ldg(ep.row_token + row0 + R) : row0 + R;
        if (orow >= 0) *reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(ep.C) + (size_t)orow * ep.ldc + n) = q;
      }
    }
  }
  __syncwarp();
}

template <int MODE>
__global__ void __launch_bounds__(threads_of(MODE), 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
               int M_max, int N, int Kd, int block_n, uint32_t idesc,
               const int32_t* __restrict__ tile_expert, const int32_t* __restrict__ num_m_tiles_dev,
               Epilogue ep, int32_t* __restrict__ status, uint32_t wait_limit, int withhold_kb,
               const int32_t* __restrict__ k_seg, int n_seg) {
  constexpr int STAGES = stages_of(MODE);
  constexpr int SB = stage_bytes_of(MODE);          // bytes per operand stage (multiple of 1024)
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;               // 128B-swizzled tiles need 1024-byte alignment
  unsigned char* smem = smem_raw + (base - raw);
  const uint32_t bars = base + STAGES * SB;                   // barrier block (8-byte aligned)
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (2 * STAGES + ACC_STAGES + a); };
  const uint32_t drain_bar = bars + 8u * (2 * STAGES + 2 * ACC_STAGES);      // abort path only: completion of the MMAs already issued
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(smem + STAGES * SB + 8 * (2 * STAGES + 2 * ACC_STAGES + 1));
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  float* out_stage = reinterpret_cast<float*>(smem + STAGES * SB + 256);        // [8 warps][32][32] (softplus only)

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  int num_m_tiles = (M_max + BLOCK_M - 1) / BLOCK_M;
  if (num_m_tiles_dev) num_m_tiles = min(num_m_tiles, *num_m_tiles_dev);
  const int M_valid = min(M_max, num_m_tiles * BLOCK_M);
  // EPI_SWIGLU: a tile holds 128 gate columns and the 128 up columns of the same hidden units
  const int n_tiles = MODE == EPI_SWIGLU ? N / 128 : (N + block_n - 1) / block_n;
  // Weight-gradient mode (k_seg != nullptr): n_seg independent problems share A and B; problem s contracts the K range
  // [k_seg[s], k_seg[s+1]) (multiples of BLOCK_K; an expert's padded row segment) and writes rows [s M_max, (s+1) M_max) of C.
  const int seg_tiles = num_m_tiles * n_tiles;
  const int total_tiles = k_seg ? n_seg * seg_tiles : seg_tiles;
  const int num_kb = (Kd + BLOCK_K - 1) / BLOCK_K;
  auto decode = [&](int tile, int& m_tile, int& n_tile, int& seg, int& kb0, int& nkb) {
    seg = 0; kb0 = 0; nkb = num_kb;
    int lt = tile;
    if (k_seg) {
      seg = tile / seg_tiles;
      lt = tile - seg * seg_tiles;
      kb0 = k_seg[seg] / BLOCK_K;
      nkb = (k_seg[seg + 1] - k_seg[seg]) / BLOCK_K;
    }
    m_tile = lt / n_tiles;
    n_tile = lt - m_tile * n_tiles;
  };
  const uint32_t stage_tx = A_STAGE_BYTES + (uint32_t)block_n * BLOCK_K * 2;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(full_bar(s), 1); mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < ACC_STAGES; ++a) { mbar_init(tfull_bar(a), 1); mbar_init(tempty_bar(a), epi_warps_of(MODE)); }
    mbar_init(drain_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_holder)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      int issued = 0;
      bool ok = true;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        int m_tile, n_tile, seg, kb0, nkb;
        decode(tile, m_tile, n_tile, seg, kb0, nkb);
        const int e = tile_expert ? tile_expert[m_tile] : 0;
        const int b_row = MODE == EPI_SWIGLU ? e * 2 * N + n_tile * 128 : e * N + n_tile * block_n;
        for (int kq = 0; kq < nkb; ++kq) {
          const int kb = kb0 + kq;
          if (!mbar_wait(empty_bar(stage), phase ^ 1u, abort_flag, wait_limit)) { ok = false; break; }
          mbar_expect_tx(full_bar(stage), stage_tx);
          const uint32_t sa = base + stage * SB;
          // fault injection (tests only): the copies of K block `withhold_kb` of this CTA's first tile are never issued,
          // so the stage never fills and the waits downstream run out
          if (!(withhold_kb >= 0 && tile == (int)blockIdx.x && kq == withhold_kb)) {
            tma_load_2d(sa, &tmap_a, full_bar(stage), kb * BLOCK_K, m_tile * BLOCK_M);
            tma_load_2d(sa + A_STAGE_BYTES, &tmap_b, full_bar(stage), kb * BLOCK_K, b_row);
            if (MODE == EPI_SWIGLU)     // second half of the B tile: the up rows of the same 128 hidden units (box = 128 rows)
              tma_load_2d(sa + A_STAGE_BYTES + 128 * BLOCK_K * 2, &tmap_b, full_bar(stage), kb * BLOCK_K, b_row + N);
          }
          ++issued;
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (!ok) {
        if (!*abort_flag) { atomicExch(status + kStatCode, ROM_ERR_DEVICE_TIMEOUT); atomicExch(status + kStatWhere, 1); }
        *abort_flag = 1;
      }
      if (*abort_flag) {
        // drain: give this CTA's copies still in flight a bounded time to land before the CTA exits
        int s = stage; uint32_t ph = phase;
        for (int i = 0; i < min(issued, STAGES); ++i) {
          if (--s < 0) { s = STAGES - 1; ph ^= 1u; }
          for (uint32_t it = 0; it < (wait_limit >> 2); ++it)
            if (mbar_try_wait(full_bar(s), ph)) break;
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int stage = 0; uint32_t phase = 0;
      int acc = 0; uint32_t acc_phase = 0;
      bool ok = true, issued_any = false;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
        if (!mbar_wait(tempty_bar(acc), acc_phase ^ 1u, abort_flag, wait_limit)) { ok = false; break; }
        tc_fence_after();
        const uint32_t tmem_d = tmem_base + (uint32_t)acc * MAX_BLOCK_N;
        int m_tile_, n_tile_, seg_, kb0_, nkb;
        decode(tile, m_tile_, n_tile_, seg_, kb0_, nkb);
        for (int kb = 0; kb < nkb; ++kb) {
          if (!mbar_wait(full_bar(stage), phase, abort_flag, wait_limit)) { ok = false; break; }
          tc_fence_after();
          const uint32_t sa = base + stage * SB;
          const uint64_t adesc = make_smem_desc(sa);
          const uint64_t bdesc = make_smem_desc(sa + A_STAGE_BYTES);
#pragma unroll
          for (int k = 0; k < BLOCK_K / UMMA_K; ++k) {
            // advance 16 elements = 32 bytes along K inside the swizzled row: +2 in the address field
            umma_bf16(tmem_d, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), idesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(empty_bar(stage));
          issued_any = true;
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        umma_commit(tfull_bar(acc));
        if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
      }
      if (!ok) {
        if (!*abort_flag) { atomicExch(status + kStatCode, ROM_ERR_DEVICE_TIMEOUT); atomicExch(status + kStatWhere, 2); }
        *abort_flag = 1;
      }
      if (*abort_flag && issued_any) {
        // the MMAs already issued may still read shared memory and write tensor memory: one more commit tracks them
        // all; wait for it (bounded) before the CTA frees its tensor memory
        umma_commit(drain_bar);
        for (uint32_t it = 0; it < (wait_limit >> 2); ++it)
          if (mbar_try_wait(drain_bar, 0)) break;
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..9)
    const int quarter = warp & 3;                 // TMEM lanes [32*quarter, 32*quarter+32) belong to this warp
    constexpr int EWQ = epi_warps_of(MODE) / 4;   // warps per lane quarter
    const int half = (warp - 2) >> 2;             // which of the EWQ warps of the quarter: takes chunks half, half+EWQ, ...
    const int n_chunks = block_n >> 5;
    int acc = 0; uint32_t acc_phase = 0;
    bool ok = true;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      int m_tile, n_tile, seg, kb0_, nkb;
      decode(tile, m_tile, n_tile, seg, kb0_, nkb);
      // warp-uniform outcome: the tensor-memory loads below need the whole warp
      if (!__all_sync(0xffffffffu, mbar_wait(tfull_bar(acc), acc_phase, abort_flag, wait_limit))) { ok = false; break; }
      tc_fence_after();
      const int row = m_tile * BLOCK_M + quarter * 32 + lane;
      bool row_ok = row < M_valid;
      size_t out_row = (size_t)row;
      float scale = 1.0f;
      size_t tok_row = (size_t)row;
      if ((MODE == EPI_OUTPROJ || (MODE == EPI_INPROJ && ep.row_token != nullptr)) && row_ok) {
        const int tok = __ldg(ep.row_token + row);      // rows are written at their token's position
        row_ok = tok >= 0;
        if (row_ok) {
          out_row = (size_t)tok;
          if (MODE == EPI_OUTPROJ) scale = __ldg(ep.row_scale + tok);
        }
      }
      if (MODE == EPI_XPROJ && ep.row_token != nullptr && row_ok) {
        // per-expert x Proj at top-1: delta_r stays in expert order (it feeds the grouped dt Proj), B and C go to the token's row
        const int tok = __ldg(ep.row_token + row);
        row_ok = tok >= 0;
        tok_row = row_ok ? (size_t)tok : 0;
      }
      const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)acc * MAX_BLOCK_N;
      const int n_base = n_tile * block_n;
      uint32_t ra[32], rb[32];
      float4 bq[8];
      if constexpr (MODE == EPI_SWIGLU) {
        // accumulator columns [0,128) = gate, [128,256) = up; this warp takes 32-column groups half and half + 2
        for (int c = half; c < 4; c += 2) {
          tmem_ld32_issue(taddr + c * 32, ra);
          tmem_ld32_issue(taddr + 128 + c * 32, rb);
          tmem_ld_wait(ra);
          tmem_ld_wait(rb);
          if (row_ok) {
            __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(ep.C) + out_row * ep.ldc + n_tile * 128 + c * 32;
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
              uint4 q;
              uint32_t* w = reinterpret_cast<uint32_t*>(&q);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                const float v0 = silu_fast(__uint_as_float(ra[j + 2 * i])) * __uint_as_float(rb[j + 2 * i]);
                const float v1 = silu_fast(__uint_as_float(ra[j + 2 * i + 1])) * __uint_as_float(rb[j + 2 * i + 1]);
                __nv_bfloat162 hh = __floats2bfloat162_rn(v0, v1);
                w[i] = *reinterpret_cast<uint32_t*>(&hh);
              }
              *reinterpret_cast<uint4*>(dst + j) = q;
            }
          }
        }
      }
      if constexpr (EWQ == 4) {
        // sixteen warps: at most two chunks each, one register buffer (the register file has no room for two)
        uint4* stage = reinterpret_cast<uint4*>(out_stage + (warp - 2) * 1024);
        const int c0 = 2 * half;                       // this warp's chunks: c0 and c0 + 1
        int n_pieces = 0;
        for (int cc = 0; cc < 2 && c0 + cc < n_chunks; ++cc) {
          tmem_ld32_issue(taddr + (c0 + cc) * 32, ra);
          load_bias<MODE>(ep, n_base + (c0 + cc) * 32, N, bq);
          tmem_ld_wait(ra);
          softplus_stage_bf16(stage, 4 * cc, ra, bq, lane);
          n_pieces += 4;
        }
        if (n_pieces > 0) {
          __syncwarp();
          softplus_flush_bf16<MODE>(ep, stage, m_tile * BLOCK_M + quarter * 32, M_valid, n_base + c0 * 32, N, n_pieces, lane);
          __syncwarp();
        }
      }
      // weight-gradient mode: problem `seg` owns its own rows of C; an empty K range leaves zeros
      Epilogue epl = ep;
      if (MODE == EPI_F32 && k_seg) epl.C = reinterpret_cast<float*>(ep.C) + (size_t)seg * M_max * ep.ldc;
      const bool zero_acc = MODE == EPI_F32 && k_seg && nkb == 0;
      int ch = (MODE == EPI_SWIGLU || EWQ == 4) ? n_chunks : half;
      if (ch < n_chunks) tmem_ld32_issue(taddr + ch * 32, ra);
      // two register buffers: while one chunk is processed the next chunk's tensor-memory load is in flight
      while (ch < n_chunks) {
        load_bias<MODE>(ep, n_base + ch * 32, N, bq);     // in flight together with the tensor-memory load
        tmem_ld_wait(ra);
        if (ch + EWQ < n_chunks) tmem_ld32_issue(taddr + (ch + EWQ) * 32, rb);
        if (zero_acc) {
#pragma unroll
          for (int i = 0; i < 32; ++i) ra[i] = 0u;
        }
        if (f32_out(MODE)) epi_softplus32<MODE>(epl, out_stage + (warp - 2) * 1024, m_tile * BLOCK_M + quarter * 32, M_valid, n_base + ch * 32, N, ra, bq, lane);
        else if (row_ok) epi_store32<MODE>(ep, out_row, tok_row, n_base + ch * 32, N, ra, scale, bq);
        ch += EWQ;
        if (ch >= n_chunks) break;
        load_bias<MODE>(ep, n_base + ch * 32, N, bq);
        tmem_ld_wait(rb);
        if (ch + EWQ < n_chunks) tmem_ld32_issue(taddr + (ch + EWQ) * 32, ra);
        if (zero_acc) {
#pragma unroll
          for (int i = 0; i < 32; ++i) rb[i] = 0u;
        }
        if (f32_out(MODE)) epi_softplus32<MODE>(epl, out_stage + (warp - 2) * 1024, m_tile * BLOCK_M + quarter * 32, M_valid, n_base + ch * 32, N, rb, bq, lane);
        else if (row_ok) epi_store32<MODE>(ep, out_row, tok_row, n_base + ch * 32, N, rb, scale, bq);
        ch += EWQ;
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(tempty_bar(acc));
      if (++acc == ACC_STAGES) { acc = 0; acc_phase ^= 1u; }
    }
    if (!ok && lane == 0) {
      if (!*abort_flag) { atomicExch(status + kStatCode, ROM_ERR_DEVICE_TIMEOUT); atomicExch(status + kStatWhere, 3); }
      *abort_flag = 1;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace

cudaError_t launch_gemm_tc(const void* A, int lda, const void* Bw, int ldb, int n_experts, int M_max, int N, int Kd,
                           const int32_t* tile_expert, const int32_t* num_m_tiles_dev, const Epilogue& epi,
                           int32_t* status, cudaStream_t st, bool test_stall) {
  // N tile: a multiple of 32 (epilogue column groups) and of 16 (UMMA N for M = 128), at most 256
  const bool swiglu = epi.mode == EPI_SWIGLU;      // N output columns from 2N rows of B per expert, loaded as two boxes of 128 rows
  if (swiglu && (N % 128 != 0 || MAX_BLOCK_N != 256)) return cudaErrorInvalidValue;
  int block_n = (swiglu || N >= MAX_BLOCK_N) ? MAX_BLOCK_N : (N + 31) / 32 * 32;
  if (epi.mode == EPI_XPROJ && block_n > XPROJ_BLOCK_N) block_n = XPROJ_BLOCK_N;
  CUtensorMap ta, tb;
  if (!make_tmap(&ta, A, (uint64_t)M_max, (uint64_t)Kd, (uint64_t)lda, BLOCK_M)) return cudaErrorInvalidValue;
  if (!make_tmap(&tb, Bw, (uint64_t)n_experts * (swiglu ? 2 * N : N), (uint64_t)Kd, (uint64_t)ldb, swiglu ? 128u : (uint32_t)block_n))
    return cudaErrorInvalidValue;
  // instruction descriptor: D = f32, A = B = bf16, both K-major, N >> 3 at bit 17, M >> 4 at bit 24
  const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(block_n >> 3) << 17) | ((uint32_t)(BLOCK_M >> 4) << 24);
  int num_sms = 0;
  cudaError_t e = current_device_sm_count(&num_sms);
  if (e != cudaSuccess) return e;
  auto kern = epi.mode == EPI_STORE ? gemm_tc_kernel<EPI_STORE> : epi.mode == EPI_XPROJ ? gemm_tc_kernel<EPI_XPROJ>
              : epi.mode == EPI_INPROJ ? gemm_tc_kernel<EPI_INPROJ> : epi.mode == EPI_OUTPROJ ? gemm_tc_kernel<EPI_OUTPROJ>
              : epi.mode == EPI_F32 ? gemm_tc_kernel<EPI_F32> : epi.mode == EPI_SWIGLU ? gemm_tc_kernel<EPI_SWIGLU>
              : epi.mode == EPI_SOFTPLUS_ROWS ? gemm_tc_kernel<EPI_SOFTPLUS_ROWS>
              : gemm_tc_kernel<EPI_SOFTPLUS>;
  const int smem_bytes = smem_bytes_of(epi.mode);
  e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  if (e != cudaSuccess) return e;
  const int n_tiles = swiglu ? N / 128 : (N + block_n - 1) / block_n;
  const long long max_tiles = (long long)((M_max + BLOCK_M - 1) / BLOCK_M) * n_tiles;
  const int grid = (int)(max_tiles < num_sms ? max_tiles : num_sms);
  kern<<<grid, threads_of(epi.mode), smem_bytes, st>>>(ta, tb, M_max, N, Kd, block_n, idesc, tile_expert, num_m_tiles_dev, epi, status,
                                                            test_stall ? WAIT_LIMIT_TEST : WAIT_LIMIT, test_stall ? 1 : -1, nullptr, 0);
  count_launch();
  return cudaGetLastError();
}

// Grouped weight gradient on the tensor cores: C[s][P, Q] (fp32) = sum over the rows r in [seg[s], seg[s+1]) of Xt[p, r] Yt[q, r].
// Xt [P, ld], Yt [Q, ld]: the activations transposed, so the contracted token rows are contiguous; seg: n_seg + 1 device offsets,
// multiples of 64 (the padded expert segments); rows outside every segment are never read.
cudaError_t launch_gemm_tc_wgrad(const void* Xt, const void* Yt, int ld, const int32_t* seg, int n_seg, int P, int Q, float* C,
                                 int32_t* status, cudaStream_t st) {
  const int block_n = Q >= MAX_BLOCK_N ? MAX_BLOCK_N : (Q + 31) / 32 * 32;
  CUtensorMap ta, tb;
  if (!make_tmap(&ta, Xt, (uint64_t)P, (uint64_t)ld, (uint64_t)ld, BLOCK_M)) return cudaErrorInvalidValue;
  if (!make_tmap(&tb, Yt, (uint64_t)Q, (uint64_t)ld, (uint64_t)ld, (uint32_t)block_n)) return cudaErrorInvalidValue;
  const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(block_n >> 3) << 17) | ((uint32_t)(BLOCK_M >> 4) << 24);
  int num_sms = 0;
  cudaError_t e = current_device_sm_count(&num_sms);
  if (e != cudaSuccess) return e;
  const int smem_bytes = smem_bytes_of(EPI_F32);
  e = cudaFuncSetAttribute(gemm_tc_kernel<EPI_F32>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes);
  if (e != cudaSuccess) return e;
  const int n_tiles = (Q + block_n - 1) / block_n;
  const long long max_tiles = (long long)n_seg * ((P + BLOCK_M - 1) / BLOCK_M) * n_tiles;
  const int grid = (int)(max_tiles < num_sms ? max_tiles : num_sms);
  const Epilogue epi{EPI_F32, C, Q, nullptr, nullptr, nullptr, 0, 0, nullptr, nullptr};
  gemm_tc_kernel<EPI_F32><<<grid, threads_of(EPI_F32), smem_bytes, st>>>(ta, tb, P, Q, ld, block_n, idesc, nullptr, nullptr, epi, status,
                                                                        WAIT_LIMIT, -1, seg, n_seg);
  count_launch();
  return cudaGetLastError();
}

}  // namespace rom
