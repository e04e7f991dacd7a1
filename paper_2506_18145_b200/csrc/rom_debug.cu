// Debug checks (ROM_FLAG_DEBUG_CHECKS): a substitute for a memory checker on machines where none can run.
//
// Every gather and scatter of the layer takes its row index from the routing tables (row of each assignment,
// assignment of each row, expert of each row tile, padded segment offsets), so validating those tables on
// the device before any kernel consumes them bounds every indexed access of the forward.  Canary words sit
// between the sub-buffers of the workspace; they are written before the first kernel and compared after the
// last, so a kernel that writes past its buffer is reported with the index of the canary it damaged.
// Violations are latched in the workspace status word (first one wins) and read with rom_get_status.
#include "rom_internal.cuh"

namespace rom {
namespace {

constexpr uint32_t kCanaryWord = 0xC0FFEE00u;

__device__ __forceinline__ void latch(int32_t* status, int where, int index) {
  if (atomicCAS(status + kStatCode, 0, (int)ROM_ERR_DEBUG_CHECK) == 0) {
    status[kStatWhere] = where;
    status[kStatIndex] = index;
  }
}

__global__ void __launch_bounds__(256)
check_tables_kernel(const int32_t* __restrict__ row_of_assign, const int32_t* __restrict__ assign_of_row,
                    const int32_t* __restrict__ tile_expert, const int32_t* __restrict__ num_m_tiles,
                    const int32_t* __restrict__ pad_offsets, int A, int rows_max, int max_m_tiles, int E, int32_t* status) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < A) {                                   // every assignment has a row inside the padded range, and the maps agree
    const int r = row_of_assign[i];
    if (r < 0 || r >= rows_max) latch(status, 10, i);
    else if (assign_of_row[r] != i) latch(status, 11, i);
  }
  if (i < rows_max) {                            // every row is padding (-1) or points back at its assignment
    const int a = assign_of_row[i];
    if (a != -1 && (a < 0 || a >= A || row_of_assign[a] != i)) latch(status, 12, i);
  }
  const int nt = *num_m_tiles;
  if (i == 0 && (nt < 0 || nt > max_m_tiles)) latch(status, 13, nt);
  if (i < min(nt, max_m_tiles)) {                // every row tile names a real expert
    const int e = tile_expert[i];
    if (e < 0 || e >= E) latch(status, 14, i);
  }
  if (i <= E) {                                  // padded segment offsets: multiples of the row tile, ascending, ending at the tile count
    const int o = pad_offsets[i];
    if (o % kTileM != 0 || o < 0 || (i > 0 && o < pad_offsets[i - 1]) || (i == E && o != nt * kTileM)) latch(status, 15, i);
  }
}

struct CanaryList { unsigned long long off[kMaxCanaries]; int n; };

__global__ void __launch_bounds__(64)
canary_kernel(char* ws, const CanaryList list, int check, int32_t* status) {
  const int c = blockIdx.x;
  if (c >= list.n) return;
  uint32_t* w = reinterpret_cast<uint32_t*>(ws + list.off[c]);
  const uint32_t want = kCanaryWord + (uint32_t)c;
  if (!check) w[threadIdx.x] = want;
  else if (w[threadIdx.x] != want) latch(status, 20, c);
}

}  // namespace

cudaError_t launch_check_tables(const rom_config& c, char* ws, const WsLayout& lay, cudaStream_t st) {
  const long long n = lay.rows_max > lay.A ? lay.rows_max : lay.A;
  check_tables_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(
      reinterpret_cast<const int32_t*>(ws + lay.row_of_assign), reinterpret_cast<const int32_t*>(ws + lay.assign_of_row),
      reinterpret_cast<const int32_t*>(ws + lay.tile_expert), reinterpret_cast<const int32_t*>(ws + lay.num_m_tiles),
      reinterpret_cast<const int32_t*>(ws + lay.pad_offsets), (int)lay.A, (int)lay.rows_max, (int)lay.max_m_tiles, c.E,
      reinterpret_cast<int32_t*>(ws + lay.status));
  count_launch();
  return cudaGetLastError();
}

cudaError_t launch_canaries(char* ws, const WsLayout& lay, bool check, cudaStream_t st) {
  if (lay.n_canary == 0) return cudaSuccess;
  CanaryList list{};
  list.n = lay.n_canary;
  for (int i = 0; i < lay.n_canary; ++i) list.off[i] = lay.canary[i];
  canary_kernel<<<lay.n_canary, 64, 0, st>>>(ws, list, check ? 1 : 0, reinterpret_cast<int32_t*>(ws + lay.status));
  count_launch();
  return cudaGetLastError();
}

}  // namespace rom
