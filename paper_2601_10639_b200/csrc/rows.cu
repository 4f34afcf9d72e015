// Row movers for a table that lives off the device: the prefetch gather
// (cache[r] = table[ids[r]]) and the gradient write-back.  Row counts are device scalars,
// so the grids are sized for the upper bound and CTAs stride over the real count.
// 16-byte accesses, one row spread across the CTA; when the table is page-locked host
// memory the loads cross the host link directly (no staging copy).
#include "stem_internal.h"

namespace stem {
namespace {

constexpr int kThreads = 256;

__global__ void __launch_bounds__(kThreads)
gather_rows_kernel(int V, int vec_per_row, const int32_t* __restrict__ ids,
                   const int32_t* __restrict__ n_ids, const uint4* __restrict__ table,
                   uint4* __restrict__ dst, int32_t* status) {
  const int n = *n_ids;
  // a CTA handles `rows_per_cta` rows per step so short rows still fill the block
  const int lanes_per_row = min(vec_per_row, kThreads);
  const int rows_per_cta = kThreads / lanes_per_row;
  const int sub = threadIdx.x / lanes_per_row, lane = threadIdx.x % lanes_per_row;
  if (sub >= rows_per_cta) return;
  for (int r = blockIdx.x * rows_per_cta + sub; r < n; r += gridDim.x * rows_per_cta) {
    int id = ids[r];
    if (id < 0 || id >= V) {
      if (lane == 0) report_error(status, STEM_ERR_ID_RANGE, r);
      id = id < 0 ? 0 : V - 1;
    }
    const uint4* src = table + static_cast<size_t>(id) * vec_per_row;
    uint4* out = dst + static_cast<size_t>(r) * vec_per_row;
    int c = lane;
    for (; c + 3 * lanes_per_row < vec_per_row; c += 4 * lanes_per_row) {
      const uint4 a0 = src[c], a1 = src[c + lanes_per_row], a2 = src[c + 2 * lanes_per_row],
                  a3 = src[c + 3 * lanes_per_row];
      out[c] = a0; out[c + lanes_per_row] = a1; out[c + 2 * lanes_per_row] = a2;
      out[c + 3 * lanes_per_row] = a3;
    }
    for (; c < vec_per_row; c += lanes_per_row) out[c] = src[c];
  }
}

__global__ void __launch_bounds__(kThreads)
writeback_rows_kernel(int vec_per_row, const uint4* __restrict__ rows,
                      const int32_t* __restrict__ unique_ids, const int32_t* __restrict__ n_rows,
                      uint4* __restrict__ host_rows, int32_t* __restrict__ host_ids,
                      int32_t* __restrict__ host_n) {
  const int n = *n_rows;
  const size_t total = static_cast<size_t>(n) * vec_per_row;
  const size_t stride = static_cast<size_t>(gridDim.x) * kThreads;
  for (size_t i = static_cast<size_t>(blockIdx.x) * kThreads + threadIdx.x; i < total; i += stride)
    host_rows[i] = rows[i];
  for (size_t i = static_cast<size_t>(blockIdx.x) * kThreads + threadIdx.x; i < static_cast<size_t>(n); i += stride)
    host_ids[i] = unique_ids[i];
  if (blockIdx.x == 0 && threadIdx.x == 0) *host_n = n;
}

}  // namespace

cudaError_t launch_gather_rows(int max_rows, int V, size_t row_bytes, const int32_t* ids,
                               const int32_t* n_ids, const void* table, void* dst,
                               int32_t* status, cudaStream_t stream) {
  if (max_rows <= 0) return cudaSuccess;
  const int vec = static_cast<int>(row_bytes / 16);
  const int lanes_per_row = vec < kThreads ? vec : kThreads;
  const int rows_per_cta = kThreads / lanes_per_row;
  int blocks = (max_rows + rows_per_cta - 1) / rows_per_cta;
  const int cap = device_sm_count() * 8;
  if (blocks > cap) blocks = cap;
  gather_rows_kernel<<<blocks, kThreads, 0, stream>>>(V, vec, ids, n_ids, static_cast<const uint4*>(table),
                                                     static_cast<uint4*>(dst), status);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_writeback_rows(int max_rows, size_t row_bytes, const void* rows,
                                  const int32_t* unique_ids, const int32_t* n_rows, void* host_rows,
                                  int32_t* host_ids, int32_t* host_n, cudaStream_t stream) {
  if (max_rows <= 0) return cudaSuccess;
  const int vec = static_cast<int>(row_bytes / 16);
  const int blocks = device_sm_count() * 4;
  writeback_rows_kernel<<<blocks, kThreads, 0, stream>>>(vec, static_cast<const uint4*>(rows), unique_ids,
                                                        n_rows, static_cast<uint4*>(host_rows), host_ids, host_n);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace stem
