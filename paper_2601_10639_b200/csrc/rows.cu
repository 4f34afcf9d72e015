// Row movers for a table that lives off the device: the prefetch gather
// (cache[r] = table[ids[r]]) and the gradient write-back.  Row counts are device scalars,
// so the grids are sized for the upper bound and CTAs stride over the real count.
// 16-byte accesses, one row spread across the CTA; when the table is page-locked host
// memory the loads cross the host link directly (no staging copy).  Kernels that talk to
// host memory are meant to run beside the contraction kernels of another layer, which hold
// every SM with one large CTA each: they are launched as kHostLinkCtas CTAs of
// kHostLinkThreads threads.  Even two of those fit next to a contraction CTA (registers,
// threads; no shared memory), so the contraction never waits for an SM, and eight 16-byte
// loads in flight per thread still cover several times the host link's bandwidth-delay
// product.
#include "stem_internal.h"

namespace stem {
namespace {

constexpr int kThreads = 256;          // device-to-device gathers
constexpr int kHostLinkCtas = 32;
constexpr int kHostLinkThreads = 128;

__global__ void __launch_bounds__(kThreads)
gather_rows_kernel(int max_rows, int V, int vec_per_row, const int32_t* __restrict__ ids,
                   const int32_t* __restrict__ n_ids, const uint4* __restrict__ table,
                   const uint4* __restrict__ hot_rows, const int32_t* __restrict__ hot_slot,
                   uint4* __restrict__ dst, int32_t* status, int32_t* stats) {
  // the count is a device scalar the host never saw: never trust it beyond the buffers' capacity
  int n = *n_ids;
  if (n > max_rows || n < 0) {
    if (blockIdx.x == 0 && threadIdx.x == 0) report_error(status, STEM_ERR_COUNT_RANGE, n);
    n = n < 0 ? 0 : max_rows;
  }
  // a CTA handles `rows_per_cta` rows per step so short rows still fill the block
  const int lanes_per_row = min(vec_per_row, static_cast<int>(blockDim.x));
  const int rows_per_cta = static_cast<int>(blockDim.x) / lanes_per_row;
  const int sub = threadIdx.x / lanes_per_row, lane = threadIdx.x % lanes_per_row;
  if (sub >= rows_per_cta) return;
  for (int r = blockIdx.x * rows_per_cta + sub; r < n; r += gridDim.x * rows_per_cta) {
    int id = ids[r];
    if (id < 0 || id >= V) {
      if (lane == 0) report_error(status, STEM_ERR_ID_RANGE, r);
      id = id < 0 ? 0 : V - 1;
    }
    // a row held in the on-device hot set is copied from there instead of crossing the host link
    const int slot = hot_slot != nullptr ? hot_slot[id] : -1;
    const uint4* src = slot >= 0 ? hot_rows + static_cast<size_t>(slot) * vec_per_row
                                 : table + static_cast<size_t>(id) * vec_per_row;
    if (stats != nullptr && lane == 0) atomicAdd(stats + (slot >= 0 ? 0 : 1), 1);
    uint4* out = dst + static_cast<size_t>(r) * vec_per_row;
    int c = lane;
    for (; c + 7 * lanes_per_row < vec_per_row; c += 8 * lanes_per_row) {
      uint4 a[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) a[j] = src[c + j * lanes_per_row];
#pragma unroll
      for (int j = 0; j < 8; ++j) out[c + j * lanes_per_row] = a[j];
    }
    for (; c + 3 * lanes_per_row < vec_per_row; c += 4 * lanes_per_row) {
      const uint4 a0 = src[c], a1 = src[c + lanes_per_row], a2 = src[c + 2 * lanes_per_row],
                  a3 = src[c + 3 * lanes_per_row];
      out[c] = a0; out[c + lanes_per_row] = a1; out[c + 2 * lanes_per_row] = a2;
      out[c + 3 * lanes_per_row] = a3;
    }
    for (; c < vec_per_row; c += lanes_per_row) out[c] = src[c];
  }
}

// Device-resident table (and hot set): the whole copy is one flat list of 16-byte vectors,
// vector i belonging to row i / vec_per_row, dealt to the threads in batches of kFlatBatch with
// the next batch's loads issued before the current batch is stored.  No thread ever waits on a
// row's id before it can ask for the row: every vector looks its id up itself (one cached 4-byte
// load shared by the whole row), so the id -> row address -> data chains of 2 * kFlatBatch
// vectors per thread overlap.
constexpr int kFlatBatch = 4;

__device__ __forceinline__ const uint4* flat_src(size_t i, int vec_per_row, int V, const int32_t* __restrict__ ids,
                                                 const uint4* __restrict__ table, const uint4* __restrict__ hot_rows,
                                                 const int32_t* __restrict__ hot_slot, int32_t* status, int32_t* stats) {
  // 32-bit division whenever the index allows (it nearly always does): far cheaper than 64-bit
  const int r = (i >> 32) == 0 ? static_cast<int>(static_cast<uint32_t>(i) / static_cast<uint32_t>(vec_per_row))
                               : static_cast<int>(i / vec_per_row);
  const int c = static_cast<int>(i - static_cast<size_t>(r) * vec_per_row);
  int id = __ldg(ids + r);
  if (id < 0 || id >= V) {
    if (c == 0) report_error(status, STEM_ERR_ID_RANGE, r);
    id = id < 0 ? 0 : V - 1;
  }
  const int slot = hot_slot != nullptr ? __ldg(hot_slot + id) : -1;
  if (stats != nullptr && c == 0) atomicAdd(stats + (slot >= 0 ? 0 : 1), 1);
  return (slot >= 0 ? hot_rows + static_cast<size_t>(slot) * vec_per_row : table + static_cast<size_t>(id) * vec_per_row) + c;
}

__global__ void __launch_bounds__(kThreads)
gather_rows_flat_kernel(int max_rows, int V, int vec_per_row, const int32_t* __restrict__ ids,
                        const int32_t* __restrict__ n_ids, const uint4* __restrict__ table,
                        const uint4* __restrict__ hot_rows, const int32_t* __restrict__ hot_slot,
                        uint4* __restrict__ dst, int32_t* status, int32_t* stats) {
  int n = *n_ids;
  if (n > max_rows || n < 0) {
    if (blockIdx.x == 0 && threadIdx.x == 0) report_error(status, STEM_ERR_COUNT_RANGE, n);
    n = n < 0 ? 0 : max_rows;
  }
  const size_t total = static_cast<size_t>(n) * vec_per_row;
  const size_t step = static_cast<size_t>(gridDim.x) * blockDim.x * kFlatBatch;
  size_t base = static_cast<size_t>(blockIdx.x) * blockDim.x * kFlatBatch + threadIdx.x;
  uint4 cur[kFlatBatch], nxt[kFlatBatch];
#pragma unroll
  for (int j = 0; j < kFlatBatch; ++j) {
    const size_t i = base + static_cast<size_t>(j) * blockDim.x;
    if (i < total) cur[j] = *flat_src(i, vec_per_row, V, ids, table, hot_rows, hot_slot, status, stats);
  }
  for (; base < total; base += step) {
    const size_t nb = base + step;
#pragma unroll
    for (int j = 0; j < kFlatBatch; ++j) {
      const size_t i = nb + static_cast<size_t>(j) * blockDim.x;
      if (i < total) nxt[j] = *flat_src(i, vec_per_row, V, ids, table, hot_rows, hot_slot, status, stats);
    }
#pragma unroll
    for (int j = 0; j < kFlatBatch; ++j) {
      const size_t i = base + static_cast<size_t>(j) * blockDim.x;
      if (i < total) dst[i] = cur[j];
    }
#pragma unroll
    for (int j = 0; j < kFlatBatch; ++j) cur[j] = nxt[j];
  }
}

__global__ void __launch_bounds__(kHostLinkThreads)
writeback_rows_kernel(int max_rows, int vec_per_row, const uint4* __restrict__ rows,
                      const int32_t* __restrict__ unique_ids, const int32_t* __restrict__ n_rows,
                      uint4* __restrict__ host_rows, int32_t* __restrict__ host_ids,
                      int32_t* __restrict__ host_n, int32_t* status) {
  int n = *n_rows;
  if (n > max_rows || n < 0) {   // clamped to what the host buffers hold, and reported
    if (blockIdx.x == 0 && threadIdx.x == 0) report_error(status, STEM_ERR_COUNT_RANGE, n);
    n = n < 0 ? 0 : max_rows;
  }
  const size_t total = static_cast<size_t>(n) * vec_per_row;
  const size_t stride = static_cast<size_t>(gridDim.x) * blockDim.x;
  size_t i = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  for (; i + 3 * stride < total; i += 4 * stride) {   // four loads in flight per thread
    const uint4 a0 = rows[i], a1 = rows[i + stride], a2 = rows[i + 2 * stride], a3 = rows[i + 3 * stride];
    host_rows[i] = a0; host_rows[i + stride] = a1; host_rows[i + 2 * stride] = a2; host_rows[i + 3 * stride] = a3;
  }
  for (; i < total; i += stride) host_rows[i] = rows[i];
  for (size_t j = static_cast<size_t>(blockIdx.x) * blockDim.x + threadIdx.x; j < static_cast<size_t>(n); j += stride)
    host_ids[j] = unique_ids[j];
  if (blockIdx.x == 0 && threadIdx.x == 0) *host_n = n;
}

// An SM cannot hold CTAs of two kernels that run under different shared-memory / L1 splits,
// and the contraction kernels need the largest shared-memory split.  Asking for the same
// split here (these kernels use no shared memory themselves) lets their CTAs share an SM
// with a contraction CTA instead of waiting for it, or making it wait.
template <typename Kernel>
cudaError_t prefer_max_shared(Kernel kernel) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
}

}  // namespace

cudaError_t launch_gather_rows(int max_rows, int V, size_t row_bytes, const int32_t* ids,
                               const int32_t* n_ids, const void* table, bool table_on_host,
                               const void* hot_rows, const int32_t* hot_slot, void* dst, int32_t* status,
                               int32_t* stats, cudaStream_t stream) {
  if (max_rows <= 0) return cudaSuccess;
  const int vec = static_cast<int>(row_bytes / 16);
  const int threads = table_on_host ? kHostLinkThreads : kThreads;
  const int lanes_per_row = vec < threads ? vec : threads;
  const int rows_per_cta = threads / lanes_per_row;
  int blocks = (max_rows + rows_per_cta - 1) / rows_per_cta;
  const int cap = table_on_host ? kHostLinkCtas : device_sm_count() * 8;
  if (blocks > cap) blocks = cap;
  if (!table_on_host) {
    // a device table: flat copy, as many CTAs as the largest possible count needs, up to 8 per SM
    const size_t per_cta = static_cast<size_t>(kThreads) * kFlatBatch;
    const size_t need = (static_cast<size_t>(max_rows) * vec + per_cta - 1) / per_cta;
    const int grid = static_cast<int>(need < static_cast<size_t>(device_sm_count()) * 8 ? need : device_sm_count() * 8);
    gather_rows_flat_kernel<<<grid > 0 ? grid : 1, kThreads, 0, stream>>>(
        max_rows, V, vec, ids, n_ids, static_cast<const uint4*>(table), static_cast<const uint4*>(hot_rows), hot_slot,
        static_cast<uint4*>(dst), status, stats);
    count_launches(1);
    return cudaGetLastError();
  }
  static PerDeviceOnce configured;
  if (cudaError_t ce = configured.run([] { return prefer_max_shared(gather_rows_kernel); })) return ce;
  gather_rows_kernel<<<blocks, threads, 0, stream>>>(max_rows, V, vec, ids, n_ids, static_cast<const uint4*>(table),
                                                    static_cast<const uint4*>(hot_rows), hot_slot,
                                                    static_cast<uint4*>(dst), status, stats);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_writeback_rows(int max_rows, size_t row_bytes, const void* rows,
                                  const int32_t* unique_ids, const int32_t* n_rows, void* host_rows,
                                  int32_t* host_ids, int32_t* host_n, int32_t* status, cudaStream_t stream) {
  if (max_rows <= 0) return cudaSuccess;
  const int vec = static_cast<int>(row_bytes / 16);
  const int blocks = kHostLinkCtas;
  static PerDeviceOnce configured;
  if (cudaError_t ce = configured.run([] { return prefer_max_shared(writeback_rows_kernel); })) return ce;
  writeback_rows_kernel<<<blocks, kHostLinkThreads, 0, stream>>>(max_rows, vec, static_cast<const uint4*>(rows), unique_ids,
                                                        n_rows, static_cast<uint4*>(host_rows), host_ids, host_n, status);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace stem
