// Frequency-ranked row cache for decoding with an off-device table (paper Section 3.4: a
// memory-efficient LFU cache over Zipfian token ids; Section 3.2.4: cached in the memory the
// removed up-projection frees).
//
// State, all caller-owned device memory: freq[V] (lookups seen per id), hot_slot[V] (slot of
// each id in the cache, -1 = not cached), hot_ids[K] (id held by each slot, -1 = empty),
// hot_rows[K, d_ff] (copies of table rows).  Two operations:
//   touch    count the lookups of one decode step, and how many of them the cache serves
//   refresh  make the cache hold the K most frequently looked-up ids seen so far (ties go to
//            the smaller id; ids never seen are not cached): ids that dropped out give up
//            their slots, ids that came in take them and have their rows copied from the
//            table over the host link.  The set is exact (least-frequently-used eviction in
//            batch form); which slot an id lands in is arbitrary.
// Integer work plus row copies; no floating point.
#include "stem_internal.h"

namespace stem {
namespace {

constexpr int kThreads = 256;
constexpr int kCopyCtas = 32;      // row copies cross the host link: same sizing as the prefetch
constexpr int kCopyThreads = 128;
constexpr int kKeyMax = 0x7ffffffe;

__global__ void __launch_bounds__(kThreads)
lfu_touch_kernel(int n, int V, const int32_t* __restrict__ ids, int32_t* freq,
                 const int32_t* __restrict__ hot_slot, int32_t* stats, int32_t* status) {
  int hits = 0, misses = 0;
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) {
    int id = ids[i];
    if (id < 0 || id >= V) {
      report_error(status, STEM_ERR_ID_RANGE, i);
      id = id < 0 ? 0 : V - 1;
    }
    atomicAdd(freq + id, 1);
    if (hot_slot[id] >= 0) ++hits; else ++misses;
  }
  if (stats != nullptr) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      hits += __shfl_xor_sync(0xffffffffu, hits, o);
      misses += __shfl_xor_sync(0xffffffffu, misses, o);
    }
    if ((threadIdx.x & 31) == 0) {
      if (hits) atomicAdd(stats, hits);
      if (misses) atomicAdd(stats + 1, misses);
    }
  }
}

// Sort key: ascending key = descending frequency; the stable sort breaks ties by id.
__global__ void __launch_bounds__(kThreads)
lfu_keys_kernel(int V, const int32_t* __restrict__ freq, int32_t* __restrict__ keys) {
  for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < V; i += gridDim.x * blockDim.x) {
    const int f = freq[i];
    keys[i] = kKeyMax - (f < 0 ? 0 : (f > kKeyMax ? kKeyMax : f));
  }
}

// in_new[id] = 1 for the ids that belong in the cache: the first K of the ranking, if seen.
__global__ void __launch_bounds__(kThreads)
lfu_mark_kernel(int K, const int32_t* __restrict__ ranking, const int32_t* __restrict__ freq,
                uint8_t* __restrict__ in_new) {
  for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < K; j += gridDim.x * blockDim.x) {
    const int id = ranking[j];
    if (freq[id] > 0) in_new[id] = 1;
  }
}

// Slots that are empty or whose id dropped out become free (and the id loses its slot); ids
// that belong in the cache and have no slot are listed as entering.  counts: [n_free, n_enter].
__global__ void __launch_bounds__(kThreads)
lfu_lists_kernel(int K, const int32_t* __restrict__ ranking, const uint8_t* __restrict__ in_new,
                 int32_t* hot_slot, int32_t* hot_ids, int32_t* free_slots, int32_t* entering,
                 int32_t* counts) {
  for (int j = blockIdx.x * blockDim.x + threadIdx.x; j < K; j += gridDim.x * blockDim.x) {
    const int held = hot_ids[j];
    if (held < 0 || !in_new[held]) {
      free_slots[atomicAdd(counts, 1)] = j;
      if (held >= 0) { hot_slot[held] = -1; hot_ids[j] = -1; }
    }
    // ids leaving (not in_new) and ids entering (in_new) are disjoint, so reading hot_slot of
    // an entering id does not race with the write above
    const int id = ranking[j];
    if (in_new[id] && hot_slot[id] < 0) entering[atomicAdd(counts + 1, 1)] = id;
  }
}

// Entering id i takes free slot i; its row is copied from the table (host memory: 16-byte
// loads across the host link, eight in flight per thread).
__global__ void __launch_bounds__(kCopyThreads)
lfu_install_kernel(int K, int vec_per_row, const int32_t* __restrict__ counts, const int32_t* __restrict__ free_slots,
                   const int32_t* __restrict__ entering, const uint4* __restrict__ table,
                   int32_t* hot_slot, int32_t* hot_ids, uint4* __restrict__ hot_rows, int32_t* n_installed) {
  // never more than counts[0] (the cache has K slots and the new set at most K ids); bounded all
  // the same, so that no count can carry a copy past the K rows of the cache
  const int n = min(min(counts[1], counts[0]), K);
  if (blockIdx.x == 0 && threadIdx.x == 0 && n_installed != nullptr) *n_installed = n;
  for (int i = blockIdx.x; i < n; i += gridDim.x) {
    const int slot = free_slots[i], id = entering[i];
    if (threadIdx.x == 0) { hot_slot[id] = slot; hot_ids[slot] = id; }
    const uint4* src = table + static_cast<size_t>(id) * vec_per_row;
    uint4* dst = hot_rows + static_cast<size_t>(slot) * vec_per_row;
    int c = threadIdx.x;
    for (; c + 7 * kCopyThreads < vec_per_row; c += 8 * kCopyThreads) {
      uint4 a[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) a[j] = src[c + j * kCopyThreads];
#pragma unroll
      for (int j = 0; j < 8; ++j) dst[c + j * kCopyThreads] = a[j];
    }
    for (; c < vec_per_row; c += kCopyThreads) dst[c] = src[c];
  }
}

size_t lfu_offsets(int V, int K, size_t* keys, size_t* ranking, size_t* in_new, size_t* lists, size_t* counts) {
  size_t o = 0;
  *keys = o;    o += align_up(static_cast<size_t>(V) * 4, 256);
  *ranking = o; o += align_up(static_cast<size_t>(V) * 4, 256);
  *in_new = o;  o += align_up(static_cast<size_t>(V), 256);
  *lists = o;   o += 2 * align_up(static_cast<size_t>(K) * 4, 256);
  *counts = o;  o += 256;
  return o;     // the sort's own scratch follows
}

}  // namespace

size_t lfu_workspace_bytes(int V, int K) {
  size_t a, b, c, d, e;
  return lfu_offsets(V, K, &a, &b, &c, &d, &e) + dedup_workspace_bytes(V, 0x7fffffff);
}

cudaError_t launch_lfu_touch(int n, int V, const int32_t* ids, int32_t* freq, const int32_t* hot_slot,
                             int32_t* stats, int32_t* status, cudaStream_t stream) {
  if (n <= 0) return cudaSuccess;
  const int blocks = (n + kThreads - 1) / kThreads < 64 ? (n + kThreads - 1) / kThreads : 64;
  lfu_touch_kernel<<<blocks, kThreads, 0, stream>>>(n, V, ids, freq, hot_slot, stats, status);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_lfu_refresh(int V, int K, size_t row_bytes, const int32_t* freq, int32_t* hot_slot,
                               int32_t* hot_ids, void* hot_rows, const void* table, int32_t* n_installed,
                               void* scratch, cudaStream_t stream) {
  size_t o_keys, o_rank, o_new, o_lists, o_counts;
  const size_t o_sort = lfu_offsets(V, K, &o_keys, &o_rank, &o_new, &o_lists, &o_counts);
  char* p = static_cast<char*>(scratch);
  int32_t* keys = reinterpret_cast<int32_t*>(p + o_keys);
  int32_t* ranking = reinterpret_cast<int32_t*>(p + o_rank);
  uint8_t* in_new = reinterpret_cast<uint8_t*>(p + o_new);
  int32_t* free_slots = reinterpret_cast<int32_t*>(p + o_lists);
  int32_t* entering = free_slots + align_up(static_cast<size_t>(K) * 4, 256) / 4;
  int32_t* counts = reinterpret_cast<int32_t*>(p + o_counts);
  const int vblocks = (V + kThreads - 1) / kThreads < 128 ? (V + kThreads - 1) / kThreads : 128;
  const int kblocks = (K + kThreads - 1) / kThreads < 128 ? (K + kThreads - 1) / kThreads : 128;
  cudaError_t e = cudaMemsetAsync(in_new, 0, static_cast<size_t>(V), stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(counts, 0, 8, stream);
  if (e != cudaSuccess) return e;
  lfu_keys_kernel<<<vblocks, kThreads, 0, stream>>>(V, freq, keys);
  const int32_t* sorted_keys = nullptr;
  e = launch_stable_sort(V, 0x7fffffff, keys, ranking, p + o_sort, &sorted_keys, nullptr, stream);
  if (e != cudaSuccess) return e;
  lfu_mark_kernel<<<kblocks, kThreads, 0, stream>>>(K, ranking, freq, in_new);
  lfu_lists_kernel<<<kblocks, kThreads, 0, stream>>>(K, ranking, in_new, hot_slot, hot_ids, free_slots, entering, counts);
  lfu_install_kernel<<<kCopyCtas, kCopyThreads, 0, stream>>>(
      K, static_cast<int>(row_bytes / 16), counts, free_slots, entering, static_cast<const uint4*>(table), hot_slot,
      hot_ids, static_cast<uint4*>(hot_rows), n_installed);
  count_launches(4);
  return cudaGetLastError();
}

}  // namespace stem
