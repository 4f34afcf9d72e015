// Token-id deduplication: a stable LSD radix sort of (id, position) pairs, 8 bits per
// pass, followed by one pass that marks the head of every run of equal ids and emits the
// distinct ids, the run offsets and each position's slot.  Integer-only: every output has
// exactly one correct value.
#include <mutex>

#include "stem_internal.h"

namespace stem {
namespace {

constexpr int kRadix = 256;
constexpr int kWarpsPerBlock = 8;

__host__ __device__ inline int elems_per_warp(int T) { return T <= (1 << 16) ? 256 : 2048; }

// Each warp owns a contiguous run of positions; counts[digit * n_warps + warp] = how many
// of its keys carry `digit` at `shift`.
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
radix_count_kernel(int T, int V, int epw, int n_warps, int shift, bool first_pass,
                   const int32_t* __restrict__ keys_in, int32_t* __restrict__ counts,
                   int32_t* status) {
  __shared__ int hist[kWarpsPerBlock][kRadix];
  const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int i = lane; i < kRadix; i += 32) hist[w][i] = 0;
  __syncwarp();
  const int gw = blockIdx.x * kWarpsPerBlock + w;
  if (gw < n_warps) {
    const int begin = gw * epw, end = min(T, begin + epw);
    for (int i = begin + lane; i < end; i += 32) {
      int key = keys_in[i];
      if (first_pass && (key < 0 || key >= V)) {
        if (status) { report_error(status, STEM_ERR_ID_RANGE, i); atomicAdd(status + 2, 1); }
        key = key < 0 ? 0 : V - 1;
      }
      atomicAdd(&hist[w][(key >> shift) & (kRadix - 1)], 1);
    }
    __syncwarp();
    for (int d = lane; d < kRadix; d += 32) counts[d * n_warps + gw] = hist[w][d];
  }
}

// Exclusive prefix sum of n ints in place, one block.
__global__ void __launch_bounds__(1024) scan_exclusive_kernel(int32_t* data, int n) {
  __shared__ int warp_sums[32];
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  const int per = (n + 1023) / 1024;
  const int begin = min(n, tid * per), end = min(n, begin + per);
  int local = 0;
  for (int i = begin; i < end; ++i) local += data[i];
  int incl = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) warp_sums[w] = incl;
  __syncthreads();
  if (w == 0) {
    int s = warp_sums[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, s, o);
      if (lane >= o) s += v;
    }
    warp_sums[lane] = s;
  }
  __syncthreads();
  int run = incl - local + (w > 0 ? warp_sums[w - 1] : 0);
  for (int i = begin; i < end; ++i) {
    const int v = data[i];
    data[i] = run;
    run += v;
  }
}

// Stable scatter: within a warp's run, keys with the same digit keep their order.
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
radix_scatter_kernel(int T, int V, int epw, int n_warps, int shift, bool first_pass,
                     const int32_t* __restrict__ keys_in, const int32_t* __restrict__ vals_in,
                     const int32_t* __restrict__ offsets, int32_t* __restrict__ keys_out,
                     int32_t* __restrict__ vals_out) {
  __shared__ int base[kWarpsPerBlock][kRadix];
  const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int gw = blockIdx.x * kWarpsPerBlock + w;
  if (gw >= n_warps) return;
  for (int d = lane; d < kRadix; d += 32) base[w][d] = offsets[d * n_warps + gw];
  __syncwarp();
  const int begin = gw * epw, end = min(T, begin + epw);
  const unsigned lt_mask = (1u << lane) - 1u;
  for (int i0 = begin; i0 < end; i0 += 32) {
    const int i = i0 + lane;
    const bool valid = i < end;
    int key = 0, val = 0;
    if (valid) {
      key = keys_in[i];
      if (first_pass) {
        key = key < 0 ? 0 : (key >= V ? V - 1 : key);
        val = i;
      } else {
        val = vals_in[i];
      }
    }
    const int digit = (key >> shift) & (kRadix - 1);
    const unsigned peers = __match_any_sync(0xffffffffu, valid ? digit : (kRadix + lane));
    const int rank = __popc(peers & lt_mask);
    int dst = 0;
    if (valid) dst = base[w][digit] + rank;
    __syncwarp();
    if (valid && rank == 0) base[w][digit] += __popc(peers);
    __syncwarp();
    if (valid) {
      keys_out[dst] = key;
      vals_out[dst] = val;
    }
  }
}

// One block walks the sorted ids: heads of runs -> unique_ids / seg_offsets, slot of every
// position -> inverse.
__global__ void __launch_bounds__(1024)
segment_heads_kernel(int T, const int32_t* __restrict__ sorted_ids, const int32_t* __restrict__ perm,
                     int32_t* __restrict__ unique_ids, int32_t* __restrict__ n_unique,
                     int32_t* __restrict__ inverse, int32_t* __restrict__ seg_offsets) {
  __shared__ int warp_sums[32];
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  const int per = (T + 1023) / 1024;
  const int begin = min(T, tid * per), end = min(T, begin + per);
  int local = 0;
  for (int p = begin; p < end; ++p)
    local += (p == 0 || sorted_ids[p] != sorted_ids[p - 1]) ? 1 : 0;
  int incl = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) warp_sums[w] = incl;
  __syncthreads();
  if (w == 0) {
    int s = warp_sums[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, s, o);
      if (lane >= o) s += v;
    }
    warp_sums[lane] = s;
  }
  __syncthreads();
  int heads_before = incl - local + (w > 0 ? warp_sums[w - 1] : 0);
  for (int p = begin; p < end; ++p) {
    const int id = sorted_ids[p];
    if (p == 0 || id != sorted_ids[p - 1]) {
      unique_ids[heads_before] = id;
      seg_offsets[heads_before] = p;
      ++heads_before;
    }
    if (inverse) inverse[perm[p]] = heads_before - 1;
  }
  if (tid == 1023) {
    const int total = warp_sums[31];
    *n_unique = total;
    seg_offsets[total] = T;
  }
}

__global__ void empty_dedup_kernel(int32_t* n_unique, int32_t* seg_offsets) {
  *n_unique = 0;
  seg_offsets[0] = 0;
}

int key_bits(int V) {
  int bits = 1;
  while (bits < 31 && (1ll << bits) < static_cast<long long>(V)) ++bits;
  return bits;
}

}  // namespace

size_t dedup_workspace_bytes(int T, int V) {
  (void)V;
  if (T <= 0) return 0;
  const int epw = elems_per_warp(T);
  const int n_warps = (T + epw - 1) / epw;
  // two key buffers, two value buffers, the digit counts
  return 4 * align_up(static_cast<size_t>(T) * 4, 256) + align_up(static_cast<size_t>(n_warps) * kRadix * 4, 256);
}

cudaError_t launch_dedup(int T, int V, const int32_t* ids, int32_t* unique_ids, int32_t* n_unique,
                         int32_t* inverse, int32_t* perm, int32_t* seg_offsets, void* scratch,
                         int32_t* status, cudaStream_t stream) {
  if (T <= 0) {
    empty_dedup_kernel<<<1, 1, 0, stream>>>(n_unique, seg_offsets);
    count_launches(1);
    return cudaGetLastError();
  }
  const int epw = elems_per_warp(T);
  const int n_warps = (T + epw - 1) / epw;
  const size_t tb = align_up(static_cast<size_t>(T) * 4, 256);
  char* p = static_cast<char*>(scratch);
  int32_t* keys[2] = {reinterpret_cast<int32_t*>(p), reinterpret_cast<int32_t*>(p + tb)};
  int32_t* vals[2] = {reinterpret_cast<int32_t*>(p + 2 * tb), reinterpret_cast<int32_t*>(p + 3 * tb)};
  int32_t* counts = reinterpret_cast<int32_t*>(p + 4 * tb);

  const int passes = (key_bits(V) + 7) / 8;
  const int blocks = (n_warps + kWarpsPerBlock - 1) / kWarpsPerBlock;
  const int32_t* kin = ids;
  const int32_t* vin = nullptr;
  for (int pass = 0; pass < passes; ++pass) {
    const bool first = pass == 0, last = pass == passes - 1;
    int32_t* kout = keys[pass & 1];
    int32_t* vout = last ? perm : vals[pass & 1];
    radix_count_kernel<<<blocks, kWarpsPerBlock * 32, 0, stream>>>(T, V, epw, n_warps, pass * 8, first,
                                                                  kin, counts, status);
    scan_exclusive_kernel<<<1, 1024, 0, stream>>>(counts, n_warps * kRadix);
    radix_scatter_kernel<<<blocks, kWarpsPerBlock * 32, 0, stream>>>(T, V, epw, n_warps, pass * 8, first,
                                                                    kin, vin, counts, kout, vout);
    count_launches(3);
    kin = kout;
    vin = vout;
  }
  segment_heads_kernel<<<1, 1024, 0, stream>>>(T, kin, perm, unique_ids, n_unique, inverse, seg_offsets);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace stem

// ---- dedup without a caller workspace ---------------------------------------------------
// Some callers cannot hand the library scratch memory because they cannot allocate any:
// a serving process whose framework reserved all of HBM at start-up for weights and KV
// cache, a plug-in that runs inside another runtime's stream callback, or a latency-bound
// loop where a cudaMalloc would synchronise the whole device.  For them the radix sort's
// ping-pong buffers and digit counts live in this fixed array, which every GPU that loads
// the library holds until the process exits (1.25 MiB).
namespace stem {
namespace {

constexpr int kStaticMaxT = 65536;
constexpr size_t kStaticScratchBytes = 4 * static_cast<size_t>(kStaticMaxT) * 4 +
                                       static_cast<size_t>(kStaticMaxT / 256) * kRadix * 4;
static __device__ __align__(256) unsigned char g_dedup_scratch[kStaticScratchBytes];

// The array's name is only a host-side handle; kernels need its device address, which
// differs per device and is looked up once per device.
std::mutex g_static_mutex;
void* g_static_ptr[64] = {nullptr};

cudaError_t static_scratch_address(void** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (g_static_ptr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_dedup_scratch);
    if (e != cudaSuccess) return e;
    g_static_ptr[dev] = p;
  }
  *out = g_static_ptr[dev];
  return cudaSuccess;
}

}  // namespace
}  // namespace stem

extern "C" int stem_dedup_ids_static(const stem_shape_t* shape, const int32_t* ids, int32_t* unique_ids,
                                     int32_t* n_unique, int32_t* inverse, int32_t* perm,
                                     int32_t* seg_offsets, int32_t* status, void* stream) {
  using namespace stem;
  if (!shape || shape->T < 0 || shape->V <= 0 || shape->V > (1 << 30)) return STEM_ERR_INVALID_ARG;
  if (shape->T > kStaticMaxT) return STEM_ERR_STATIC_LIMIT;
  if (!unique_ids || !n_unique || !perm || !seg_offsets || (shape->T > 0 && !ids)) return STEM_ERR_INVALID_ARG;
  if (dedup_workspace_bytes(shape->T, shape->V) > kStaticScratchBytes) return STEM_ERR_STATIC_LIMIT;
  void* scratch = nullptr;
  if (static_scratch_address(&scratch) != cudaSuccess) { cudaGetLastError(); return STEM_ERR_CUDA; }
  // Nothing in the scratch has to start at zero: every pass writes each digit count and each
  // key/value slot it later reads, so whatever the previous call left behind is overwritten.
  cudaError_t e = launch_dedup(shape->T, shape->V, ids, unique_ids, n_unique, inverse, perm, seg_offsets,
                               scratch, status, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? STEM_OK : STEM_ERR_CUDA;
}

extern "C" int stem_dedup_static_max_tokens(void) { return stem::kStaticMaxT; }
