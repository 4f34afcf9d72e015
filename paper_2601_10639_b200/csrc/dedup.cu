// Token-id deduplication: a stable LSD radix sort of (id, position) pairs, 8 bits per
// pass (a count kernel and a scatter kernel per pass), followed by two kernels that mark
// the head of every run of equal ids and emit the distinct ids, the run offsets and each
// position's slot.  Batches of up to 1024 positions take a one-launch path (rank sort in
// shared memory).  Integer-only: every output has exactly one correct value.
#include <mutex>

#include "stem_internal.h"

namespace stem {
namespace {

constexpr int kRadix = 256;
constexpr int kWarps = 32;              // warps per CTA
constexpr int kCtaThreads = kWarps * 32;
constexpr int kMaxCtas = 64;

// Work split: CTA c owns positions [c * 32 * epw, (c + 1) * 32 * epw), warp w of it the
// w-th run of epw positions.  Few, large CTAs keep the cross-CTA bookkeeping (one digit
// histogram per CTA) small enough for every CTA to re-derive its offsets by itself.
struct Split { int n_ctas, epw; };
__host__ __device__ inline Split make_split(int T) {
  int n_ctas = (T + 1023) / 1024;
  n_ctas = n_ctas < 1 ? 1 : (n_ctas > kMaxCtas ? kMaxCtas : n_ctas);
  const int per_cta = (T + n_ctas - 1) / n_ctas;
  const int epw = ((per_cta + kWarps - 1) / kWarps + 31) / 32 * 32;
  return {n_ctas, epw};
}

// The kernels of one dedup call are launched with programmatic stream serialisation: each
// may be scheduled while its predecessor is still draining, waits here for the predecessor's
// results to be complete and visible, and then lets its own successor be scheduled.  That
// takes most of the launch gaps out of a chain of six few-microsecond kernels.
__device__ __forceinline__ void pdl_wait_then_release() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kernel)(KArgs...), int grid, int block, cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(grid));
  cfg.blockDim = dim3(static_cast<unsigned>(block));
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

__device__ __forceinline__ int clamp_id(int key, int V) { return key < 0 ? 0 : (key >= V ? V - 1 : key); }

// Per-warp digit histograms of this CTA's keys, in shared memory.
__device__ __forceinline__ void warp_histograms(int (*hist)[kRadix], int T, int V, int epw, int shift,
                                                bool first_pass, const int32_t* __restrict__ keys_in,
                                                int32_t* status) {
  const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int i = lane; i < kRadix; i += 32) hist[w][i] = 0;
  __syncwarp();
  const int begin = (blockIdx.x * kWarps + w) * epw, end = min(T, begin + epw);
  for (int i = begin + lane; i < end; i += 32) {
    int key = keys_in[i];
    if (first_pass) {
      if (status != nullptr && (key < 0 || key >= V)) {
        report_error(status, STEM_ERR_ID_RANGE, i);
        atomicAdd(status + 2, 1);
      }
      key = clamp_id(key, V);
    }
    atomicAdd(&hist[w][(key >> shift) & (kRadix - 1)], 1);
  }
}

// cta_hist[c][d] = number of keys of CTA c whose digit at `shift` is d.
__global__ void __launch_bounds__(kCtaThreads)
radix_count_kernel(int T, int V, int epw, int shift, bool first_pass, const int32_t* __restrict__ keys_in,
                   int32_t* __restrict__ cta_hist, int32_t* status) {
  pdl_wait_then_release();
  __shared__ int hist[kWarps][kRadix];
  warp_histograms(hist, T, V, epw, shift, first_pass, keys_in, status);
  __syncthreads();
  if (threadIdx.x < kRadix) {
    int sum = 0;
#pragma unroll 8
    for (int w = 0; w < kWarps; ++w) sum += hist[w][threadIdx.x];
    cta_hist[blockIdx.x * kRadix + threadIdx.x] = sum;
  }
}

// Stable scatter.  Every CTA derives its own output offsets from all CTAs' histograms:
// keys with a smaller digit first, then equal digits of earlier CTAs, then of earlier warps.
__global__ void __launch_bounds__(kCtaThreads)
radix_scatter_kernel(int T, int V, int epw, int shift, bool first_pass, const int32_t* __restrict__ keys_in,
                     const int32_t* __restrict__ vals_in, const int32_t* __restrict__ cta_hist,
                     int32_t* __restrict__ keys_out, int32_t* __restrict__ vals_out) {
  pdl_wait_then_release();
  __shared__ int hist[kWarps][kRadix];
  __shared__ int warp_tot[kRadix / 32];
  warp_histograms(hist, T, V, epw, shift, first_pass, keys_in, nullptr);
  __syncthreads();
  const int w = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int before = 0, total = 0;
  if (threadIdx.x < kRadix) {
    for (int c = 0; c < static_cast<int>(gridDim.x); ++c) {
      const int v = cta_hist[c * kRadix + threadIdx.x];
      total += v;
      if (c < static_cast<int>(blockIdx.x)) before += v;
    }
    int incl = total;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) warp_tot[w] = incl;
    total = incl - total;  // exclusive prefix inside this warp of digits
  }
  __syncthreads();
  if (threadIdx.x < kRadix) {
    int base = total + before;
    for (int ww = 0; ww < w; ++ww) base += warp_tot[ww];
    for (int ww = 0; ww < kWarps; ++ww) {  // turn per-warp counts into per-warp start offsets
      const int cnt = hist[ww][threadIdx.x];
      hist[ww][threadIdx.x] = base;
      base += cnt;
    }
  }
  __syncthreads();
  const int begin = (blockIdx.x * kWarps + w) * epw, end = min(T, begin + epw);
  const unsigned lt_mask = (1u << lane) - 1u;
  for (int i0 = begin; i0 < end; i0 += 32) {
    const int i = i0 + lane;
    const bool valid = i < end;
    int key = 0, val = 0;
    if (valid) {
      key = keys_in[i];
      if (first_pass) { key = clamp_id(key, V); val = i; } else { val = vals_in[i]; }
    }
    const int digit = (key >> shift) & (kRadix - 1);
    const unsigned peers = __match_any_sync(0xffffffffu, valid ? digit : (kRadix + lane));
    const int rank = __popc(peers & lt_mask);
    int dst = 0;
    if (valid) dst = hist[w][digit] + rank;
    __syncwarp();
    if (valid && rank == 0) hist[w][digit] += __popc(peers);
    __syncwarp();
    if (valid) { keys_out[dst] = key; vals_out[dst] = val; }
  }
}

__device__ __forceinline__ bool is_head(const int32_t* __restrict__ sorted_ids, int p) {
  return p == 0 || sorted_ids[p] != sorted_ids[p - 1];
}

// Heads of runs of equal ids, counted per CTA chunk.
__global__ void __launch_bounds__(kCtaThreads)
heads_count_kernel(int T, int per_cta, const int32_t* __restrict__ sorted_ids, int32_t* __restrict__ cta_heads) {
  pdl_wait_then_release();
  const int begin = blockIdx.x * per_cta, end = min(T, begin + per_cta);
  int local = 0;
  for (int p = begin + threadIdx.x; p < end; p += kCtaThreads) local += is_head(sorted_ids, p) ? 1 : 0;
  __shared__ int s_sum;
  if (threadIdx.x == 0) s_sum = 0;
  __syncthreads();
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) local += __shfl_xor_sync(0xffffffffu, local, o);
  if ((threadIdx.x & 31) == 0 && local) atomicAdd(&s_sum, local);
  __syncthreads();
  if (threadIdx.x == 0) cta_heads[blockIdx.x] = s_sum;
}

// unique_ids / seg_offsets at the heads, slot of every position -> inverse.
__global__ void __launch_bounds__(kCtaThreads)
heads_write_kernel(int T, int per_cta, const int32_t* __restrict__ sorted_ids, const int32_t* __restrict__ perm,
                   const int32_t* __restrict__ cta_heads, int32_t* __restrict__ unique_ids,
                   int32_t* __restrict__ n_unique, int32_t* __restrict__ inverse,
                   int32_t* __restrict__ seg_offsets) {
  pdl_wait_then_release();
  __shared__ int warp_sums[kWarps];
  __shared__ int s_before;
  const int tid = threadIdx.x, lane = tid & 31, w = tid >> 5;
  if (w == 0) {
    int v = 0;
    for (int c = lane; c < static_cast<int>(blockIdx.x); c += 32) v += cta_heads[c];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (lane == 0) s_before = v;
  }
  const int cta_begin = blockIdx.x * per_cta, cta_end = min(T, cta_begin + per_cta);
  const int per_thread = (per_cta + kCtaThreads - 1) / kCtaThreads;
  const int begin = min(cta_end, cta_begin + tid * per_thread), end = min(cta_end, begin + per_thread);
  int local = 0;
  for (int p = begin; p < end; ++p) local += is_head(sorted_ids, p) ? 1 : 0;
  int incl = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) warp_sums[w] = incl;
  __syncthreads();
  if (w == 0) {
    int v = warp_sums[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int u = __shfl_up_sync(0xffffffffu, v, o);
      if (lane >= o) v += u;
    }
    warp_sums[lane] = v;
  }
  __syncthreads();
  int heads = s_before + incl - local + (w > 0 ? warp_sums[w - 1] : 0);  // heads before `begin`
  for (int p = begin; p < end; ++p) {
    const int id = sorted_ids[p];
    if (is_head(sorted_ids, p)) {
      unique_ids[heads] = id;
      seg_offsets[heads] = p;
      ++heads;
    }
    if (inverse) inverse[perm[p]] = heads - 1;
  }
  if (blockIdx.x == gridDim.x - 1 && tid == 0) {
    const int total = s_before + warp_sums[kWarps - 1];
    *n_unique = total;
    seg_offsets[total] = T;
  }
}

// A batch of at most kCtaThreads positions (decode steps) in one launch by one CTA: every
// thread ranks its own (id, position) pair against all others in shared memory, which is the
// stable sort; run heads and slots follow from one block-wide scan.  Same outputs as the
// radix path, without its six launch latencies.
__global__ void __launch_bounds__(kCtaThreads)
dedup_small_kernel(int T, int V, const int32_t* __restrict__ ids, int32_t* __restrict__ unique_ids,
                   int32_t* __restrict__ n_unique, int32_t* __restrict__ inverse, int32_t* __restrict__ perm,
                   int32_t* __restrict__ seg_offsets, int32_t* status) {
  __shared__ int s_id[kCtaThreads];       // ids by position, then ids in sorted order
  __shared__ int s_sorted[kCtaThreads];
  __shared__ int s_perm[kCtaThreads];
  __shared__ int s_warp[kWarps];
  const int t = threadIdx.x, lane = t & 31, w = t >> 5;
  int id = 0x7fffffff;
  if (t < T) {
    id = ids[t];
    if (id < 0 || id >= V) {
      if (status != nullptr) { report_error(status, STEM_ERR_ID_RANGE, t); atomicAdd(status + 2, 1); }
      id = clamp_id(id, V);
    }
  }
  s_id[t] = id;
  __syncthreads();
  if (t < T) {
    int rank = 0;
    for (int j = 0; j < T; ++j) {
      const int other = s_id[j];
      rank += (other < id || (other == id && j < t)) ? 1 : 0;
    }
    s_sorted[rank] = id;
    s_perm[rank] = t;
  }
  __syncthreads();
  // thread t now owns sorted position t
  const bool head = t < T && (t == 0 || s_sorted[t] != s_sorted[t - 1]);
  int incl = head ? 1 : 0;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  if (lane == 31) s_warp[w] = incl;
  __syncthreads();
  if (w == 0) {
    int v = s_warp[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int u = __shfl_up_sync(0xffffffffu, v, o);
      if (lane >= o) v += u;
    }
    s_warp[lane] = v;
  }
  __syncthreads();
  const int slot = incl + (w > 0 ? s_warp[w - 1] : 0) - 1;   // slot of sorted position t
  if (t < T) {
    perm[t] = s_perm[t];
    if (head) { unique_ids[slot] = s_sorted[t]; seg_offsets[slot] = t; }
    if (inverse) inverse[s_perm[t]] = slot;
  }
  if (t == 0) {
    const int total = s_warp[kWarps - 1];
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
  // two key buffers, two value buffers, per-CTA digit histograms, per-CTA head counts
  return 4 * align_up(static_cast<size_t>(T) * 4, 256) + static_cast<size_t>(kMaxCtas) * kRadix * 4 + 256;
}

// Stable LSD radix sort of n keys in [0, V): perm = positions in sorted order; *sorted_keys
// points at the sorted keys (inside scratch).  scratch: dedup_workspace_bytes(n, V) bytes.
cudaError_t launch_stable_sort(int n, int V, const int32_t* keys_in, int32_t* perm, void* scratch,
                               const int32_t** sorted_keys, int32_t* status, cudaStream_t stream) {
  const Split sp = make_split(n);
  const size_t tb = align_up(static_cast<size_t>(n) * 4, 256);
  char* p = static_cast<char*>(scratch);
  int32_t* keys[2] = {reinterpret_cast<int32_t*>(p), reinterpret_cast<int32_t*>(p + tb)};
  int32_t* vals[2] = {reinterpret_cast<int32_t*>(p + 2 * tb), reinterpret_cast<int32_t*>(p + 3 * tb)};
  int32_t* cta_hist = reinterpret_cast<int32_t*>(p + 4 * tb);
  const int passes = (key_bits(V) + 7) / 8;
  const int32_t* kin = keys_in;
  const int32_t* vin = nullptr;
  for (int pass = 0; pass < passes; ++pass) {
    const bool first = pass == 0, last = pass == passes - 1;
    int32_t* kout = keys[pass & 1];
    int32_t* vout = last ? perm : vals[pass & 1];
    cudaError_t e = launch_chained(radix_count_kernel, sp.n_ctas, kCtaThreads, stream, n, V, sp.epw, pass * 8, first,
                                   kin, cta_hist, status);
    if (e != cudaSuccess) return e;
    e = launch_chained(radix_scatter_kernel, sp.n_ctas, kCtaThreads, stream, n, V, sp.epw, pass * 8, first, kin, vin,
                       static_cast<const int32_t*>(cta_hist), kout, vout);
    if (e != cudaSuccess) return e;
    count_launches(2);
    kin = kout;
    vin = vout;
  }
  *sorted_keys = kin;
  return cudaSuccess;
}

cudaError_t launch_dedup(int T, int V, const int32_t* ids, int32_t* unique_ids, int32_t* n_unique,
                         int32_t* inverse, int32_t* perm, int32_t* seg_offsets, void* scratch,
                         int32_t* status, cudaStream_t stream) {
  if (T <= 0) {
    empty_dedup_kernel<<<1, 1, 0, stream>>>(n_unique, seg_offsets);
    count_launches(1);
    return cudaGetLastError();
  }
  if (T <= kCtaThreads) {
    dedup_small_kernel<<<1, kCtaThreads, 0, stream>>>(T, V, ids, unique_ids, n_unique, inverse, perm, seg_offsets,
                                                    status);
    count_launches(1);
    return cudaGetLastError();
  }
  const Split sp = make_split(T);
  const size_t tb = align_up(static_cast<size_t>(T) * 4, 256);
  int32_t* cta_heads = reinterpret_cast<int32_t*>(static_cast<char*>(scratch) + 4 * tb) + kMaxCtas * kRadix;
  const int32_t* kin = nullptr;
  if (cudaError_t e = launch_stable_sort(T, V, ids, perm, scratch, &kin, status, stream)) return e;
  const int per_cta = sp.epw * kWarps;
  cudaError_t e = launch_chained(heads_count_kernel, sp.n_ctas, kCtaThreads, stream, T, per_cta, kin, cta_heads);
  if (e != cudaSuccess) return e;
  e = launch_chained(heads_write_kernel, sp.n_ctas, kCtaThreads, stream, T, per_cta, kin,
                     static_cast<const int32_t*>(perm), static_cast<const int32_t*>(cta_heads), unique_ids, n_unique,
                     inverse, seg_offsets);
  count_launches(2);
  return e != cudaSuccess ? e : cudaGetLastError();
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
constexpr size_t kStaticScratchBytes = 1310720;  // 1.25 MiB >= dedup_workspace_bytes(kStaticMaxT, .)
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
