// Table-gradient reduce: dE_rows[r,:] = sum over the positions p of segment r of
// dU[perm[p],:], in a fixed order, without floating-point atomics.
//
// The sorted position range [0,T) is cut into blocks of at most kSegBlk positions.  One CTA per
// (block, column slab) walks its positions in order, accumulating in fp32 registers.  A run
// whose segment lies wholly inside the block is final and is written to dE_rows; a run whose
// segment crosses a block edge (at most the first and the last run of a block) goes to a
// partial row.  The CTAs that hold parts of such a segment count themselves off on an
// integer counter; the one that arrives last adds the segment's partial rows in block order
// and writes the row.  Which CTA that is varies from run to run, the order of the additions
// does not, so the result is bitwise reproducible.  One launch; HBM-bound: every dU row is
// read once with 16-byte loads, coalesced along d_ff.
#include "stem_internal.h"

namespace stem {
namespace {

constexpr int kSegBlk = 64;     // most sorted positions per CTA (the launch picks blk_len <= kSegBlk)
constexpr int kCtasPerSm = 7;   // register budget the kernel is compiled for
constexpr int kThreads = 128;   // pass 1: one thread per vector of columns
constexpr int kBatch = 8;       // rows requested before the first is consumed

template <typename T> struct Vec;
template <> struct Vec<float> {
  static constexpr int N = 4;
  __device__ static uint4 load_raw(const float* p) { return __ldg(reinterpret_cast<const uint4*>(p)); }
  __device__ static void add(float* acc, const uint4& q) {
    acc[0] += __uint_as_float(q.x); acc[1] += __uint_as_float(q.y);
    acc[2] += __uint_as_float(q.z); acc[3] += __uint_as_float(q.w);
  }
  __device__ static void store(float* p, const float* v) {
    *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  }
};
template <> struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static uint4 load_raw(const __nv_bfloat16* p) { return __ldg(reinterpret_cast<const uint4*>(p)); }
  __device__ static void add(float* acc, const uint4& q) {
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      acc[2 * i] += __uint_as_float(w[i] << 16);
      acc[2 * i + 1] += __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
  __device__ static void store(__nv_bfloat16* p, const float* v) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
      w[i] = *reinterpret_cast<const uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  }
};

// A thread owns VI consecutive columns; rows are written in the output type's vectors.
template <int VI, typename TOut>
__device__ __forceinline__ void store_row(TOut* dst, const float (&v)[VI]) {
#pragma unroll
  for (int i = 0; i < VI; i += Vec<TOut>::N) Vec<TOut>::store(dst + i, v + i);
}

// Scratch layout: arrival counters [n_blk][n_slabs] (one per block in which a crossing
// segment can start, per column slab; zeroed before each launch), then 2 partial rows per
// block.
__host__ __device__ inline size_t partial_offset_bytes(int n_blk, int n_slabs) {
  return (static_cast<size_t>(n_blk) * n_slabs * 4 + 255) / 256 * 256;
}

template <typename TIn, typename TOut>
__global__ void __launch_bounds__(kThreads, kCtasPerSm)
segreduce_kernel(int T, int F, int blk_len, const TIn* __restrict__ dU, const int32_t* __restrict__ perm,
                 const int32_t* __restrict__ seg_offsets, const int32_t* __restrict__ n_unique,
                 TOut* __restrict__ dE_rows, int32_t* __restrict__ counters, float* partial) {
  constexpr int VI = (Vec<TIn>::N > Vec<TOut>::N) ? Vec<TIn>::N : Vec<TOut>::N;
  constexpr int LD = VI / Vec<TIn>::N;  // 16-byte loads per row per thread
  __shared__ int s_off[kSegBlk + 1];    // offsets of the segments that can touch this block
  __shared__ int s_row[kSegBlk];
  __shared__ int s_loc[kSegBlk];        // position -> index into s_off
  __shared__ int s_finish[2];           // crossing segments this CTA must finish (index into s_off), or -1
  const int blk = blockIdx.x;
  const int p0 = blk * blk_len;
  const int cnt = min(blk_len, T - p0);
  const int n_u = *n_unique;

  // r_first = largest r with seg_offsets[r] <= p0, found with kThreads pivots per round
  // (two rounds for a few thousand segments instead of a dozen dependent loads).
  int lo = 0, hi = n_u;  // seg_offsets[lo] <= p0 < seg_offsets[hi]
  while (hi - lo > 1) {
    const int step = (hi - lo + kThreads) / (kThreads + 1);
    const int piv = lo + (static_cast<int>(threadIdx.x) + 1) * step;
    const int hit = (piv < hi && seg_offsets[piv] <= p0) ? 1 : 0;
    const int n_hit = __syncthreads_count(hit);
    const int new_lo = lo + n_hit * step;
    hi = min(hi, new_lo + step);
    lo = new_lo;
  }
  const int r_first = lo;
  if (threadIdx.x <= kSegBlk) {
    const int r = r_first + threadIdx.x;
    s_off[threadIdx.x] = r <= n_u ? seg_offsets[r] : 0x7fffffff;
  }
  if (threadIdx.x < cnt) s_row[threadIdx.x] = perm[p0 + threadIdx.x];
  __syncthreads();
  if (threadIdx.x < cnt) {
    const int p = p0 + threadIdx.x;
    int a = 0, b = kSegBlk;  // s_off[a] <= p; at most kSegBlk segments start inside the block
    while (b - a > 1) {
      const int mid = (a + b) >> 1;
      if (s_off[mid] <= p) a = mid; else b = mid;
    }
    if (s_off[b] <= p) a = b;
    s_loc[threadIdx.x] = a;
  }
  __syncthreads();
  const int col = (blockIdx.y * kThreads + threadIdx.x) * VI;
  const bool col_ok = col < F;

  float acc[VI];
#pragma unroll
  for (int i = 0; i < VI; ++i) acc[i] = 0.0f;
  bool first_run = true;
  for (int b0 = 0; col_ok && b0 < cnt; b0 += kBatch) {
    uint4 raw[kBatch][LD];
#pragma unroll
    for (int j = 0; j < kBatch; ++j) {
      if (b0 + j < cnt) {
        const TIn* src = dU + static_cast<size_t>(s_row[b0 + j]) * F + col;
#pragma unroll
        for (int i = 0; i < LD; ++i) raw[j][i] = Vec<TIn>::load_raw(src + i * Vec<TIn>::N);
      }
    }
#pragma unroll
    for (int j = 0; j < kBatch; ++j) {
      const int q = b0 + j;
      if (q < cnt) {
#pragma unroll
        for (int i = 0; i < LD; ++i) Vec<TIn>::add(acc + i * Vec<TIn>::N, raw[j][i]);
        const int loc = s_loc[q];
        const bool run_ends = (q + 1 == cnt) || (s_loc[q + 1] != loc);
        if (run_ends) {
          const bool whole = s_off[loc] >= p0 && s_off[loc + 1] <= p0 + blk_len;
          if (whole) {
            store_row<VI, TOut>(dE_rows + static_cast<size_t>(r_first + loc) * F + col, acc);
          } else {
            store_row<VI, float>(partial + static_cast<size_t>(2 * blk + (first_run ? 0 : 1)) * F + col, acc);
          }
#pragma unroll
          for (int i = 0; i < VI; ++i) acc[i] = 0.0f;
          first_run = false;
        }
      }
    }
  }

  // ---- crossing segments: the last CTA to arrive adds the parts ----------------------------
  // At most two per block: the segment of the first position (if it began earlier or runs on)
  // and that of the last position (if it runs on).  s_off[0] <= p0, so index 0 is the first.
  __threadfence();   // this CTA's partial rows are visible before it counts itself off
  __syncthreads();
  if (threadIdx.x == 0) {
    const int n_slabs = gridDim.y;
    const int j_first = 0, j_last = s_loc[cnt - 1];
    for (int which = 0; which < 2; ++which) {
      const int j = which == 0 ? j_first : j_last;
      int fin = -1;
      const bool whole = s_off[j] >= p0 && s_off[j + 1] <= p0 + blk_len;
      if (!whole && !(which == 1 && j_last == j_first)) {
        const int start_blk = s_off[j] / blk_len, last_blk = (s_off[j + 1] - 1) / blk_len;
        const int old = atomicAdd(&counters[start_blk * n_slabs + blockIdx.y], 1);
        if (old == last_blk - start_blk) fin = j;
      }
      s_finish[which] = fin;
    }
  }
  __syncthreads();
#pragma unroll
  for (int which = 0; which < 2; ++which) {
    const int j = s_finish[which];
    if (j < 0 || !col_ok) continue;
    __threadfence();   // the other CTAs' partial rows, published before their count, are visible
    const int seg_begin = s_off[j], seg_end = s_off[j + 1];
    const int start_blk = seg_begin / blk_len, last_blk = (seg_end - 1) / blk_len;
#pragma unroll
    for (int i = 0; i < VI; ++i) acc[i] = 0.0f;
    for (int b = start_blk; b <= last_blk; ++b) {
      // the segment's run is the first run of block b, unless b is the block it starts in
      // and it does not start at that block's first position
      const int slot = (b > start_blk || seg_begin == start_blk * blk_len) ? 2 * b : 2 * b + 1;
      const float* src = partial + static_cast<size_t>(slot) * F + col;
#pragma unroll
      for (int i = 0; i < VI; i += 4) {
        const float4 q = __ldcg(reinterpret_cast<const float4*>(src + i));
        acc[i] += q.x; acc[i + 1] += q.y; acc[i + 2] += q.z; acc[i + 3] += q.w;
      }
    }
    store_row<VI, TOut>(dE_rows + static_cast<size_t>(r_first + j) * F + col, acc);
  }
}

template <typename TIn, typename TOut>
cudaError_t launch_typed(int T, int F, const void* dU, const int32_t* perm, const int32_t* seg_offsets,
                         const int32_t* n_unique, void* dE_rows, void* scratch, cudaStream_t stream) {
  constexpr int VI = (Vec<TIn>::N > Vec<TOut>::N) ? Vec<TIn>::N : Vec<TOut>::N;
  const int n_slabs = (F + kThreads * VI - 1) / (kThreads * VI);
  // Block length: as long as allowed, then shortened so that the CTAs fill a whole number of
  // waves of the resident CTA slots (a ragged last wave of full-length blocks costs more than
  // evenly shorter blocks).
  static int ctas_per_sm = 0;
  if (ctas_per_sm == 0) {
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, segreduce_kernel<TIn, TOut>, kThreads, 0) != cudaSuccess || n < 1)
      n = 1;
    ctas_per_sm = n;
  }
  const int per_wave = device_sm_count() * ctas_per_sm / n_slabs > 0 ? device_sm_count() * ctas_per_sm / n_slabs : 1;
  const int min_blk = (T + kSegBlk - 1) / kSegBlk;
  const int waves = (min_blk + per_wave - 1) / per_wave;
  int blk_len = (T + waves * per_wave - 1) / (waves * per_wave);
  if (blk_len < 8) blk_len = 8 < T ? 8 : T;
  if (blk_len > kSegBlk) blk_len = kSegBlk;
  const int n_blk = (T + blk_len - 1) / blk_len;
  int32_t* counters = static_cast<int32_t*>(scratch);
  float* partial = reinterpret_cast<float*>(static_cast<char*>(scratch) + partial_offset_bytes(n_blk, n_slabs));
  cudaError_t e = cudaMemsetAsync(counters, 0, static_cast<size_t>(n_blk) * n_slabs * sizeof(int32_t), stream);
  if (e != cudaSuccess) return e;
  segreduce_kernel<TIn, TOut><<<dim3(n_blk, n_slabs), kThreads, 0, stream>>>(
      T, F, blk_len, static_cast<const TIn*>(dU), perm, seg_offsets, n_unique, static_cast<TOut*>(dE_rows), counters, partial);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace

size_t segreduce_workspace_bytes(int T, int F) {
  if (T <= 0) return 0;
  // bounds over every launch shape: blocks of at least 8 positions, the narrowest slab
  const size_t n_blk = (static_cast<size_t>(T) + 7) / 8;
  const int n_slabs = (F + kThreads * 4 - 1) / (kThreads * 4);
  return partial_offset_bytes(static_cast<int>(n_blk), n_slabs) + align_up(2 * n_blk * static_cast<size_t>(F) * sizeof(float), 256);
}

cudaError_t launch_segreduce(int T, int F, int in_dtype, int out_dtype, const void* dU,
                             const int32_t* perm, const int32_t* seg_offsets,
                             const int32_t* n_unique, void* dE_rows, void* scratch,
                             cudaStream_t stream) {
  if (T <= 0) return cudaSuccess;
  if (in_dtype == STEM_DTYPE_FP32) {
    if (out_dtype == STEM_DTYPE_FP32)
      return launch_typed<float, float>(T, F, dU, perm, seg_offsets, n_unique, dE_rows, scratch, stream);
    return launch_typed<float, __nv_bfloat16>(T, F, dU, perm, seg_offsets, n_unique, dE_rows, scratch, stream);
  }
  if (out_dtype == STEM_DTYPE_FP32)
    return launch_typed<__nv_bfloat16, float>(T, F, dU, perm, seg_offsets, n_unique, dE_rows, scratch, stream);
  return launch_typed<__nv_bfloat16, __nv_bfloat16>(T, F, dU, perm, seg_offsets, n_unique, dE_rows, scratch, stream);
}

}  // namespace stem
