// Table-gradient reduce: dE_rows[r,:] = sum over the positions p of segment r of
// dU[perm[p],:], in a fixed order, without floating-point atomics.
//
// The sorted position range [0,T) is cut into blocks of kSegBlk positions.  Pass 1: one CTA
// per (block, column slab) walks its positions in order, accumulating in fp32 registers.
// A run whose segment lies wholly inside the block is final and is written to dE_rows; a
// run whose segment crosses a block edge (at most the first and the last run of a block)
// goes to a partial row.  Pass 2: the CTA of the block in which a crossing segment starts
// adds that segment's partial rows in block order.  Both orders depend on the index arrays
// only, so the result is bitwise reproducible.  HBM-bound: every dU row is read once with
// 16-byte loads, coalesced along d_ff.
#include "stem_internal.h"

namespace stem {
namespace {

constexpr int kSegBlk = 64;
constexpr int kThreads = 256;
constexpr int kBatch = 8;

template <typename T> struct Vec;
template <> struct Vec<float> {
  static constexpr int N = 4;
  __device__ static void load(const float* p, float (&v)[4]) {
    const float4 q = __ldg(reinterpret_cast<const float4*>(p));
    v[0] = q.x; v[1] = q.y; v[2] = q.z; v[3] = q.w;
  }
  __device__ static void store(float* p, const float (&v)[4]) {
    *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
  }
};
template <> struct Vec<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static void load(const __nv_bfloat16* p, float (&v)[8]) {
    const uint4 q = __ldg(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      v[2 * i] = __uint_as_float(w[i] << 16);
      v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
    }
  }
  __device__ static void store(__nv_bfloat16* p, const float (&v)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
      w[i] = *reinterpret_cast<const uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  }
};

// largest r in [0, n_u) with seg_offsets[r] <= p   (p < T = seg_offsets[n_u])
__device__ __forceinline__ int segment_of(const int32_t* seg_offsets, int n_u, int p) {
  int lo = 0, hi = n_u;  // invariant: seg_offsets[lo] <= p < seg_offsets[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (seg_offsets[mid] <= p) lo = mid; else hi = mid;
  }
  return lo;
}

// A thread owns VI consecutive columns; rows are written in the output type's vectors.
template <int VI, typename TOut>
__device__ __forceinline__ void store_row(TOut* dst, const float (&v)[VI]) {
#pragma unroll
  for (int i = 0; i < VI; i += Vec<TOut>::N) {
    float t[Vec<TOut>::N];
#pragma unroll
    for (int j = 0; j < Vec<TOut>::N; ++j) t[j] = v[i + j];
    Vec<TOut>::store(dst + i, t);
  }
}

template <typename TIn, typename TOut>
__global__ void __launch_bounds__(kThreads)
segreduce_pass1_kernel(int T, int F, const TIn* __restrict__ dU, const int32_t* __restrict__ perm,
                       const int32_t* __restrict__ seg_offsets, const int32_t* __restrict__ n_unique,
                       TOut* __restrict__ dE_rows, float* __restrict__ partial) {
  constexpr int VI = (Vec<TIn>::N > Vec<TOut>::N) ? Vec<TIn>::N : Vec<TOut>::N;
  __shared__ int s_row[kSegBlk];
  __shared__ int s_seg[kSegBlk];
  __shared__ int s_seg_begin[kSegBlk];
  __shared__ int s_seg_end[kSegBlk];
  const int blk = blockIdx.x;
  const int p0 = blk * kSegBlk;
  const int cnt = min(kSegBlk, T - p0);
  const int n_u = *n_unique;
  if (threadIdx.x < cnt) {
    const int p = p0 + threadIdx.x;
    const int r = segment_of(seg_offsets, n_u, p);
    s_row[threadIdx.x] = perm[p];
    s_seg[threadIdx.x] = r;
    s_seg_begin[threadIdx.x] = seg_offsets[r];
    s_seg_end[threadIdx.x] = seg_offsets[r + 1];
  }
  __syncthreads();
  const int col = (blockIdx.y * kThreads + threadIdx.x) * VI;
  if (col >= F) return;

  float acc[VI];
#pragma unroll
  for (int i = 0; i < VI; ++i) acc[i] = 0.0f;
  bool first_run = true;

  for (int b0 = 0; b0 < cnt; b0 += kBatch) {
    float v[kBatch][VI];
#pragma unroll
    for (int j = 0; j < kBatch; ++j) {
      if (b0 + j < cnt) {
        const TIn* src = dU + static_cast<size_t>(s_row[b0 + j]) * F + col;
#pragma unroll
        for (int i = 0; i < VI; i += Vec<TIn>::N) {
          float t[Vec<TIn>::N];
          Vec<TIn>::load(src + i, t);
#pragma unroll
          for (int q = 0; q < Vec<TIn>::N; ++q) v[j][i + q] = t[q];
        }
      }
    }
#pragma unroll
    for (int j = 0; j < kBatch; ++j) {
      const int q = b0 + j;
      if (q < cnt) {
#pragma unroll
        for (int i = 0; i < VI; ++i) acc[i] += v[j][i];
        const bool run_ends = (q + 1 == cnt) || (s_seg[q + 1] != s_seg[q]);
        if (run_ends) {
          const bool whole = s_seg_begin[q] >= p0 && s_seg_end[q] <= p0 + kSegBlk;
          if (whole) {
            store_row<VI, TOut>(dE_rows + static_cast<size_t>(s_seg[q]) * F + col, acc);
          } else {
            float* dst = partial + (static_cast<size_t>(2 * blk + (first_run ? 0 : 1))) * F + col;
            store_row<VI, float>(dst, acc);
          }
#pragma unroll
          for (int i = 0; i < VI; ++i) acc[i] = 0.0f;
          first_run = false;
        }
      }
    }
  }
}

template <typename TOut, int VI>
__global__ void __launch_bounds__(kThreads)
segreduce_pass2_kernel(int T, int F, const int32_t* __restrict__ seg_offsets,
                       const int32_t* __restrict__ n_unique, const float* __restrict__ partial,
                       TOut* __restrict__ dE_rows) {
  const int blk = blockIdx.x;
  const int p0 = blk * kSegBlk;
  const int p_last = min(T, p0 + kSegBlk) - 1;
  const int n_u = *n_unique;
  // the segment of this block's last position; this CTA owns it iff it starts here and
  // runs past the block's end
  const int r = segment_of(seg_offsets, n_u, p_last);
  const int seg_begin = seg_offsets[r], seg_end = seg_offsets[r + 1];
  if (seg_begin < p0 || seg_end <= p0 + kSegBlk) return;
  const int col = (blockIdx.y * kThreads + threadIdx.x) * VI;
  if (col >= F) return;
  const int b_last = (seg_end - 1) / kSegBlk;
  float acc[VI];
#pragma unroll
  for (int i = 0; i < VI; ++i) acc[i] = 0.0f;
  for (int b = blk; b <= b_last; ++b) {
    // the segment's run is the first run of block b unless b is the starting block and the
    // segment does not begin exactly at the block's first position
    const int slot = (b > blk || seg_begin == p0) ? 2 * b : 2 * b + 1;
    const float* src = partial + static_cast<size_t>(slot) * F + col;
#pragma unroll
    for (int i = 0; i < VI; i += 4) {
      const float4 q = *reinterpret_cast<const float4*>(src + i);
      acc[i] += q.x; acc[i + 1] += q.y; acc[i + 2] += q.z; acc[i + 3] += q.w;
    }
  }
  store_row<VI, TOut>(dE_rows + static_cast<size_t>(r) * F + col, acc);
}

template <typename TIn, typename TOut>
cudaError_t launch_typed(int T, int F, const void* dU, const int32_t* perm, const int32_t* seg_offsets,
                         const int32_t* n_unique, void* dE_rows, void* scratch, cudaStream_t stream) {
  constexpr int VI = (Vec<TIn>::N > Vec<TOut>::N) ? Vec<TIn>::N : Vec<TOut>::N;
  const int n_blk = (T + kSegBlk - 1) / kSegBlk;
  dim3 grid(n_blk, (F + kThreads * VI - 1) / (kThreads * VI));
  segreduce_pass1_kernel<TIn, TOut><<<grid, kThreads, 0, stream>>>(
      T, F, static_cast<const TIn*>(dU), perm, seg_offsets, n_unique, static_cast<TOut*>(dE_rows),
      static_cast<float*>(scratch));
  segreduce_pass2_kernel<TOut, VI><<<grid, kThreads, 0, stream>>>(
      T, F, seg_offsets, n_unique, static_cast<const float*>(scratch), static_cast<TOut*>(dE_rows));
  count_launches(2);
  return cudaGetLastError();
}

}  // namespace

size_t segreduce_workspace_bytes(int T, int F) {
  if (T <= 0) return 0;
  const size_t n_blk = (static_cast<size_t>(T) + kSegBlk - 1) / kSegBlk;
  return align_up(2 * n_blk * static_cast<size_t>(F) * sizeof(float), 256);
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
