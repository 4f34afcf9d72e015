// Table-gradient reduce: dE_rows[r,:] = sum over the positions p of segment r of
// dU[perm[p],:], in a fixed order, without floating-point atomics.
//
// The sorted position range [0,T) is cut into blocks of at most kSegBlk positions.  One CTA per
// (block, column slab) walks its positions in order, accumulating in fp32 registers.  A run
// whose segment lies wholly inside the block is final and is written to dE_rows; a run whose
// segment crosses a block edge (at most the first and the last run of a block) goes to a
// partial row, and the block in which such a segment starts leaves a note (row, first and last
// position).  A second, small kernel reads the notes and adds each crossing segment's partial
// rows in block order.  No counters, no atomics, no state that outlives the call: the order of
// every addition is fixed, so the result is bitwise reproducible.  Both kernels are launched
// with programmatic stream serialisation and wait for the grid before them first, so they cost
// no full launch boundary inside a chain of such kernels.  HBM-bound: every dU row is read once
// with 16-byte loads, coalesced along d_ff.
#include "ptx_sm100.cuh"
#include "stem_internal.h"

namespace stem {
namespace {

constexpr int kSegBlk = 64;     // most sorted positions per CTA (the launch picks blk_len <= kSegBlk)
constexpr int kCtasPerSm = 7;   // register budget the kernel is compiled for
constexpr int kThreads = 128;   // pass 1: one thread per vector of columns
constexpr int kBatch = 8;       // rows requested before the first is consumed
constexpr int kFinBatch = 8;    // finishing kernel: partial rows requested before the first is added

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

// Scratch layout: one note per block (int4: row of the crossing segment that starts in the
// block or -1, its first position, its end position, unused; written by the block's CTA of
// column slab 0 on every launch), then 2 partial rows per block.
__host__ __device__ inline size_t partial_offset_bytes(int n_blk) {
  return (static_cast<size_t>(n_blk) * sizeof(int4) + 255) / 256 * 256;
}

template <typename TIn, typename TOut>
__global__ void __launch_bounds__(kThreads, kCtasPerSm)
segreduce_kernel(int T, int F, int blk_len, const TIn* __restrict__ dU, const int32_t* __restrict__ perm,
                 const int32_t* __restrict__ seg_offsets, const int32_t* __restrict__ n_unique,
                 TOut* __restrict__ dE_rows, int4* __restrict__ notes, float* partial) {
  constexpr int VI = (Vec<TIn>::N > Vec<TOut>::N) ? Vec<TIn>::N : Vec<TOut>::N;
  constexpr int LD = VI / Vec<TIn>::N;  // 16-byte loads per row per thread
  __shared__ int s_off[kSegBlk + 1];    // offsets of the segments that can touch this block
  __shared__ int s_row[kSegBlk];
  __shared__ int s_loc[kSegBlk];        // position -> index into s_off
  const int blk = blockIdx.x;
  const int p0 = blk * blk_len;
  const int cnt = min(blk_len, T - p0);
  // everything below reads what earlier kernels of the stream produced
  ptx::grid_dependency_wait();
  ptx::grid_launch_dependents();
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
  // Rows are requested kHalf at a time, two requests in flight: while one half-batch is being
  // added, the next one is already on its way, so a thread never sits without loads outstanding
  // (the memory system, not the adds, sets the pace of this kernel).
  constexpr int kHalf = kBatch / 2;
  uint4 raw[2][kHalf][LD];
  auto request = [&](int buf, int first) {
#pragma unroll
    for (int j = 0; j < kHalf; ++j) {
      if (first + j < cnt) {
        const TIn* src = dU + static_cast<size_t>(s_row[first + j]) * F + col;
#pragma unroll
        for (int i = 0; i < LD; ++i) raw[buf][j][i] = Vec<TIn>::load_raw(src + i * Vec<TIn>::N);
      }
    }
  };
  auto consume = [&](int buf, int first) {
#pragma unroll
    for (int j = 0; j < kHalf; ++j) {
      const int q = first + j;
      if (q < cnt) {
#pragma unroll
        for (int i = 0; i < LD; ++i) Vec<TIn>::add(acc + i * Vec<TIn>::N, raw[buf][j][i]);
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
  };
  if (col_ok) {
    request(0, 0);
    for (int b0 = 0; b0 < cnt; b0 += kBatch) {
      request(1, b0 + kHalf);
      consume(0, b0);
      request(0, b0 + kBatch);
      consume(1, b0 + kHalf);
    }
  }

  // ---- the note for the finishing kernel: the crossing segment that starts in this block ------
  // Only the segment of the block's last position can start here and run on.  s_off[0] <= p0.
  if (blockIdx.y == 0 && threadIdx.x == 0) {
    const int j = s_loc[cnt - 1];
    const bool starts_here = s_off[j] >= p0, runs_on = s_off[j + 1] > p0 + blk_len;
    notes[blk] = (starts_here && runs_on) ? make_int4(r_first + j, s_off[j], s_off[j + 1], 0) : make_int4(-1, 0, 0, 0);
  }
}

// Finishing kernel: one CTA per (block, slab of 4 * kThreads columns), one 4-column vector per
// thread.  If a crossing segment starts in the block, add its partial rows in block order and
// write the row.
template <typename TOut>
__global__ void __launch_bounds__(kThreads)
segfinish_kernel(int F, int blk_len, const int4* __restrict__ notes, const float* __restrict__ partial,
                 TOut* __restrict__ dE_rows) {
  ptx::grid_dependency_wait();
  ptx::grid_launch_dependents();
  const int4 note = __ldcg(notes + blockIdx.x);
  if (note.x < 0) return;
  const int seg_begin = note.y, seg_end = note.z;
  const int start_blk = blockIdx.x, last_blk = (seg_end - 1) / blk_len;
  const int col = (blockIdx.y * kThreads + threadIdx.x) * 4;
  if (col >= F) return;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  // parts are requested kFinBatch at a time and added in block order: a segment of a frequent id
  // spans dozens of blocks, and one load latency per block would make this launch a serial tail
  for (int b0 = start_blk; b0 <= last_blk; b0 += kFinBatch) {
    float4 q[kFinBatch];
#pragma unroll
    for (int i = 0; i < kFinBatch; ++i) {
      const int b = b0 + i;
      if (b <= last_blk) {
        // the segment's run is the first run of block b, unless b is the block it starts in
        // and it does not start at that block's first position
        const int slot = (b > start_blk || seg_begin == start_blk * blk_len) ? 2 * b : 2 * b + 1;
        q[i] = __ldcg(reinterpret_cast<const float4*>(partial + static_cast<size_t>(slot) * F + col));
      }
    }
#pragma unroll
    for (int i = 0; i < kFinBatch; ++i) {
      if (b0 + i <= last_blk) { acc.x += q[i].x; acc.y += q[i].y; acc.z += q[i].z; acc.w += q[i].w; }
    }
  }
  TOut* dst = dE_rows + static_cast<size_t>(note.x) * F + col;
  dst[0] = from_f32<TOut>(acc.x); dst[1] = from_f32<TOut>(acc.y);
  dst[2] = from_f32<TOut>(acc.z); dst[3] = from_f32<TOut>(acc.w);
}

// Resident CTAs of the first kernel per SM, per device (an occupancy query is not free).
template <typename TIn, typename TOut>
int ctas_per_sm() {
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 1;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, segreduce_kernel<TIn, TOut>, kThreads, 0) != cudaSuccess || n < 1)
      n = 1;
    cached[dev] = n;
  }
  return cached[dev];
}

template <typename TIn, typename TOut>
cudaError_t launch_typed(int T, int F, const void* dU, const int32_t* perm, const int32_t* seg_offsets,
                         const int32_t* n_unique, void* dE_rows, void* scratch, cudaStream_t stream) {
  constexpr int VI = (Vec<TIn>::N > Vec<TOut>::N) ? Vec<TIn>::N : Vec<TOut>::N;
  const int n_slabs = (F + kThreads * VI - 1) / (kThreads * VI);
  // Block length: as long as allowed, then shortened so that the CTAs fill a whole number of
  // waves of the resident CTA slots (a ragged last wave of full-length blocks costs more than
  // evenly shorter blocks).
  const int resident = ctas_per_sm<TIn, TOut>();
  const int per_wave = device_sm_count() * resident / n_slabs > 0 ? device_sm_count() * resident / n_slabs : 1;
  const int min_blk = (T + kSegBlk - 1) / kSegBlk;
  const int waves = (min_blk + per_wave - 1) / per_wave;
  int blk_len = (T + waves * per_wave - 1) / (waves * per_wave);
  if (blk_len < 8) blk_len = 8 < T ? 8 : T;
  if (blk_len > kSegBlk) blk_len = kSegBlk;
  const int n_blk = (T + blk_len - 1) / blk_len;
  int4* notes = static_cast<int4*>(scratch);
  float* partial = reinterpret_cast<float*>(static_cast<char*>(scratch) + partial_offset_bytes(n_blk));
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(n_blk, n_slabs);
  cfg.blockDim = dim3(kThreads);
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, segreduce_kernel<TIn, TOut>, T, F, blk_len, static_cast<const TIn*>(dU), perm,
                                     seg_offsets, n_unique, static_cast<TOut*>(dE_rows), notes, partial);
  count_launches(1);
  if (e != cudaSuccess) return e;
  cfg.gridDim = dim3(n_blk, (F + 4 * kThreads - 1) / (4 * kThreads));
  e = cudaLaunchKernelEx(&cfg, segfinish_kernel<TOut>, F, blk_len, static_cast<const int4*>(notes),
                         static_cast<const float*>(partial), static_cast<TOut*>(dE_rows));
  count_launches(1);
  return e != cudaSuccess ? e : cudaGetLastError();
}

}  // namespace

size_t segreduce_workspace_bytes(int T, int F) {
  if (T <= 0) return 0;
  // bounds over every launch shape: blocks of at least 8 positions, the narrowest slab
  const size_t n_blk = (static_cast<size_t>(T) + 7) / 8;
  return partial_offset_bytes(static_cast<int>(n_blk)) + align_up(2 * n_blk * static_cast<size_t>(F) * sizeof(float), 256);
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
