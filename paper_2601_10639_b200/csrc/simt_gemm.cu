// FMA-pipe contraction kernels with the layer's fused epilogues.
//
// These carry the fp32 configuration (tensor cores have no true fp32 MMA: kind::tf32
// rounds inputs to a 10-bit mantissa, which cannot meet a 1e-5 error bound) and serve as
// a slow cross-check for the bf16 tensor-core kernels (STEM_FLAG_SIMT).
#include "stem_internal.h"

namespace stem {
namespace {

constexpr int TM = 64, TN = 64, TK = 16;

template <typename T, int KIND>
__device__ __forceinline__ void epilogue_elem(const EpiParams& ep, int m, int n, int N, int row_id,
                                              float acc) {
  const size_t o = static_cast<size_t>(m) * N + n;
  if (KIND == kEpiStore) {
    if (ep.out_fp32) {
      float* p = static_cast<float*>(ep.out) + o;
      *p = ep.accumulate ? *p + acc : acc;
    } else {
      T* p = static_cast<T*>(ep.out) + o;
      *p = from_f32<T>(ep.accumulate ? to_f32(*p) + acc : acc);
    }
  } else if (KIND == kEpiAdd) {
    const float u = to_f32(static_cast<const T*>(ep.E)[static_cast<size_t>(row_id) * N + n]);
    static_cast<T*>(ep.H)[o] = from_f32<T>(acc + u);
  } else if (KIND == kEpiGate) {
    const float u = to_f32(static_cast<const T*>(ep.E)[static_cast<size_t>(row_id) * N + n]);
    const float s = sigmoid_f32(acc);
    static_cast<T*>(ep.H)[o] = from_f32<T>(acc * s * u);
    if (ep.G) static_cast<T*>(ep.G)[o] = from_f32<T>(acc);
  } else {
    const float u = to_f32(static_cast<const T*>(ep.E)[static_cast<size_t>(row_id) * N + n]);
    const float g = to_f32(static_cast<const T*>(ep.Gin)[o]);
    const float s = sigmoid_f32(g);
    static_cast<T*>(ep.H)[o] = from_f32<T>(acc * (g * s));                          // dU
    static_cast<T*>(ep.G)[o] = from_f32<T>(acc * u * (s * (1.0f + g * (1.0f - s))));  // dG
  }
}

template <typename T, bool A_MN, bool B_MN, int KIND>
__global__ void __launch_bounds__(256)
simt_gemm_kernel(int M, int N, int K, const T* __restrict__ A, const T* __restrict__ B, EpiParams ep) {
  __shared__ float As[TK][TM + 4];
  __shared__ float Bs[TK][TN + 4];
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const int m0 = blockIdx.y * TM, n0 = blockIdx.x * TN;
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;

  for (int k0 = 0; k0 < K; k0 += TK) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int idx = tid + i * 256;
      int mm, kk;
      if (A_MN) { mm = idx % TM; kk = idx / TM; } else { kk = idx % TK; mm = idx / TK; }
      const int gm = m0 + mm, gk = k0 + kk;
      float v = 0.0f;
      if (gm < M && gk < K)
        v = to_f32(A_MN ? A[static_cast<size_t>(gk) * M + gm] : A[static_cast<size_t>(gm) * K + gk]);
      As[kk][mm] = v;
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int idx = tid + i * 256;
      int nn, kk;
      if (B_MN) { nn = idx % TN; kk = idx / TN; } else { kk = idx % TK; nn = idx / TK; }
      const int gn = n0 + nn, gk = k0 + kk;
      float v = 0.0f;
      if (gn < N && gk < K)
        v = to_f32(B_MN ? B[static_cast<size_t>(gk) * N + gn] : B[static_cast<size_t>(gn) * K + gk]);
      Bs[kk][nn] = v;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      float a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
    }
    __syncthreads();
  }

#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= M) continue;
    int row_id = 0;
    if (KIND != kEpiStore) {
      row_id = ep.ids != nullptr ? ep.ids[m] : m;
      if (row_id < 0 || row_id >= ep.V) {
        report_error(ep.status, STEM_ERR_ID_RANGE, m);
        row_id = row_id < 0 ? 0 : ep.V - 1;
      }
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n < N) epilogue_elem<T, KIND>(ep, m, n, N, row_id, acc[i][j]);
    }
  }
}

template <typename T, bool A_MN, bool B_MN>
cudaError_t launch_kind(int M, int N, int K, const void* A, const void* B, EpiKind kind,
                        const EpiParams& ep, cudaStream_t stream) {
  dim3 grid((N + TN - 1) / TN, (M + TM - 1) / TM);
  const T* a = static_cast<const T*>(A);
  const T* b = static_cast<const T*>(B);
  switch (kind) {
    case kEpiStore: simt_gemm_kernel<T, A_MN, B_MN, kEpiStore><<<grid, 256, 0, stream>>>(M, N, K, a, b, ep); break;
    case kEpiGate: simt_gemm_kernel<T, A_MN, B_MN, kEpiGate><<<grid, 256, 0, stream>>>(M, N, K, a, b, ep); break;
    case kEpiDH: simt_gemm_kernel<T, A_MN, B_MN, kEpiDH><<<grid, 256, 0, stream>>>(M, N, K, a, b, ep); break;
    case kEpiAdd: simt_gemm_kernel<T, A_MN, B_MN, kEpiAdd><<<grid, 256, 0, stream>>>(M, N, K, a, b, ep); break;
  }
  count_launches(1);
  return cudaGetLastError();
}

template <typename T>
cudaError_t launch_layout(int M, int N, int K, const void* A, bool a_mn, const void* B, bool b_mn,
                          EpiKind kind, const EpiParams& ep, cudaStream_t stream) {
  if (!a_mn && !b_mn) return launch_kind<T, false, false>(M, N, K, A, B, kind, ep, stream);
  if (!a_mn && b_mn) return launch_kind<T, false, true>(M, N, K, A, B, kind, ep, stream);
  if (a_mn && !b_mn) return launch_kind<T, true, false>(M, N, K, A, B, kind, ep, stream);
  return launch_kind<T, true, true>(M, N, K, A, B, kind, ep, stream);
}

}  // namespace

cudaError_t launch_simt_gemm(int dtype, int M, int N, int K, const void* A, bool a_mn,
                             const void* B, bool b_mn, EpiKind kind, const EpiParams& ep,
                             cudaStream_t stream) {
  if (M <= 0 || N <= 0) return cudaSuccess;
  if (dtype == STEM_DTYPE_FP32)
    return launch_layout<float>(M, N, K, A, a_mn, B, b_mn, kind, ep, stream);
  return launch_layout<__nv_bfloat16>(M, N, K, A, a_mn, B, b_mn, kind, ep, stream);
}

}  // namespace stem
