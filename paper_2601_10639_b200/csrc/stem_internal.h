// Internal declarations shared by the translation units of libstem.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <cstddef>
#include <cstdint>

#include "../../include/stem.h"

namespace stem {

constexpr size_t kStatusBytes = 256;  // head of every workspace
// status word layout (int32): [0] first error code, [1] detail, [2] count of bad ids
struct StatusWord {
  int32_t code;
  int32_t detail;
  int32_t bad_ids;
};

__device__ __forceinline__ void report_error(int32_t* status, int32_t code, int32_t detail) {
  if (status == nullptr) return;
  if (atomicCAS(status, 0, code) == 0) status[1] = detail;
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// ---- element helpers ----------------------------------------------------------------
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) {
  return __float2bfloat16_rn(v);
}

__device__ __forceinline__ float sigmoid_f32(float g) { return 1.0f / (1.0f + expf(-g)); }

// ---- epilogue descriptions (shared by the FMA and the tensor-core GEMM front ends) ---
enum EpiKind : int { kEpiStore = 0, kEpiGate = 1, kEpiDH = 2, kEpiAdd = 3, kEpiDagger = 4 };

struct EpiParams {
  // kEpiStore: out[m*ld + n] = acc              (out_fp32 selects fp32 or bf16/T storage)
  //            accumulate: out[m*ld + n] += acc   (gradient accumulation over micro-batches)
  void* out = nullptr;
  int out_fp32 = 0;
  int accumulate = 0;
  // kEpiGate:  g = acc; H = SiLU(g) * E[ids[m], n]; optional G = g
  // kEpiDH:    dh = acc; g = G[m,n]; u = E[ids[m], n];
  //            dU = dh * SiLU(g); dG = dh * u * SiLU'(g)
  // kEpiAdd:   H[m,n] = acc + E[ids[m], n]      (bf16/T storage; in place when E == H)
  // ids == nullptr in kEpiGate / kEpiDH / kEpiAdd means ids[m] = m: E is then a [M,N] matrix
  const int32_t* ids = nullptr;
  const void* E = nullptr;
  int V = 0;
  void* H = nullptr;    // kEpiGate: H out          kEpiDH: dU out
  void* G = nullptr;    // kEpiGate: G out (opt.)   kEpiDH: dG out
  const void* Gin = nullptr;  // kEpiDH: saved G
  // kEpiDagger (two products of the same A tile, gate = acc and up = acc2):
  //            U = acc2 + E[ids[m], n]; H = SiLU(acc) * U; optional G = acc, optional U out
  void* U = nullptr;
  int32_t* status = nullptr;
  // kEpiStore, optional: scratch for partial tiles when the last round of tiles is split
  // along k (tc_gemm_scratch_bytes()); without it every tile is computed whole
  void* sk_scratch = nullptr;
  size_t sk_bytes = 0;
};

// C[m,n] = sum_k A(m,k) B(n,k); a_mn/b_mn: operand stored with the M (N) index contiguous.
// FMA-pipe kernels, any T in {float, bf16}; fp32 accumulation.
cudaError_t launch_simt_gemm(int dtype, int M, int N, int K, const void* A, bool a_mn,
                             const void* B, bool b_mn, EpiKind kind, const EpiParams& ep,
                             cudaStream_t stream);

// tcgen05 / TMEM / TMA kernels, bf16 inputs.  Returns cudaErrorNotSupported when the
// shape cannot be described to TMA (the caller decides what to do).
// pair: run on CTA pairs (cta_group::2, 256-row tiles) rather than single CTAs.
cudaError_t launch_tc_gemm(int M, int N, int K, const void* A, bool a_mn, const void* B,
                           bool b_mn, EpiKind kind, const EpiParams& ep, bool pair, cudaStream_t stream);

// Two token-contracted products in one launch (the two weight gradients of the layer):
//   out1[m,n] = sum_k A1(k,m) B1(k,n)   and   out2[m,n] = sum_k A2(k,m) B2(k,n),
// all four operands stored [K, .] row-major (MN-major), both outputs of ep.out_fp32's type, the
// same ep.accumulate.  Their tiles share one work list, so the pair fills the SMs where each
// product alone leaves some idle; ep.out is ignored (out1 / out2 are the outputs).
cudaError_t launch_tc_gemm_token_pair(int K, int M1, int N1, const void* A1, const void* B1, void* out1, int M2,
                                      int N2, const void* A2, const void* B2, void* out2, const EpiParams& ep,
                                      bool pair, cudaStream_t stream);

// The dagger variant's gate and up products of the same x tile in one launch (CTA pairs, two
// accumulators): G = A B_gate^T, Up = A B_up^T, then U = Up + E[ids], H = SiLU(G) * U in the
// epilogue; outputs ep.H and, when not NULL, ep.G and ep.U.  All operands K-major.
cudaError_t launch_tc_gemm_dagger(int M, int N, int K, const void* A, const void* B_gate, const void* B_up,
                                  const EpiParams& ep, cudaStream_t stream);

size_t tc_gemm_scratch_bytes();

// ---- index path ----------------------------------------------------------------------
size_t dedup_workspace_bytes(int T, int V);
cudaError_t launch_dedup(int T, int V, const int32_t* ids, int32_t* unique_ids, int32_t* n_unique,
                         int32_t* inverse, int32_t* perm, int32_t* seg_offsets, void* scratch,
                         int32_t* status, cudaStream_t stream);

// Stable radix sort of n keys in [0, V) (the sort inside launch_dedup): perm = positions in
// sorted order, *sorted_keys = the sorted keys (inside scratch, dedup_workspace_bytes(n, V)).
cudaError_t launch_stable_sort(int n, int V, const int32_t* keys_in, int32_t* perm, void* scratch,
                               const int32_t** sorted_keys, int32_t* status, cudaStream_t stream);

// ---- table-gradient reduce --------------------------------------------------------------
size_t segreduce_workspace_bytes(int T, int F);
cudaError_t launch_segreduce(int T, int F, int in_dtype, int out_dtype, const void* dU,
                             const int32_t* perm, const int32_t* seg_offsets,
                             const int32_t* n_unique, void* dE_rows, void* scratch,
                             cudaStream_t stream);

// ---- row movers ---------------------------------------------------------------------------
// table_on_host: the table is page-locked host memory read over the host link; the launch
// is then kept small enough to share the SMs with a running contraction kernel.
cudaError_t launch_gather_rows(int max_rows, int V, size_t row_bytes, const int32_t* ids,
                               const int32_t* n_ids, const void* table, bool table_on_host,
                               const void* hot_rows, const int32_t* hot_slot, void* dst, int32_t* status,
                               int32_t* stats, cudaStream_t stream);
cudaError_t launch_writeback_rows(int max_rows, size_t row_bytes, const void* rows,
                                  const int32_t* unique_ids, const int32_t* n_rows, void* host_rows,
                                  int32_t* host_ids, int32_t* host_n, int32_t* status, cudaStream_t stream);

// ---- frequency-ranked row cache ------------------------------------------------------------
size_t lfu_workspace_bytes(int V, int K);
cudaError_t launch_lfu_touch(int n, int V, const int32_t* ids, int32_t* freq, const int32_t* hot_slot,
                             int32_t* stats, int32_t* status, cudaStream_t stream);
cudaError_t launch_lfu_refresh(int V, int K, size_t row_bytes, const int32_t* freq, int32_t* hot_slot,
                               int32_t* hot_ids, void* hot_rows, const void* table, int32_t* n_installed,
                               void* scratch, cudaStream_t stream);

// ---- table sharded over GPUs: requests of the row exchange ---------------------------------
size_t shard_route_workspace_bytes(int n_max, int G);
cudaError_t launch_shard_route(int n_max, int T, int G, const int32_t* unique_ids, const int32_t* n_unique,
                               const int32_t* inverse, int32_t* send_local, int32_t* send_slot,
                               int32_t* send_counts, int32_t* token_slot, void* scratch, int32_t* status,
                               cudaStream_t stream);

// Bounded-wait self-test (selftest.cu): one thread waits at most limit_cycles on a barrier that
// is completed first (arrive != 0) or never.
cudaError_t launch_selftest_wait(int32_t* status, long long limit_cycles, int arrive, cudaStream_t stream);

int device_sm_count();

// Function attributes (shared-memory size, preferred split) are per device: `done` is a
// per-call-site table that remembers on which devices `set()` has already succeeded.
struct PerDeviceOnce {
  bool done[64] = {};
  template <typename F> cudaError_t run(F set) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    if (done[dev]) return cudaSuccess;
    e = set();
    if (e == cudaSuccess) done[dev] = true;
    return e;
  }
};
void count_launches(int n);  // bookkeeping for stem_launch_count()

}  // namespace stem
