// C ABI of libstem: argument checks, workspace carve-up and kernel sequencing.
#include <cstdio>
#include <cstring>

#include "stem_internal.h"

namespace stem {

int device_sm_count() {
  static int cached[64] = {0};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev] = n;
  }
  return cached[dev];
}

namespace {

thread_local char g_cuda_msg[256] = "";

int cuda_fail(cudaError_t e) {
  snprintf(g_cuda_msg, sizeof(g_cuda_msg), "CUDA error: %s", cudaGetErrorString(e));
  return STEM_ERR_CUDA;
}

bool is_sm100() {
  static int cached[64] = {0};  // 0 unknown, 1 yes, 2 no
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return false;
  if (cached[dev] == 0) {
    int major = 0;
    cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    cached[dev] = major == 10 ? 1 : 2;
  }
  return cached[dev] == 1;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

size_t elem_bytes(int dtype) { return dtype == STEM_DTYPE_FP32 ? 4 : 2; }

int check_shape(const stem_shape_t* s) {
  if (!s) return STEM_ERR_INVALID_ARG;
  if (s->dtype != STEM_DTYPE_FP32 && s->dtype != STEM_DTYPE_BF16) return STEM_ERR_INVALID_ARG;
  if (s->grad_dtype != STEM_DTYPE_FP32 && s->grad_dtype != STEM_DTYPE_BF16) return STEM_ERR_INVALID_ARG;
  if (s->T < 0 || s->d_model <= 0 || s->d_ff <= 0 || s->V <= 0) return STEM_ERR_INVALID_ARG;
  if (s->T > (1 << 22) || s->V > (1 << 30)) return STEM_ERR_UNSUPPORTED_SHAPE;
  if (s->dtype == STEM_DTYPE_FP32 && s->grad_dtype != STEM_DTYPE_FP32) return STEM_ERR_INVALID_ARG;
  const int mult = s->dtype == STEM_DTYPE_BF16 ? 8 : 4;
  if (s->d_model % mult || s->d_ff % mult) return STEM_ERR_UNSUPPORTED_SHAPE;
  return STEM_OK;
}

struct WsLayout {
  size_t dedup_off, dedup_bytes;
  size_t h_off, h_bytes;     // forward: H when the caller keeps none
  size_t du_off, dg_off, tf_bytes, part_off, part_bytes;
  size_t total;
};

WsLayout ws_layout(const stem_shape_t* s) {
  WsLayout w{};
  const size_t tf = align_up(static_cast<size_t>(s->T) * s->d_ff * elem_bytes(s->dtype), 256);
  w.tf_bytes = tf;
  w.dedup_off = kStatusBytes;
  w.dedup_bytes = dedup_workspace_bytes(s->T, s->V);
  w.h_off = kStatusBytes;
  w.h_bytes = tf;
  w.du_off = kStatusBytes;
  w.dg_off = w.du_off + tf;
  w.part_off = w.dg_off + tf;
  w.part_bytes = segreduce_workspace_bytes(s->T, s->d_ff);
  size_t m = w.dedup_off + w.dedup_bytes;
  if (w.h_off + w.h_bytes > m) m = w.h_off + w.h_bytes;
  if (w.part_off + w.part_bytes > m) m = w.part_off + w.part_bytes;
  w.total = align_up(m, 256);
  return w;
}

int32_t* status_of(void* ws) { return static_cast<int32_t*>(ws); }

bool use_tc(const stem_shape_t* s) {
  return s->dtype == STEM_DTYPE_BF16 && !(s->flags & STEM_FLAG_SIMT);
}

cudaError_t gemm(const stem_shape_t* s, int M, int N, int K, const void* A, bool a_mn, const void* B,
                 bool b_mn, EpiKind kind, const EpiParams& ep, cudaStream_t st) {
  if (use_tc(s)) return launch_tc_gemm(M, N, K, A, a_mn, B, b_mn, kind, ep, st);
  return launch_simt_gemm(s->dtype, M, N, K, A, a_mn, B, b_mn, kind, ep, st);
}

int pinned_or_device(const void* p, const void** dev_ptr) {
  cudaPointerAttributes attr;
  if (cudaPointerGetAttributes(&attr, p) != cudaSuccess) { cudaGetLastError(); return STEM_ERR_NOT_PINNED; }
  if (attr.type == cudaMemoryTypeUnregistered) return STEM_ERR_NOT_PINNED;
  *dev_ptr = attr.devicePointer ? attr.devicePointer : p;
  return STEM_OK;
}

}  // namespace
}  // namespace stem

using namespace stem;

extern "C" {

int stem_version(void) { return 100; }

const char* stem_status_string(int code) {
  switch (code) {
    case STEM_OK: return "ok";
    case STEM_ERR_INVALID_ARG: return "invalid argument (null or misaligned pointer, bad dtype or size)";
    case STEM_ERR_UNSUPPORTED_SHAPE: return "unsupported shape (T > 2^22, V > 2^30, or d_model/d_ff not a multiple of 8 (bf16) / 4 (fp32))";
    case STEM_ERR_UNSUPPORTED_ARCH: return "device is not compute capability 10.x (sm_100a)";
    case STEM_ERR_WORKSPACE_TOO_SMALL: return "workspace smaller than stem_workspace_bytes()";
    case STEM_ERR_NOT_PINNED: return "host pointer is not page-locked (cudaHostAlloc / cudaHostRegister)";
    case STEM_ERR_CUDA: return g_cuda_msg[0] ? g_cuda_msg : "CUDA error";
    case STEM_ERR_TIMEOUT: return "device: a bounded pipeline wait expired";
    case STEM_ERR_ID_RANGE: return "device: token id outside [0,V) (clamped)";
    default: return "unknown status";
  }
}

int stem_workspace_bytes(const stem_shape_t* shape, size_t* bytes) {
  if (!bytes) return STEM_ERR_INVALID_ARG;
  if (int rc = check_shape(shape)) return rc;
  *bytes = ws_layout(shape).total;
  return STEM_OK;
}

int stem_init_workspace(void* ws, size_t ws_bytes, void* stream) {
  if (!ws || !aligned16(ws)) return STEM_ERR_INVALID_ARG;
  if (ws_bytes < kStatusBytes) return STEM_ERR_WORKSPACE_TOO_SMALL;
  cudaError_t e = cudaMemsetAsync(ws, 0, kStatusBytes, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? STEM_OK : cuda_fail(e);
}

int stem_query_status(const void* ws, void* stream, int32_t* status_out) {
  if (!ws || !status_out) return STEM_ERR_INVALID_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e = cudaMemcpyAsync(status_out, ws, sizeof(int32_t), cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  return e == cudaSuccess ? STEM_OK : cuda_fail(e);
}

int stem_dedup_ids(const stem_shape_t* shape, const int32_t* ids, int32_t* unique_ids, int32_t* n_unique,
                   int32_t* inverse, int32_t* perm, int32_t* seg_offsets, void* ws, size_t ws_bytes,
                   void* stream) {
  if (int rc = check_shape(shape)) return rc;
  if (!unique_ids || !n_unique || !perm || !seg_offsets || !ws || !aligned16(ws)) return STEM_ERR_INVALID_ARG;
  if (shape->T > 0 && !ids) return STEM_ERR_INVALID_ARG;
  const WsLayout w = ws_layout(shape);
  if (ws_bytes < w.total) return STEM_ERR_WORKSPACE_TOO_SMALL;
  cudaError_t e = launch_dedup(shape->T, shape->V, ids, unique_ids, n_unique, inverse, perm, seg_offsets,
                               static_cast<char*>(ws) + w.dedup_off, status_of(ws), static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? STEM_OK : cuda_fail(e);
}

int stem_ffn_forward(const stem_shape_t* shape, const void* x, const int32_t* ids, const void* W_gate,
                     const void* E, const void* W_down, void* y, void* G_save, void* H_save, void* ws,
                     size_t ws_bytes, void* stream) {
  if (int rc = check_shape(shape)) return rc;
  if (!ws || !aligned16(ws)) return STEM_ERR_INVALID_ARG;
  if (shape->T == 0) return STEM_OK;
  if (!x || !ids || !W_gate || !E || !W_down || !y) return STEM_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(W_gate) || !aligned16(E) || !aligned16(W_down) || !aligned16(y) ||
      !aligned16(G_save) || !aligned16(H_save))
    return STEM_ERR_INVALID_ARG;
  const WsLayout w = ws_layout(shape);
  if (ws_bytes < w.total) return STEM_ERR_WORKSPACE_TOO_SMALL;
  if (use_tc(shape) && !is_sm100()) return STEM_ERR_UNSUPPORTED_ARCH;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int T = shape->T, d = shape->d_model, F = shape->d_ff;
  void* H = H_save ? H_save : static_cast<char*>(ws) + w.h_off;

  EpiParams gate;
  gate.ids = ids; gate.E = E; gate.V = shape->V; gate.H = H; gate.G = G_save; gate.status = status_of(ws);
  cudaError_t e = gemm(shape, T, F, d, x, false, W_gate, false, kEpiGate, gate, st);   // G = x W_gate^T, fused lookup
  if (e != cudaSuccess) return cuda_fail(e);
  EpiParams down;
  down.out = y; down.out_fp32 = shape->dtype == STEM_DTYPE_FP32; down.status = status_of(ws);
  e = gemm(shape, T, d, F, H, false, W_down, false, kEpiStore, down, st);              // y = H W_down^T
  return e == cudaSuccess ? STEM_OK : cuda_fail(e);
}

int stem_ffn_backward(const stem_shape_t* shape, const void* dy, const void* x, const int32_t* ids,
                      const void* W_gate, const void* E, const void* W_down, const void* G_save,
                      const void* H_save, const int32_t* perm, const int32_t* seg_offsets,
                      const int32_t* n_unique, void* dx, void* dW_gate, void* dW_down, void* dE_rows,
                      const int32_t* unique_ids, void* ws, size_t ws_bytes, void* stream) {
  (void)unique_ids;
  if (int rc = check_shape(shape)) return rc;
  if (!ws || !aligned16(ws)) return STEM_ERR_INVALID_ARG;
  if (shape->T == 0) return STEM_OK;
  if (!dy || !x || !ids || !W_gate || !E || !W_down || !G_save) return STEM_ERR_INVALID_ARG;
  if (dW_down && !H_save) return STEM_ERR_INVALID_ARG;
  if (dE_rows && (!perm || !seg_offsets || !n_unique)) return STEM_ERR_INVALID_ARG;
  if (!aligned16(dy) || !aligned16(x) || !aligned16(W_gate) || !aligned16(E) || !aligned16(W_down) ||
      !aligned16(G_save) || !aligned16(H_save) || !aligned16(dx) || !aligned16(dW_gate) ||
      !aligned16(dW_down) || !aligned16(dE_rows))
    return STEM_ERR_INVALID_ARG;
  const WsLayout w = ws_layout(shape);
  if (ws_bytes < w.total) return STEM_ERR_WORKSPACE_TOO_SMALL;
  if (use_tc(shape) && !is_sm100()) return STEM_ERR_UNSUPPORTED_ARCH;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int T = shape->T, d = shape->d_model, F = shape->d_ff;
  const int grad_fp32 = shape->grad_dtype == STEM_DTYPE_FP32;
  char* base = static_cast<char*>(ws);
  void* dU = base + w.du_off;
  void* dG = base + w.dg_off;

  // dH = dy W_down (contraction over d_model; W_down is [d, F]: F contiguous), fused
  // dU = dH SiLU(G), dG = dH E[ids] SiLU'(G)
  EpiParams dh;
  dh.ids = ids; dh.E = E; dh.V = shape->V; dh.H = dU; dh.G = dG; dh.Gin = G_save; dh.status = status_of(ws);
  cudaError_t e = gemm(shape, T, F, d, dy, false, W_down, true, kEpiDH, dh, st);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dW_down) {  // dW_down[i,j] = sum_t dy[t,i] H[t,j]
    EpiParams p; p.out = dW_down; p.out_fp32 = grad_fp32; p.status = status_of(ws);
    e = gemm(shape, d, F, T, dy, true, H_save, true, kEpiStore, p, st);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  if (dE_rows) {
    e = launch_segreduce(T, F, shape->dtype, shape->grad_dtype, dU, perm, seg_offsets, n_unique, dE_rows,
                         base + w.part_off, st);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  if (dW_gate) {  // dW_gate[j,k] = sum_t dG[t,j] x[t,k]
    EpiParams p; p.out = dW_gate; p.out_fp32 = grad_fp32; p.status = status_of(ws);
    e = gemm(shape, F, d, T, dG, true, x, true, kEpiStore, p, st);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  if (dx) {  // dx = dG W_gate (contraction over d_ff; W_gate is [F, d]: d contiguous)
    EpiParams p; p.out = dx; p.out_fp32 = shape->dtype == STEM_DTYPE_FP32; p.status = status_of(ws);
    e = gemm(shape, T, d, F, dG, false, W_gate, true, kEpiStore, p, st);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  return STEM_OK;
}

int stem_prefetch_rows(const stem_shape_t* shape, const int32_t* ids, const int32_t* n_ids, const void* table,
                       void* dev_cache, void* ws, void* stream) {
  if (int rc = check_shape(shape)) return rc;
  if (shape->T == 0) return STEM_OK;
  if (!ids || !n_ids || !table || !dev_cache || !aligned16(table) || !aligned16(dev_cache)) return STEM_ERR_INVALID_ARG;
  const void* src = nullptr;
  if (int rc = pinned_or_device(table, &src)) return rc;
  const int max_rows = shape->T < shape->V ? shape->T : shape->V;
  const size_t row_bytes = static_cast<size_t>(shape->d_ff) * elem_bytes(shape->dtype);
  cudaError_t e = launch_gather_rows(max_rows, shape->V, row_bytes, ids, n_ids, src, dev_cache,
                                     ws ? status_of(ws) : nullptr, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? STEM_OK : cuda_fail(e);
}

int stem_writeback_rows(const stem_shape_t* shape, const void* dE_rows, const int32_t* unique_ids,
                        const int32_t* n_rows, void* host_rows, int32_t* host_ids, int32_t* host_n,
                        void* stream) {
  if (int rc = check_shape(shape)) return rc;
  if (shape->T == 0) return STEM_OK;
  if (!dE_rows || !unique_ids || !n_rows || !host_rows || !host_ids || !host_n || !aligned16(dE_rows) ||
      !aligned16(host_rows))
    return STEM_ERR_INVALID_ARG;
  const void *hr = nullptr, *hi = nullptr, *hn = nullptr;
  if (int rc = pinned_or_device(host_rows, &hr)) return rc;
  if (int rc = pinned_or_device(host_ids, &hi)) return rc;
  if (int rc = pinned_or_device(host_n, &hn)) return rc;
  const int max_rows = shape->T < shape->V ? shape->T : shape->V;
  const size_t row_bytes = static_cast<size_t>(shape->d_ff) * elem_bytes(shape->grad_dtype);
  cudaError_t e = launch_writeback_rows(max_rows, row_bytes, dE_rows, unique_ids, n_rows, const_cast<void*>(hr),
                                        static_cast<int32_t*>(const_cast<void*>(hi)),
                                        static_cast<int32_t*>(const_cast<void*>(hn)), static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? STEM_OK : cuda_fail(e);
}

int stem_gemm_bf16(int32_t M, int32_t N, int32_t K, const void* A, int32_t a_mn, const void* B, int32_t b_mn,
                   void* C, int32_t c_fp32, int32_t flags, void* ws, void* stream) {
  if (M < 0 || N < 0 || K <= 0) return STEM_ERR_INVALID_ARG;
  if (M == 0 || N == 0) return STEM_OK;
  if (!A || !B || !C || !ws || !aligned16(A) || !aligned16(B) || !aligned16(C)) return STEM_ERR_INVALID_ARG;
  if ((M % 8) || (N % 8) || (K % 8)) return STEM_ERR_UNSUPPORTED_SHAPE;
  EpiParams p; p.out = C; p.out_fp32 = c_fp32; p.status = status_of(ws);
  cudaError_t e;
  if (flags & STEM_FLAG_SIMT) {
    e = launch_simt_gemm(STEM_DTYPE_BF16, M, N, K, A, a_mn != 0, B, b_mn != 0, kEpiStore, p, static_cast<cudaStream_t>(stream));
  } else {
    if (!is_sm100()) return STEM_ERR_UNSUPPORTED_ARCH;
    e = launch_tc_gemm(M, N, K, A, a_mn != 0, B, b_mn != 0, kEpiStore, p, static_cast<cudaStream_t>(stream));
  }
  return e == cudaSuccess ? STEM_OK : cuda_fail(e);
}

}  // extern "C"
