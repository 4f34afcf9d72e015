// C ABI of libstem: argument checks, workspace carve-up and kernel sequencing.
#include <atomic>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <vector>

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
std::atomic<long long> g_launches{0};
}
void count_launches(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

namespace {

thread_local char g_cuda_msg[256] = "";

// Optional per-step timing: a pair of CUDA events around each step of the path, recorded
// on the caller's stream.  Off by default; a few microseconds per step when on.
struct ProfRecord { const char* name; cudaEvent_t begin, end; };
std::mutex g_prof_mutex;
bool g_prof_on = false;
std::vector<ProfRecord> g_prof;        // records of the current session
std::vector<cudaEvent_t> g_event_pool;  // events kept for reuse

cudaEvent_t take_event() {
  if (!g_event_pool.empty()) { cudaEvent_t e = g_event_pool.back(); g_event_pool.pop_back(); return e; }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}

// The end event of one step doubles as the begin event of the next when nothing else was
// launched by the library on that stream in between, which halves the events a step costs.
cudaEvent_t g_prof_last_end = nullptr;
cudaStream_t g_prof_last_stream = nullptr;
long long g_prof_last_launches = -1;

struct ProfScope {
  cudaStream_t st; int idx = -1;
  ProfScope(const char* name, cudaStream_t s) : st(s) {
    std::lock_guard<std::mutex> lock(g_prof_mutex);
    if (!g_prof_on) return;
    ProfRecord r{name, nullptr, nullptr};
    if (g_prof_last_end != nullptr && g_prof_last_stream == st &&
        g_prof_last_launches == g_launches.load(std::memory_order_relaxed)) {
      r.begin = g_prof_last_end;
    } else {
      r.begin = take_event();
      cudaEventRecord(r.begin, st);
    }
    r.end = take_event();
    g_prof.push_back(r);
    idx = static_cast<int>(g_prof.size()) - 1;
  }
  ~ProfScope() {
    if (idx < 0) return;
    std::lock_guard<std::mutex> lock(g_prof_mutex);
    if (idx >= static_cast<int>(g_prof.size())) return;
    cudaEventRecord(g_prof[idx].end, st);
    g_prof_last_end = g_prof[idx].end;
    g_prof_last_stream = st;
    g_prof_last_launches = g_launches.load(std::memory_order_relaxed);
  }
};

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
  size_t du_off, dg_off, tf_bytes, part_off, part_bytes, sk_off, sk_bytes;
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
  // partial tiles of the token-contracted gradients (dW_down, dW_gate): live while dG is
  w.sk_off = align_up(w.part_off + w.part_bytes, 1024);
  w.sk_bytes = s->dtype == STEM_DTYPE_BF16 ? tc_gemm_scratch_bytes() : 0;
  size_t m = w.dedup_off + w.dedup_bytes;
  if (w.h_off + w.h_bytes > m) m = w.h_off + w.h_bytes;
  if (w.sk_off + w.sk_bytes > m) m = w.sk_off + w.sk_bytes;
  w.total = align_up(m, 256);
  return w;
}

int32_t* status_of(void* ws) { return static_cast<int32_t*>(ws); }

bool use_tc(const stem_shape_t* s) {
  return s->dtype == STEM_DTYPE_BF16 && !(s->flags & STEM_FLAG_SIMT);
}

cudaError_t gemm(const stem_shape_t* s, int M, int N, int K, const void* A, bool a_mn, const void* B,
                 bool b_mn, EpiKind kind, const EpiParams& ep, cudaStream_t st) {
  if (use_tc(s)) return launch_tc_gemm(M, N, K, A, a_mn, B, b_mn, kind, ep, !(s->flags & STEM_FLAG_SINGLE_CTA), st);
  return launch_simt_gemm(s->dtype, M, N, K, A, a_mn, B, b_mn, kind, ep, st);
}

int pinned_or_device(const void* p, const void** dev_ptr, bool* on_host = nullptr) {
  cudaPointerAttributes attr;
  if (cudaPointerGetAttributes(&attr, p) != cudaSuccess) { cudaGetLastError(); return STEM_ERR_NOT_PINNED; }
  if (attr.type == cudaMemoryTypeUnregistered) return STEM_ERR_NOT_PINNED;
  *dev_ptr = attr.devicePointer ? attr.devicePointer : p;
  if (on_host) *on_host = attr.type == cudaMemoryTypeHost;
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
    case STEM_ERR_COUNT_RANGE: return "device: a row count exceeded the capacity of the row buffers (clamped)";
    case STEM_ERR_STATIC_LIMIT: return "size exceeds the fixed scratch of the allocation-free entry point (T > 65536)";
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
  ProfScope prof("dedup", static_cast<cudaStream_t>(stream));
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
  cudaError_t e;
  {
    ProfScope prof("gate_gemm", st);
    e = gemm(shape, T, F, d, x, false, W_gate, false, kEpiGate, gate, st);   // G = x W_gate^T, fused lookup
  }
  if (e != cudaSuccess) return cuda_fail(e);
  EpiParams down;
  down.out = y; down.out_fp32 = shape->dtype == STEM_DTYPE_FP32; down.status = status_of(ws);
  // few row tiles and a long contraction (decode steps): the tiles may be cut along k
  down.sk_scratch = static_cast<char*>(ws) + w.sk_off; down.sk_bytes = w.sk_bytes;
  {
    ProfScope prof("down_gemm", st);
    e = gemm(shape, T, d, F, H, false, W_down, false, kEpiStore, down, st);              // y = H W_down^T
  }
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
  cudaError_t e;
  {
    ProfScope prof("dh_gemm", st);
    e = gemm(shape, T, F, d, dy, false, W_down, true, kEpiDH, dh, st);
  }
  if (e != cudaSuccess) return cuda_fail(e);
  // Table gradient first: the tail of dU is still in L2 behind the dH kernel.
  if (dE_rows) {
    ProfScope prof("seg_reduce", st);
    e = launch_segreduce(T, F, shape->dtype, shape->grad_dtype, dU, perm, seg_offsets, n_unique, dE_rows,
                         base + w.part_off, st);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  EpiParams gp; gp.out_fp32 = grad_fp32; gp.status = status_of(ws);
  gp.accumulate = (shape->flags & STEM_FLAG_ACCUM_GRADS) != 0;
  gp.sk_scratch = base + w.sk_off; gp.sk_bytes = w.sk_bytes;
  if (dW_down && dW_gate && use_tc(shape)) {
    // dW_down[i,j] = sum_t dy[t,i] H[t,j] and dW_gate[j,k] = sum_t dG[t,j] x[t,k] in ONE launch: both
    // contract over the tokens, and their output tiles together fill the SMs (at the 350M shape
    // each has 44 tiles for 74 CTA pairs) with one split tail and one fix-up instead of two
    ProfScope prof("dw_pair_gemm", st);
    e = launch_tc_gemm_token_pair(T, d, F, dy, H_save, dW_down, F, d, dG, x, dW_gate, gp,
                                  !(shape->flags & STEM_FLAG_SINGLE_CTA), st);
    if (e != cudaSuccess) return cuda_fail(e);
  } else {
    if (dW_down) {  // dW_down[i,j] = sum_t dy[t,i] H[t,j]
      EpiParams p = gp; p.out = dW_down;
      ProfScope prof("dw_down_gemm", st);
      e = gemm(shape, d, F, T, dy, true, H_save, true, kEpiStore, p, st);
      if (e != cudaSuccess) return cuda_fail(e);
    }
    if (dW_gate) {  // dW_gate[j,k] = sum_t dG[t,j] x[t,k]
      EpiParams p = gp; p.out = dW_gate;
      ProfScope prof("dw_gate_gemm", st);
      e = gemm(shape, F, d, T, dG, true, x, true, kEpiStore, p, st);
      if (e != cudaSuccess) return cuda_fail(e);
    }
  }
  if (dx) {  // dx = dG W_gate (contraction over d_ff; W_gate is [F, d]: d contiguous)
    EpiParams p; p.out = dx; p.out_fp32 = shape->dtype == STEM_DTYPE_FP32; p.status = status_of(ws);
    p.sk_scratch = base + w.sk_off; p.sk_bytes = w.sk_bytes;
    ProfScope prof("dx_gemm", st);
    e = gemm(shape, T, d, F, dG, false, W_gate, true, kEpiStore, p, st);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  return STEM_OK;
}

// ---- table sharded over GPUs ---------------------------------------------------------------
int stem_shard_route_workspace_bytes(int32_t n_max, int32_t G, size_t* bytes) {
  if (!bytes || n_max < 0 || G < 1 || G > 1024) return STEM_ERR_INVALID_ARG;
  if (n_max > (1 << 22)) return STEM_ERR_UNSUPPORTED_SHAPE;
  *bytes = shard_route_workspace_bytes(n_max, G);
  return STEM_OK;
}

int stem_shard_route(int32_t n_max, int32_t T, int32_t G, const int32_t* unique_ids, const int32_t* n_unique,
                     const int32_t* inverse, int32_t* send_local, int32_t* send_slot, int32_t* send_counts,
                     int32_t* token_slot, void* route_ws, size_t route_ws_bytes, void* stream) {
  if (n_max < 0 || T < 0 || G < 1 || G > 1024) return STEM_ERR_INVALID_ARG;
  if (n_max > (1 << 22) || T > (1 << 22)) return STEM_ERR_UNSUPPORTED_SHAPE;
  if (!send_counts || !route_ws || !aligned16(route_ws)) return STEM_ERR_INVALID_ARG;
  if (n_max > 0 && (!unique_ids || !n_unique || !send_local || !send_slot)) return STEM_ERR_INVALID_ARG;
  if (token_slot && T > 0 && !inverse) return STEM_ERR_INVALID_ARG;
  if (route_ws_bytes < shard_route_workspace_bytes(n_max, G)) return STEM_ERR_WORKSPACE_TOO_SMALL;
  ProfScope prof("shard_route", static_cast<cudaStream_t>(stream));
  // no status word: the sort keys are made here and cannot be out of range
  cudaError_t e = launch_shard_route(n_max, T, G, unique_ids, n_unique, inverse, send_local, send_slot, send_counts,
                                     token_slot, route_ws, nullptr, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? STEM_OK : cuda_fail(e);
}

int stem_gather_rows(const stem_shape_t* shape, const int32_t* ids, const int32_t* n_ids, const void* table,
                     void* out, void* ws, void* stream) {
  if (int rc = check_shape(shape)) return rc;
  if (shape->T == 0) return STEM_OK;
  if (!ids || !n_ids || !table || !out || !aligned16(table) || !aligned16(out)) return STEM_ERR_INVALID_ARG;
  const void* src = nullptr;
  bool on_host = false;
  if (int rc = pinned_or_device(table, &src, &on_host)) return rc;
  const size_t row_bytes = static_cast<size_t>(shape->d_ff) * elem_bytes(shape->dtype);
  ProfScope prof("gather_rows", static_cast<cudaStream_t>(stream));
  cudaError_t e = launch_gather_rows(shape->T, shape->V, row_bytes, ids, n_ids, src, on_host, nullptr, nullptr, out,
                                     ws ? status_of(ws) : nullptr, nullptr, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? STEM_OK : cuda_fail(e);
}

int stem_reduce_rows(const stem_shape_t* shape, const void* rows_in, const int32_t* perm,
                     const int32_t* seg_offsets, const int32_t* n_unique, void* rows_out, void* ws,
                     size_t ws_bytes, void* stream) {
  if (int rc = check_shape(shape)) return rc;
  if (!ws || !aligned16(ws)) return STEM_ERR_INVALID_ARG;
  if (shape->T == 0) return STEM_OK;
  if (!rows_in || !perm || !seg_offsets || !n_unique || !rows_out || !aligned16(rows_in) || !aligned16(rows_out))
    return STEM_ERR_INVALID_ARG;
  const WsLayout w = ws_layout(shape);
  if (ws_bytes < w.total) return STEM_ERR_WORKSPACE_TOO_SMALL;
  ProfScope prof("reduce_rows", static_cast<cudaStream_t>(stream));
  cudaError_t e = launch_segreduce(shape->T, shape->d_ff, shape->grad_dtype, shape->grad_dtype, rows_in, perm,
                                   seg_offsets, n_unique, rows_out, static_cast<char*>(ws) + w.part_off,
                                   static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? STEM_OK : cuda_fail(e);
}

// ---- STEM-dagger: the up-projection is kept and the table row is added to its output -------
int stem_dagger_forward(const stem_shape_t* shape, const void* x, const int32_t* ids, const void* W_gate,
                        const void* W_up, const void* E, const void* W_down, void* y, void* G_save, void* H_save,
                        void* U_save, void* ws, size_t ws_bytes, void* stream) {
  if (int rc = check_shape(shape)) return rc;
  if (!ws || !aligned16(ws)) return STEM_ERR_INVALID_ARG;
  if (shape->T == 0) return STEM_OK;
  if (!x || !ids || !W_gate || !W_up || !E || !W_down || !y || !U_save) return STEM_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(W_gate) || !aligned16(W_up) || !aligned16(E) || !aligned16(W_down) || !aligned16(y) ||
      !aligned16(G_save) || !aligned16(H_save) || !aligned16(U_save))
    return STEM_ERR_INVALID_ARG;
  const WsLayout w = ws_layout(shape);
  if (ws_bytes < w.total) return STEM_ERR_WORKSPACE_TOO_SMALL;
  if (use_tc(shape) && !is_sm100()) return STEM_ERR_UNSUPPORTED_ARCH;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int T = shape->T, d = shape->d_model, F = shape->d_ff;
  void* H = H_save ? H_save : static_cast<char*>(ws) + w.h_off;
  cudaError_t e;
  if (use_tc(shape) && (shape->flags & STEM_FLAG_DAGGER_FUSED) && !(shape->flags & STEM_FLAG_SINGLE_CTA)) {
    // One kernel for both products of x: the gate and up tiles of the same x rows accumulate side
    // by side in tensor memory, and the epilogue forms U = up + E[ids], H = SiLU(gate) (.) U in
    // registers.  x is streamed once, and U reaches memory only as the copy backward needs.
    // Opt-in: two accumulator sets leave room for 128-column tiles only, every A block is then read
    // from shared memory once per product, and shared-memory bandwidth makes this launch about a
    // fifth slower than the two launches it replaces (measured at the 1B shape).
    EpiParams du;
    du.ids = ids; du.E = E; du.V = shape->V; du.H = H; du.G = G_save; du.U = U_save; du.status = status_of(ws);
    ProfScope prof("gate_up_gemm", st);
    e = launch_tc_gemm_dagger(T, F, d, x, W_gate, W_up, du, st);
    if (e != cudaSuccess) return cuda_fail(e);
  } else {
    {  // U = x W_up^T + E[ids]: the lookup is added in the up GEMM's epilogue
      EpiParams up;
      up.ids = ids; up.E = E; up.V = shape->V; up.H = U_save; up.status = status_of(ws);
      ProfScope prof("up_gemm", st);
      e = gemm(shape, T, F, d, x, false, W_up, false, kEpiAdd, up, st);
    }
    if (e != cudaSuccess) return cuda_fail(e);
    {  // G = x W_gate^T, H = SiLU(G) (.) U: the gate epilogue with U as a [T, d_ff] "table" indexed by position
      EpiParams gate;
      gate.ids = nullptr; gate.E = U_save; gate.V = T; gate.H = H; gate.G = G_save; gate.status = status_of(ws);
      ProfScope prof("gate_gemm", st);
      e = gemm(shape, T, F, d, x, false, W_gate, false, kEpiGate, gate, st);
    }
    if (e != cudaSuccess) return cuda_fail(e);
  }
  EpiParams down;
  down.out = y; down.out_fp32 = shape->dtype == STEM_DTYPE_FP32; down.status = status_of(ws);
  down.sk_scratch = static_cast<char*>(ws) + w.sk_off; down.sk_bytes = w.sk_bytes;
  {
    ProfScope prof("down_gemm", st);
    e = gemm(shape, T, d, F, H, false, W_down, false, kEpiStore, down, st);
  }
  return e == cudaSuccess ? STEM_OK : cuda_fail(e);
}

int stem_dagger_backward(const stem_shape_t* shape, const void* dy, const void* x, const void* W_gate,
                         const void* W_up, const void* W_down, const void* G_save, const void* H_save,
                         const void* U_save, const int32_t* perm, const int32_t* seg_offsets,
                         const int32_t* n_unique, void* dx, void* dW_gate, void* dW_up, void* dW_down, void* dE_rows,
                         void* ws, size_t ws_bytes, void* stream) {
  if (int rc = check_shape(shape)) return rc;
  if (!ws || !aligned16(ws)) return STEM_ERR_INVALID_ARG;
  if (shape->T == 0) return STEM_OK;
  if (!dy || !x || !W_gate || !W_up || !W_down || !G_save || !U_save) return STEM_ERR_INVALID_ARG;
  if (dW_down && !H_save) return STEM_ERR_INVALID_ARG;
  if (dE_rows && (!perm || !seg_offsets || !n_unique)) return STEM_ERR_INVALID_ARG;
  if (!aligned16(dy) || !aligned16(x) || !aligned16(W_gate) || !aligned16(W_up) || !aligned16(W_down) ||
      !aligned16(G_save) || !aligned16(H_save) || !aligned16(U_save) || !aligned16(dx) || !aligned16(dW_gate) ||
      !aligned16(dW_up) || !aligned16(dW_down) || !aligned16(dE_rows))
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
  cudaError_t e;
  {  // dH = dy W_down; dU = dH SiLU(G) (gradient of U = W_up x + E[ids]); dG = dH U SiLU'(G)
    EpiParams dh;
    dh.ids = nullptr; dh.E = U_save; dh.V = T; dh.H = dU; dh.G = dG; dh.Gin = G_save; dh.status = status_of(ws);
    ProfScope prof("dh_gemm", st);
    e = gemm(shape, T, F, d, dy, false, W_down, true, kEpiDH, dh, st);
  }
  if (e != cudaSuccess) return cuda_fail(e);
  auto grad = [&](const char* name, void* out, int M, int N, const void* A, const void* Bm) {
    EpiParams p; p.out = out; p.out_fp32 = grad_fp32; p.status = status_of(ws);
    p.accumulate = (shape->flags & STEM_FLAG_ACCUM_GRADS) != 0;
    p.sk_scratch = base + w.sk_off; p.sk_bytes = w.sk_bytes;
    ProfScope prof(name, st);
    return gemm(shape, M, N, T, A, true, Bm, true, kEpiStore, p, st);   // contraction over the tokens
  };
  if (dW_down && (e = grad("dw_down_gemm", dW_down, d, F, dy, H_save)) != cudaSuccess) return cuda_fail(e);
  if (dE_rows) {
    ProfScope prof("seg_reduce", st);
    e = launch_segreduce(T, F, shape->dtype, shape->grad_dtype, dU, perm, seg_offsets, n_unique, dE_rows,
                         base + w.part_off, st);
    if (e != cudaSuccess) return cuda_fail(e);
  }
  if (dW_gate && (e = grad("dw_gate_gemm", dW_gate, F, d, dG, x)) != cudaSuccess) return cuda_fail(e);
  if (dW_up && (e = grad("dw_up_gemm", dW_up, F, d, dU, x)) != cudaSuccess) return cuda_fail(e);
  if (dx) {  // dx = dG W_gate + dU W_up: the second product is added onto the first in its epilogue
    EpiParams p; p.out = dx; p.out_fp32 = shape->dtype == STEM_DTYPE_FP32; p.status = status_of(ws);
    {
      ProfScope prof("dx_gemm", st);
      e = gemm(shape, T, d, F, dG, false, W_gate, true, kEpiStore, p, st);
    }
    if (e != cudaSuccess) return cuda_fail(e);
    EpiParams a; a.ids = nullptr; a.E = dx; a.V = T; a.H = dx; a.status = status_of(ws);
    ProfScope prof("dx_up_gemm", st);
    e = gemm(shape, T, d, F, dU, false, W_up, true, kEpiAdd, a, st);
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
  bool on_host = false;
  if (int rc = pinned_or_device(table, &src, &on_host)) return rc;
  const int max_rows = shape->T < shape->V ? shape->T : shape->V;
  const size_t row_bytes = static_cast<size_t>(shape->d_ff) * elem_bytes(shape->dtype);
  ProfScope prof("prefetch_rows", static_cast<cudaStream_t>(stream));
  cudaError_t e = launch_gather_rows(max_rows, shape->V, row_bytes, ids, n_ids, src, on_host, nullptr, nullptr,
                                     dev_cache, ws ? status_of(ws) : nullptr, nullptr,
                                     static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? STEM_OK : cuda_fail(e);
}

int stem_prefetch_rows_hot(const stem_shape_t* shape, const int32_t* ids, const int32_t* n_ids, const void* table,
                           const void* hot_rows, const int32_t* hot_slot, void* dev_cache, int32_t* stats, void* ws,
                           void* stream) {
  if (int rc = check_shape(shape)) return rc;
  if (shape->T == 0) return STEM_OK;
  if (!ids || !n_ids || !table || !dev_cache || !hot_rows || !hot_slot || !aligned16(table) || !aligned16(dev_cache) ||
      !aligned16(hot_rows))
    return STEM_ERR_INVALID_ARG;
  const void* src = nullptr;
  bool on_host = false;
  if (int rc = pinned_or_device(table, &src, &on_host)) return rc;
  const int max_rows = shape->T < shape->V ? shape->T : shape->V;
  const size_t row_bytes = static_cast<size_t>(shape->d_ff) * elem_bytes(shape->dtype);
  ProfScope prof("prefetch_rows", static_cast<cudaStream_t>(stream));
  cudaError_t e = launch_gather_rows(max_rows, shape->V, row_bytes, ids, n_ids, src, on_host, hot_rows, hot_slot,
                                     dev_cache, ws ? status_of(ws) : nullptr, stats, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? STEM_OK : cuda_fail(e);
}

int stem_lfu_workspace_bytes(int32_t V, int32_t K, size_t* bytes) {
  if (!bytes || V <= 0 || K <= 0 || K > V || V > (1 << 30)) return STEM_ERR_INVALID_ARG;
  *bytes = lfu_workspace_bytes(V, K);
  return STEM_OK;
}

int stem_lfu_touch(int32_t n, int32_t V, const int32_t* ids, int32_t* freq, const int32_t* hot_slot,
                   int32_t* stats, void* stream) {
  if (n < 0 || V <= 0) return STEM_ERR_INVALID_ARG;
  if (n == 0) return STEM_OK;
  if (!ids || !freq || !hot_slot) return STEM_ERR_INVALID_ARG;
  ProfScope prof("lfu_touch", static_cast<cudaStream_t>(stream));
  cudaError_t e = launch_lfu_touch(n, V, ids, freq, hot_slot, stats, nullptr, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? STEM_OK : cuda_fail(e);
}

int stem_lfu_refresh(const stem_shape_t* shape, int32_t K, const int32_t* freq, int32_t* hot_slot, int32_t* hot_ids,
                     void* hot_rows, const void* table, int32_t* n_installed, void* lfu_ws, size_t lfu_ws_bytes,
                     void* stream) {
  if (int rc = check_shape(shape)) return rc;
  if (K <= 0 || K > shape->V || !freq || !hot_slot || !hot_ids || !hot_rows || !table || !lfu_ws ||
      !aligned16(hot_rows) || !aligned16(table) || !aligned16(lfu_ws))
    return STEM_ERR_INVALID_ARG;
  if (lfu_ws_bytes < lfu_workspace_bytes(shape->V, K)) return STEM_ERR_WORKSPACE_TOO_SMALL;
  const void* src = nullptr;
  if (int rc = pinned_or_device(table, &src)) return rc;
  const size_t row_bytes = static_cast<size_t>(shape->d_ff) * elem_bytes(shape->dtype);
  ProfScope prof("lfu_refresh", static_cast<cudaStream_t>(stream));
  cudaError_t e = launch_lfu_refresh(shape->V, K, row_bytes, freq, hot_slot, hot_ids, hot_rows, src, n_installed, lfu_ws,
                                     static_cast<cudaStream_t>(stream));
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
  ProfScope prof("writeback_rows", static_cast<cudaStream_t>(stream));
  cudaError_t e = launch_writeback_rows(max_rows, row_bytes, dE_rows, unique_ids, n_rows, const_cast<void*>(hr),
                                        static_cast<int32_t*>(const_cast<void*>(hi)),
                                        static_cast<int32_t*>(const_cast<void*>(hn)), nullptr,
                                        static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? STEM_OK : cuda_fail(e);
}

int stem_writeback_rows_dma(const stem_shape_t* shape, const void* dE_rows, const int32_t* unique_ids,
                            int32_t n_rows, void* host_rows, int32_t* host_ids, void* stream) {
  if (int rc = check_shape(shape)) return rc;
  const int max_rows = shape->T < shape->V ? shape->T : shape->V;
  if (n_rows < 0 || n_rows > max_rows) return STEM_ERR_INVALID_ARG;
  if (n_rows == 0) return STEM_OK;
  if (!dE_rows || !unique_ids || !host_rows || !host_ids) return STEM_ERR_INVALID_ARG;
  const void* unused = nullptr;
  if (int rc = pinned_or_device(host_rows, &unused)) return rc;
  if (int rc = pinned_or_device(host_ids, &unused)) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t row_bytes = static_cast<size_t>(shape->d_ff) * elem_bytes(shape->grad_dtype);
  ProfScope prof("writeback_rows", st);
  cudaError_t e = cudaMemcpyAsync(host_rows, dE_rows, row_bytes * n_rows, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(host_ids, unique_ids, sizeof(int32_t) * static_cast<size_t>(n_rows), cudaMemcpyDeviceToHost, st);
  return e == cudaSuccess ? STEM_OK : cuda_fail(e);
}

int stem_gemm_bf16(int32_t M, int32_t N, int32_t K, const void* A, int32_t a_mn, const void* B, int32_t b_mn,
                   void* C, int32_t c_fp32, int32_t flags, void* ws, void* stream) {
  if (M < 0 || N < 0 || K <= 0) return STEM_ERR_INVALID_ARG;
  if (M == 0 || N == 0) return STEM_OK;
  if (!A || !B || !C || !ws || !aligned16(A) || !aligned16(B) || !aligned16(C)) return STEM_ERR_INVALID_ARG;
  if ((N % 8) || ((a_mn ? M : K) % 8) || ((b_mn ? N : K) % 8)) return STEM_ERR_UNSUPPORTED_SHAPE;
  EpiParams p; p.out = C; p.out_fp32 = c_fp32; p.status = status_of(ws);
  cudaError_t e;
  if (flags & STEM_FLAG_SIMT) {
    e = launch_simt_gemm(STEM_DTYPE_BF16, M, N, K, A, a_mn != 0, B, b_mn != 0, kEpiStore, p, static_cast<cudaStream_t>(stream));
  } else {
    if (!is_sm100()) return STEM_ERR_UNSUPPORTED_ARCH;
    e = launch_tc_gemm(M, N, K, A, a_mn != 0, B, b_mn != 0, kEpiStore, p, !(flags & STEM_FLAG_SINGLE_CTA),
                       static_cast<cudaStream_t>(stream));
  }
  return e == cudaSuccess ? STEM_OK : cuda_fail(e);
}

int stem_selftest_wait(void* ws, long long limit_cycles, int arrive, void* stream) {
  if (!ws || !aligned16(ws)) return STEM_ERR_INVALID_ARG;
  if (limit_cycles < 1 || limit_cycles > 2000000000ll) return STEM_ERR_INVALID_ARG;
  cudaError_t e = launch_selftest_wait(status_of(ws), limit_cycles, arrive, static_cast<cudaStream_t>(stream));
  return e == cudaSuccess ? STEM_OK : cuda_fail(e);
}

long long stem_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int stem_profile_enable(int on) {
  std::lock_guard<std::mutex> lock(g_prof_mutex);
  if (on) {
    // every end event once, and the begin events that are not some record's end event
    for (size_t i = 0; i < g_prof.size(); ++i) {
      g_event_pool.push_back(g_prof[i].end);
      if (i == 0 || g_prof[i].begin != g_prof[i - 1].end) g_event_pool.push_back(g_prof[i].begin);
    }
    g_prof.clear();
    g_prof_last_end = nullptr;
  }
  g_prof_on = on != 0;
  return STEM_OK;
}

int stem_profile_count(void) {
  std::lock_guard<std::mutex> lock(g_prof_mutex);
  return static_cast<int>(g_prof.size());
}

int stem_profile_get(int i, const char** name, float* ms) {
  std::lock_guard<std::mutex> lock(g_prof_mutex);
  if (i < 0 || i >= static_cast<int>(g_prof.size()) || !name || !ms) return STEM_ERR_INVALID_ARG;
  cudaError_t e = cudaEventSynchronize(g_prof[i].end);
  if (e == cudaSuccess) e = cudaEventElapsedTime(ms, g_prof[i].begin, g_prof[i].end);
  if (e != cudaSuccess) return cuda_fail(e);
  *name = g_prof[i].name;
  return STEM_OK;
}

namespace {
// Arena of the host-buffer step: the workspace, the saved activations and index arrays, and
// TWO slots of input (x, dy, ids) and output (y, dx) buffers, so the copies of one call
// overlap the kernels of its neighbours.
struct Arena {
  size_t ws, ws_bytes, x[2], dy[2], ids[2], y[2], dx[2], n_u[2], G, H, inverse, perm, seg, total;
};
Arena arena_layout(const stem_shape_t* s) {
  Arena a{};
  const size_t T = s->T, td = align_up(T * s->d_model * elem_bytes(s->dtype), 256),
               tf = align_up(T * s->d_ff * elem_bytes(s->dtype), 256), ti = align_up((T + 1) * 4, 256);
  const size_t R = static_cast<size_t>(s->T < s->V ? s->T : s->V);
  size_t o = 0;
  a.ws = o; a.ws_bytes = ws_layout(s).total; o += a.ws_bytes;
  for (int k = 0; k < 2; ++k) {
    a.x[k] = o; o += td;  a.dy[k] = o; o += td;  a.ids[k] = o; o += ti;
    a.y[k] = o; o += td;  a.dx[k] = o; o += td;
    a.n_u[k] = o; o += 256;   // this call's row count, kept until its copy to the host has run
  }
  a.G = o; o += tf;  a.H = o; o += tf;
  a.inverse = o; o += ti;  a.perm = o; o += ti;  a.seg = o; o += align_up((R + 1) * 4, 256);
  a.total = o;
  return a;
}

// Copy streams and hand-over events of the host-buffer step, one set per device, created on
// first use (host-side objects; no device memory).
struct StepPipe {
  bool ready = false;
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t x_in[2], dy_in[2], y_done[2], bwd_done[2], out_done[2];
  bool used[2] = {false, false};
  unsigned long long calls = 0;
};
std::mutex g_pipe_mutex;
StepPipe g_pipe[64];

cudaError_t pipe_get(StepPipe** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
  StepPipe& p = g_pipe[dev];
  if (!p.ready) {
    if ((e = cudaStreamCreateWithFlags(&p.in, cudaStreamNonBlocking)) != cudaSuccess) return e;
    if ((e = cudaStreamCreateWithFlags(&p.out, cudaStreamNonBlocking)) != cudaSuccess) return e;
    for (int k = 0; k < 2; ++k)
      for (cudaEvent_t* ev : {&p.x_in[k], &p.dy_in[k], &p.y_done[k], &p.bwd_done[k], &p.out_done[k]})
        if ((e = cudaEventCreateWithFlags(ev, cudaEventDisableTiming)) != cudaSuccess) return e;
    p.ready = true;
  }
  *out = &p;
  return cudaSuccess;
}
}  // namespace

int stem_step_arena_bytes(const stem_shape_t* shape, size_t* bytes) {
  if (!bytes) return STEM_ERR_INVALID_ARG;
  if (int rc = check_shape(shape)) return rc;
  *bytes = arena_layout(shape).total;
  return STEM_OK;
}

int stem_ffn_step_host(const stem_shape_t* shape, const void* host_x, const int32_t* host_ids, const void* host_dy,
                       const void* W_gate, const void* E, const void* W_down, void* host_y, void* host_dx,
                       void* dW_gate, void* dW_down, void* dE_rows, int32_t* unique_ids, int32_t* n_unique,
                       int32_t* host_n_unique, void* arena, size_t arena_bytes, void* stream) {
  if (int rc = check_shape(shape)) return rc;
  if (!arena || !aligned16(arena)) return STEM_ERR_INVALID_ARG;
  if (shape->T == 0) return STEM_OK;
  if (!host_x || !host_ids || !host_dy || !host_y || !host_dx || !unique_ids || !n_unique) return STEM_ERR_INVALID_ARG;
  const Arena a = arena_layout(shape);
  if (arena_bytes < a.total) return STEM_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  StepPipe* pp = nullptr;
  cudaError_t e = pipe_get(&pp);
  if (e != cudaSuccess) return cuda_fail(e);
  StepPipe& p = *pp;
  const int k = static_cast<int>(p.calls++ & 1);   // slot of this call
  char* base = static_cast<char*>(arena);
  const size_t td = static_cast<size_t>(shape->T) * shape->d_model * elem_bytes(shape->dtype);
  int32_t* ids = reinterpret_cast<int32_t*>(base + a.ids[k]);
  int32_t* perm = reinterpret_cast<int32_t*>(base + a.perm);
  int32_t* seg = reinterpret_cast<int32_t*>(base + a.seg);
#define STEP_CUDA(call) do { e = (call); if (e != cudaSuccess) return cuda_fail(e); } while (0)
  // inputs: the slot is free once the backward pass of the call that used it last is done
  if (p.used[k]) STEP_CUDA(cudaStreamWaitEvent(p.in, p.bwd_done[k], 0));
  {
    ProfScope prof("h2d_inputs", p.in);
    STEP_CUDA(cudaMemcpyAsync(ids, host_ids, static_cast<size_t>(shape->T) * 4, cudaMemcpyHostToDevice, p.in));
    STEP_CUDA(cudaMemcpyAsync(base + a.x[k], host_x, td, cudaMemcpyHostToDevice, p.in));
    STEP_CUDA(cudaEventRecord(p.x_in[k], p.in));
    STEP_CUDA(cudaMemcpyAsync(base + a.dy[k], host_dy, td, cudaMemcpyHostToDevice, p.in));
    STEP_CUDA(cudaEventRecord(p.dy_in[k], p.in));
  }
  // compute on the caller's stream; y/dx of this slot must have left for the host first
  STEP_CUDA(cudaStreamWaitEvent(st, p.x_in[k], 0));
  if (p.used[k]) STEP_CUDA(cudaStreamWaitEvent(st, p.out_done[k], 0));
  if (int rc = stem_dedup_ids(shape, ids, unique_ids, n_unique, reinterpret_cast<int32_t*>(base + a.inverse), perm, seg,
                              base + a.ws, a.ws_bytes, stream)) return rc;
  if (int rc = stem_ffn_forward(shape, base + a.x[k], ids, W_gate, E, W_down, base + a.y[k], base + a.G, base + a.H,
                                base + a.ws, a.ws_bytes, stream)) return rc;
  STEP_CUDA(cudaEventRecord(p.y_done[k], st));
  STEP_CUDA(cudaStreamWaitEvent(st, p.dy_in[k], 0));
  if (int rc = stem_ffn_backward(shape, base + a.dy[k], base + a.x[k], ids, W_gate, E, W_down, base + a.G, base + a.H,
                                 perm, seg, n_unique, base + a.dx[k], dW_gate, dW_down, dE_rows, unique_ids,
                                 base + a.ws, a.ws_bytes, stream)) return rc;
  // The caller's n_unique scalar is rewritten by the next call's dedup long before this call's
  // output copies run: the count that goes to the host is taken from a word of this slot (copied
  // here, behind the last kernel, where the stream has an event boundary anyway).
  if (host_n_unique) STEP_CUDA(cudaMemcpyAsync(base + a.n_u[k], n_unique, 4, cudaMemcpyDeviceToDevice, st));
  STEP_CUDA(cudaEventRecord(p.bwd_done[k], st));
  // outputs
  STEP_CUDA(cudaStreamWaitEvent(p.out, p.y_done[k], 0));
  {
    ProfScope prof("d2h_outputs", p.out);
    STEP_CUDA(cudaMemcpyAsync(host_y, base + a.y[k], td, cudaMemcpyDeviceToHost, p.out));
    STEP_CUDA(cudaStreamWaitEvent(p.out, p.bwd_done[k], 0));
    STEP_CUDA(cudaMemcpyAsync(host_dx, base + a.dx[k], td, cudaMemcpyDeviceToHost, p.out));
    if (host_n_unique) STEP_CUDA(cudaMemcpyAsync(host_n_unique, base + a.n_u[k], 4, cudaMemcpyDeviceToHost, p.out));
  }
  STEP_CUDA(cudaEventRecord(p.out_done[k], p.out));
  p.used[k] = true;
  return STEM_OK;
}

int stem_ffn_step_host_flush(void* stream) {
  std::lock_guard<std::mutex> lock(g_pipe_mutex);
  StepPipe* pp = nullptr;
  cudaError_t e = pipe_get(&pp);
  if (e != cudaSuccess) return cuda_fail(e);
  for (int k = 0; k < 2; ++k)
    if (pp->used[k]) STEP_CUDA(cudaStreamWaitEvent(static_cast<cudaStream_t>(stream), pp->out_done[k], 0));
#undef STEP_CUDA
  return STEM_OK;
}

}  // extern "C"
