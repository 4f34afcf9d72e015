/*
 * libstem -- the STEM feed-forward layer on NVIDIA B200 (sm_100a), C ABI.
 *
 * The layer (paper Section 3.1, "STEM", the layer equation):
 *
 *     y_t = W_down ( SiLU(W_gate x_t) (.) E[id_t] )          for every position t
 *
 * with W_gate in R^{d_ff x d_model}, W_down in R^{d_model x d_ff} (orientations of
 * Section 2, "Background") and a layer-local table E in R^{V x d_ff} (the paper's U_l)
 * that replaces the dense up-projection of a SwiGLU block.  SiLU(z) = z * sigmoid(z);
 * no bias terms (Table 1 caption); token ids are 0-based.
 *
 * Conventions shared by every entry point
 *   - All matrices are dense row-major: x,y,dy,dx [T,d_model]; W_gate,dW_gate
 *     [d_ff,d_model]; W_down,dW_down [d_model,d_ff]; E [V,d_ff]; G,H [T,d_ff].
 *   - Unless a parameter says "host", pointers are device pointers, 16-byte aligned.
 *     The caller owns every buffer, the workspace included.  The library allocates no
 *     device memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls
 *     only enqueue work; they do not synchronise unless stated.  Calls are re-entrant across
 *     distinct workspaces.  On ONE workspace, issue them on one stream in the documented order:
 *     the regions of a workspace are shared between calls (stem_dedup_ids' sort scratch, the H
 *     of a forward call that was given no H_save, and backward's dU / dG all start at the same
 *     offset), so e.g. stem_dedup_ids on a workspace destroys an unsaved H that still lives in it.
 *   - Outputs are overwritten, except the weight gradients under STEM_FLAG_ACCUM_GRADS.
 *   - Return value: STEM_OK or a negative STEM_ERR_* code.  Conditions only the device
 *     can see (an id outside [0,V), a pipeline wait that ran out) are recorded in the
 *     workspace's status word and read back with stem_query_status().  A bad id is
 *     clamped into range so no access leaves the table.  Nothing traps, prints from the
 *     device or throws; there is no CPU fallback.
 *   - dtype 0: fp32 storage and fp32 FMA arithmetic.  dtype 1: bf16 storage, bf16
 *     tensor-core products accumulated in fp32, elementwise math in fp32, results
 *     rounded to bf16 (round to nearest even) when stored.
 *   - Shape limits: T <= 2^22; d_model and d_ff multiples of 8 (bf16) or 4 (fp32);
 *     V <= 2^30.  T = 0 is accepted by every call and does nothing.
 */
#ifndef STEM_H_
#define STEM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define STEM_OK 0
#define STEM_ERR_INVALID_ARG (-1)
#define STEM_ERR_UNSUPPORTED_SHAPE (-2)
#define STEM_ERR_UNSUPPORTED_ARCH (-3)
#define STEM_ERR_WORKSPACE_TOO_SMALL (-4)
#define STEM_ERR_NOT_PINNED (-5)
#define STEM_ERR_CUDA (-6)
#define STEM_ERR_TIMEOUT (-7)  /* device: a bounded pipeline wait expired          */
#define STEM_ERR_ID_RANGE (-8) /* device: a token id was outside [0,V) (clamped)  */
#define STEM_ERR_STATIC_LIMIT (-9) /* size beyond the fixed scratch of an allocation-free call */
#define STEM_ERR_COUNT_RANGE (-10) /* device: a row count (device scalar) exceeded the buffers' capacity (clamped) */

#define STEM_DTYPE_FP32 0
#define STEM_DTYPE_BF16 1

#define STEM_FLAG_SIMT 1 /* run the bf16 contractions on the plain-FMA kernels (debug aid) */
#define STEM_FLAG_SINGLE_CTA 2 /* tensor-core contractions on single CTAs instead of CTA pairs (debug aid) */
/* Backward adds the weight gradients (dW_gate, dW_down, and dW_up of the dagger variant) to what
 * the caller's buffers hold instead of overwriting them: gradient accumulation over
 * micro-batches.  Not a step of the paper's method; dx and dE_rows are still overwritten (the
 * rows of dE_rows belong to this call's unique ids).  With bf16 gradients the product is rounded
 * to bf16 before the bf16 add. */
#define STEM_FLAG_ACCUM_GRADS 4
/* stem_dagger_forward: compute the gate and up products of x in ONE launch with two accumulators in
 * tensor memory (U = up + E[ids] and H = SiLU(gate) (.) U formed in its epilogue) instead of two
 * launches that pass U through memory.  Same results within rounding (H is formed from the
 * unrounded U).  Saves one pass over x and one read of U; measured slower on B200 at the 1B shape
 * (the tile must shrink to 256 x 128 per product and shared-memory bandwidth binds), so it is off by
 * default.  CTA pairs only: ignored with STEM_FLAG_SINGLE_CTA or STEM_FLAG_SIMT. */
#define STEM_FLAG_DAGGER_FUSED 8

typedef struct {
  int32_t T;          /* positions in this call (batch x sequence)                 */
  int32_t d_model;    /* d                                                          */
  int32_t d_ff;       /* F                                                          */
  int32_t V;          /* rows of E addressable by ids                               */
  int32_t dtype;      /* STEM_DTYPE_*: x, y, dy, dx, W_gate, W_down, E, G, H        */
  int32_t grad_dtype; /* STEM_DTYPE_*: dW_gate, dW_down, dE_rows                    */
  int32_t flags;      /* STEM_FLAG_* bits                                           */
} stem_shape_t;

/* Library version, major*10000 + minor*100 + patch. */
int stem_version(void);

/* Text for a STEM_ERR_* code (static storage). */
const char* stem_status_string(int code);

/* Bytes of workspace that any call with this shape needs (the maximum over calls).
 * The first 256 bytes of a workspace hold the status word. */
int stem_workspace_bytes(const stem_shape_t* shape, size_t* bytes /*host, out*/);

/* Clear the status word.  Call once after allocating a workspace (and to re-arm it
 * after an error was read). */
int stem_init_workspace(void* ws, size_t ws_bytes, void* stream);

/* Synchronises `stream`, then copies the status word to *status_out (host):
 * STEM_OK, STEM_ERR_TIMEOUT, STEM_ERR_ID_RANGE or STEM_ERR_COUNT_RANGE.  The word is sticky: the first
 * error stays until stem_init_workspace(). */
int stem_query_status(const void* ws, void* stream, int32_t* status_out /*host*/);

/*
 * Token deduplication (Section 3.4 "System Implementation": the batch's token ids are
 * deduplicated so only uniq(B*L) rows move; Table 1, "Communication").  The paper
 * names the step; the arrays are defined here, each with exactly one correct value:
 *   perm[T]          positions sorted by (ids[t], t) ascending (stable radix sort by id)
 *   unique_ids[n_u]  the distinct ids, ascending
 *   seg_offsets[n_u+1]  index in perm where each id's run starts; seg_offsets[n_u] = T
 *   inverse[T]       inverse[t] = r with unique_ids[r] == ids[t]
 *   n_unique         device scalar n_u
 * unique_ids needs room for min(T,V) entries, seg_offsets for min(T,V)+1.  `inverse`
 * may be NULL.  Entries past n_u are left untouched.
 */
int stem_dedup_ids(const stem_shape_t* shape, const int32_t* ids, int32_t* unique_ids,
                   int32_t* n_unique, int32_t* inverse, int32_t* perm, int32_t* seg_offsets,
                   void* ws, size_t ws_bytes, void* stream);

/*
 * stem_dedup_ids for callers that cannot allocate device memory (the paper has no
 * counterpart; this is a deployment aid).  Think of an inference server whose framework
 * claimed all of HBM for weights and KV cache at start-up, a plug-in invoked from inside
 * another runtime that forbids allocation on its threads, or a latency-critical loop in
 * which a cudaMalloc would stall every stream of the device: none of them can produce
 * the workspace stem_dedup_ids wants.  Here the sort's scratch is a fixed 1.25 MiB array
 * compiled into the library (held by every GPU that loads it, until the process exits),
 * so the call takes inputs and outputs only and calls no allocator of any kind.
 *   - Same outputs, bit for bit, as stem_dedup_ids.  Only shape->T and shape->V are read.
 *   - Limit: T <= stem_dedup_static_max_tokens() (65536); larger T returns
 *     STEM_ERR_STATIC_LIMIT and launches nothing.
 *   - status: optional device int32[4], zeroed by the caller; receives STEM_ERR_ID_RANGE
 *     if an id is outside [0,V) (ids are clamped either way).  NULL = not reported.
 *   - The first call on each device looks up the array's device address; make that first
 *     call before starting any stream capture on that device.
 *   - All calls on a device share the one array: two calls whose kernels can overlap on
 *     the GPU (different streams, no ordering between them) race.  Order them.  The array
 *     keeps the previous call's contents; nothing in it needs clearing between calls.
 */
int stem_dedup_ids_static(const stem_shape_t* shape, const int32_t* ids, int32_t* unique_ids,
                          int32_t* n_unique, int32_t* inverse, int32_t* perm, int32_t* seg_offsets,
                          int32_t* status, void* stream);
int stem_dedup_static_max_tokens(void);

/*
 * Forward (Section 3.1, the layer equation).  Two kernels:
 *   G = x W_gate^T, H = SiLU(G) (.) E[ids]   -- the row lookup is fused in the GEMM's
 *                                               epilogue; E[ids] is never materialised
 *   y = H W_down^T
 * G_save, H_save: optional [T,d_ff] outputs (dtype) kept for backward; either may be
 * NULL (H then lives in the workspace).  With a prefetched row cache, pass
 * ids := inverse and E := dev_cache with shape->V = rows of the cache.
 */
int stem_ffn_forward(const stem_shape_t* shape, const void* x, const int32_t* ids,
                     const void* W_gate, const void* E, const void* W_down, void* y,
                     void* G_save, void* H_save, void* ws, size_t ws_bytes, void* stream);

/*
 * Backward.  The paper states no formulas (training is implied: Table 1 notes, Section
 * 3.4); these are the chain rule of the layer equation for L = sum dy (.) y:
 *   dH = dy W_down;  dU = dH (.) SiLU(G);  dG = dH (.) E[ids] (.) SiLU'(G)
 *   dW_down = dy^T H;  dW_gate = dG^T x;  dx = dG W_gate
 *   dE_rows[r] = sum of dU[t] over the positions t with ids[t] == unique_ids[r]
 *                (fixed summation order: the result is bitwise reproducible)
 * When both weight gradients are asked for, the two token-contracted products run as one launch
 * whose tiles share the SMs.
 * G_save, H_save: what stem_ffn_forward saved (required).  perm, seg_offsets, n_unique,
 * unique_ids: from stem_dedup_ids on the same ids.  dE_rows [min(T,V), d_ff]
 * (grad_dtype): rows >= n_u are left untouched; ids absent from the call have no row
 * (their gradient is zero).  dW_gate, dW_down in grad_dtype; dx in dtype.  Any of dx,
 * dW_gate, dW_down, dE_rows may be NULL to skip that output.  With STEM_FLAG_ACCUM_GRADS in
 * shape->flags, dW_gate and dW_down are added to instead of overwritten.
 */
int stem_ffn_backward(const stem_shape_t* shape, const void* dy, const void* x, const int32_t* ids,
                      const void* W_gate, const void* E, const void* W_down, const void* G_save,
                      const void* H_save, const int32_t* perm, const int32_t* seg_offsets,
                      const int32_t* n_unique, void* dx, void* dW_gate, void* dW_down,
                      void* dE_rows, const int32_t* unique_ids, void* ws, size_t ws_bytes,
                      void* stream);

/*
 * STEM-dagger (Appendix, "Additional Architecture Ablation Study": the variant that keeps the
 * up-projection and adds the token's table row to its output):
 *     y_t = W_down ( SiLU(W_gate x_t) (.) (W_up x_t + E[id_t]) )
 * Forward: U = x W_up^T + E[ids] (the lookup is added in the up GEMM's epilogue), G = x W_gate^T,
 * H = SiLU(G) (.) U, y = H W_down^T (STEM_FLAG_DAGGER_FUSED: the first three in one launch).  W_up [d_ff,d_model] like W_gate.  U_save [T,d_ff] (dtype) is
 * a required output (the backward pass needs it); G_save, H_save as in stem_ffn_forward.
 * Backward (chain rule, as for the layer itself): dH = dy W_down; dU = dH (.) SiLU(G);
 * dG = dH (.) U (.) SiLU'(G); dW_down = dy^T H; dW_gate = dG^T x; dW_up = dU^T x;
 * dx = dG W_gate + dU W_up; dE_rows[r] = sum of dU[t] over the positions of unique_ids[r].
 * perm, seg_offsets, n_unique from stem_dedup_ids; any of dx, dW_gate, dW_up, dW_down, dE_rows
 * may be NULL.  Same workspace as the layer's calls.
 */
int stem_dagger_forward(const stem_shape_t* shape, const void* x, const int32_t* ids, const void* W_gate,
                        const void* W_up, const void* E, const void* W_down, void* y, void* G_save,
                        void* H_save, void* U_save, void* ws, size_t ws_bytes, void* stream);
int stem_dagger_backward(const stem_shape_t* shape, const void* dy, const void* x, const void* W_gate,
                         const void* W_up, const void* W_down, const void* G_save, const void* H_save,
                         const void* U_save, const int32_t* perm, const int32_t* seg_offsets,
                         const int32_t* n_unique, void* dx, void* dW_gate, void* dW_up, void* dW_down,
                         void* dE_rows, void* ws, size_t ws_bytes, void* stream);

/*
 * Row prefetch for a table kept off the device (Section 3.4: tables offloaded to CPU
 * memory, rows of the deduplicated ids prefetched asynchronously with layer compute;
 * Figure 1(c)):   dev_cache[r,:] = table[ids[r],:]   for r < *n_ids.
 * table: [V,d_ff] (dtype) in page-locked host memory (cudaHostAlloc / cudaHostRegister;
 * checked, else STEM_ERR_NOT_PINNED) or in device memory (a compact on-device gather).
 * ids: device, normally unique_ids; n_ids: device scalar, so no host round trip is
 * needed between dedup and prefetch.  dev_cache: device [min(T,V), d_ff].  Run it on a
 * side stream to overlap the previous layer's GEMMs.  A count outside [0, min(T,V)] is clamped
 * to the cache's capacity and recorded in the status word as STEM_ERR_COUNT_RANGE (ws not NULL).
 */
int stem_prefetch_rows(const stem_shape_t* shape, const int32_t* ids, const int32_t* n_ids,
                       const void* table, void* dev_cache, void* ws, void* stream);

/*
 * Row prefetch with an on-device hot set (Section 3.2.4, "Prefetching cost": traffic is cut
 * further by caching the most frequently used embeddings in the memory the removed
 * up-projection frees; Section 3.4 names an LFU cache).  As stem_prefetch_rows, but a row
 * whose id has a slot in the hot set is copied from device memory instead of the table:
 *   dev_cache[r,:] = hot_slot[ids[r]] >= 0 ? hot_rows[hot_slot[ids[r]],:] : table[ids[r],:]
 * hot_rows: device [K,d_ff] (dtype), copies of table rows; hot_slot: device int32 [V], slot of
 * each id or -1.  Which rows to keep hot (and replacing them as frequencies drift) is the
 * caller's policy; the result equals stem_prefetch_rows' whenever hot_rows mirrors the table.
 * stats: optional device int32[2], incremented by the number of rows served from the hot
 * set ([0]) and from the table ([1]).
 */
int stem_prefetch_rows_hot(const stem_shape_t* shape, const int32_t* ids, const int32_t* n_ids,
                           const void* table, const void* hot_rows, const int32_t* hot_slot,
                           void* dev_cache, int32_t* stats, void* ws, void* stream);

/*
 * Frequency-ranked ("LFU") maintenance of the hot set used by stem_prefetch_rows_hot, for
 * decoding with an off-device table (Section 3.4: token ids are Zipfian, so a memory-efficient
 * LFU cache serves most lookups -- the paper reports more than 80 % hits; Section 3.2.4: the
 * cache lives in the memory the removed up-projection frees).  State, all caller-owned device
 * memory, initialised by the caller: freq int32 [V] = 0, hot_slot int32 [V] = -1, hot_ids
 * int32 [K] = -1 (id held by each slot), hot_rows [K,d_ff].
 *   stem_lfu_touch    one decode step's lookups: freq[ids[i]] += 1 for i < n; stats (optional
 *                     device int32[2]) += {lookups the cache serves, lookups it misses}.
 *   stem_lfu_refresh  afterwards the cache holds exactly the K ids with the largest freq (ties
 *                     to the smaller id; ids with freq 0 are never cached): ids that dropped
 *                     out lose their slots, ids that came in take them and their rows are
 *                     copied from `table` (page-locked host or device memory, [V,d_ff]).  Which
 *                     slot an id gets is arbitrary.  *n_installed (optional device int32) =
 *                     rows copied.  lfu_ws: device scratch of stem_lfu_workspace_bytes(V, K).
 * The paper gives no algorithm for its cache; this is least-frequently-used eviction applied
 * in batches (call refresh every few steps).
 */
int stem_lfu_workspace_bytes(int32_t V, int32_t K, size_t* bytes /*host, out*/);
int stem_lfu_touch(int32_t n, int32_t V, const int32_t* ids, int32_t* freq, const int32_t* hot_slot,
                   int32_t* stats, void* stream);
int stem_lfu_refresh(const stem_shape_t* shape, int32_t K, const int32_t* freq, int32_t* hot_slot,
                     int32_t* hot_ids, void* hot_rows, const void* table, int32_t* n_installed,
                     void* lfu_ws, size_t lfu_ws_bytes, void* stream);

/*
 * Gradient write-back for an off-device table (Table 1 notes: the table's gradients are
 * transferred back to CPU for the optimizer update):
 *   host_rows[r,:] = dE_rows[r,:] for r < *n_rows;  host_ids[r] = unique_ids[r];
 *   *host_n = *n_rows.
 * host_rows [min(T,V), d_ff] (grad_dtype), host_ids [min(T,V)], host_n [1]: page-locked
 * host memory (checked).  The device writes them directly; they are complete once
 * `stream` has been synchronised.  A count outside [0, min(T,V)] is clamped to that range (the
 * host buffers hold no more); *host_n receives the clamped value.
 */
int stem_writeback_rows(const stem_shape_t* shape, const void* dE_rows, const int32_t* unique_ids,
                        const int32_t* n_rows, void* host_rows, int32_t* host_ids,
                        int32_t* host_n, void* stream);

/*
 * The same write-back through the GPU's copy engine, for callers that know the row count on
 * the host (n_rows, a value): two asynchronous device-to-host copies on `stream`,
 * host_rows[0:n_rows,:] and host_ids[0:n_rows].  Prefer it when the write-back overlaps other
 * kernels: stores issued by SM code that saturate the host link's outbound direction also
 * delay the GPU's own command fetch over that link, and with it every kernel launched
 * meanwhile; copy-engine traffic does not.  A caller that pipelines layers can read
 * *n_unique back one layer ahead without draining the GPU.
 */
int stem_writeback_rows_dma(const stem_shape_t* shape, const void* dE_rows, const int32_t* unique_ids,
                            int32_t n_rows, void* host_rows, int32_t* host_ids, void* stream);

/*
 * Plain contraction on the same tensor-core kernel the layer uses (the y = H W_down^T
 * step is exactly this; exposed for testing and reuse):
 *   C[m,n] = sum_k A(m,k) B(n,k),  C row-major [M,N] (bf16 if c_fp32 == 0, else fp32).
 * a_mn == 0: A stored [M,K] row-major (K contiguous); a_mn == 1: A stored [K,M]
 * row-major (M contiguous).  b_mn likewise for B ([N,K] or [K,N]).  N and the contiguous
 * extent of each operand must be multiples of 8.  bf16 inputs, fp32 accumulation.
 * ws: a workspace (status word only).
 */
int stem_gemm_bf16(int32_t M, int32_t N, int32_t K, const void* A, int32_t a_mn, const void* B,
                   int32_t b_mn, void* C, int32_t c_fp32, int32_t flags, void* ws, void* stream);

/*
 * Table sharded over G GPUs (Section 3.4, "parallel embeddings": the table is always sharded
 * across the available GPUs, whatever the backbone's parallelism; the cost is one exchange of
 * the deduplicated rows, uniq(BL) x d_ff, Table 1).  The paper does not fix the row assignment;
 * here GPU g owns the rows with id mod G == g and keeps row id at local index id / G.
 *
 * stem_shard_route turns a batch's distinct ids into the requests of that exchange:
 *   send_local [n_max]  local row index asked of its owner, grouped by owner (owner 0 first),
 *                       ascending id inside a group; entries [0, *n_unique) are written
 *   send_slot  [n_max]  index into unique_ids of request j (where the answer's row, and later
 *                       its gradient row, belongs)
 *   send_counts [G]     requests per owner (device; the caller copies them to the host to size
 *                       the exchange)
 *   token_slot [T]      request whose answer is position t's row, or NULL: the layer is then
 *                       run with ids = token_slot and E = the [n_unique, d_ff] rows as they
 *                       came back, V = n_unique
 * unique_ids [n_max], n_unique [1], inverse [T]: outputs of stem_dedup_ids (device).
 * n_max >= *n_unique (normally min(T, V)); 1 <= G <= 1024.  route_ws: device scratch of
 * stem_shard_route_workspace_bytes(n_max, G) bytes, 16-byte aligned.  Integer work only.
 *
 * stem_reduce_rows is the table-gradient reduce as a call of its own, for the owner's side of
 * the return exchange: rows_out[r,:] = sum over the positions p of segment r of
 * rows_in[perm[p],:], in a fixed order.  shape->T = rows received, shape->d_ff = row length,
 * rows_in and rows_out in shape->grad_dtype; perm, seg_offsets, n_unique from stem_dedup_ids
 * over the received local row indices; rows_out [min(T,V), d_ff]; ws as for
 * stem_ffn_backward with this shape.
 */
/* The owner's side of the row exchange: out[r,:] = table[ids[r],:] for r < *n_ids, where ids
 * may repeat (several GPUs may ask for the same row), so up to shape->T rows are written
 * whatever shape->V is.  table [V,d_ff] and out [T,d_ff] in shape->dtype, device memory (or
 * table in page-locked host memory); ids, n_ids: device; ws: any initialised workspace
 * (status word only) or NULL. */
int stem_gather_rows(const stem_shape_t* shape, const int32_t* ids, const int32_t* n_ids, const void* table,
                     void* out, void* ws, void* stream);
int stem_shard_route_workspace_bytes(int32_t n_max, int32_t G, size_t* bytes /*host, out*/);
int stem_shard_route(int32_t n_max, int32_t T, int32_t G, const int32_t* unique_ids, const int32_t* n_unique,
                     const int32_t* inverse, int32_t* send_local, int32_t* send_slot, int32_t* send_counts,
                     int32_t* token_slot, void* route_ws, size_t route_ws_bytes, void* stream);
int stem_reduce_rows(const stem_shape_t* shape, const void* rows_in, const int32_t* perm,
                     const int32_t* seg_offsets, const int32_t* n_unique, void* rows_out, void* ws,
                     size_t ws_bytes, void* stream);

/*
 * One training step of the layer from host buffers (the composition of the calls above,
 * in the order Section 3.4 gives for training: ids deduplicated, forward, backward, table
 * gradients reduced per unique id):
 *   copy host_x, host_ids, host_dy to the device; stem_dedup_ids; stem_ffn_forward;
 *   stem_ffn_backward; copy y and dx back to host_y, host_dx (and n_u to host_n_unique
 *   when it is not NULL).
 * host_*: host memory ([T,d_model] in dtype; ids [T] int32), page-locked for the copies
 * to be asynchronous.  W_gate, E, W_down: device-resident parameters.  dW_gate, dW_down,
 * dE_rows, unique_ids [min(T,V)], n_unique [1]: device outputs, as in stem_ffn_backward
 * (they stay on the device for the optimizer; valid in `stream` order).  arena: device
 * scratch of stem_step_arena_bytes() bytes holding the workspace (call stem_init_workspace
 * on it once), every intermediate, and two slots of input and output buffers.
 * Pipelining: the kernels run on `stream`; the copies run on two copy streams the library
 * creates per device on first use (host-side objects only), chained to the kernels with
 * events.  Successive calls alternate between the two slots, so the host-to-device copy
 * of call k+1 and the device-to-host copy of call k-1 overlap the kernels of call k.
 * Consequences for the caller: the host INPUT buffers of a call must stay unchanged, and
 * its host OUTPUT buffers are not complete, until stem_ffn_step_host_flush(stream) has
 * been called and `stream` synchronised (flush makes `stream` wait for every outstanding
 * output copy; it is cheap and may be called after every step at the price of the
 * overlap).  Calls on one device are serialised by a lock; use one arena at a time.
 */
int stem_step_arena_bytes(const stem_shape_t* shape, size_t* bytes /*host, out*/);
int stem_ffn_step_host(const stem_shape_t* shape, const void* host_x, const int32_t* host_ids,
                       const void* host_dy, const void* W_gate, const void* E, const void* W_down,
                       void* host_y, void* host_dx, void* dW_gate, void* dW_down, void* dE_rows,
                       int32_t* unique_ids, int32_t* n_unique, int32_t* host_n_unique /*host*/,
                       void* arena, size_t arena_bytes, void* stream);
int stem_ffn_step_host_flush(void* stream);

/*
 * Self-test of the device-side bounded wait (no counterpart in the paper).  Every wait inside
 * the contraction kernels (on a TMA copy, on the tensor cores, on the epilogue) gives up after
 * a cycle limit, records STEM_ERR_TIMEOUT in the status word and lets the kernel unwind instead
 * of hanging the GPU.  This call runs that wait alone: one thread of one small CTA waits on a
 * barrier for at most limit_cycles SM clocks (1 .. 2e9).  arrive == 0: nothing ever completes the
 * barrier, the wait runs out, stem_query_status(ws) then returns STEM_ERR_TIMEOUT (detail 100)
 * and stem_init_workspace re-arms the word.  arrive != 0: the barrier is completed first, the
 * wait succeeds and the status stays as it was.  No copy or MMA is in flight either way; the
 * kernel always returns.  ws: an initialised workspace (status word only).
 */
int stem_selftest_wait(void* ws, long long limit_cycles, int arrive, void* stream);

/*
 * Instrumentation (no counterpart in the paper).  stem_launch_count: kernels this library
 * has launched in this process.  stem_profile_enable(1) clears earlier records and starts
 * recording one CUDA-event pair per step of the path (dedup, gate_gemm, down_gemm,
 * dh_gemm, seg_reduce, dw_pair_gemm (or dw_down_gemm, dw_gate_gemm), dx_gemm, prefetch_rows,
 * writeback_rows, h2d_inputs, d2h_outputs) on the stream of each call; (0) stops.
 * stem_profile_get waits for record i to finish and returns its name (static storage) and
 * its duration in milliseconds.
 */
long long stem_launch_count(void);
int stem_profile_enable(int on);
int stem_profile_count(void);
int stem_profile_get(int i, const char** name /*host, out*/, float* ms /*host, out*/);

#ifdef __cplusplus
}
#endif
#endif /* STEM_H_ */
