// Routing for a table whose rows are spread over G GPUs (paper Section 3.4, "parallel
// embeddings": whatever the backbone's parallelism, the STEM table is sharded across the
// available GPUs).  The paper does not say how rows are assigned; here GPU g owns the rows with
// id mod G == g and stores row id at local index id / G, which spreads the frequent (small)
// ids of a Zipfian vocabulary evenly.
//
// Given the batch's distinct ids (ascending, from the dedup), this produces what one exchange
// of rows each way needs:
//   send_local[j]  local row index to ask its owner for, grouped by owner (owner 0 first),
//                  ascending id inside a group
//   send_slot[j]   which distinct id (index into unique_ids) request j is
//   send_counts[g] requests addressed to owner g
//   token_slot[t]  for every position t, the request j whose answer is its row: the rows come
//                  back in request order, and the layer reads them through this index
// Integer work only; the order is fixed by a stable sort, so it does not depend on timing.
#include "stem_internal.h"

namespace stem {
namespace {

constexpr int kThreads = 256;

// key = owner of each distinct id; entries past n_unique sort last
__global__ void __launch_bounds__(kThreads)
shard_keys_kernel(int n_max, int G, const int32_t* __restrict__ unique_ids, const int32_t* __restrict__ n_unique,
                  int32_t* __restrict__ keys, int32_t* __restrict__ send_counts) {
  const int n = *n_unique;
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < G) send_counts[i] = 0;
  if (i < n_max) keys[i] = i < n ? unique_ids[i] % G : G;
}

// after the stable sort by owner: request j is distinct id order[j]
__global__ void __launch_bounds__(kThreads)
shard_requests_kernel(int n_max, int G, const int32_t* __restrict__ unique_ids, const int32_t* __restrict__ n_unique,
                      const int32_t* __restrict__ order, int32_t* __restrict__ send_local,
                      int32_t* __restrict__ send_slot, int32_t* __restrict__ request_of, int32_t* send_counts) {
  const int n = *n_unique;
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= n_max || j >= n) return;
  const int u = order[j];
  const int id = unique_ids[u];
  send_local[j] = id / G;
  send_slot[j] = u;
  request_of[u] = j;
  atomicAdd(send_counts + id % G, 1);   // integer counts: the result does not depend on the order
}

__global__ void __launch_bounds__(kThreads)
shard_token_slot_kernel(int T, const int32_t* __restrict__ inverse, const int32_t* __restrict__ request_of,
                        int32_t* __restrict__ token_slot) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t < T) token_slot[t] = request_of[inverse[t]];
}

size_t route_offsets(int n_max, size_t* keys, size_t* order, size_t* request_of) {
  const size_t tb = align_up(static_cast<size_t>(n_max) * 4, 256);
  *keys = 0; *order = tb; *request_of = 2 * tb;
  return 3 * tb;   // the sort's own scratch follows
}

}  // namespace

size_t shard_route_workspace_bytes(int n_max, int G) {
  size_t a, b, c;
  return route_offsets(n_max, &a, &b, &c) + dedup_workspace_bytes(n_max, G + 1);
}

cudaError_t launch_shard_route(int n_max, int T, int G, const int32_t* unique_ids, const int32_t* n_unique,
                               const int32_t* inverse, int32_t* send_local, int32_t* send_slot,
                               int32_t* send_counts, int32_t* token_slot, void* scratch, int32_t* status,
                               cudaStream_t stream) {
  if (n_max <= 0) return cudaMemsetAsync(send_counts, 0, static_cast<size_t>(G) * 4, stream);
  size_t o_keys, o_order, o_req;
  const size_t o_sort = route_offsets(n_max, &o_keys, &o_order, &o_req);
  char* p = static_cast<char*>(scratch);
  int32_t* keys = reinterpret_cast<int32_t*>(p + o_keys);
  int32_t* order = reinterpret_cast<int32_t*>(p + o_order);
  int32_t* request_of = reinterpret_cast<int32_t*>(p + o_req);
  const int blocks = ((n_max > G ? n_max : G) + kThreads - 1) / kThreads;
  shard_keys_kernel<<<blocks, kThreads, 0, stream>>>(n_max, G, unique_ids, n_unique, keys, send_counts);
  const int32_t* sorted = nullptr;
  cudaError_t e = launch_stable_sort(n_max, G + 1, keys, order, p + o_sort, &sorted, status, stream);
  if (e != cudaSuccess) return e;
  shard_requests_kernel<<<blocks, kThreads, 0, stream>>>(n_max, G, unique_ids, n_unique, order, send_local, send_slot,
                                                        request_of, send_counts);
  count_launches(2);
  if (token_slot != nullptr && T > 0) {
    shard_token_slot_kernel<<<(T + kThreads - 1) / kThreads, kThreads, 0, stream>>>(T, inverse, request_of, token_slot);
    count_launches(1);
  }
  return cudaGetLastError();
}

}  // namespace stem
