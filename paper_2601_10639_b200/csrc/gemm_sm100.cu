// bf16 contraction on the 5th-generation tensor cores (tcgen05), fp32 accumulators in
// tensor memory, operands staged by TMA -- with the layer's elementwise work fused into
// the epilogue.
//
//   C[m,n] = sum_k A(m,k) B(n,k)
//
// One persistent CTA per SM, warp-specialised:
//   warp 0      one thread issues TMA loads into a STAGES-deep shared-memory ring
//   warp 1      allocates TMEM; one thread issues tcgen05.mma (128 x BN x 16 per
//               instruction, four per 64-wide k block) and commits to mbarriers
//   warps 2..9  epilogue: tcgen05.ld the finished 128 x BN fp32 tile (one row per thread,
//               two warps per TMEM lane quarter, each taking half of the columns), apply
//               the fused elementwise step, and hand the result to TMA: each warp writes a
//               32-row x 32-column block into its own swizzled shared-memory buffer and
//               one lane issues a tensor store, so global writes are whole lines issued
//               by the copy engine instead of 32 scattered sectors per instruction.  The
//               table row and the saved G are fetched one 32-column chunk ahead of the
//               arithmetic, with 32-byte loads, so their latency hides behind the
//               previous chunk
// Two accumulator tiles live in TMEM (2 x BN columns), so the epilogue of tile i overlaps
// the MMAs of tile i+1.  Operands may be K-major or MN-major (the backward pass contracts
// over the token dimension, which is the slow index of every [T, .] tensor); both use the
// 128-byte swizzle, selected in the instruction and shared-memory descriptors.
//
// Every wait is bounded.  On expiry the role records STEM_ERR_TIMEOUT in the status word,
// raises a CTA-wide abort flag, and all roles unwind: copies in flight are waited for
// (again bounded), TMEM is freed, the kernel returns.
#include <cuda.h>

#include "ptx_sm100.cuh"
#include "stem_internal.h"

namespace stem {
namespace {

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int UMMA_K = 16;
constexpr int kEpiWarps = 8;
constexpr int kThreads = 64 + 32 * kEpiWarps;
constexpr long long kWaitLimitCycles = 2000000000ll;  // ~1 s at boost clock
constexpr int kAtomBytes = 64 * BK * 2;                // one 64(MN) x BK swizzled block

// CTAS = 2: two CTAs of a cluster share every MMA (cta_group::2).  Each stages its own 128
// rows of A and half of the BN columns of B, so a stage is 32 KB instead of 48 KB and the
// operand bytes fetched per flop drop by a third.
// DUAL: two products of the same A tile per stage (B operands of both, side by side) and three
// output blocks per epilogue warp.
template <int BN, int STAGES, int CTAS, bool DUAL = false>
struct Smem {
  static constexpr int kABytes = BM * BK * 2;
  static constexpr int kBBytes = (BN / CTAS) * BK * 2;          // one B operand
  static constexpr int kStageBytes = kABytes + (DUAL ? 2 : 1) * kBBytes;
  // per epilogue warp: two (DUAL: three) 2 KB output blocks (32 rows x 32 bf16) or one 4 KB block (fp32)
  static constexpr int kOutOffset = STAGES * kStageBytes;
  static constexpr int kOutBytesPerWarp = DUAL ? 6144 : 4096;
  static constexpr int kBarOffset = kOutOffset + kEpiWarps * kOutBytesPerWarp;
  // full[STAGES], empty[STAGES], tmem_full[2], tmem_empty[2], drain, tmem address, abort
  static constexpr int kNumBars = 2 * STAGES + 5;
  static constexpr int kTotal = kBarOffset + kNumBars * 8 + 16 + 1024;  // + alignment slack
};

// sigmoid(g) = 0.5 tanh(g / 2) + 0.5 with the hardware tanh (one special-function op instead of
// an exponential and a reciprocal; absolute error ~2^-12, far below the bf16 rounding of
// everything this feeds).
__device__ __forceinline__ float fast_sigmoid(float g) {
  float t;
  asm("tanh.approx.f32 %0, %1;" : "=f"(t) : "f"(0.5f * g));
  return fmaf(t, 0.5f, 0.5f);
}

// ---- 32-column row segments: global <-> registers -------------------------------------
// WIDE: the row pitch and base are multiples of 32 bytes, so 256-bit accesses are legal and
// a 16-column group is wholly inside or outside the matrix.  Otherwise 128-bit accesses.
// NC: the memory is read-only for the whole kernel, so the non-coherent path may serve it.  The
// add epilogue can run in place (its addend is the buffer it overwrites): it reads with plain
// loads.
template <bool NC>
__device__ __forceinline__ void ldg256(const void* p, uint32_t* r) {
  if (NC) {
    asm volatile("ld.global.nc.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "l"(p));
  } else {
    asm volatile("ld.global.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
                 : "l"(p) : "memory");
  }
}
template <bool NC>
__device__ __forceinline__ void ldg128(const void* p, uint32_t* r) {
  uint4 q;
  if (NC) {
    q = __ldg(static_cast<const uint4*>(p));
  } else {
    asm volatile("ld.global.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(q.x), "=r"(q.y), "=r"(q.z), "=r"(q.w) : "l"(p) : "memory");
  }
  r[0] = q.x; r[1] = q.y; r[2] = q.z; r[3] = q.w;
}

// 32 bf16 (16 registers) starting at column n of a row; p points at column n.
template <bool WIDE, bool NC = true>
__device__ __forceinline__ void load_bf16x32(const __nv_bfloat16* p, int n, int N, uint32_t (&r)[16]) {
  if (WIDE) {
#pragma unroll
    for (int h = 0; h < 2; ++h) if (n + 16 * h < N) ldg256<NC>(p + 16 * h, r + 8 * h);
  } else {
#pragma unroll
    for (int q = 0; q < 4; ++q) if (n + 8 * q < N) ldg128<NC>(p + 8 * q, r + 4 * q);
  }
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// One row (lane) of a 32-row block into the warp's staging buffer, in the layout the
// output tensor maps expect.  bf16: 64-byte rows, 64-byte swizzle (16-byte piece j of row
// r sits at piece j ^ ((r >> 1) & 3)).  fp32: 128-byte rows, 128-byte swizzle (piece j at
// j ^ (r & 7)).  Both patterns are bank-conflict free for 16-byte stores by 8 lanes.
__device__ __forceinline__ void stage_row_bf16(uint32_t buf, int lane, const uint32_t (&o)[16]) {
  const uint32_t row = buf + lane * 64, x = (lane >> 1) & 3;
#pragma unroll
  for (int j = 0; j < 4; ++j)
    ptx::st_shared_v4(row + ((j ^ x) << 4), o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
}
__device__ __forceinline__ void stage_row_f32(uint32_t buf, int lane, const uint32_t (&o)[32]) {
  const uint32_t row = buf + lane * 128, x = lane & 7;
#pragma unroll
  for (int j = 0; j < 8; ++j)
    ptx::st_shared_v4(row + ((j ^ x) << 4), o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
}

// Fused elementwise step on 32 consecutive columns of one output row: results go to the
// warp's staging buffer (first output at buf, second at buf + 2048).  e and g hold the
// table row segment and the saved pre-activation (bf16 pairs), fetched earlier.
// kEpiDagger: acc = the gate product, up = the up product of the same 32 columns:
// U = up + E[id], H = SiLU(acc) * U; outputs H, then (optional) G = acc and U.
__device__ __forceinline__ void epilogue_row32_dagger(const EpiParams& ep, uint32_t buf, int lane,
                                                      const uint32_t (&acc)[32], const uint32_t (&up)[32],
                                                      const uint32_t (&e)[16]) {
  uint32_t h[16], go[16], uo[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const float a0 = __uint_as_float(acc[2 * i]), a1 = __uint_as_float(acc[2 * i + 1]);
    const float u0 = __uint_as_float(up[2 * i]) + bf16_lo(e[i]), u1 = __uint_as_float(up[2 * i + 1]) + bf16_hi(e[i]);
    h[i] = pack_bf16(a0 * fast_sigmoid(a0) * u0, a1 * fast_sigmoid(a1) * u1);
    go[i] = pack_bf16(a0, a1);
    uo[i] = pack_bf16(u0, u1);
  }
  stage_row_bf16(buf, lane, h);
  if (ep.G) stage_row_bf16(buf + 2048, lane, go);
  if (ep.U) stage_row_bf16(buf + 4096, lane, uo);
}

template <int KIND>
__device__ __forceinline__ void epilogue_row32(const EpiParams& ep, uint32_t buf, int lane,
                                               const uint32_t (&acc)[32], const uint32_t (&e)[16],
                                               const uint32_t (&g)[16]) {
  if (KIND == kEpiStore) {
    if (ep.out_fp32) {
      stage_row_f32(buf, lane, acc);
    } else {
      uint32_t o[16];
#pragma unroll
      for (int i = 0; i < 16; ++i) o[i] = pack_bf16(__uint_as_float(acc[2 * i]), __uint_as_float(acc[2 * i + 1]));
      stage_row_bf16(buf, lane, o);
    }
  } else if (KIND == kEpiAdd) {
    uint32_t o[16];
#pragma unroll
    for (int i = 0; i < 16; ++i)
      o[i] = pack_bf16(__uint_as_float(acc[2 * i]) + bf16_lo(e[i]), __uint_as_float(acc[2 * i + 1]) + bf16_hi(e[i]));
    stage_row_bf16(buf, lane, o);
  } else if (KIND == kEpiGate) {
    uint32_t h[16], go[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const float a0 = __uint_as_float(acc[2 * i]), a1 = __uint_as_float(acc[2 * i + 1]);
      h[i] = pack_bf16(a0 * fast_sigmoid(a0) * bf16_lo(e[i]), a1 * fast_sigmoid(a1) * bf16_hi(e[i]));
      go[i] = pack_bf16(a0, a1);
    }
    stage_row_bf16(buf, lane, h);
    if (ep.G) stage_row_bf16(buf + 2048, lane, go);
  } else {
    uint32_t du[16], dg[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const float a0 = __uint_as_float(acc[2 * i]), a1 = __uint_as_float(acc[2 * i + 1]);
      const float g0 = bf16_lo(g[i]), g1 = bf16_hi(g[i]);
      const float s0 = fast_sigmoid(g0), s1 = fast_sigmoid(g1);
      du[i] = pack_bf16(a0 * (g0 * s0), a1 * (g1 * s1));
      dg[i] = pack_bf16(a0 * bf16_lo(e[i]) * (s0 * (1.0f + g0 * (1.0f - s0))),
                        a1 * bf16_hi(e[i]) * (s1 * (1.0f + g1 * (1.0f - s1))));
    }
    stage_row_bf16(buf, lane, du);
    stage_row_bf16(buf + 2048, lane, dg);
  }
}

struct TileCoord { int m_blk, n_blk; };
__device__ __forceinline__ TileCoord tile_coord(int tile, int tiles_m, int tiles_n, int group_m) {
  const int per_group = group_m * tiles_n;
  const int g = tile / per_group;
  const int first_m = g * group_m;
  const int gsize = min(group_m, tiles_m - first_m);
  const int in = tile - g * per_group;
  return {first_m + in % gsize, in / gsize};
}

// ---- work list ----------------------------------------------------------------------------
// Tiles [0, dp_tiles) are handed out whole, round robin over the P persistent CTAs (pairs).
// When the tile count leaves a ragged last round, each of the remaining tiles is cut into
// `split` pieces along k (equal k ranges) and the pieces are handed out round robin, ordered
// k range first, so the pieces in flight together cover the same k range of different
// tiles and share their operand panels in L2 exactly as whole tiles do.  A piece writes raw
// fp32 sums to its slot of a partial-tile matrix; a small fix-up kernel adds each tile's
// pieces in ascending k order, so the result does not depend on timing.
struct Work { int tile, kb0, kb1, slot; };  // slot < 0: a whole tile, written to the output

struct WorkList {
  int p, P, dp_tiles, num_tiles, k_blocks, split;
  // i-th work item of CTA (pair) p; false when the list is exhausted
  __device__ __forceinline__ bool get(int i, Work& w) const {
    const int n_dp = dp_tiles > p ? (dp_tiles - p + P - 1) / P : 0;
    if (i < n_dp) { w = {p + i * P, 0, k_blocks, -1}; return true; }
    const int tail = num_tiles - dp_tiles;
    const int q = p + (i - n_dp) * P;          // piece number
    if (q >= tail * split) return false;
    const int ik = q / tail, j = q - ik * tail;  // k range, tail tile
    w = {dp_tiles + j, static_cast<int>(static_cast<long long>(k_blocks) * ik / split),
         static_cast<int>(static_cast<long long>(k_blocks) * (ik + 1) / split), q};
    return true;
  }
};

template <bool A_MN, bool B_MN, int KIND, int BN, int STAGES, bool WIDE, int CTAS>
__global__ void __launch_bounds__(kThreads, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmC0, const __grid_constant__ CUtensorMap tmC1,
               const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmB2,
               const __grid_constant__ CUtensorMap tmC2,
               int M, int N, int K, int M2, int N2, int group_m, int dp_tiles, int split, EpiParams ep) {
  constexpr bool kDual = KIND == kEpiDagger;      // two products (gate, up) of every A tile
  using L = Smem<BN, STAGES, CTAS, kDual>;
  constexpr int kAccCols = kDual ? 2 * BN : BN;   // TMEM columns of one accumulator set
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = ptx::smem_u32(smem_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  uint8_t* base_ptr = smem_raw + (base - raw);
  const uint32_t bars = base + L::kBarOffset;
  auto full_bar = [&](int s) { return bars + 8u * s; };
  auto empty_bar = [&](int s) { return bars + 8u * (STAGES + s); };
  auto tfull_bar = [&](int a) { return bars + 8u * (2 * STAGES + a); };
  auto tempty_bar = [&](int a) { return bars + 8u * (2 * STAGES + 2 + a); };
  const uint32_t drain_bar = bars + 8u * (2 * STAGES + 4);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + L::kBarOffset + L::kNumBars * 8);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + L::kBarOffset + L::kNumBars * 8 + 4);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // A work unit is one BM*CTAS x BN output tile, handled by one CTA or one CTA pair.
  const uint32_t rank = CTAS == 2 ? ptx::cluster_ctarank() : 0u;
  const int unit0 = blockIdx.x / CTAS, unit_stride = gridDim.x / CTAS;
  const int tiles_m = (M + BM * CTAS - 1) / (BM * CTAS), tiles_n = (N + BN - 1) / BN;
  // A second product with the same contraction length may ride in the same launch (plain stores
  // only): its tiles are numbered after the first product's and share one work list, so the two
  // fill the machine together where each alone would leave SMs idle.
  const int tiles_m2 = KIND == kEpiStore && M2 > 0 ? (M2 + BM * CTAS - 1) / (BM * CTAS) : 0;
  const int tiles_n2 = KIND == kEpiStore && M2 > 0 ? (N2 + BN - 1) / BN : 0;
  const int num_tiles1 = tiles_m * tiles_n;
  const int num_tiles = num_tiles1 + tiles_m2 * tiles_n2;
  const int k_blocks = (K + BK - 1) / BK;
  constexpr uint32_t kTmemCols = 2 * kAccCols;
  static_assert(kTmemCols <= 512, "two accumulator sets must fit the 512 TMEM columns");
  const WorkList work{unit0, unit_stride, dp_tiles, num_tiles, k_blocks, split};

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(full_bar(s), 1); ptx::mbar_init(empty_bar(s), 1); }
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(tfull_bar(a), 1); ptx::mbar_init(tempty_bar(a), kEpiWarps * CTAS); }
    ptx::mbar_init(drain_bar, 1);
    *abort_flag = 0;
    ptx::fence_mbar_init();
    ptx::prefetch_tensormap(&tmA);
    ptx::prefetch_tensormap(&tmB);
    ptx::prefetch_tensormap(&tmC0);
    if (KIND == kEpiGate || KIND == kEpiDH || kDual) ptx::prefetch_tensormap(&tmC1);
    if (kDual) { ptx::prefetch_tensormap(&tmB2); ptx::prefetch_tensormap(&tmC2); }
    if (KIND == kEpiStore && M2 > 0) {
      ptx::prefetch_tensormap(&tmA2);
      ptx::prefetch_tensormap(&tmB2);
      ptx::prefetch_tensormap(&tmC2);
    }
  }
  if (warp == 1) {
    if (CTAS == 2) {
      ptx::tmem_alloc_pair(ptx::smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
      ptx::tmem_relinquish_pair();
    } else {
      ptx::tmem_alloc(ptx::smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
      ptx::tmem_relinquish();
    }
  }
  ptx::tc_fence_before();
  // in a pair, the other CTA's barriers and TMEM must exist before anything targets them
  if (CTAS == 2) ptx::cluster_sync(); else __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  // Everything above touched only this CTA's own resources, so it may overlap the tail of the
  // previous kernel in the stream; everything below reads or overwrites global memory.
  ptx::grid_dependency_wait();
  ptx::grid_launch_dependents();

  int issued = 0;  // producer: k blocks handed to TMA so far

  if (warp == 0) {
    if (lane == 0) {
      int s = 0; uint32_t ph = 0;
      bool ok = true;
      Work w;
      for (int i = 0; ok && work.get(i, w); ++i) {
        const bool second = KIND == kEpiStore && w.tile >= num_tiles1;
        const TileCoord tc = second ? tile_coord(w.tile - num_tiles1, tiles_m2, tiles_n2, group_m)
                                    : tile_coord(w.tile, tiles_m, tiles_n, group_m);
        const CUtensorMap* mapA = second ? &tmA2 : &tmA;
        const CUtensorMap* mapB = second ? &tmB2 : &tmB;
        // this CTA's rows of A and its share of the columns of B
        const int m0 = (tc.m_blk * CTAS + rank) * BM, n0 = tc.n_blk * BN + rank * (BN / CTAS);
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
          if (!ptx::mbar_wait_bounded(empty_bar(s), ph ^ 1u, abort_flag, kWaitLimitCycles)) {
            report_error(ep.status, STEM_ERR_TIMEOUT, 1);
            *abort_flag = 1; ok = false; break;
          }
          const uint32_t a_dst = base + s * L::kStageBytes;
          const uint32_t b_dst = a_dst + L::kABytes;
          // The MMA issuer (rank 0) waits on its own full barrier for the bytes of both CTAs.
          if (rank == 0) ptx::mbar_arrive_expect_tx(full_bar(s), CTAS * L::kStageBytes);
          const uint32_t fb = CTAS == 2 ? ptx::mapa(full_bar(s), 0) : full_bar(s);
          auto load = [&](uint32_t dst, const CUtensorMap* map, int c0, int c1) {
            if (CTAS == 2) ptx::tma_load_2d_pair(dst, map, fb, c0, c1); else ptx::tma_load_2d(dst, map, fb, c0, c1);
          };
          const int k0 = kb * BK;
          if (A_MN) {
#pragma unroll
            for (int j = 0; j < BM / 64; ++j) load(a_dst + j * kAtomBytes, mapA, m0 + 64 * j, k0);
          } else {
            load(a_dst, mapA, k0, m0);
          }
          if (B_MN) {
#pragma unroll
            for (int j = 0; j < BN / CTAS / 64; ++j) load(b_dst + j * kAtomBytes, mapB, n0 + 64 * j, k0);
          } else {
            load(b_dst, mapB, k0, n0);
            if (kDual) load(b_dst + L::kBBytes, &tmB2, k0, n0);    // the up-projection's rows of the same columns
          }
          ++issued;
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      constexpr uint32_t idesc = ptx::make_idesc_bf16(BM * CTAS, BN, A_MN, B_MN);
      auto commit = [&](uint32_t bar) {   // in a pair the barrier of both CTAs is signalled
        if (CTAS == 2) ptx::mma_commit_pair(bar, 3); else ptx::mma_commit(bar);
      };
      int s = 0; uint32_t ph = 0;
      int acc = 0; uint32_t aph = 0;
      bool ok = true;
      Work w;
      for (int i = 0; ok && work.get(i, w); ++i) {
        if (!ptx::mbar_wait_bounded(tempty_bar(acc), aph ^ 1u, abort_flag, kWaitLimitCycles)) {
          report_error(ep.status, STEM_ERR_TIMEOUT, 3);
          *abort_flag = 1; ok = false; break;
        }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + acc * kAccCols;
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
          if (!ptx::mbar_wait_bounded(full_bar(s), ph, abort_flag, kWaitLimitCycles)) {
            report_error(ep.status, STEM_ERR_TIMEOUT, 2);
            *abort_flag = 1; ok = false; break;
          }
          ptx::tc_fence_after();
          const uint32_t a_src = base + s * L::kStageBytes;
          const uint32_t b_src = a_src + L::kABytes;
#pragma unroll
          for (int kk = 0; kk < BK / UMMA_K; ++kk) {
            // K-major: 16 k elements = 32 bytes inside the 128-byte swizzled row; 8-row
            // groups 1024 bytes apart.  MN-major: 16 k rows of 128 bytes; 64-wide MN blocks
            // kAtomBytes apart, 8-row k groups 1024 bytes apart.
            const uint64_t ad = A_MN ? ptx::make_smem_desc(a_src + kk * (UMMA_K * 128), kAtomBytes, 1024)
                                     : ptx::make_smem_desc(a_src + kk * (UMMA_K * 2), 16, 1024);
            const uint64_t bd = B_MN ? ptx::make_smem_desc(b_src + kk * (UMMA_K * 128), kAtomBytes, 1024)
                                     : ptx::make_smem_desc(b_src + kk * (UMMA_K * 2), 16, 1024);
            if (CTAS == 2) ptx::mma_bf16_ss_pair(d_tmem, ad, bd, idesc, (kb > w.kb0 || kk > 0) ? 1u : 0u);
            else ptx::mma_bf16_ss(d_tmem, ad, bd, idesc, (kb > w.kb0 || kk > 0) ? 1u : 0u);
          }
          if (kDual) {   // the same A block against the second B operand, into the second accumulator
#pragma unroll
            for (int kk = 0; kk < BK / UMMA_K; ++kk) {
              const uint64_t ad = ptx::make_smem_desc(a_src + kk * (UMMA_K * 2), 16, 1024);
              const uint64_t bd2 = ptx::make_smem_desc(b_src + L::kBBytes + kk * (UMMA_K * 2), 16, 1024);
              if (CTAS == 2) ptx::mma_bf16_ss_pair(d_tmem + BN, ad, bd2, idesc, (kb > w.kb0 || kk > 0) ? 1u : 0u);
              else ptx::mma_bf16_ss(d_tmem + BN, ad, bd2, idesc, (kb > w.kb0 || kk > 0) ? 1u : 0u);
            }
          }
          commit(empty_bar(s));
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
        commit(tfull_bar(acc));
        if (++acc == 2) { acc = 0; aph ^= 1u; }
      }
      if (!ok) {
        // let MMAs already issued finish before TMEM is freed
        if (CTAS == 2) ptx::mma_commit_pair(drain_bar, 1); else ptx::mma_commit(drain_bar);
        int zero = 0;
        ptx::mbar_wait_bounded(drain_bar, 0, &zero, kWaitLimitCycles);
      }
    }
  } else {
    const int q = warp & 3;                 // TMEM lane quarter this warp may read
    const int half = (warp - 2) >> 2;       // which half of the tile's columns it handles
    constexpr int kChunks = BN / 2 / 32;    // 32-column chunks per thread per tile
    const uint32_t out_buf = base + L::kOutOffset + (warp - 2) * L::kOutBytesPerWarp;
    const bool second_out = KIND == kEpiDH || ((KIND == kEpiGate || kDual) && ep.G != nullptr);
    constexpr bool kReadOnlyE = KIND != kEpiAdd;   // the add epilogue may overwrite its addend
    int acc = 0; uint32_t aph = 0;
    bool ok = true;
    Work w;
    for (int i = 0; ok && work.get(i, w); ++i) {
      const bool second = KIND == kEpiStore && w.tile >= num_tiles1;
      const TileCoord tc = second ? tile_coord(w.tile - num_tiles1, tiles_m2, tiles_n2, group_m)
                                  : tile_coord(w.tile, tiles_m, tiles_n, group_m);
      const CUtensorMap* mapC = second ? &tmC2 : &tmC0;
      const int M_ = second ? M2 : M, N_ = second ? N2 : N;    // extents of the product this tile belongs to
      const int m_warp = (tc.m_blk * CTAS + rank) * BM + q * 32;  // first row of this warp's 32-row block
      const int m = m_warp + lane;
      const int n0 = tc.n_blk * BN + half * (BN / 2);
      const bool row_ok = m < M_;
      const size_t row_off = static_cast<size_t>(m) * N;
      const __nv_bfloat16* e_row = nullptr;
      const __nv_bfloat16* g_row = nullptr;
      if (KIND != kEpiStore && row_ok) {
        int id = ep.ids != nullptr ? ep.ids[m] : m;
        if (id < 0 || id >= ep.V) {
          report_error(ep.status, STEM_ERR_ID_RANGE, m);
          id = id < 0 ? 0 : ep.V - 1;
        }
        e_row = static_cast<const __nv_bfloat16*>(ep.E) + static_cast<size_t>(id) * N;
        if (KIND == kEpiDH) g_row = static_cast<const __nv_bfloat16*>(ep.Gin) + row_off;
      }
      // operands of the first chunk are requested before waiting for the accumulator
      uint32_t e_next[16], g_next[16];
      if (KIND != kEpiStore && row_ok) {
        load_bf16x32<WIDE, kReadOnlyE>(e_row + n0, n0, N, e_next);
        if (KIND == kEpiDH) load_bf16x32<WIDE>(g_row + n0, n0, N, g_next);
      }
      bool mine = ptx::mbar_wait_bounded(tfull_bar(acc), aph, abort_flag, kWaitLimitCycles);
      mine = __all_sync(0xffffffffu, mine);
      if (!mine) {
        if (lane == 0) { report_error(ep.status, STEM_ERR_TIMEOUT, 4); *abort_flag = 1; }
        ok = false; break;
      }
      ptx::tc_fence_after();
      const uint32_t t_row = tmem_base + acc * kAccCols + half * (BN / 2) + (static_cast<uint32_t>(q * 32) << 16);
#pragma unroll
      for (int c = 0; c < kChunks; ++c) {
        uint32_t e_cur[16], g_cur[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) { e_cur[i] = e_next[i]; g_cur[i] = g_next[i]; }
        const int n = n0 + c * 32;
        if (KIND != kEpiStore && row_ok && c + 1 < kChunks) {
          load_bf16x32<WIDE, kReadOnlyE>(e_row + n + 32, n + 32, N, e_next);
          if (KIND == kEpiDH) load_bf16x32<WIDE>(g_row + n + 32, n + 32, N, g_next);
        }
        uint32_t v[32], v2[kDual ? 32 : 1];
        ptx::tmem_ld_32x32(t_row + c * 32, v);
        if constexpr (kDual) ptx::tmem_ld_32x32(t_row + BN + c * 32, v2);
        ptx::tmem_ld_wait();
        if (c + 1 == kChunks) {
          // the accumulator has been read out: hand it back to the MMA issuer
          ptx::tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            if (rank == 0) ptx::mbar_arrive(tempty_bar(acc)); else ptx::mbar_arrive_cluster(ptx::mapa(tempty_bar(acc), 0));
          }
        }
        // the staging buffer is free once the previous chunk's tensor stores have read it
        if (lane == 0) ptx::bulk_wait_read_all();
        __syncwarp();
        if (KIND == kEpiStore && w.slot >= 0) {
          // a piece of a tile: raw fp32 sums into the piece's slot of the partial-tile matrix
          // (tmC1: [slots * BM * CTAS, BN] fp32), finished by the fix-up kernel
          stage_row_f32(out_buf, lane, v);
          ptx::fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            ptx::tma_store_2d(&tmC1, out_buf, half * (BN / 2) + c * 32, (w.slot * CTAS + rank) * BM + q * 32);
            ptx::bulk_commit_group();
          }
        } else {
          if constexpr (kDual) epilogue_row32_dagger(ep, out_buf, lane, v, v2, e_cur);
          else epilogue_row32<KIND>(ep, out_buf, lane, v, e_cur, g_cur);
          ptx::fence_proxy_async();
          __syncwarp();
          if (lane == 0 && m_warp < M_ && n < N_) {
            if (KIND == kEpiStore && ep.accumulate) ptx::tma_reduce_add_2d(mapC, out_buf, n, m_warp);
            else ptx::tma_store_2d(mapC, out_buf, n, m_warp);
            if (second_out) ptx::tma_store_2d(&tmC1, out_buf + 2048, n, m_warp);
            if (kDual && ep.U != nullptr) ptx::tma_store_2d(&tmC2, out_buf + 4096, n, m_warp);
            ptx::bulk_commit_group();
          }
        }
      }
      if (++acc == 2) { acc = 0; aph ^= 1u; }
    }
    // every tensor store of this warp must be complete before the CTA may exit
    if (lane == 0) ptx::bulk_wait_all();
  }

  __syncthreads();
  if (*abort_flag != 0 && threadIdx.x == 0) {
    // wait (bounded) for TMA copies still in flight: the last issue into each stage.  The
    // bytes of a pair's second CTA are counted on the first CTA's barriers, which it cannot
    // poll; it waits out a fixed interval instead (far longer than a copy takes).
    int zero = 0;
    if (rank == 0) {
      for (int s = 0; s < STAGES; ++s) {
        int last = -1;
        for (int j = issued - 1; j >= 0 && j >= issued - STAGES; --j)
          if (j % STAGES == s) { last = j; break; }
        if (last >= 0) ptx::mbar_wait_bounded(full_bar(s), (last / STAGES) & 1, &zero, kWaitLimitCycles / 16);
      }
    } else {
      const long long t0 = clock64();
      while (clock64() - t0 < 2000000ll) { }
    }
  }
  // Neither CTA of a pair may exit (or free TMEM) while the other can still signal its
  // barriers, read its shared memory or write its accumulators.  Every role reaches this
  // point in bounded time, so the cluster barrier cannot hang.
  if (CTAS == 2) ptx::cluster_sync(); else __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after();
    if (CTAS == 2) ptx::tmem_dealloc_pair(tmem_base, kTmemCols); else ptx::tmem_dealloc(tmem_base, kTmemCols);
  }
}

// Fix-up for the tail tiles: output tile = sum of its pieces in ascending k order (piece ik of
// tail tile j is slot ik * tail + j).  One CTA per (tail tile, kFixRows-row band); a thread
// requests its element of every piece before it adds the first, so the launch is bound by
// bandwidth (the partial tiles mostly still sit in L2), not by a chain of load latencies.
constexpr int kMaxSplit = 8;   // most pieces a tail tile is cut into
constexpr int kFixRows = 8;    // rows of a tile per fix-up CTA
template <int BN, int CTAS>
__global__ void __launch_bounds__(256)
tail_fixup_kernel(int M, int N, int dp_tiles, int tail, int split, int tiles_m, int tiles_n, int group_m,
                  const float* __restrict__ partial, void* __restrict__ out, int out_fp32, int accumulate,
                  int M2, int N2, int tiles_m2, int tiles_n2, void* __restrict__ out2) {
  constexpr int TM = BM * CTAS;
  ptx::grid_dependency_wait();
  ptx::grid_launch_dependents();
  const int j = blockIdx.x;
  // tiles of a second product riding in the same launch are numbered after the first product's
  const int num_tiles1 = tiles_m * tiles_n;
  const bool second = dp_tiles + j >= num_tiles1;
  const TileCoord tc = second ? tile_coord(dp_tiles + j - num_tiles1, tiles_m2, tiles_n2, group_m)
                              : tile_coord(dp_tiles + j, tiles_m, tiles_n, group_m);
  if (second) { M = M2; N = N2; out = out2; }
  const int r0 = blockIdx.y * kFixRows;
  for (int e = threadIdx.x; e < kFixRows * (BN / 4); e += 256) {
    const int r = r0 + e / (BN / 4), c = (e % (BN / 4)) * 4;
    const int m = tc.m_blk * TM + r, nn = tc.n_blk * BN + c;
    if (m >= M || nn >= N) continue;
    float4 v[kMaxSplit];
#pragma unroll
    for (int ik = 0; ik < kMaxSplit; ++ik) {
      if (ik < split) {
        const size_t slot = static_cast<size_t>(ik) * tail + j;
        v[ik] = __ldcg(reinterpret_cast<const float4*>(partial + (slot * TM + r) * BN + c));
      }
    }
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int ik = 0; ik < kMaxSplit; ++ik) {
      if (ik < split) { acc.x += v[ik].x; acc.y += v[ik].y; acc.z += v[ik].z; acc.w += v[ik].w; }
    }
    const size_t o = static_cast<size_t>(m) * N + nn;   // N is a multiple of 8: 4 columns never straddle the edge
    if (out_fp32) {
      float4* p = reinterpret_cast<float4*>(static_cast<float*>(out) + o);
      if (accumulate) { const float4 v = *p; acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w; }
      *p = acc;
    } else {
      uint2* p = reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(out) + o);
      if (accumulate) {
        const uint2 v = *p;
        acc.x += bf16_lo(v.x); acc.y += bf16_hi(v.x); acc.z += bf16_lo(v.y); acc.w += bf16_hi(v.y);
      }
      uint2 pk;
      pk.x = pack_bf16(acc.x, acc.y);
      pk.y = pack_bf16(acc.z, acc.w);
      *p = pk;
    }
  }
}

// ---- host side ---------------------------------------------------------------------------
using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                              CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                              CUtensorMapFloatOOBfill);

EncodeFn get_encode_fn() {
  static EncodeFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeFn>(p);
  }();
  return fn;
}

// Row-major bf16 matrix [rows, cols] (cols contiguous); box = 64 columns x box_rows rows.
bool encode_map(CUtensorMap* map, const void* ptr, int rows, int cols, int box_rows) {
  EncodeFn fn = get_encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(cols) * 2};
  const cuuint32_t box[2] = {64u, static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t estr[2] = {1u, 1u};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Output matrix [rows, cols] row-major, bf16 or fp32; box = 32 columns x 32 rows, swizzled
// over the box's row length (64 bytes for bf16, 128 bytes for fp32).
bool encode_out_map(CUtensorMap* map, const void* ptr, int rows, int cols, bool fp32) {
  EncodeFn fn = get_encode_fn();
  if (!fn) return false;
  const cuuint64_t esz = fp32 ? 4 : 2;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(cols) * esz};
  const cuuint32_t box[2] = {32u, 32u};
  const cuuint32_t estr[2] = {1u, 1u};
  return fn(map, fp32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
            const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            fp32 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// A second product C2 = A2 B2^T with the same contraction length and operand layouts, carried by
// the same launch (plain stores only); M == 0 means none.
// The same parameter slots carry the second B operand (B) and the third output (C) of the
// two-product kind kEpiDagger, with M == 0 and `maps` set.
struct SecondMaps { CUtensorMap A, B, C; int M = 0, N = 0; void* out = nullptr; bool maps = false; };

template <bool A_MN, bool B_MN, int KIND, int BN, int STAGES, bool WIDE, int CTAS>
cudaError_t launch_inst(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmC0,
                        const CUtensorMap& tmC1, int M, int N, int K, const EpiParams& ep, int sk_tail,
                        int sk_split, const SecondMaps& sec, cudaStream_t stream) {
  using L = Smem<BN, STAGES, CTAS, KIND == kEpiDagger>;
  static_assert(L::kTotal <= 232448, "exceeds the shared memory a CTA can have");
  auto kern = tc_gemm_kernel<A_MN, B_MN, KIND, BN, STAGES, WIDE, CTAS>;
  static PerDeviceOnce configured;
  if (cudaError_t ce = configured.run([&] {
        return cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal);
      }))
    return ce;
  // persistent: one CTA (or one pair) per SM (pair of SMs), each walking its work list
  const int tiles_m = (M + BM * CTAS - 1) / (BM * CTAS), tiles_n = (N + BN - 1) / BN;
  const int tiles_m2 = sec.M > 0 ? (sec.M + BM * CTAS - 1) / (BM * CTAS) : 0, tiles_n2 = sec.M > 0 ? (sec.N + BN - 1) / BN : 0;
  const int units = tiles_m * tiles_n + tiles_m2 * tiles_n2;
  const int slots = device_sm_count() / CTAS;
  const int P = sk_tail > 0 ? slots : (units < slots ? units : slots);
  const int dp_tiles = sk_tail > 0 ? units - sk_tail : units;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(CTAS * P));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = L::kTotal;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = CTAS;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  const bool second_maps = sec.M > 0 || sec.maps;
  cudaError_t e = cudaLaunchKernelEx(&cfg, kern, tmA, tmB, tmC0, tmC1, sec.M > 0 ? sec.A : tmA, second_maps ? sec.B : tmB,
                                     second_maps ? sec.C : tmC0, M, N, K, sec.M, sec.N, 8, dp_tiles, sk_split, ep);
  count_launches(1);
  if (e == cudaSuccess && sk_tail > 0) {
    cudaLaunchConfig_t fcfg = {};
    fcfg.gridDim = dim3(sk_tail, BM * CTAS / kFixRows);
    fcfg.blockDim = dim3(256);
    fcfg.stream = stream;
    fcfg.attrs = attr + 1;
    fcfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&fcfg, tail_fixup_kernel<BN, CTAS>, M, N, dp_tiles, sk_tail, sk_split, tiles_m, tiles_n, 8,
                           static_cast<const float*>(ep.sk_scratch), ep.out, static_cast<int>(ep.out_fp32),
                           static_cast<int>(ep.accumulate), sec.M, sec.N, tiles_m2, tiles_n2, sec.out);
    count_launches(1);
  }
  return e != cudaSuccess ? e : cudaGetLastError();
}

struct SecondProduct { int M = 0, N = 0; const void* A = nullptr; const void* B = nullptr; void* out = nullptr; };

template <bool A_MN, bool B_MN, int KIND, int CTAS, int BN = 256>
cudaError_t launch_bn(const void* A, const void* B, int M, int N, int K, const EpiParams& ep,
                      const SecondProduct& second, cudaStream_t stream) {
  // 192 KB of operand ring either way: 4 stages of 48 KB, or 6 stages of 32 KB per CTA of a pair
  // (8 stages of 24 KB for the 128-column tiles of decode-sized batches)
  constexpr int STAGES = BN == 256 ? (CTAS == 2 ? 6 : 4) : (CTAS == 2 ? 8 : 5);
  CUtensorMap tmA, tmB;
  const bool okA = A_MN ? encode_map(&tmA, A, K, M, BK) : encode_map(&tmA, A, M, K, BM);
  const bool okB = B_MN ? encode_map(&tmB, B, K, N, BK) : encode_map(&tmB, B, N, K, BN / CTAS);
  if (!okA || !okB) return cudaErrorNotSupported;
  CUtensorMap tmC0, tmC1;
  SecondMaps sec;
  bool okC;
  int sk_tail = 0, sk_split = 1;  // tiles of the ragged last round, pieces per tile along k
  if (KIND == kEpiStore) {
    okC = encode_out_map(&tmC0, ep.out, M, N, ep.out_fp32 != 0);
    tmC1 = tmC0;
    if (second.M > 0) {
      sec.M = second.M; sec.N = second.N; sec.out = second.out;
      okC = okC && (A_MN ? encode_map(&sec.A, second.A, K, second.M, BK) : encode_map(&sec.A, second.A, second.M, K, BM));
      okC = okC && (B_MN ? encode_map(&sec.B, second.B, K, second.N, BK) : encode_map(&sec.B, second.B, second.N, K, BN / CTAS));
      okC = okC && encode_out_map(&sec.C, second.out, second.M, second.N, ep.out_fp32 != 0);
    }
    // The last round costs ceil(tail * split / slots) / split tile times instead of one.
    // Worth it when that saves clearly more than the partial tiles and the fix-up launch
    // cost (10-25 us together); a tile time is ~ 2 TM BN K flops at ~11 TFLOP/s per SM.
    constexpr int TM = BM * CTAS;
    const int units = ((M + TM - 1) / TM) * ((N + BN - 1) / BN) +
                      (second.M > 0 ? ((second.M + TM - 1) / TM) * ((second.N + BN - 1) / BN) : 0);
    const int slots = device_sm_count() / CTAS;
    const int k_blocks = (K + BK - 1) / BK;
    const int tail = units % slots;
    const size_t slot_bytes = static_cast<size_t>(TM) * BN * sizeof(float);
    const double tile_us = 2.0 * TM * BN * static_cast<double>(K) / (11.0e6 * CTAS);
    if (tail > 0 && ep.sk_scratch != nullptr) {
      int best = 1;
      double best_cost = 1.0;
      for (int sp = 2; sp <= kMaxSplit; ++sp) {
        if (static_cast<size_t>(tail) * sp * slot_bytes > ep.sk_bytes || k_blocks / sp < 4) break;
        const double cost = static_cast<double>((tail * sp + slots - 1) / slots) / sp;
        if (cost < best_cost - 0.04) { best_cost = cost; best = sp; }
      }
      if (best > 1 && (1.0 - best_cost) * tile_us > 25.0) {
        sk_tail = tail;
        sk_split = best;
        okC = okC && encode_out_map(&tmC1, ep.sk_scratch, tail * best * TM, BN, true);
      }
    }
  } else {
    okC = encode_out_map(&tmC0, ep.H, M, N, false);
    if (ep.G) okC = okC && encode_out_map(&tmC1, ep.G, M, N, false); else tmC1 = tmC0;
  }
  if (!okC) return cudaErrorNotSupported;
  auto a32 = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 31u) == 0; };
  const bool wide = (N % 16 == 0) && a32(ep.E) && a32(ep.Gin);
  if (wide) return launch_inst<A_MN, B_MN, KIND, BN, STAGES, true, CTAS>(tmA, tmB, tmC0, tmC1, M, N, K, ep, sk_tail, sk_split, sec, stream);
  return launch_inst<A_MN, B_MN, KIND, BN, STAGES, false, CTAS>(tmA, tmB, tmC0, tmC1, M, N, K, ep, sk_tail, sk_split, sec, stream);
}

template <bool A_MN, bool B_MN, int KIND>
cudaError_t launch_ctas(const void* A, const void* B, int M, int N, int K, const EpiParams& ep, bool pair,
                        cudaStream_t stream) {
  if constexpr (KIND == kEpiGate) {
    // A decode-sized batch (one row of tiles) leaves most CTA pairs without a tile and makes the
    // one tile a pair has a serial chain of load, multiply, epilogue.  Halving the tile width
    // doubles the pairs at work and halves that chain; beyond 256 rows the extra passes over x
    // cost more than they save (measured: 256 rows 22.6 -> 20.5 us, 512 rows 23.8 -> 28.8 us).
    if (pair && M <= 256 && (N + 127) / 128 <= device_sm_count() / 2)
      return launch_bn<A_MN, B_MN, KIND, 2, 128>(A, B, M, N, K, ep, SecondProduct{}, stream);
  }
  if (pair) return launch_bn<A_MN, B_MN, KIND, 2>(A, B, M, N, K, ep, SecondProduct{}, stream);
  return launch_bn<A_MN, B_MN, KIND, 1>(A, B, M, N, K, ep, SecondProduct{}, stream);
}

}  // namespace

cudaError_t launch_tc_gemm_dagger(int M, int N, int K, const void* A, const void* B_gate, const void* B_up,
                                  const EpiParams& ep, cudaStream_t stream) {
  if (M <= 0 || N <= 0) return cudaSuccess;
  if (K <= 0 || (N % 8) || (K % 8)) return cudaErrorNotSupported;
  // CTA pairs; 256 x 128 tiles of BOTH products: 2 x 2 x 128 accumulator columns fill TMEM, and a
  // stage holds the A block and the two B blocks (32 KB per CTA), five stages deep
  constexpr int BN = 128, STAGES = 5, CTAS = 2;
  CUtensorMap tmA, tmB, tmC0, tmC1;
  SecondMaps sec;
  sec.maps = true;
  bool ok = encode_map(&tmA, A, M, K, BM) && encode_map(&tmB, B_gate, N, K, BN / CTAS) &&
            encode_map(&sec.B, B_up, N, K, BN / CTAS) && encode_out_map(&tmC0, ep.H, M, N, false);
  if (ep.G) ok = ok && encode_out_map(&tmC1, ep.G, M, N, false); else tmC1 = tmC0;
  if (ep.U) ok = ok && encode_out_map(&sec.C, ep.U, M, N, false); else sec.C = tmC0;
  if (!ok) return cudaErrorNotSupported;
  auto a32 = [](const void* p) { return (reinterpret_cast<uintptr_t>(p) & 31u) == 0; };
  if ((N % 16 == 0) && a32(ep.E))
    return launch_inst<false, false, kEpiDagger, BN, STAGES, true, CTAS>(tmA, tmB, tmC0, tmC1, M, N, K, ep, 0, 1, sec, stream);
  return launch_inst<false, false, kEpiDagger, BN, STAGES, false, CTAS>(tmA, tmB, tmC0, tmC1, M, N, K, ep, 0, 1, sec, stream);
}

cudaError_t launch_tc_gemm_token_pair(int K, int M1, int N1, const void* A1, const void* B1, void* out1, int M2,
                                      int N2, const void* A2, const void* B2, void* out2, const EpiParams& ep,
                                      bool pair, cudaStream_t stream) {
  if (K <= 0 || M1 <= 0 || N1 <= 0 || M2 <= 0 || N2 <= 0) return cudaErrorNotSupported;
  if ((M1 % 8) || (N1 % 8) || (M2 % 8) || (N2 % 8)) return cudaErrorNotSupported;
  EpiParams p = ep;
  p.out = out1;
  SecondProduct second;
  second.M = M2; second.N = N2; second.A = A2; second.B = B2; second.out = out2;
  if (pair) return launch_bn<true, true, kEpiStore, 2>(A1, B1, M1, N1, K, p, second, stream);
  return launch_bn<true, true, kEpiStore, 1>(A1, B1, M1, N1, K, p, second, stream);
}

size_t tc_gemm_scratch_bytes() {
  // room for 296 partial 256 x 256 fp32 tiles: up to four pieces for each of the at most 73
  // tail tiles of a pair launch (twice as many 128 x 256 tiles for single CTAs)
  return static_cast<size_t>(4) * 148 * 128 * 256 * sizeof(float);
}

cudaError_t launch_tc_gemm(int M, int N, int K, const void* A, bool a_mn, const void* B, bool b_mn,
                           EpiKind kind, const EpiParams& ep, bool pair, cudaStream_t stream) {
  if (M <= 0 || N <= 0) return cudaSuccess;
  // TMA needs 16-byte row pitches (the contiguous extent of each operand a multiple of 8
  // elements); the epilogue stores 8 columns at a time.
  if (K <= 0 || (N % 8) || ((a_mn ? M : K) % 8) || ((b_mn ? N : K) % 8)) return cudaErrorNotSupported;
  // layer call sites: gate (K,K,gate)  down (K,K,store)  dH (K,MN,dh)  dx (K,MN,store)
  //                   dW_down / dW_gate (MN,MN,store); the plain-GEMM entry adds (MN,K,store)
  if (!a_mn && !b_mn) {
    if (kind == kEpiGate) return launch_ctas<false, false, kEpiGate>(A, B, M, N, K, ep, pair, stream);
    if (kind == kEpiAdd) return launch_ctas<false, false, kEpiAdd>(A, B, M, N, K, ep, pair, stream);
    if (kind == kEpiStore) return launch_ctas<false, false, kEpiStore>(A, B, M, N, K, ep, pair, stream);
  } else if (!a_mn && b_mn) {
    if (kind == kEpiDH) return launch_ctas<false, true, kEpiDH>(A, B, M, N, K, ep, pair, stream);
    if (kind == kEpiAdd) return launch_ctas<false, true, kEpiAdd>(A, B, M, N, K, ep, pair, stream);
    if (kind == kEpiStore) return launch_ctas<false, true, kEpiStore>(A, B, M, N, K, ep, pair, stream);
  } else if (a_mn && b_mn) {
    if (kind == kEpiStore) return launch_ctas<true, true, kEpiStore>(A, B, M, N, K, ep, pair, stream);
  } else {
    if (kind == kEpiStore) return launch_ctas<true, false, kEpiStore>(A, B, M, N, K, ep, pair, stream);
  }
  return cudaErrorNotSupported;
}

}  // namespace stem
