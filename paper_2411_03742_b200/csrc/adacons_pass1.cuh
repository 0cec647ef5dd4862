// Pass 1 (Eq. 7 of arXiv 2411.03742): column sums, then per worker N p_i = sum_k g_ik s_k and q_i = sum_k g_ik^2,
// one partial record per block (or per segment a block meets).  All variants: TMA-staged tiles for N <= 64, tall
// tiles for N <= 256, column sums + dot products for larger N, thread-block clusters (opt-in), per-segment, generic.
#pragma once

#include "adacons_common.cuh"

namespace adacons {

// ----------------------------------------------------------------------------------------------
// Pass 1, TMA-staged (N <= 64, 16-byte aligned rows).
//
// A tile is WC boxes of N rows x 512 bytes, laid side by side; the 8 warps form a WR x WC grid
// (WR * WC = 8): warp (rw, cw) reads box cw and rows rw, rw+WR, ... (NR of them); lane l owns the
// 16-byte column group l of the box.  Per tile every thread
//   1. copies its NR row vectors from shared memory to registers,
//   2. adds them up (partial column sums); with WR > 1 the WR partials are exchanged through
//      shared memory and added in a fixed order (p1_xch_finish), giving the column sums s,
//   3. accumulates, per row, sum x*s and sum x*x in fp32 (two lanes of packed fp32 FMA).
// One elected thread refills a stage by TMA as soon as the block has copied it to registers.
//
// Two kernels share these steps: pass1_tma_kernel (one set of coefficients for the whole vector;
// a block owns tiles b, b+grid, ...) and pass1_seg_kernel (one set per segment; a block owns a
// contiguous tile range and writes one partial record per segment it meets).
// ----------------------------------------------------------------------------------------------
template <int DT, int NR_, int WR_>
struct P1 {
  static constexpr int NR = NR_, WR = WR_;
  static constexpr int WC = kWarps / WR;
  static constexpr int VEC = Elem<DT>::kVec;
  static constexpr int NP = VEC / 2;
  static constexpr int BOXC = kBoxRowBytes / Elem<DT>::kBytes;   // columns per box
  static constexpr int TILEC = WC * BOXC;                        // columns per tile
  static constexpr int kXchOne = WR * WC * 32 * VEC;             // floats of one exchange buffer
  static constexpr int kXchFloats = (WR > 1) ? 2 * kXchOne : 0;
  static constexpr int kRedFloats = kWarps * NR * 2;
  static constexpr int kOuterFloats = 2 * NR * kThreads;        // second-level accumulators, [2][NR][thread]
  static constexpr int kBlockThreads = kThreads;
};

struct P1Smem {            // carve-up of the dynamic shared memory of both pass-1 kernels
  unsigned char* stage_base;
  float* xch;
  float* red;
  float* outer;
  uint64_t* full;
};
template <class C>
__device__ __forceinline__ P1Smem p1_carve(unsigned char* raw, int stages, uint32_t stage_bytes) {
  P1Smem s;
  s.stage_base = raw;
  s.xch = reinterpret_cast<float*>(raw + static_cast<size_t>(stages) * stage_bytes);
  s.red = s.xch + C::kXchFloats;
  s.outer = s.red + C::kRedFloats;
  s.full = reinterpret_cast<uint64_t*>(s.outer + C::kOuterFloats);
  return s;
}

// rows of this thread from a landed stage (zeros for rows >= N)
template <class C>
__device__ __forceinline__ void p1_load_rows(uint4 (&v)[C::NR], const unsigned char* box_lane, int rw, int N) {
  if (N == C::NR * C::WR) {                  // every row exists (block-uniform): no per-row test
#pragma unroll
    for (int j = 0; j < C::NR; ++j) v[j] = ld_shared_v4(box_lane + (rw + C::WR * j) * kBoxRowBytes);
  } else {
#pragma unroll
    for (int j = 0; j < C::NR; ++j) {
      const int row = rw + C::WR * j;
      v[j] = (row < N) ? ld_shared_v4(box_lane + row * kBoxRowBytes) : make_uint4(0u, 0u, 0u, 0u);
    }
  }
}
template <int DT, class C>
__device__ __forceinline__ void p1_colsum(const uint4 (&v)[C::NR], float2 (&sp)[C::NP]) {
#pragma unroll
  for (int h = 0; h < C::NP; ++h) sp[h] = make_float2(0.f, 0.f);
#pragma unroll
  for (int j = 0; j < C::NR; ++j)
#pragma unroll
    for (int h = 0; h < C::NP; ++h) sp[h] = __fadd2_rn(sp[h], unpack_pair<DT>(v[j], h));
}
// exchange layout [rw][cw][16-byte half h2][lane][4 floats]: conflict-free 16-byte accesses
template <class C>
__device__ __forceinline__ void p1_xch_write(float* xbuf, const float2 (&sp)[C::NP], int rw, int cw, int lane) {
#pragma unroll
  for (int h2 = 0; h2 < C::VEC / 4; ++h2) {
    const float4 w4 = make_float4(sp[2 * h2].x, sp[2 * h2].y, sp[2 * h2 + 1].x, sp[2 * h2 + 1].y);
    *reinterpret_cast<float4*>(xbuf + ((rw * C::WC + cw) * (C::VEC / 4) + h2) * 128 + lane * 4) = w4;
  }
}
template <class C>
__device__ __forceinline__ void p1_xch_read(const float* xbuf, float2 (&sp)[C::NP], int cw, int lane) {
#pragma unroll
  for (int h = 0; h < C::NP; ++h) sp[h] = make_float2(0.f, 0.f);
#pragma unroll
  for (int r = 0; r < C::WR; ++r)
#pragma unroll
    for (int h2 = 0; h2 < C::VEC / 4; ++h2) {
      const float4 w4 = *reinterpret_cast<const float4*>(xbuf + ((r * C::WC + cw) * (C::VEC / 4) + h2) * 128 + lane * 4);
      sp[2 * h2] = __fadd2_rn(sp[2 * h2], make_float2(w4.x, w4.y));
      sp[2 * h2 + 1] = __fadd2_rn(sp[2 * h2 + 1], make_float2(w4.z, w4.w));
    }
}
// Where a tile's partial column sums are written, and how they become the column sums.
// WR < 8: double-buffered partials, every thread adds the WR partials of its own column group.
// WR = 8: adding 8 partials per thread costs more than the tile's own arithmetic warrants, so the
// 256 threads first finish one column each (the 8 partials in rw order) into the second half of
// the exchange area, meet at a second barrier, and read back the finished sums of their group.
template <class C>
__device__ __forceinline__ float* p1_xch_buffer(float* xch, int k) {
  return (C::WR == 8) ? xch : xch + (k & 1) * C::kXchOne;
}
template <class C>
__device__ __forceinline__ void p1_xch_finish(float* xch, int k, float2 (&sp)[C::NP], int cw, int lane) {
  if constexpr (C::WR == 8) {
    constexpr int per = C::kXchOne / C::WR;
    float* sbuf = xch + C::kXchOne;
    for (int idx = threadIdx.x; idx < per; idx += kThreads) {
      float a = 0.f;
#pragma unroll
      for (int r = 0; r < C::WR; ++r) a += xch[r * per + idx];
      sbuf[idx] = a;
    }
    __syncthreads();
#pragma unroll
    for (int h2 = 0; h2 < C::VEC / 4; ++h2) {
      const float4 w4 = *reinterpret_cast<const float4*>(sbuf + (cw * (C::VEC / 4) + h2) * 128 + lane * 4);
      sp[2 * h2] = make_float2(w4.x, w4.y);
      sp[2 * h2 + 1] = make_float2(w4.z, w4.w);
    }
  } else if constexpr (C::WR > 1) {
    p1_xch_read<C>(xch + (k & 1) * C::kXchOne, sp, cw, lane);
  }
}
template <int DT, class C>
__device__ __forceinline__ void p1_accumulate(const uint4 (&v)[C::NR], const float2 (&sp)[C::NP],
                                              float2 (&pacc)[C::NR], float2 (&qacc)[C::NR]) {
#pragma unroll
  for (int j = 0; j < C::NR; ++j)
#pragma unroll
    for (int h = 0; h < C::NP; ++h) {
      const float2 x = unpack_pair<DT>(v[j], h);
      pacc[j] = __ffma2_rn(x, sp[h], pacc[j]);
      qacc[j] = __ffma2_rn(x, x, qacc[j]);
    }
}
// same, counting only the columns lo <= col < hi; col0 = column of this lane's first element
template <int DT, class C>
__device__ __forceinline__ void p1_accumulate_masked(const uint4 (&v)[C::NR], const float2 (&sp)[C::NP],
                                                     float2 (&pacc)[C::NR], float2 (&qacc)[C::NR],
                                                     long long col0, long long lo, long long hi) {
#pragma unroll
  for (int j = 0; j < C::NR; ++j)
#pragma unroll
    for (int h = 0; h < C::NP; ++h) {
      float2 x = unpack_pair<DT>(v[j], h);
      const long long c = col0 + 2 * h;
      if (c < lo || c >= hi) x.x = 0.f;
      if (c + 1 < lo || c + 1 >= hi) x.y = 0.f;
      pacc[j] = __ffma2_rn(x, sp[h], pacc[j]);
      qacc[j] = __ffma2_rn(x, x, qacc[j]);
    }
}
// Two-level accumulation.  A thread's fp32 sums are folded into second-level accumulators (in
// shared memory, one slot per thread and row) every kFoldTiles tiles.  Long fp32 sums of squares of
// bf16 values are not merely noisy but biased: such squares have few, structured significant bits,
// so once the running sum is large they round down more often than up (q was 9e-6 low after 18k
// terms per accumulator at d = 340M).  Kept below ~128 terms the first level is exact for typical
// data, and the second level adds full-width values, whose rounding is unbiased.
constexpr int kFoldTiles = 32;
template <class C>
__device__ __forceinline__ void p1_outer_clear(float* outer) {
#pragma unroll
  for (int j = 0; j < 2 * C::NR; ++j) outer[j * C::kBlockThreads + threadIdx.x] = 0.f;
}
template <class C>
__device__ __forceinline__ void p1_fold(float2 (&pacc)[C::NR], float2 (&qacc)[C::NR], float* outer) {
#pragma unroll
  for (int j = 0; j < C::NR; ++j) {
    outer[j * C::kBlockThreads + threadIdx.x] += pacc[j].x + pacc[j].y;
    outer[(C::NR + j) * C::kBlockThreads + threadIdx.x] += qacc[j].x + qacc[j].y;
    pacc[j] = qacc[j] = make_float2(0.f, 0.f);
  }
}
// Block partial of the accumulators (both levels): lanes (fixed xor tree), then the WC warps that
// share a row (fixed order).  dst_p[0..rows) = N p_i (un-divided), dst_q[0..rows) = q_i.  Contains
// two barriers; both levels are reset.
template <class C>
__device__ __forceinline__ void p1_block_store(float2 (&pacc)[C::NR], float2 (&qacc)[C::NR], float* outer, float* red,
                                               float* dst_p, float* dst_q, int rows) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  p1_fold<C>(pacc, qacc, outer);
#pragma unroll
  for (int j = 0; j < C::NR; ++j) {
    float p = outer[j * kThreads + tid], q = outer[(C::NR + j) * kThreads + tid];
    outer[j * kThreads + tid] = 0.f;
    outer[(C::NR + j) * kThreads + tid] = 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      p += __shfl_xor_sync(0xffffffffu, p, o);
      q += __shfl_xor_sync(0xffffffffu, q, o);
    }
    if (lane == 0) {
      red[(warp * C::NR + j) * 2 + 0] = p;
      red[(warp * C::NR + j) * 2 + 1] = q;
    }
  }
  __syncthreads();
  if (tid < rows) {
    const int r_w = tid % C::WR, j = tid / C::WR;
    float p = 0.f, q = 0.f;
#pragma unroll
    for (int c = 0; c < C::WC; ++c) {
      p += red[((c * C::WR + r_w) * C::NR + j) * 2 + 0];
      q += red[((c * C::WR + r_w) * C::NR + j) * 2 + 1];
    }
    dst_p[tid] = p;
    dst_q[tid] = q;
  }
  __syncthreads();
}
// After a bounded wait expired: wait (bounded) for the copies still in flight into this block's
// shared memory so that the block may exit, and report.
__device__ __forceinline__ void p1_drain_after_timeout(uint64_t* full, int stages, int issued, uint32_t* flags) {
  for (int k = (issued > stages ? issued - stages : 0); k < issued; ++k)
    (void)mbar_wait_bounded(&full[k % stages], static_cast<uint32_t>(k / stages) & 1u);
  atomicOr(flags, kFlagTimeout);
}

struct Pass1Params {
  int N;
  int num_tiles;        // ceil(d / tile columns)
  int stages;           // ring depth
  uint32_t stage_bytes; // WC * N * 512
  float* partials;      // [gridDim.x][2N]: N p_i (un-divided) then q_i
  uint32_t* flags;      // device status word
};

template <int DT, int NR, int WR>
__global__ void __launch_bounds__(kThreads, 2)
pass1_tma_kernel(const __grid_constant__ CUtensorMap tmap, const Pass1Params prm) {
  using C = P1<DT, NR, WR>;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  __shared__ int s_abort;
  const int N = prm.N;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int cw = warp / WR, rw = warp % WR;
  const P1Smem sm = p1_carve<C>(smem_raw, prm.stages, prm.stage_bytes);

  if (tid == 0) {
    s_abort = 0;
    for (int s = 0; s < prm.stages; ++s) mbar_init(&sm.full[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async_smem();
  }
  __syncthreads();
  pdl_launch_dependents();

  const int first = blockIdx.x;
  const int stride = gridDim.x;
  const int my_tiles = first < prm.num_tiles ? (prm.num_tiles - first + stride - 1) / stride : 0;

  auto issue = [&](int k, int s) {   // elected thread: fill stage s with tile k of this block
    const int col0 = (first + k * stride) * C::TILEC;
    mbar_expect_tx(&sm.full[s], prm.stage_bytes);
#pragma unroll
    for (int c = 0; c < C::WC; ++c)
      tma_load_2d(sm.stage_base + static_cast<size_t>(s) * prm.stage_bytes + static_cast<size_t>(c) * N * kBoxRowBytes,
                  &tmap, &sm.full[s], col0 + c * C::BOXC, 0);
  };
  int issued = 0;                    // meaningful in thread 0 only
  if (tid == 0) {
    const int pre = my_tiles < prm.stages ? my_tiles : prm.stages;
    for (int k = 0; k < pre; ++k) issue(k, k);
    issued = pre;
  }

  float2 pacc[NR], qacc[NR];
#pragma unroll
  for (int j = 0; j < NR; ++j) pacc[j] = qacc[j] = make_float2(0.f, 0.f);
  p1_outer_clear<C>(sm.outer);

  int s = 0;
  uint32_t parity = 0;
  for (int k = 0; k < my_tiles; ++k) {
    uint4 v[NR];
    if (mbar_wait_bounded(&sm.full[s], parity)) {
      p1_load_rows<C>(v, sm.stage_base + static_cast<size_t>(s) * prm.stage_bytes +
                             static_cast<size_t>(cw) * N * kBoxRowBytes + lane * 16, rw, N);
    } else {
#pragma unroll
      for (int j = 0; j < NR; ++j) v[j] = make_uint4(0u, 0u, 0u, 0u);
      atomicOr(&s_abort, 1);
    }
    float2 sp[C::NP];
    p1_colsum<DT, C>(v, sp);
    float* xbuf = p1_xch_buffer<C>(sm.xch, k);
    if (WR > 1) p1_xch_write<C>(xbuf, sp, rw, cw, lane);
    __syncthreads();   // every thread holds its rows in registers; exchange buffer is written
    if (s_abort) break;
    if (tid == 0 && k + prm.stages < my_tiles) {
      fence_proxy_async_smem();
      issue(k + prm.stages, s);
      issued = k + prm.stages + 1;
    }
    p1_xch_finish<C>(sm.xch, k, sp, cw, lane);
    p1_accumulate<DT, C>(v, sp, pacc, qacc);
    if ((k & (kFoldTiles - 1)) == kFoldTiles - 1) p1_fold<C>(pacc, qacc, sm.outer);
    if (++s == prm.stages) { s = 0; parity ^= 1u; }
  }

  float* dst = prm.partials + static_cast<size_t>(blockIdx.x) * 2 * N;
  if (s_abort) {
    if (tid == 0) p1_drain_after_timeout(sm.full, prm.stages, issued, prm.flags);
    if (tid < 2 * N) dst[tid] = 0.f;
    return;
  }
  p1_block_store<C>(pacc, qacc, sm.outer, sm.red, dst, dst + N, N);
}

// ---- pass 1 for more than 64 workers: column sums first, then dot products per 64-row chunk -----
// With N > 64 a tile of all rows no longer fits the ring.  colsum_kernel streams the matrix once
// and leaves the column sums s (fp32) in scratch; pass1_dot_kernel then runs once per chunk of 64
// rows with the same boxes, ring and warp grid as pass1_tma_kernel<DT, 8, 8>, reading s instead of
// exchanging partial sums, and writes its rows' slice of the block partial.  Pass 1 costs two
// reads of the matrix instead of one.
template <int DT>
__global__ void __launch_bounds__(kThreads)
colsum_kernel(const unsigned char* __restrict__ grads, float* __restrict__ s_out, int N, long long row_bytes,
              long long num_vec, int tail_elems) {
  constexpr int VEC = Elem<DT>::kVec;
  constexpr int NP = VEC / 2;
  constexpr int U = 8;
  const long long v = static_cast<long long>(blockIdx.x) * kThreads + threadIdx.x;
  if (v >= num_vec) return;
  const unsigned char* col = grads + v * 16;
  float2 acc[NP];
#pragma unroll
  for (int h = 0; h < NP; ++h) acc[h] = make_float2(0.f, 0.f);
  int i0 = 0;
  for (; i0 + U <= N; i0 += U) {
    uint4 x[U];
#pragma unroll
    for (int u = 0; u < U; ++u) x[u] = ld_stream_v4(col + static_cast<long long>(i0 + u) * row_bytes);
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int h = 0; h < NP; ++h) acc[h] = __fadd2_rn(acc[h], unpack_pair<DT>(x[u], h));
  }
  for (; i0 < N; ++i0) {
    const uint4 x = ld_stream_v4(col + static_cast<long long>(i0) * row_bytes);
#pragma unroll
    for (int h = 0; h < NP; ++h) acc[h] = __fadd2_rn(acc[h], unpack_pair<DT>(x, h));
  }
  float* dst = s_out + v * VEC;
#pragma unroll
  for (int e = 0; e < VEC; ++e) {
    float x = (e & 1) ? acc[e / 2].y : acc[e / 2].x;
    if (tail_elems != 0 && v == num_vec - 1 && e >= tail_elems) x = 0.f;   // row padding is not data
    dst[e] = x;
  }
}

struct Pass1DotParams {
  int N;                // all workers (row pitch of the partials)
  int r0;               // first row of this chunk
  int rows;             // rows in this chunk (<= 64)
  int num_tiles;
  int stages;
  uint32_t stage_bytes; // 64 * 512
  const float* s;       // column sums, zero past d, padded to a whole tile
  float* partials;      // [gridDim.x][2N]
  uint32_t* flags;
};

template <int DT>
__global__ void __launch_bounds__(kThreads, 2)
pass1_dot_kernel(const __grid_constant__ CUtensorMap tmap, const Pass1DotParams prm) {
  using C = P1<DT, 8, 8>;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  __shared__ int s_abort;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int rw = warp;                               // WR = 8, WC = 1
  const P1Smem sm = p1_carve<C>(smem_raw, prm.stages, prm.stage_bytes);
  if (tid == 0) {
    s_abort = 0;
    for (int s = 0; s < prm.stages; ++s) mbar_init(&sm.full[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async_smem();
  }
  __syncthreads();
  const int first = blockIdx.x, stride = gridDim.x;
  const int my_tiles = first < prm.num_tiles ? (prm.num_tiles - first + stride - 1) / stride : 0;
  auto issue = [&](int k, int s) {
    mbar_expect_tx(&sm.full[s], prm.stage_bytes);
    tma_load_2d(sm.stage_base + static_cast<size_t>(s) * prm.stage_bytes, &tmap, &sm.full[s],
                (first + k * stride) * C::TILEC, prm.r0);
  };
  int issued = 0;
  if (tid == 0) {
    const int pre = my_tiles < prm.stages ? my_tiles : prm.stages;
    for (int k = 0; k < pre; ++k) issue(k, k);
    issued = pre;
  }
  float2 pacc[8], qacc[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) pacc[j] = qacc[j] = make_float2(0.f, 0.f);
  p1_outer_clear<C>(sm.outer);
  int s = 0;
  uint32_t parity = 0;
  for (int k = 0; k < my_tiles; ++k) {
    // column sums of this thread's 16-byte group (in flight while the tile lands)
    float2 sp[C::NP];
    const float* sv = prm.s + static_cast<long long>(first + k * stride) * C::TILEC + lane * C::VEC;
#pragma unroll
    for (int h2 = 0; h2 < C::VEC / 4; ++h2) {
      const float4 w4 = __ldg(reinterpret_cast<const float4*>(sv) + h2);
      sp[2 * h2] = make_float2(w4.x, w4.y);
      sp[2 * h2 + 1] = make_float2(w4.z, w4.w);
    }
    uint4 v[8];
    if (mbar_wait_bounded(&sm.full[s], parity)) {
      p1_load_rows<C>(v, sm.stage_base + static_cast<size_t>(s) * prm.stage_bytes + lane * 16, rw, 64);
    } else {
#pragma unroll
      for (int j = 0; j < 8; ++j) v[j] = make_uint4(0u, 0u, 0u, 0u);
      atomicOr(&s_abort, 1);
    }
    __syncthreads();                                   // the stage is in registers
    if (s_abort) break;
    if (tid == 0 && k + prm.stages < my_tiles) {
      fence_proxy_async_smem();
      issue(k + prm.stages, s);
      issued = k + prm.stages + 1;
    }
    p1_accumulate<DT, C>(v, sp, pacc, qacc);
    if ((k & (kFoldTiles - 1)) == kFoldTiles - 1) p1_fold<C>(pacc, qacc, sm.outer);
    if (++s == prm.stages) { s = 0; parity ^= 1u; }
  }
  float* dst = prm.partials + static_cast<size_t>(blockIdx.x) * 2 * prm.N;
  if (s_abort) {
    if (tid == 0) p1_drain_after_timeout(sm.full, prm.stages, issued, prm.flags);
    if (tid < prm.rows) { dst[prm.r0 + tid] = 0.f; dst[prm.N + prm.r0 + tid] = 0.f; }
    return;
  }
  p1_block_store<C>(pacc, qacc, sm.outer, sm.red, dst + prm.r0, dst + prm.N + prm.r0, prm.rows);
}

// ---- pass 1 for 64 < N <= 256 in one read, one block per tile: taller, narrower boxes ------------
// More rows than pass1_tma_kernel's tallest tile at a fraction of the width, so a stage is still
// 32 KB: 128 rows x 256 bytes (LPR = 16 lanes per row: a HALF-warp owns a row) or 256 rows x 128
// bytes (LPR = 8: a quarter-warp; TMA moves 128-byte box rows at 4.6 TB/s at most on this GPU, which
// is still more than two reads at full speed).  With TH = 512 threads and LPR = 16 a block takes
// 256 rows x 256 bytes (64 KB per stage, one block per SM).  Lane l of warp w belongs to row group
// g = (32 / LPR) w + l / LPR and owns the 16-byte column group l % LPR of rows g, g + G, ...,
// g + 7 G (8 rows, as before; G = 8 * 32 / LPR groups; rows past N are zero-filled by TMA).  The
// groups' partial column sums are exchanged through shared memory in two steps -- every thread
// first finishes one column of its share of the groups, in group order, then all read the sums of
// their own columns -- and the lane reduction at the end stays inside the LPR lanes of a row.
// Same partial-record layout as pass1_tma_kernel.
template <int DT, int LPR, int TH = kThreads>
struct P1H {
  static constexpr int NR = 8;
  static constexpr int kBlockThreads = TH;
  static constexpr int VEC = Elem<DT>::kVec;
  static constexpr int NP = VEC / 2;
  static constexpr int kLanesPerRow = LPR;
  static constexpr int kGroups = (TH / 32) * (32 / LPR), kRows = kGroups * NR;
  static constexpr int kBoxRowBytesH = LPR * 16;
  static constexpr int TILEC = kBoxRowBytesH / Elem<DT>::kBytes;   // columns per tile
  static constexpr int PARTS = TH / TILEC;                         // threads per column in the first exchange step
  static constexpr int kGroupsPerPart = kGroups / PARTS;
  static constexpr uint32_t kStageBytes = kRows * kBoxRowBytesH;   // 32 KB (64 KB with 512 threads)
  static constexpr int kXchFloats = kGroups * TILEC;
  static constexpr int kSumFloats = PARTS * TILEC;                 // = TH
  static constexpr int kRedFloats = kGroups * NR * 2;
  static constexpr int kOuterFloats = 2 * NR * TH;
  static constexpr size_t kFixedBytes = (kXchFloats + kSumFloats + kRedFloats + kOuterFloats) * sizeof(float);
};

template <int DT, int LPR, int TH>
__global__ void __launch_bounds__(TH, TH == kThreads ? 2 : 1)
pass1_tall_kernel(const __grid_constant__ CUtensorMap tmap, const Pass1Params prm) {
  using C = P1H<DT, LPR, TH>;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  __shared__ int s_abort;
  const int N = prm.N;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = (32 / LPR) * warp + lane / LPR, cl = lane % LPR;
  unsigned char* stage_base = smem_raw;
  float* xch = reinterpret_cast<float*>(smem_raw + static_cast<size_t>(prm.stages) * C::kStageBytes);
  float* sums = xch + C::kXchFloats;
  float* red = sums + C::kSumFloats;
  float* outer = red + C::kRedFloats;
  uint64_t* full = reinterpret_cast<uint64_t*>(outer + C::kOuterFloats);
  if (tid == 0) {
    s_abort = 0;
    for (int s = 0; s < prm.stages; ++s) mbar_init(&full[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async_smem();
  }
  __syncthreads();
  pdl_launch_dependents();
  const int first = blockIdx.x, stride = gridDim.x;
  const int my_tiles = first < prm.num_tiles ? (prm.num_tiles - first + stride - 1) / stride : 0;
  auto issue = [&](int k, int s) {
    mbar_expect_tx(&full[s], C::kStageBytes);
    tma_load_2d(stage_base + static_cast<size_t>(s) * C::kStageBytes, &tmap, &full[s], (first + k * stride) * C::TILEC, 0);
  };
  int issued = 0;
  if (tid == 0) {
    const int pre = my_tiles < prm.stages ? my_tiles : prm.stages;
    for (int k = 0; k < pre; ++k) issue(k, k);
    issued = pre;
  }
  float2 pacc[C::NR], qacc[C::NR];
#pragma unroll
  for (int j = 0; j < C::NR; ++j) pacc[j] = qacc[j] = make_float2(0.f, 0.f);
  p1_outer_clear<C>(outer);
  int s = 0;
  uint32_t parity = 0;
  for (int k = 0; k < my_tiles; ++k) {
    uint4 v[C::NR];
    if (mbar_wait_bounded(&full[s], parity)) {
      const unsigned char* mine = stage_base + static_cast<size_t>(s) * C::kStageBytes + g * C::kBoxRowBytesH + cl * 16;
#pragma unroll
      for (int j = 0; j < C::NR; ++j) v[j] = ld_shared_v4(mine + j * (C::kGroups * C::kBoxRowBytesH));
    } else {
#pragma unroll
      for (int j = 0; j < C::NR; ++j) v[j] = make_uint4(0u, 0u, 0u, 0u);
      atomicOr(&s_abort, 1);
    }
    float2 sp[C::NP];
    p1_colsum<DT, C>(v, sp);
#pragma unroll
    for (int h2 = 0; h2 < C::VEC / 4; ++h2)            // this group's partial sums of the thread's VEC columns
      *reinterpret_cast<float4*>(xch + g * C::TILEC + cl * C::VEC + 4 * h2) =
          make_float4(sp[2 * h2].x, sp[2 * h2].y, sp[2 * h2 + 1].x, sp[2 * h2 + 1].y);
    __syncthreads();                                    // the stage is in registers; the partials are written
    if (s_abort) break;
    if (tid == 0 && k + prm.stages < my_tiles) {
      fence_proxy_async_smem();
      issue(k + prm.stages, s);
      issued = k + prm.stages + 1;
    }
    {                                                   // step 1: one column, this thread's share of the groups, in group order
      const int c = tid % C::TILEC, part = tid / C::TILEC;
      float a = 0.f;
#pragma unroll
      for (int r = 0; r < C::kGroupsPerPart; ++r) a += xch[(part * C::kGroupsPerPart + r) * C::TILEC + c];
      sums[part * C::TILEC + c] = a;
    }
    __syncthreads();
#pragma unroll
    for (int h = 0; h < C::NP; ++h) sp[h] = make_float2(0.f, 0.f);
#pragma unroll
    for (int part = 0; part < C::PARTS; ++part)         // step 2: the parts in order
#pragma unroll
      for (int h2 = 0; h2 < C::VEC / 4; ++h2) {
        const float4 w4 = *reinterpret_cast<const float4*>(sums + part * C::TILEC + cl * C::VEC + 4 * h2);
        sp[2 * h2] = __fadd2_rn(sp[2 * h2], make_float2(w4.x, w4.y));
        sp[2 * h2 + 1] = __fadd2_rn(sp[2 * h2 + 1], make_float2(w4.z, w4.w));
      }
    p1_accumulate<DT, C>(v, sp, pacc, qacc);
    if ((k & (kFoldTiles - 1)) == kFoldTiles - 1) p1_fold<C>(pacc, qacc, outer);
    if (++s == prm.stages) { s = 0; parity ^= 1u; }
  }
  float* dst = prm.partials + static_cast<size_t>(blockIdx.x) * 2 * N;
  if (s_abort) {
    if (tid == 0) p1_drain_after_timeout(full, prm.stages, issued, prm.flags);
    for (int i = tid; i < 2 * N; i += TH) dst[i] = 0.f;
    return;
  }
  // block partial: both accumulation levels, the lanes of a row by a fixed xor tree; every row has one owner group
  p1_fold<C>(pacc, qacc, outer);
#pragma unroll
  for (int j = 0; j < C::NR; ++j) {
    float p = outer[j * TH + tid], q = outer[(C::NR + j) * TH + tid];
#pragma unroll
    for (int o = LPR / 2; o > 0; o >>= 1) {
      p += __shfl_xor_sync(0xffffffffu, p, o);
      q += __shfl_xor_sync(0xffffffffu, q, o);
    }
    if (cl == 0) {
      red[(g * C::NR + j) * 2 + 0] = p;
      red[(g * C::NR + j) * 2 + 1] = q;
    }
  }
  __syncthreads();
  if (tid < N) {                                        // row tid = group tid % kGroups, its (tid / kGroups)-th row
    const int rg = tid % C::kGroups, rj = tid / C::kGroups;
    dst[tid] = red[(rg * C::NR + rj) * 2 + 0];
    dst[N + tid] = red[(rg * C::NR + rj) * 2 + 1];
  }
}

// ---- pass 1 for 64 < N <= 512 in ONE read of the matrix: a thread-block cluster per column tile ----
// A cluster of C = 2, 4 or 8 blocks owns column tiles c, c + clusters, ...; block r of the cluster
// stages rows [64 r, 64 r + 64) of a tile (one TMA box; rows past N are zero-filled, a block with
// no rows at all stages nothing), adds them up as pass1_tma_kernel<DT, 8, 8> does, and leaves its
// 64-row column sums in its own shared memory.  After a cluster barrier every block reads the C
// partial column sums through distributed shared memory and adds them in rank order -- all blocks
// get the same bits -- and accumulates x*s and x*x for its own rows.  The partial sums are
// double-buffered, so one cluster barrier per tile suffices: a block overwrites buffer k & 1 only
// after the barrier of tile k + 1, which its peers reach after they have read tile k's sums.
// A cluster writes ONE partial record, each block its rows' slice.  A block whose wait on a copy
// expired keeps meeting its peers at every barrier (with zeros) so that nobody is left waiting.
__device__ __forceinline__ uint32_t cluster_ctarank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t cluster_nctarank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t cluster_id_x() { uint32_t r; asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t cluster_count_x() { uint32_t r; asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// 16 bytes from the shared memory of block `rank` of this cluster, at the address `local` has here
__device__ __forceinline__ float4 ld_cluster_v4(const float* local, uint32_t rank) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(smem_addr(local)), "r"(rank));
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(remote) : "memory");
  return v;
}

struct Pass1ClusterParams {
  int N;
  int num_tiles;
  int stages;
  uint32_t stage_bytes; // 64 * 512
  float* partials;      // [clusters][2N]
  uint32_t* flags;
};

template <int DT>
__global__ void __launch_bounds__(kThreads, 2)
pass1_cluster_kernel(const __grid_constant__ CUtensorMap tmap, const Pass1ClusterParams prm) {
  using C = P1<DT, 8, 8>;
  constexpr int VEC = C::VEC;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  __shared__ int s_abort;
  __shared__ __align__(16) float s_col[2][C::TILEC];    // this block's column sums of its 64 rows, in the exchange layout
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int rw = warp;                                  // WR = 8, WC = 1
  const uint32_t rank = cluster_ctarank(), csize = cluster_nctarank();
  const int cid = static_cast<int>(cluster_id_x()), ncl = static_cast<int>(cluster_count_x());
  const int r0 = static_cast<int>(rank) * 64;
  const int rows = prm.N - r0 < 0 ? 0 : (prm.N - r0 < 64 ? prm.N - r0 : 64);
  const bool idle = rows == 0;                          // a block beyond the last row only meets the barriers
  const P1Smem sm = p1_carve<C>(smem_raw, prm.stages, prm.stage_bytes);
  if (tid == 0) {
    s_abort = 0;
    for (int s = 0; s < prm.stages; ++s) mbar_init(&sm.full[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async_smem();
  }
  __syncthreads();
  const int my_tiles = cid < prm.num_tiles ? (prm.num_tiles - cid + ncl - 1) / ncl : 0;   // the same in every block of the cluster
  auto issue = [&](int k, int s) {
    mbar_expect_tx(&sm.full[s], prm.stage_bytes);
    tma_load_2d(sm.stage_base + static_cast<size_t>(s) * prm.stage_bytes, &tmap, &sm.full[s], (cid + k * ncl) * C::TILEC, r0);
  };
  int issued = 0;
  if (tid == 0 && !idle) {
    const int pre = my_tiles < prm.stages ? my_tiles : prm.stages;
    for (int k = 0; k < pre; ++k) issue(k, k);
    issued = pre;
  }
  float2 pacc[8], qacc[8];
#pragma unroll
  for (int j = 0; j < 8; ++j) pacc[j] = qacc[j] = make_float2(0.f, 0.f);
  p1_outer_clear<C>(sm.outer);
  int s = 0;
  uint32_t parity = 0;
  bool dead = false;                                    // block-uniform: a wait expired earlier
  for (int k = 0; k < my_tiles; ++k) {
    uint4 v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = make_uint4(0u, 0u, 0u, 0u);
    if (!idle && !dead) {
      if (mbar_wait_bounded(&sm.full[s], parity)) p1_load_rows<C>(v, sm.stage_base + static_cast<size_t>(s) * prm.stage_bytes + lane * 16, rw, 64);
      else atomicOr(&s_abort, 1);
    }
    float2 sp[C::NP];
    p1_colsum<DT, C>(v, sp);
    p1_xch_write<C>(sm.xch, sp, rw, 0, lane);
    __syncthreads();                                    // the stage is in registers, the partials are written
    if (s_abort) dead = true;
    if (tid == 0 && !idle && !dead && k + prm.stages < my_tiles) {
      fence_proxy_async_smem();
      issue(k + prm.stages, s);
      issued = k + prm.stages + 1;
    }
    float* mine = s_col[k & 1];
    for (int idx = tid; idx < C::TILEC; idx += kThreads) {   // this block's 64-row sum of one column, row warps in order
      float a = 0.f;
#pragma unroll
      for (int r = 0; r < 8; ++r) a += sm.xch[r * C::TILEC + idx];
      mine[idx] = a;
    }
    cluster_sync_all();
#pragma unroll
    for (int h = 0; h < C::NP; ++h) sp[h] = make_float2(0.f, 0.f);
    for (uint32_t r = 0; r < csize; ++r)                // blocks in rank order: the same sum everywhere
#pragma unroll
      for (int h2 = 0; h2 < VEC / 4; ++h2) {
        const float4 w4 = ld_cluster_v4(mine + h2 * 128 + lane * 4, r);
        sp[2 * h2] = __fadd2_rn(sp[2 * h2], make_float2(w4.x, w4.y));
        sp[2 * h2 + 1] = __fadd2_rn(sp[2 * h2 + 1], make_float2(w4.z, w4.w));
      }
    p1_accumulate<DT, C>(v, sp, pacc, qacc);
    if ((k & (kFoldTiles - 1)) == kFoldTiles - 1) p1_fold<C>(pacc, qacc, sm.outer);
    if (++s == prm.stages) { s = 0; parity ^= 1u; }
  }
  cluster_sync_all();                                   // nobody leaves while a peer may still read its column sums
  float* dst = prm.partials + static_cast<size_t>(cid) * 2 * prm.N;
  if (dead) {
    if (tid == 0) p1_drain_after_timeout(sm.full, prm.stages, issued, prm.flags);
    if (tid < rows) { dst[r0 + tid] = 0.f; dst[prm.N + r0 + tid] = 0.f; }
    return;
  }
  if (!idle) p1_block_store<C>(pacc, qacc, sm.outer, sm.red, dst + r0, dst + prm.N + r0, rows);
}

// ---- per-segment ("layer-wise") pass 1 ----------------------------------------------------------
// Block b owns the contiguous tile range [b*T/G, (b+1)*T/G).  The column sums of a tile do not
// depend on the segments; only the destination of x*s and x*x does.  The block keeps accumulators
// for its current segment and, whenever that segment ends inside (or at the end of) a tile,
// reduces them to one record and moves on; a tile that contains a boundary is accumulated once per
// segment it meets, with the columns outside the segment masked to zero.  Records of set s are
// contiguous: record (rec_begin[s] + b - set_first_block[s]) belongs to block b.
struct Pass1SegParams {
  int N;
  int num_tiles;
  int stages;
  uint32_t stage_bytes;
  long long d;
  const long long* seg_off;       // [S+1]
  const int* blk_first_seg;       // [grid] segment that contains the block's first column
  const int* blk_last_seg;        // [grid] segment that contains the block's last column
  const int* rec_begin;           // [S]
  const int* set_first_block;     // [S]
  float* records;                 // [num_records][2N]
  uint32_t* flags;
};

template <int DT, int NR, int WR>
__global__ void __launch_bounds__(kThreads, 2)
pass1_seg_kernel(const __grid_constant__ CUtensorMap tmap, const Pass1SegParams prm) {
  using C = P1<DT, NR, WR>;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  __shared__ int s_abort;
  const int N = prm.N;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int cw = warp / WR, rw = warp % WR;
  const P1Smem sm = p1_carve<C>(smem_raw, prm.stages, prm.stage_bytes);

  if (tid == 0) {
    s_abort = 0;
    for (int s = 0; s < prm.stages; ++s) mbar_init(&sm.full[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async_smem();
  }
  __syncthreads();
  pdl_launch_dependents();

  const int b = blockIdx.x, G = gridDim.x;
  const int t0 = static_cast<int>(static_cast<long long>(b) * prm.num_tiles / G);
  const int t1 = static_cast<int>(static_cast<long long>(b + 1) * prm.num_tiles / G);
  const int my_tiles = t1 - t0;

  auto issue = [&](int k, int s) {
    const int col0 = (t0 + k) * C::TILEC;
    mbar_expect_tx(&sm.full[s], prm.stage_bytes);
#pragma unroll
    for (int c = 0; c < C::WC; ++c)
      tma_load_2d(sm.stage_base + static_cast<size_t>(s) * prm.stage_bytes + static_cast<size_t>(c) * N * kBoxRowBytes,
                  &tmap, &sm.full[s], col0 + c * C::BOXC, 0);
  };
  int issued = 0;
  if (tid == 0) {
    const int pre = my_tiles < prm.stages ? my_tiles : prm.stages;
    for (int k = 0; k < pre; ++k) issue(k, k);
    issued = pre;
  }

  float2 pacc[NR], qacc[NR];
#pragma unroll
  for (int j = 0; j < NR; ++j) pacc[j] = qacc[j] = make_float2(0.f, 0.f);
  p1_outer_clear<C>(sm.outer);

  int seg = prm.blk_first_seg[b];
  const int last_seg = prm.blk_last_seg[b];
  long long seg_end = prm.seg_off[seg + 1];
  auto record = [&](int sg) -> float* {
    return prm.records + static_cast<size_t>(prm.rec_begin[sg] + b - prm.set_first_block[sg]) * 2 * N;
  };

  int s = 0;
  uint32_t parity = 0;
  for (int k = 0; k < my_tiles; ++k) {
    uint4 v[NR];
    if (mbar_wait_bounded(&sm.full[s], parity)) {
      p1_load_rows<C>(v, sm.stage_base + static_cast<size_t>(s) * prm.stage_bytes +
                             static_cast<size_t>(cw) * N * kBoxRowBytes + lane * 16, rw, N);
    } else {
#pragma unroll
      for (int j = 0; j < NR; ++j) v[j] = make_uint4(0u, 0u, 0u, 0u);
      atomicOr(&s_abort, 1);
    }
    float2 sp[C::NP];
    p1_colsum<DT, C>(v, sp);
    float* xbuf = p1_xch_buffer<C>(sm.xch, k);
    if (WR > 1) p1_xch_write<C>(xbuf, sp, rw, cw, lane);
    __syncthreads();
    if (s_abort) break;
    if (tid == 0 && k + prm.stages < my_tiles) {
      fence_proxy_async_smem();
      issue(k + prm.stages, s);
      issued = k + prm.stages + 1;
    }
    p1_xch_finish<C>(sm.xch, k, sp, cw, lane);

    const long long tile_lo = static_cast<long long>(t0 + k) * C::TILEC;
    const long long tile_hi = tile_lo + C::TILEC < prm.d ? tile_lo + C::TILEC : prm.d;
    if (seg_end > tile_hi || seg >= last_seg) {
      p1_accumulate<DT, C>(v, sp, pacc, qacc);                  // whole tile inside the current segment
    } else {
      const long long col0 = tile_lo + cw * C::BOXC + lane * C::VEC;
      long long lo = tile_lo;
      for (;;) {                                                // block-uniform control flow
        const long long hi = seg_end < tile_hi ? seg_end : tile_hi;
        if (hi > lo) p1_accumulate_masked<DT, C>(v, sp, pacc, qacc, col0, lo, hi);
        if (seg_end <= tile_hi && seg < last_seg) {
          p1_block_store<C>(pacc, qacc, sm.outer, sm.red, record(seg), record(seg) + N, N);
          ++seg;
          seg_end = prm.seg_off[seg + 1];
          lo = hi;                                              // empty segments fall through here
        } else {
          break;
        }
      }
    }
    if ((k & (kFoldTiles - 1)) == kFoldTiles - 1) p1_fold<C>(pacc, qacc, sm.outer);
    if (++s == prm.stages) { s = 0; parity ^= 1u; }
  }

  if (s_abort) {
    if (tid == 0) p1_drain_after_timeout(sm.full, prm.stages, issued, prm.flags);
    return;   // the records keep whatever they held; the status word says the result is invalid
  }
  p1_block_store<C>(pacc, qacc, sm.outer, sm.red, record(seg), record(seg) + N, N);
}

// ----------------------------------------------------------------------------------------------
// Pass 1, generic (any N <= 1024, any alignment, any d).  Thread t of a block owns CPT columns
// of a 256*CPT-column tile; it sums them over the rows (scalar, coalesced loads), then walks
// the rows again (cache hits), reduces x*s and x*x over the warp with a fixed xor tree and lets
// lane 0 add the result into the warp's own shared-memory accumulator.  Slow but always valid.
// ----------------------------------------------------------------------------------------------
template <int DT> __device__ __forceinline__ float load_elem(const void* base, long long idx);
template <> __device__ __forceinline__ float load_elem<0>(const void* base, long long idx) {
  return __ldg(reinterpret_cast<const float*>(base) + idx);
}
template <> __device__ __forceinline__ float load_elem<1>(const void* base, long long idx) {
  const unsigned short u = __ldg(reinterpret_cast<const unsigned short*>(base) + idx);
  return __uint_as_float(static_cast<uint32_t>(u) << 16);
}

template <int DT>
__global__ void __launch_bounds__(kThreads)
pass1_generic_kernel(const void* __restrict__ grads, int N, long long d, long long pitch, int num_tiles,
                     float* __restrict__ partials) {
  constexpr int CPT = 4;
  extern __shared__ float acc[];                   // [kWarps][N][2]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int i = tid; i < kWarps * N * 2; i += kThreads) acc[i] = 0.f;
  __syncthreads();
  float* mine = acc + static_cast<size_t>(warp) * N * 2;
  for (int t = blockIdx.x; t < num_tiles; t += gridDim.x) {
    const long long c0 = static_cast<long long>(t) * (kThreads * CPT) + tid;
    float s[CPT];
#pragma unroll
    for (int c = 0; c < CPT; ++c) s[c] = 0.f;
    for (int i = 0; i < N; ++i)
#pragma unroll
      for (int c = 0; c < CPT; ++c) {
        const long long col = c0 + c * kThreads;
        if (col < d) s[c] += load_elem<DT>(grads, static_cast<long long>(i) * pitch + col);
      }
    for (int i = 0; i < N; ++i) {
      float p = 0.f, q = 0.f;
#pragma unroll
      for (int c = 0; c < CPT; ++c) {
        const long long col = c0 + c * kThreads;
        if (col < d) {
          const float x = load_elem<DT>(grads, static_cast<long long>(i) * pitch + col);
          p = fmaf(x, s[c], p);
          q = fmaf(x, x, q);
        }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        p += __shfl_xor_sync(0xffffffffu, p, o);
        q += __shfl_xor_sync(0xffffffffu, q, o);
      }
      if (lane == 0) {
        mine[2 * i] += p;
        mine[2 * i + 1] += q;
      }
    }
  }
  __syncthreads();
  for (int i = tid; i < N; i += kThreads) {
    float p = 0.f, q = 0.f;
    for (int w = 0; w < kWarps; ++w) {
      p += acc[(static_cast<size_t>(w) * N + i) * 2];
      q += acc[(static_cast<size_t>(w) * N + i) * 2 + 1];
    }
    partials[static_cast<size_t>(blockIdx.x) * 2 * N + i] = p;
    partials[static_cast<size_t>(blockIdx.x) * 2 * N + N + i] = q;
  }
}

}  // namespace adacons
