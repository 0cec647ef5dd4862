// Device code of the AdaCons aggregation library (sm_100a only).
//
// Three steps per aggregation (Algorithm 1 of arXiv 2411.03742, run on one device):
//   pass1_*   stream the N x d matrix once: column sums s_k = sum_j g_jk, then per worker
//             N p_i = sum_k g_ik s_k and q_i = sum_k g_ik^2 (Eq. 7).  One partial per block.
//   coeff_*   fixed-order fp64 reduction of the partials, a_i = p_i/sqrt(q_i), sorted
//             momentum (Eq. 11), sum-to-one weights (Eq. 12-13).
//   pass2_*   stream the matrix again: out_k = cast(sum_i gamma_i g_ik) (Eq. 12).
//
// Everything is deterministic: fixed block->tile assignment, fixed per-thread order, fixed
// shuffle trees, fixed-order cross-block sums, no floating-point atomics.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace adacons {

constexpr int kThreads = 256;          // threads per block in both streaming passes
constexpr int kWarps = kThreads / 32;
constexpr int kBoxRowBytes = 512;      // one row of one TMA box: 32 lanes x 16 bytes
constexpr int kMaxFastN = 64;          // largest N served by the TMA-staged pass 1
constexpr int kMaxN = 1024;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;  // bounded mbarrier wait: 2 s

constexpr uint32_t kFlagZeroRow = 1u, kFlagDegenerateZ = 2u, kFlagNonfinite = 4u,
                   kFlagNegZ = 8u, kFlagTimeout = 0x100u;

template <int DT> struct Elem;                       // DT: 0 = fp32, 1 = bf16
template <> struct Elem<0> { static constexpr int kVec = 4, kBytes = 4; };
template <> struct Elem<1> { static constexpr int kVec = 8, kBytes = 2; };

// ----------------------------------------------------------------------------------------------
// small PTX helpers
// ----------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_addr(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_addr(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Wait for a phase of an mbarrier, but never for longer than kWaitLimitNs.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_timer_ns();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (global_timer_ns() - t0 > kWaitLimitNs) return false;
  }
}
// 2-D tiled TMA load global -> shared, completion reported on an mbarrier.
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, uint64_t* bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_addr(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_addr(bar)), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
// Programmatic dependent launch: a kernel launched with the stream-serialisation attribute may
// start before its predecessor in the stream has finished; it must call pdl_wait() before it
// touches anything the predecessor writes.  Without the attribute both are no-ops.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ uint4 ld_shared_v4(const void* p) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(smem_addr(p)));
  return v;
}
__device__ __forceinline__ uint4 ld_stream_v4(const void* p) {   // read-once global data
  uint4 v;
  asm("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// 32 bytes with one instruction (sm_100 has 256-bit global loads and stores); p must be 32-byte aligned
__device__ __forceinline__ void ld_stream_v8(const void* p, uint4& a, uint4& b) {
  asm("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
      : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w), "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w) : "l"(p));
}
__device__ __forceinline__ void st_global_v8(void* p, const uint4& a, const uint4& b, unsigned long long policy) {
  if (policy != 0ull)
    asm volatile("st.global.L2::cache_hint.v8.u32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8}, %9;"
                 ::"l"(p), "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w), "l"(policy) : "memory");
  else
    asm volatile("st.global.v8.u32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 ::"l"(p), "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w) : "memory");
}

// A 16-byte vector as VEC/2 pairs of fp32 values (bf16 -> fp32 is exact: a 16-bit shift).
template <int DT> __device__ __forceinline__ float2 unpack_pair(const uint4& v, int k);
template <> __device__ __forceinline__ float2 unpack_pair<0>(const uint4& v, int k) {
  return k == 0 ? make_float2(__uint_as_float(v.x), __uint_as_float(v.y))
                : make_float2(__uint_as_float(v.z), __uint_as_float(v.w));
}
template <> __device__ __forceinline__ float2 unpack_pair<1>(const uint4& v, int k) {
  const uint32_t u = k == 0 ? v.x : k == 1 ? v.y : k == 2 ? v.z : v.w;
  return make_float2(__uint_as_float(u << 16), __uint_as_float(u & 0xffff0000u));
}
__device__ __forceinline__ uint32_t pack_bf16x2_rn(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

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
  for (int j = 0; j < 2 * C::NR; ++j) outer[j * kThreads + threadIdx.x] = 0.f;
}
template <class C>
__device__ __forceinline__ void p1_fold(float2 (&pacc)[C::NR], float2 (&qacc)[C::NR], float* outer) {
#pragma unroll
  for (int j = 0; j < C::NR; ++j) {
    outer[j * kThreads + threadIdx.x] += pacc[j].x + pacc[j].y;
    outer[(C::NR + j) * kThreads + threadIdx.x] += qacc[j].x + qacc[j].y;
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

// ---- pass 1 for 64 < N <= 128 in one read, one block per tile: boxes of 128 rows x 256 bytes ------
// Twice the rows of pass1_tma_kernel's tallest tile at half the width, so a stage is still 32 KB.
// A HALF-warp owns a row: lane l of warp w belongs to row group g = 2 w + (l >> 4) and owns the
// 16-byte column group l & 15 of rows g, g + 16, ..., g + 112 (8 rows, as before; rows past N are
// zero-filled by TMA).  The 16 groups' partial column sums are exchanged through shared memory in
// two steps -- every thread first finishes one column of a quarter or half of the groups, in group
// order, then all read the sums of their own columns -- and the lane reduction at the end stays
// inside a half-warp.  Same partial-record layout as pass1_tma_kernel.
template <int DT>
struct P1H {
  static constexpr int NR = 8;
  static constexpr int VEC = Elem<DT>::kVec;
  static constexpr int NP = VEC / 2;
  static constexpr int kRows = 128, kGroups = 16;
  static constexpr int kBoxRowBytesH = 256;
  static constexpr int TILEC = kBoxRowBytesH / Elem<DT>::kBytes;   // 128 (bf16) / 64 (fp32) columns per tile
  static constexpr int PARTS = kThreads / TILEC;                   // threads per column in the first exchange step
  static constexpr int kGroupsPerPart = kGroups / PARTS;
  static constexpr uint32_t kStageBytes = kRows * kBoxRowBytesH;   // 32 KB
  static constexpr int kXchFloats = kGroups * TILEC;
  static constexpr int kSumFloats = PARTS * TILEC;                 // = kThreads
  static constexpr int kRedFloats = kGroups * NR * 2;
  static constexpr int kOuterFloats = 2 * NR * kThreads;
  static constexpr size_t kFixedBytes = (kXchFloats + kSumFloats + kRedFloats + kOuterFloats) * sizeof(float);
};

template <int DT>
__global__ void __launch_bounds__(kThreads, 2)
pass1_tall_kernel(const __grid_constant__ CUtensorMap tmap, const Pass1Params prm) {
  using C = P1H<DT>;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  __shared__ int s_abort;
  const int N = prm.N;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = 2 * warp + (lane >> 4), cl = lane & 15;
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
    for (int i = tid; i < 2 * N; i += kThreads) dst[i] = 0.f;
    return;
  }
  // block partial: both accumulation levels, lanes of a half-warp by a fixed xor tree; every row has one owner group
  p1_fold<C>(pacc, qacc, outer);
#pragma unroll
  for (int j = 0; j < C::NR; ++j) {
    float p = outer[j * kThreads + tid], q = outer[(C::NR + j) * kThreads + tid];
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) {
      p += __shfl_xor_sync(0xffffffffu, p, o);
      q += __shfl_xor_sync(0xffffffffu, q, o);
    }
    if (cl == 0) {
      red[(g * C::NR + j) * 2 + 0] = p;
      red[(g * C::NR + j) * 2 + 1] = q;
    }
  }
  __syncthreads();
  if (tid < N) {                                        // row tid = group tid % 16, its (tid / 16)-th row
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

// ----------------------------------------------------------------------------------------------
// Coefficient step: one block per coefficient set.  The partial records of the set are added in
// fp64 in a fixed order (threads split them into `groups` interleaved subsequences, which are
// then added in group order); afterwards thread i = worker i.
// ----------------------------------------------------------------------------------------------
struct CoeffParams {
  int N;
  int num_partials;      // global mode: records 0..num_partials-1 belong to the one set
  int sets;
  double beta;
  int momentum, sorted, normalize;
  const float* partials; // [records][2N]
  const int* rec_begin;  // per set (nullptr in global mode)
  const int* rec_count;
  const long long* seg_off; // per-segment mode: [sets + 1] column offsets (nullptr in global mode)
  double* coef;          // [5][sets][N]: a, a~, gamma, p, q   (enum adacons_coeff order)
  float* gamma_f32;      // [sets][N]   weights as pass 2 reads them
  double* m;             // [sets][N]   momentum state, in place
  double* z;             // [sets]      normaliser Z = sum_i u_i of the last call (NaN if not computed)
  uint32_t* flags;       // device status word (OR)
  long long* step;       // aggregation counter
};

// Work arrays in shared memory: sh_part holds part_cap doubles (at least 2N), sh_a, sh_u and sh_m N each.
// The records are split into `groups` interleaved subsequences, which fixes the order of the fp64
// sum; groups follows from N, part_cap and group_threads alone (not from the block size), so two
// kernels that pass the same values add the same records in the same order.
__device__ __forceinline__ void coeff_core(const CoeffParams& prm, const int set, double* sh_part, const int part_cap,
                                           const int group_threads, double* sh_a, double* sh_u, double* sh_m) {
  __shared__ int sh_bad, sh_zero;
  __shared__ double sh_Z;
  __shared__ int sh_uniform;
  const int N = prm.N, i = threadIdx.x, T = blockDim.x;
  const int V = 2 * N;
  const size_t per = static_cast<size_t>(prm.sets) * N;   // stride between coefficient kinds
  if (i == 0) { sh_bad = 0; sh_zero = 0; }
  if (i < N) sh_m[i] = prm.m[static_cast<size_t>(set) * N + i];   // the old state, fetched while the partials are summed
  const int begin = prm.rec_begin ? prm.rec_begin[set] : 0;
  const int count = prm.rec_count ? prm.rec_count[set] : prm.num_partials;
  const float* base = prm.partials + static_cast<size_t>(begin) * V;
  // A record is V = 2N floats, read as 16-byte (N even) or 8-byte vectors; `groups` interleaved
  // subsequences of the records are summed in parallel (at most 32, and groups * V <= part_cap).
  const int w = (V % 4 == 0) ? 4 : 2;
  const int units = V / w;
  int groups = group_threads / units;
  if (groups > 32) groups = 32;
  if (groups > part_cap / V) groups = part_cap / V;
  if (groups < 1) groups = 1;
  for (int slot = i; slot < units * groups; slot += T) {
    const int g = slot / units, u = slot - g * units;
    double acc[4] = {0.0, 0.0, 0.0, 0.0};
    const float* src = base + static_cast<size_t>(u) * w;
    if (w == 4) {
      // eight records in flight, added in record order (the latency of a round trip to L2 is what this step costs)
      int c = g;
      for (; c + 7 * groups < count; c += 8 * groups) {
        float4 x[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) x[j] = __ldcg(reinterpret_cast<const float4*>(src + static_cast<size_t>(c + j * groups) * V));
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          acc[0] += static_cast<double>(x[j].x); acc[1] += static_cast<double>(x[j].y);
          acc[2] += static_cast<double>(x[j].z); acc[3] += static_cast<double>(x[j].w);
        }
      }
      for (; c < count; c += groups) {
        const float4 x = __ldcg(reinterpret_cast<const float4*>(src + static_cast<size_t>(c) * V));
        acc[0] += static_cast<double>(x.x); acc[1] += static_cast<double>(x.y);
        acc[2] += static_cast<double>(x.z); acc[3] += static_cast<double>(x.w);
      }
    } else {
#pragma unroll 4
      for (int c = g; c < count; c += groups) {
        const float2 x = __ldcg(reinterpret_cast<const float2*>(src + static_cast<size_t>(c) * V));
        acc[0] += static_cast<double>(x.x); acc[1] += static_cast<double>(x.y);
      }
    }
    for (int e = 0; e < w; ++e) sh_part[g * V + u * w + e] = acc[e];
  }
  __syncthreads();
  double p = 0.0, q = 0.0;
  if (i < N) {
    double P = 0.0, Q = 0.0;
    for (int g = 0; g < groups; ++g) { P += sh_part[g * V + i]; Q += sh_part[g * V + N + i]; }
    p = P / static_cast<double>(N);   // gbar is the mean of the workers (text before Eq. 7)
    q = Q;
    if (!(isfinite(p) && isfinite(q))) atomicOr(&sh_bad, 1);
    if (q == 0.0) atomicOr(&sh_zero, 1);
    prm.coef[3 * per + set * N + i] = p;
    prm.coef[4 * per + set * N + i] = q;
  }
  __syncthreads();
  // A segment without columns is no layer: its all-zero statistics take the usual fallbacks
  // (weights 1/N, state unchanged at zero) but are no degeneracy of the data and raise no flag.
  const bool empty_set = prm.seg_off != nullptr && prm.seg_off[set + 1] == prm.seg_off[set];
  uint32_t flags = (sh_zero && !empty_set) ? kFlagZeroRow : 0u;
  const double uniform = 1.0 / static_cast<double>(N);
  if (sh_bad) {   // non-finite statistic: plain mean, momentum state left as it was
    if (i < N) {
      const double nan = __longlong_as_double(0x7ff8000000000000ll);
      prm.coef[0 * per + set * N + i] = nan;
      prm.coef[1 * per + set * N + i] = nan;
      prm.coef[2 * per + set * N + i] = uniform;
      prm.gamma_f32[set * N + i] = static_cast<float>(uniform);
    }
    if (i == 0) {
      atomicOr(prm.flags, flags | kFlagNonfinite);
      prm.z[set] = __longlong_as_double(0x7ff8000000000000ll);
      if (set == 0) atomicAdd(reinterpret_cast<unsigned long long*>(prm.step), 1ull);   // no round trip
    }
    return;
  }
  const double rq = q > 0.0 ? sqrt(q) : 0.0;
  const double a = q > 0.0 ? p / rq : 0.0;                       // Eq. 7
  if (i < N) sh_a[i] = a;
  __syncthreads();
  double at = a;
  if (i < N && prm.momentum) {
    int rank = i;
    if (prm.sorted) {                                            // stable ascending rank, Eq. 11
      rank = 0;
      for (int j = 0; j < N; ++j) {
        const double aj = sh_a[j];
        rank += (aj < a || (aj == a && j < i)) ? 1 : 0;
      }
    }
    // spelled out so that every kernel this is inlined into rounds the same way (one product, one fused step)
    at = __fma_rn(prm.beta, sh_m[rank], __dmul_rn(1.0 - prm.beta, a));
    prm.m[static_cast<size_t>(set) * N + rank] = at;              // exactly one writer per slot
  }
  const double u = q > 0.0 ? at / rq : 0.0;                      // unit-column P: weight on raw g_i
  if (i < N) sh_u[i] = u;
  __syncthreads();
  if (i == 0) {
    double Z = 0.0, A = 0.0;
    for (int j = 0; j < N; ++j) { Z += sh_u[j]; A += fabs(sh_u[j]); }
    sh_Z = Z;
    prm.z[set] = Z;
    sh_uniform = 0;
    if (prm.normalize) {
      if (!isfinite(Z) || fabs(Z) <= 1e-12 * A) { sh_uniform = 1; if (!empty_set) flags |= kFlagDegenerateZ; }
      else if (Z < 0.0) flags |= kFlagNegZ;
    }
    if (flags) atomicOr(prm.flags, flags);
    if (set == 0) atomicAdd(reinterpret_cast<unsigned long long*>(prm.step), 1ull);   // no round trip
  }
  __syncthreads();
  if (i < N) {
    double g;
    if (prm.normalize) g = sh_uniform ? uniform : u / sh_Z;      // Eq. 12-13
    else g = u * uniform;                                         // lambda = 1, 1/N of Eq. 8
    prm.coef[0 * per + set * N + i] = a;
    prm.coef[1 * per + set * N + i] = at;
    prm.coef[2 * per + set * N + i] = g;
    prm.gamma_f32[set * N + i] = static_cast<float>(g);
  }
}

__device__ __forceinline__ void coeff_body(const CoeffParams& prm, const int set) {
  __shared__ double sh_part[2 * kMaxN];
  __shared__ double sh_a[kMaxN];
  __shared__ double sh_u[kMaxN];
  __shared__ double sh_m[kMaxN];
  coeff_core(prm, set, sh_part, 2 * kMaxN, static_cast<int>(blockDim.x), sh_a, sh_u, sh_m);
}

__global__ void __launch_bounds__(kMaxN)
coeff_kernel(const CoeffParams prm) {
  pdl_launch_dependents();
  pdl_wait();                                              // pass 1 has finished and is visible
  coeff_body(prm, blockIdx.x);
}

// ----------------------------------------------------------------------------------------------
// Pass 2, vectorised (16-byte aligned rows).  Threads own 16-byte column groups (or pairs of
// them); blocks are numbered from the END of the vector, so the columns pass 1 read last are read
// first.  (That order is harmless but buys nothing measurable on B200: a pass 2 over 819 MB takes
// 0.119 ms whether the preceding sweep read the same matrix or another one, in either direction,
// and evict_last hints on the sweep's last 16-128 MB move it by under 3 %.)  Rows are added in
// index order with fp32 FMA.
// SEG = true: one weight set per segment.  blk_seg[2b] >= 0 names the single segment that holds
// all columns of block b; otherwise it is -(s+1), s = segment of the block's lowest column, and
// blk_seg[2b+1] is the segment of its highest column (see "blocks that span segment boundaries").
// ----------------------------------------------------------------------------------------------
// `policy` is an L2 eviction-priority descriptor (0 = none).  The 16-byte kernel writes its
// result with evict_last: the 680 MB-scale result is only 1/N of the traffic but, left to the
// default policy, its dirty lines leave L2 scattered among the reads and cost DRAM far more than
// their size (pass 2 without stores: 5.81 ms; with: 6.40 ms; with evict_last: 6.27 ms on bert64).
// The 32-byte kernel chooses per launch (see pass2_wide_kernel).
__device__ __forceinline__ unsigned long long l2_policy_evict_last() {
  unsigned long long pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
template <int DT, int NP>
__device__ __forceinline__ uint4 pass2_pack(const float2 (&acc)[NP]) {   // one RNE rounding to the storage type
  if constexpr (DT == 0)
    return make_uint4(__float_as_uint(acc[0].x), __float_as_uint(acc[0].y), __float_as_uint(acc[1].x),
                      __float_as_uint(acc[1].y));
  else
    return make_uint4(pack_bf16x2_rn(acc[0].x, acc[0].y), pack_bf16x2_rn(acc[1].x, acc[1].y),
                      pack_bf16x2_rn(acc[NP - 2].x, acc[NP - 2].y), pack_bf16x2_rn(acc[NP - 1].x, acc[NP - 1].y));
}
template <int DT, int NP>
__device__ __forceinline__ void pass2_store(unsigned char* out, long long v, const float2 (&acc)[NP],
                                            unsigned long long policy = 0ull) {
  const uint4 o = pass2_pack<DT, NP>(acc);
  if (policy != 0ull)
    asm volatile("st.global.L2::cache_hint.v4.u32 [%0], {%1,%2,%3,%4}, %5;"
                 ::"l"(out + v * 16), "r"(o.x), "r"(o.y), "r"(o.z), "r"(o.w), "l"(policy) : "memory");
  else
    *reinterpret_cast<uint4*>(out + v * 16) = o;
}

// Block -> column mapping shared by both vectorised pass-2 kernels (and by the host's per-block
// segment plan): the row's 16-byte groups are paired (group 2w with 2w+1; with an odd count the last
// pair has one member) and block b owns the kPass2BlockPairs pairs below num_pairs - b * kPass2BlockPairs,
// i.e. groups [2 * (num_pairs - (b+1) * 256), 2 * (num_pairs - b * 256)) clipped to [0, num_vec).
constexpr int kPass2BlockPairs = kThreads;
constexpr int kPass2BlockVecs = 2 * kPass2BlockPairs;   // 16-byte groups per block: 8 KB of every row
constexpr int kPass2Rows = 8;      // narrow kernel: rows per batch, 2 * kPass2Rows 16-byte loads in flight per thread
constexpr int kPass2WideRows = 4;  // wide kernel: rows per batch, kPass2WideRows 32-byte loads in flight per thread

// The last 16-byte group of a row holds only `tail_elems` real columns when d is not a multiple of
// the vector width (rows padded to a 16-byte pitch): store those element by element.
template <int DT, int NP>
__device__ __forceinline__ void pass2_store_tail(unsigned char* out, long long v, const float2 (&acc)[NP], int tail_elems) {
  constexpr int VEC = Elem<DT>::kVec;
#pragma unroll
  for (int e = 0; e < VEC; ++e) {
    if (e >= tail_elems) break;
    const float x = (e & 1) ? acc[e / 2].y : acc[e / 2].x;
    if constexpr (DT == 0) reinterpret_cast<float*>(out)[v * VEC + e] = x;
    else reinterpret_cast<unsigned short*>(out)[v * VEC + e] = static_cast<unsigned short>(pack_bf16x2_rn(x, 0.f) & 0xffffu);
  }
}
template <int DT, int NP>
__device__ __forceinline__ void pass2_store_any(unsigned char* out, long long v, const float2 (&acc)[NP],
                                                long long num_vec, int tail_elems, unsigned long long policy = 0ull) {
  if (tail_elems != 0 && v == num_vec - 1) pass2_store_tail<DT, NP>(out, v, acc, tail_elems);
  else pass2_store<DT, NP>(out, v, acc, policy);
}

// One 16-byte group with a single weight set taken from shared memory, rows one at a time.
template <int DT>
__device__ __forceinline__ void pass2_single_vector(const unsigned char* __restrict__ grads, unsigned char* __restrict__ out,
                                                    const float* g_s, int N, long long row_bytes, long long v,
                                                    long long num_vec, int tail_elems, unsigned long long policy) {
  constexpr int NP = Elem<DT>::kVec / 2;
  float2 a1[NP];
#pragma unroll
  for (int h = 0; h < NP; ++h) a1[h] = make_float2(0.f, 0.f);
  for (int i = 0; i < N; ++i) {
    const uint4 x = ld_stream_v4(grads + v * 16 + static_cast<long long>(i) * row_bytes);
    const float2 g2 = make_float2(g_s[i], g_s[i]);
#pragma unroll
    for (int h = 0; h < NP; ++h) a1[h] = __ffma2_rn(unpack_pair<DT>(x, h), g2, a1[h]);
  }
  pass2_store_any<DT, NP>(out, v, a1, num_vec, tail_elems, policy);
}

// One 16-byte group of a block that spans a segment boundary: every column finds its own segment
// (sg0 = segment of the block's lowest column; segments ascend, empty ones are skipped).
template <int DT>
__device__ __forceinline__ void pass2_mixed_vector(const unsigned char* __restrict__ grads, unsigned char* __restrict__ out,
                                                   const float* __restrict__ gamma, int N, long long row_bytes, long long v,
                                                   long long num_vec, int tail_elems, const long long* __restrict__ seg_off,
                                                   int sg0, unsigned long long policy) {
  constexpr int VEC = Elem<DT>::kVec;
  constexpr int NP = VEC / 2;
  int sg = sg0;
  int seg_of[VEC];
  const long long d_cols = (num_vec - 1) * VEC + (tail_elems ? tail_elems : VEC);
#pragma unroll
  for (int e = 0; e < VEC; ++e) {
    const long long c = v * VEC + e;
    if (c < d_cols)
      while (c >= seg_off[sg + 1]) ++sg;
    seg_of[e] = sg;                              // padding columns: any set, never stored
  }
  const unsigned char* col = grads + v * 16;
  float2 acc[NP];
#pragma unroll
  for (int h = 0; h < NP; ++h) acc[h] = make_float2(0.f, 0.f);
  for (int i = 0; i < N; ++i) {
    const uint4 x = ld_stream_v4(col + static_cast<long long>(i) * row_bytes);
#pragma unroll
    for (int h = 0; h < NP; ++h) {
      const float2 xv = unpack_pair<DT>(x, h);
      const float2 g2 = make_float2(gamma[static_cast<size_t>(seg_of[2 * h]) * N + i],
                                    gamma[static_cast<size_t>(seg_of[2 * h + 1]) * N + i]);
      acc[h] = __ffma2_rn(xv, g2, acc[h]);
    }
  }
  pass2_store_any<DT, NP>(out, v, acc, num_vec, tail_elems, policy);
}

// ---- blocks that span segment boundaries (SEG kernels) -------------------------------------------
// Such a block keeps the weights of ALL segments it touches in shared memory ([nseg][N], at most
// kSegSmemFloats floats and kSegSmemSegs segments) next to their column offsets.  A thread whose
// columns lie in one segment -- all but the few that straddle a boundary -- runs the ordinary
// vector loop with that segment's row of weights; a straddling thread looks the weight of each of
// its columns up in shared memory.  Blocks that touch more segments than fit fall back to
// pass2_mixed_vector (weights from global memory).
constexpr int kSegSmemFloats = 4096;
constexpr int kSegSmemSegs = 128;

// index (relative to the block's first segment) of the segment that holds column c
__device__ __forceinline__ int seg_find(const long long* off_s, int nseg, long long c) {
  int lo = 0, hi = nseg - 1;
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (off_s[mid + 1] > c) hi = mid; else lo = mid + 1;
  }
  return lo;
}

template <int DT>
__device__ __noinline__ void pass2_mixed_vector_smem(   // rare (threads that straddle a boundary): kept out of the vector loop's registers
    const unsigned char* __restrict__ grads, unsigned char* __restrict__ out,
                                                        const float* g_seg, const long long* off_s, int nseg, int N,
                                                        long long row_bytes, long long v, long long num_vec, int tail_elems,
                                                        unsigned long long policy) {
  constexpr int VEC = Elem<DT>::kVec;
  constexpr int NP = VEC / 2;
  const long long d_cols = (num_vec - 1) * VEC + (tail_elems ? tail_elems : VEC);
  int sg = seg_find(off_s, nseg, v * VEC);
  int seg_of[VEC];
#pragma unroll
  for (int e = 0; e < VEC; ++e) {
    const long long c = v * VEC + e;
    if (c < d_cols)
      while (c >= off_s[sg + 1]) ++sg;
    seg_of[e] = sg * N;                          // padding columns: any set, never stored
  }
  const unsigned char* col = grads + v * 16;
  float2 acc[NP];
#pragma unroll
  for (int h = 0; h < NP; ++h) acc[h] = make_float2(0.f, 0.f);
  constexpr int U = 4;                           // rows in flight: this thread's block waits for it
  int i0 = 0;
  for (; i0 + U <= N; i0 += U) {
    uint4 x[U];
#pragma unroll
    for (int u = 0; u < U; ++u) x[u] = ld_stream_v4(col + static_cast<long long>(i0 + u) * row_bytes);
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int h = 0; h < NP; ++h)
        acc[h] = __ffma2_rn(unpack_pair<DT>(x[u], h),
                            make_float2(g_seg[seg_of[2 * h] + i0 + u], g_seg[seg_of[2 * h + 1] + i0 + u]), acc[h]);
  }
  for (; i0 < N; ++i0) {
    const uint4 x = ld_stream_v4(col + static_cast<long long>(i0) * row_bytes);
#pragma unroll
    for (int h = 0; h < NP; ++h)
      acc[h] = __ffma2_rn(unpack_pair<DT>(x, h), make_float2(g_seg[seg_of[2 * h] + i0], g_seg[seg_of[2 * h + 1] + i0]), acc[h]);
  }
  pass2_store_any<DT, NP>(out, v, acc, num_vec, tail_elems, policy);
}

// The same for a complete 32-byte pair (groups 2w and 2w + 1): one 256-bit load per row, four rows in
// flight, so that a straddling thread needs no more round trips to memory than its neighbours and
// does not keep its block waiting.
template <int DT>
__device__ __noinline__ void pass2_mixed_pair_smem(const unsigned char* __restrict__ grads, unsigned char* __restrict__ out,
                                                   const float* g_seg, const long long* off_s, int nseg, int N,
                                                   long long row_bytes, long long w, long long num_vec, int tail_elems,
                                                   unsigned long long policy) {
  constexpr int VEC = Elem<DT>::kVec;
  constexpr int NP = VEC / 2;
  const long long v0 = 2 * w;
  const long long d_cols = (num_vec - 1) * VEC + (tail_elems ? tail_elems : VEC);
  int sg = seg_find(off_s, nseg, v0 * VEC);
  int seg_of[2 * VEC];
#pragma unroll
  for (int e = 0; e < 2 * VEC; ++e) {
    const long long c = v0 * VEC + e;
    if (c < d_cols)
      while (c >= off_s[sg + 1]) ++sg;
    seg_of[e] = sg * N;
  }
  const unsigned char* col = grads + w * 32;
  float2 acc[2][NP];
#pragma unroll
  for (int g = 0; g < 2; ++g)
#pragma unroll
    for (int h = 0; h < NP; ++h) acc[g][h] = make_float2(0.f, 0.f);
  constexpr int U = 4;
  int i0 = 0;
  for (; i0 + U <= N; i0 += U) {
    uint4 x[U][2];
#pragma unroll
    for (int u = 0; u < U; ++u) ld_stream_v8(col + static_cast<long long>(i0 + u) * row_bytes, x[u][0], x[u][1]);
#pragma unroll
    for (int u = 0; u < U; ++u)
#pragma unroll
      for (int g = 0; g < 2; ++g)
#pragma unroll
        for (int h = 0; h < NP; ++h)
          acc[g][h] = __ffma2_rn(unpack_pair<DT>(x[u][g], h),
                                 make_float2(g_seg[seg_of[g * VEC + 2 * h] + i0 + u], g_seg[seg_of[g * VEC + 2 * h + 1] + i0 + u]),
                                 acc[g][h]);
  }
  for (; i0 < N; ++i0) {
    uint4 x[2];
    ld_stream_v8(col + static_cast<long long>(i0) * row_bytes, x[0], x[1]);
#pragma unroll
    for (int g = 0; g < 2; ++g)
#pragma unroll
      for (int h = 0; h < NP; ++h)
        acc[g][h] = __ffma2_rn(unpack_pair<DT>(x[g], h),
                               make_float2(g_seg[seg_of[g * VEC + 2 * h] + i0], g_seg[seg_of[g * VEC + 2 * h + 1] + i0]), acc[g][h]);
  }
  pass2_store_any<DT, NP>(out, v0, acc[0], num_vec, tail_elems, policy);
  pass2_store_any<DT, NP>(out, v0 + 1, acc[1], num_vec, tail_elems, policy);
}

// Loads the weights and offsets of segments sg0..sg1 into shared memory; false if they do not fit.
__device__ __forceinline__ bool seg_block_setup(float* g_seg, long long* off_s, const float* __restrict__ gamma,
                                                const long long* __restrict__ seg_off, int sg0, int sg1, int N) {
  const int nseg = sg1 - sg0 + 1;
  if (nseg > kSegSmemSegs || nseg * N > kSegSmemFloats) return false;
  for (int idx = threadIdx.x; idx < nseg * N; idx += kThreads) g_seg[idx] = gamma[static_cast<size_t>(sg0) * N + idx];
  for (int j = threadIdx.x; j <= nseg; j += kThreads) off_s[j] = seg_off[sg0 + j];
  return true;
}

// Narrow kernel (buffers 16-byte but not 32-byte aligned): thread t of block b owns the groups
// lo + t and lo + 256 + t of the block's range, one 16-byte load each.
template <int DT, bool SEG, int U = kPass2Rows>
__global__ void __launch_bounds__(kThreads)
pass2_vec_kernel(const unsigned char* __restrict__ grads, unsigned char* __restrict__ out,
                 const float* __restrict__ gamma, int N, long long row_bytes, long long num_vec,
                 const int* __restrict__ blk_seg, const long long* __restrict__ seg_off, int tail_elems) {
  constexpr int VEC = Elem<DT>::kVec;
  constexpr int NP = VEC / 2;
  constexpr int CG = 2;
  __shared__ float g_s[SEG ? kSegSmemFloats : kMaxN];
  __shared__ long long off_s[SEG ? kSegSmemSegs + 1 : 1];
  const unsigned long long keep = l2_policy_evict_last();
  pdl_wait();                                        // the coefficient step has finished
  int code = 0;
  if (SEG) code = blk_seg[2 * blockIdx.x];
  const long long num_pairs = (num_vec + 1) / 2;
  const long long base = 2 * (num_pairs - (static_cast<long long>(blockIdx.x) + 1) * kPass2BlockPairs) + threadIdx.x;
  if (!SEG || code >= 0) {
    const float* gsrc = gamma + static_cast<size_t>(SEG ? code : 0) * N;
    for (int i = threadIdx.x; i < N; i += kThreads) g_s[i] = gsrc[i];
    __syncthreads();
    if (base >= 0 && base + (CG - 1) * kThreads < num_vec) {   // both groups exist (all but the edge blocks)
      float2 acc[CG][NP];
#pragma unroll
      for (int g = 0; g < CG; ++g)
#pragma unroll
        for (int h = 0; h < NP; ++h) acc[g][h] = make_float2(0.f, 0.f);
      const unsigned char* col = grads + base * 16;
      int i0 = 0;
      for (; i0 + U <= N; i0 += U) {
        uint4 x[U][CG];
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
          for (int g = 0; g < CG; ++g)
            x[u][g] = ld_stream_v4(col + static_cast<long long>(i0 + u) * row_bytes + g * (kThreads * 16));
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const float gm = g_s[i0 + u];
          const float2 g2 = make_float2(gm, gm);
#pragma unroll
          for (int g = 0; g < CG; ++g)
#pragma unroll
            for (int h = 0; h < NP; ++h) acc[g][h] = __ffma2_rn(unpack_pair<DT>(x[u][g], h), g2, acc[g][h]);
        }
      }
      for (; i0 < N; ++i0) {
        const float gm = g_s[i0];
        const float2 g2 = make_float2(gm, gm);
#pragma unroll
        for (int g = 0; g < CG; ++g) {
          const uint4 x = ld_stream_v4(col + static_cast<long long>(i0) * row_bytes + g * (kThreads * 16));
#pragma unroll
          for (int h = 0; h < NP; ++h) acc[g][h] = __ffma2_rn(unpack_pair<DT>(x, h), g2, acc[g][h]);
        }
      }
#pragma unroll
      for (int g = 0; g < CG; ++g) pass2_store_any<DT, NP>(out, base + g * kThreads, acc[g], num_vec, tail_elems, keep);
    } else {
      for (int g = 0; g < CG; ++g) {
        const long long v = base + g * kThreads;
        if (v >= 0 && v < num_vec) pass2_single_vector<DT>(grads, out, g_s, N, row_bytes, v, num_vec, tail_elems, keep);
      }
    }
  } else if (SEG) {
    // the block spans segment boundaries: weights of all its segments in shared memory if they fit
    const int sg0 = -code - 1, sg1 = blk_seg[2 * blockIdx.x + 1];
    const bool fits = seg_block_setup(g_s, off_s, gamma, seg_off, sg0, sg1, N);   // block-uniform
    __syncthreads();
    const long long d_cols = (num_vec - 1) * VEC + (tail_elems ? tail_elems : VEC);
    for (int g = 0; g < CG; ++g) {
      const long long v = base + g * kThreads;
      if (v < 0 || v >= num_vec) continue;
      if (!fits) {
        pass2_mixed_vector<DT>(grads, out, gamma, N, row_bytes, v, num_vec, tail_elems, seg_off, sg0, keep);
        continue;
      }
      const int nseg = sg1 - sg0 + 1;
      const int sl = seg_find(off_s, nseg, v * VEC);
      const long long c_last = (v * VEC + VEC < d_cols ? v * VEC + VEC : d_cols) - 1;
      if (c_last < off_s[sl + 1])                      // the whole group lies in one segment
        pass2_single_vector<DT>(grads, out, g_s + sl * N, N, row_bytes, v, num_vec, tail_elems, keep);
      else
        pass2_mixed_vector_smem<DT>(grads, out, g_s, off_s, nseg, N, row_bytes, v, num_vec, tail_elems, keep);
    }
  }
}

// 32 contiguous bytes (two 16-byte column groups) of every row, weights from shared memory: one
// 256-bit streaming load per row, U rows in flight, rows added in index order.
template <int DT, int U>
__device__ __forceinline__ void pass2_wide_pair(const unsigned char* __restrict__ col, const float* g_s, int N,
                                                long long row_bytes, float2 (&acc)[2][Elem<DT>::kVec / 2]) {
  constexpr int NP = Elem<DT>::kVec / 2;
#pragma unroll
  for (int g = 0; g < 2; ++g)
#pragma unroll
    for (int h = 0; h < NP; ++h) acc[g][h] = make_float2(0.f, 0.f);
  int i0 = 0;
  for (; i0 + U <= N; i0 += U) {
    uint4 x[U][2];
#pragma unroll
    for (int u = 0; u < U; ++u) ld_stream_v8(col + static_cast<long long>(i0 + u) * row_bytes, x[u][0], x[u][1]);
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const float gm = g_s[i0 + u];
      const float2 g2 = make_float2(gm, gm);
#pragma unroll
      for (int g = 0; g < 2; ++g)
#pragma unroll
        for (int h = 0; h < NP; ++h) acc[g][h] = __ffma2_rn(unpack_pair<DT>(x[u][g], h), g2, acc[g][h]);
    }
  }
  for (; i0 < N; ++i0) {
    uint4 x[2];
    ld_stream_v8(col + static_cast<long long>(i0) * row_bytes, x[0], x[1]);
    const float gm = g_s[i0];
    const float2 g2 = make_float2(gm, gm);
#pragma unroll
    for (int g = 0; g < 2; ++g)
#pragma unroll
      for (int h = 0; h < NP; ++h) acc[g][h] = __ffma2_rn(unpack_pair<DT>(x[g], h), g2, acc[g][h]);
  }
}

// The same sum for a thread of a block that spans segment boundaries: its first `split` elements
// take the weights `ga` (one segment), the rest `gb` (the next one); split = 2 VEC when the whole
// pair lies in one segment.  Every thread of such a block runs this loop, so a warp with a
// straddling thread does not execute two different loops one after the other.
template <int DT, int U>
__device__ __forceinline__ void pass2_wide_pair_two(const unsigned char* __restrict__ col, const float* ga, const float* gb,
                                                    int split, int N, long long row_bytes,
                                                    float2 (&acc)[2][Elem<DT>::kVec / 2]) {
  constexpr int VEC = Elem<DT>::kVec;
  constexpr int NP = VEC / 2;
#pragma unroll
  for (int g = 0; g < 2; ++g)
#pragma unroll
    for (int h = 0; h < NP; ++h) acc[g][h] = make_float2(0.f, 0.f);
  int i0 = 0;
  for (; i0 + U <= N; i0 += U) {
    uint4 x[U][2];
#pragma unroll
    for (int u = 0; u < U; ++u) ld_stream_v8(col + static_cast<long long>(i0 + u) * row_bytes, x[u][0], x[u][1]);
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const float a = ga[i0 + u], b = gb[i0 + u];
#pragma unroll
      for (int g = 0; g < 2; ++g)
#pragma unroll
        for (int h = 0; h < NP; ++h) {
          const int e = g * VEC + 2 * h;
          acc[g][h] = __ffma2_rn(unpack_pair<DT>(x[u][g], h), make_float2(e < split ? a : b, e + 1 < split ? a : b), acc[g][h]);
        }
    }
  }
  for (; i0 < N; ++i0) {
    uint4 x[2];
    ld_stream_v8(col + static_cast<long long>(i0) * row_bytes, x[0], x[1]);
    const float a = ga[i0], b = gb[i0];
#pragma unroll
    for (int g = 0; g < 2; ++g)
#pragma unroll
      for (int h = 0; h < NP; ++h) {
        const int e = g * VEC + 2 * h;
        acc[g][h] = __ffma2_rn(unpack_pair<DT>(x[g], h), make_float2(e < split ? a : b, e + 1 < split ? a : b), acc[g][h]);
      }
  }
}

// Wide kernel (grads, out and the row pitch 32-byte aligned): thread t of block b owns pair
// w = num_pairs - (b+1) * 256 + t, i.e. 32 contiguous bytes of every row, fetched with one 256-bit
// load per row (U rows in flight) and written with one 256-bit store.  The loads are no faster
// than 16-byte ones (a read-only sweep runs at the same 7.5-7.7 TB/s either way), but the result
// costs less: a warp stores 1 KB contiguous per instruction and the whole pass takes 2.3 % less
// (6.19 -> 6.05 ms on 43.5 GB, same GPU, same run).  With the wide store the L2 evict_last hint no
// longer pays for a result larger than L2 (6.07 with, 6.05 without, and the next pass 1 is slower
// with it), so such a result is written with plain stores.  A result that fits in L2
// (keep_in_l2 != 0) is still written evict_last: it then stays in L2, where the next call
// overwrites it and its consumer finds it, and never costs DRAM bandwidth at all.
template <int DT, bool SEG, int U = kPass2WideRows>
__global__ void __launch_bounds__(kThreads, 4)     // four blocks per SM: the rare per-column path may spill, the vector loop does not
pass2_wide_kernel(const unsigned char* __restrict__ grads, unsigned char* __restrict__ out,
                  const float* __restrict__ gamma, int N, long long row_bytes, long long num_vec,
                  const int* __restrict__ blk_seg, const long long* __restrict__ seg_off, int tail_elems, int keep_in_l2) {
  constexpr int VEC = Elem<DT>::kVec;
  constexpr int NP = VEC / 2;
  __shared__ float g_s[SEG ? kSegSmemFloats : kMaxN];
  __shared__ long long off_s[SEG ? kSegSmemSegs + 1 : 1];
  const unsigned long long keep = keep_in_l2 ? l2_policy_evict_last() : 0ull;
  pdl_wait();                                        // the coefficient step has finished
  int code = 0;
  if (SEG) code = blk_seg[2 * blockIdx.x];
  const long long num_pairs = (num_vec + 1) / 2;
  const long long w = num_pairs - (static_cast<long long>(blockIdx.x) + 1) * kPass2BlockPairs + threadIdx.x;
  const long long v0 = 2 * w;
  const float* gw = g_s;                             // this thread's row of weights
  const float* gw2 = g_s;                            // ... and that of the next segment, if its 32 bytes hold a boundary
  int split = 2 * VEC;                               // elements of the pair that belong to the first of the two
  bool mixed_block = false;
  bool many = false;                                 // its 32 bytes hold more than one boundary
  int nseg = 1;
  if (!SEG || code >= 0) {
    const float* gsrc = gamma + static_cast<size_t>(SEG ? code : 0) * N;
    for (int i = threadIdx.x; i < N; i += kThreads) g_s[i] = gsrc[i];
    __syncthreads();
    if (w < 0) return;
  } else {
    // the block spans segment boundaries: weights of all its segments in shared memory if they fit
    const int sg0 = -code - 1, sg1 = blk_seg[2 * blockIdx.x + 1];
    const bool fits = seg_block_setup(g_s, off_s, gamma, seg_off, sg0, sg1, N);   // block-uniform
    __syncthreads();
    if (!fits) {
      // too many tiny segments for shared memory: single 16-byte groups, weights from global memory;
      // thread t takes groups lo + t and lo + 256 + t so that a warp's loads stay contiguous
      const long long lo = 2 * (num_pairs - (static_cast<long long>(blockIdx.x) + 1) * kPass2BlockPairs);
      for (int g = 0; g < 2; ++g) {
        const long long v = lo + threadIdx.x + g * kThreads;
        if (v >= 0 && v < num_vec)
          pass2_mixed_vector<DT>(grads, out, gamma, N, row_bytes, v, num_vec, tail_elems, seg_off, sg0, keep);
      }
      return;
    }
    if (w < 0) return;
    mixed_block = true;
    nseg = sg1 - sg0 + 1;
    const long long d_cols = (num_vec - 1) * VEC + (tail_elems ? tail_elems : VEC);
    const int sl = seg_find(off_s, nseg, v0 * VEC);
    const long long c_last = (v0 * VEC + 2 * VEC < d_cols ? v0 * VEC + 2 * VEC : d_cols) - 1;
    gw = gw2 = g_s + sl * N;
    if (c_last >= off_s[sl + 1]) {                   // a boundary inside the pair: the next non-empty segment takes over
      split = static_cast<int>(off_s[sl + 1] - v0 * VEC);
      int s2 = sl + 1;
      while (off_s[s2 + 1] <= off_s[sl + 1]) ++s2;   // ends: the block's last segment holds c_last
      gw2 = g_s + s2 * N;
      many = c_last >= off_s[s2 + 1];
    }
  }
  if (SEG && many) {                                 // rare: segments of a few columns
    if (v0 + 1 < num_vec) pass2_mixed_pair_smem<DT>(grads, out, g_s, off_s, nseg, N, row_bytes, w, num_vec, tail_elems, keep);
    else pass2_mixed_vector_smem<DT>(grads, out, g_s, off_s, nseg, N, row_bytes, v0, num_vec, tail_elems, keep);
    return;
  }
  if (SEG && mixed_block && v0 + 1 >= num_vec && split < 2 * VEC) {   // an odd row's last group with a boundary inside
    pass2_mixed_vector_smem<DT>(grads, out, g_s, off_s, nseg, N, row_bytes, v0, num_vec, tail_elems, keep);
    return;
  }
  if (v0 + 1 < num_vec) {                            // the pair is complete (all but an odd row's last group)
    float2 acc[2][NP];
    if (SEG && mixed_block) pass2_wide_pair_two<DT, U>(grads + w * 32, gw, gw2, split, N, row_bytes, acc);
    else pass2_wide_pair<DT, U>(grads + w * 32, gw, N, row_bytes, acc);
    if (tail_elems != 0 && v0 + 1 == num_vec - 1) {            // the row's last group is partial
      pass2_store<DT, NP>(out, v0, acc[0], keep);
      pass2_store_tail<DT, NP>(out, v0 + 1, acc[1], tail_elems);
    } else {
      st_global_v8(out + w * 32, pass2_pack<DT, NP>(acc[0]), pass2_pack<DT, NP>(acc[1]), keep);
    }
  } else {
    pass2_single_vector<DT>(grads, out, gw, N, row_bytes, v0, num_vec, tail_elems, keep);
  }
}

// Pass 2, generic: one thread per column, scalar loads.
template <int DT>
__global__ void __launch_bounds__(kThreads)
pass2_generic_kernel(const void* __restrict__ grads, void* __restrict__ out, const float* __restrict__ gamma,
                     int N, long long d, long long pitch) {
  __shared__ float g_s[kMaxN];
  pdl_wait();
  for (int i = threadIdx.x; i < N; i += kThreads) g_s[i] = gamma[i];
  __syncthreads();
  const long long k = static_cast<long long>(blockIdx.x) * kThreads + threadIdx.x;
  if (k >= d) return;
  float acc = 0.f;
  for (int i = 0; i < N; ++i) acc = fmaf(load_elem<DT>(grads, static_cast<long long>(i) * pitch + k), g_s[i], acc);
  if constexpr (DT == 0) reinterpret_cast<float*>(out)[k] = acc;
  else reinterpret_cast<unsigned short*>(out)[k] = static_cast<unsigned short>(pack_bf16x2_rn(acc, 0.f) & 0xffffu);
}

// ----------------------------------------------------------------------------------------------
// Edges of a matrix whose rows start off a 16-byte boundary (every row by the same amount: the row
// pitch is a multiple of 16 bytes).  The vectorised kernels then run on the aligned body -- from
// each row's first 16-byte boundary on -- and these two one-block kernels do the few columns left:
// edge_stats_kernel adds the first `head` (< 8) columns' share of Eq. 7 as one more partial record,
// edge_combine_kernel forms Eq. 12 for the head columns and for the last `tail` (< 8) columns that
// do not fill a 16-byte group (element-wise, so nothing is read or written past the vector).
// ----------------------------------------------------------------------------------------------
template <int DT>
__global__ void __launch_bounds__(kThreads)
edge_stats_kernel(const void* __restrict__ grads, int N, long long pitch, int head, float* __restrict__ record) {
  __shared__ float x[kMaxFastN * 8];
  __shared__ float s[8];
  const int tid = threadIdx.x;
  for (int idx = tid; idx < N * head; idx += kThreads) {
    const int i = idx / head, k = idx - i * head;
    x[i * 8 + k] = load_elem<DT>(grads, static_cast<long long>(i) * pitch + k);
  }
  __syncthreads();
  if (tid < head) {
    float a = 0.f;
    for (int i = 0; i < N; ++i) a += x[i * 8 + tid];
    s[tid] = a;
  }
  __syncthreads();
  if (tid < N) {
    float pp = 0.f, qq = 0.f;
    for (int k = 0; k < head; ++k) {
      const float v = x[tid * 8 + k];
      pp = fmaf(v, s[k], pp);
      qq = fmaf(v, v, qq);
    }
    record[tid] = pp;
    record[N + tid] = qq;
  }
}

template <int DT>
__global__ void __launch_bounds__(32)
edge_combine_kernel(const void* __restrict__ grads, void* __restrict__ out, const float* __restrict__ gamma, int N,
                    long long d, long long pitch, int head, int tail) {
  __shared__ float g_s[kMaxFastN];
  for (int i = threadIdx.x; i < N; i += 32) g_s[i] = gamma[i];
  __syncthreads();
  const int k = threadIdx.x;
  if (k >= head + tail) return;
  const long long col = k < head ? k : d - tail + (k - head);
  float acc = 0.f;
  for (int i = 0; i < N; ++i) acc = fmaf(load_elem<DT>(grads, static_cast<long long>(i) * pitch + col), g_s[i], acc);
  if constexpr (DT == 0) reinterpret_cast<float*>(out)[col] = acc;
  else reinterpret_cast<unsigned short*>(out)[col] = static_cast<unsigned short>(pack_bf16x2_rn(acc, 0.f) & 0xffffu);
}

// ----------------------------------------------------------------------------------------------
// Single-pass path for problems that fit in the grid's shared memory (N*d*sizeof(element) up to
// about 148 x 160 KB): ONE cooperative kernel reads the matrix from HBM once.  Block b keeps all N
// rows of its column slice in shared memory, computes its partial statistics (Eq. 7), meets the
// other blocks at a grid barrier, block 0 runs the coefficient step (Eq. 11, Eq. 12-13), a second
// grid barrier, and every block forms its slice of sum_i gamma_i g_i (Eq. 12) from shared memory.
// The barriers are counters in global memory; the launch is cooperative, so all blocks are
// resident, and every wait is bounded (2 s), after which the block raises the time-out flag and
// leaves.
// ----------------------------------------------------------------------------------------------
constexpr int kFusedThreads = 1024;

struct FusedParams {
  int N;
  long long num_vec;            // 16-byte column groups per row (the last may be partial)
  int tail_elems;               // real columns in the last group (0 = all)
  long long row_bytes;
  int vec_per_block;            // column groups owned by one block (shared-memory row pitch)
  const unsigned char* grads;
  unsigned char* out;
  unsigned long long* barrier;  // monotonically increasing arrival counter
  CoeffParams coeff;            // partials [gridDim.x][2N], sets = 1
};

__device__ __forceinline__ bool grid_barrier_bounded(unsigned long long* counter, unsigned int G, uint32_t* flags) {
  __shared__ int s_ok;
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned long long old = atomicAdd(counter, 1ull);
    const unsigned long long target = (old / G + 1ull) * G;
    const unsigned long long t0 = global_timer_ns();
    int ok = 1;
    for (;;) {
      unsigned long long cur;
      asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(cur) : "l"(counter) : "memory");
      if (cur >= target) break;
      if (global_timer_ns() - t0 > kWaitLimitNs) { ok = 0; atomicOr(flags, kFlagTimeout); break; }
    }
    __threadfence();
    s_ok = ok;
  }
  __syncthreads();
  return s_ok != 0;
}

template <int DT>
__global__ void __launch_bounds__(kFusedThreads, 1)
fused_small_kernel(const FusedParams prm) {
  constexpr int VEC = Elem<DT>::kVec;
  constexpr int NP = VEC / 2;
  constexpr int kW = kFusedThreads / 32;
  extern __shared__ __align__(16) unsigned char fs_raw[];
  const int N = prm.N, vpb = prm.vec_per_block;
  uint4* tile = reinterpret_cast<uint4*>(fs_raw);                                   // [N][vpb]
  float* acc = reinterpret_cast<float*>(fs_raw + static_cast<size_t>(N) * vpb * 16); // [kW][N][2]
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long vb0 = static_cast<long long>(blockIdx.x) * vpb;
  long long rem = prm.num_vec - vb0;
  const int nv = rem <= 0 ? 0 : (rem < vpb ? static_cast<int>(rem) : vpb);

  // ---- the only read of the matrix from HBM
  for (int idx = tid; idx < N * nv; idx += kFusedThreads) {
    const int row = idx / nv, v = idx - row * nv;
    uint4 x = ld_stream_v4(prm.grads + static_cast<long long>(row) * prm.row_bytes + (vb0 + v) * 16);
    if (prm.tail_elems != 0 && vb0 + v == prm.num_vec - 1) {     // row padding is not data: zero it
      uint32_t wds[4] = {x.x, x.y, x.z, x.w};
      constexpr int kPerWord = 4 / Elem<DT>::kBytes;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int first = k * kPerWord;
        if (first >= prm.tail_elems) wds[k] = 0u;
        else if (kPerWord == 2 && first + 1 >= prm.tail_elems) wds[k] &= 0x0000ffffu;
      }
      x = make_uint4(wds[0], wds[1], wds[2], wds[3]);
    }
    tile[row * vpb + v] = x;
  }
  for (int i = tid; i < kW * N * 2; i += kFusedThreads) acc[i] = 0.f;
  __syncthreads();

  // ---- statistics of the slice: a warp takes 32 column groups at a time
  float* mine = acc + static_cast<size_t>(warp) * N * 2;
  for (int v0 = warp * 32; v0 < nv; v0 += kFusedThreads) {
    const int v = v0 + lane;
    const bool valid = v < nv;
    float2 sp[NP];
#pragma unroll
    for (int h = 0; h < NP; ++h) sp[h] = make_float2(0.f, 0.f);
    if (valid)
      for (int i = 0; i < N; ++i) {
        const uint4 x = tile[i * vpb + v];
#pragma unroll
        for (int h = 0; h < NP; ++h) sp[h] = __fadd2_rn(sp[h], unpack_pair<DT>(x, h));
      }
    for (int i = 0; i < N; ++i) {
      float2 pa = make_float2(0.f, 0.f), qa = make_float2(0.f, 0.f);
      if (valid) {
        const uint4 x = tile[i * vpb + v];
#pragma unroll
        for (int h = 0; h < NP; ++h) {
          const float2 xv = unpack_pair<DT>(x, h);
          pa = __ffma2_rn(xv, sp[h], pa);
          qa = __ffma2_rn(xv, xv, qa);
        }
      }
      float p = pa.x + pa.y, q = qa.x + qa.y;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        p += __shfl_xor_sync(0xffffffffu, p, o);
        q += __shfl_xor_sync(0xffffffffu, q, o);
      }
      if (lane == 0) { mine[2 * i] += p; mine[2 * i + 1] += q; }
    }
  }
  __syncthreads();
  float* part = const_cast<float*>(prm.coeff.partials) + static_cast<size_t>(blockIdx.x) * 2 * N;
  for (int i = tid; i < N; i += kFusedThreads) {
    float p = 0.f, q = 0.f;
    for (int w = 0; w < kW; ++w) { p += acc[(static_cast<size_t>(w) * N + i) * 2]; q += acc[(static_cast<size_t>(w) * N + i) * 2 + 1]; }
    part[i] = p;
    part[N + i] = q;
  }
  if (!grid_barrier_bounded(prm.barrier, gridDim.x, prm.coeff.flags)) return;

  if (blockIdx.x == 0) coeff_body(prm.coeff, 0);
  if (!grid_barrier_bounded(prm.barrier, gridDim.x, prm.coeff.flags)) return;

  // ---- weighted combination of the slice, from shared memory
  float* g_s = acc;                                   // reuse: N floats
  for (int i = tid; i < N; i += kFusedThreads) g_s[i] = __ldcg(prm.coeff.gamma_f32 + i);
  __syncthreads();
  for (int v = tid; v < nv; v += kFusedThreads) {
    float2 o[NP];
#pragma unroll
    for (int h = 0; h < NP; ++h) o[h] = make_float2(0.f, 0.f);
    for (int i = 0; i < N; ++i) {
      const uint4 x = tile[i * vpb + v];
      const float2 g2 = make_float2(g_s[i], g_s[i]);
#pragma unroll
      for (int h = 0; h < NP; ++h) o[h] = __ffma2_rn(unpack_pair<DT>(x, h), g2, o[h]);
    }
    pass2_store_any<DT, NP>(prm.out, vb0 + v, o, prm.num_vec, prm.tail_elems);
  }
}

// ----------------------------------------------------------------------------------------------
// One launch, two reads: pass 1, the coefficient step and pass 2 in ONE cooperative kernel, for
// matrices too large for shared memory but small enough that two kernel boundaries and a third
// launch are a visible share of the step (hundreds of MB to a few GB).
//   phase 1  exactly pass1_tma_kernel's loop; the block's partial goes to global memory.
//   ticket   every block takes a ticket (integer atomic).  Nobody waits here: the block that draws
//            the last ticket of the launch adds up all partials in index order (so the result does
//            not depend on who came last), runs Eq. 7 / 11 / 12-13 and publishes the weights with
//            a release store of the launch's generation number.
//   phase 2  the other blocks poll that word (bounded, 2 s) while their first copies of phase 2
//            are already in flight (fetching needs no weights), then all blocks form
//            sum_i gamma_i g_i for the 4 KB-per-row column tiles b, b + grid, ... counted from the
//            END of the vector -- the columns phase 1 read last come first.  The matrix is staged
//            by TMA in chunks of 8 rows; a thread owns 16 bytes of every row and adds the rows up
//            in index order, the order and rounding of the pass-2 kernels: the same output bytes.
// The launch is cooperative (all blocks resident), the grid is phase 1's.  sync[0] is the ticket
// counter, sync[1] the published generation; both only grow, a launch owns tickets
// [gen * grid, (gen + 1) * grid), so the kernel can be replayed from a CUDA graph; sync[2], the
// tile counter of phase 2, is set by the block that publishes the weights.
// ----------------------------------------------------------------------------------------------
// One thread waits until a monotonically growing word in global memory reaches `want` (written
// with a release store by another block of the same launch), for at most kWaitLimitNs.
__device__ __forceinline__ bool wait_generation_bounded(const unsigned long long* word, unsigned long long want, uint32_t* flags) {
  const unsigned long long t0 = global_timer_ns();
  bool ok = true;
  for (;;) {
    unsigned long long cur;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(cur) : "l"(word) : "memory");
    if (cur >= want) break;
    if (global_timer_ns() - t0 > kWaitLimitNs) { ok = false; atomicOr(flags, kFlagTimeout); break; }
  }
  __threadfence();
  return ok;
}

struct MidParams {
  Pass1Params p1;
  CoeffParams coeff;               // sets = 1, partials = p1.partials, num_partials = gridDim.x
  const unsigned char* grads;
  unsigned char* out;
  long long row_bytes;
  long long num_vec;               // 16-byte column groups per row (the last may be partial)
  int tail_elems;
  int keep_in_l2;                  // the result fits in L2: store it evict_last
  int stages2;                     // depth of phase 2's ring (stages of 8 boxes x min(N, 8) rows x 512 bytes)
  unsigned long long* sync;        // [0] tickets drawn, [1] generations published, [2] phase-2 tile counter
};

constexpr int kMidPartCap = 2 * kMaxN;   // as coeff_kernel (1024 threads): the same summation order, the same bits
constexpr int kMidChunkRows = 8;   // rows of one phase-2 stage
constexpr int kMidMaxStages2 = 8;

template <int DT, int NR, int WR>
__global__ void __launch_bounds__(kThreads, 2)
mid_fused_kernel(const __grid_constant__ CUtensorMap tmap, const __grid_constant__ CUtensorMap tmap2, const MidParams prm) {
  using C = P1<DT, NR, WR>;
  constexpr int NP = Elem<DT>::kVec / 2;
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  __shared__ int s_abort;
  __shared__ int s_role;                       // 0 = waits for the weights, 1 = computes them, -1 = gave up
  __shared__ unsigned long long s_gen;
  __shared__ float g_s[kMaxFastN];
  __shared__ __align__(8) uint64_t s_full2[kMidMaxStages2];
  __shared__ long long s_item_tile[kMidMaxStages2];   // per stage: the tile id of the item it holds (-1: the ring ends here)
  __shared__ int s_item_chunk[kMidMaxStages2];        // ... and which chunk of rows
  const Pass1Params& p1 = prm.p1;
  const int N = p1.N;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int cw = warp / WR, rw = warp % WR;
  const P1Smem sm = p1_carve<C>(smem_raw, p1.stages, p1.stage_bytes);

  if (tid == 0) {
    s_abort = 0;
    for (int s = 0; s < p1.stages; ++s) mbar_init(&sm.full[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async_smem();
  }
  __syncthreads();

  // ---- phase 1 (Eq. 7): as pass1_tma_kernel
  const int first = blockIdx.x;
  const int stride = gridDim.x;
  const int my_tiles = first < p1.num_tiles ? (p1.num_tiles - first + stride - 1) / stride : 0;
  auto issue = [&](int k, int s) {
    const int col0 = (first + k * stride) * C::TILEC;
    mbar_expect_tx(&sm.full[s], p1.stage_bytes);
#pragma unroll
    for (int c = 0; c < C::WC; ++c)
      tma_load_2d(sm.stage_base + static_cast<size_t>(s) * p1.stage_bytes + static_cast<size_t>(c) * N * kBoxRowBytes,
                  &tmap, &sm.full[s], col0 + c * C::BOXC, 0);
  };
  int issued = 0;
  if (tid == 0) {
    const int pre = my_tiles < p1.stages ? my_tiles : p1.stages;
    for (int k = 0; k < pre; ++k) issue(k, k);
    issued = pre;
  }
  float2 pacc[NR], qacc[NR];
#pragma unroll
  for (int j = 0; j < NR; ++j) pacc[j] = qacc[j] = make_float2(0.f, 0.f);
  p1_outer_clear<C>(sm.outer);
  {
    int s = 0;
    uint32_t parity = 0;
    for (int k = 0; k < my_tiles; ++k) {
      uint4 v[NR];
      if (mbar_wait_bounded(&sm.full[s], parity)) {
        p1_load_rows<C>(v, sm.stage_base + static_cast<size_t>(s) * p1.stage_bytes +
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
      if (tid == 0 && k + p1.stages < my_tiles) {
        fence_proxy_async_smem();
        issue(k + p1.stages, s);
        issued = k + p1.stages + 1;
      }
      p1_xch_finish<C>(sm.xch, k, sp, cw, lane);
      p1_accumulate<DT, C>(v, sp, pacc, qacc);
      if ((k & (kFoldTiles - 1)) == kFoldTiles - 1) p1_fold<C>(pacc, qacc, sm.outer);
      if (++s == p1.stages) { s = 0; parity ^= 1u; }
    }
  }
  float* dst = p1.partials + static_cast<size_t>(blockIdx.x) * 2 * N;
  const bool aborted = s_abort != 0;           // block-uniform (read after the loop's barrier)
  if (aborted) {
    if (tid == 0) p1_drain_after_timeout(sm.full, p1.stages, issued, p1.flags);
    if (tid < 2 * N) dst[tid] = 0.f;
    __syncthreads();
  } else {
    p1_block_store<C>(pacc, qacc, sm.outer, sm.red, dst, dst + N, N);   // ends with a barrier
  }

  // ---- phase 2 set-up: a ring of row chunks (see below).  Nothing of phase 1 lives in shared
  // memory any more; its barriers are invalidated before their bytes are reused.
  // Column tiles of phase 2 are handed out dynamically -- an output element is formed entirely
  // inside one thread, so who computes which tile cannot change a bit of the result, and blocks
  // that run slower simply take fewer tiles.  Tile ids count from the END of the vector.  The
  // first kStatic ids of a block are fixed (b, b + grid, ...), enough to fill its ring before the
  // weights exist; later ids come from a counter that the block publishing the weights sets to
  // kStatic * grid first.  The elected thread fetches the next id one tile ahead of its use.
  const int RB = N < kMidChunkRows ? N : kMidChunkRows;       // rows per chunk = rows of one box
  const int RC = (N + RB - 1) / RB;                           // chunks per column tile
  const uint32_t stage2_bytes = static_cast<uint32_t>(kWarps) * RB * kBoxRowBytes;
  constexpr int T2COLS = kWarps * C::BOXC;                    // columns per phase-2 tile: 4 KB of every row
  const long long tiles2 = (prm.num_vec * C::VEC + T2COLS - 1) / T2COLS;
  const int kStatic = (prm.stages2 + RC - 1) / RC;
  // the ticket first: its round trip to L2 overlaps the set-up of phase 2's barriers
  unsigned long long ticket = 0ull;
  if (tid == 0) {
    __threadfence();                                            // this block's partial is visible ...
    ticket = atomicAdd(&prm.sync[0], 1ull);                     // ... before its ticket is
    for (int s = 0; s < p1.stages; ++s) asm volatile("mbarrier.inval.shared::cta.b64 [%0];" ::"r"(smem_addr(&sm.full[s])) : "memory");
    for (int s = 0; s < prm.stages2; ++s) { mbar_init(&s_full2[s], 1); s_item_tile[s] = -1; }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async_smem();                                 // phase 1 wrote these bytes with ordinary stores
  }
  // producer state (elected thread only)
  long long p_tile = -1;          // id of the tile being issued (-1: none left)
  int p_chunk = 0;                // next chunk of it
  int p_static = 0;               // static ids taken so far
  long long p_next_dyn = -1;      // dynamic id fetched ahead (valid once the weights are published)
  bool p_dyn_ready = false;
  int issued2 = 0;                // items issued (for the drain after a time-out)
  auto next_tile = [&]() -> long long {
    if (p_static < kStatic) {
      const long long id = first + static_cast<long long>(p_static) * stride;
      ++p_static;
      return id < tiles2 ? id : -1;
    }
    if (!p_dyn_ready) return -1;                               // not before the weights are published (initial fill only)
    const long long id = p_next_dyn;
    if (id >= tiles2) return -1;
    p_next_dyn = static_cast<long long>(atomicAdd(&prm.sync[2], 1ull));   // for the tile after this one
    return id;
  };
  auto issue_next = [&](int s) -> bool {  // put the next item into stage s; false when there is none
    if (p_tile < 0 || p_chunk == RC) {
      p_tile = next_tile();
      p_chunk = 0;
      if (p_tile < 0) { s_item_tile[s] = -1; return false; }
    }
    s_item_tile[s] = p_tile;
    s_item_chunk[s] = p_chunk;
    const int col0 = static_cast<int>((tiles2 - 1 - p_tile) * T2COLS);
    const int row0 = p_chunk * RB;
    mbar_expect_tx(&s_full2[s], stage2_bytes);
#pragma unroll
    for (int w = 0; w < kWarps; ++w)
      tma_load_2d(smem_raw + static_cast<size_t>(s) * stage2_bytes + static_cast<size_t>(w) * RB * kBoxRowBytes, &tmap2,
                  &s_full2[s], col0 + w * C::BOXC, row0);
    ++p_chunk;
    ++issued2;
    return true;
  };

  // ---- the last block of the launch computes the weights (Eq. 7, 11, 12-13)
  if (tid == 0) {
    s_gen = ticket / gridDim.x;
    s_role = ((ticket + 1ull) % gridDim.x == 0ull) ? 1 : 0;
    __threadfence();
    if (s_role == 0 && !aborted)                                // fetching needs no weights: fill the ring while waiting
      for (int s = 0; s < prm.stages2; ++s)
        if (!issue_next(s)) break;
  }
  __syncthreads();
  if (s_role == 1) {
    // this block's ring is idle until it has published the weights: it holds the work arrays
    double* work = reinterpret_cast<double*>(smem_raw);
    coeff_core(prm.coeff, 0, work, kMidPartCap, kMaxN, work + kMidPartCap, work + kMidPartCap + kMaxFastN,
               work + kMidPartCap + 2 * kMaxFastN);
    __syncthreads();
    if (tid == 0) {
      prm.sync[2] = static_cast<unsigned long long>(kStatic) * gridDim.x;   // first dynamic tile id of this launch
      __threadfence();
      const unsigned long long g = s_gen + 1ull;
      asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(prm.sync + 1), "l"(g) : "memory");
      if (!aborted) {
        fence_proxy_async_smem();
        for (int s = 0; s < prm.stages2; ++s)
          if (!issue_next(s)) break;
      }
    }
  } else if (tid == 0) {
    if (!wait_generation_bounded(prm.sync + 1, s_gen + 1ull, p1.flags)) s_role = -1;
  }
  __syncthreads();
  if (aborted) return;                                          // nothing of phase 2 was issued
  if (s_role < 0) {                                             // the weights never came: wait for the copies in flight, leave
    if (tid == 0) p1_drain_after_timeout(s_full2, prm.stages2, issued2, p1.flags);
    return;
  }
  if (tid == 0) {                                               // the counter is valid now: fetch the first dynamic id ahead
    p_next_dyn = static_cast<long long>(atomicAdd(&prm.sync[2], 1ull));
    p_dyn_ready = true;
  }
  if (tid < kMaxFastN) g_s[tid] = tid < N ? __ldcg(prm.coeff.gamma_f32 + tid) : 0.f;
  __syncthreads();

  // ---- phase 2 (Eq. 12).  A stage holds RB rows of a 4 KB-per-row column tile: one TMA box of
  // RB x 512 bytes per warp.  Thread (warp, lane) owns the 16-byte column group `lane` of its warp's
  // box and walks the row chunks of a tile in order, adding gamma_i * g_i row by row into registers
  // (the order and rounding of the pass-2 kernels); after the last chunk it stores its 16 bytes.
  // No data crosses threads.
  const unsigned long long keep = prm.keep_in_l2 ? l2_policy_evict_last() : 0ull;
  float2 acc[NP];
#pragma unroll
  for (int h = 0; h < NP; ++h) acc[h] = make_float2(0.f, 0.f);
  int s2 = 0;
  uint32_t parity2 = 0;
  for (;;) {
    const long long tile = s_item_tile[s2];                     // written by the elected thread at least one barrier ago
    if (tile < 0) break;
    const int rc = s_item_chunk[s2];
    uint4 xr[kMidChunkRows];
    const unsigned char* box = smem_raw + static_cast<size_t>(s2) * stage2_bytes + static_cast<size_t>(warp) * RB * kBoxRowBytes + lane * 16;
    if (mbar_wait_bounded(&s_full2[s2], parity2)) {
#pragma unroll
      for (int r = 0; r < kMidChunkRows; ++r) xr[r] = r < RB ? ld_shared_v4(box + r * kBoxRowBytes) : make_uint4(0u, 0u, 0u, 0u);
    } else {
#pragma unroll
      for (int r = 0; r < kMidChunkRows; ++r) xr[r] = make_uint4(0u, 0u, 0u, 0u);
      atomicOr(&s_abort, 1);
    }
    __syncthreads();                                            // the stage is in registers; its item fields are read
    if (s_abort) break;
    if (tid == 0) {
      fence_proxy_async_smem();
      (void)issue_next(s2);
    }
    const int rbase = rc * RB;
#pragma unroll
    for (int r = 0; r < kMidChunkRows; ++r) {
      if (r < RB && rbase + r < N) {
        const float gm = g_s[rbase + r];
        const float2 g2 = make_float2(gm, gm);
#pragma unroll
        for (int h = 0; h < NP; ++h) acc[h] = __ffma2_rn(unpack_pair<DT>(xr[r], h), g2, acc[h]);
      }
    }
    if (rc == RC - 1) {
      const long long v = (tiles2 - 1 - tile) * (T2COLS / C::VEC) + warp * 32 + lane;
      if (v < prm.num_vec) pass2_store_any<DT, NP>(prm.out, v, acc, prm.num_vec, prm.tail_elems, keep);
#pragma unroll
      for (int h = 0; h < NP; ++h) acc[h] = make_float2(0.f, 0.f);
    }
    if (++s2 == prm.stages2) { s2 = 0; parity2 ^= 1u; }
  }
  if (s_abort) {
    if (tid == 0) p1_drain_after_timeout(s_full2, prm.stages2, issued2, p1.flags);
    return;
  }
}

// Self-test of the bounded waits (no data path): which = 0 waits on an mbarrier that nobody arrives
// on, which = 1 on a grid barrier that expects one more block than exists, which = 2 on a
// generation word that nobody advances.  All give up after
// kWaitLimitNs, raise the time-out flag and return; the context stays usable.
__global__ void selftest_wait_kernel(int which, unsigned long long* barrier, uint32_t* flags) {
  __shared__ __align__(8) uint64_t bar;
  if (which == 0) {
    if (threadIdx.x == 0) {
      mbar_init(&bar, 1);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    if (threadIdx.x == 0 && !mbar_wait_bounded(&bar, 0u)) atomicOr(flags, kFlagTimeout);
  } else if (which == 1) {
    (void)grid_barrier_bounded(barrier, gridDim.x + 1u, flags);
  } else {
    // the one-launch kernel's wait for the weights: a generation that nobody publishes
    if (threadIdx.x == 0) (void)wait_generation_bounded(barrier + 2, barrier[2] + 1ull, flags);
  }
}

__global__ void reset_kernel(double* m, long long n, uint32_t* flags, long long* step, unsigned long long* barrier) {
  for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < n;
       i += static_cast<long long>(gridDim.x) * blockDim.x)
    m[i] = 0.0;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    *flags = 0u; *step = 0;
    barrier[0] = 0ull; barrier[1] = 0ull; barrier[2] = 0ull;    // grid barrier; ticket counter and generation of the one-launch kernel
  }
}

}  // namespace adacons
