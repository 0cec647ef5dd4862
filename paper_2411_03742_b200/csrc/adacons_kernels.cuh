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
// 2-D tiled TMA load global -> shared, completion reported on an mbarrier (no multicast).
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, uint64_t* bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_addr(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_addr(bar)), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
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
// A block owns column tiles  t = blockIdx.x, blockIdx.x + gridDim.x, ...  A tile is WC boxes of
// N rows x 512 bytes, laid side by side; the 8 warps form a WR x WC grid (WR * WC = 8): warp
// (rw, cw) reads box cw and rows rw, rw+WR, ... (NR of them); lane l owns the 16-byte column
// group l of the box.  Per tile every thread
//   1. copies its NR row vectors from shared memory to registers,
//   2. adds them up (partial column sums); with WR > 1 the WR partials are exchanged through
//      shared memory and added in a fixed order, giving the column sums s of the tile,
//   3. accumulates, per row, sum x*s and sum x*x in fp32 (two lanes of packed fp32 FMA).
// One elected thread refills a stage by TMA as soon as the block has copied it to registers.
// ----------------------------------------------------------------------------------------------
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
  constexpr int WC = kWarps / WR;
  constexpr int VEC = Elem<DT>::kVec;
  constexpr int NP = VEC / 2;
  constexpr int BOXC = kBoxRowBytes / Elem<DT>::kBytes;   // columns per box
  constexpr int TILEC = WC * BOXC;                        // columns per tile

  extern __shared__ __align__(1024) unsigned char smem_raw[];
  const int N = prm.N;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int cw = warp / WR, rw = warp % WR;

  unsigned char* stage_base = smem_raw;
  unsigned char* after = smem_raw + static_cast<size_t>(prm.stages) * prm.stage_bytes;
  float* xch = reinterpret_cast<float*>(after);                           // [2][WR][WC*32*VEC]
  constexpr int kXchFloats = (WR > 1) ? 2 * WR * WC * 32 * VEC : 0;
  float* red = xch + kXchFloats;                                          // [kWarps][NR][2]
  uint64_t* full = reinterpret_cast<uint64_t*>(red + kWarps * NR * 2);    // [stages]
  __shared__ int s_abort;

  if (tid == 0) {
    s_abort = 0;
    for (int s = 0; s < prm.stages; ++s) mbar_init(&full[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async_smem();
  }
  __syncthreads();

  const int first = blockIdx.x;
  const int stride = gridDim.x;
  const int my_tiles = first < prm.num_tiles ? (prm.num_tiles - first + stride - 1) / stride : 0;

  auto issue = [&](int k) {   // elected thread: fill stage k % stages with tile k of this block
    const int s = k % prm.stages;
    const int col0 = (first + k * stride) * TILEC;
    mbar_expect_tx(&full[s], prm.stage_bytes);
#pragma unroll
    for (int c = 0; c < WC; ++c)
      tma_load_2d(stage_base + static_cast<size_t>(s) * prm.stage_bytes + static_cast<size_t>(c) * N * kBoxRowBytes,
                  &tmap, &full[s], col0 + c * BOXC, 0);
  };
  if (tid == 0) {
    const int pre = my_tiles < prm.stages ? my_tiles : prm.stages;
    for (int k = 0; k < pre; ++k) issue(k);
  }

  float2 pacc[NR], qacc[NR];
#pragma unroll
  for (int j = 0; j < NR; ++j) pacc[j] = qacc[j] = make_float2(0.f, 0.f);

  bool timed_out = false;
  int issued_upto = my_tiles < prm.stages ? my_tiles : prm.stages;   // meaningful in thread 0 only

  for (int k = 0; k < my_tiles; ++k) {
    const int s = k % prm.stages;
    const uint32_t parity = static_cast<uint32_t>(k / prm.stages) & 1u;
    uint4 v[NR];
#pragma unroll
    for (int j = 0; j < NR; ++j) v[j] = make_uint4(0u, 0u, 0u, 0u);
    if (mbar_wait_bounded(&full[s], parity)) {
      const unsigned char* box = stage_base + static_cast<size_t>(s) * prm.stage_bytes +
                                 static_cast<size_t>(cw) * N * kBoxRowBytes + lane * 16;
#pragma unroll
      for (int j = 0; j < NR; ++j) {
        const int row = rw + WR * j;
        if (row < N) v[j] = ld_shared_v4(box + row * kBoxRowBytes);
      }
    } else {
      timed_out = true;
      atomicOr(&s_abort, 1);
    }

    // partial column sums over this warp's rows (rows in index order)
    float2 sp[NP];
#pragma unroll
    for (int h = 0; h < NP; ++h) sp[h] = make_float2(0.f, 0.f);
#pragma unroll
    for (int j = 0; j < NR; ++j)
#pragma unroll
      for (int h = 0; h < NP; ++h) sp[h] = __fadd2_rn(sp[h], unpack_pair<DT>(v[j], h));

    float* xbuf = xch + (k & 1) * (WR * WC * 32 * VEC);
    if (WR > 1) {
      // layout [rw][cw][half h2][lane][4 floats]: conflict-free 16-byte accesses
#pragma unroll
      for (int h2 = 0; h2 < VEC / 4; ++h2) {
        float4 w4 = make_float4(sp[2 * h2].x, sp[2 * h2].y, sp[2 * h2 + 1].x, sp[2 * h2 + 1].y);
        *reinterpret_cast<float4*>(xbuf + ((rw * WC + cw) * (VEC / 4) + h2) * 128 + lane * 4) = w4;
      }
    }
    __syncthreads();   // every thread holds its rows in registers; exchange buffer is written
    if (s_abort) break;
    if (tid == 0 && k + prm.stages < my_tiles) {
      fence_proxy_async_smem();
      issue(k + prm.stages);
      issued_upto = k + prm.stages + 1;
    }
    if (WR > 1) {
#pragma unroll
      for (int h = 0; h < NP; ++h) sp[h] = make_float2(0.f, 0.f);
#pragma unroll
      for (int r = 0; r < WR; ++r)
#pragma unroll
        for (int h2 = 0; h2 < VEC / 4; ++h2) {
          const float4 w4 = *reinterpret_cast<const float4*>(xbuf + ((r * WC + cw) * (VEC / 4) + h2) * 128 + lane * 4);
          sp[2 * h2] = __fadd2_rn(sp[2 * h2], make_float2(w4.x, w4.y));
          sp[2 * h2 + 1] = __fadd2_rn(sp[2 * h2 + 1], make_float2(w4.z, w4.w));
        }
    }
#pragma unroll
    for (int j = 0; j < NR; ++j)
#pragma unroll
      for (int h = 0; h < NP; ++h) {
        const float2 x = unpack_pair<DT>(v[j], h);
        pacc[j] = __ffma2_rn(x, sp[h], pacc[j]);
        qacc[j] = __ffma2_rn(x, x, qacc[j]);
      }
  }

  if (s_abort) {
    // Leave cleanly: wait (bounded) for the copies still in flight into this block's shared
    // memory, report, and write zero partials so that the finish kernel reads defined data.
    if (tid == 0) {
      for (int k = 0; k < issued_upto; ++k) {
        // stages whose latest fill has not been consumed: the last `stages` issued tiles
        if (k + prm.stages >= issued_upto)
          (void)mbar_wait_bounded(&full[k % prm.stages], static_cast<uint32_t>(k / prm.stages) & 1u);
      }
      atomicOr(prm.flags, kFlagTimeout);
    }
    (void)timed_out;
    if (tid < 2 * N) prm.partials[static_cast<size_t>(blockIdx.x) * 2 * N + tid] = 0.f;
    return;
  }

  // block partial: lanes (fixed xor tree), then the WC warps that share a row (fixed order)
#pragma unroll
  for (int j = 0; j < NR; ++j) {
    float p = pacc[j].x + pacc[j].y, q = qacc[j].x + qacc[j].y;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      p += __shfl_xor_sync(0xffffffffu, p, o);
      q += __shfl_xor_sync(0xffffffffu, q, o);
    }
    if (lane == 0) {
      red[(warp * NR + j) * 2 + 0] = p;
      red[(warp * NR + j) * 2 + 1] = q;
    }
  }
  __syncthreads();
  if (tid < N) {
    const int r_w = tid % WR, j = tid / WR;
    float p = 0.f, q = 0.f;
#pragma unroll
    for (int c = 0; c < WC; ++c) {
      p += red[((c * WR + r_w) * NR + j) * 2 + 0];
      q += red[((c * WR + r_w) * NR + j) * 2 + 1];
    }
    prm.partials[static_cast<size_t>(blockIdx.x) * 2 * N + tid] = p;
    prm.partials[static_cast<size_t>(blockIdx.x) * 2 * N + N + tid] = q;
  }
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
pass1_generic_kernel(const void* __restrict__ grads, int N, long long d, int num_tiles, float* __restrict__ partials) {
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
        if (col < d) s[c] += load_elem<DT>(grads, static_cast<long long>(i) * d + col);
      }
    for (int i = 0; i < N; ++i) {
      float p = 0.f, q = 0.f;
#pragma unroll
      for (int c = 0; c < CPT; ++c) {
        const long long col = c0 + c * kThreads;
        if (col < d) {
          const float x = load_elem<DT>(grads, static_cast<long long>(i) * d + col);
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
// Coefficient step: one block per coefficient set, thread i = worker i.
// ----------------------------------------------------------------------------------------------
struct CoeffParams {
  int N;
  int num_partials;      // rows of `partials` to add up (fixed order 0..num_partials-1)
  int sets;              // coefficient sets (1 = whole vector); partials are [num_partials][sets][2N]
  double beta;
  int momentum, sorted, normalize;
  const float* partials;
  double* coef;          // [5][sets][N]: a, a~, gamma, p, q   (enum adacons_coeff order)
  float* gamma_f32;      // [sets][N]   weights as pass 2 reads them
  double* m;             // [sets][N]   momentum state, in place
  uint32_t* flags;       // device status word (OR)
  long long* step;       // aggregation counter
};

__global__ void __launch_bounds__(kMaxN)
coeff_kernel(const CoeffParams prm) {
  __shared__ double sh_a[kMaxN];
  __shared__ double sh_u[kMaxN];
  __shared__ int sh_bad, sh_zero;
  __shared__ double sh_Z;
  __shared__ int sh_uniform;
  const int N = prm.N, i = threadIdx.x, set = blockIdx.x;
  const size_t per = static_cast<size_t>(prm.sets) * N;   // stride between coefficient kinds
  if (i == 0) { sh_bad = 0; sh_zero = 0; }
  __syncthreads();
  double p = 0.0, q = 0.0;
  if (i < N) {
    double P = 0.0, Q = 0.0;
    const float* base = prm.partials + static_cast<size_t>(set) * 2 * N;
    const size_t row = static_cast<size_t>(prm.sets) * 2 * N;
    for (int c = 0; c < prm.num_partials; ++c) {
      P += static_cast<double>(base[c * row + i]);
      Q += static_cast<double>(base[c * row + N + i]);
    }
    p = P / static_cast<double>(N);   // gbar is the mean of the workers (text before Eq. 7)
    q = Q;
    if (!(isfinite(p) && isfinite(q))) atomicOr(&sh_bad, 1);
    if (q == 0.0) atomicOr(&sh_zero, 1);
    prm.coef[3 * per + set * N + i] = p;
    prm.coef[4 * per + set * N + i] = q;
  }
  __syncthreads();
  uint32_t flags = sh_zero ? kFlagZeroRow : 0u;
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
      if (set == 0) *prm.step += 1;
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
    double* slot = prm.m + static_cast<size_t>(set) * N + rank;
    at = prm.beta * (*slot) + (1.0 - prm.beta) * a;              // exactly one writer per slot
    *slot = at;
  }
  const double u = q > 0.0 ? at / rq : 0.0;                      // unit-column P: weight on raw g_i
  if (i < N) sh_u[i] = u;
  __syncthreads();
  if (i == 0) {
    double Z = 0.0, A = 0.0;
    for (int j = 0; j < N; ++j) { Z += sh_u[j]; A += fabs(sh_u[j]); }
    sh_Z = Z;
    sh_uniform = 0;
    if (prm.normalize) {
      if (!isfinite(Z) || fabs(Z) <= 1e-12 * A) { sh_uniform = 1; flags |= kFlagDegenerateZ; }
      else if (Z < 0.0) flags |= kFlagNegZ;
    }
    if (flags) atomicOr(prm.flags, flags);
    if (set == 0) *prm.step += 1;
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

// ----------------------------------------------------------------------------------------------
// Pass 2, vectorised (16-byte aligned rows).  One thread per 16-byte column group; the groups
// are visited from the END of the vector so that the columns pass 1 touched last, which are
// still in L2, are read first.  Rows are added in index order with fp32 FMA.
// ----------------------------------------------------------------------------------------------
template <int DT>
__global__ void __launch_bounds__(kThreads)
pass2_vec_kernel(const unsigned char* __restrict__ grads, unsigned char* __restrict__ out,
                 const float* __restrict__ gamma, int N, long long row_bytes, long long num_vec) {
  constexpr int VEC = Elem<DT>::kVec;
  constexpr int NP = VEC / 2;
  constexpr int U = 8;                               // row loads in flight per thread
  __shared__ float g_s[kMaxN];
  for (int i = threadIdx.x; i < N; i += kThreads) g_s[i] = gamma[i];
  __syncthreads();
  const long long v = num_vec - 1 - (static_cast<long long>(blockIdx.x) * kThreads + threadIdx.x);
  if (v < 0) return;
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
    for (int u = 0; u < U; ++u) {
      const float g = g_s[i0 + u];
      const float2 g2 = make_float2(g, g);
#pragma unroll
      for (int h = 0; h < NP; ++h) acc[h] = __ffma2_rn(unpack_pair<DT>(x[u], h), g2, acc[h]);
    }
  }
  for (; i0 < N; ++i0) {
    const uint4 x = ld_stream_v4(col + static_cast<long long>(i0) * row_bytes);
    const float g = g_s[i0];
    const float2 g2 = make_float2(g, g);
#pragma unroll
    for (int h = 0; h < NP; ++h) acc[h] = __ffma2_rn(unpack_pair<DT>(x, h), g2, acc[h]);
  }
  uint4 o;
  if constexpr (DT == 0) {
    o = make_uint4(__float_as_uint(acc[0].x), __float_as_uint(acc[0].y), __float_as_uint(acc[1].x),
                   __float_as_uint(acc[1].y));
  } else {
    o = make_uint4(pack_bf16x2_rn(acc[0].x, acc[0].y), pack_bf16x2_rn(acc[1].x, acc[1].y),
                   pack_bf16x2_rn(acc[NP - 2].x, acc[NP - 2].y), pack_bf16x2_rn(acc[NP - 1].x, acc[NP - 1].y));
  }
  *reinterpret_cast<uint4*>(out + v * 16) = o;
}

// Pass 2, generic: one thread per column, scalar loads.
template <int DT>
__global__ void __launch_bounds__(kThreads)
pass2_generic_kernel(const void* __restrict__ grads, void* __restrict__ out, const float* __restrict__ gamma,
                     int N, long long d) {
  __shared__ float g_s[kMaxN];
  for (int i = threadIdx.x; i < N; i += kThreads) g_s[i] = gamma[i];
  __syncthreads();
  const long long k = static_cast<long long>(blockIdx.x) * kThreads + threadIdx.x;
  if (k >= d) return;
  float acc = 0.f;
  for (int i = 0; i < N; ++i) acc = fmaf(load_elem<DT>(grads, static_cast<long long>(i) * d + k), g_s[i], acc);
  if constexpr (DT == 0) reinterpret_cast<float*>(out)[k] = acc;
  else reinterpret_cast<unsigned short*>(out)[k] = static_cast<unsigned short>(pack_bf16x2_rn(acc, 0.f) & 0xffffu);
}

__global__ void reset_kernel(double* m, long long n, uint32_t* flags, long long* step) {
  for (long long i = blockIdx.x * static_cast<long long>(blockDim.x) + threadIdx.x; i < n;
       i += static_cast<long long>(gridDim.x) * blockDim.x)
    m[i] = 0.0;
  if (blockIdx.x == 0 && threadIdx.x == 0) { *flags = 0u; *step = 0; }
}

}  // namespace adacons
