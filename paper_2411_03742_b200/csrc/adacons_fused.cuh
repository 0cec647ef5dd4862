// Kernels that run all three steps in one launch (matrix resident in shared memory: one read; mid-size matrices:
// two reads), the self-test of the bounded waits and the reset kernel.
#pragma once

#include "adacons_common.cuh"
#include "adacons_pass1.cuh"
#include "adacons_coeff.cuh"
#include "adacons_pass2.cuh"

namespace adacons {

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
