// Pass 1 (Eq. 7) for rows that start at arbitrary element offsets: the staged kernel fed by one tensor map per row class.
#pragma once

#include "adacons_pass1.cuh"

namespace adacons {

// ----------------------------------------------------------------------------------------------
// A row pitch that is not a multiple of 16 bytes (contiguous rows of an odd length) puts every row
// at another offset from a 16-byte boundary, and one tensor map cannot describe that: its strides
// must be multiples of 16 bytes.  But k = 16 / gcd(pitch in bytes, 16) rows further on (k = 2, 4 or
// 8) the offset repeats, so the rows r, r + k, r + 2k, ... form a matrix with a legal stride: the
// matrix is described by k tensor maps, class c holding rows c, c + k, ..., each based at the
// 16-byte boundary at or below its first body column.  A tile is k boxes (per column warp) of
// rows-of-the-class x 512 bytes; a row lands `shift_c` bytes into its 512-byte slot, the same shift
// for every tile.  A thread reads the aligned 16 bytes that hold the start of its column group and
// the next 16, and shifts the group into place (realign_16: which words it takes is a branch on the
// row, which a warp takes as one).  The 512-byte slot holds 31 whole groups behind a shift of up to
// 15 bytes, so lane 31 of every warp idles: a tile is 31 groups wide per column warp.  From there on
// the tile is pass1_tma_kernel's: same warp grid, exchange of partial column sums, accumulation
// and partial record.
//
// The body the kernel covers is whole 16-byte column groups [head, head + body_cols) with head =
// one vector width, so that a map's base never lies before its first row, and with at least one
// vector width left after it; each map's extent ends with the body, and the tensor copy zero-fills
// what lies beyond, so nothing past a row is read.  The columns before and after the body are one
// more partial record (edge_stats_kernel).
// ----------------------------------------------------------------------------------------------
constexpr int kShiftMaxClasses = 8;
constexpr int kShiftGroups = 31;     // column groups of a 512-byte slot that are whole whatever the shift

struct ShiftMaps {
  CUtensorMap m[kShiftMaxClasses];
};

struct Pass1ShiftParams {
  int N;
  int num_tiles;                 // ceil(body groups / (WC * 31))
  int stages;
  uint32_t stage_bytes;          // WC * N * 512
  int classes;                   // k
  int class_base[kShiftMaxClasses];   // first slot of class c in a box: rows of the classes before it
  int class_shift[kShiftMaxClasses];  // bytes by which the rows of class c land late in their slots
  float* partials;
  uint32_t* flags;
};

template <int DT, int NR, int WR>
__global__ void __launch_bounds__(kThreads, 2)
pass1_shift_kernel(const __grid_constant__ ShiftMaps maps, const Pass1ShiftParams prm) {
  using C = P1<DT, NR, WR>;
  constexpr int VEC = C::VEC;
  constexpr int kTileGroupCols = kShiftGroups * VEC;          // body columns per column warp and tile
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

  // slot and shift of this thread's rows: row r is entry r / k of class r % k
  int slot[NR];
  uint32_t shifts = 0;
#pragma unroll
  for (int j = 0; j < NR; ++j) {
    const int row = rw + WR * j;
    const int c = row % prm.classes;
    slot[j] = prm.class_base[c] + row / prm.classes;
    shifts |= static_cast<uint32_t>(prm.class_shift[c]) << (4 * j);
  }

  // elected thread: fill stage s with tile k of this block, one box per class and column warp
  auto issue = [&](int k, int s) {
    const int g0 = (first + k * stride) * C::WC * kTileGroupCols;     // first body column of the tile
    unsigned char* stage = sm.stage_base + static_cast<size_t>(s) * prm.stage_bytes;
    mbar_expect_tx(&sm.full[s], prm.stage_bytes);
#pragma unroll
    for (int w = 0; w < C::WC; ++w)
      for (int c = 0; c < prm.classes; ++c) {
        if (c >= N) break;                                            // fewer rows than classes: the rest are empty
        tma_load_2d(stage + (static_cast<size_t>(w) * N + prm.class_base[c]) * kBoxRowBytes, &maps.m[c], &sm.full[s],
                    g0 + w * kTileGroupCols, 0);
      }
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
      const unsigned char* box_lane = sm.stage_base + static_cast<size_t>(s) * prm.stage_bytes +
                                      static_cast<size_t>(cw) * N * kBoxRowBytes + lane * 16;
#pragma unroll
      for (int j = 0; j < NR; ++j) {
        if (rw + WR * j < N && lane < kShiftGroups) {
          const unsigned char* p = box_lane + slot[j] * kBoxRowBytes;
          v[j] = realign_16(ld_shared_v4(p), ld_shared_v4(p + 16), static_cast<int>((shifts >> (4 * j)) & 15u));
        } else {
          v[j] = make_uint4(0u, 0u, 0u, 0u);
        }
      }
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

}  // namespace adacons
