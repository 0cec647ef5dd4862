// Pass 1 for bf16 and N <= 64 on the tensor cores: the Gram matrix of every column tile (Eq. 7, third line).
#pragma once

#include "adacons_pass1.cuh"

namespace adacons {

// ----------------------------------------------------------------------------------------------
// Eq. 7 writes the statistic two ways: N p_i = <g_i, sum_j g_j> (what pass1_tma_kernel computes:
// column sums, then dot products) and N p_i = sum_j <g_i, g_j>, the row sums of the Gram matrix
// G G^T, whose diagonal is q_i.  This kernel takes the second form: no column sums, no exchange
// between warps, no block-wide barrier per tile, and under one instruction per element instead of
// four -- at the price of 64 x 64 products per column where 2 x 64 are needed, which only the
// tensor cores can afford.
//
// Tiles and ring as in pass1_dot_kernel: TMA boxes of 64 rows x 512 bytes (256 columns; rows past N
// and columns past d arrive as zeros), full/empty mbarriers per stage, thread 0 issues the copies.
// A row's 512 bytes are eight 64-byte spans of 32 columns.  Warp w works on spans 2 (w / 2) and
// 2 (w / 2) + 1 of every tile and on one half of the Gram matrix's upper block triangle (16 x 16
// blocks (a, b), a <= b): warps with even w own (0,0) (0,1) (0,2) (0,3) (1,1), odd ones (1,2) (1,3)
// (2,2) (2,3) (3,3) -- five blocks, 40 accumulators a thread, either way.
//
// Operands come straight from the unswizzled tile with 16-byte shared loads, no ldmatrix: lane
// (g = lane / 4, t = lane % 4) loads bytes [16 t, 16 t + 16) of the span from rows g, g + 8 of each
// 16-row block (rows with odd g take their two spans in the other order and swap registers, which
// keeps the loads free of bank conflicts although all rows start on the same bank).  Its four bf16 pairs serve as the k-slots (2t, 2t+1) and (2t+8, 2t+9) of two
// m16n8k16 steps.  That permutes the columns inside a span -- harmless, since the contraction index
// of A and B = A^T is permuted alike -- and the registers of a row block are at once its A fragment
// and the B fragments of its two 8-row halves.
//
// Accumulation has two levels: the MMA accumulators take `fold_tiles` tiles (4 chained MMAs per
// tile), then they are added in fp32 (round to nearest) to second-level sums in shared memory and
// cleared, so that a sum never chains more than 4 fold_tiles tensor-core additions.  That matters:
// the tensor cores round the running sum toward zero (measured on a sum of squares: -4e-8 relative
// per chained MMA, i.e. -2e-6 with 16 tiles per fold and -1.4e-4 without folding on 40 M columns).  At the end each warp folds its blocks into row sums (rows of (a, b) for block a's rows,
// columns of an off-diagonal (a, b) for block b's rows, by symmetry) and diagonal entries, in a
// fixed order; the eight warps' results are added in warp order.  Same partial record as
// pass1_tma_kernel: N p_i (un-divided), then q_i.
// ----------------------------------------------------------------------------------------------
struct GramParams {
  int N;
  int num_tiles;        // ceil(d / 256)
  int stages;           // ring depth
  int fold_tiles;       // tiles per first-level accumulation (>= 1)
  float* partials;      // [gridDim.x][2N]
  uint32_t* flags;
};

constexpr int kGramRows = 64;
constexpr uint32_t kGramStageBytes = kGramRows * kBoxRowBytes;   // 32 KB
constexpr int kGramAcc = 40;                                     // accumulators per thread: 5 blocks x 2 halves x 4
constexpr size_t kGramSecondBytes = static_cast<size_t>(kGramAcc) * kThreads * sizeof(float);

__host__ __device__ constexpr int gram_block_a(int set, int i) { return set == 0 ? (i < 4 ? 0 : 1) : (i < 2 ? 1 : (i < 4 ? 2 : 3)); }
__host__ __device__ constexpr int gram_block_b(int set, int i) { return set == 0 ? (i < 4 ? i : 1) : (i == 0 ? 2 : (i == 1 ? 3 : (i == 2 ? 2 : 3))); }

__device__ __forceinline__ void mma_bf16_m16n8k16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                                  uint32_t b0, uint32_t b1) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

// One warp's share of every tile of the block.  Returns with the warp's 40 sums in acc (both levels added).
template <int SET>
__device__ __forceinline__ void gram_warp_loop(const CUtensorMap* tmap, const GramParams& prm, unsigned char* stage_base,
                                               uint64_t* full, uint64_t* empty, float* second, volatile int* s_abort,
                                               int* issued_out, float (&acc)[5][2][4]) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t = lane & 3;
  const bool odd = (g & 1) != 0;
  const int first_off = odd ? 64 : 0;
  const int first = blockIdx.x, stride = gridDim.x;
  const int my_tiles = first < prm.num_tiles ? (prm.num_tiles - first + stride - 1) / stride : 0;
  int issued = 0;
  if (tid == 0) {
    const int pre = my_tiles < prm.stages ? my_tiles : prm.stages;
    for (int k = 0; k < pre; ++k) {
      mbar_expect_tx(&full[k], kGramStageBytes);
      tma_load_2d(stage_base + static_cast<size_t>(k) * kGramStageBytes, tmap, &full[k], (first + k * stride) * 256, 0);
    }
    issued = pre;
  }
#pragma unroll
  for (int i = 0; i < 5; ++i)
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[i][h][e] = 0.f;
#pragma unroll
  for (int e = 0; e < kGramAcc; ++e) second[e * kThreads] = 0.f;
  int s = 0, in_fold = 0;
  uint32_t parity = 0;
  for (int k = 0; k < my_tiles; ++k) {
    // warp-uniform decisions: the MMAs and warp barriers below need all 32 lanes
    if (__any_sync(0xffffffffu, *s_abort != 0)) break;
    const bool landed = mbar_wait_bounded(&full[s], parity);
    if (!__all_sync(0xffffffffu, landed)) { if (lane == 0) *s_abort = 1; break; }
    // The warp's two spans are 128 consecutive bytes of a row.  Rows are 512 bytes apart, so the two
    // rows of a quarter-warp (g even, g odd) would meet on the same banks; instead the odd row reads
    // its spans in the other order and swaps registers afterwards: every 16-byte load is conflict-free.
    const unsigned char* mine = stage_base + static_cast<size_t>(s) * kGramStageBytes + g * kBoxRowBytes + (warp >> 1) * 128 + t * 16;
    uint4 f[4][2][2];                              // [row block][span][8-row half]: rows 16 rb + 8 half + g
    auto load_block = [&](const int rb) {
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const unsigned char* p = mine + (16 * rb + 8 * half) * kBoxRowBytes;
        const uint4 l1 = ld_shared_v4(p + first_off), l2 = ld_shared_v4(p + (64 - first_off));
        f[rb][0][half] = make_uint4(odd ? l2.x : l1.x, odd ? l2.y : l1.y, odd ? l2.z : l1.z, odd ? l2.w : l1.w);
        f[rb][1][half] = make_uint4(odd ? l1.x : l2.x, odd ? l1.y : l2.y, odd ? l1.z : l2.z, odd ? l1.w : l2.w);
      }
    };
    auto block_pair = [&](const int i) {           // both spans, both k-steps of each, both halves of block b
      const int a = gram_block_a(SET, i), b = gram_block_b(SET, i);
#pragma unroll
      for (int sp = 0; sp < 2; ++sp) {
#pragma unroll
        for (int h = 0; h < 2; ++h)
          mma_bf16_m16n8k16(acc[i][h], f[a][sp][0].x, f[a][sp][1].x, f[a][sp][0].y, f[a][sp][1].y, f[b][sp][h].x, f[b][sp][h].y);
#pragma unroll
        for (int h = 0; h < 2; ++h)
          mma_bf16_m16n8k16(acc[i][h], f[a][sp][0].z, f[a][sp][1].z, f[a][sp][0].w, f[a][sp][1].w, f[b][sp][h].z, f[b][sp][h].w);
      }
    };
    auto release_stage = [&]() {                   // the warp has read all it needs of this stage
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[s]);
    };
    if (SET == 0) {                                // (0,0) (0,1) (0,2) (0,3) (1,1): block 0 stays, the others pass through
      load_block(0); block_pair(0);
      load_block(1); block_pair(1); block_pair(4);
      load_block(2); block_pair(2);
      load_block(3); release_stage(); block_pair(3);
    } else {                                       // (1,2) (1,3) (2,2) (2,3) (3,3)
      load_block(1); load_block(2); block_pair(0); block_pair(2);
      load_block(3); release_stage(); block_pair(1); block_pair(3); block_pair(4);
    }
    if (tid == 0 && k + prm.stages < my_tiles) {   // refill this stage once all eight warps have let go of it
      if (!mbar_wait_bounded(&empty[s], parity)) { *s_abort = 1; }
      else {
        fence_proxy_async_smem();
        mbar_expect_tx(&full[s], kGramStageBytes);
        tma_load_2d(stage_base + static_cast<size_t>(s) * kGramStageBytes, tmap, &full[s], (first + (k + prm.stages) * stride) * 256, 0);
        issued = k + prm.stages + 1;
      }
    }
    __syncwarp();
    if (++in_fold == prm.fold_tiles) {
      in_fold = 0;
#pragma unroll
      for (int i = 0; i < 5; ++i)
#pragma unroll
        for (int h = 0; h < 2; ++h)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            float* p = second + ((i * 2 + h) * 4 + e) * kThreads;
            *p = __fadd_rn(*p, acc[i][h][e]);
            acc[i][h][e] = 0.f;
          }
    }
    if (++s == prm.stages) { s = 0; parity ^= 1u; }
  }
#pragma unroll
  for (int i = 0; i < 5; ++i)
#pragma unroll
    for (int h = 0; h < 2; ++h)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[i][h][e] = __fadd_rn(second[((i * 2 + h) * 4 + e) * kThreads], acc[i][h][e]);
  if (tid == 0) *issued_out = issued;
}

// The warp's blocks folded into row sums W[64] and diagonal entries D[64] (this warp's slice of shared memory, zeroed by the caller).
template <int SET>
__device__ __forceinline__ void gram_warp_fold(const float (&acc)[5][2][4], float* W, float* D) {
  const int lane = threadIdx.x & 31, g = lane >> 2, t = lane & 3;
#pragma unroll
  for (int i = 0; i < 5; ++i) {
    const int a = gram_block_a(SET, i), b = gram_block_b(SET, i);
    float r_lo = __fadd_rn(__fadd_rn(acc[i][0][0], acc[i][0][1]), __fadd_rn(acc[i][1][0], acc[i][1][1]));   // row 16a + g
    float r_hi = __fadd_rn(__fadd_rn(acc[i][0][2], acc[i][0][3]), __fadd_rn(acc[i][1][2], acc[i][1][3]));   // row 16a + 8 + g
#pragma unroll
    for (int o = 1; o <= 2; o <<= 1) {
      r_lo += __shfl_xor_sync(0xffffffffu, r_lo, o);
      r_hi += __shfl_xor_sync(0xffffffffu, r_hi, o);
    }
    if (t == 0) { W[16 * a + g] += r_lo; W[16 * a + 8 + g] += r_hi; }
    __syncwarp();
    if (a != b) {                                  // by symmetry the block's column sums belong to block b's rows
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        float c_even = __fadd_rn(acc[i][h][0], acc[i][h][2]);   // column 2t of the half, rows g and g + 8
        float c_odd = __fadd_rn(acc[i][h][1], acc[i][h][3]);    // column 2t + 1
#pragma unroll
        for (int o = 4; o <= 16; o <<= 1) {
          c_even += __shfl_xor_sync(0xffffffffu, c_even, o);
          c_odd += __shfl_xor_sync(0xffffffffu, c_odd, o);
        }
        if (g == 0) { W[16 * b + 8 * h + 2 * t] += c_even; W[16 * b + 8 * h + 2 * t + 1] += c_odd; }
      }
      __syncwarp();
    } else if (t == (g >> 1)) {                    // the diagonal: entry (m, m) sits in the lane whose columns hold m
      D[16 * a + g] = (g & 1) ? acc[i][0][1] : acc[i][0][0];
      D[16 * a + 8 + g] = (g & 1) ? acc[i][1][3] : acc[i][1][2];
    }
  }
}

__global__ void __launch_bounds__(kThreads, 2)
pass1_gram_kernel(const __grid_constant__ CUtensorMap tmap, const GramParams prm) {
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  __shared__ int s_abort;
  __shared__ int s_issued;
  const int N = prm.N;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  unsigned char* stage_base = smem_raw;
  float* second = reinterpret_cast<float*>(smem_raw + static_cast<size_t>(prm.stages) * kGramStageBytes) + tid;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem_raw + static_cast<size_t>(prm.stages) * kGramStageBytes + kGramSecondBytes);
  uint64_t* empty = full + prm.stages;
  if (tid == 0) {
    s_abort = 0;
    s_issued = 0;
    for (int s = 0; s < prm.stages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], kWarps); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    fence_proxy_async_smem();
  }
  __syncthreads();
  pdl_launch_dependents();
  float acc[5][2][4];
  if (warp & 1) gram_warp_loop<1>(&tmap, prm, stage_base, full, empty, second, &s_abort, &s_issued, acc);
  else gram_warp_loop<0>(&tmap, prm, stage_base, full, empty, second, &s_abort, &s_issued, acc);
  __syncthreads();                                 // every warp is done with the ring (or gave up)
  float* dst = prm.partials + static_cast<size_t>(blockIdx.x) * 2 * N;
  if (s_abort) {
    if (tid == 0) p1_drain_after_timeout(full, prm.stages, s_issued, prm.flags);
    for (int i = tid; i < 2 * N; i += kThreads) dst[i] = 0.f;
    return;
  }
  // the ring's memory now holds the warps' results: [warp][row sums 64 | diagonal 64]
  float* R = reinterpret_cast<float*>(smem_raw);
  for (int i = lane; i < 2 * kGramRows; i += 32) R[warp * 2 * kGramRows + i] = 0.f;
  __syncwarp();
  if (warp & 1) gram_warp_fold<1>(acc, R + warp * 2 * kGramRows, R + warp * 2 * kGramRows + kGramRows);
  else gram_warp_fold<0>(acc, R + warp * 2 * kGramRows, R + warp * 2 * kGramRows + kGramRows);
  __syncthreads();
  if (tid < 2 * kGramRows) {
    float v = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) v += R[w * 2 * kGramRows + tid];
    const int row = tid & (kGramRows - 1);
    if (row < N) dst[(tid >= kGramRows ? N : 0) + row] = v;
  }
}

}  // namespace adacons
