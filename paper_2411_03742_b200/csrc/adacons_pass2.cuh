// Pass 2 (Eq. 12): out_k = cast(sum_i gamma_i g_ik), rows added in index order, one rounding to the storage type.
#pragma once

#include "adacons_common.cuh"
#include "adacons_pass1.cuh"   // load_elem

namespace adacons {

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
// Pass 2 for rows that start anywhere (a row pitch that is not a multiple of 16 bytes, or `out` off
// a 16-byte boundary by another amount than the rows): vector loads all the same.  The body of the
// vector is cut into 16-byte groups of OUT (so the stores are aligned); the 16 bytes of row i that
// belong to a group start `shift_i` bytes into an aligned 16-byte group of the matrix, the same
// shift for every group of the row.  A thread loads that aligned group and the next one and
// extracts its bytes with funnel shifts; which words it takes depends on the row alone, so the
// choice is a branch the whole grid takes alike.  The second load is the first load of the
// neighbouring thread (an L1 hit).  Rows are added in index order with the rounding of the other
// pass-2 kernels, so the bytes agree with theirs.  The body leaves out the first 16 to 31 bytes and
// the last 16 to 31 bytes of the vector (edge_combine_kernel), so no load leaves a row.
// ----------------------------------------------------------------------------------------------
constexpr int kPass2ShiftRows = 4;   // rows per batch: 2 * kPass2ShiftRows 16-byte loads in flight per thread

// grads: byte address of element (0, 0); body_off: byte offset of the body's first column within a row;
// out_body: the (16-byte aligned) address of that column in the result; num_groups 16-byte groups follow.
template <int DT>
__global__ void __launch_bounds__(kThreads)
pass2_shift_kernel(const unsigned char* __restrict__ grads, unsigned char* __restrict__ out_body, const float* __restrict__ gamma,
                   int N, long long row_bytes, long long body_off, long long num_groups) {
  constexpr int NP = Elem<DT>::kVec / 2;
  constexpr int U = kPass2ShiftRows;
  __shared__ float g_s[kMaxN];
  __shared__ unsigned char shift_s[kMaxN];
  pdl_wait();
  for (int i = threadIdx.x; i < N; i += kThreads) {
    g_s[i] = gamma[i];
    shift_s[i] = static_cast<unsigned char>((reinterpret_cast<unsigned long long>(grads) + static_cast<unsigned long long>(i) * row_bytes + body_off) & 15ull);
  }
  __syncthreads();
  const long long j = static_cast<long long>(blockIdx.x) * kThreads + threadIdx.x;
  if (j >= num_groups) return;
  const unsigned char* col = grads + body_off + j * 16;
  float2 acc[NP];
#pragma unroll
  for (int h = 0; h < NP; ++h) acc[h] = make_float2(0.f, 0.f);
  for (int i0 = 0; i0 < N; i0 += U) {
    uint4 lo[U], hi[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int i = i0 + u < N ? i0 + u : N - 1;     // rows past the end repeat the last one and get weight 0
      const unsigned char* a = col + static_cast<long long>(i) * row_bytes - shift_s[i];
      lo[u] = ld_nc_v4(a);
      hi[u] = ld_nc_v4(a + 16);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int i = i0 + u < N ? i0 + u : N - 1;
      const float g = i0 + u < N ? g_s[i] : 0.f;
      const uint4 x = realign_16(lo[u], hi[u], shift_s[i]);
      const float2 g2 = make_float2(g, g);
#pragma unroll
      for (int h = 0; h < NP; ++h) acc[h] = __ffma2_rn(unpack_pair<DT>(x, h), g2, acc[h]);
    }
  }
  pass2_store<DT, NP>(out_body, j, acc);
}

// ----------------------------------------------------------------------------------------------
// Edges of a matrix whose rows start off a 16-byte boundary (every row by the same amount: the row
// pitch is a multiple of 16 bytes).  The vectorised kernels then run on the aligned body -- from
// each row's first 16-byte boundary on -- and these two one-block kernels do the few columns left:
// edge_stats_kernel adds the share of the first `head` and the last `tail` columns (24 in all at
// most) in Eq. 7 as one more partial record,
// edge_combine_kernel forms Eq. 12 for the first `head` and the last `tail` columns (32 in all at
// most; element-wise, so nothing is read or written past the vector).
// ----------------------------------------------------------------------------------------------
constexpr int kEdgeCols = 24;   // most columns the statistics edge kernel takes (head + tail)
template <int DT>
__global__ void __launch_bounds__(kThreads)
edge_stats_kernel(const void* __restrict__ grads, int N, long long d, long long pitch, int head, int tail, float* __restrict__ record) {
  __shared__ float x[kMaxFastN * kEdgeCols];
  __shared__ float s[kEdgeCols];
  const int tid = threadIdx.x;
  const int cols = head + tail;                    // columns [0, head) and [d - tail, d)
  for (int idx = tid; idx < N * cols; idx += kThreads) {
    const int i = idx / cols, k = idx - i * cols;
    const long long col = k < head ? k : d - tail + (k - head);
    x[i * kEdgeCols + k] = load_elem<DT>(grads, static_cast<long long>(i) * pitch + col);
  }
  __syncthreads();
  if (tid < cols) {
    float a = 0.f;
    for (int i = 0; i < N; ++i) a += x[i * kEdgeCols + tid];
    s[tid] = a;
  }
  __syncthreads();
  if (tid < N) {
    float pp = 0.f, qq = 0.f;
    for (int k = 0; k < cols; ++k) {
      const float v = x[tid * kEdgeCols + k];
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
  __shared__ float g_s[kMaxN];
  for (int i = threadIdx.x; i < N; i += 32) g_s[i] = gamma[i];
  __syncthreads();
  const int k = threadIdx.x;                       // head + tail <= 32
  if (k >= head + tail) return;
  const long long col = k < head ? k : d - tail + (k - head);
  float acc = 0.f;
  for (int i = 0; i < N; ++i) acc = fmaf(load_elem<DT>(grads, static_cast<long long>(i) * pitch + col), g_s[i], acc);
  if constexpr (DT == 0) reinterpret_cast<float*>(out)[col] = acc;
  else reinterpret_cast<unsigned short*>(out)[col] = static_cast<unsigned short>(pack_bf16x2_rn(acc, 0.f) & 0xffffu);
}

}  // namespace adacons
