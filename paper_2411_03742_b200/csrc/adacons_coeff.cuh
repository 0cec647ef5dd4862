// The coefficient step (Eq. 7, Eq. 11, Eq. 12-13; Algorithm 1 steps 2-3): from the partial records to the weights.
#pragma once

#include "adacons_common.cuh"

namespace adacons {

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
  // Column-sharded use (coeff_kernel only).  A statistics record of one set is 2N + 1 doubles: the N
  // sums sum_k g_ik s_k over the set's columns (N p_i of Eq. 7 before the division), the N squared
  // norms q_i, and the number of columns.  stats_out != nullptr: write this set's record (from the
  // partial records, in the usual order) and stop -- no coefficient, no state change.  stats_in !=
  // nullptr: take the statistics from `shards` records per set, [shard][set][2N + 1], added in shard
  // order, instead of from partial records.
  double* stats_out = nullptr;
  const double* stats_in = nullptr;
  int shards = 0;
  long long cols = 0;    // global mode: columns of the one set (for the record's last entry)
};

// Work arrays in shared memory: sh_part holds part_cap doubles (at least 2N), sh_a, sh_u and sh_m N each.
// The records are split into `groups` interleaved subsequences, which fixes the order of the fp64
// sum; groups follows from N, part_cap and group_threads alone (not from the block size), so two
// kernels that pass the same values add the same records in the same order.
// EXT: the kernel honours stats_out / stats_in (the fused kernels have no use for them).
template <bool EXT = false>
__device__ __forceinline__ void coeff_core(const CoeffParams& prm, const int set, double* sh_part, const int part_cap,
                                           const int group_threads, double* sh_a, double* sh_u, double* sh_m) {
  __shared__ int sh_bad, sh_zero, sh_nocols;
  __shared__ double sh_Z;
  __shared__ int sh_uniform;
  const int N = prm.N, i = threadIdx.x, T = blockDim.x;
  const int V = 2 * N;
  const size_t per = static_cast<size_t>(prm.sets) * N;   // stride between coefficient kinds
  if (i == 0) { sh_bad = 0; sh_zero = 0; }   // sh_nocols: written by one thread, and only read, with external statistics
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
  const bool external = EXT && prm.stats_in != nullptr;
  if (external) {                                          // the shards' records of this set, in shard order
    groups = 1;
    const size_t rec = static_cast<size_t>(V) + 1;
    for (int e = i; e <= V; e += T) {
      double acc = 0.0;
      for (int r = 0; r < prm.shards; ++r) acc += prm.stats_in[(static_cast<size_t>(r) * prm.sets + set) * rec + e];
      if (e < V) sh_part[e] = acc;
      else sh_nocols = acc == 0.0 ? 1 : 0;
    }
  }
  for (int slot = i; !external && slot < units * groups; slot += T) {
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
    if (EXT && prm.stats_out != nullptr) {
      double* rec = prm.stats_out + static_cast<size_t>(set) * (V + 1);
      rec[i] = P;
      rec[N + i] = Q;
      if (i == 0) rec[V] = static_cast<double>(prm.seg_off ? prm.seg_off[set + 1] - prm.seg_off[set] : prm.cols);
    }
    p = P / static_cast<double>(N);   // gbar is the mean of the workers (text before Eq. 7)
    q = Q;
    if (!(isfinite(p) && isfinite(q))) atomicOr(&sh_bad, 1);
    if (q == 0.0) atomicOr(&sh_zero, 1);
    prm.coef[3 * per + set * N + i] = p;
    prm.coef[4 * per + set * N + i] = q;
  }
  if (EXT && prm.stats_out != nullptr) return;              // uniform: the whole block leaves
  __syncthreads();
  // A segment without columns is no layer: its all-zero statistics take the usual fallbacks
  // (weights 1/N, state unchanged at zero) but are no degeneracy of the data and raise no flag.
  // (with external statistics: no columns on any shard)
  const bool empty_set = external ? sh_nocols != 0 : (prm.seg_off != nullptr && prm.seg_off[set + 1] == prm.seg_off[set]);
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

template <bool EXT = false>
__device__ __forceinline__ void coeff_body(const CoeffParams& prm, const int set) {
  __shared__ double sh_part[2 * kMaxN];
  __shared__ double sh_a[kMaxN];
  __shared__ double sh_u[kMaxN];
  __shared__ double sh_m[kMaxN];
  coeff_core<EXT>(prm, set, sh_part, 2 * kMaxN, static_cast<int>(blockDim.x), sh_a, sh_u, sh_m);
}

__global__ void __launch_bounds__(kMaxN)
coeff_kernel(const CoeffParams prm) {
  pdl_launch_dependents();
  pdl_wait();                                              // pass 1 has finished and is visible
  coeff_body<true>(prm, blockIdx.x);
}

}  // namespace adacons
