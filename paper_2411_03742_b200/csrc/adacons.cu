// Host side of the AdaCons aggregation library: context, launch plan and the C ABI declared in
// include/adacons.h.  All arithmetic of the method runs in the kernels of adacons_kernels.cuh;
// this file validates arguments, owns device memory and launches.
#include "adacons.h"

#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <pthread.h>
#include <new>
#include <vector>

#include "adacons_kernels.cuh"

using namespace adacons;

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// TMA coordinates are 32-bit: longer vectors are walked in column chunks of this many elements,
// each with its own tensor map and its own slice of the partial records.
constexpr long long kChunkCols = 1ll << 30;

// The opt-in limit on dynamic shared memory is a property of a kernel (per device), not of a
// context, and contexts of different shapes share kernel instantiations.  Every kernel therefore
// gets one fixed limit that covers all plans; a plan's own size only goes into its launches.
constexpr size_t kPass1SmemBudget = 110 * 1024;                    // two blocks per SM
constexpr size_t kPass1SmemCap = 112 * 1024;                       // budget + barriers
constexpr size_t kFusedSmemCap = 160 * 1024;
constexpr size_t kGenericSmemCap = static_cast<size_t>(kWarps) * kMaxN * 2 * sizeof(float);
// Largest matrix (bytes) that takes the one-launch kernel by default: beyond it two kernel
// boundaries are a negligible share of the step and the separate kernels are at least as fast.
constexpr long long kOneLaunchMaxBytes = 1ll << 30;
// Ring depth of the one-launch kernel's second phase.  Two stages of 32 KB per block (two blocks per
// SM) keep enough bytes in flight; a third made the phase 3-5 % slower on both mid-size workloads.
constexpr int kMidStages2 = 2;
static_assert(kMidStages2 >= 2 && kMidStages2 <= kMidMaxStages2, "the ring needs two stages: a stage's item fields are rewritten one barrier after they are read");

bool set_smem_cap(const void* kernel, size_t cap) {
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(cap)) == cudaSuccess)
    return true;
  cudaGetLastError();
  return false;
}

struct Pass1Plan {            // TMA-staged pass 1 for this (N, dtype)
  bool available = false;
  int NR = 0, WR = 0;
  int tile_cols = 0;
  int num_tiles = 0;
  int stages = 0;
  uint32_t stage_bytes = 0;
  size_t smem_bytes = 0;
  int grid = 0;
  const void* kernel = nullptr;
};

}  // namespace

struct adacons_ctx {
  int N = 0;
  long long d = 0;
  int dtype = 0;
  int elem_bytes = 4;
  long long pitch = 0;                  // elements between the starts of two rows (>= d)
  int device = 0;
  int num_sms = 0;
  long long l2_bytes = 0;
  std::vector<long long> seg_offsets;   // S + 1 entries
  int num_segments = 1;

  // options
  double beta = 0.99;
  int momentum = 1, sorted = 1, normalize = 1, per_segment = 0, overlap_launch = 1, fused_small = 1;

  // plans
  Pass1Plan fast;
  int generic_grid = 0;
  int generic_tiles = 0;
  size_t generic_smem = 0;
  int max_partials = 0;

  // device memory
  float* partials = nullptr;      // [max_partials][2N]
  double* coef = nullptr;         // [5][sets][N]
  float* gamma_f32 = nullptr;     // [sets][N]
  double* m = nullptr;            // [sets][N]
  double* z = nullptr;            // [sets]
  uint32_t* flags = nullptr;
  long long* step = nullptr;
  void* staging = nullptr;        // adacons_aggregate_host: N*pitch + d elements
  size_t staging_bytes = 0;
  size_t scratch_bytes = 0;

  // more than 64 workers: column sums to scratch, then dot products per 64-row chunk
  bool big_available = false;
  int big_grid = 0, big_tiles = 0, big_stages = 0;
  size_t big_smem = 0;
  float* d_colsum = nullptr;            // [big_tiles * tile columns], zero past d
  size_t colsum_bytes = 0;
  CUtensorMap tmap_big;
  const void* tmap_big_for = nullptr;
  // 64 < N <= 256: one read of the matrix, one block per tile of 128 rows x 256 bytes or 256 rows x 128 bytes
  bool tall_available = false;
  int tall_grid = 0, tall_tiles = 0, tall_stages = 0;
  size_t tall_smem = 0;
  int tall_tiles_opt = 1;               // ADACONS_OPT_TALL_TILES
  CUtensorMap tmap_tall;
  const void* tmap_tall_for = nullptr;
  // 64 < N <= 512: one read of the matrix by clusters of 2, 4 or 8 blocks (64 rows each)
  bool cl_available = false;
  int cl_size = 0, cl_grid = 0, cl_tiles = 0;
  size_t cl_smem = 0;
  int cluster_pass1 = 0;                // ADACONS_OPT_CLUSTER_PASS1 (opt-in)
  int shifted_loads = 1;                // ADACONS_OPT_SHIFTED_LOADS
  Pass1Plan shift;                      // pass1_shift_kernel: rows at arbitrary element offsets (N <= 64)
  long long shift_body_cols = 0;
  int shift_head = 0, shift_tail = 0;
  ShiftMaps shift_maps;                 // one tensor map per row class, for the matrix at shift_maps_for
  const void* shift_maps_for = nullptr;
  int shift_classes = 1, shift_class_base[kShiftMaxClasses] = {0}, shift_class_shift[kShiftMaxClasses] = {0};
  // bf16, N <= 64: pass 1 from the Gram matrix on the tensor cores (pass1_gram_kernel)
  bool gram_available = false;
  int gram_grid = 0, gram_tiles = 0, gram_stages = 2;
  size_t gram_smem = 0;
  int gram_fold = 0;                    // ADACONS_OPT_GRAM_PASS1: 0 = off, n >= 1 = on, n tiles per first-level sum
  int last_launches = 3;

  // single-pass path for problems that fit in the grid's shared memory
  bool fused_available = false;
  int fused_grid = 0, fused_vpb = 0;
  size_t fused_smem = 0;
  unsigned long long* d_barrier = nullptr;

  // one launch for mid-size matrices: pass 1, coefficient step and pass 2 in one cooperative kernel
  bool mid_available = false;
  int mid_grid = 0, mid_stages2 = 0;
  size_t mid_smem = 0;
  const void* mid_kernel = nullptr;
  CUtensorMap tmap_mid2;                // phase 2: boxes of min(N, 8) rows x 512 bytes
  const void* tmap_mid2_for = nullptr;
  int one_launch = 1;                   // ADACONS_OPT_ONE_LAUNCH: 0 never, 1 by size, 2 whenever possible

  // per-segment ("layer-wise") plan, built when ADACONS_OPT_PER_SEGMENT is switched on
  int seg_grid = 0;               // blocks of pass1_seg_kernel
  int seg_records = 0;
  const void* seg_kernel = nullptr;
  long long* d_seg_off = nullptr;       // [S+1]
  int* d_blk_first_seg = nullptr;       // [seg_grid]
  int* d_blk_last_seg = nullptr;        // [seg_grid]
  int* d_rec_begin = nullptr;           // [S]
  int* d_rec_count = nullptr;           // [S]
  int* d_set_first_block = nullptr;     // [S]
  float* d_records = nullptr;           // [seg_records][2N]
  int* d_pass2_blk_seg = nullptr;       // [pass-2 blocks][2]: segment code, last segment
  size_t seg_bytes = 0;

  EncodeTiledFn encode = nullptr;
  int num_chunks = 1;                   // ceil(d / kChunkCols)
  std::vector<CUtensorMap> tmaps;       // one per column chunk; tmaps[0] covers everything when d <= 2^30
  const void* tmap_for = nullptr;

  CUtensorMap tmap_body;                // pass 1 on the aligned body of a matrix whose rows start off a 16-byte boundary
  const void* tmap_body_for = nullptr;
  int aligned_body = 1;                 // ADACONS_OPT_ALIGNED_BODY
  int last_path = 0;
  int last_pass2 = 0;                   // 0 none, 1 generic, 2 16-byte vectors, 3 32-byte vectors
  long long total_launches = 0;

  // optional per-kernel timing (ADACONS_OPT_PROFILE)
  static constexpr int kProfSlots = 64;
  int profile = 0;
  long long prof_calls = 0;
  cudaEvent_t prof_ev[kProfSlots][4] = {};
  bool prof_ready = false;

  int sets() const { return per_segment ? num_segments : 1; }
};

namespace {

template <int DT, int NR, int WR>
const void* pass1_fn() { return reinterpret_cast<const void*>(&pass1_tma_kernel<DT, NR, WR>); }

const void* select_pass1(int dtype, int NR, int WR) {
#define ADACONS_PICK(DT)                                     \
  if (WR == 1) {                                             \
    if (NR == 1) return pass1_fn<DT, 1, 1>();                \
    if (NR == 2) return pass1_fn<DT, 2, 1>();                \
    if (NR == 4) return pass1_fn<DT, 4, 1>();                \
    return pass1_fn<DT, 8, 1>();                             \
  }                                                          \
  if (WR == 2) return pass1_fn<DT, 8, 2>();                  \
  if (WR == 4) return pass1_fn<DT, 8, 4>();                  \
  return pass1_fn<DT, 8, 8>();
  if (dtype == ADACONS_F32) { ADACONS_PICK(0) }
  ADACONS_PICK(1)
#undef ADACONS_PICK
}

template <int DT, int NR, int WR>
const void* pass1_shift_fn() { return reinterpret_cast<const void*>(&pass1_shift_kernel<DT, NR, WR>); }

const void* select_pass1_shift(int dtype, int NR, int WR) {
#define ADACONS_PICK(DT)                                     \
  if (WR == 1) {                                             \
    if (NR == 1) return pass1_shift_fn<DT, 1, 1>();          \
    if (NR == 2) return pass1_shift_fn<DT, 2, 1>();          \
    if (NR == 4) return pass1_shift_fn<DT, 4, 1>();          \
    return pass1_shift_fn<DT, 8, 1>();                       \
  }                                                          \
  if (WR == 2) return pass1_shift_fn<DT, 8, 2>();            \
  if (WR == 4) return pass1_shift_fn<DT, 8, 4>();            \
  return pass1_shift_fn<DT, 8, 8>();
  if (dtype == ADACONS_F32) { ADACONS_PICK(0) }
  ADACONS_PICK(1)
#undef ADACONS_PICK
}

template <int DT, int NR, int WR>
const void* pass1_seg_fn() { return reinterpret_cast<const void*>(&pass1_seg_kernel<DT, NR, WR>); }

const void* select_pass1_seg(int dtype, int NR, int WR) {
#define ADACONS_PICK(DT)                                     \
  if (WR == 1) {                                             \
    if (NR == 1) return pass1_seg_fn<DT, 1, 1>();            \
    if (NR == 2) return pass1_seg_fn<DT, 2, 1>();            \
    if (NR == 4) return pass1_seg_fn<DT, 4, 1>();            \
    return pass1_seg_fn<DT, 8, 1>();                         \
  }                                                          \
  if (WR == 2) return pass1_seg_fn<DT, 8, 2>();              \
  if (WR == 4) return pass1_seg_fn<DT, 8, 4>();              \
  return pass1_seg_fn<DT, 8, 8>();
  if (dtype == ADACONS_F32) { ADACONS_PICK(0) }
  ADACONS_PICK(1)
#undef ADACONS_PICK
}

template <int DT, int NR, int WR>
const void* mid_fn() { return reinterpret_cast<const void*>(&mid_fused_kernel<DT, NR, WR>); }

const void* select_mid(int dtype, int NR, int WR) {
#define ADACONS_PICK(DT)                                     \
  if (WR == 1) {                                             \
    if (NR == 1) return mid_fn<DT, 1, 1>();                  \
    if (NR == 2) return mid_fn<DT, 2, 1>();                  \
    if (NR == 4) return mid_fn<DT, 4, 1>();                  \
    return mid_fn<DT, 8, 1>();                               \
  }                                                          \
  if (WR == 2) return mid_fn<DT, 8, 2>();                    \
  if (WR == 4) return mid_fn<DT, 8, 4>();                    \
  return mid_fn<DT, 8, 8>();
  if (dtype == ADACONS_F32) { ADACONS_PICK(0) }
  ADACONS_PICK(1)
#undef ADACONS_PICK
}

// Launch with (or without) the programmatic-stream-serialisation attribute.
template <typename... KArgs, typename... Args>
cudaError_t launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, bool pdl,
                          Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

int plan_fast(adacons_ctx* c) {
  Pass1Plan& f = c->fast;
  f.available = false;
  const int N = c->N;
  if (N > kMaxFastN) return ADACONS_OK;
  if ((c->pitch * c->elem_bytes) % 16 != 0) return ADACONS_OK;
  if (c->encode == nullptr) return ADACONS_OK;
  c->num_chunks = static_cast<int>((c->d + kChunkCols - 1) / kChunkCols);
  c->tmap_for = nullptr;
  const long long first_cols = c->d < kChunkCols ? c->d : kChunkCols;   // columns of the first (largest) chunk
  int WR, NR;
  if (N <= 8) { WR = 1; NR = N <= 1 ? 1 : N <= 2 ? 2 : N <= 4 ? 4 : 8; }
  else if (N <= 16) { WR = 2; NR = 8; }
  else if (N <= 32) { WR = 4; NR = 8; }
  else { WR = 8; NR = 8; }
  const int WC = kWarps / WR;
  const int vec = c->dtype == ADACONS_F32 ? 4 : 8;
  f.NR = NR; f.WR = WR;
  f.tile_cols = WC * (kBoxRowBytes / c->elem_bytes);
  f.num_tiles = static_cast<int>((first_cols + f.tile_cols - 1) / f.tile_cols);
  f.stage_bytes = static_cast<uint32_t>(WC) * N * kBoxRowBytes;
  const size_t xch = WR > 1 ? static_cast<size_t>(2) * WR * WC * 32 * vec * sizeof(float) : 0;
  const size_t fixed = xch + static_cast<size_t>(kWarps) * NR * 2 * sizeof(float) +
                       static_cast<size_t>(2) * NR * kThreads * sizeof(float);   // exchange, block reduce, second-level sums
  const size_t budget = kPass1SmemBudget;
  int stages = static_cast<int>((budget - fixed - 64) / f.stage_bytes);
  if (stages > 8) stages = 8;
  if (stages < 2) stages = 2;
  f.stages = stages;
  f.smem_bytes = static_cast<size_t>(stages) * f.stage_bytes + fixed + static_cast<size_t>(stages) * 8;
  f.kernel = select_pass1(c->dtype, NR, WR);
  if (f.smem_bytes > kPass1SmemCap || !set_smem_cap(f.kernel, kPass1SmemCap)) return ADACONS_ECUDA;
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, f.kernel, kThreads, f.smem_bytes) != cudaSuccess ||
      per_sm < 1) {
    cudaGetLastError();
    return ADACONS_ECUDA;
  }
  f.grid = per_sm * c->num_sms;
  if (f.grid > f.num_tiles) f.grid = f.num_tiles;
  f.available = true;
  return ADACONS_OK;
}

// N <= 64, rows at arbitrary element offsets (any pitch): one tensor map per class of rows that share an
// offset from a 16-byte boundary (pass1_shift_kernel).  The body is the whole 16-byte column groups
// between one vector width of head columns and one to two vector widths of tail columns.
int plan_shift(adacons_ctx* c) {
  Pass1Plan& f = c->shift;
  f.available = false;
  c->shift_maps_for = nullptr;
  const int N = c->N;
  const int vec = 16 / c->elem_bytes;
  if (N > kMaxFastN || c->d < 4 * vec || c->d > kChunkCols || c->encode == nullptr) return ADACONS_OK;
  // A tensor copy costs the copy engine a fixed 30 ns or so besides its bytes, so the k classes must not be too
  // thin: with 4 KB per copy (8 rows) the kernel reads at 4.4-5.0 TB/s, with 1 KB at 2.3-2.6 TB/s.  The scalar
  // kernel does 2.6-3.4 TB/s on fp32 and 1.2-1.5 TB/s on bf16, hence: bf16 always, fp32 from 4 rows per class on.
  {
    const unsigned rem = static_cast<unsigned>((static_cast<unsigned long long>(c->pitch) * c->elem_bytes) % 16);
    const int k = rem == 0 ? 1 : static_cast<int>(16u / (rem & (~rem + 1u)));
    if (c->dtype == ADACONS_F32 && N < 4 * k) return ADACONS_OK;
  }
  c->shift_head = vec;
  c->shift_body_cols = (c->d - 2 * vec) / vec * vec;
  c->shift_tail = static_cast<int>(c->d - vec - c->shift_body_cols);
  int WR, NR;
  if (N <= 8) { WR = 1; NR = N <= 1 ? 1 : N <= 2 ? 2 : N <= 4 ? 4 : 8; }
  else if (N <= 16) { WR = 2; NR = 8; }
  else if (N <= 32) { WR = 4; NR = 8; }
  else { WR = 8; NR = 8; }
  const int WC = kWarps / WR;
  f.NR = NR; f.WR = WR;
  f.tile_cols = WC * kShiftGroups * vec;
  f.num_tiles = static_cast<int>((c->shift_body_cols + f.tile_cols - 1) / f.tile_cols);
  f.stage_bytes = static_cast<uint32_t>(WC) * N * kBoxRowBytes;
  const size_t xch = WR > 1 ? static_cast<size_t>(2) * WR * WC * 32 * vec * sizeof(float) : 0;
  const size_t fixed = xch + static_cast<size_t>(kWarps) * NR * 2 * sizeof(float) + static_cast<size_t>(2) * NR * kThreads * sizeof(float);
  int stages = static_cast<int>((kPass1SmemBudget - fixed - 64) / f.stage_bytes);
  if (stages > 8) stages = 8;
  if (stages < 2) stages = 2;
  f.stages = stages;
  f.smem_bytes = static_cast<size_t>(stages) * f.stage_bytes + fixed + static_cast<size_t>(stages) * 8;
  f.kernel = select_pass1_shift(c->dtype, NR, WR);
  int per_sm = 0;
  if (f.smem_bytes > kPass1SmemCap || !set_smem_cap(f.kernel, kPass1SmemCap) ||
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, f.kernel, kThreads, f.smem_bytes) != cudaSuccess || per_sm < 1) {
    cudaGetLastError();
    return ADACONS_OK;
  }
  f.grid = per_sm * c->num_sms;
  if (f.grid > f.num_tiles) f.grid = f.num_tiles;
  f.available = true;
  return ADACONS_OK;
}

// The tensor maps of pass1_shift_kernel for a matrix at `grads`: rows c, c + k, c + 2k, ... (k = 16 / gcd(pitch in
// bytes, 16)) start at the same offset from a 16-byte boundary and are k * pitch apart, a legal stride.
int encode_shift_maps(adacons_ctx* c, const void* grads) {
  if (c->shift_maps_for == grads) return ADACONS_OK;
  const unsigned long long g0 = reinterpret_cast<unsigned long long>(grads);
  const unsigned long long row_bytes = static_cast<unsigned long long>(c->pitch) * c->elem_bytes;
  const unsigned rem = static_cast<unsigned>(row_bytes % 16);
  int k = 1;
  if (rem != 0) k = static_cast<int>(16u / (rem & (~rem + 1u)));      // gcd(rem, 16) is rem's lowest set bit
  c->shift_classes = k;
  int base_slot = 0;
  for (int cl = 0; cl < k; ++cl) {
    const int rows = cl < c->N ? (c->N - cl + k - 1) / k : 0;
    c->shift_class_base[cl] = base_slot;
    base_slot += rows;
    c->shift_class_shift[cl] = 0;
    if (rows == 0) continue;
    const unsigned long long a = g0 + static_cast<unsigned long long>(cl) * row_bytes + static_cast<unsigned long long>(c->shift_head) * c->elem_bytes;
    const unsigned shift = static_cast<unsigned>(a % 16);
    c->shift_class_shift[cl] = static_cast<int>(shift);
    const cuuint64_t dims[2] = {static_cast<cuuint64_t>(c->shift_body_cols) + shift / c->elem_bytes, static_cast<cuuint64_t>(rows)};
    const cuuint64_t strides[1] = {static_cast<cuuint64_t>(k) * row_bytes};
    const cuuint32_t box[2] = {static_cast<cuuint32_t>(kBoxRowBytes / c->elem_bytes), static_cast<cuuint32_t>(rows)};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = c->encode(&c->shift_maps.m[cl],
                                 c->dtype == ADACONS_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                                 2, reinterpret_cast<void*>(a - shift), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                 CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return ADACONS_ECUDA;
  }
  c->shift_maps_for = grads;
  return ADACONS_OK;
}

// N > 64 on the aligned path: needs d floats of scratch for the column sums.
int plan_big(adacons_ctx* c) {
  c->big_available = false;
  if (c->N <= kMaxFastN) return ADACONS_OK;
  if ((c->pitch * c->elem_bytes) % 16 != 0 || c->encode == nullptr || c->d > kChunkCols) return ADACONS_OK;
  const int tile_cols = kBoxRowBytes / c->elem_bytes;
  c->big_tiles = static_cast<int>((c->d + tile_cols - 1) / tile_cols);
  const uint32_t stage_bytes = 64u * kBoxRowBytes;
  const int vec = c->dtype == ADACONS_F32 ? 4 : 8;
  const size_t fixed = static_cast<size_t>(2) * 8 * 32 * vec * sizeof(float) + static_cast<size_t>(kWarps) * 8 * 2 * sizeof(float) +
                       static_cast<size_t>(2) * 8 * kThreads * sizeof(float);
  c->big_stages = 2;
  c->big_smem = static_cast<size_t>(c->big_stages) * stage_bytes + fixed + static_cast<size_t>(c->big_stages) * 8;
  const void* k = c->dtype == ADACONS_F32 ? reinterpret_cast<const void*>(&pass1_dot_kernel<0>)
                                          : reinterpret_cast<const void*>(&pass1_dot_kernel<1>);
  int per_sm = 0;
  if (c->big_smem > kPass1SmemCap || !set_smem_cap(k, kPass1SmemCap) ||
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, kThreads, c->big_smem) != cudaSuccess || per_sm < 1) {
    cudaGetLastError();
    return ADACONS_OK;
  }
  c->big_grid = per_sm * c->num_sms;
  if (c->big_grid > c->big_tiles) c->big_grid = c->big_tiles;
  const size_t need = static_cast<size_t>(c->big_tiles) * tile_cols * sizeof(float);
  if (need > c->colsum_bytes) {
    cudaFree(c->d_colsum);
    c->d_colsum = nullptr;
    c->colsum_bytes = 0;
    if (cudaMalloc(&c->d_colsum, need) != cudaSuccess) { cudaGetLastError(); return ADACONS_ENOMEM; }
    c->colsum_bytes = need;
  }
  if (cudaMemset(c->d_colsum, 0, c->colsum_bytes) != cudaSuccess) return ADACONS_ECUDA;
  c->big_available = true;
  return ADACONS_OK;
}

// 64 < N <= 256 on the aligned path, one block per tile (pass1_tall_kernel): tiles of 128 rows x 256 bytes
// (N <= 128); beyond, 256 rows x 256 bytes with 512 threads (one block per SM) or, on request
// (ADACONS_OPT_TALL_TILES = 2), 256 rows x 128 bytes with 256 threads.
struct TallVariant {
  const void* kernel;
  int threads, box_bytes, box_rows;
  size_t fixed_bytes, stage_bytes;
};
template <int DT, int LPR, int TH>
TallVariant tall_variant_of() {
  using C = P1H<DT, LPR, TH>;
  return TallVariant{reinterpret_cast<const void*>(&pass1_tall_kernel<DT, LPR, TH>), TH, C::kBoxRowBytesH, C::kRows,
                     C::kFixedBytes, C::kStageBytes};
}
TallVariant tall_variant(int dtype, int N, int opt) {
  const bool f32 = dtype == ADACONS_F32;
  if (N <= 128) return f32 ? tall_variant_of<0, 16, 256>() : tall_variant_of<1, 16, 256>();
  if (opt == 2) return f32 ? tall_variant_of<0, 8, 256>() : tall_variant_of<1, 8, 256>();
  return f32 ? tall_variant_of<0, 16, 512>() : tall_variant_of<1, 16, 512>();
}

int plan_tall(adacons_ctx* c) {
  c->tall_available = false;
  if (c->N <= kMaxFastN || c->N > 256) return ADACONS_OK;
  if ((c->pitch * c->elem_bytes) % 16 != 0 || c->encode == nullptr || c->d > kChunkCols) return ADACONS_OK;
  const TallVariant v = tall_variant(c->dtype, c->N, c->tall_tiles_opt);
  const int tile_cols = v.box_bytes / c->elem_bytes;
  c->tall_tiles = static_cast<int>((c->d + tile_cols - 1) / tile_cols);
  // 256 threads: two blocks per SM share its shared memory; 512 threads: one block has it all
  const size_t budget = v.threads == kThreads ? kPass1SmemBudget : 2 * kPass1SmemBudget;
  int stages = static_cast<int>((budget - v.fixed_bytes - 64) / v.stage_bytes);
  if (stages > 8) stages = 8;
  if (stages < 2) return ADACONS_OK;
  const size_t smem = stages * v.stage_bytes + v.fixed_bytes + static_cast<size_t>(stages) * 8;
  const size_t cap = v.threads == kThreads ? kPass1SmemCap : 2 * kPass1SmemCap;
  int per_sm = 0;
  if (smem > cap || !set_smem_cap(v.kernel, cap) ||
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, v.kernel, v.threads, smem) != cudaSuccess || per_sm < 1) {
    cudaGetLastError();
    return ADACONS_OK;
  }
  c->tall_stages = stages;
  c->tall_smem = smem;
  c->tall_grid = per_sm * c->num_sms;
  if (c->tall_grid > c->tall_tiles) c->tall_grid = c->tall_tiles;
  c->tmap_tall_for = nullptr;
  c->tall_available = true;
  return ADACONS_OK;
}

int encode_map_tall(adacons_ctx* c, const void* grads) {
  if (c->tmap_tall_for == grads) return ADACONS_OK;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(c->d), static_cast<cuuint64_t>(c->N)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(c->pitch) * c->elem_bytes};
  const TallVariant v = tall_variant(c->dtype, c->N, c->tall_tiles_opt);
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(v.box_bytes / c->elem_bytes), static_cast<cuuint32_t>(v.box_rows)};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = c->encode(&c->tmap_tall,
                               c->dtype == ADACONS_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                               2, const_cast<void*>(grads), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                               CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return ADACONS_ECUDA;
  c->tmap_tall_for = grads;
  return ADACONS_OK;
}

// 64 < N <= 512 on the aligned path: clusters of ceil(N / 64) blocks rounded up to 2, 4 or 8.
// Shares the tensor map (boxes of 64 rows) and the shared-memory carve-up of the N > 64 path.
// Opt-in (ADACONS_OPT_CLUSTER_PASS1): the blocks of a cluster meet at a barrier once per tile, and a
// block cannot prefetch past it, so pass 1 runs latency-bound.  Measured, pass 1 alone, bf16 unless
// noted: N = 128, d = 20 M: 1.47 ms against 1.51 ms for the two-read form (fp32, d = 10 M: 1.13
// against 1.47); N = 256, d = 8 M: 1.77 against 1.20; N = 512, d = 4 M: 4.22 against 1.22.

int plan_cluster(adacons_ctx* c) {
  c->cl_available = false;
  if (c->N <= kMaxFastN || c->N > 512) return ADACONS_OK;
  if ((c->pitch * c->elem_bytes) % 16 != 0 || c->encode == nullptr || c->d > kChunkCols) return ADACONS_OK;
  const int tile_cols = kBoxRowBytes / c->elem_bytes;
  c->cl_tiles = static_cast<int>((c->d + tile_cols - 1) / tile_cols);
  c->cl_size = c->N <= 128 ? 2 : c->N <= 256 ? 4 : 8;
  const uint32_t stage_bytes = 64u * kBoxRowBytes;
  const int vec = c->dtype == ADACONS_F32 ? 4 : 8;
  const size_t fixed = static_cast<size_t>(2) * 8 * 32 * vec * sizeof(float) + static_cast<size_t>(kWarps) * 8 * 2 * sizeof(float) +
                       static_cast<size_t>(2) * 8 * kThreads * sizeof(float);
  const size_t smem = 2 * static_cast<size_t>(stage_bytes) + fixed + 2 * 8;
  const void* k = c->dtype == ADACONS_F32 ? reinterpret_cast<const void*>(&pass1_cluster_kernel<0>)
                                          : reinterpret_cast<const void*>(&pass1_cluster_kernel<1>);
  if (smem > kPass1SmemCap || !set_smem_cap(k, kPass1SmemCap)) return ADACONS_OK;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(c->cl_size) * 8); cfg.blockDim = dim3(kThreads); cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = static_cast<unsigned>(c->cl_size); attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  int clusters = 0;
  if (cudaOccupancyMaxActiveClusters(&clusters, k, &cfg) != cudaSuccess || clusters < 1) { cudaGetLastError(); return ADACONS_OK; }
  if (clusters > c->cl_tiles) clusters = c->cl_tiles;
  c->cl_grid = clusters * c->cl_size;
  c->cl_smem = smem;
  c->cl_available = true;
  return ADACONS_OK;
}

// bf16 and N <= 64 on the aligned path: the Gram-matrix pass 1 (pass1_gram_kernel); shares tmap_big (64-row boxes).
int plan_gram(adacons_ctx* c) {
  c->gram_available = false;
  if (c->dtype != ADACONS_BF16 || c->N > kMaxFastN) return ADACONS_OK;
  if ((c->pitch * c->elem_bytes) % 16 != 0 || c->encode == nullptr || c->d > kChunkCols) return ADACONS_OK;
  c->gram_tiles = static_cast<int>((c->d + 255) / 256);
  c->gram_stages = 2;
  c->gram_smem = static_cast<size_t>(c->gram_stages) * kGramStageBytes + kGramSecondBytes + static_cast<size_t>(2 * c->gram_stages) * 8;
  const void* k = reinterpret_cast<const void*>(&pass1_gram_kernel);
  int per_sm = 0;
  if (c->gram_smem > kPass1SmemCap || !set_smem_cap(k, kPass1SmemCap) ||
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, kThreads, c->gram_smem) != cudaSuccess || per_sm < 1) {
    cudaGetLastError();
    return ADACONS_OK;
  }
  c->gram_grid = per_sm * c->num_sms;
  if (c->gram_grid > c->gram_tiles) c->gram_grid = c->gram_tiles;
  c->gram_available = true;
  return ADACONS_OK;
}

int encode_map_big(adacons_ctx* c, const void* grads) {
  if (c->tmap_big_for == grads) return ADACONS_OK;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(c->d), static_cast<cuuint64_t>(c->N)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(c->pitch) * c->elem_bytes};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(kBoxRowBytes / c->elem_bytes), 64u};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = c->encode(&c->tmap_big,
                               c->dtype == ADACONS_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                               2, const_cast<void*>(grads), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                               CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return ADACONS_ECUDA;
  c->tmap_big_for = grads;
  return ADACONS_OK;
}

int plan_fused(adacons_ctx* c) {
  c->fused_available = false;
  int coop = 0;
  if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, c->device) != cudaSuccess || !coop) {
    cudaGetLastError();
    return ADACONS_OK;
  }
  if ((c->pitch * c->elem_bytes) % 16 != 0) return ADACONS_OK;
  const long long num_vec = (c->d * c->elem_bytes + 15) / 16;
  long long grid = (num_vec + 63) / 64;
  if (grid > c->num_sms) grid = c->num_sms;
  if (grid < 1) grid = 1;
  const long long vpb = (num_vec + grid - 1) / grid;
  const size_t smem = static_cast<size_t>(c->N) * vpb * 16 + static_cast<size_t>(kFusedThreads / 32) * c->N * 2 * sizeof(float);
  if (smem > kFusedSmemCap) return ADACONS_OK;
  const void* k = c->dtype == ADACONS_F32 ? reinterpret_cast<const void*>(&fused_small_kernel<0>)
                                          : reinterpret_cast<const void*>(&fused_small_kernel<1>);
  int per_sm = 0;
  if (!set_smem_cap(k, kFusedSmemCap) ||
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, kFusedThreads, smem) != cudaSuccess) {
    cudaGetLastError();
    return ADACONS_OK;
  }
  if (per_sm < 1) return ADACONS_OK;
  c->fused_grid = static_cast<int>(grid);
  c->fused_vpb = static_cast<int>(vpb);
  c->fused_smem = smem;
  c->fused_available = true;
  return ADACONS_OK;
}

// The one-launch kernel shares pass 1's plan (tiles, ring, shared memory); it needs a cooperative
// launch of pass 1's grid and one column chunk.
int plan_mid(adacons_ctx* c) {
  c->mid_available = false;
  if (!c->fast.available || c->num_chunks != 1) return ADACONS_OK;
  int coop = 0;
  if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, c->device) != cudaSuccess || !coop) {
    cudaGetLastError();
    return ADACONS_OK;
  }
  const void* k = select_mid(c->dtype, c->fast.NR, c->fast.WR);
  // phase 2 re-uses the dynamic shared memory as a ring of stages of 8 boxes x min(N, 8) rows x 512 bytes
  const size_t stage2 = static_cast<size_t>(kWarps) * (c->N < kMidChunkRows ? c->N : kMidChunkRows) * kBoxRowBytes;
  const int stages2 = kMidStages2;
  size_t smem = c->fast.smem_bytes;
  if (smem < stages2 * stage2) smem = stages2 * stage2;
  const size_t work = (static_cast<size_t>(kMidPartCap) + 3 * kMaxFastN) * sizeof(double);   // the coefficient step's arrays
  if (smem < work) smem = work;
  int per_sm = 0;
  if (smem > kPass1SmemCap || !set_smem_cap(k, kPass1SmemCap) ||
      cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k, kThreads, smem) != cudaSuccess || per_sm < 1) {
    cudaGetLastError();
    return ADACONS_OK;
  }
  c->mid_stages2 = stages2;
  c->mid_smem = smem;
  c->tmap_mid2_for = nullptr;
  int grid = per_sm * c->num_sms;
  if (grid > c->fast.grid) grid = c->fast.grid;       // never more blocks than pass 1 would use (or than tiles)
  c->mid_grid = grid;
  c->mid_kernel = k;
  c->mid_available = true;
  return ADACONS_OK;
}

// Tensor map of column chunk `ch` (columns [ch * 2^30, ...)) of the matrix at `grads`.
int encode_chunk_map(const adacons_ctx* c, const void* grads, int ch, CUtensorMap* out) {
  const long long col0 = static_cast<long long>(ch) * kChunkCols;
  const long long cols = c->d - col0 < kChunkCols ? c->d - col0 : kChunkCols;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(c->N)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(c->pitch) * c->elem_bytes};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(kBoxRowBytes / c->elem_bytes), static_cast<cuuint32_t>(c->N)};
  const cuuint32_t estr[2] = {1, 1};
  void* base = const_cast<unsigned char*>(static_cast<const unsigned char*>(grads)) + col0 * c->elem_bytes;
  const CUresult r = c->encode(out, c->dtype == ADACONS_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                               2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                               CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? ADACONS_OK : ADACONS_ECUDA;
}

// Tensor map of the one-launch kernel's second phase: the same matrix, boxes of min(N, 8) rows.
int encode_map_mid2(adacons_ctx* c, const void* grads) {
  if (c->tmap_mid2_for == grads) return ADACONS_OK;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(c->d), static_cast<cuuint64_t>(c->N)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(c->pitch) * c->elem_bytes};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(kBoxRowBytes / c->elem_bytes),
                             static_cast<cuuint32_t>(c->N < kMidChunkRows ? c->N : kMidChunkRows)};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = c->encode(&c->tmap_mid2,
                               c->dtype == ADACONS_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                               2, const_cast<void*>(grads), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                               CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return ADACONS_ECUDA;
  c->tmap_mid2_for = grads;
  return ADACONS_OK;
}

// Tensor map of the aligned body: columns [head, d) of every row, starting on a 16-byte boundary.
int encode_map_body(adacons_ctx* c, const void* grads, int head) {
  if (c->tmap_body_for == grads) return ADACONS_OK;
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(c->d - head), static_cast<cuuint64_t>(c->N)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(c->pitch) * c->elem_bytes};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(kBoxRowBytes / c->elem_bytes), static_cast<cuuint32_t>(c->N)};
  const cuuint32_t estr[2] = {1, 1};
  void* base = const_cast<unsigned char*>(static_cast<const unsigned char*>(grads)) + static_cast<size_t>(head) * c->elem_bytes;
  const CUresult r = c->encode(&c->tmap_body, c->dtype == ADACONS_F32 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16,
                               2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                               CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return ADACONS_ECUDA;
  c->tmap_body_for = grads;
  return ADACONS_OK;
}

// All chunk maps of a context (its vector was sized when the plan was made).
int encode_map(adacons_ctx* c, const void* grads) {
  if (c->tmap_for == grads) return ADACONS_OK;
  for (int ch = 0; ch < c->num_chunks; ++ch) {
    const int rc = encode_chunk_map(c, grads, ch, &c->tmaps[static_cast<size_t>(ch)]);
    if (rc != ADACONS_OK) return rc;
  }
  c->tmap_for = grads;
  return ADACONS_OK;
}

bool launch_ok() { return cudaGetLastError() == cudaSuccess; }

struct DeviceGuard {   // make the context's device current for the duration of a call
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() {
    int cur = -1;
    if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
  }
};

int alloc_sets(adacons_ctx* c) {   // (re)allocate everything whose size depends on sets()
  cudaFree(c->coef); cudaFree(c->gamma_f32); cudaFree(c->m); cudaFree(c->z);
  c->coef = nullptr; c->gamma_f32 = nullptr; c->m = nullptr; c->z = nullptr;
  const size_t sets = static_cast<size_t>(c->sets());
  const size_t N = static_cast<size_t>(c->N);
  const size_t b_coef = 5 * sets * N * sizeof(double);
  const size_t b_gam = sets * N * sizeof(float);
  const size_t b_m = sets * N * sizeof(double);
  if (cudaMalloc(&c->coef, b_coef) != cudaSuccess || cudaMalloc(&c->gamma_f32, b_gam) != cudaSuccess ||
      cudaMalloc(&c->m, b_m) != cudaSuccess || cudaMalloc(&c->z, sets * sizeof(double)) != cudaSuccess) {
    cudaGetLastError();
    return ADACONS_ENOMEM;
  }
  if (cudaMemset(c->coef, 0, b_coef) != cudaSuccess || cudaMemset(c->gamma_f32, 0, b_gam) != cudaSuccess ||
      cudaMemset(c->m, 0, b_m) != cudaSuccess || cudaMemset(c->z, 0, sets * sizeof(double)) != cudaSuccess)
    return ADACONS_ECUDA;
  const size_t b_part = static_cast<size_t>(c->max_partials) * 2 * N * sizeof(float);
  c->scratch_bytes = b_part + b_coef + b_gam + b_m + sizeof(uint32_t) + sizeof(long long) + c->seg_bytes;
  return ADACONS_OK;
}

void free_seg_plan(adacons_ctx* c) {
  cudaFree(c->d_seg_off); cudaFree(c->d_blk_first_seg); cudaFree(c->d_blk_last_seg); cudaFree(c->d_rec_begin);
  cudaFree(c->d_rec_count); cudaFree(c->d_set_first_block); cudaFree(c->d_records); cudaFree(c->d_pass2_blk_seg);
  c->d_seg_off = nullptr; c->d_blk_first_seg = c->d_blk_last_seg = c->d_rec_begin = c->d_rec_count = nullptr;
  c->d_set_first_block = c->d_pass2_blk_seg = nullptr; c->d_records = nullptr;
  c->seg_bytes = 0;
  cudaGetLastError();
}

template <typename T>
int upload(T** dst, const std::vector<T>& src, size_t* bytes) {
  const size_t b = (src.empty() ? 1 : src.size()) * sizeof(T);
  if (cudaMalloc(dst, b) != cudaSuccess) { cudaGetLastError(); return ADACONS_ENOMEM; }
  if (!src.empty() && cudaMemcpy(*dst, src.data(), src.size() * sizeof(T), cudaMemcpyHostToDevice) != cudaSuccess) {
    cudaGetLastError();
    return ADACONS_ECUDA;
  }
  *bytes += b;
  return ADACONS_OK;
}

// Host plan of the per-segment mode: which block meets which segments, where each (set, block)
// partial record lives, and which segment each pass-2 block works in.
int build_seg_plan(adacons_ctx* c) {
  if (!c->fast.available || c->num_chunks != 1) return ADACONS_EALIGN;   // needs the TMA path: N <= 64, 16-byte row pitch, d <= 2^30
  free_seg_plan(c);
  const int S = c->num_segments;
  const std::vector<long long>& off = c->seg_offsets;
  auto seg_of = [&](long long col) {   // the (non-empty) segment that contains column `col`
    int lo = 0, hi = S;                // first index with off[idx] > col, minus one
    while (lo < hi) { const int mid = (lo + hi) / 2; if (off[mid + 1] > col) hi = mid; else lo = mid + 1; }
    return lo;
  };
  const int T = c->fast.num_tiles;
  int G = c->fast.grid < T ? c->fast.grid : T;
  const long long tilec = c->fast.tile_cols;
  std::vector<int> first(G), last(G), rec_begin(S, 0), rec_count(S, 0), set_first(S, 0);
  for (int b = 0; b < G; ++b) {
    const long long t0 = static_cast<long long>(b) * T / G, t1 = static_cast<long long>(b + 1) * T / G;
    const long long c0 = t0 * tilec, c1 = t1 * tilec < c->d ? t1 * tilec : c->d;
    first[b] = seg_of(c0);
    last[b] = seg_of(c1 - 1);
    for (int sgm = first[b]; sgm <= last[b]; ++sgm) {
      if (rec_count[sgm] == 0) set_first[sgm] = b;
      rec_count[sgm] += 1;
    }
  }
  int R = 0;
  for (int sgm = 0; sgm < S; ++sgm) { rec_begin[sgm] = R; R += rec_count[sgm]; }
  // pass 2: block bid owns the pairs of 16-byte groups [num_pairs - (bid+1)*P, num_pairs - bid*P), P = 256,
  // i.e. groups [2*(num_pairs - (bid+1)*P), 2*(num_pairs - bid*P)) clipped to [0, num_vec) -- both vectorised kernels
  const int vec = c->dtype == ADACONS_F32 ? 4 : 8;
  const long long num_vec = (c->d + vec - 1) / vec;
  const long long num_pairs = (num_vec + 1) / 2;
  const long long blocks2 = (num_pairs + kPass2BlockPairs - 1) / kPass2BlockPairs;
  std::vector<int> blk(static_cast<size_t>(2 * blocks2));   // per block: code, last segment
  for (long long bid = 0; bid < blocks2; ++bid) {
    long long vlo = 2 * (num_pairs - (bid + 1) * kPass2BlockPairs);
    if (vlo < 0) vlo = 0;
    long long vhi = 2 * (num_pairs - bid * kPass2BlockPairs) - 1;
    if (vhi > num_vec - 1) vhi = num_vec - 1;
    const long long chi = vhi * vec + vec - 1 < c->d - 1 ? vhi * vec + vec - 1 : c->d - 1;
    const int slo = seg_of(vlo * vec), shi = seg_of(chi);
    blk[static_cast<size_t>(2 * bid)] = slo == shi ? slo : -(slo + 1);
    blk[static_cast<size_t>(2 * bid + 1)] = shi;
  }
  size_t bytes = 0;
  int rc;
  if ((rc = upload(&c->d_seg_off, off, &bytes)) != ADACONS_OK) return rc;
  if ((rc = upload(&c->d_blk_first_seg, first, &bytes)) != ADACONS_OK) return rc;
  if ((rc = upload(&c->d_blk_last_seg, last, &bytes)) != ADACONS_OK) return rc;
  if ((rc = upload(&c->d_rec_begin, rec_begin, &bytes)) != ADACONS_OK) return rc;
  if ((rc = upload(&c->d_rec_count, rec_count, &bytes)) != ADACONS_OK) return rc;
  if ((rc = upload(&c->d_set_first_block, set_first, &bytes)) != ADACONS_OK) return rc;
  if ((rc = upload(&c->d_pass2_blk_seg, blk, &bytes)) != ADACONS_OK) return rc;
  const size_t rb = static_cast<size_t>(R > 0 ? R : 1) * 2 * c->N * sizeof(float);
  if (cudaMalloc(&c->d_records, rb) != cudaSuccess) { cudaGetLastError(); return ADACONS_ENOMEM; }
  if (cudaMemset(c->d_records, 0, rb) != cudaSuccess) return ADACONS_ECUDA;
  bytes += rb;
  c->seg_grid = G;
  c->seg_records = R;
  c->seg_bytes = bytes;
  c->seg_kernel = select_pass1_seg(c->dtype, c->fast.NR, c->fast.WR);
  if (!set_smem_cap(c->seg_kernel, kPass1SmemCap)) return ADACONS_ECUDA;
  return ADACONS_OK;
}

}  // namespace

extern "C" {

int adacons_version(void) { return 100; }

const char* adacons_strerror(int code) {
  switch (code) {
    case ADACONS_OK: return "success";
    case ADACONS_EINVAL: return "invalid argument";
    case ADACONS_EALIGN: return "misaligned buffer";
    case ADACONS_ENOMEM: return "out of memory";
    case ADACONS_ECUDA: return "CUDA call failed or no CUDA device";
    case ADACONS_EARCH: return "device is not compute capability 10.x (sm_100)";
    case ADACONS_ETIMEOUT: return "a bounded on-device wait expired";
    case ADACONS_ELIMIT: return "problem exceeds the fixed scratch of the allocation-free entry point (N > 64)";
    default: return "unknown error code";
  }
}

int adacons_create(adacons_ctx** out, int N, int64_t d, int dtype, const int64_t* seg_offsets, int num_segments) {
  if (out == nullptr) return ADACONS_EINVAL;
  *out = nullptr;
  if (N < 1 || N > kMaxN || d < 1 || d >= (1ll << 40)) return ADACONS_EINVAL;
  if (dtype != ADACONS_F32 && dtype != ADACONS_BF16) return ADACONS_EINVAL;
  if (num_segments < 0 || (num_segments > 0 && seg_offsets == nullptr)) return ADACONS_EINVAL;
  if (num_segments > 0) {
    if (seg_offsets[0] != 0 || seg_offsets[num_segments] != d) return ADACONS_EINVAL;
    for (int s = 0; s < num_segments; ++s)
      if (seg_offsets[s + 1] < seg_offsets[s]) return ADACONS_EINVAL;
  }
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return ADACONS_ECUDA; }
  int major = 0, sms = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
    cudaGetLastError();
    return ADACONS_ECUDA;
  }
  if (major != 10) return ADACONS_EARCH;
  int l2 = 0;
  if (cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev) != cudaSuccess) { cudaGetLastError(); l2 = 0; }

  adacons_ctx* c = new (std::nothrow) adacons_ctx();
  if (c == nullptr) return ADACONS_ENOMEM;
  c->N = N; c->d = d; c->pitch = d; c->dtype = dtype; c->elem_bytes = dtype == ADACONS_F32 ? 4 : 2;
  c->device = dev; c->num_sms = sms; c->l2_bytes = l2;
  if (num_segments > 0) {
    c->num_segments = num_segments;
    c->seg_offsets.assign(seg_offsets, seg_offsets + num_segments + 1);
  } else {
    c->num_segments = 1;
    c->seg_offsets = {0, static_cast<long long>(d)};
  }

  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
      qres == cudaDriverEntryPointSuccess)
    c->encode = reinterpret_cast<EncodeTiledFn>(fn);
  else
    cudaGetLastError();

  int rc = plan_fast(c);
  if (rc != ADACONS_OK) { delete c; return rc; }
  c->tmaps.resize(static_cast<size_t>(c->num_chunks));

  // generic path: always available
  c->generic_tiles = static_cast<int>((d + kThreads * 4 - 1) / (kThreads * 4));
  c->generic_smem = static_cast<size_t>(kWarps) * N * 2 * sizeof(float);
  if (!set_smem_cap(reinterpret_cast<const void*>(&pass1_generic_kernel<0>), kGenericSmemCap) ||
      !set_smem_cap(reinterpret_cast<const void*>(&pass1_generic_kernel<1>), kGenericSmemCap)) {
    delete c;
    return ADACONS_ECUDA;
  }
  c->generic_grid = sms * 4;
  if (c->generic_grid > c->generic_tiles) c->generic_grid = c->generic_tiles;
  c->max_partials = c->generic_grid;
  if (c->fast.available && c->fast.grid * c->num_chunks > c->max_partials) c->max_partials = c->fast.grid * c->num_chunks;
  plan_fused(c);
  if (c->fused_available && c->fused_grid > c->max_partials) c->max_partials = c->fused_grid;
  plan_mid(c);
  rc = plan_big(c);
  if (rc != ADACONS_OK) { adacons_destroy(c); return rc; }
  if (c->big_available && c->big_grid > c->max_partials) c->max_partials = c->big_grid;
  plan_cluster(c);
  if (c->cl_available && c->cl_grid / c->cl_size > c->max_partials) c->max_partials = c->cl_grid / c->cl_size;
  plan_gram(c);
  if (c->gram_available && c->gram_grid > c->max_partials) c->max_partials = c->gram_grid;
  plan_shift(c);
  if (c->shift.available && c->shift.grid > c->max_partials) c->max_partials = c->shift.grid;
  plan_tall(c);
  if (c->tall_available && c->tall_grid > c->max_partials) c->max_partials = c->tall_grid;

  if (cudaMalloc(&c->flags, sizeof(uint32_t)) != cudaSuccess || cudaMalloc(&c->step, sizeof(long long)) != cudaSuccess ||
      cudaMalloc(&c->d_barrier, 4 * sizeof(unsigned long long)) != cudaSuccess) {
    cudaGetLastError(); adacons_destroy(c); return ADACONS_ENOMEM;
  }
  if (cudaMemset(c->flags, 0, sizeof(uint32_t)) != cudaSuccess || cudaMemset(c->step, 0, sizeof(long long)) != cudaSuccess ||
      cudaMemset(c->d_barrier, 0, 4 * sizeof(unsigned long long)) != cudaSuccess) {
    adacons_destroy(c); return ADACONS_ECUDA;
  }
  c->max_partials += 1;                  // room for the record of the head columns (aligned-body path)
  const size_t b_part = static_cast<size_t>(c->max_partials) * 2 * N * sizeof(float);
  if (cudaMalloc(&c->partials, b_part) != cudaSuccess) { cudaGetLastError(); adacons_destroy(c); return ADACONS_ENOMEM; }
  if (cudaMemset(c->partials, 0, b_part) != cudaSuccess) { adacons_destroy(c); return ADACONS_ECUDA; }
  rc = alloc_sets(c);
  if (rc != ADACONS_OK) { adacons_destroy(c); return rc; }
  if (cudaDeviceSynchronize() != cudaSuccess) { adacons_destroy(c); return ADACONS_ECUDA; }
  *out = c;
  return ADACONS_OK;
}

int adacons_destroy(adacons_ctx* c) {
  if (c == nullptr) return ADACONS_OK;
  DeviceGuard g(c->device);
  cudaFree(c->partials); cudaFree(c->coef); cudaFree(c->gamma_f32); cudaFree(c->m); cudaFree(c->z);
  cudaFree(c->flags); cudaFree(c->step); cudaFree(c->staging); cudaFree(c->d_barrier); cudaFree(c->d_colsum);
  free_seg_plan(c);
  if (c->prof_ready)
    for (int s = 0; s < adacons_ctx::kProfSlots; ++s)
      for (int e = 0; e < 4; ++e) cudaEventDestroy(c->prof_ev[s][e]);
  cudaGetLastError();
  delete c;
  return ADACONS_OK;
}

}  // extern "C"

namespace {

// Which part of a step a call runs: all of it, or one half of the column-sharded form.
enum Phase { kWholeStep = 0, kStatisticsOnly = 1, kFromStatistics = 2 };

int run_step(adacons_ctx* c, const void* grads, void* out, void* cuda_stream, Phase phase, double* stats_out,
             const double* stats_in, int shards) {
  if (c == nullptr || grads == nullptr) return ADACONS_EINVAL;
  if (phase != kStatisticsOnly && out == nullptr) return ADACONS_EINVAL;
  if (phase == kStatisticsOnly && (stats_out == nullptr || reinterpret_cast<uintptr_t>(stats_out) % 8 != 0)) return ADACONS_EINVAL;
  if (phase == kFromStatistics && (stats_in == nullptr || shards < 1 || reinterpret_cast<uintptr_t>(stats_in) % 8 != 0)) return ADACONS_EINVAL;
  // an option change that ran out of memory half-way leaves the context without its buffers
  if (c->partials == nullptr || c->coef == nullptr || c->gamma_f32 == nullptr || c->m == nullptr || c->z == nullptr)
    return ADACONS_ENOMEM;
  // with padded rows the vector loads may touch the last row's padding too: the matrix is N * pitch elements
  const size_t gbytes = static_cast<size_t>(c->N) * c->pitch * c->elem_bytes;
  const size_t obytes = static_cast<size_t>(c->d) * c->elem_bytes;
  // the statistics half writes no result: `out` then only stands for "as aligned as grads"
  const uintptr_t g0 = reinterpret_cast<uintptr_t>(grads), o0 = phase == kStatisticsOnly ? g0 : reinterpret_cast<uintptr_t>(out);
  if (phase != kStatisticsOnly && o0 < g0 + gbytes && g0 < o0 + obytes) return ADACONS_EINVAL;   // out overlaps grads
  DeviceGuard guard(c->device);
  if (!guard.ok) return ADACONS_ECUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const bool pitch16 = (c->pitch * c->elem_bytes) % 16 == 0;
  const bool aligned = (g0 % 16 == 0) && (o0 % 16 == 0) && pitch16;
  const bool g_aligned = (g0 % 16 == 0) && pitch16;      // pass 1 only reads the matrix
  // rows that start off a 16-byte boundary, all by the same amount: `head` columns up to the boundary
  const int head = (pitch16 && g0 % 16 != 0 && g0 % c->elem_bytes == 0) ? static_cast<int>((16 - g0 % 16) / c->elem_bytes) : 0;
  const long long num_vec = (c->d * c->elem_bytes + 15) / 16;              // 16-byte column groups per row
  const int tail_elems = static_cast<int>((c->d * c->elem_bytes % 16) / c->elem_bytes);   // 0: the last group is full
  const long long row_bytes = c->pitch * c->elem_bytes;
  const int N = c->N;
  int num_partials = 0;
  int extra_launches = 0;
  cudaEvent_t* ev = (phase == kWholeStep && c->profile && c->prof_ready) ? c->prof_ev[c->prof_calls % adacons_ctx::kProfSlots] : nullptr;
  if (ev) cudaEventRecord(ev[0], st);

  // the coefficient kernel may be launched while pass 1 still runs (it waits for it on the device);
  // event records between the kernels would defeat that
  const bool pdl = (ev == nullptr) && c->overlap_launch && phase != kFromStatistics;
  const bool seg = c->per_segment != 0;
  if (seg && !(aligned && c->fast.available && c->seg_kernel != nullptr)) return ADACONS_EALIGN;

  // ---- single-pass path: the whole matrix fits in the grid's shared memory ----
  if (phase == kWholeStep && !seg && aligned && c->fused_available && c->fused_small) {
    FusedParams f;
    f.N = N; f.num_vec = num_vec; f.tail_elems = tail_elems; f.row_bytes = row_bytes; f.vec_per_block = c->fused_vpb;
    f.grads = static_cast<const unsigned char*>(grads); f.out = static_cast<unsigned char*>(out);
    f.barrier = c->d_barrier;
    CoeffParams& q = f.coeff;
    q.N = N; q.num_partials = c->fused_grid; q.sets = 1; q.beta = c->beta;
    q.momentum = c->momentum; q.sorted = c->sorted; q.normalize = c->normalize;
    q.partials = c->partials; q.rec_begin = nullptr; q.rec_count = nullptr; q.seg_off = nullptr;
    q.coef = c->coef; q.gamma_f32 = c->gamma_f32; q.m = c->m; q.z = c->z; q.flags = c->flags; q.step = c->step;
    const void* k = c->dtype == ADACONS_F32 ? reinterpret_cast<const void*>(&fused_small_kernel<0>)
                                            : reinterpret_cast<const void*>(&fused_small_kernel<1>);
    void* args[1] = {&f};
    if (cudaLaunchCooperativeKernel(k, dim3(c->fused_grid), dim3(kFusedThreads), args, c->fused_smem, st) != cudaSuccess) {
      cudaGetLastError();
      return ADACONS_ECUDA;
    }
    if (ev) { cudaEventRecord(ev[1], st); cudaEventRecord(ev[2], st); cudaEventRecord(ev[3], st); c->prof_calls += 1; }
    c->last_path = 3;
    c->last_pass2 = 0;
    c->last_launches = 1;
    c->total_launches += 1;
    return ADACONS_OK;
  }

  // ---- one launch, two reads: mid-size matrices ----
  if (phase == kWholeStep && !seg && aligned && c->mid_available &&
      (c->one_launch == 2 ||
       (c->one_launch == 1 && static_cast<long long>(c->N) * row_bytes <= kOneLaunchMaxBytes))) {
    int rc = encode_map(c, grads);
    if (rc == ADACONS_OK) rc = encode_map_mid2(c, grads);
    if (rc != ADACONS_OK) return rc;
    MidParams mp;
    mp.p1.N = N; mp.p1.num_tiles = c->fast.num_tiles; mp.p1.stages = c->fast.stages; mp.p1.stage_bytes = c->fast.stage_bytes;
    mp.p1.partials = c->partials; mp.p1.flags = c->flags;
    CoeffParams& q = mp.coeff;
    q.N = N; q.num_partials = c->mid_grid; q.sets = 1; q.beta = c->beta;
    q.momentum = c->momentum; q.sorted = c->sorted; q.normalize = c->normalize;
    q.partials = c->partials; q.rec_begin = nullptr; q.rec_count = nullptr; q.seg_off = nullptr;
    q.coef = c->coef; q.gamma_f32 = c->gamma_f32; q.m = c->m; q.z = c->z; q.flags = c->flags; q.step = c->step;
    mp.grads = static_cast<const unsigned char*>(grads); mp.out = static_cast<unsigned char*>(out);
    mp.row_bytes = row_bytes; mp.num_vec = num_vec; mp.tail_elems = tail_elems;
    mp.keep_in_l2 = static_cast<long long>(obytes) <= c->l2_bytes ? 1 : 0;
    mp.stages2 = c->mid_stages2;
    mp.sync = c->d_barrier + 1;
    void* args[3] = {&c->tmaps[0], &c->tmap_mid2, &mp};
    if (cudaLaunchCooperativeKernel(c->mid_kernel, dim3(c->mid_grid), dim3(kThreads), args, c->mid_smem, st) != cudaSuccess) {
      cudaGetLastError();
      return ADACONS_ECUDA;
    }
    if (ev) { cudaEventRecord(ev[1], st); cudaEventRecord(ev[2], st); cudaEventRecord(ev[3], st); c->prof_calls += 1; }
    c->last_path = 5;
    c->last_pass2 = 4;
    c->last_launches = 1;
    c->total_launches += 1;
    return ADACONS_OK;
  }

  // ---- pass 1 (Eq. 7) ----
  if (phase == kFromStatistics) {
    // the statistics come from the caller
  } else if (seg) {
    int rc = encode_map(c, grads);
    if (rc != ADACONS_OK) return rc;
    Pass1SegParams p;
    p.N = N; p.num_tiles = c->fast.num_tiles; p.stages = c->fast.stages; p.stage_bytes = c->fast.stage_bytes;
    p.d = c->d; p.seg_off = c->d_seg_off; p.blk_first_seg = c->d_blk_first_seg; p.blk_last_seg = c->d_blk_last_seg;
    p.rec_begin = c->d_rec_begin; p.set_first_block = c->d_set_first_block; p.records = c->d_records;
    p.flags = c->flags;
    void* args[2] = {&c->tmaps[0], &p};
    if (cudaLaunchKernel(c->seg_kernel, dim3(c->seg_grid), dim3(kThreads), args, c->fast.smem_bytes, st) != cudaSuccess) {
      cudaGetLastError();
      return ADACONS_ECUDA;
    }
    num_partials = 0;
    c->last_path = 1;
  } else if (g_aligned && c->gram_available && c->gram_fold > 0) {
    int rc = encode_map_big(c, grads);
    if (rc != ADACONS_OK) return rc;
    GramParams p;
    p.N = N; p.num_tiles = c->gram_tiles; p.stages = c->gram_stages; p.fold_tiles = c->gram_fold;
    p.partials = c->partials; p.flags = c->flags;
    void* args[2] = {&c->tmap_big, &p};
    if (cudaLaunchKernel(reinterpret_cast<const void*>(&pass1_gram_kernel), dim3(c->gram_grid), dim3(kThreads), args,
                         c->gram_smem, st) != cudaSuccess) {
      cudaGetLastError();
      return ADACONS_ECUDA;
    }
    num_partials = c->gram_grid;
    c->last_path = 9;
  } else if (g_aligned && c->fast.available) {
    int rc = encode_map(c, grads);
    if (rc != ADACONS_OK) return rc;
    for (int ch = 0; ch < c->num_chunks; ++ch) {      // one launch per column chunk of 2^30 (normally one)
      const long long col0 = static_cast<long long>(ch) * kChunkCols;
      const long long cols = c->d - col0 < kChunkCols ? c->d - col0 : kChunkCols;
      Pass1Params p;
      p.N = N; p.num_tiles = static_cast<int>((cols + c->fast.tile_cols - 1) / c->fast.tile_cols);
      p.stages = c->fast.stages; p.stage_bytes = c->fast.stage_bytes;
      p.partials = c->partials + static_cast<size_t>(ch) * c->fast.grid * 2 * N; p.flags = c->flags;
      void* args[2] = {&c->tmaps[static_cast<size_t>(ch)], &p};
      if (cudaLaunchKernel(c->fast.kernel, dim3(c->fast.grid), dim3(kThreads), args, c->fast.smem_bytes, st) != cudaSuccess) {
        cudaGetLastError();
        return ADACONS_ECUDA;
      }
      if (ch > 0) extra_launches += 1;
    }
    num_partials = c->fast.grid * c->num_chunks;
    c->last_path = 1;
  } else if (head > 0 && c->aligned_body && c->fast.available && c->num_chunks == 1 && c->d > head) {
    // the TMA-staged kernel on the aligned body, the head columns as one more partial record
    int rc = encode_map_body(c, grads, head);
    if (rc != ADACONS_OK) return rc;
    Pass1Params p;
    p.N = N; p.num_tiles = static_cast<int>((c->d - head + c->fast.tile_cols - 1) / c->fast.tile_cols);
    p.stages = c->fast.stages; p.stage_bytes = c->fast.stage_bytes; p.partials = c->partials; p.flags = c->flags;
    void* args[2] = {&c->tmap_body, &p};
    if (cudaLaunchKernel(c->fast.kernel, dim3(c->fast.grid), dim3(kThreads), args, c->fast.smem_bytes, st) != cudaSuccess) {
      cudaGetLastError();
      return ADACONS_ECUDA;
    }
    float* rec = c->partials + static_cast<size_t>(c->fast.grid) * 2 * N;
    if (c->dtype == ADACONS_F32) edge_stats_kernel<0><<<1, kThreads, 0, st>>>(grads, N, c->d, c->pitch, head, 0, rec);
    else edge_stats_kernel<1><<<1, kThreads, 0, st>>>(grads, N, c->d, c->pitch, head, 0, rec);
    if (!launch_ok()) return ADACONS_ECUDA;
    extra_launches += 1;
    num_partials = c->fast.grid + 1;
    c->last_path = 8;
  } else if (g_aligned && c->tall_available && c->tall_tiles_opt && !c->cluster_pass1) {
    int rc = encode_map_tall(c, grads);
    if (rc != ADACONS_OK) return rc;
    Pass1Params p;
    const TallVariant v = tall_variant(c->dtype, N, c->tall_tiles_opt);
    p.N = N; p.num_tiles = c->tall_tiles; p.stages = c->tall_stages; p.stage_bytes = static_cast<uint32_t>(v.stage_bytes);
    p.partials = c->partials; p.flags = c->flags;
    void* args[2] = {&c->tmap_tall, &p};
    if (cudaLaunchKernel(v.kernel, dim3(c->tall_grid), dim3(v.threads), args, c->tall_smem, st) != cudaSuccess) {
      cudaGetLastError();
      return ADACONS_ECUDA;
    }
    num_partials = c->tall_grid;
    c->last_path = 7;
  } else if (g_aligned && c->cl_available && c->cluster_pass1) {
    int rc = encode_map_big(c, grads);
    if (rc != ADACONS_OK) return rc;
    Pass1ClusterParams p;
    p.N = N; p.num_tiles = c->cl_tiles; p.stages = 2; p.stage_bytes = 64u * kBoxRowBytes;
    p.partials = c->partials; p.flags = c->flags;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(c->cl_grid)); cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = c->cl_smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = static_cast<unsigned>(c->cl_size); attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    const cudaError_t e1 = c->dtype == ADACONS_F32 ? cudaLaunchKernelEx(&cfg, pass1_cluster_kernel<0>, c->tmap_big, p)
                                                   : cudaLaunchKernelEx(&cfg, pass1_cluster_kernel<1>, c->tmap_big, p);
    if (e1 != cudaSuccess) { cudaGetLastError(); return ADACONS_ECUDA; }
    num_partials = c->cl_grid / c->cl_size;
    c->last_path = 6;
  } else if (g_aligned && c->big_available) {
    int rc = encode_map_big(c, grads);
    if (rc != ADACONS_OK) return rc;
    const unsigned cblocks = static_cast<unsigned>((num_vec + kThreads - 1) / kThreads);
    const unsigned char* g8 = static_cast<const unsigned char*>(grads);
    if (c->dtype == ADACONS_F32) colsum_kernel<0><<<cblocks, kThreads, 0, st>>>(g8, c->d_colsum, N, row_bytes, num_vec, tail_elems);
    else colsum_kernel<1><<<cblocks, kThreads, 0, st>>>(g8, c->d_colsum, N, row_bytes, num_vec, tail_elems);
    if (!launch_ok()) return ADACONS_ECUDA;
    const void* k = c->dtype == ADACONS_F32 ? reinterpret_cast<const void*>(&pass1_dot_kernel<0>)
                                            : reinterpret_cast<const void*>(&pass1_dot_kernel<1>);
    for (int r0 = 0; r0 < N; r0 += 64) {
      Pass1DotParams p;
      p.N = N; p.r0 = r0; p.rows = N - r0 < 64 ? N - r0 : 64; p.num_tiles = c->big_tiles; p.stages = c->big_stages;
      p.stage_bytes = 64u * kBoxRowBytes; p.s = c->d_colsum; p.partials = c->partials; p.flags = c->flags;
      void* args[2] = {&c->tmap_big, &p};
      if (cudaLaunchKernel(k, dim3(c->big_grid), dim3(kThreads), args, c->big_smem, st) != cudaSuccess) {
        cudaGetLastError();
        return ADACONS_ECUDA;
      }
      extra_launches += 1;
    }
    num_partials = c->big_grid;
    c->last_path = 4;
  } else if (c->shifted_loads && c->shift.available && g0 % c->elem_bytes == 0) {
    // rows at arbitrary element offsets: a tensor map per class of equally offset rows, shifted into place in
    // registers; head and tail columns as one more record
    int rc = encode_shift_maps(c, grads);
    if (rc != ADACONS_OK) return rc;
    Pass1ShiftParams p;
    p.N = N; p.num_tiles = c->shift.num_tiles; p.stages = c->shift.stages; p.stage_bytes = c->shift.stage_bytes;
    p.classes = c->shift_classes;
    for (int cl = 0; cl < kShiftMaxClasses; ++cl) { p.class_base[cl] = c->shift_class_base[cl]; p.class_shift[cl] = c->shift_class_shift[cl]; }
    p.partials = c->partials; p.flags = c->flags;
    void* args[2] = {&c->shift_maps, &p};
    if (cudaLaunchKernel(c->shift.kernel, dim3(c->shift.grid), dim3(kThreads), args, c->shift.smem_bytes, st) != cudaSuccess) {
      cudaGetLastError();
      return ADACONS_ECUDA;
    }
    float* rec = c->partials + static_cast<size_t>(c->shift.grid) * 2 * N;
    if (c->dtype == ADACONS_F32) edge_stats_kernel<0><<<1, kThreads, 0, st>>>(grads, N, c->d, c->pitch, c->shift_head, c->shift_tail, rec);
    else edge_stats_kernel<1><<<1, kThreads, 0, st>>>(grads, N, c->d, c->pitch, c->shift_head, c->shift_tail, rec);
    if (!launch_ok()) return ADACONS_ECUDA;
    extra_launches += 1;
    num_partials = c->shift.grid + 1;
    c->last_path = 10;
  } else {
    if (c->dtype == ADACONS_F32)
      pass1_generic_kernel<0><<<c->generic_grid, kThreads, c->generic_smem, st>>>(grads, N, c->d, c->pitch, c->generic_tiles, c->partials);
    else
      pass1_generic_kernel<1><<<c->generic_grid, kThreads, c->generic_smem, st>>>(grads, N, c->d, c->pitch, c->generic_tiles, c->partials);
    if (!launch_ok()) return ADACONS_ECUDA;
    num_partials = c->generic_grid;
    c->last_path = 2;
  }
  if (ev) cudaEventRecord(ev[1], st);

  // ---- coefficients (Eq. 11, Eq. 12-13) ----
  CoeffParams q;
  q.N = N; q.num_partials = num_partials; q.sets = c->sets(); q.beta = c->beta;
  q.momentum = c->momentum; q.sorted = c->sorted; q.normalize = c->normalize;
  q.partials = seg ? c->d_records : c->partials;
  q.rec_begin = seg ? c->d_rec_begin : nullptr;
  q.rec_count = seg ? c->d_rec_count : nullptr;
  q.seg_off = seg ? c->d_seg_off : nullptr;
  q.coef = c->coef; q.gamma_f32 = c->gamma_f32; q.m = c->m; q.z = c->z;
  q.flags = c->flags; q.step = c->step;
  q.cols = c->d;
  if (phase == kStatisticsOnly) q.stats_out = stats_out;
  if (phase == kFromStatistics) { q.stats_in = stats_in; q.shards = shards; }
  int cthreads = 1024;
  if (seg) { cthreads = ((2 * N + 31) / 32) * 32; if (cthreads > 1024) cthreads = 1024; }
  if (launch_kernel(coeff_kernel, dim3(c->sets()), dim3(cthreads), 0, st, pdl, q) != cudaSuccess) {
    cudaGetLastError();
    return ADACONS_ECUDA;
  }
  if (ev) cudaEventRecord(ev[2], st);
  if (phase == kStatisticsOnly) {
    c->last_launches = 2 + extra_launches;
    c->total_launches += c->last_launches;
    return ADACONS_OK;
  }

  // ---- pass 2 (Eq. 12) ----
  cudaError_t e2;
  if (aligned) {
    const long long num_pairs = (num_vec + 1) / 2;
    const unsigned blocks = static_cast<unsigned>((num_pairs + kPass2BlockPairs - 1) / kPass2BlockPairs);
    const unsigned char* g8 = static_cast<const unsigned char*>(grads);
    unsigned char* o8 = static_cast<unsigned char*>(out);
    const int* bs = c->d_pass2_blk_seg;
    const long long* so = c->d_seg_off;
    // 32-byte aligned buffers and pitch: one 256-bit load and store per thread and row
    const bool wide = (g0 % 32 == 0) && (o0 % 32 == 0) && (row_bytes % 32 == 0);
    // a result that fits in L2 is kept there (evict_last stores); a larger one is written plainly
    const int keep = static_cast<long long>(obytes) <= c->l2_bytes ? 1 : 0;
#define ADACONS_LAUNCH_PASS2(KERNEL) \
    launch_kernel(KERNEL, dim3(blocks), dim3(kThreads), 0, st, false, g8, o8, c->gamma_f32, N, row_bytes, num_vec, bs, so, tail_elems)
#define ADACONS_LAUNCH_PASS2W(KERNEL) \
    launch_kernel(KERNEL, dim3(blocks), dim3(kThreads), 0, st, false, g8, o8, c->gamma_f32, N, row_bytes, num_vec, bs, so, tail_elems, keep)
    if (c->dtype == ADACONS_F32) {
      if (wide) e2 = seg ? ADACONS_LAUNCH_PASS2W((pass2_wide_kernel<0, true>)) : ADACONS_LAUNCH_PASS2W((pass2_wide_kernel<0, false>));
      else e2 = seg ? ADACONS_LAUNCH_PASS2((pass2_vec_kernel<0, true>)) : ADACONS_LAUNCH_PASS2((pass2_vec_kernel<0, false>));
    } else {
      if (wide) e2 = seg ? ADACONS_LAUNCH_PASS2W((pass2_wide_kernel<1, true>)) : ADACONS_LAUNCH_PASS2W((pass2_wide_kernel<1, false>));
      else e2 = seg ? ADACONS_LAUNCH_PASS2((pass2_vec_kernel<1, true>)) : ADACONS_LAUNCH_PASS2((pass2_vec_kernel<1, false>));
    }
#undef ADACONS_LAUNCH_PASS2
#undef ADACONS_LAUNCH_PASS2W
    c->last_pass2 = wide ? 3 : 2;
  } else if (!seg && head > 0 && c->aligned_body && (o0 % 16 == g0 % 16) && c->d > head) {
    // grads and out start off a 16-byte boundary by the same amount: the vector kernels on the whole
    // 16-byte groups of the aligned body, the head and the ragged tail element by element
    const int vec = 16 / c->elem_bytes;
    const long long body = c->d - head;
    const long long nv = body / vec;                                    // whole groups only
    const int tail = static_cast<int>(body - nv * vec);
    const unsigned char* g8 = static_cast<const unsigned char*>(grads) + static_cast<size_t>(head) * c->elem_bytes;
    unsigned char* o8 = static_cast<unsigned char*>(out) + static_cast<size_t>(head) * c->elem_bytes;
    e2 = cudaSuccess;
    if (nv > 0) {
      const long long np2 = (nv + 1) / 2;
      const unsigned blocks = static_cast<unsigned>((np2 + kPass2BlockPairs - 1) / kPass2BlockPairs);
      const bool wide = (reinterpret_cast<uintptr_t>(g8) % 32 == 0) && (reinterpret_cast<uintptr_t>(o8) % 32 == 0) && (row_bytes % 32 == 0);
      const int keep = static_cast<long long>(obytes) <= c->l2_bytes ? 1 : 0;
      const int* nobs = nullptr; const long long* noso = nullptr;
      if (c->dtype == ADACONS_F32)
        e2 = wide ? launch_kernel(pass2_wide_kernel<0, false>, dim3(blocks), dim3(kThreads), 0, st, false, g8, o8, c->gamma_f32, N, row_bytes, nv, nobs, noso, 0, keep)
                  : launch_kernel(pass2_vec_kernel<0, false>, dim3(blocks), dim3(kThreads), 0, st, false, g8, o8, c->gamma_f32, N, row_bytes, nv, nobs, noso, 0);
      else
        e2 = wide ? launch_kernel(pass2_wide_kernel<1, false>, dim3(blocks), dim3(kThreads), 0, st, false, g8, o8, c->gamma_f32, N, row_bytes, nv, nobs, noso, 0, keep)
                  : launch_kernel(pass2_vec_kernel<1, false>, dim3(blocks), dim3(kThreads), 0, st, false, g8, o8, c->gamma_f32, N, row_bytes, nv, nobs, noso, 0);
    }
    if (e2 == cudaSuccess) {
      if (c->dtype == ADACONS_F32) edge_combine_kernel<0><<<1, 32, 0, st>>>(grads, out, c->gamma_f32, N, c->d, c->pitch, head, tail);
      else edge_combine_kernel<1><<<1, 32, 0, st>>>(grads, out, c->gamma_f32, N, c->d, c->pitch, head, tail);
      e2 = cudaGetLastError();
      extra_launches += (nv > 0) ? 1 : 0;
    }
    c->last_pass2 = 5;
  } else if (!seg && c->shifted_loads && g0 % c->elem_bytes == 0 && o0 % c->elem_bytes == 0 && c->d >= 4 * (16 / c->elem_bytes)) {
    // rows (or out) at any element offset: 16-byte groups of out, each row's bytes realigned in registers
    const int vec = 16 / c->elem_bytes;
    const int head = static_cast<int>(((16 - o0 % 16) % 16) / c->elem_bytes) + vec;        // vec .. 2 vec - 1 columns
    const long long groups = (c->d - 2 * vec - head) / vec + 1;                             // >= 1; the last one ends 2 vec columns before d at the latest
    const int tail = static_cast<int>(c->d - head - groups * vec);                          // vec .. 2 vec - 1 columns
    const unsigned char* g8 = static_cast<const unsigned char*>(grads);
    unsigned char* o8 = static_cast<unsigned char*>(out) + static_cast<size_t>(head) * c->elem_bytes;
    const long long body_off = static_cast<long long>(head) * c->elem_bytes;
    const unsigned blocks = static_cast<unsigned>((groups + kThreads - 1) / kThreads);
    if (c->dtype == ADACONS_F32)
      e2 = launch_kernel(pass2_shift_kernel<0>, dim3(blocks), dim3(kThreads), 0, st, false, g8, o8, c->gamma_f32, N, row_bytes, body_off, groups);
    else
      e2 = launch_kernel(pass2_shift_kernel<1>, dim3(blocks), dim3(kThreads), 0, st, false, g8, o8, c->gamma_f32, N, row_bytes, body_off, groups);
    if (e2 == cudaSuccess) {
      if (c->dtype == ADACONS_F32) edge_combine_kernel<0><<<1, 32, 0, st>>>(grads, out, c->gamma_f32, N, c->d, c->pitch, head, tail);
      else edge_combine_kernel<1><<<1, 32, 0, st>>>(grads, out, c->gamma_f32, N, c->d, c->pitch, head, tail);
      e2 = cudaGetLastError();
      extra_launches += 1;
    }
    c->last_pass2 = 6;
  } else {
    const unsigned blocks = static_cast<unsigned>((c->d + kThreads - 1) / kThreads);
    if (c->dtype == ADACONS_F32)
      e2 = launch_kernel(pass2_generic_kernel<0>, dim3(blocks), dim3(kThreads), 0, st, false, grads, out, c->gamma_f32, N, c->d, c->pitch);
    else
      e2 = launch_kernel(pass2_generic_kernel<1>, dim3(blocks), dim3(kThreads), 0, st, false, grads, out, c->gamma_f32, N, c->d, c->pitch);
    c->last_pass2 = 1;
  }
  if (e2 != cudaSuccess) { cudaGetLastError(); return ADACONS_ECUDA; }
  if (ev) { cudaEventRecord(ev[3], st); c->prof_calls += 1; }
  c->last_launches = (phase == kFromStatistics ? 2 : 3) + extra_launches;
  c->total_launches += c->last_launches;
  return ADACONS_OK;
}

}  // namespace

extern "C" {

int adacons_aggregate(adacons_ctx* c, const void* grads, void* out, void* cuda_stream) {
  return run_step(c, grads, out, cuda_stream, kWholeStep, nullptr, nullptr, 0);
}

int adacons_pass1(adacons_ctx* c, const void* grads, double* stats, void* cuda_stream) {
  return run_step(c, grads, nullptr, cuda_stream, kStatisticsOnly, stats, nullptr, 0);
}

int adacons_finish(adacons_ctx* c, const void* grads, void* out, const double* stats, int shards, void* cuda_stream) {
  return run_step(c, grads, out, cuda_stream, kFromStatistics, nullptr, stats, shards);
}

int adacons_aggregate_host(adacons_ctx* c, const void* host_grads, void* host_out, void* cuda_stream) {
  if (c == nullptr || host_grads == nullptr || host_out == nullptr) return ADACONS_EINVAL;
  DeviceGuard guard(c->device);
  if (!guard.ok) return ADACONS_ECUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t gbytes = (static_cast<size_t>(c->N - 1) * c->pitch + c->d) * c->elem_bytes;
  const size_t obytes = static_cast<size_t>(c->d) * c->elem_bytes;
  const size_t gpad = (static_cast<size_t>(c->N) * c->pitch * c->elem_bytes + 255) / 256 * 256;
  if (c->staging != nullptr && c->staging_bytes < gpad + obytes) {
    cudaFree(c->staging);
    c->staging = nullptr;
    c->scratch_bytes -= c->staging_bytes;
  }
  if (c->staging == nullptr) {
    if (cudaMalloc(&c->staging, gpad + obytes) != cudaSuccess) { cudaGetLastError(); return ADACONS_ENOMEM; }
    c->staging_bytes = gpad + obytes;
    c->scratch_bytes += gpad + obytes;
  }
  unsigned char* dg = static_cast<unsigned char*>(c->staging);
  unsigned char* dout = dg + gpad;
  if (cudaMemcpyAsync(dg, host_grads, gbytes, cudaMemcpyHostToDevice, st) != cudaSuccess) { cudaGetLastError(); return ADACONS_ECUDA; }
  const int rc = adacons_aggregate(c, dg, dout, cuda_stream);
  if (rc != ADACONS_OK) return rc;
  if (cudaMemcpyAsync(host_out, dout, obytes, cudaMemcpyDeviceToHost, st) != cudaSuccess) { cudaGetLastError(); return ADACONS_ECUDA; }
  if (cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return ADACONS_ECUDA; }
  return ADACONS_OK;
}

int adacons_reset(adacons_ctx* c, void* cuda_stream) {
  if (c == nullptr) return ADACONS_EINVAL;
  if (c->m == nullptr) return ADACONS_ENOMEM;
  DeviceGuard guard(c->device);
  if (!guard.ok) return ADACONS_ECUDA;
  const long long n = static_cast<long long>(c->sets()) * c->N;
  reset_kernel<<<static_cast<unsigned>((n + 255) / 256 < 1024 ? (n + 255) / 256 : 1024), 256, 0,
                 static_cast<cudaStream_t>(cuda_stream)>>>(c->m, n, c->flags, c->step, c->d_barrier);
  if (!launch_ok()) return ADACONS_ECUDA;
  c->total_launches += 1;
  return ADACONS_OK;
}

int adacons_set_option(adacons_ctx* c, int key, double value) {
  if (c == nullptr) return ADACONS_EINVAL;
  switch (key) {
    case ADACONS_OPT_BETA:
      if (!(value >= 0.0 && value < 1.0)) return ADACONS_EINVAL;
      c->beta = value; return ADACONS_OK;
    case ADACONS_OPT_MOMENTUM: c->momentum = value != 0.0; return ADACONS_OK;
    case ADACONS_OPT_SORTED: c->sorted = value != 0.0; return ADACONS_OK;
    case ADACONS_OPT_NORMALIZE: c->normalize = value != 0.0; return ADACONS_OK;
    case ADACONS_OPT_PER_SEGMENT: {
      const int want = value != 0.0;
      if (want == c->per_segment) return ADACONS_OK;
      DeviceGuard guard(c->device);
      if (!guard.ok) return ADACONS_ECUDA;
      if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return ADACONS_ECUDA; }
      if (want) {
        const int rc = build_seg_plan(c);
        if (rc != ADACONS_OK) { free_seg_plan(c); return rc; }
      } else {
        free_seg_plan(c);
      }
      c->per_segment = want;
      int rc = alloc_sets(c);                      // state, coefficients: one set per segment; zeroed
      if (rc != ADACONS_OK) return rc;
      if (cudaMemset(c->flags, 0, sizeof(uint32_t)) != cudaSuccess || cudaMemset(c->step, 0, sizeof(long long)) != cudaSuccess)
        return ADACONS_ECUDA;
      return ADACONS_OK;
    }
    case ADACONS_OPT_OVERLAP_LAUNCH: c->overlap_launch = value != 0.0; return ADACONS_OK;
    case ADACONS_OPT_FUSED_SMALL: c->fused_small = value != 0.0; return ADACONS_OK;
    case ADACONS_OPT_CLUSTER_PASS1: c->cluster_pass1 = value != 0.0; return ADACONS_OK;
    case ADACONS_OPT_GRAM_PASS1:
      if (value < 0.0 || value > 32.0 || value != static_cast<double>(static_cast<int>(value))) return ADACONS_EINVAL;
      c->gram_fold = static_cast<int>(value);
      return ADACONS_OK;
    case ADACONS_OPT_TALL_TILES: {
      if (value != 0.0 && value != 1.0 && value != 2.0) return ADACONS_EINVAL;
      const int before = c->tall_tiles_opt;
      c->tall_tiles_opt = static_cast<int>(value);
      if (c->tall_tiles_opt != 0 && before != 0 && c->tall_tiles_opt != before && c->N > 128) {   // another tile shape
        DeviceGuard guard(c->device);
        if (!guard.ok) return ADACONS_ECUDA;
        plan_tall(c);
        if (c->tall_available && c->tall_grid > c->max_partials) { c->tall_tiles_opt = before; plan_tall(c); return ADACONS_ENOMEM; }
      }
      return ADACONS_OK;
    }
    case ADACONS_OPT_ALIGNED_BODY: c->aligned_body = value != 0.0; return ADACONS_OK;
    case ADACONS_OPT_SHIFTED_LOADS: c->shifted_loads = value != 0.0; return ADACONS_OK;
    case ADACONS_OPT_ONE_LAUNCH:
      if (value != 0.0 && value != 1.0 && value != 2.0) return ADACONS_EINVAL;
      c->one_launch = static_cast<int>(value); return ADACONS_OK;
    case ADACONS_OPT_ROW_PITCH: {
      const long long pitch = static_cast<long long>(value);
      if (static_cast<double>(pitch) != value || pitch < c->d || pitch >= (1ll << 40)) return ADACONS_EINVAL;
      if (pitch == c->pitch) return ADACONS_OK;
      DeviceGuard guard(c->device);
      if (!guard.ok) return ADACONS_ECUDA;
      if (cudaDeviceSynchronize() != cudaSuccess) { cudaGetLastError(); return ADACONS_ECUDA; }
      c->pitch = pitch;
      c->tmap_for = nullptr;
      c->tmap_mid2_for = nullptr;
      c->tmap_tall_for = nullptr;
      c->tmap_body_for = nullptr;
      int rc = plan_fast(c);
      if (rc != ADACONS_OK) return rc;
      c->tmaps.resize(static_cast<size_t>(c->num_chunks));
      plan_fused(c);
      plan_mid(c);
      // the grid barrier and the ticket counter count in units of a plan's grid: start them afresh
      if (cudaMemset(c->d_barrier, 0, 4 * sizeof(unsigned long long)) != cudaSuccess) return ADACONS_ECUDA;
      c->tmap_big_for = nullptr;
      rc = plan_big(c);
      if (rc != ADACONS_OK) return rc;
      plan_cluster(c);
      plan_tall(c);
      plan_gram(c);
      plan_shift(c);
      int need = c->generic_grid;
      if (c->fast.available && c->fast.grid * c->num_chunks > need) need = c->fast.grid * c->num_chunks;
      if (c->fused_available && c->fused_grid > need) need = c->fused_grid;
      if (c->big_available && c->big_grid > need) need = c->big_grid;
      if (c->cl_available && c->cl_grid / c->cl_size > need) need = c->cl_grid / c->cl_size;
      if (c->tall_available && c->tall_grid > need) need = c->tall_grid;
      if (c->gram_available && c->gram_grid > need) need = c->gram_grid;
      if (c->shift.available && c->shift.grid > need) need = c->shift.grid;
      need += 1;                             // the head columns' record (aligned-body path)
      if (need > c->max_partials) {          // the other paths may use more blocks than the old plan
        cudaFree(c->partials);
        c->partials = nullptr;
        c->max_partials = need;
        const size_t b_part = static_cast<size_t>(need) * 2 * c->N * sizeof(float);
        if (cudaMalloc(&c->partials, b_part) != cudaSuccess) { cudaGetLastError(); return ADACONS_ENOMEM; }
        if (cudaMemset(c->partials, 0, b_part) != cudaSuccess) return ADACONS_ECUDA;
      }
      if (c->per_segment) {
        rc = build_seg_plan(c);
        if (rc != ADACONS_OK) { free_seg_plan(c); c->per_segment = 0; alloc_sets(c); return rc; }
      }
      return ADACONS_OK;
    }
    case ADACONS_OPT_PROFILE: {
      DeviceGuard guard(c->device);
      if (!guard.ok) return ADACONS_ECUDA;
      if (value != 0.0 && !c->prof_ready) {
        for (int s = 0; s < adacons_ctx::kProfSlots; ++s)
          for (int e = 0; e < 4; ++e)
            if (cudaEventCreate(&c->prof_ev[s][e]) != cudaSuccess) { cudaGetLastError(); return ADACONS_ECUDA; }
        c->prof_ready = true;
      }
      c->profile = value != 0.0;
      c->prof_calls = 0;
      return ADACONS_OK;
    }
    default: return ADACONS_EINVAL;
  }
}

int adacons_get_option(adacons_ctx* c, int key, double* value) {
  if (c == nullptr || value == nullptr) return ADACONS_EINVAL;
  switch (key) {
    case ADACONS_OPT_BETA: *value = c->beta; return ADACONS_OK;
    case ADACONS_OPT_MOMENTUM: *value = c->momentum; return ADACONS_OK;
    case ADACONS_OPT_SORTED: *value = c->sorted; return ADACONS_OK;
    case ADACONS_OPT_NORMALIZE: *value = c->normalize; return ADACONS_OK;
    case ADACONS_OPT_PER_SEGMENT: *value = c->per_segment; return ADACONS_OK;
    case ADACONS_OPT_PROFILE: *value = c->profile; return ADACONS_OK;
    case ADACONS_OPT_OVERLAP_LAUNCH: *value = c->overlap_launch; return ADACONS_OK;
    case ADACONS_OPT_FUSED_SMALL: *value = c->fused_small; return ADACONS_OK;
    case ADACONS_OPT_ONE_LAUNCH: *value = c->one_launch; return ADACONS_OK;
    case ADACONS_OPT_TALL_TILES: *value = c->tall_tiles_opt; return ADACONS_OK;
    case ADACONS_OPT_ALIGNED_BODY: *value = c->aligned_body; return ADACONS_OK;
    case ADACONS_OPT_SHIFTED_LOADS: *value = c->shifted_loads; return ADACONS_OK;
    case ADACONS_OPT_CLUSTER_PASS1: *value = c->cluster_pass1; return ADACONS_OK;
    case ADACONS_OPT_GRAM_PASS1: *value = c->gram_fold; return ADACONS_OK;
    case ADACONS_OPT_ROW_PITCH: *value = static_cast<double>(c->pitch); return ADACONS_OK;
    default: return ADACONS_EINVAL;
  }
}

int adacons_get_coeffs(adacons_ctx* c, int which, double* host, void* cuda_stream) {
  if (c == nullptr || host == nullptr || which < 0 || which > ADACONS_COEFF_Q) return ADACONS_EINVAL;
  DeviceGuard guard(c->device);
  if (!guard.ok) return ADACONS_ECUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t n = static_cast<size_t>(c->sets()) * c->N;
  if (cudaMemcpyAsync(host, c->coef + static_cast<size_t>(which) * n, n * sizeof(double), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return ADACONS_ECUDA; }
  return ADACONS_OK;
}

int adacons_get_normaliser(adacons_ctx* c, double* host_z, void* cuda_stream) {
  if (c == nullptr || host_z == nullptr) return ADACONS_EINVAL;
  DeviceGuard guard(c->device);
  if (!guard.ok) return ADACONS_ECUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(host_z, c->z, static_cast<size_t>(c->sets()) * sizeof(double), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return ADACONS_ECUDA; }
  return ADACONS_OK;
}

int adacons_get_state(adacons_ctx* c, double* host_m, int64_t* step, void* cuda_stream) {
  if (c == nullptr) return ADACONS_EINVAL;
  DeviceGuard guard(c->device);
  if (!guard.ok) return ADACONS_ECUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t n = static_cast<size_t>(c->sets()) * c->N;
  long long s = 0;
  if (host_m && cudaMemcpyAsync(host_m, c->m, n * sizeof(double), cudaMemcpyDeviceToHost, st) != cudaSuccess) { cudaGetLastError(); return ADACONS_ECUDA; }
  if (step && cudaMemcpyAsync(&s, c->step, sizeof(long long), cudaMemcpyDeviceToHost, st) != cudaSuccess) { cudaGetLastError(); return ADACONS_ECUDA; }
  if (cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return ADACONS_ECUDA; }
  if (step) *step = s;
  return ADACONS_OK;
}

int adacons_set_state(adacons_ctx* c, const double* host_m, int64_t step, void* cuda_stream) {
  if (c == nullptr || host_m == nullptr || step < 0) return ADACONS_EINVAL;
  DeviceGuard guard(c->device);
  if (!guard.ok) return ADACONS_ECUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  const size_t n = static_cast<size_t>(c->sets()) * c->N;
  const long long s = step;
  if (cudaMemcpyAsync(c->m, host_m, n * sizeof(double), cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaMemcpyAsync(c->step, &s, sizeof(long long), cudaMemcpyHostToDevice, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return ADACONS_ECUDA; }
  return ADACONS_OK;
}

int adacons_get_status(adacons_ctx* c, uint32_t* flags, void* cuda_stream) {
  if (c == nullptr || flags == nullptr) return ADACONS_EINVAL;
  DeviceGuard guard(c->device);
  if (!guard.ok) return ADACONS_ECUDA;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(flags, c->flags, sizeof(uint32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return ADACONS_ECUDA; }
  return ADACONS_OK;
}

int adacons_get_profile(adacons_ctx* c, double ms[3], int64_t* calls, void* cuda_stream) {
  if (c == nullptr || ms == nullptr || calls == nullptr) return ADACONS_EINVAL;
  if (!c->prof_ready || c->prof_calls == 0) return ADACONS_EINVAL;
  DeviceGuard guard(c->device);
  if (!guard.ok) return ADACONS_ECUDA;
  if (cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) { cudaGetLastError(); return ADACONS_ECUDA; }
  const long long n = c->prof_calls < adacons_ctx::kProfSlots ? c->prof_calls : adacons_ctx::kProfSlots;
  double sum[3] = {0.0, 0.0, 0.0};
  for (long long s = 0; s < n; ++s)
    for (int k = 0; k < 3; ++k) {
      float t = 0.f;
      if (cudaEventElapsedTime(&t, c->prof_ev[s][k], c->prof_ev[s][k + 1]) != cudaSuccess) { cudaGetLastError(); return ADACONS_ECUDA; }
      sum[k] += t;
    }
  for (int k = 0; k < 3; ++k) ms[k] = sum[k] / static_cast<double>(n);
  *calls = n;
  return ADACONS_OK;
}

int adacons_selftest_bounded_wait(adacons_ctx* c, int which, void* cuda_stream) {
  if (c == nullptr || which < 0 || which > 2) return ADACONS_EINVAL;
  DeviceGuard guard(c->device);
  if (!guard.ok) return ADACONS_ECUDA;
  selftest_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(which, c->d_barrier, c->flags);
  if (!launch_ok()) return ADACONS_ECUDA;
  c->total_launches += 1;
  return ADACONS_OK;
}

int adacons_get_info(adacons_ctx* c, int key, int64_t* value) {
  if (c == nullptr || value == nullptr) return ADACONS_EINVAL;
  switch (key) {
    case ADACONS_INFO_NUM_SEGMENTS: *value = c->num_segments; return ADACONS_OK;
    case ADACONS_INFO_COEFF_SETS: *value = c->sets(); return ADACONS_OK;
    case ADACONS_INFO_PASS1_BLOCKS: *value = c->fast.available ? c->fast.grid : c->generic_grid; return ADACONS_OK;
    case ADACONS_INFO_SCRATCH_BYTES: *value = static_cast<int64_t>(c->scratch_bytes); return ADACONS_OK;
    case ADACONS_INFO_LAUNCHES_PER_CALL: *value = c->last_launches; return ADACONS_OK;
    case ADACONS_INFO_LAST_PATH: *value = c->last_path; return ADACONS_OK;
    case ADACONS_INFO_TOTAL_LAUNCHES: *value = c->total_launches; return ADACONS_OK;
    case ADACONS_INFO_LAST_PASS2: *value = c->last_pass2; return ADACONS_OK;
    case ADACONS_INFO_STATS_DOUBLES: *value = static_cast<int64_t>(c->sets()) * (2 * c->N + 1); return ADACONS_OK;
    default: return ADACONS_EINVAL;
  }
}

}  // extern "C"

// ------------------------------------------------------------------------------------------------
// Allocation-free consensus statistics (adacons_stats_noalloc).
//
// The block partials of pass 1 go to a fixed array in the library's device image instead of
// memory from cudaMalloc.  In host code the array's name is only a handle: the device address is
// fetched once per device with cudaGetSymbolAddress (that device current) and passed to the
// kernels like any other pointer.
// ------------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_noalloc_scratch[ADACONS_NOALLOC_SCRATCH_BYTES];

namespace {

constexpr int kNoAllocMaxDevices = 64;
constexpr size_t kNoAllocPartialBytes =
    static_cast<size_t>(ADACONS_NOALLOC_MAX_BLOCKS) * 2 * ADACONS_NOALLOC_MAX_N * sizeof(float);

struct NoAllocDevice {
  bool ready = false;
  unsigned char* scratch = nullptr;   // device address of g_noalloc_scratch on this device
  EncodeTiledFn encode = nullptr;
  int sms = 0;
  // launch plan of the most recent shape (a hook calls with the same shape every step)
  bool plan_valid = false;
  int plan_N = 0, plan_dtype = 0, plan_chunks = 1;
  long long plan_d = 0;
  Pass1Plan plan;
};
NoAllocDevice g_noalloc_dev[kNoAllocMaxDevices];
pthread_mutex_t g_noalloc_mutex = PTHREAD_MUTEX_INITIALIZER;

// Sum the block partials in index order (fp64) into the caller's buffer: p (divided by N), then q.
__global__ void stats_finish_kernel(const float* __restrict__ partials, int num_partials, int N,
                                    const uint32_t* __restrict__ flag, double* __restrict__ pq_out) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= 2 * N) return;
  if (*flag & kFlagTimeout) { pq_out[i] = __longlong_as_double(0x7ff8000000000000ll); return; }
  double acc = 0.0;
  for (int c = 0; c < num_partials; ++c) acc += static_cast<double>(partials[static_cast<size_t>(c) * 2 * N + i]);
  pq_out[i] = i < N ? acc / static_cast<double>(N) : acc;
}

int noalloc_setup(int dev, NoAllocDevice** out) {
  if (dev < 0 || dev >= kNoAllocMaxDevices) return ADACONS_EINVAL;
  pthread_mutex_lock(&g_noalloc_mutex);
  NoAllocDevice& nd = g_noalloc_dev[dev];
  int rc = ADACONS_OK;
  if (!nd.ready) {
    void* ptr = nullptr;
    int major = 0;
    if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&nd.sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
      cudaGetLastError(); rc = ADACONS_ECUDA;
    } else if (major != 10) {
      rc = ADACONS_EARCH;
    } else if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess || ptr == nullptr) {
      cudaGetLastError(); rc = ADACONS_ECUDA;
    } else {
      nd.scratch = static_cast<unsigned char*>(ptr);
      void* fn = nullptr;
      cudaDriverEntryPointQueryResult qres;
      if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
          qres == cudaDriverEntryPointSuccess)
        nd.encode = reinterpret_cast<EncodeTiledFn>(fn);
      else
        cudaGetLastError();
      nd.ready = true;
    }
  }
  pthread_mutex_unlock(&g_noalloc_mutex);
  *out = &nd;
  return rc;
}

}  // namespace

extern "C" int adacons_stats_noalloc(const void* grads, int N, int64_t d, int dtype, double* pq_out,
                                     void* cuda_stream) {
  if (grads == nullptr || pq_out == nullptr) return ADACONS_EINVAL;
  if (N < 1 || d < 1 || d >= (1ll << 31)) return ADACONS_EINVAL;
  if (dtype != ADACONS_F32 && dtype != ADACONS_BF16) return ADACONS_EINVAL;
  if (N > ADACONS_NOALLOC_MAX_N) return ADACONS_ELIMIT;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return ADACONS_ECUDA; }
  NoAllocDevice* nd = nullptr;
  int rc = noalloc_setup(dev, &nd);
  if (rc != ADACONS_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

  // A context object on the host stack only carries the launch plan; it owns no device memory.
  // The plan (kernel attributes, occupancy query) is made once per shape and kept.
  adacons_ctx plan;
  plan.N = N; plan.d = d; plan.pitch = d; plan.dtype = dtype; plan.elem_bytes = dtype == ADACONS_F32 ? 4 : 2;
  plan.device = dev; plan.num_sms = nd->sms; plan.encode = nd->encode;
  pthread_mutex_lock(&g_noalloc_mutex);
  if (nd->plan_valid && nd->plan_N == N && nd->plan_d == d && nd->plan_dtype == dtype) {
    plan.fast = nd->plan;
    plan.num_chunks = nd->plan_chunks;
    rc = ADACONS_OK;
  } else {
    rc = plan_fast(&plan);
    if (rc == ADACONS_OK) {
      nd->plan = plan.fast; nd->plan_chunks = plan.num_chunks;
      nd->plan_N = N; nd->plan_d = d; nd->plan_dtype = dtype; nd->plan_valid = true;
    }
  }
  pthread_mutex_unlock(&g_noalloc_mutex);
  if (rc != ADACONS_OK) return rc;

  float* partials = reinterpret_cast<float*>(nd->scratch);
  uint32_t* flag = reinterpret_cast<uint32_t*>(nd->scratch + kNoAllocPartialBytes);
  if (cudaMemsetAsync(flag, 0, sizeof(uint32_t), st) != cudaSuccess) { cudaGetLastError(); return ADACONS_ECUDA; }

  const bool aligned = (reinterpret_cast<uintptr_t>(grads) % 16 == 0) && ((d * plan.elem_bytes) % 16 == 0);
  int blocks;
  if (aligned && plan.fast.available) {
    CUtensorMap maps[2];                                // d < 2^31: at most two chunks; nothing is allocated
    if (plan.num_chunks > 2) return ADACONS_EINVAL;
    for (int ch = 0; ch < plan.num_chunks; ++ch) {
      rc = encode_chunk_map(&plan, grads, ch, &maps[ch]);
      if (rc != ADACONS_OK) return rc;
    }
    int grid = plan.fast.grid;
    if (grid * plan.num_chunks > ADACONS_NOALLOC_MAX_BLOCKS) grid = ADACONS_NOALLOC_MAX_BLOCKS / plan.num_chunks;
    for (int ch = 0; ch < plan.num_chunks; ++ch) {      // column chunks of 2^30 (32-bit TMA coordinates)
      const long long col0 = static_cast<long long>(ch) * kChunkCols;
      const long long cols = d - col0 < kChunkCols ? d - col0 : kChunkCols;
      Pass1Params p;
      p.N = N; p.num_tiles = static_cast<int>((cols + plan.fast.tile_cols - 1) / plan.fast.tile_cols);
      p.stages = plan.fast.stages; p.stage_bytes = plan.fast.stage_bytes;
      p.partials = partials + static_cast<size_t>(ch) * grid * 2 * N; p.flags = flag;
      void* args[2] = {&maps[ch], &p};
      if (cudaLaunchKernel(plan.fast.kernel, dim3(grid), dim3(kThreads), args, plan.fast.smem_bytes, st) != cudaSuccess) {
        cudaGetLastError();
        return ADACONS_ECUDA;
      }
    }
    blocks = grid * plan.num_chunks;
  } else {
    const int tiles = static_cast<int>((d + kThreads * 4 - 1) / (kThreads * 4));
    blocks = nd->sms * 4;
    if (blocks > tiles) blocks = tiles;
    if (blocks > ADACONS_NOALLOC_MAX_BLOCKS) blocks = ADACONS_NOALLOC_MAX_BLOCKS;
    const size_t smem = static_cast<size_t>(kWarps) * N * 2 * sizeof(float);   // <= 4 KB for N <= 64
    if (dtype == ADACONS_F32) pass1_generic_kernel<0><<<blocks, kThreads, smem, st>>>(grads, N, d, d, tiles, partials);
    else pass1_generic_kernel<1><<<blocks, kThreads, smem, st>>>(grads, N, d, d, tiles, partials);
    if (!launch_ok()) return ADACONS_ECUDA;
  }
  stats_finish_kernel<<<(2 * N + 127) / 128, 128, 0, st>>>(partials, blocks, N, flag, pq_out);
  if (!launch_ok()) return ADACONS_ECUDA;
  return ADACONS_OK;
}
