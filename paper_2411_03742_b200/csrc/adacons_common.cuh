// Constants, status flags and the small PTX helpers shared by every kernel of the AdaCons library (sm_100a).
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

__device__ __forceinline__ uint4 ld_nc_v4(const void* p) {   // read-only path, L1 allocation allowed
  uint4 v;
  asm("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
// bytes [shift, shift + 16) of the 32 bytes lo:hi; shift is a multiple of 2
__device__ __forceinline__ uint4 realign_16(const uint4& lo, const uint4& hi, const int shift) {
  const uint32_t r = static_cast<uint32_t>(shift & 3) * 8u;
  switch (shift >> 2) {
    case 0: return make_uint4(__funnelshift_r(lo.x, lo.y, r), __funnelshift_r(lo.y, lo.z, r), __funnelshift_r(lo.z, lo.w, r), __funnelshift_r(lo.w, hi.x, r));
    case 1: return make_uint4(__funnelshift_r(lo.y, lo.z, r), __funnelshift_r(lo.z, lo.w, r), __funnelshift_r(lo.w, hi.x, r), __funnelshift_r(hi.x, hi.y, r));
    case 2: return make_uint4(__funnelshift_r(lo.z, lo.w, r), __funnelshift_r(lo.w, hi.x, r), __funnelshift_r(hi.x, hi.y, r), __funnelshift_r(hi.y, hi.z, r));
    default: return make_uint4(__funnelshift_r(lo.w, hi.x, r), __funnelshift_r(hi.x, hi.y, r), __funnelshift_r(hi.y, hi.z, r), __funnelshift_r(hi.z, hi.w, r));
  }
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

}  // namespace adacons
