// Pieces shared by the two scan kernels (8-bit codes: scan.cu, 4-bit codes: scan4.cu): packed
// fp32 accumulators, the vector reduction into the list partial, and the bulk-copy / mbarrier
// wrappers used for the table fetch.
#pragma once

#include "common.cuh"

namespace pqhsa {

// Packed accumulators: the Gc partial sums of a token live in 64-bit registers holding two
// floats each, so one table entry is added with add.f32x2 (two lanes per instruction).
template <int GC> struct Acc;
template <> struct Acc<4> {
  unsigned long long lo, hi;
  __device__ __forceinline__ void zero() { lo = 0ull; hi = 0ull; }
  __device__ __forceinline__ void load(uint32_t saddr) {
    asm volatile("ld.shared.v2.b64 {%0, %1}, [%2];" : "=l"(lo), "=l"(hi) : "r"(saddr));
  }
  __device__ __forceinline__ void merge(const Acc& o) {
    asm("add.rn.f32x2 %0, %0, %1;" : "+l"(lo) : "l"(o.lo));
    asm("add.rn.f32x2 %0, %0, %1;" : "+l"(hi) : "l"(o.hi));
  }
  __device__ __forceinline__ void get(float (&f)[4]) const {
    f[0] = __uint_as_float((uint32_t)lo); f[1] = __uint_as_float((uint32_t)(lo >> 32));
    f[2] = __uint_as_float((uint32_t)hi); f[3] = __uint_as_float((uint32_t)(hi >> 32));
  }
};
template <> struct Acc<2> {
  unsigned long long lo;
  __device__ __forceinline__ void zero() { lo = 0ull; }
  __device__ __forceinline__ void load(uint32_t saddr) {
    asm volatile("ld.shared.b64 %0, [%1];" : "=l"(lo) : "r"(saddr));
  }
  __device__ __forceinline__ void merge(const Acc& o) {
    asm("add.rn.f32x2 %0, %0, %1;" : "+l"(lo) : "l"(o.lo));
  }
  __device__ __forceinline__ void get(float (&f)[2]) const {
    f[0] = __uint_as_float((uint32_t)lo); f[1] = __uint_as_float((uint32_t)(lo >> 32));
  }
};
template <> struct Acc<1> {
  float v;
  __device__ __forceinline__ void zero() { v = 0.f; }
  __device__ __forceinline__ void load(uint32_t saddr) {
    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(saddr));
  }
  __device__ __forceinline__ void merge(const Acc& o) { v += o.v; }
  __device__ __forceinline__ void get(float (&f)[1]) const { f[0] = v; }
};

template <int GC> __device__ __forceinline__ void load_vec(float (&f)[GC], const float* p);
template <> __device__ __forceinline__ void load_vec<1>(float (&f)[1], const float* p) { f[0] = *p; }
template <> __device__ __forceinline__ void load_vec<2>(float (&f)[2], const float* p) {
  const float2 v = *reinterpret_cast<const float2*>(p);
  f[0] = v.x; f[1] = v.y;
}
template <> __device__ __forceinline__ void load_vec<4>(float (&f)[4], const float* p) {
  const float4 v = *reinterpret_cast<const float4*>(p);
  f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
}

template <int GC> __device__ __forceinline__ void red_add(float* dst, const float (&e)[GC]) {
  if constexpr (GC == 4)
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(dst), "f"(e[0]), "f"(e[1]),
                 "f"(e[2]), "f"(e[3]) : "memory");
  else if constexpr (GC == 2)
    asm volatile("red.global.add.v2.f32 [%0], {%1, %2};" ::"l"(dst), "f"(e[0]), "f"(e[1]) : "memory");
  else
    asm volatile("red.global.add.f32 [%0], %1;" ::"l"(dst), "f"(e[0]) : "memory");
}

constexpr float kOverflowGuardLog2 = 96.0f;   // exp2 arguments above this trigger the rebuild
// The reference of a segment's exp-sums is set this far above the maximum of the CTA's first
// round of tiles, so that a later, larger logit (heavy-tailed keys: the maximum of 57 K tokens
// is far above the maximum of the first 512) still lands below the overflow guard and the
// segment is not rebuilt; terms are kept down to 2^-40 of the first round's maximum, as before.
// exp2 arguments then run from -120 to +96, inside the fp32 range (2^-120 is a normal number).
constexpr float kRefHeadroomLog2 = 80.0f;
constexpr float kRefHeadroom = kRefHeadroomLog2 / kLog2e;             // in units of the scores
constexpr float kScanNegligibleLog2 = kNegligibleLog2 - kRefHeadroomLog2;
constexpr int kMbarSpinLimit = 1 << 22;

// ---- bulk async copy global -> shared, completion on an mbarrier (TMA, no tensor map)
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)),
               "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}
// Bounded wait: returns false if the phase did not complete within the spin limit.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  for (int it = 0; it < kMbarSpinLimit; ++it) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    if (done) return true;
  }
  return false;
}

}  // namespace pqhsa
