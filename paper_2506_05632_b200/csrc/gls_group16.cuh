// gls_group16.cuh -- building blocks of the vocabulary sweeps: 256-bit streaming loads, groups of
// 16 logits held in registers (bf16 pairs or fp32), two-wide fp32 arithmetic, the group-wise
// log-sum-exp, and a Philox4x32 variant that derives its round keys on the fly.
#pragma once
#include "gls_kernels.cuh"

namespace gls {

// 32 bytes per lane in one instruction (sm_100a): a warp reads 1 KB contiguous.
struct Words8 {
  uint32_t w[8];
};
__device__ __forceinline__ Words8 ld_stream32(const void* p) {
  Words8 v;
  asm volatile("ld.global.nc.L1::no_allocate.v8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(v.w[0]), "=r"(v.w[1]), "=r"(v.w[2]), "=r"(v.w[3]), "=r"(v.w[4]),
                 "=r"(v.w[5]), "=r"(v.w[6]), "=r"(v.w[7])
               : "l"(p));
  return v;
}

__device__ __forceinline__ float lg2_approx(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// two-wide fp32 arithmetic (sm_100a)
__device__ __forceinline__ unsigned long long pack_f32x2(float a, float b) {
  unsigned long long r;
  asm("mov.b64 %0, {%1,%2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long r, float& a, float& b) {
  asm("mov.b64 {%0,%1}, %2;" : "=f"(a), "=f"(b) : "l"(r));
}
__device__ __forceinline__ unsigned long long fma_f32x2(unsigned long long a, unsigned long long b,
                                                        unsigned long long c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ unsigned long long mul_f32x2(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
__device__ __forceinline__ unsigned long long add_f32x2(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// 16 tokens of one lane: bf16 -> 8 words (two tokens each), fp32 -> 16 words
template <int DT>
struct Group16;
template <>
struct Group16<kBF16> {
  Words8 a;
};
template <>
struct Group16<kF32> {
  Words8 a, b;
};

__device__ __forceinline__ void load16_vec(Group16<kBF16>& g, const char* p) { g.a = ld_stream32(p); }
__device__ __forceinline__ void load16_vec(Group16<kF32>& g, const char* p) {
  g.a = ld_stream32(p);
  g.b = ld_stream32(p + 32);
}
// scalar loader for ragged tails and rows that are not 32-byte aligned; out of range -> -inf
__device__ __forceinline__ void load16_scalar(Group16<kBF16>& g, const char* rowp, int tok, int end) {
#pragma unroll
  for (int t = 0; t < 8; ++t) {
    const uint32_t lo = tok + 2 * t < end ? (uint32_t)__ldg((const unsigned short*)rowp + tok + 2 * t) : 0xff80u;
    const uint32_t hi = tok + 2 * t + 1 < end ? (uint32_t)__ldg((const unsigned short*)rowp + tok + 2 * t + 1) : 0xff80u;
    g.a.w[t] = lo | (hi << 16);
  }
}
__device__ __forceinline__ void load16_scalar(Group16<kF32>& g, const char* rowp, int tok, int end) {
#pragma unroll
  for (int t = 0; t < 8; ++t) {
    g.a.w[t] = tok + t < end ? __float_as_uint(__ldg((const float*)rowp + tok + t)) : 0xff800000u;
    g.b.w[t] = tok + 8 + t < end ? __float_as_uint(__ldg((const float*)rowp + tok + 8 + t)) : 0xff800000u;
  }
}

// max over the 16 logits, ignoring NaN
__device__ __forceinline__ float group16_max(const Group16<kBF16>& g) {
  const uint32_t x = max_bf16x2(max_bf16x2(max_bf16x2(g.a.w[0], g.a.w[1]), max_bf16x2(g.a.w[2], g.a.w[3])),
                                max_bf16x2(max_bf16x2(g.a.w[4], g.a.w[5]), max_bf16x2(g.a.w[6], g.a.w[7])));
  return fmaxf(bf16_lo(x), bf16_hi(x));
}
__device__ __forceinline__ float group16_max(const Group16<kF32>& g) {
  float m = -CUDART_INF_F;
#pragma unroll
  for (int t = 0; t < 8; ++t)
    m = fmaxf(m, fmaxf(__uint_as_float(g.a.w[t]), __uint_as_float(g.b.w[t])));
  return m;
}
// logit t (0..15) of the group, t a compile-time constant after unrolling
template <int DT>
__device__ __forceinline__ float group16_get(const Group16<DT>& g, int t);
template <>
__device__ __forceinline__ float group16_get<kBF16>(const Group16<kBF16>& g, int t) {
  return (t & 1) ? bf16_hi(g.a.w[t >> 1]) : bf16_lo(g.a.w[t >> 1]);
}
template <>
__device__ __forceinline__ float group16_get<kF32>(const Group16<kF32>& g, int t) {
  return __uint_as_float(t < 8 ? g.a.w[t] : g.b.w[t - 8]);
}

// (logit t - lm, logit t+1 - lm) as an fp32 pair, t even.  bf16: the mixed-precision add takes
// the 16-bit halves of the word as they are (bf16 + fp32 -> fp32, rounded once), so the pair is
// never unpacked.
__device__ __forceinline__ unsigned long long group16_diff2(const Group16<kBF16>& g, int t, float nlm,
                                                            unsigned long long) {
  unsigned short lo, hi;
  asm("mov.b32 {%0,%1}, %2;" : "=h"(lo), "=h"(hi) : "r"(g.a.w[t >> 1]));
  float d0, d1;
  asm("add.rn.f32.bf16 %0, %1, %2;" : "=f"(d0) : "h"(lo), "f"(nlm));
  asm("add.rn.f32.bf16 %0, %1, %2;" : "=f"(d1) : "h"(hi), "f"(nlm));
  return pack_f32x2(d0, d1);
}
__device__ __forceinline__ unsigned long long group16_diff2(const Group16<kF32>& g, int t, float,
                                                            unsigned long long nlm2) {
  return add_f32x2(pack_f32x2(group16_get<kF32>(g, t), group16_get<kF32>(g, t + 1)), nlm2);
}

constexpr float kGroupLseFloor = -1.0e30f;  // finite stand-in for "no finite logit seen yet"

// Softmax statistics of 16 logits: lm = reference exponent, ls2 = two partial sums of
// 2^((a - lm) c2).  lm is not a running maximum: it moves only when a group's maximum exceeds it
// by more than 2^kLseHeadroom (then it jumps to that maximum), so the rescaling branch is taken a
// handful of times per row instead of whenever any lane sees a new maximum; terms are at most
// 2^kLseHeadroom, far from fp32 overflow for any row length.  The loop assumes finite-or-(-inf)
// logits and checks nothing: a NaN or +inf logit turns the lane's sum into NaN or +inf, which
// the caller detects once at the end of the work item and repairs with the sweep's careful redo.
constexpr float kLseHeadroom = 64.0f;
template <int DT>
__device__ __forceinline__ void lse16(const Group16<DT>& g, float amax, float c2, float& lm,
                                      unsigned long long& ls2) {
  if (fmaf(amax - lm, c2, -kLseHeadroom) > 0.f) {
    if (amax < CUDART_INF_F) {
      const float r = ex2_approx((lm - amax) * c2);
      ls2 = fma_f32x2(ls2, pack_f32x2(r, r), 0ull);
      lm = amax;
    }
  }
  // (a - lm) first, then the scale: the difference is exact (or rounded at 2^-24 of itself), so
  // the exponent is good to 1e-7 of its own size however large the logits are; a * c2 - lm * c2
  // would carry the rounding of the two large products
  const unsigned long long c22 = pack_f32x2(c2, c2), nlm2 = pack_f32x2(-lm, -lm);
#pragma unroll
  for (int t = 0; t < 16; t += 2) {
    float e0, e1;
    unpack_f32x2(mul_f32x2(group16_diff2(g, t, -lm, nlm2), c22), e0, e1);
    ls2 = add_f32x2(ls2, pack_f32x2(ex2_approx(e0), ex2_approx(e1)));
  }
}

// dynamic shared memory of the sweep and reduction kernels
extern __shared__ __align__(16) unsigned char gls_smem_raw[];

// Philox4x32 with the round keys derived on the fly (the batched path runs out of line and has no
// cheap access to the kernel parameter's precomputed round keys).
template <int ROUNDS>
__device__ __forceinline__ void philox4x32_keyed(uint32_t k0, uint32_t k1, int rounds_rt, uint32_t c0,
                                                 uint32_t c1, uint32_t c2, uint32_t c3,
                                                 uint32_t (&out)[4]) {
  const int n = ROUNDS > 0 ? ROUNDS : rounds_rt;
#pragma unroll
  for (int r = 0; r < n; ++r) {
    const unsigned long long p0 = (unsigned long long)kPhiloxM0 * c0;
    const unsigned long long p1 = (unsigned long long)kPhiloxM1 * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    c1 = (uint32_t)p1;
    c3 = (uint32_t)p0;
    c0 = n0;
    c2 = n2;
    k0 += kPhiloxW0;
    k1 += kPhiloxW1;
  }
  out[0] = c0;
  out[1] = c1;
  out[2] = c2;
  out[3] = c3;
}


}  // namespace gls
