// gls_sweep3.cuh -- the vocabulary sweep for noise_spec 3 (8 coarse + 40 refinement bits).
//
// One Philox4x32 call yields the coarse bytes of 16 consecutive tokens, so the generator -- whose
// 32x32->64-bit multiplies are the scarcest resource of this path on sm_100a -- runs once per 16
// tokens.  With m a lower bound on the row's best score, token i can only matter if
// S_i <= exp(logit_i/T - m), and S_i = -log1p(-v_i) >= v_i >= h_i / 256 with h_i its coarse byte.
// Hence, per group of 16 tokens, with 2^x = 256 * 2^(max logit * c - m'):
//   - if x <= 0 (the usual case), only tokens with h == 0 can matter: a zero-byte test on the
//     four generator words settles the group;
//   - otherwise the group is "wide" (a few dozen per row): bytes below 2^x can matter.
// Candidate groups are not examined on the spot: the lane pushes the group (the four generator
// words, its block index tagged with ceil(x), and its 16 logits as loaded) on a small per-warp
// queue in shared memory and the sweep goes on.  When 32 groups are queued the warp evaluates
// them together, one group per lane: per-token test on the coarse byte, refinement bits from the
// second generator stream, the filter on the 48-bit uniform, and for the survivors the fp32 score
// logit/T - ln(-log1p(-v)).  Batching turns what would be a divergent detour in most iterations
// (a zero byte turns up in 1 of 16 groups) into dense work done once per ~10 iterations, and
// because the entry carries the logits the batched path never goes back to global memory.  The
// filter has no false negatives, so the result equals a full evaluation (Sec. 3 step 2 /
// Algorithm 2 draft loop and Y_j line of arXiv 2506.05632, log domain).
//
// Work decomposition: a work item is one (row, vocabulary slice), owned by one CTA (2 warps for
// bf16 rows, 8 for fp32); per iteration a lane takes 16 consecutive tokens (one 32-byte load of
// bf16, two of fp32), a warp 512 and the CTA 1024 or 4096 contiguous tokens.  Warps never wait on one another: they share the bound
// m through one tagged shared-memory word, each warp writes its own partial result, and the
// split-V reduction merges them.  The batched evaluation is called from an outer loop so that
// the hot loop contains no call.  A fused variant (MULTI) races one row under several noise
// streams at once for the compression encoder of Sec. 5.1.
#pragma once
#include "gls_kernels.cuh"

namespace gls {

constexpr int kS3LaneTokens = 16;
constexpr int kS3WarpTokens = 32 * kS3LaneTokens;               // 512

// Launch shape per element type, chosen by measurement.  bf16 rows are bound by the noise
// arithmetic: few warps per row and ~100 registers per thread (2 warps x 10 CTAs per SM) beat
// wider CTAs by 15 %, because longer per-warp items amortise the per-item set-up and more
// registers let the two generator chains of a step overlap.  fp32 rows are bound by HBM and want
// the memory parallelism of 8 warps x 3 CTAs.
template <int DT>
struct S3Cfg {
  static constexpr int kWarps = DT == kBF16 ? 2 : 8;
  static constexpr int kCtasPerSM = DT == kBF16 ? 10 : 3;
  static constexpr int kCtaTokens = kWarps * kS3WarpTokens;  // tokens one CTA consumes per iteration
};
constexpr int kS3MaxWarps = 8;
constexpr int kS3MaxCtaTokens = kS3MaxWarps * kS3WarpTokens;

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

// the group as loaded, to 16-byte aligned shared memory
__device__ __forceinline__ void store_group16(uint32_t* dst, const Group16<kBF16>& g) {
  reinterpret_cast<uint4*>(dst)[0] = make_uint4(g.a.w[0], g.a.w[1], g.a.w[2], g.a.w[3]);
  reinterpret_cast<uint4*>(dst)[1] = make_uint4(g.a.w[4], g.a.w[5], g.a.w[6], g.a.w[7]);
}
__device__ __forceinline__ void store_group16(uint32_t* dst, const Group16<kF32>& g) {
  reinterpret_cast<uint4*>(dst)[0] = make_uint4(g.a.w[0], g.a.w[1], g.a.w[2], g.a.w[3]);
  reinterpret_cast<uint4*>(dst)[1] = make_uint4(g.a.w[4], g.a.w[5], g.a.w[6], g.a.w[7]);
  reinterpret_cast<uint4*>(dst)[2] = make_uint4(g.b.w[0], g.b.w[1], g.b.w[2], g.b.w[3]);
  reinterpret_cast<uint4*>(dst)[3] = make_uint4(g.b.w[4], g.b.w[5], g.b.w[6], g.b.w[7]);
}

constexpr float kS3LseFloor = -1.0e30f;  // finite stand-in for "no finite logit seen yet"

// Softmax statistics of 16 logits: lm = reference exponent, ls2 = two partial sums of
// 2^((a - lm) c2).  lm is not a running maximum: it moves only when a group's maximum exceeds it
// by more than 2^kLseHeadroom (then it jumps to that maximum), so the rescaling branch is taken a
// handful of times per row instead of whenever any lane sees a new maximum; terms are at most
// 2^kLseHeadroom, far from fp32 overflow for any row length.  The loop assumes finite-or-(-inf)
// logits and checks nothing: a NaN or +inf logit turns the lane's sum into NaN or +inf, which
// the caller detects once at the end of the work item and repairs with lse_redo_careful().
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

// The lane's share of a work item again, token by token, leaving out NaN and +inf logits (they
// cannot define a probability).  Rare: only rows that hold such values come here.
template <int DT>
__device__ __noinline__ void lse_redo_careful(const char* rowp, int tok0, int n_iter, int tok_end,
                                              float c2, float* lm_out, float* ls_out) {
  float lm = kS3LseFloor, ls = 0.f;
  for (int it = 0; it < n_iter; ++it) {
    const int tok = tok0 + it * S3Cfg<DT>::kCtaTokens;
    for (int t = 0; t < kS3LaneTokens; ++t) {
      if (tok + t >= tok_end) break;
      const float a = load_logit<DT>(rowp, tok + t);
      if (!(a < CUDART_INF_F) || a == -CUDART_INF_F) continue;
      if (a > lm) {
        ls *= ex2_approx((lm - a) * c2);
        lm = a;
      }
      ls += ex2_approx((a - lm) * c2);
    }
  }
  *lm_out = lm;
  *ls_out = ls;
}

// Any zero byte among the 16 coarse bytes?  (exact as a yes / no for the four words together)
__device__ __forceinline__ bool any_zero_byte(const uint32_t (&w)[4]) {
  const uint32_t z = ((w[0] - 0x01010101u) & ~w[0]) | ((w[1] - 0x01010101u) & ~w[1]) |
                     ((w[2] - 0x01010101u) & ~w[2]) | ((w[3] - 0x01010101u) & ~w[3]);
  return (z & 0x80808080u) != 0u;
}
// bit t set iff byte t of the word is zero (exact per byte)
__device__ __forceinline__ uint32_t zero_byte_mask4(uint32_t v) {
  const uint32_t t = ~(((v & 0x7f7f7f7fu) + 0x7f7f7f7fu) | v | 0x7f7f7f7fu);  // 0x80 per zero byte
  return (((t >> 7) * 0x00204081u) >> 21) & 0xfu;
}

// ------------------------------------------------------------------------------------------
// Shared memory of the sweep CTA (dynamic, so that the batched path below can reach it too)
// ------------------------------------------------------------------------------------------
struct S3WarpCtx {  // what the batched path needs to know about the warp's current work item
  const uint8_t* bins;
  uint32_t c1, pos, seq;
  uint32_t key0, key1;  // Philox key (round keys are key + r * Weyl constants)
  float inv_t;
  int msg, tok_end;
};
// A queue entry holds everything the batched path needs, so that it never goes back to global
// memory for the logits: 4 generator words, block index | kb << 28, and the group's 16 logits as
// loaded (8 words of bf16, 16 of fp32).  Entries are 16-byte aligned for 128-bit accesses.
template <int DT>
struct S3Entry {
  static constexpr int kDataWords = DT == kBF16 ? 8 : 16;
  static constexpr int kWords = 8 + (DT == kBF16 ? 8 : 24);  // 64 or 128 bytes
  // Groups per warp queue: a batch is taken at 32 queued groups, and one step of the sweep can
  // add 32 more (64 for bf16, whose sweep handles two groups per lane and step).
  static constexpr int kCap = DT == kBF16 ? 96 : 64;
};
template <int DT>
struct S3Shared {
  unsigned long long m_tag;  // (item tag << 32) | ordered code of the CTA-wide bound on the best score
  S3WarpCtx ctx[S3Cfg<DT>::kWarps];
  Top2 best[S3Cfg<DT>::kWarps * 32];  // per-thread candidates, touched by the batched path only
  __align__(16) uint32_t queue[S3Cfg<DT>::kWarps][S3Entry<DT>::kCap * S3Entry<DT>::kWords];
};
extern __shared__ __align__(16) unsigned char s3_smem_raw[];
template <int DT>
__device__ __forceinline__ S3Shared<DT>& s3_shared() {
  return *reinterpret_cast<S3Shared<DT>*>(s3_smem_raw);
}

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

// logit t (0..15, a run-time index) of a queued group
template <int DT>
__device__ __forceinline__ float entry_logit(const uint32_t* data, int t) {
  if (DT == kBF16) {
    const uint32_t w = data[t >> 1];
    return (t & 1) ? bf16_hi(w) : bf16_lo(w);
  }
  return __uint_as_float(data[t]);
}

// ------------------------------------------------------------------------------------------
// Batched evaluation of queued groups: lane l < n takes entry first + l of its warp's queue.
// Candidate tokens of a group: those whose coarse byte is below 2^kb (kb = 0, the usual case:
// zero bytes only); in a very wide group (kb > 3) those whose byte passes the per-token test
// h < 256 * 2^(logit c + nm).  A candidate with a non-zero byte takes that per-token test first;
// then the lane draws its 40 refinement bits, applies the filter to the 48-bit uniform and scores
// the survivors in fp32.  Returns the best lower bound found (ordered code, 0 if none).
// ------------------------------------------------------------------------------------------
template <int DT, int ROUNDS, bool MULTI>
__device__ __noinline__ uint32_t s3_flush(int rounds_rt, int first, int n, float nm) {
  S3Shared<DT>& sh = s3_shared<DT>();
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const S3WarpCtx cx = sh.ctx[warp];
  const uint32_t* e = sh.queue[warp] + (first + lane) * S3Entry<DT>::kWords;
  const uint32_t* data = e + 8;
  const float c2 = cx.inv_t * kLog2e;
  const float nm8 = nm + 8.0f;
  uint32_t msk = 0u, blk = 0u;
  uint32_t w0 = 0u, w1 = 0u, w2 = 0u, w3 = 0u;
  uint32_t ks = 0u;  // noise stream of the entry (fused multi-stream race only)
  if (lane < n) {
    const uint4 cw = *reinterpret_cast<const uint4*>(e);
    w0 = cw.x; w1 = cw.y; w2 = cw.z; w3 = cw.w;
    blk = e[4];
    if (MULTI) ks = e[5];
    // kb: the group's coarse bytes can matter only below 2^kb (0: zero bytes only)
    const uint32_t kb = blk >> 28;
    blk &= 0x0fffffffu;
    if (kb > 3u) {
      // very wide group: test every token's byte against the token's own threshold
#pragma unroll
      for (int t = 0; t < 16; ++t) {
        const uint32_t wt = t < 4 ? w0 : t < 8 ? w1 : t < 12 ? w2 : w3;
        const float h = (float)((wt >> (8 * (t & 3))) & 0xffu);
        if (h < ex2_approx(fmaf(entry_logit<DT>(data, t), c2, nm8))) msk |= 1u << t;  // false for NaN
      }
    } else {
      // bytes below 2^kb: clear their low kb bits and look for zero bytes
      const uint32_t keep = 0x01010101u * ((0xffu << kb) & 0xffu);
      msk = zero_byte_mask4(w0 & keep) | (zero_byte_mask4(w1 & keep) << 4) |
            (zero_byte_mask4(w2 & keep) << 8) | (zero_byte_mask4(w3 & keep) << 12);
    }
  }
  Top2 b = sh.best[threadIdx.x];
  float lower = -CUDART_INF_F;
  while (__any_sync(0xffffffffu, msk != 0u)) {
    if (msk != 0u) {
      const int t = __ffs(msk) - 1;
      msk &= msk - 1u;
      const int i = (int)(blk << 4) + t;
      if (i < cx.tok_end) {
        const float a = entry_logit<DT>(data, t);
        const uint32_t wt = t < 4 ? w0 : t < 8 ? w1 : t < 12 ? w2 : w3;
        const uint32_t h = (wt >> (8 * (t & 3))) & 0xffu;
        // NaN and +inf never win; a non-zero byte must pass its own coarse test first
        if (a < CUDART_INF_F && (h == 0u || (float)h < ex2_approx(fmaf(a, c2, nm8)))) {
          uint32_t f[4];
          philox4x32_keyed<ROUNDS>(cx.key0, cx.key1, rounds_rt, (uint32_t)i >> 1,
                                   cx.c1 + ks + (2u << 16), cx.pos, cx.seq, f);
          const uint32_t lo = (i & 1) ? f[2] : f[0], hi = ((i & 1) ? f[3] : f[1]) & 0xffu;
          const float v = fmaf((float)h, 0x1p-8f,
                               fmaf((float)hi, 0x1p-16f, fmaf((float)lo, 0x1p-48f, 0x1p-49f)));
          if (v < ex2_approx(fmaf(a, c2, nm)) &&
              (cx.bins == nullptr || (int)__ldg(cx.bins + i) == cx.msg)) {
            float ln_s;
            const float s = score_f32(a, cx.inv_t, v, &ln_s);
            // fused race: the candidate is (token, stream), ordered by token first
            top2_offer(b, s, MULTI ? (int)(((uint32_t)i << 3) | ks) : i);
            lower = fmaxf(lower, s - score_slack(s, ln_s));
          }
        }
      }
    }
  }
  sh.best[threadIdx.x] = b;
  __syncwarp();
  return __reduce_max_sync(0xffffffffu, enc_ordered(lower));
}

// ------------------------------------------------------------------------------------------
// The kernel
// ------------------------------------------------------------------------------------------
template <int DT, bool LSE, int ROUNDS, bool MULTI = false>
__global__ void __launch_bounds__(S3Cfg<DT>::kWarps * 32, S3Cfg<DT>::kCtasPerSM)
sweep3_kernel(const __grid_constant__ SweepArgs A) {
  S3Shared<DT>& sh = s3_shared<DT>();
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  constexpr int ES = DT == kBF16 ? 2 : 4;
  constexpr bool PREFETCH = DT == kBF16;       // fp32 groups are 16 registers: no second copy
  constexpr int kS3CtaTokens = S3Cfg<DT>::kCtaTokens;
  constexpr int kSweepWarps3 = S3Cfg<DT>::kWarps;
  constexpr int STEP = kS3CtaTokens * ES;      // bytes between a lane's consecutive groups
  typedef Group16<DT> G;
  uint32_t* const queue = sh.queue[warp];
  volatile unsigned long long* const m_tag = &sh.m_tag;

  if (threadIdx.x == 0) sh.m_tag = 0ull;
  __syncthreads();

  uint32_t tag = 0u;
  for (long long item = blockIdx.x; item < A.n_items; item += gridDim.x) {
    ++tag;
    const int split = (int)(item / A.rows);
    const int row = (int)(item - (long long)split * A.rows);
    const int tok_begin = split * A.chunk;
    const int tok_end = min(A.V, tok_begin + A.chunk);
    uint32_t c1, pos, seq;
    const char* rowp;
    float c2;
    {
      const int j = row % A.J;
      const int bk = row / A.J;
      const int k = bk % A.K;
      const int b = bk / A.K;
      rowp = (const char*)A.data + (b * A.sb + k * A.sk + j * A.sj) * ES;
      c1 = ((uint32_t)k & A.kmask) | (A.domain << 16);
      pos = A.pos_base + (uint32_t)j;
      seq = A.seq_ids ? __ldg(A.seq_ids + b) : A.seq_base + (uint32_t)b;
      const float inv_t = A.inv_t[k];
      c2 = inv_t * kLog2e;
      __syncwarp();  // the previous item's batched path is done with the context
      if (lane == 0) {
        S3WarpCtx cx;
        cx.bins = A.bins ? A.bins + A.bins_sb * b : nullptr;
        cx.c1 = c1; cx.pos = pos; cx.seq = seq;
        cx.key0 = A.rk[0]; cx.key1 = A.rk[1];
        cx.inv_t = inv_t;
        cx.msg = (A.bins && A.msg) ? (int)__ldg(A.msg + b) : 0;
        cx.tok_end = tok_end;
        sh.ctx[warp] = cx;
      }
      top2_init(sh.best[threadIdx.x]);
      __syncwarp();
    }
    const bool aligned = (((uintptr_t)rowp) & 31) == 0;
    // this warp's iterations: tokens base_w + it * kS3CtaTokens + [0, 512)
    const int base_w = tok_begin + warp * kS3WarpTokens;
    const int span = tok_end - base_w;
    const int n_iter = span > 0 ? (span + kS3CtaTokens - 1) / kS3CtaTokens : 0;
    const int n_full = (aligned && span >= kS3WarpTokens) ? (span - kS3WarpTokens) / kS3CtaTokens + 1 : 0;
    const int tok0 = base_w + lane * kS3LaneTokens;

    uint32_t m_enc = __ldcg(A.hints + row);  // bound published by earlier slices of the row
    float lm = kS3LseFloor;
    unsigned long long ls2 = 0ull;
    int qn = 0;

    // ---- warm start: a valid lower bound from the coarse bytes of the lane's first group -----
    // v < (h + 1) / 256  =>  S = -log1p(-v) < x / (1 - x), x = (h + 1) / 256, so the token's score
    // exceeds logit/T - ln(x / (1 - x)).  Each lane takes the best such bound over its 16 tokens.
    if (n_iter > 0) {
      G g;
      if (n_full > 0) load16_vec(g, rowp + (size_t)tok0 * ES);
      else load16_scalar(g, rowp, tok0, tok_end);
      uint32_t cw[4];
      philox4x32<ROUNDS>(A.rk, A.rounds, (uint32_t)tok0 >> 4, c1, pos, seq, cw);
      float lb2 = -CUDART_INF_F;  // log2 units
      int tb = 0;
#pragma unroll
      for (int t = 0; t < 16; ++t) {
        const float a = group16_get<DT>(g, t);
        const uint32_t h = (cw[t >> 2] >> (8 * (t & 3))) & 0xffu;
        // log2 of exp(logit/T) (1 - x) / x
        const float key = fmaf(a, c2, lg2_approx((float)(255u - h)) - lg2_approx((float)(h + 1u)));
        if (h < 255u && a < CUDART_INF_F && key > lb2) {
          lb2 = key;
          tb = t;
        }
      }
      float lb = -CUDART_INF_F;
      const S3WarpCtx& cx = sh.ctx[warp];
      if (lb2 > -CUDART_INF_F && tok0 + tb < tok_end &&
          (cx.bins == nullptr || (int)__ldg(cx.bins + tok0 + tb) == cx.msg)) {
        lb = lb2 * 0.6931471805599453f;
        // lg2.approx and the roundings are good to ~1e-6 relative of |lb2| + 8
        lb -= 0x1p-16f * (16.0f + fabsf(lb));
      }
      const uint32_t e = __reduce_max_sync(0xffffffffu, enc_ordered(lb));
      if (e > m_enc) m_enc = e;
      if (lane == 0 && m_enc > 0u)
        atomicMax((unsigned long long*)&sh.m_tag, ((unsigned long long)tag << 32) | m_enc);
    }
    float nm8 = filter_offset(dec_ordered(m_enc)) + 8.0f;

    // one group of 16 tokens per lane
    auto process = [&](const G& g, int tok) {
      uint32_t cw[4];
      philox4x32<ROUNDS>(A.rk, A.rounds, (uint32_t)tok >> 4, c1, pos, seq, cw);
      const float amax = group16_max(g);
      const float x = fmaf(amax, c2, nm8);  // log2 of 256 * 2^(amax c + nm)
      const bool wide = x > 0.f;             // non-zero coarse bytes may matter, those below 2^x
      const bool pass = any_zero_byte(cw) | wide;
      if (LSE) lse16<DT>(g, amax, c2, lm, ls2);
      const unsigned long long mt = *m_tag;  // bound published by the other warps of the CTA
      uint32_t m_new = ((uint32_t)(mt >> 32) == tag) ? (uint32_t)mt : 0u;
      const unsigned bal = __ballot_sync(0xffffffffu, pass);
      if (bal != 0u) {
        if (pass) {
          uint32_t* e = queue + (qn + __popc(bal & ((1u << lane) - 1u))) * S3Entry<DT>::kWords;
          const uint32_t kb = wide ? (uint32_t)min(15, __float2int_ru(x)) : 0u;
          *reinterpret_cast<uint4*>(e) = make_uint4(cw[0], cw[1], cw[2], cw[3]);
          e[4] = ((uint32_t)tok >> 4) | (kb << 28);
          store_group16(e + 8, g);
        }
        qn += __popc(bal);
      }
      if (m_new > m_enc) {
        m_enc = m_new;
        nm8 = filter_offset(dec_ordered(m_enc)) + 8.0f;
      }
    };

    // two groups per lane in one step (bf16): two independent generator chains in flight hide
    // each other's latency, and the loop and polling overhead is paid once for 32 tokens
    auto process2 = [&](const G& g0, const G& g1, int tok) {
      uint32_t cw0[4], cw1[4];
      philox4x32<ROUNDS>(A.rk, A.rounds, (uint32_t)tok >> 4, c1, pos, seq, cw0);
      philox4x32<ROUNDS>(A.rk, A.rounds, (uint32_t)(tok + kS3CtaTokens) >> 4, c1, pos, seq, cw1);
      const float amax0 = group16_max(g0), amax1 = group16_max(g1);
      const float x0 = fmaf(amax0, c2, nm8), x1 = fmaf(amax1, c2, nm8);
      const bool wide0 = x0 > 0.f, wide1 = x1 > 0.f;
      const bool pass0 = any_zero_byte(cw0) | wide0, pass1 = any_zero_byte(cw1) | wide1;
      if (LSE) {
        lse16<DT>(g0, amax0, c2, lm, ls2);
        lse16<DT>(g1, amax1, c2, lm, ls2);
      }
      const unsigned long long mt = *m_tag;
      const uint32_t m_new = ((uint32_t)(mt >> 32) == tag) ? (uint32_t)mt : 0u;
      const unsigned bal0 = __ballot_sync(0xffffffffu, pass0);
      const unsigned bal1 = __ballot_sync(0xffffffffu, pass1);
      if (pass0) {
        uint32_t* e = queue + (qn + __popc(bal0 & ((1u << lane) - 1u))) * S3Entry<DT>::kWords;
        const uint32_t kb = wide0 ? (uint32_t)min(15, __float2int_ru(x0)) : 0u;
        *reinterpret_cast<uint4*>(e) = make_uint4(cw0[0], cw0[1], cw0[2], cw0[3]);
        e[4] = ((uint32_t)tok >> 4) | (kb << 28);
        store_group16(e + 8, g0);
      }
      qn += __popc(bal0);
      if (pass1) {
        uint32_t* e = queue + (qn + __popc(bal1 & ((1u << lane) - 1u))) * S3Entry<DT>::kWords;
        const uint32_t kb = wide1 ? (uint32_t)min(15, __float2int_ru(x1)) : 0u;
        *reinterpret_cast<uint4*>(e) = make_uint4(cw1[0], cw1[1], cw1[2], cw1[3]);
        e[4] = ((uint32_t)(tok + kS3CtaTokens) >> 4) | (kb << 28);
        store_group16(e + 8, g1);
      }
      qn += __popc(bal1);
      if (m_new > m_enc) {
        m_enc = m_new;
        nm8 = filter_offset(dec_ordered(m_enc)) + 8.0f;
      }
    };

    // ---- fused multi-stream race (Sec. 5.1 encoder: Y = argmin over tokens AND streams of
    //      S_i^(k) / weight_i): the group is loaded, maximised and summed once, then each of the
    //      multi_k noise streams takes its turn as one step of the inner loop.
    if constexpr (MULTI) {
      const int ns = A.multi_k;
      const uint32_t smask = A.kmask;
      const char* p = rowp + (size_t)tok0 * ES;
      int tok = tok0;
      int it = 0, st = 0;
      G g;
      float amax = 0.f;
      for (;;) {
#pragma unroll 1
        while (it < n_iter && qn < 32) {
          if (st == 0) {
            if (it < n_full) load16_vec(g, p);
            else load16_scalar(g, rowp, tok, tok_end);
            amax = group16_max(g);
            if (LSE) lse16<DT>(g, amax, c2, lm, ls2);
          }
          uint32_t cw[4];
          philox4x32<ROUNDS>(A.rk, A.rounds, (uint32_t)tok >> 4, c1 + ((uint32_t)st & smask), pos, seq, cw);
          const float x = fmaf(amax, c2, nm8);
          const bool wide = x > 0.f;
          const bool pass = any_zero_byte(cw) | wide;
          const unsigned long long mt = *m_tag;
          const uint32_t m_new = ((uint32_t)(mt >> 32) == tag) ? (uint32_t)mt : 0u;
          const unsigned bal = __ballot_sync(0xffffffffu, pass);
          if (pass) {
            uint32_t* e = queue + (qn + __popc(bal & ((1u << lane) - 1u))) * S3Entry<DT>::kWords;
            const uint32_t kb = wide ? (uint32_t)min(15, __float2int_ru(x)) : 0u;
            *reinterpret_cast<uint4*>(e) = make_uint4(cw[0], cw[1], cw[2], cw[3]);
            e[4] = ((uint32_t)tok >> 4) | (kb << 28);
            e[5] = (uint32_t)st & smask;
            store_group16(e + 8, g);
          }
          qn += __popc(bal);
          if (m_new > m_enc) {
            m_enc = m_new;
            nm8 = filter_offset(dec_ordered(m_enc)) + 8.0f;
          }
          if (++st == ns) {
            st = 0;
            ++it;
            p += STEP;
            tok += kS3CtaTokens;
          }
        }
        if (qn < 32) break;
        __syncwarp();
        qn -= 32;
        const uint32_t e = s3_flush<DT, ROUNDS, MULTI>(A.rounds, qn, 32, nm8 - 8.0f);
        if (e > m_enc) {
          m_enc = e;
          nm8 = filter_offset(dec_ordered(m_enc)) + 8.0f;
          if (lane == 0)
            atomicMax((unsigned long long*)&sh.m_tag, ((unsigned long long)tag << 32) | e);
        }
      }
    } else
    // ---- the sweep.  The inner loop runs until 32 groups are queued; the batched evaluation is
    //      called from the outer loop so that the inner loop carries no call (its state would
    //      otherwise be spilled around the call on every iteration).  One call site serves full
    //      (vector) and ragged (scalar) iterations; with PREFETCH the next group's load is issued
    //      before the current one is used.
    {
      const char* p = rowp + (size_t)tok0 * ES;
      int tok = tok0;
      int it = 0;
      constexpr bool PAIR = DT == kBF16;
      G nxt, nxt1;
      if (PAIR) {
        if (n_full >= 2) {
          load16_vec(nxt, p);
          load16_vec(nxt1, p + STEP);
        }
      } else if (PREFETCH && n_full > 0) {
        load16_vec(nxt, p);
      }
      for (;;) {
        if (PAIR) {
          // pairs of full iterations, the next pair's loads in flight
#pragma unroll 1
          for (; it + 2 <= n_full && qn < 32; it += 2) {
            const G g0 = nxt, g1 = nxt1;
            if (it + 4 <= n_full) {
              load16_vec(nxt, p + 2 * STEP);
              load16_vec(nxt1, p + 3 * STEP);
            }
            process2(g0, g1, tok);
            p += 2 * STEP;
            tok += 2 * kS3CtaTokens;
          }
          // what is left: at most one full iteration, then the ragged ones
#pragma unroll 1
          for (; it + 2 > n_full && it < n_iter && qn < 32; ++it) {
            G g;
            if (it < n_full) load16_vec(g, p);
            else load16_scalar(g, rowp, tok, tok_end);
            process(g, tok);
            p += STEP;
            tok += kS3CtaTokens;
          }
        } else {
#pragma unroll 1
          for (; it < n_iter && qn < 32; ++it) {
            G g;
            if (it < n_full) {
              if (PREFETCH) {
                g = nxt;
                if (it + 1 < n_full) load16_vec(nxt, p + STEP);
              } else {
                load16_vec(g, p);
              }
            } else {
              load16_scalar(g, rowp, tok, tok_end);
            }
            process(g, tok);
            p += STEP;
            tok += kS3CtaTokens;
          }
        }
        if (qn < 32) break;
        __syncwarp();
        const int nb = min(qn, 32);
        qn -= nb;
        const uint32_t e = s3_flush<DT, ROUNDS, MULTI>(A.rounds, qn, nb, nm8 - 8.0f);
        if (e > m_enc) {
          m_enc = e;
          nm8 = filter_offset(dec_ordered(m_enc)) + 8.0f;
          if (lane == 0)
            atomicMax((unsigned long long*)&sh.m_tag, ((unsigned long long)tag << 32) | e);
        }
      }
    }
    // ---- drain the queue ---------------------------------------------------------------------
    if (qn > 0) {
      __syncwarp();
      const uint32_t e = s3_flush<DT, ROUNDS, MULTI>(A.rounds, 0, qn, nm8 - 8.0f);
      if (e > m_enc) m_enc = e;
      qn = 0;
    }

    // ---- combine the lanes; every warp writes its own partial result ---------------------------
    Top2 t2 = sh.best[threadIdx.x];
    top2_warp_merge(t2);
    float ls = 0.f;
    if (LSE) {
      float s0, s1;
      unpack_f32x2(ls2, s0, s1);
      if (__any_sync(0xffffffffu, !(s0 + s1 < CUDART_INF_F))) {  // NaN or +inf logits in the slice
        float rl, rs;
        lse_redo_careful<DT>(rowp, tok0, n_iter, tok_end, c2, &rl, &rs);
        lm = rl;
        s0 = rs;
        s1 = 0.f;
      }
      float wm = lm;
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, d));
      ls = (s0 + s1) * ex2_approx((lm - wm) * c2);
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, d);
      lm = wm;
    }
    if (lane == 0) {
      Partial pr;
      pr.s1 = t2.s1; pr.i1 = t2.i1; pr.s2 = t2.s2; pr.i2 = t2.i2;
      pr.lm = lm; pr.ls = ls; pr.pad0 = 0; pr.pad1 = 0;
      A.partials[((long long)row * A.splits + split) * kSweepWarps3 + warp] = pr;
      if (A.splits > 1 && m_enc > 0u) atomicMax(A.hints + row, m_enc);
    }
  }
}

}  // namespace gls
