// gls_kernels.cuh -- device code shared by every kernel of libgls (Philox4x32, the exact fp64
// noise and score, the top-2 tracker, the filter's margins) and the sweep for noise_spec 1, the
// literal "one uniform per token" reading of Sec. 3 of arXiv 2506.05632.
//
// One pass over each row of logits computes, per (row, vocabulary slice):
//   - the two best candidates of the Gumbel-max race  argmax_i (logit_i / T - ln S_i)
//     (Sec. 3 step 2 / Algorithm 1, log domain), with S_i generated in registers from the
//     counter-based generator described in include/gls.h;
//   - optionally the running (max, sum) of the row's softmax normaliser, needed where rows
//     with different normalisers meet in the min over k (Algorithm 2, the Y_j line).
//
// The sweep never evaluates a logarithm for a token that cannot win.  With m a lower bound on
// the row's final best score, token i can only matter if  S_i <= exp(logit_i/T - m), and
// S_i = -log1p(-v_i) >= v_i.  So per group of 8 consecutive tokens one test
// "min word < 2^(max logit * c - m')" decides, and only groups that pass look at their tokens one
// by one (fp32 score from the full word).  The filter has no false negatives (margins below), so
// the result equals a full evaluation.  (The default layout, noise_spec 4, has its own sweep in
// gls_sweep4.cuh.)
#pragma once
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

namespace gls {

// Range checks of the kernels' own indices, compiled in with -DGLS_DEBUG_BOUNDS (the tests run
// the small shapes once under it; the memory checker of the toolkit is not available on every
// installation).  A violated check records (site, value, limit) in a device word array, counts it,
// and the guarded access is skipped; nothing traps.  Without the option the macro only evaluates to
// true and costs nothing.
__device__ unsigned int g_bounds_fault[4];  // [0] count, [1] first site, [2] its value, [3] its limit
#ifdef GLS_DEBUG_BOUNDS
__device__ __forceinline__ bool bounds_ok(long long v, long long lo, long long hi, unsigned site) {
  if (v >= lo && v < hi) return true;
  if (atomicAdd(&g_bounds_fault[0], 1u) == 0u) {
    g_bounds_fault[1] = site;
    g_bounds_fault[2] = (unsigned)v;
    g_bounds_fault[3] = (unsigned)hi;
  }
  return false;
}
#define GLS_IN_RANGE(v, lo, hi, site) (::gls::bounds_ok((long long)(v), (long long)(lo), (long long)(hi), (site)))
#else
#define GLS_IN_RANGE(v, lo, hi, site) (true)
#endif

constexpr int kMaxK = 64;
constexpr int kWarpTokens = 256;  // tokens one warp consumes per iteration (8 per lane)
constexpr float kLog2e = 1.4426950408889634f;

enum : int { kF32 = 0, kBF16 = 1 };

// Published Philox4x32 constants (Salmon et al., SC'11).
constexpr uint32_t kPhiloxM0 = 0xD2511F53u;
constexpr uint32_t kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u;
constexpr uint32_t kPhiloxW1 = 0xBB67AE85u;

// Per (row, slice) result of the sweep: the two best fp32 scores with their tokens, and the
// slice's softmax statistics (lm = max logit seen, ls = sum 2^((logit - lm) * c)).
struct __align__(16) Partial {
  float s1;
  int i1;
  float s2;
  int i2;
  float lm;
  float ls;
  int pad0, pad1;
};

// Per row: exact (fp64) score of the winner, its token, and the row's log-sum-exp.
struct __align__(16) RowResult {
  double score;
  double lse;
  int idx;
  int pad0, pad1, pad2;
};

struct SweepArgs {
  const void* data;       // rows [B][K][J][V]
  long long sb, sk, sj;   // element strides
  int K, J, V;
  // Optional second set of rows (the fused draft + verify call): rows [rows1, rows) of the call
  // are rows [b][k][j] of `data2` with J2 positions per (b, k) and the temperature inv_t2; rows
  // [0, rows1) are those of `data`.  data2 == NULL: one set, rows1 == rows.
  const void* data2;
  long long sb2, sk2, sj2;
  int J2, rows1;
  float inv_t2;
  int chunk;              // tokens per slice
  int splits;             // slices per row
  int parts;              // partial-result slots per row (slices x producers per slice)
  int parts1, parts2;     // slots in use per row of the first / second set (0: all of them)
  int rows;               // B * K * J
  int multi_k;            // > 0: one race per row over this many noise streams (fused encoder)
  long long n_items;      // row_count * splits
  int row_begin, row_count;  // the rows this launch sweeps: [row_begin, row_begin + row_count)
  float inv_t[kMaxK];     // 1/T per k
  uint32_t rk[32];        // Philox round keys: rk[2r], rk[2r+1]
  int rounds;
  uint32_t seq_base;
  const uint32_t* seq_ids;
  uint32_t pos_base;
  uint32_t domain;        // 0 decoding, 1 compression
  uint32_t kmask;         // 0xffff, or 0 when every k shares the noise of k = 0
  const uint8_t* bins;    // NULL, or candidate labels
  long long bins_sb;
  const uint8_t* msg;     // [B] label a candidate must carry (decoder side)
  // Rows that are computed, not read (compression from the source, Appendix C with the Gaussian
  // model of Appendix D.3): candidates gu [N][gD], sources ga [B][gD], side information
  // gt [B][K][gD]; gu == NULL otherwise.  g_dec: the rows are decoder rows (b, k), else encoder
  // rows b.
  const float* gu;
  const float* ga;
  const float* gt;
  int gD, g_dec;
  double g_s2_eta, g_s2_zeta, g_s2_prior;
  uint32_t* hints;        // [rows] ordered-int encoding of a lower bound on the row's best score
  Partial* partials;      // [n_items]
};

// ------------------------------------------------------------------------------------------
// small helpers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));  // a NaN operand is ignored
  return d;
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

__device__ __forceinline__ uint4 ld_stream16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// order-preserving map float -> uint32 (for atomicMax); 0 decodes to -inf
__device__ __forceinline__ uint32_t enc_ordered(float f) {
  uint32_t b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float dec_ordered(uint32_t e) {
  if (e <= 0x007fffffu) return -CUDART_INF_F;  // at or below the code of -inf (0 = never written)
  uint32_t b = (e & 0x80000000u) ? (e & 0x7fffffffu) : ~e;
  return __uint_as_float(b);
}

// ------------------------------------------------------------------------------------------
// Philox4x32: (c0,c1,c2,c3) <- (hi(M1 c2)^c1^k0, lo(M1 c2), hi(M0 c0)^c3^k1, lo(M0 c0)) per round,
// round keys precomputed on the host.
// ------------------------------------------------------------------------------------------
template <int ROUNDS>
__device__ __forceinline__ void philox4x32(const uint32_t* __restrict__ rk, int rounds_rt,
                                           uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                           uint32_t (&out)[4]) {
  const int n = ROUNDS > 0 ? ROUNDS : rounds_rt;
#pragma unroll
  for (int r = 0; r < n; ++r) {
    const unsigned long long p0 = (unsigned long long)kPhiloxM0 * c0;
    const unsigned long long p1 = (unsigned long long)kPhiloxM1 * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ rk[2 * r];
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ rk[2 * r + 1];
    c1 = (uint32_t)p1;
    c3 = (uint32_t)p0;
    c0 = n0;
    c2 = n2;
  }
  out[0] = c0;
  out[1] = c1;
  out[2] = c2;
  out[3] = c3;
}

// Identity of one noise stream: everything of the counter except the token block.
struct StreamKey {
  uint32_t c1;  // k | domain << 16
  uint32_t pos;
  uint32_t seq;
};

// The uniform of token i under noise_spec 1: v = (word + 0.5) * 2^-32.
template <int ROUNDS>
__device__ __forceinline__ double uniform_exact(const SweepArgs& A, const StreamKey& sk, int i) {
  uint32_t o[4];
  philox4x32<ROUNDS>(A.rk, A.rounds, (uint32_t)i >> 2, sk.c1, sk.pos, sk.seq, o);
  const uint32_t t = (uint32_t)i & 3u;
  const uint32_t w = t == 0 ? o[0] : t == 1 ? o[1] : t == 2 ? o[2] : o[3];
  return ((double)w + 0.5) * 0x1p-32;
}

// The exponential S_i of token i in fp64.  noise_spec 1: S = -log1p(-v) (Sec. 3: S = -ln U,
// U = 1 - v).  noise_spec 4: the group of 16 is built from its minimum M = -log1p(-v0) / 16,
// v0 = (w * 2^16 + r + 0.5) * 2^-48: S = M at position loc of the group, M - log1p(-v_i) at the
// others, v_i = (u_i + 0.5) * 2^-32 (an exact sampler of 16 i.i.d. Exp(1) values).
template <int SPEC, int ROUNDS>
__device__ __forceinline__ double noise_exact(const SweepArgs& A, const StreamKey& sk, int i) {
  if (SPEC != 4) return -log1p(-uniform_exact<ROUNDS>(A, sk, i));
  uint32_t o[4];
  const uint32_t g = (uint32_t)i >> 4;
  philox4x32<ROUNDS>(A.rk, A.rounds, ((g >> 7) << 5) | (g & 31u), sk.c1, sk.pos, sk.seq, o);
  const uint32_t j = (g >> 5) & 3u;
  const uint32_t w = j == 0 ? o[0] : j == 1 ? o[1] : j == 2 ? o[2] : o[3];
  philox4x32<ROUNDS>(A.rk, A.rounds, g, sk.c1 + (2u << 16), sk.pos, sk.seq, o);
  const uint32_t r = o[0] & 0xffffu, loc = (o[0] >> 16) & 15u;
  const double m = -log1p(-((double)w * 65536.0 + (double)r + 0.5) * 0x1p-48) / 16.0;
  if (((uint32_t)i & 15u) == loc) return m;
  philox4x32<ROUNDS>(A.rk, A.rounds, (uint32_t)i >> 2, sk.c1 + (4u << 16), sk.pos, sk.seq, o);
  const uint32_t t = (uint32_t)i & 3u;
  const uint32_t u = t == 0 ? o[0] : t == 1 ? o[1] : t == 2 ? o[2] : o[3];
  return m + (-log1p(-((double)u + 0.5) * 0x1p-32));
}

// Where row `row` of the call lives and which (b, k, j) it is.
struct RowLoc {
  const char* rowp;
  int b, k, j;
  float inv_t;
  bool second;
};
template <int ES>
__device__ __forceinline__ RowLoc locate_row(const SweepArgs& A, int row) {
  RowLoc r;
  r.second = A.data2 != nullptr && row >= A.rows1;
  const int rr = r.second ? row - A.rows1 : row;
  const int J = r.second ? A.J2 : A.J;
  r.j = rr % J;
  const int bk = rr / J;
  r.k = bk % A.K;
  r.b = bk / A.K;
  if (r.second) {
    r.rowp = (const char*)A.data2 + (r.b * A.sb2 + r.k * A.sk2 + r.j * A.sj2) * ES;
    r.inv_t = A.inv_t2;
  } else {
    r.rowp = (const char*)A.data + (r.b * A.sb + r.k * A.sk + r.j * A.sj) * ES;
    r.inv_t = A.inv_t[r.k];
  }
  return r;
}

template <int DT>
__device__ __forceinline__ float load_logit(const void* row, long long i) {
  if (DT == kF32) return __ldg((const float*)row + i);
  return __uint_as_float((uint32_t)__ldg((const unsigned short*)row + i) << 16);
}

// Importance log-weight of candidate i for source sample b (decoder k if A.g_dec) in fp64
// (Appendix C; Gaussian model of Appendix D.3 per dimension; terms common to a row dropped):
//   encoder  sum_d -(u - a)^2 / (2 s2_eta) + u^2 / (2 s2_prior)
//   decoder  sum_d -(u - t / s2_T)^2 / (2 (s2_W - 1 / s2_T)) + u^2 / (2 s2_prior)
__device__ __forceinline__ double gauss_logw64(const SweepArgs& A, int b, int k, long long i) {
  const double s2T = 1.0 + A.g_s2_zeta, s2W = 1.0 + A.g_s2_eta;
  const double var = A.g_dec ? s2W - 1.0 / s2T : A.g_s2_eta;
  const float* mu = A.g_dec ? A.gt + ((long long)b * A.K + k) * A.gD : A.ga + (long long)b * A.gD;
  const float* u = A.gu + i * A.gD;
  double acc = 0.0;
  for (int d = 0; d < A.gD; ++d) {
    const double x = (double)__ldg(u + d);
    const double m = A.g_dec ? (double)__ldg(mu + d) / s2T : (double)__ldg(mu + d);
    const double diff = x - m;
    acc += -(diff * diff) / (2.0 * var) + (x * x) / (2.0 * A.g_s2_prior);
  }
  return acc;
}

// Exact score of one token in fp64: logit/T - ln S, S = -log1p(-v)  (Sec. 3: S = -ln U, U = 1 - v).
// (b, k) are only used for rows that are computed from the source.
template <int DT, int SPEC, int ROUNDS>
__device__ __noinline__ double exact_score(const SweepArgs& A, const void* row,
                                           const StreamKey& sk, int i, float inv_t, int b, int k) {
  const double a = A.gu != nullptr ? gauss_logw64(A, b, k, i)
                                   : (double)load_logit<DT>(row, i) * (double)inv_t;
  return a - log(noise_exact<SPEC, ROUNDS>(A, sk, i));
}

// Exp(1) from the uniform v = (word + frac) * 2^-32, frac in (0, 1) standing for further bits
// and the half-step offset: -log1p(-v), through the complement 1 - v = (~word + 1 - frac) * 2^-32
// when v > 1/2, so that the conversion of the word to fp32 can never round v up to 1.
__device__ __forceinline__ float exp1_from_word(uint32_t word, float frac) {
  if (word & 0x80000000u) return -logf(fmaf((float)(~word), 0x1p-32f, (1.0f - frac) * 0x1p-32f));
  return -log1pf(-fmaf((float)word, 0x1p-32f, frac * 0x1p-32f));
}

// fp32 score from the exponential; |error| is well below score_slack().
__device__ __forceinline__ float score_f32(float a, float inv_t, float s_noise, float* ln_s) {
  const float l = logf(s_noise);
  *ln_s = l;
  return fmaf(a, inv_t, -l);
}
// Bound on |fp32 score - exact score| used to (a) keep the filter's running bound below the
// truth and (b) decide when two candidates must be re-evaluated in fp64.
__device__ __forceinline__ float score_slack(float s, float ln_s) {
  return 0x1p-17f * (1.0f + fabsf(s) + fabsf(ln_s));
}

// Exponent offset of the filter for a running lower bound m on the best score (natural-log
// units): a token passes iff coarse(v) < 2^(logit * c + nm).  The margin covers the rounding of
// c, of the fma and of ex2.approx (together < 1e-5 for |logit * c| < 2^10), so no token whose
// exact score reaches m is ever rejected.
__device__ __forceinline__ float filter_offset(float m) {
  if (m == -CUDART_INF_F) return CUDART_INF_F;
  const float ml = m * kLog2e;
  return fmaf(fabsf(ml), 0x1p-20f, 0x1p-12f) - ml;
}

struct Top2 {
  float s1;
  int i1;
  float s2;
  int i2;
};
__device__ __forceinline__ void top2_init(Top2& t) {
  t.s1 = -CUDART_INF_F;
  t.i1 = -1;
  t.s2 = -CUDART_INF_F;
  t.i2 = -1;
}
// order: score descending, then token ascending
__device__ __forceinline__ bool beats(float s, int i, float s0, int i0) {
  return i0 < 0 || s > s0 || (s == s0 && i < i0);
}
__device__ __forceinline__ void top2_offer(Top2& t, float s, int i) {
  if (i < 0 || i == t.i1 || i == t.i2) return;  // the two leaders are distinct candidates
  if (beats(s, i, t.s1, t.i1)) {
    t.s2 = t.s1;
    t.i2 = t.i1;
    t.s1 = s;
    t.i1 = i;
  } else if (beats(s, i, t.s2, t.i2)) {
    t.s2 = s;
    t.i2 = i;
  }
}
__device__ __forceinline__ void top2_warp_merge(Top2& t) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) {
    const float os1 = __shfl_xor_sync(0xffffffffu, t.s1, d);
    const int oi1 = __shfl_xor_sync(0xffffffffu, t.i1, d);
    const float os2 = __shfl_xor_sync(0xffffffffu, t.s2, d);
    const int oi2 = __shfl_xor_sync(0xffffffffu, t.i2, d);
    top2_offer(t, os1, oi1);
    top2_offer(t, os2, oi2);
  }
}

// ------------------------------------------------------------------------------------------
// Per-token examination of one lane's group of 8 tokens (rare path).
//   a[8]   logits (excluded / out-of-range tokens hold -inf)
//   w[8]   the tokens' generator words
// ------------------------------------------------------------------------------------------
template <int ROUNDS>
__device__ __noinline__ void examine_group(int tok0, const float (&a)[8], const uint32_t* w,
                                           float inv_t, float c2, float m, const uint8_t* bins,
                                           int msg, Top2& best) {
  float nm = filter_offset(m);
#pragma unroll 1
  for (int t = 0; t < 8; ++t) {
    const float at = a[t];
    if (!(at < CUDART_INF_F)) continue;  // NaN and +inf never win
    const float thr = ex2_approx(fmaf(at, c2, nm));
    const uint32_t wt = w[t];
    if (!(__uint2float_rd(wt) < thr * 4294967296.0f)) continue;
    const int i = tok0 + t;
    if (bins != nullptr && (int)__ldg(bins + i) != msg) continue;
    float ln_s;
    const float s = score_f32(at, inv_t, exp1_from_word(wt, 0.5f), &ln_s);
    top2_offer(best, s, i);
    const float lower = s - score_slack(s, ln_s);
    if (lower > m) {
      m = lower;
      nm = filter_offset(m);
    }
  }
}

// running lower bound implied by a lane's best candidate
__device__ __forceinline__ float lane_bound(const Top2& t) {
  if (t.i1 < 0) return -CUDART_INF_F;
  // ln S is not kept; |ln S| <= 34 for v >= 2^-49, use that worst case
  return t.s1 - 0x1p-17f * (35.0f + fabsf(t.s1));
}

// ------------------------------------------------------------------------------------------
// The sweep.  Each warp owns work items (row, slice); per iteration a lane takes 8 consecutive
// tokens (one 16-byte load of bf16, two of fp32), so a warp reads 512 B / 1 KB contiguous.
// ------------------------------------------------------------------------------------------
constexpr int kSweepThreads = 256;

template <int DT>
struct Group {
  uint4 q0, q1;  // q1 only used by fp32
};

template <int DT>
__device__ __forceinline__ Group<DT> load_group_vec(const char* rowp, int tok) {
  Group<DT> g;
  if (DT == kBF16) {
    g.q0 = ld_stream16(rowp + (size_t)tok * 2);
    g.q1 = make_uint4(0, 0, 0, 0);
  } else {
    g.q0 = ld_stream16(rowp + (size_t)tok * 4);
    g.q1 = ld_stream16(rowp + (size_t)tok * 4 + 16);
  }
  return g;
}

// scalar loader for ragged tails and rows that are not 16-byte aligned; out-of-range -> -inf
template <int DT>
__device__ __forceinline__ Group<DT> load_group_scalar(const char* rowp, int tok, int V) {
  Group<DT> g;
  uint32_t e[8];
#pragma unroll
  for (int t = 0; t < 8; ++t) {
    const int i = tok + t;
    if (DT == kBF16)
      e[t] = i < V ? (uint32_t)__ldg((const unsigned short*)rowp + i) : 0xff80u;
    else
      e[t] = i < V ? __float_as_uint(__ldg((const float*)rowp + i)) : 0xff800000u;
  }
  if (DT == kBF16) {
    g.q0 = make_uint4(e[0] | (e[1] << 16), e[2] | (e[3] << 16), e[4] | (e[5] << 16),
                      e[6] | (e[7] << 16));
    g.q1 = make_uint4(0, 0, 0, 0);
  } else {
    g.q0 = make_uint4(e[0], e[1], e[2], e[3]);
    g.q1 = make_uint4(e[4], e[5], e[6], e[7]);
  }
  return g;
}

template <int DT>
__device__ __forceinline__ void unpack_group(const Group<DT>& g, float (&a)[8]) {
  if (DT == kBF16) {
    a[0] = bf16_lo(g.q0.x); a[1] = bf16_hi(g.q0.x);
    a[2] = bf16_lo(g.q0.y); a[3] = bf16_hi(g.q0.y);
    a[4] = bf16_lo(g.q0.z); a[5] = bf16_hi(g.q0.z);
    a[6] = bf16_lo(g.q0.w); a[7] = bf16_hi(g.q0.w);
  } else {
    a[0] = __uint_as_float(g.q0.x); a[1] = __uint_as_float(g.q0.y);
    a[2] = __uint_as_float(g.q0.z); a[3] = __uint_as_float(g.q0.w);
    a[4] = __uint_as_float(g.q1.x); a[5] = __uint_as_float(g.q1.y);
    a[6] = __uint_as_float(g.q1.z); a[7] = __uint_as_float(g.q1.w);
  }
}

// max over the group, ignoring NaN
template <int DT>
__device__ __forceinline__ float group_max(const Group<DT>& g) {
  if (DT == kBF16) {
    const uint32_t x = max_bf16x2(max_bf16x2(g.q0.x, g.q0.y), max_bf16x2(g.q0.z, g.q0.w));
    return fmaxf(bf16_lo(x), bf16_hi(x));
  } else {
    const float x0 = fmaxf(fmaxf(__uint_as_float(g.q0.x), __uint_as_float(g.q0.y)),
                           fmaxf(__uint_as_float(g.q0.z), __uint_as_float(g.q0.w)));
    const float x1 = fmaxf(fmaxf(__uint_as_float(g.q1.x), __uint_as_float(g.q1.y)),
                           fmaxf(__uint_as_float(g.q1.z), __uint_as_float(g.q1.w)));
    return fmaxf(x0, x1);
  }
}

// Softmax statistics of one group: lm = running max, ls = sum 2^((a - lm) * c2).
// Fast path assumes finite-or-(-inf) logits; anything else is redone token by token.
__device__ __forceinline__ void lse_group(const float (&a)[8], float amax, float c2, float& lm,
                                          float& ls) {
  bool careful = false;
  if (amax > lm) {
    if (amax == CUDART_INF_F) {
      careful = true;
    } else {
      ls *= ex2_approx((lm - amax) * c2);
      lm = amax;
    }
  }
  float gs = 0.f;
  if (!careful) {
#pragma unroll
    for (int t = 0; t < 8; ++t) gs += ex2_approx((a[t] - lm) * c2);
    careful = !(gs <= 16.0f);  // a NaN logit poisons the sum
  }
  if (careful) {
    float vmax = -CUDART_INF_F;
#pragma unroll
    for (int t = 0; t < 8; ++t)
      if (a[t] < CUDART_INF_F) vmax = fmaxf(vmax, a[t]);  // false for NaN and +inf
    if (vmax > lm) {
      ls *= ex2_approx((lm - vmax) * c2);
      lm = vmax;
    }
    gs = 0.f;
#pragma unroll
    for (int t = 0; t < 8; ++t)
      if (a[t] < CUDART_INF_F) gs += ex2_approx((a[t] - lm) * c2);
  }
  ls += gs;
}

constexpr float kLseFloor = -3.0e38f;  // finite stand-in for "no finite logit seen yet"

template <int DT, bool LSE, int ROUNDS>
__global__ void __launch_bounds__(kSweepThreads, 4)
sweep_kernel(const __grid_constant__ SweepArgs A) {
  const int lane = threadIdx.x & 31;
  const long long warp0 = (long long)blockIdx.x * (kSweepThreads / 32) + (threadIdx.x >> 5);
  const long long nwarps = (long long)gridDim.x * (kSweepThreads / 32);
  constexpr int ES = DT == kBF16 ? 2 : 4;

  for (long long item = warp0; item < A.n_items; item += nwarps) {
    const int row = (int)(item / A.splits);
    const int split = (int)(item - (long long)row * A.splits);
    const int j = row % A.J;
    const int bk = row / A.J;
    const int k = bk % A.K;
    const int b = bk / A.K;
    const char* rowp = (const char*)A.data + (b * A.sb + k * A.sk + j * A.sj) * ES;
    StreamKey sk;
    sk.c1 = ((uint32_t)k & A.kmask) | (A.domain << 16);
    sk.pos = A.pos_base + (uint32_t)j;
    sk.seq = A.seq_ids ? __ldg(A.seq_ids + b) : A.seq_base + (uint32_t)b;
    const float inv_t = A.inv_t[k];
    const float c2 = inv_t * kLog2e;
    const uint8_t* bins = A.bins ? A.bins + A.bins_sb * b : nullptr;
    const int msg = (A.bins && A.msg) ? (int)__ldg(A.msg + b) : 0;
    const int tok_begin = split * A.chunk;
    const int tok_end = min(A.V, tok_begin + A.chunk);
    const bool aligned = (((uintptr_t)rowp) & 15) == 0;
    // iterations whose 256 tokens are all in range can use vector loads
    const int n_full = aligned ? (tok_end - tok_begin) / kWarpTokens : 0;
    const int n_iter = (tok_end - tok_begin + kWarpTokens - 1) / kWarpTokens;

    float m = dec_ordered(__ldcg(A.hints + row));  // best lower bound published so far
    float nm = filter_offset(m);
    Top2 best;
    top2_init(best);
    float lm = kLseFloor, ls = 0.f;

    Group<DT> cur, nxt;
    int tok = tok_begin + lane * 8;
    if (n_full > 0) cur = load_group_vec<DT>(rowp, tok);
    for (int it = 0; it < n_iter; ++it, tok += kWarpTokens) {
      const bool full = it < n_full;
      if (!full) cur = load_group_scalar<DT>(rowp, tok, tok_end);
      if (it + 1 < n_full) nxt = load_group_vec<DT>(rowp, tok + kWarpTokens);

      // the group's eight generator words and the smallest of them
      uint32_t w[8];
      {
        uint32_t o[4];
        philox4x32<ROUNDS>(A.rk, A.rounds, (uint32_t)tok >> 2, sk.c1, sk.pos, sk.seq, o);
        w[0] = o[0]; w[1] = o[1]; w[2] = o[2]; w[3] = o[3];
        philox4x32<ROUNDS>(A.rk, A.rounds, ((uint32_t)tok >> 2) + 1u, sk.c1, sk.pos, sk.seq, o);
        w[4] = o[0]; w[5] = o[1]; w[6] = o[2]; w[7] = o[3];
      }
      const uint32_t wm = min(min(min(w[0], w[1]), min(w[2], w[3])),
                              min(min(w[4], w[5]), min(w[6], w[7])));
      const float vlow = __uint2float_rd(wm);  // lower bound on 2^32 min_t v_t
      const float amax = group_max<DT>(cur);
      const float thr = ex2_approx(fmaf(amax, c2, nm)) * 4294967296.0f;
      const bool pass = vlow < thr;

      if (LSE) {
        float a[8];
        unpack_group<DT>(cur, a);
        lse_group(a, amax, c2, lm, ls);
      }

      if (__any_sync(0xffffffffu, pass)) {
        if (pass) {
          float a[8];
          unpack_group<DT>(cur, a);
          examine_group<ROUNDS>(tok, a, w, inv_t, c2, m, bins, msg, best);
        }
        // share the improved bound with the warp and with the other slices of the row
        float mb = lane_bound(best);
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) mb = fmaxf(mb, __shfl_xor_sync(0xffffffffu, mb, d));
        if (mb > m) {
          m = mb;
          if (lane == 0) atomicMax(A.hints + row, enc_ordered(m));
        }
        const float mg = dec_ordered(__ldcg(A.hints + row));
        if (mg > m) m = mg;
        nm = filter_offset(m);
      } else if ((it & 15) == 15) {
        const float mg = dec_ordered(__ldcg(A.hints + row));
        if (mg > m) {
          m = mg;
          nm = filter_offset(m);
        }
      }
      cur = nxt;
    }

    // combine the lanes
    top2_warp_merge(best);
    if (LSE) {
      float wm = lm;
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, d));
      float s = ls * ex2_approx((lm - wm) * c2);
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) s += __shfl_xor_sync(0xffffffffu, s, d);
      lm = wm;
      ls = s;
    }
    if (lane == 0) {
      Partial p;
      p.s1 = best.s1; p.i1 = best.i1; p.s2 = best.s2; p.i2 = best.i2;
      p.lm = lm; p.ls = ls; p.pad0 = 0; p.pad1 = 0;
      if (GLS_IN_RANGE(item, 0, A.n_items, 10u)) A.partials[item] = p;
    }
  }
}

}  // namespace gls
