// gls_sweep4.cuh -- the vocabulary sweep for noise_spec 4 (groups of 16 exponentials built from
// their minimum).
//
// Under noise_spec 4 the 16 tokens 16g .. 16g+15 of group g share one number M_g ~ Exp(16), the
// smallest of their 16 exponentials: S_i = M_g at one uniformly placed token and M_g + Exp(1) at
// the other fifteen -- an exact sampler of 16 i.i.d. Exp(1) values (memorylessness), i.e. of
// Sec. 3's S_i = -ln U_i of arXiv 2506.05632.  One Philox4x32 call yields the 32 coarse bits w of
// M for FOUR groups, so the generator -- whose 32x32->64-bit multiplies are the scarcest
// resource of this path on sm_100a -- runs once per 64 tokens, and
//     S_i >= M_g = -log1p(-v0) / 16 >= v0 / 16 >= w * 2^-36        for every token of the group.
// With m a lower bound on the row's best score, a token can only matter if S_i <= exp(a_i - m)
// (a_i = logit_i / T), hence a group only if  w * 2^-32 <= 16 * exp(max a - m): a group maximum,
// two multiply-adds, an integer multiply-add and one compare per 16 tokens (the right-hand side
// is replaced by an upper bound that needs no ex2).  A few dozen groups per row pass.  They
// are not examined on the spot: the lane pushes (w, g) on a small per-warp queue in shared
// memory and the sweep goes on; when 32 groups are queued the warp evaluates them together, one
// group per lane (the 16 refinement bits and the position of the minimum from a second
// generator stream, a per-token test against M, and for the survivors their own Exp(1) from a
// third stream and the fp32 score a_i - ln S_i).  The filter has no false negatives, so the
// result equals a full evaluation (Sec. 3 step 2 / Algorithm 2 draft loop and Y_j line, log
// domain).
//
// Work decomposition: a work item is one (row, vocabulary slice), owned by one CTA.  Per step a
// warp takes 2048 contiguous tokens: lane l holds groups l, l + 32, l + 64, l + 96 of the step
// (four 32-byte loads of bf16, eight of fp32, each warp-wide load 1 KB contiguous), which are
// exactly the four groups served by its generator call.  Warps never wait on one another: they
// share the bound m through one tagged shared-memory word, each warp writes its own partial
// result, and the split-V reduction merges them.  The batched evaluation is called from an outer
// loop so that the hot loop contains no call.  A fused variant (MULTI) races one row under
// several noise streams at once for the compression encoder of Sec. 5.1.
#pragma once
#include "gls_group16.cuh"

namespace gls {

#ifndef GLS_S4_BF16_WARPS
#define GLS_S4_BF16_WARPS 1
#define GLS_S4_BF16_CTAS 16
#endif
#ifndef GLS_S4_BF16_PREFETCH
#define GLS_S4_BF16_PREFETCH 1
#endif
#ifndef GLS_S4_F32_WARPS
#define GLS_S4_F32_WARPS 8
#define GLS_S4_F32_CTAS 2
#endif
constexpr int kS4LaneGroups = 4;                                // groups per lane and step
constexpr int kS4WarpGroups = 32 * kS4LaneGroups;               // 128
constexpr int kS4WarpTokens = 16 * kS4WarpGroups;               // 2048
// Groups per warp queue: a batch is taken at 32 queued groups, and one step can add 128 more.
constexpr int kS4QueueCap = 32 + kS4WarpGroups;

// Launch shapes, chosen by measurement.  A lane holds its four groups in registers (32 for bf16,
// 64 for fp32); every shape runs under a 128-register budget.
//   shape 1, bf16 rows: the next step's loads are issued before the current step is used (32 more
//     registers), one warp per CTA and 16 CTAs per SM (at the time of the choice config 4 ran at
//     6.48 / 4.90 TB/s against 6.05 / 4.75 TB/s for 2 warps x 10 CTAs without the prefetch);
//   shape 0, fp32 rows of at least 2^19 tokens: 8 warps x 2 CTAs, no prefetch (config 5 decoders
//     6.58 TB/s against 5.96 TB/s for 1 x 16);
//   shape 2, shorter fp32 rows and the fused multi-stream race: 1 warp x 16 CTAs, so that a warp's
//     share of a row stays tens of steps long (rows of 128k tokens: 5.14 / 5.01 TB/s per draft /
//     target call against 4.62 / 4.24 TB/s for 8 x 2).
constexpr int kS4ShapeF32Wide = 0, kS4ShapeBf16 = 1, kS4ShapeF32Narrow = 2;
constexpr long long kS4WideMinTokens = 1LL << 19;
template <int SH>
struct S4Cfg {
  static constexpr int kDT = SH == kS4ShapeBf16 ? kBF16 : kF32;
  static constexpr int kWarps =
      SH == kS4ShapeBf16 ? GLS_S4_BF16_WARPS : SH == kS4ShapeF32Wide ? GLS_S4_F32_WARPS : 1;
  static constexpr int kCtasPerSM =
      SH == kS4ShapeBf16 ? GLS_S4_BF16_CTAS : SH == kS4ShapeF32Wide ? GLS_S4_F32_CTAS : 16;
  static constexpr int kCtaTokens = kWarps * kS4WarpTokens;
  // the next step's loads are issued before the current step is used (bf16: 32 more registers)
  static constexpr bool kPrefetch = SH == kS4ShapeBf16 ? (GLS_S4_BF16_PREFETCH != 0) : false;
};
constexpr int kS4MaxCtaTokens = 8 * kS4WarpTokens;

struct S4WarpCtx {  // what the batched path needs to know about the warp's current work item
  const char* rowp;
  const uint8_t* bins;
  uint32_t c1, pos, seq;
  uint32_t key0, key1;
  float inv_t;
  int msg, tok_end;
};
template <int SH>
struct S4Shared {
  unsigned long long m_tag;  // (item tag << 32) | ordered code of the CTA-wide bound on the best score
  S4WarpCtx ctx[S4Cfg<SH>::kWarps];
  Top2 best[S4Cfg<SH>::kWarps * 32];
  uint2 queue[S4Cfg<SH>::kWarps][kS4QueueCap];  // (coarse word, group | stream << 28)
};
template <int SH>
__device__ __forceinline__ S4Shared<SH>& s4_shared() {
  return *reinterpret_cast<S4Shared<SH>*>(gls_smem_raw);
}

// lower bound on word * 2^-32 from its top 23 bits, without an integer-to-float conversion
__device__ __forceinline__ float coarse_lower(uint32_t w) {
  return __uint_as_float(0x3f800000u | (w >> 9)) - 1.0f;
}

// An upper bound on 2^x without the special-function unit (which the log-sum-exp keeps busy):
// with xs = sat(x / 126 + 1) in [0, 1], i.e. x clamped to [-126, 0], the integer
// round(32768 (x clamped)) is placed in the low mantissa bits of a float by a magic-number
// multiply-add and moved into exponent and mantissa position by one integer multiply-add: the
// result is 2^floor(x) (1 + frac(x)) >= 2^x (the chord of a convex function), at most 6.2 % above
// it.  The caller passes x / 126 + 1 with x already raised by 2^-9 to cover the roundings (of
// c2 / 126, 2^-24 * 126 in xs, half a unit of 2^-15 in the integer).  NaN gives 2^-126.
__device__ __forceinline__ float exp2_upper_from_scaled(float amax, float c2s, float nms) {
  float xs;
  asm("fma.rn.sat.f32 %0, %1, %2, %3;" : "=f"(xs) : "f"(amax), "f"(c2s), "f"(nms));
  const float t = fmaf(xs, 4128768.0f, 12582912.0f - 4128768.0f);  // 126 * 32768; 1.5 * 2^23
  return __uint_as_float(__float_as_uint(t) * 256u + 0xff800000u);
}
// the second and third argument of exp2_upper_from_scaled for x = amax * c2 + nm4
__device__ __forceinline__ float scaled_offset(float nm4) {
  return fmaf(nm4 + 0x1p-9f, 1.0f / 126.0f, 1.0f + 0x1p-22f);
}

// generator call that serves group g (and g + 32, g + 64, g + 96 when g mod 128 < 32)
__device__ __forceinline__ uint32_t s4_call_index(uint32_t g) { return ((g >> 7) << 5) | (g & 31u); }

// ------------------------------------------------------------------------------------------
// Batched evaluation of queued groups: lane l < n takes entry first + l of its warp's queue.
// The lane draws the group's refinement bits and the position of its minimum, computes M, keeps
// the tokens with a_t - ln M above the bound (S_t >= M), and scores the survivors in fp32, one
// per round, drawing the token's own exponential unless it is the group's minimum.  Returns the
// best lower bound found (ordered code, 0 if none).
// ------------------------------------------------------------------------------------------
template <int SH, int ROUNDS, bool MULTI>
__device__ __noinline__ uint32_t s4_flush(int rounds_rt, int first, int n, float nm) {
  constexpr int DT = S4Cfg<SH>::kDT;
  S4Shared<SH>& sh = s4_shared<SH>();
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const S4WarpCtx cx = sh.ctx[warp];
  const float c2 = cx.inv_t * kLog2e;
  uint32_t msk = 0u, g = 0u, ks = 0u;
  int loc = -1;
  float M = 1.f;
  float lb = -CUDART_INF_F;
  if (lane < n) {
    const uint2 e = sh.queue[warp][GLS_IN_RANGE(first + lane, 0, kS4QueueCap, 25u) ? first + lane : 0];
    g = e.y;
    if (MULTI) {
      ks = g >> 28;
      g &= 0x0fffffffu;
    }
    uint32_t f[4];
    philox4x32_keyed<ROUNDS>(cx.key0, cx.key1, rounds_rt, g, cx.c1 + ks + (2u << 16), cx.pos, cx.seq, f);
    loc = (int)((f[0] >> 16) & 15u);
    M = exp1_from_word(e.x, ((float)(f[0] & 0xffffu) + 0.5f) * 0x1p-16f) * 0.0625f;
    // the token at the minimum has S = M exactly: its score is a lower bound for the row at once
    const int il = (int)(g << 4) + loc;
    if (il < cx.tok_end && (cx.bins == nullptr || (int)__ldg(cx.bins + il) == cx.msg)) {
      const float a = load_logit<DT>(cx.rowp, il);
      if (a < CUDART_INF_F) {  // false for NaN
        const float ln_s = logf(M);
        const float s = fmaf(a, cx.inv_t, -ln_s);
        lb = s - score_slack(s, ln_s);
      }
    }
  }
  nm = fminf(nm, filter_offset(dec_ordered(__reduce_max_sync(0xffffffffu, enc_ordered(lb)))));
  if (lane < n) {
    // token t can matter only if a_t c2 + nm - log2(M) >= 0 (S_t >= M); lg2.approx and the
    // rounding of M are good to 2^-20, the extra 2^-10 covers them
    const float nmM = nm - lg2_approx(M) + 0x1p-10f;
    const int i0 = (int)(g << 4);
#pragma unroll
    for (int t = 0; t < 16; ++t) {
      if (i0 + t < cx.tok_end) {
        const float a = load_logit<DT>(cx.rowp, i0 + t);
        if (a < CUDART_INF_F && fmaf(a, c2, nmM) >= 0.f) msk |= 1u << t;  // false for NaN
      }
    }
  }
  Top2 b = sh.best[threadIdx.x];
  float lower = -CUDART_INF_F;
  while (__any_sync(0xffffffffu, msk != 0u)) {
    if (msk != 0u) {
      const int t = __ffs(msk) - 1;
      msk &= msk - 1u;
      const int i = (int)(g << 4) + t;
      if (cx.bins == nullptr || (int)__ldg(cx.bins + i) == cx.msg) {
        const float a = load_logit<DT>(cx.rowp, i);
        float s_noise = M;
        if (t != loc) {
          uint32_t f[4];
          philox4x32_keyed<ROUNDS>(cx.key0, cx.key1, rounds_rt, (uint32_t)i >> 2,
                                   cx.c1 + ks + (4u << 16), cx.pos, cx.seq, f);
          const uint32_t u = (i & 2) ? ((i & 1) ? f[3] : f[2]) : ((i & 1) ? f[1] : f[0]);
          s_noise = M + exp1_from_word(u, 0.5f);
        }
        const float ln_s = logf(s_noise);
        const float s = fmaf(a, cx.inv_t, -ln_s);
        // fused race: the candidate is (token, stream), ordered by token first
        top2_offer(b, s, MULTI ? (int)(((uint32_t)i << 3) | ks) : i);
        lower = fmaxf(lower, s - score_slack(s, ln_s));
      }
    }
  }
  sh.best[threadIdx.x] = b;
  __syncwarp();
  return __reduce_max_sync(0xffffffffu, enc_ordered(lower));
}

// The lane's share of a work item again for the softmax sum, token by token, leaving out NaN and
// +inf logits (they cannot define a probability).  Rare: only rows that hold such values.
template <int SH>
__device__ __noinline__ void lse4_redo_careful(const char* rowp, int tok0, int n_steps, int tok_end,
                                               float c2, float* lm_out, float* ls_out) {
  constexpr int DT = S4Cfg<SH>::kDT;
  float lm = kGroupLseFloor, ls = 0.f;
  for (int s = 0; s < n_steps; ++s) {
    for (int j = 0; j < kS4LaneGroups; ++j) {
      const int tok = tok0 + s * S4Cfg<SH>::kCtaTokens + j * 512;
      for (int t = 0; t < 16; ++t) {
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
  }
  *lm_out = lm;
  *ls_out = ls;
}

// ------------------------------------------------------------------------------------------
// The kernel
// ------------------------------------------------------------------------------------------
// One work item: slice `split` of row `row`, swept by the calling CTA; rows are cut into `splits`
// slices of `chunk` tokens.
template <int SH, bool LSE, int ROUNDS, bool MULTI>
__device__ __forceinline__ void s4_item(const SweepArgs& A, int row, int split, uint32_t tag,
                                        const int chunk, const int splits) {
  constexpr int DT = S4Cfg<SH>::kDT;
  S4Shared<SH>& sh = s4_shared<SH>();
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  constexpr int ES = DT == kBF16 ? 2 : 4;
  constexpr int kWarps = S4Cfg<SH>::kWarps;
  constexpr int kCtaTokens = S4Cfg<SH>::kCtaTokens;
  typedef Group16<DT> G;
  uint2* const queue = sh.queue[warp];
  volatile unsigned long long* const m_tag = &sh.m_tag;
  {
    const int tok_begin = split * chunk;  // a multiple of 2048
    const int tok_end = min(A.V, tok_begin + chunk);
    uint32_t c1, pos, seq;
    const char* rowp;
    float c2;
    {
      const RowLoc rl = locate_row<ES>(A, row);
      const int j = rl.j, k = rl.k, b = rl.b;
      rowp = rl.rowp;
      // the fused multi-stream race enumerates the streams itself, whatever the row's k
      c1 = (MULTI ? 0u : ((uint32_t)k & A.kmask)) | (A.domain << 16);
      pos = A.pos_base + (uint32_t)j;
      seq = A.seq_ids ? __ldg(A.seq_ids + b) : A.seq_base + (uint32_t)b;
      const float inv_t = rl.inv_t;
      c2 = inv_t * kLog2e;
      __syncwarp();  // the previous item's batched path is done with the context
      if (lane == 0) {
        S4WarpCtx cx;
        cx.rowp = rowp;
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
    // this warp's steps: tokens base_w + s * kCtaTokens + [0, 2048)
    const int base_w = tok_begin + warp * kS4WarpTokens;
    const int span = tok_end - base_w;
    const int n_steps = span > 0 ? (span + kCtaTokens - 1) / kCtaTokens : 0;
    const int n_full = (aligned && span >= kS4WarpTokens) ? (span - kS4WarpTokens) / kCtaTokens + 1 : 0;
    const int tok0 = base_w + lane * 16;  // the lane's first group; its others follow at +512 tokens

    // bound published by earlier slices of the row (the hint words are cleared only when rows are cut)
    uint32_t m_enc = splits > 1 ? __ldcg(A.hints + row) : 0u;
    float lm = kGroupLseFloor;
    unsigned long long ls2 = 0ull;
    int qn = 0;

    // the lane's four groups of step s
    auto load_step = [&](auto& g, int s) {
      const int tok = tok0 + s * kCtaTokens;
      if (s < n_full) {
        const char* p = rowp + (size_t)tok * ES;
#pragma unroll
        for (int j = 0; j < kS4LaneGroups; ++j)
          if (GLS_IN_RANGE(tok + j * 512 + 15, 0, tok_end, 22u)) load16_vec(g[j], p + j * 512 * ES);
      } else {
#pragma unroll
        for (int j = 0; j < kS4LaneGroups; ++j) load16_scalar(g[j], rowp, tok + j * 512, tok_end);
      }
    };
    // coarse words of the lane's four groups of step s under noise stream c1s
    auto coarse_step = [&](uint32_t (&cw)[4], int s, uint32_t c1s) {
      const uint32_t g0 = (uint32_t)(tok0 + s * kCtaTokens) >> 4;  // g0 mod 128 == lane
      philox4x32<ROUNDS>(A.rk, A.rounds, s4_call_index(g0), c1s, pos, seq, cw);
    };

    // shapes that keep the next step's loads in flight request the first step now, so that it
    // arrives while the warm start computes (which then takes its data from the same registers)
    constexpr bool PREFETCH = S4Cfg<SH>::kPrefetch && !MULTI;
    G nxt[PREFETCH ? kS4LaneGroups : 1];
    if (PREFETCH && n_steps > 0) load_step(nxt, 0);

    // ---- warm start: evaluate, per lane, the most promising group of the first step; skipped
    //      when an earlier slice of the row has already published a bound ---------------------
    if (n_steps > 0 && m_enc == 0u) {
      G g[kS4LaneGroups];
      uint32_t cw[4];
      if constexpr (PREFETCH) {
#pragma unroll
        for (int j = 0; j < kS4LaneGroups; ++j) g[j] = nxt[j];
      } else {
        load_step(g, 0);
      }
      coarse_step(cw, 0, c1);
      float bkey = -CUDART_INF_F;
      int bj = -1;
#pragma unroll
      for (int j = 0; j < kS4LaneGroups; ++j) {
        // log2 of an upper bound on exp(score) of the group's tokens, up to a constant
        const float key = fmaf(group16_max(g[j]), c2, -lg2_approx(coarse_lower(cw[j]) + 0x1p-24f));
        if (key > bkey && tok0 + j * 512 < tok_end) {  // false for NaN
          bkey = key;
          bj = j;
        }
      }
      const bool pass = bj >= 0;
      const unsigned bal = __ballot_sync(0xffffffffu, pass);
      if (pass) {
        const uint32_t w = bj == 0 ? cw[0] : bj == 1 ? cw[1] : bj == 2 ? cw[2] : cw[3];
        const int qi = __popc(bal & ((1u << lane) - 1u));
        if (GLS_IN_RANGE(qi, 0, kS4QueueCap, 20u)) queue[qi] = make_uint2(w, ((uint32_t)tok0 >> 4) + 32u * bj);
      }
      const int nb = __popc(bal);
      __syncwarp();
      if (nb > 0) {
        const uint32_t e = s4_flush<SH, ROUNDS, MULTI>(A.rounds, 0, nb, filter_offset(dec_ordered(m_enc)));
        if (e > m_enc) m_enc = e;
      }
    }
    if (kWarps > 1 && lane == 0 && m_enc > 0u)
      atomicMax((unsigned long long*)&sh.m_tag, ((unsigned long long)tag << 32) | m_enc);
    float nm4 = filter_offset(dec_ordered(m_enc)) + 4.0f;
    const float c2s = c2 * (1.0f / 126.0f);
    float nms = scaled_offset(nm4);

    // one group: candidate iff coarse_lower(w) <= (an upper bound on) 2^(amax c2 + nm + 4)
    auto test_group = [&](float amax, uint32_t w, uint32_t gidx) {
      const bool pass = coarse_lower(w) <= exp2_upper_from_scaled(amax, c2s, nms);
      const unsigned bal = __ballot_sync(0xffffffffu, pass);
      if (bal != 0u) {
        if (pass) {
          const int qi = qn + __popc(bal & ((1u << lane) - 1u));
          if (GLS_IN_RANGE(qi, 0, kS4QueueCap, 21u)) queue[qi] = make_uint2(w, gidx);
        }
        qn += __popc(bal);
      }
    };
    auto poll_bound = [&]() {
      if (kWarps == 1) return;
      const unsigned long long mt = *m_tag;  // bound published by the other warps of the CTA
      const uint32_t m_new = ((uint32_t)(mt >> 32) == tag) ? (uint32_t)mt : 0u;
      if (m_new > m_enc) {
        m_enc = m_new;
        nm4 = filter_offset(dec_ordered(m_enc)) + 4.0f;
        nms = scaled_offset(nm4);
      }
    };
    auto flush_batch = [&](bool last) {
      __syncwarp();
      const int nb = min(qn, 32);
      qn -= nb;
      uint32_t e = s4_flush<SH, ROUNDS, MULTI>(A.rounds, qn, nb, nm4 - 4.0f);
      // the slices of a row trade their bounds through the row's hint word at batch time (not
      // after the item's last batch: nothing is left to filter, and the item publishes its bound
      // when it ends)
      if (splits > 1 && !last) {
        uint32_t h = 0u;
        if (lane == 0) h = e > m_enc ? atomicMax(A.hints + row, e) : __ldcg(A.hints + row);
        e = max(e, __shfl_sync(0xffffffffu, h, 0));
      }
      if (e > m_enc) {
        m_enc = e;
        nm4 = filter_offset(dec_ordered(m_enc)) + 4.0f;
        nms = scaled_offset(nm4);
        if (kWarps > 1 && lane == 0)
          atomicMax((unsigned long long*)&sh.m_tag, ((unsigned long long)tag << 32) | e);
      }
    };

    if constexpr (MULTI) {
      // ---- fused multi-stream race (Sec. 5.1 encoder: Y = argmin over tokens AND streams of
      //      S_i^(k) / weight_i): a step is loaded, maximised and summed once, then each of the
      //      multi_k noise streams takes its turn as one pass of the inner loop.
      const int ns = A.multi_k;
      const uint32_t smask = A.kmask;
      G g[kS4LaneGroups];
      float amax[kS4LaneGroups];
      int s = 0, st = 0;
      for (;;) {
#pragma unroll 1
        while (s < n_steps && qn < 32) {
          if (st == 0) {
            load_step(g, s);
#pragma unroll
            for (int j = 0; j < kS4LaneGroups; ++j) {
              amax[j] = group16_max(g[j]);
              if (LSE) lse16<DT>(g[j], amax[j], c2, lm, ls2);
            }
          }
          const uint32_t ks = (uint32_t)st & smask;
          uint32_t cw[4];
          coarse_step(cw, s, c1 + ks);
          const uint32_t g0 = (uint32_t)(tok0 + s * kCtaTokens) >> 4;
#pragma unroll
          for (int j = 0; j < kS4LaneGroups; ++j) test_group(amax[j], cw[j], (g0 + 32u * j) | (ks << 28));
          poll_bound();
          if (++st == ns) {
            st = 0;
            ++s;
          }
        }
        if (qn < 32) break;
        flush_batch(false);
      }
    } else {
      // ---- the sweep.  The inner loop runs until 32 groups are queued; the batched evaluation
      //      is called from the outer loop so that the inner loop carries no call.
      int s = 0;
      for (;;) {
#pragma unroll 1
        for (; s < n_steps && qn < 32; ++s) {
          G g[kS4LaneGroups];
          uint32_t cw[4];
          if constexpr (PREFETCH) {
#pragma unroll
            for (int j = 0; j < kS4LaneGroups; ++j) g[j] = nxt[j];
            if (s + 1 < n_steps) load_step(nxt, s + 1);
          } else {
            load_step(g, s);
          }
          coarse_step(cw, s, c1);
          const uint32_t g0 = (uint32_t)(tok0 + s * kCtaTokens) >> 4;
#pragma unroll
          for (int j = 0; j < kS4LaneGroups; ++j) {
            const float amax = group16_max(g[j]);
            if (LSE) lse16<DT>(g[j], amax, c2, lm, ls2);
            test_group(amax, cw[j], g0 + 32u * j);
          }
          poll_bound();
        }
        if (qn < 32) break;
        flush_batch(false);
      }
    }
    // ---- drain the queue ---------------------------------------------------------------------
    while (qn > 0) flush_batch(qn <= 32);

    // ---- combine the lanes; every warp writes its own partial result ---------------------------
    Top2 t2 = sh.best[threadIdx.x];
    top2_warp_merge(t2);
    float ls = 0.f;
    if (LSE) {
      float s0, s1;
      unpack_f32x2(ls2, s0, s1);
      if (__any_sync(0xffffffffu, !(s0 + s1 < CUDART_INF_F))) {  // NaN or +inf logits in the slice
        float rl, rs;
        lse4_redo_careful<SH>(rowp, tok0, n_steps, tok_end, c2, &rl, &rs);
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
      if (GLS_IN_RANGE(split * kWarps + warp, 0, A.parts, 23u) && GLS_IN_RANGE(row, 0, A.rows, 24u))
        A.partials[(long long)row * A.parts + split * kWarps + warp] = pr;
      if (splits > 1 && m_enc > 0u) atomicMax(A.hints + row, m_enc);
    }
  }
}

// LSEMODE 0: races only (draft side, decoders); 1: races and the rows' log-sum-exp (target side,
// encoder); 2: two sets of rows in one launch, the first without and the second with the
// log-sum-exp (the fused draft + verify call).
template <int SH, int LSEMODE, int ROUNDS, bool MULTI = false>
__global__ void __launch_bounds__(S4Cfg<SH>::kWarps * 32, S4Cfg<SH>::kCtasPerSM)
sweep4_kernel(const __grid_constant__ SweepArgs A) {
  S4Shared<SH>& sh = s4_shared<SH>();
  if (threadIdx.x == 0) sh.m_tag = 0ull;
  __syncthreads();
  uint32_t tag = 0u;
  for (long long item = blockIdx.x; item < A.n_items; item += gridDim.x) {
    ++tag;
    const int split = (int)(item / A.row_count);
    const int row = A.row_begin + (int)(item - (long long)split * A.row_count);
    if constexpr (LSEMODE == 2) {
      if (row >= A.rows1)
        s4_item<SH, true, ROUNDS, false>(A, row, split, tag, A.chunk, A.splits);
      else
        s4_item<SH, false, ROUNDS, false>(A, row, split, tag, A.chunk, A.splits);
    } else {
      s4_item<SH, LSEMODE == 1, ROUNDS, MULTI>(A, row, split, tag, A.chunk, A.splits);
    }
  }
  // this block has no more work: a dependent launch (the reduction) may start to be scheduled
  asm volatile("griddepcontrol.launch_dependents;");
}

// ------------------------------------------------------------------------------------------
// Rows named by a list in device memory (the position-by-position verification of Algorithm 2:
// the rows of a position are those of the drafts still active there, known only on the device).
// The slicing follows from the number of listed rows, by the rule of the host-side plan; slices
// are at least four steps long.
// ------------------------------------------------------------------------------------------
struct ListedSlicing {
  int chunk, splits;
};
__host__ __device__ __forceinline__ int listed_max_splits(int V, int cta_tokens) {
  const int steps = (V + cta_tokens - 1) / cta_tokens;
  return steps >= 8 ? steps / 4 : 1;
}
__host__ __device__ __forceinline__ ListedSlicing listed_slicing(int n_rows, int V, int cta_tokens,
                                                                 int grid) {
  const int steps = (V + cta_tokens - 1) / cta_tokens;
  const int cap = listed_max_splits(V, cta_tokens);
  // Few rows (less than half a launch): as many slices per row as keep the items within one
  // round.  Otherwise the fewest slices for which the items fill the launch and the last round of
  // items leaves at most 15 % of it idle (or every CTA gets a dozen items).
  int want = cap;
  if (2 * (long long)n_rows < grid) {
    want = n_rows > 0 ? grid / n_rows : 1;
    if (want > cap) want = cap;
  } else {
    for (int sp = 1; sp < cap; ++sp) {
      const long long items = (long long)n_rows * sp;
      if (items < grid) continue;
      const long long rounds = (items + grid - 1) / grid;
      if (items >= 12LL * grid || (rounds * grid - items) * 100 <= 15 * rounds * grid) {
        want = sp;
        break;
      }
    }
  }
  const int chunk_steps = (steps + want - 1) / want;
  ListedSlicing r;
  r.chunk = chunk_steps * cta_tokens;
  r.splits = (steps + chunk_steps - 1) / chunk_steps;
  return r;
}

// Races and log-sum-exp of the rows list[0 .. *count): the target side of one phase (MULTI: every
// row under all of the call's noise streams at once, Appendix B).
template <int SH, int ROUNDS, bool MULTI>
__global__ void __launch_bounds__(S4Cfg<SH>::kWarps * 32, S4Cfg<SH>::kCtasPerSM)
sweep4_listed_kernel(const __grid_constant__ SweepArgs A, const int* __restrict__ list,
                     const int* __restrict__ count) {
  S4Shared<SH>& sh = s4_shared<SH>();
  if (threadIdx.x == 0) sh.m_tag = 0ull;
  __syncthreads();
  // the kernel that wrote the list (launched before this one) is complete
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int n = __ldcg(count);
  const ListedSlicing sl = listed_slicing(n, A.V, S4Cfg<SH>::kCtaTokens, (int)gridDim.x);
  const long long n_items = (long long)n * sl.splits;
  uint32_t tag = 0u;
  for (long long item = blockIdx.x; item < n_items; item += gridDim.x) {
    ++tag;
    const int split = (int)(item / n);
    const int row = __ldcg(list + (int)(item - (long long)split * n));
    if (GLS_IN_RANGE(row, 0, A.rows, 27u))
      s4_item<SH, true, ROUNDS, MULTI>(A, row, split, tag, sl.chunk, sl.splits);
  }
  asm volatile("griddepcontrol.launch_dependents;");
}

}  // namespace gls
