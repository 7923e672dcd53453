// gls_gauss.cuh -- compression from the source: the races of Sec. 5.1 over importance weights
// that are computed on the fly (Appendix C of arXiv 2506.05632 with the Gaussian model of
// Sec. 5.2 / Appendix D.3, applied per dimension), instead of being streamed from memory.
//
// The log-weight of candidate u_i for a row with mean mu and variance v is
//     sum_d -(u_id - mu_d)^2 / (2 v) + u_id^2 / (2 s2_prior)
// (encoder row b: mu = a_b, v = s2_eta; decoder row (b, k): mu = t_bk / s2_T, v = s2_W - 1 / s2_T).
// Streaming precomputed weights reads 4 bytes per (row, candidate); computing them needs the
// D coordinates of the candidate, which are the same for every row.  So the loop nest is turned
// around: a CTA takes a tile of 2048 candidates (the 128 noise groups that 32 generator calls
// serve), keeps its coordinates in shared memory, pre-scaled by 1 / sqrt(2 v), and walks over the
// rows, four at a time.  Per row block a lane computes the 4 x 16 weights of its group of 16
// candidates in two-wide fp32 arithmetic (one add and one multiply-add per coordinate and pair),
// then the group test of the sweep (gls_sweep4.cuh) decides from the coarse word of the group's
// minimum whether any of the 16 can still win; candidate groups are examined in batches, exactly
// as in the sweep, and the leaders are re-scored in fp64 by the reduction kernel, which
// recomputes their weights from the source in fp64.  Per (row, tile) one partial result is
// written (only if the tile produced a candidate, or carries a share of the log-sum-exp).
#pragma once
#include "gls_sweep4.cuh"

namespace gls {

constexpr int kGTile = 2048;        // candidates per tile = 128 groups of 16
constexpr int kGWarps = 4;          // warp w owns groups 32 w .. 32 w + 31 of the tile
constexpr int kGRows = 2;           // rows per block (2 x 16 weights per lane stay under 128 registers)
constexpr int kGPad = 16;           // floats per group in shared memory; its four 16-byte chunks are
                                    // stored XOR-swizzled by (group >> 1) & 3: conflict-free 128-bit reads
constexpr int kGMaxD = 16;
constexpr int kGMaxK = 8;
constexpr int kGFlushAt = 8;                    // a batch is taken as soon as this many groups are queued
constexpr int kGQueue = kGFlushAt + 32;         // one (row, stream) test adds at most 32 per warp
constexpr int kGMaxQuads = 4;                   // warp quads per CTA, each walking its own row blocks

struct GaussRowCtx {  // one row of the current block
  uint32_t c1, pos, seq;  // noise stream (c1 without the stream number in the encoder pass)
  uint32_t m_enc;         // ordered code of the row's bound
  int row, b;             // row number (-1: past the end), source sample
  int msg;                // label a candidate must carry (decoder pass with labels)
  float nms;              // the group test's offset for the bound the row had when the block was set up
};
struct __align__(16) GaussEntry {  // a queued group: coarse word, group | stream << 28, row slot, weights
  uint32_t w, g, slot, pad;
  float a[16];
};
// Shared memory of one warp quad (four warps that walk the same row blocks); the coarse words
// [stream-row][word][lane] follow it, then the next quad's block.
struct __align__(16) GaussQuad {
  // [2]: the block being worked on and the next one, which is set up meanwhile
  float mu[2][kGMaxD][kGRows];                    // twice the scaled means of the block's rows
  GaussRowCtx ctx[2][kGRows];
  Top2 best[2][kGWarps][kGRows];                  // per warp and row slot
  float lse_m[2][kGWarps][kGRows], lse_s[2][kGWarps][kGRows];
  GaussEntry queue[kGWarps][kGQueue];
};
// Layout: quads x (GaussQuad, coarse words [2][kGRows * streams][4][32]), labels [128][4], then the
// tile [(D + 1)][128 * kGPad] floats, plane D holding the part of a weight that depends on the
// candidate alone.
__host__ __device__ inline size_t gauss_quad_bytes(int streams) {
  return sizeof(GaussQuad) + (size_t)2 * kGRows * streams * 4 * 32 * sizeof(uint32_t);
}
__host__ __device__ inline size_t gauss_smem_bytes(int D, int streams, int quads) {
  return (size_t)quads * gauss_quad_bytes(streams) + 128 * 4 * sizeof(uint32_t) +
         (size_t)(D + 1) * 128 * kGPad * sizeof(float);
}

// Batched evaluation of queued groups (cf. s4_flush): lane l < n takes entry first + l.  Entries
// may belong to different rows of the block; each lane works under its own row's key and bound.
// The lanes' results are merged per row slot into sh.best[warp][slot]; improved bounds go to the
// row's context and to its hint word.
template <int ROUNDS, bool ENC>
__device__ __noinline__ void gauss_flush(const SweepArgs& A, GaussQuad& sh, int buf, int first, int n) {
  const int lane = threadIdx.x & 31;
  const int warp = (threadIdx.x >> 5) & (kGWarps - 1);
  constexpr float c2 = kLog2e;
  uint32_t msk = 0u, g = 0u, ks = 0u;
  int loc = -1, slot = 0;
  float M = 1.f, lg2M = 0.f, nm = CUDART_INF_F;
  const GaussEntry& e =
      sh.queue[warp][GLS_IN_RANGE(first + (lane < n ? lane : 0), 0, kGQueue, 33u) ? first + (lane < n ? lane : 0) : 0];
  Top2 b;
  top2_init(b);
  float lower = -CUDART_INF_F;
  const uint8_t* bins = nullptr;
  GaussRowCtx cx = sh.ctx[buf][0];
  if (lane < n) {
    slot = (int)e.slot;
    cx = sh.ctx[buf][slot];
    bins = A.bins ? A.bins + A.bins_sb * cx.b : nullptr;
    g = e.g;
    ks = g >> 28;
    g &= 0x0fffffffu;
    uint32_t f[4];
    philox4x32<ROUNDS>(A.rk, A.rounds, g, cx.c1 + ks + (2u << 16), cx.pos, cx.seq, f);
    loc = (int)((f[0] >> 16) & 15u);
    M = exp1_from_word(e.w, ((float)(f[0] & 0xffffu) + 0.5f) * 0x1p-16f) * 0.0625f;
    lg2M = lg2_approx(M);
    nm = filter_offset(dec_ordered(cx.m_enc));
    // the candidate at the minimum has S = M exactly: its score bounds the row's best at once
    const long long il = ((long long)g << 4) + loc;
    const float a = e.a[loc];
    if (a > -CUDART_INF_F && a < CUDART_INF_F &&
        (ENC || bins == nullptr || (int)__ldg(bins + il) == cx.msg)) {
      const float ln_s = logf(M);
      const float s = a - ln_s;
      nm = fminf(nm, filter_offset(s - score_slack(s, ln_s)));
    }
    const float nmM = nm - lg2M + 0x1p-10f;
#pragma unroll
    for (int t = 0; t < 16; ++t) {
      const float at = e.a[t];
      if (at < CUDART_INF_F && fmaf(at, c2, nmM) >= 0.f) msk |= 1u << t;  // false for NaN
    }
  }
  while (__any_sync(0xffffffffu, msk != 0u)) {
    if (msk != 0u) {
      const int t = __ffs(msk) - 1;
      msk &= msk - 1u;
      const long long i = ((long long)g << 4) + t;
      const float a = e.a[t];
      if (fmaf(a, c2, nm - lg2M + 0x1p-10f) >= 0.f &&
          (ENC || bins == nullptr || (int)__ldg(bins + i) == cx.msg)) {
        float s_noise = M;
        if (t != loc) {
          uint32_t f[4];
          philox4x32<ROUNDS>(A.rk, A.rounds, (uint32_t)(i >> 2), cx.c1 + ks + (4u << 16), cx.pos,
                             cx.seq, f);
          const uint32_t u = (i & 2) ? ((i & 1) ? f[3] : f[2]) : ((i & 1) ? f[1] : f[0]);
          s_noise = M + exp1_from_word(u, 0.5f);
        }
        const float ln_s = logf(s_noise);
        const float s = a - ln_s;
        // encoder pass: the candidate is (token, stream), ordered by token first
        top2_offer(b, s, ENC ? (int)(((uint32_t)i << 3) | ks) : (int)i);
        const float lo = s - score_slack(s, ln_s);
        lower = fmaxf(lower, lo);
        nm = fminf(nm, filter_offset(lo));
      }
    }
  }
  // merge the lanes' results per row slot
#pragma unroll
  for (int r = 0; r < kGRows; ++r) {
    Top2 m = b;
    float lo = lower;
    if (!(lane < n && slot == r)) {
      top2_init(m);
      lo = -CUDART_INF_F;
    }
    if (!__any_sync(0xffffffffu, m.i1 >= 0)) continue;
    top2_warp_merge(m);
    const uint32_t enc = __reduce_max_sync(0xffffffffu, enc_ordered(lo));
    if (lane == 0) {
      Top2 cur = sh.best[buf][warp][r];
      top2_offer(cur, m.s1, m.i1);
      top2_offer(cur, m.s2, m.i2);
      sh.best[buf][warp][r] = cur;
      const uint32_t old = atomicMax(&sh.ctx[buf][r].m_enc, enc);
      if (enc > old) atomicMax(A.hints + sh.ctx[buf][r].row, enc);
    }
  }
  __syncwarp();
}

// ------------------------------------------------------------------------------------------
// The kernel.  Grid: tiles x row ranges.  ENC: rows are source samples b, each raced under the
// A.multi_k noise streams at once, with the log-sum-exp of the weights; otherwise rows are
// decoder rows (b, k) under stream k, restricted to the candidates labelled A.msg[b].
//   row range r of n_ranges covers rows [r * rows_per_range, ...); blockIdx.x = tile * n_ranges + r
// ------------------------------------------------------------------------------------------
template <int ROUNDS, bool ENC>
__global__ void __launch_bounds__(kGMaxQuads * kGWarps * 32, 1)
gauss_sweep_kernel(const __grid_constant__ SweepArgs A, int n_ranges, int rows_per_range,
                   long long N, float scale /* 1 / sqrt(2 v) of this pass */) {
  // blockDim.x = quads * 128: every quad of warps walks its own row blocks over the shared tile
  const int n_quads = (int)blockDim.x >> 7;
  const int quad = (int)threadIdx.x >> 7;
  const int tq = (int)threadIdx.x & 127;  // thread within the quad
  const int lane = threadIdx.x & 31;
  const int warp = (threadIdx.x >> 5) & (kGWarps - 1);  // warp within the quad
  const int D = A.gD;
  const int K = A.K;
  const int tile = blockIdx.x / n_ranges;
  const int range = blockIdx.x - tile * n_ranges;
  const int row_lo = range * rows_per_range;
  const int row_hi = min(A.rows, row_lo + rows_per_range);
  const long long cand0 = (long long)tile * kGTile;
  const int n_streams = ENC ? A.multi_k : 1;
  constexpr int kPlane = 128 * kGPad;
  const size_t quad_bytes = gauss_quad_bytes(n_streams);
  GaussQuad& sh = *reinterpret_cast<GaussQuad*>(gls_smem_raw + (size_t)quad * quad_bytes);
  uint32_t (*const xw_all)[4][32] =  // [2 * kGRows * n_streams][4][32]: buffer p starts at p * kGRows * n_streams
      reinterpret_cast<uint32_t(*)[4][32]>(gls_smem_raw + (size_t)quad * quad_bytes + sizeof(GaussQuad));
  const int xw_stride = kGRows * n_streams;
  uint32_t (*const labels)[4] =
      reinterpret_cast<uint32_t(*)[4]>(gls_smem_raw + (size_t)n_quads * quad_bytes);
  float* const us = reinterpret_cast<float*>(gls_smem_raw + (size_t)n_quads * quad_bytes + 128 * 4 * sizeof(uint32_t));
  auto quad_sync = [&]() { asm volatile("bar.sync %0, %1;" ::"r"(quad + 1), "r"(kGWarps * 32) : "memory"); };

  // ---- the tile's coordinates, scaled, to shared memory; plane D holds the candidate's own part
  //      of the weight, -inf for candidates past the end (their weights become -inf)
  {
    const float half_inv_prior = (float)(0.5 / A.g_s2_prior);
    for (int c = threadIdx.x; c < kGTile; c += (int)blockDim.x) {
      const long long i = cand0 + c;
      const int grp = c >> 4, t = c & 15;
      const int at = grp * kGPad + 4 * ((t >> 2) ^ ((grp >> 1) & 3)) + (t & 3);
      float nrm = 0.f, nrm_s = 0.f;
      for (int d = 0; d < D; ++d) {
        const float x = i < N ? __ldg(A.gu + i * D + d) : 0.f;
        const float xs = x * scale;
        nrm = fmaf(x, x, nrm);
        nrm_s = fmaf(xs, xs, nrm_s);
        us[d * kPlane + at] = xs;
      }
      // the part of the weight that does not depend on the row: |u|^2 / (2 s2_prior), in the
      // decoder pass (dot-product form, below) less |u s|^2
      us[D * kPlane + at] = i < N ? (ENC ? nrm * half_inv_prior : fmaf(nrm, half_inv_prior, -nrm_s))
                                  : -CUDART_INF_F;
    }
  }
  // decoder pass with one label array for all samples: the tile's labels, so that the group test
  // can look at the eligible candidates only (with L_max labels the best eligible score lies about
  // ln L_max below the best overall, and that many more groups would pass a test on all sixteen)
  const bool use_labels = !ENC && A.bins != nullptr && A.bins_sb == 0;
  if (use_labels) {
    for (int c = threadIdx.x; c < kGTile; c += (int)blockDim.x) {
      const long long i = cand0 + c;
      reinterpret_cast<uint8_t*>(&labels[0][0])[c] = i < N ? __ldg(A.bins + i) : (uint8_t)0;
    }
  }
  // What the next block needs: scaled means, contexts, coarse words.  The global loads are issued
  // early (fetch, before the arithmetic of the current block) and their values parked in a few
  // registers; commit writes them to shared memory once the current block is done with it.
  float pf_mu[1] = {0.f};  // kGRows * D <= 64 values, one per thread
  uint32_t pf_seq = 0u, pf_hint = 0u;
  int pf_msg = 0;
  auto fetch = [&](int row0) {
    const int idx = tq;
    if (idx < kGRows * D) {
      const int r = idx / D, d = idx - r * D;
      const int row = row0 + r;
      float m = 0.f;
      if (row < row_hi) {
        if (ENC) m = __ldg(A.ga + (long long)row * D + d);
        else m = __ldg(A.gt + (long long)row * D + d) / (float)(1.0 + A.g_s2_zeta);
      }
      pf_mu[0] = m * scale;
    }
    if (tq < kGRows) {
      const int row = row0 + tq;
      if (row < row_hi) {
        const int b = ENC ? row : row / K;
        pf_seq = A.seq_ids ? __ldg(A.seq_ids + b) : A.seq_base + (uint32_t)b;
        pf_msg = (!ENC && A.bins && A.msg) ? (int)__ldg(A.msg + b) : 0;
        pf_hint = __ldcg(A.hints + row);
      }
    }
  };
  auto commit = [&](int row0, int buf) {
    const int idx = tq;
    if (idx < kGRows * D) {
      const int r = idx / D, d = idx - r * D;
      sh.mu[buf][d][r] = ENC ? pf_mu[0] : 2.0f * pf_mu[0];  // decoder pass: doubled, the cross term's factor
    }
    if (tq < kGRows) {
      const int r = tq;
      const int row = row0 + r;
      GaussRowCtx cx;
      cx.row = row < row_hi ? row : -1;
      const int b = ENC ? row : row / K;
      const int k = ENC ? 0 : row - b * K;
      cx.b = b;
      cx.c1 = ((uint32_t)k & A.kmask) | (A.domain << 16);
      cx.pos = A.pos_base;
      cx.seq = pf_seq;
      cx.msg = pf_msg;
      cx.m_enc = cx.row >= 0 ? pf_hint : 0u;
      cx.nms = scaled_offset(filter_offset(dec_ordered(cx.m_enc)) + 4.0f);
      sh.ctx[buf][r] = cx;
    }
  };
  // coarse words of the block's stream-rows: warp w computes stream-rows sr = w, w + 4, ...
  auto coarse_words = [&](int row0, int buf) {
    for (int sr = warp; sr < kGRows * n_streams; sr += kGWarps) {
      const int r = sr / n_streams, ks = sr - r * n_streams;
      const int row = row0 + r;
      if (row >= row_hi) continue;
      const int b = ENC ? row : row / K;
      const int k = ENC ? 0 : row - b * K;
      const uint32_t c1 = ((ENC ? (uint32_t)ks : (uint32_t)k) & A.kmask) | (A.domain << 16);
      const uint32_t seq = A.seq_ids ? __ldg(A.seq_ids + b) : A.seq_base + (uint32_t)b;
      uint32_t cw[4];
      philox4x32<ROUNDS>(A.rk, A.rounds, ((uint32_t)tile << 5) | (uint32_t)lane, c1, A.pos_base, seq, cw);
      uint32_t (*const xo)[32] = xw_all[buf * xw_stride + sr];
      xo[0][lane] = cw[0];
      xo[1][lane] = cw[1];
      xo[2][lane] = cw[2];
      xo[3][lane] = cw[3];
    }
  };
  // The blocks of rows are walked in a rotated order that differs from tile to tile: CTAs that run
  // at the same time then work on different rows, so that a row's bound, once some tile has found
  // one and published it in the row's hint word, is there for (almost) every other tile.  In
  // lockstep every CTA of the first wave would meet every row without a bound and examine all of
  // its groups.
  const int n_blocks = (row_hi - row_lo + kGRows - 1) / kGRows;
  const int rot = (int)(((uint32_t)tile * 2654435761u >> 8) % (uint32_t)n_blocks);
  auto block_row = [&](int it) { return row_lo + ((it + rot) % n_blocks) * kGRows; };
  __syncthreads();  // the tile is in shared memory
  // every row slot's running results start empty in both buffers
  if (tq < 2 * kGWarps * kGRows) top2_init((&sh.best[0][0][0])[tq]);
  if (quad < n_blocks) {
    fetch(block_row(quad));
    commit(block_row(quad), 0);
    coarse_words(block_row(quad), 0);
  }
  quad_sync();

  const int gl = warp * 32 + lane;                      // the lane's group within the tile
  const uint32_t gidx = (uint32_t)tile * 128u + (uint32_t)gl;  // ... and in the whole row
  const float* const ug = us + gl * kGPad;
  const int sw = (gl >> 1) & 3;  // chunk q of the group sits at position q ^ sw
  GaussEntry* const queue = sh.queue[warp];
  const bool group_in_range = cand0 + (long long)gl * 16 < N;

  int buf = 0;  // the buffer of the block being worked on
  for (int it = quad; it < n_blocks; it += n_quads, buf ^= 1) {
    const int row0 = block_row(it);
    uint32_t (*const xw)[4][32] = xw_all + buf * xw_stride;
    if (it + n_quads < n_blocks) fetch(block_row(it + n_quads));
    // ---- weights of the lane's 16 candidates for the block's four rows -----------------------
    // With us = u s and ms = m s (s = 1 / sqrt(2 v)) the weight is
    //   |u|^2 / (2 s2_prior) - |us - ms|^2 = (|u|^2 / (2 s2_prior) - |us|^2) + us . (2 ms) - |ms|^2.
    // Decoder pass: the first term sits in plane D of the tile, the last is one number per row, and
    // the middle one is a dot product, one two-wide multiply-add per coordinate and pair of
    // candidates instead of a difference and a multiply-add.  The cancellation costs eps times the
    // size of the terms (a few 1e-6 for the decoders' wide conditionals), inside the margin of the
    // group test and the window in which the reduction re-scores the leaders in fp64.  The encoder
    // pass keeps the differences: its weights also feed the log-sum-exp that normalises the
    // encoder's score, and a narrow encoder target (large s) would cost it its 1e-5.
    unsigned long long acc[kGRows][8];
    float m2acc[kGRows];
#pragma unroll
    for (int r = 0; r < kGRows; ++r) {
      m2acc[r] = 0.f;
#pragma unroll
      for (int p = 0; p < 8; ++p) acc[r][p] = 0ull;
    }
#pragma unroll 2
    for (int d = 0; d < D; ++d) {
      const float2 m2 = *reinterpret_cast<const float2*>(&sh.mu[buf][d][0]);
      unsigned long long up[8];
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float4 v = *reinterpret_cast<const float4*>(ug + d * kPlane + 4 * (q ^ sw));
        up[2 * q] = pack_f32x2(v.x, v.y);
        up[2 * q + 1] = pack_f32x2(v.z, v.w);
      }
      const float mr[kGRows] = {m2.x, m2.y};
#pragma unroll
      for (int r = 0; r < kGRows; ++r) {
        if constexpr (ENC) {
          // all differences first, then all multiply-adds: a dependent pair issued back to back
          // would stall on its own latency
          const unsigned long long nm2 = pack_f32x2(-mr[r], -mr[r]);
          unsigned long long diff[8];
#pragma unroll
          for (int p = 0; p < 8; ++p) diff[p] = add_f32x2(up[p], nm2);
#pragma unroll
          for (int p = 0; p < 8; ++p) acc[r][p] = fma_f32x2(diff[p], diff[p], acc[r][p]);
        } else {
          const unsigned long long tm2 = pack_f32x2(mr[r], mr[r]);
          m2acc[r] = fmaf(mr[r], mr[r], m2acc[r]);
#pragma unroll
          for (int p = 0; p < 8; ++p) acc[r][p] = fma_f32x2(up[p], tm2, acc[r][p]);
        }
      }
    }
    float pn[16];
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const float4 v = *reinterpret_cast<const float4*>(ug + D * kPlane + 4 * (q ^ sw));
      pn[4 * q] = v.x; pn[4 * q + 1] = v.y; pn[4 * q + 2] = v.z; pn[4 * q + 3] = v.w;
    }
    // ---- per row: group maximum, log-sum-exp (encoder), group test per stream ------------------
    int qn = 0;
    uint32_t lab[4] = {0u, 0u, 0u, 0u};
    if (use_labels) {
      const uint4 lv = *reinterpret_cast<const uint4*>(&labels[gl][0]);
      lab[0] = lv.x; lab[1] = lv.y; lab[2] = lv.z; lab[3] = lv.w;
    }
#pragma unroll
    for (int r = 0; r < kGRows; ++r) {
      const GaussRowCtx cx = sh.ctx[buf][r];
      if (cx.row < 0) continue;  // uniform over the CTA
      float wgt[16];
      float amax = -CUDART_INF_F;
      const float nm2 = -0.25f * m2acc[r];  // decoder pass: -|ms|^2 (the means are stored doubled)
#pragma unroll
      for (int p = 0; p < 8; ++p) {
        float s0, s1;
        unpack_f32x2(acc[r][p], s0, s1);
        wgt[2 * p] = ENC ? pn[2 * p] - s0 : (pn[2 * p] + nm2) + s0;
        wgt[2 * p + 1] = ENC ? pn[2 * p + 1] - s1 : (pn[2 * p + 1] + nm2) + s1;
        amax = fmaxf(amax, fmaxf(wgt[2 * p], wgt[2 * p + 1]));
      }
      if (ENC) {
        // the lane's share of sum_i exp(weight_i), relative to its own maximum; lanes are merged
        // with the usual rescaling
        float lm = amax, ls = 0.f;
        if (amax > -CUDART_INF_F) {
#pragma unroll
          for (int t = 0; t < 16; ++t) ls += ex2_approx((wgt[t] - amax) * kLog2e);
        } else {
          lm = kGroupLseFloor;
        }
        float wm = lm;
#pragma unroll
        for (int dd = 16; dd > 0; dd >>= 1) wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, dd));
        ls *= ex2_approx((lm - wm) * kLog2e);
#pragma unroll
        for (int dd = 16; dd > 0; dd >>= 1) ls += __shfl_xor_sync(0xffffffffu, ls, dd);
        if (lane == 0) {
          sh.lse_m[buf][warp][r] = wm;
          sh.lse_s[buf][warp][r] = ls;
        }
      }
      const float thr = exp2_upper_from_scaled(amax, kLog2e * (1.0f / 126.0f), cx.nms);
      for (int ks = 0; ks < n_streams; ++ks) {
        const uint32_t w = xw[r * n_streams + ks][warp][lane];
        bool pass = group_in_range && coarse_lower(w) <= thr;
        if (use_labels && pass) {
          // second look, for the few groups that pass on all sixteen: the maximum over the
          // candidates that carry the transmitted label (with L_max labels the best eligible
          // score lies about ln L_max lower, and that many more groups pass the first test)
          const uint32_t m4 = (uint32_t)cx.msg * 0x01010101u;
          float emax = -CUDART_INF_F;
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint32_t eq = __vcmpeq4(lab[q], m4);  // 0xff per matching byte
#pragma unroll
            for (int t = 0; t < 4; ++t)
              if (eq & (1u << (8 * t))) emax = fmaxf(emax, wgt[4 * q + t]);
          }
          pass = coarse_lower(w) <= exp2_upper_from_scaled(emax, kLog2e * (1.0f / 126.0f), cx.nms);
        }
        const unsigned bal = __ballot_sync(0xffffffffu, pass);
        if (bal != 0u) {
          if (pass) {
            const int qi = qn + __popc(bal & ((1u << lane) - 1u));
            GaussEntry& e = queue[GLS_IN_RANGE(qi, 0, kGQueue, 30u) ? qi : 0];
            e.w = w;
            e.g = gidx | (((uint32_t)ks & A.kmask) << 28);
            e.slot = (uint32_t)r;
#pragma unroll
            for (int t = 0; t < 16; ++t) e.a[t] = wgt[t];
          }
          qn += __popc(bal);
          while (qn >= kGFlushAt) {  // enough for a batch: evaluate it now (rare after the first rows)
            __syncwarp();
            const int nb = min(qn, 32);
            qn -= nb;
            gauss_flush<ROUNDS, ENC>(A, sh, buf, qn, nb);
          }
        }
      }
    }
    while (qn > 0) {
      __syncwarp();
      const int nb = min(qn, 32);
      qn -= nb;
      gauss_flush<ROUNDS, ENC>(A, sh, buf, qn, nb);
    }
    // ---- the next block is set up in the other buffer (its global values were fetched before
    //      this block's arithmetic); one barrier per block
    if (it + n_quads < n_blocks) {
      commit(block_row(it + n_quads), buf ^ 1);
      coarse_words(block_row(it + n_quads), buf ^ 1);
    }
    quad_sync();  // this block's results and the next block's set-up are in shared memory
    // ---- warp r (< rows per block) merges row slot r of this block, writes its partial result and
    //      empties the slot for the block after next, while the other warps go on: buffer `buf` is
    //      written again only after the next barrier, which this warp reaches after the merge
    {
      const int r = warp;
      const int row = row0 + r;
      if (r < kGRows && lane == 0) {
        Top2 m = sh.best[buf][0][r];
        float lm = kGroupLseFloor, ls = 0.f;
#pragma unroll
        for (int w2 = 1; w2 < kGWarps; ++w2) {
          top2_offer(m, sh.best[buf][w2][r].s1, sh.best[buf][w2][r].i1);
          top2_offer(m, sh.best[buf][w2][r].s2, sh.best[buf][w2][r].i2);
        }
#pragma unroll
        for (int w2 = 0; w2 < kGWarps; ++w2) top2_init(sh.best[buf][w2][r]);
        if (ENC) {
#pragma unroll
          for (int w2 = 0; w2 < kGWarps; ++w2) lm = fmaxf(lm, sh.lse_m[buf][w2][r]);
#pragma unroll
          for (int w2 = 0; w2 < kGWarps; ++w2)
            ls += sh.lse_s[buf][w2][r] * ex2_approx((sh.lse_m[buf][w2][r] - lm) * kLog2e);
        }
        if (row < row_hi && (m.i1 >= 0 || (ENC && ls > 0.f))) {
          Partial pr;
          pr.s1 = m.s1; pr.i1 = m.i1; pr.s2 = m.s2; pr.i2 = m.i2;
          pr.lm = lm; pr.ls = ls; pr.pad0 = 0; pr.pad1 = 0;
          if (GLS_IN_RANGE(tile, 0, A.parts, 31u) && GLS_IN_RANGE(row, 0, A.rows, 32u))
            A.partials[(long long)row * A.parts + tile] = pr;
        }
      }
    }
  }
  asm volatile("griddepcontrol.launch_dependents;");
}

}  // namespace gls
