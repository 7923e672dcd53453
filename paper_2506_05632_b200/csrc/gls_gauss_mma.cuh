// gls_gauss_mma.cuh -- decoder pass of the compression from the source on the tensor cores.
//
// A decoder row's importance log-weight of candidate u (Appendix C, Gaussian model of Appendix D.3)
// is, with us = u s, ms = m s, s = 1 / sqrt(2 v),
//     |u|^2 / (2 s2_prior) - |us - ms|^2 = P(u) + us . (2 ms) - |ms|^2,
// P(u) = |u|^2 / (2 s2_prior) - |us|^2: a [rows x D] x [D x candidates] product plus one term per
// candidate and one per row -- the one dense contraction of this library.  Here a warp takes 16
// rows at a time and the CTA's tile of 2048 candidates, eight candidates per tensor-core
// instruction (mma.sync m16n8k8, tf32 operands, fp32 accumulation; D = 16 is two of them).  The
// products only serve the group test: a group of 16 candidates is examined further if the largest
// of its (approximate) weights, raised by a bound on the tf32 rounding of the operands, passes the
// test of the sweep -- so the filter still has no false negatives -- and the groups that pass are
// re-evaluated exactly (fp32 differences from the candidates in global memory, then the same
// batched evaluation as everywhere else; the reduction re-scores the leaders in fp64).
//
// A warp owns its 16 rows for the whole tile: no barrier between warps after the tile is loaded.
#pragma once
#include "gls_gauss.cuh"

namespace gls {

constexpr int kMWarps = 16;     // warps per CTA, each with its own blocks of rows
constexpr int kMRows = 16;      // rows per block (the M of the tensor-core tile)
constexpr int kMQueue = 48;     // queued groups per warp: a batch is taken at 32, a group adds <= 16
constexpr int kMD = 16;         // coordinates (two k-steps of eight)

struct GaussMmaRow {  // a row of the warp's block
  uint32_t c1, pos, seq, m_enc;
  int row, b, msg;
  float nms;     // the group test's offset for the row's current bound
  float margin;  // bound on the rounding error of the row's approximate weights
  float m2;      // |ms|^2
  float pad0, pad1;
};
struct __align__(16) GaussMmaWarp {
  GaussMmaRow ctx[kMRows];
  Top2 best[kMRows];
  float ms[kMRows][kMD];      // scaled means, for the exact re-evaluation
  uint2 queue[kMQueue];       // (coarse word, group | row slot << 28)
};
// Layout: tile [2048][16] floats (scaled, tf32-rounded, coordinates permuted so that a lane's four
// operands of a column are one 16-byte read), P [2048], labels [2048] bytes, the warps' blocks.
__host__ __device__ inline size_t gauss_mma_smem_bytes() {
  return (size_t)kGTile * kMD * sizeof(float) + (size_t)kGTile * sizeof(float) + kGTile +
         (size_t)kMWarps * sizeof(GaussMmaWarp);
}

__device__ __forceinline__ uint32_t to_tf32(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return r;
}
__device__ __forceinline__ void mma_tf32_16x8x8(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// where coordinate d of a candidate sits in the tile: lane q of a quad reads positions 4q .. 4q+3
// = coordinates (q, q + 4, 8 + q, 12 + q), its operands of the two k-steps
__host__ __device__ __forceinline__ int mma_coord_pos(int d) {
  const int kk = d >> 3, kidx = d & 7;
  return 4 * (kidx & 3) + 2 * kk + (kidx >> 2);
}

// Batched evaluation of queued groups: lane l < n takes entry first + l of the warp's queue,
// recomputes its group's 16 weights exactly (fp32 differences from the candidates in global
// memory, as the encoder pass forms them), then proceeds as gauss_flush does: the refinement bits
// and the position of the group's minimum, the candidates that can still matter under the row's
// bound and the transmitted label, their own exponentials, their scores.  Results are merged per
// row into wp.best; improved bounds go to the row's context and hint word.
template <int ROUNDS>
__device__ __noinline__ void gauss_mma_flush(const SweepArgs& A, GaussMmaWarp& wp, int first, int n,
                                             long long N, float scale, float half_inv_prior) {
  const int lane = threadIdx.x & 31;
  constexpr float c2 = kLog2e;
  uint32_t msk = 0u, g = 0u, w = 0u;
  int loc = -1, slot = -1;
  float M = 1.f, lg2M = 0.f, nm = CUDART_INF_F;
  float a[16];
#pragma unroll
  for (int t = 0; t < 16; ++t) a[t] = -CUDART_INF_F;
  Top2 b;
  top2_init(b);
  float lower = -CUDART_INF_F;
  const uint8_t* bins = nullptr;
  GaussMmaRow cx = wp.ctx[0];
  if (lane < n) {
    const uint2 e = wp.queue[GLS_IN_RANGE(first + lane, 0, kMQueue, 34u) ? first + lane : 0];
    w = e.x;
    slot = (int)(e.y >> 28);
    g = e.y & 0x0fffffffu;
    cx = wp.ctx[slot];
    bins = A.bins ? A.bins + A.bins_sb * cx.b : nullptr;
    // the group's weights, exactly
    float ms[kMD];
#pragma unroll
    for (int d = 0; d < kMD; ++d) ms[d] = wp.ms[slot][d];
#pragma unroll 4
    for (int t = 0; t < 16; ++t) {
      const long long i = ((long long)g << 4) + t;
      if (i < N) {
        const float4* up = reinterpret_cast<const float4*>(A.gu + i * kMD);
        float nrm = 0.f, acc = 0.f;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float4 v = __ldg(up + q);
          const float x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            nrm = fmaf(x[j], x[j], nrm);
            const float df = x[j] * scale - ms[4 * q + j];
            acc = fmaf(df, df, acc);
          }
        }
        a[t] = nrm * half_inv_prior - acc;
      }
    }
    uint32_t f[4];
    philox4x32<ROUNDS>(A.rk, A.rounds, g, cx.c1 + (2u << 16), cx.pos, cx.seq, f);
    loc = (int)((f[0] >> 16) & 15u);
    M = exp1_from_word(w, ((float)(f[0] & 0xffffu) + 0.5f) * 0x1p-16f) * 0.0625f;
    lg2M = lg2_approx(M);
    nm = filter_offset(dec_ordered(cx.m_enc));
    // the candidate at the minimum has S = M exactly: its score bounds the row's best at once
    const long long il = ((long long)g << 4) + loc;
    float al = -CUDART_INF_F;
#pragma unroll
    for (int t = 0; t < 16; ++t)
      if (t == loc) al = a[t];
    if (al > -CUDART_INF_F && al < CUDART_INF_F && (bins == nullptr || (int)__ldg(bins + il) == cx.msg)) {
      const float ln_s = logf(M);
      const float s = al - ln_s;
      nm = fminf(nm, filter_offset(s - score_slack(s, ln_s)));
    }
    const float nmM = nm - lg2M + 0x1p-10f;
#pragma unroll
    for (int t = 0; t < 16; ++t)
      if (a[t] < CUDART_INF_F && fmaf(a[t], c2, nmM) >= 0.f) msk |= 1u << t;  // false for NaN
  }
  while (__any_sync(0xffffffffu, msk != 0u)) {
    if (msk != 0u) {
      const int t = __ffs(msk) - 1;
      msk &= msk - 1u;
      const long long i = ((long long)g << 4) + t;
      float at = -CUDART_INF_F;
#pragma unroll
      for (int u = 0; u < 16; ++u)
        if (u == t) at = a[u];
      if (fmaf(at, c2, nm - lg2M + 0x1p-10f) >= 0.f && (bins == nullptr || (int)__ldg(bins + i) == cx.msg)) {
        float s_noise = M;
        if (t != loc) {
          uint32_t f[4];
          philox4x32<ROUNDS>(A.rk, A.rounds, (uint32_t)(i >> 2), cx.c1 + (4u << 16), cx.pos, cx.seq, f);
          const uint32_t u = (i & 2) ? ((i & 1) ? f[3] : f[2]) : ((i & 1) ? f[1] : f[0]);
          s_noise = M + exp1_from_word(u, 0.5f);
        }
        const float ln_s = logf(s_noise);
        const float s = at - ln_s;
        top2_offer(b, s, (int)i);
        const float lo = s - score_slack(s, ln_s);
        lower = fmaxf(lower, lo);
        nm = fminf(nm, filter_offset(lo));
      }
    }
  }
  // merge the lanes' results row by row (the batch holds entries of at most 16 rows)
  unsigned todo = __ballot_sync(0xffffffffu, lane < n);
  while (todo != 0u) {
    const int r = __shfl_sync(0xffffffffu, slot, __ffs(todo) - 1);
    const bool mine = lane < n && slot == r;
    todo &= ~__ballot_sync(0xffffffffu, mine);
    Top2 m = b;
    float lo = lower;
    if (!mine) {
      top2_init(m);
      lo = -CUDART_INF_F;
    }
    if (!__any_sync(0xffffffffu, m.i1 >= 0)) continue;
    top2_warp_merge(m);
    const uint32_t enc = __reduce_max_sync(0xffffffffu, enc_ordered(lo));
    if (lane == 0) {
      Top2 cur = wp.best[r];
      top2_offer(cur, m.s1, m.i1);
      top2_offer(cur, m.s2, m.i2);
      wp.best[r] = cur;
      if (enc > wp.ctx[r].m_enc) {
        wp.ctx[r].m_enc = enc;
        wp.ctx[r].nms = scaled_offset(filter_offset(dec_ordered(enc)) + 4.0f);
        atomicMax(A.hints + wp.ctx[r].row, enc);
      }
    }
  }
  __syncwarp();
}

// ------------------------------------------------------------------------------------------
// The kernel.  Grid: tiles x row ranges (as gauss_sweep_kernel); rows are decoder rows (b, k)
// under stream k, restricted to the candidates labelled A.msg[b].  D = 16.
// ------------------------------------------------------------------------------------------
template <int ROUNDS, bool LABELS /* one label array for all samples: test eligible candidates only */>
__global__ void __launch_bounds__(kMWarps * 32, 1)
gauss_dec_mma_kernel(const __grid_constant__ SweepArgs A, int n_ranges, int rows_per_range, long long N,
                     float scale /* 1 / sqrt(2 v) of the decoders' conditional */) {
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const int K = A.K;
  const int tile = blockIdx.x / n_ranges;
  const int range = blockIdx.x - tile * n_ranges;
  const int row_lo = range * rows_per_range;
  const int row_hi = min(A.rows, row_lo + rows_per_range);
  const long long cand0 = (long long)tile * kGTile;
  float* const ut = reinterpret_cast<float*>(gls_smem_raw);               // [2048][16]
  float* const pc = ut + (size_t)kGTile * kMD;                             // [2048]
  uint8_t* const labels = reinterpret_cast<uint8_t*>(pc + kGTile);         // [2048]
  GaussMmaWarp& wp = reinterpret_cast<GaussMmaWarp*>(labels + kGTile)[warp];
  __shared__ uint32_t umax_bits;  // largest |u s| of the tile (as ordered bits of a non-negative float)
  const float half_inv_prior = (float)(0.5 / A.g_s2_prior);
  constexpr bool use_labels = LABELS;
  if (threadIdx.x == 0) umax_bits = 0u;
  __syncthreads();
  // ---- the tile: scaled coordinates rounded to tf32, P(u), labels
  {
    float umax = 0.f;
    for (int c = threadIdx.x; c < kGTile; c += (int)blockDim.x) {
      const long long i = cand0 + c;
      float nrm = 0.f, nrm_s = 0.f;
      float xs[kMD];
#pragma unroll
      for (int d = 0; d < kMD; ++d) xs[d] = 0.f;
      if (i < N) {
        const float4* up = reinterpret_cast<const float4*>(A.gu + i * kMD);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          const float4 v = __ldg(up + q);
          const float x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float s1 = x[j] * scale;
            nrm = fmaf(x[j], x[j], nrm);
            nrm_s = fmaf(s1, s1, nrm_s);
            xs[4 * q + j] = __uint_as_float(to_tf32(s1));
          }
        }
      }
      // positions 4 q .. 4 q + 3 hold coordinates (q, q + 4, 8 + q, 12 + q): see mma_coord_pos
#pragma unroll
      for (int q = 0; q < 4; ++q)
        *reinterpret_cast<float4*>(ut + c * kMD + 4 * q) = make_float4(xs[q], xs[q + 4], xs[q + 8], xs[q + 12]);
      pc[c] = i < N ? fmaf(nrm, half_inv_prior, -nrm_s) : -CUDART_INF_F;
      labels[c] = (use_labels && i < N) ? __ldg(A.bins + i) : (uint8_t)0;
      umax = fmaxf(umax, nrm_s);
    }
    umax = sqrtf(umax) * (1.0f + 0x1p-20f);
    atomicMax(&umax_bits, __float_as_uint(umax));
  }
  __syncthreads();
  const float umax = __uint_as_float(umax_bits);

  const int g = lane >> 2, q = lane & 3;      // the lane's rows (g, g + 8) and column pair of a tile
  const int my_row = (q & 1) ? g + 8 : g;     // the row this lane tests (q = 0, 1; q = 2, 3 duplicate)
  const uint32_t lt = (1u << lane) - 1u;

  // The blocks of 16 rows are walked in an order rotated per tile (cf. gauss_sweep_kernel): CTAs
  // that run at the same time work on different rows, so a row's bound is found once and then
  // shared through its hint word.
  const int n_blocks = (row_hi - row_lo + kMRows - 1) / kMRows;
  const int rot = n_blocks > 0 ? (int)(((uint32_t)tile * 2654435761u >> 8) % (uint32_t)n_blocks) : 0;
  for (int it = warp; it < n_blocks; it += kMWarps) {
    const int row0 = row_lo + ((it + rot) % n_blocks) * kMRows;
    // ---- the block's rows: context, scaled means, tensor-core operand
    __syncwarp();
    if (lane < kMRows) {
      const int row = row0 + lane;
      GaussMmaRow cx;
      cx.row = row < row_hi ? row : -1;
      const int b = row < row_hi ? row / K : 0;
      const int k = row < row_hi ? row - b * K : 0;
      cx.b = b;
      cx.c1 = ((uint32_t)k & A.kmask) | (A.domain << 16);
      cx.pos = A.pos_base;
      cx.seq = A.seq_ids ? __ldg(A.seq_ids + b) : A.seq_base + (uint32_t)b;
      cx.msg = (A.bins && A.msg) ? (int)__ldg(A.msg + b) : 0;
      cx.m_enc = cx.row >= 0 ? __ldcg(A.hints + row) : 0u;
      cx.nms = scaled_offset(filter_offset(dec_ordered(cx.m_enc)) + 4.0f);
      float m2 = 0.f, r2 = 0.f;
      const float inv_s2t = 1.0f / (float)(1.0 + A.g_s2_zeta);
#pragma unroll
      for (int d = 0; d < kMD; ++d) {
        const float m = cx.row >= 0 ? __ldg(A.gt + (long long)row * kMD + d) * inv_s2t * scale : 0.f;
        wp.ms[lane][d] = m;
        m2 = fmaf(m, m, m2);
        const float tm = __uint_as_float(to_tf32(2.0f * m));
        r2 = fmaf(tm, tm, r2);
      }
      cx.m2 = m2;
      // |sum_d us_d tm_d - exact| <= 2^-10 |us| |tm| (each operand rounded to 11 significant bits)
      // plus the fp32 accumulation and the roundings of the other two terms; a little more than
      // that is added
      cx.margin = 0x1.2p-10f * umax * sqrtf(r2) + 3e-5f;
      cx.pad0 = cx.pad1 = 0.f;
      wp.ctx[lane] = cx;
      top2_init(wp.best[lane]);
    }
    __syncwarp();
    uint32_t af[2][4];  // A fragments of the two k-steps: rows (g, g + 8), coordinates (q, q + 4) + 8 kk
#pragma unroll
    for (int kk = 0; kk < 2; ++kk) {
      af[kk][0] = to_tf32(2.0f * wp.ms[g][8 * kk + q]);
      af[kk][1] = to_tf32(2.0f * wp.ms[g + 8][8 * kk + q]);
      af[kk][2] = to_tf32(2.0f * wp.ms[g][8 * kk + q + 4]);
      af[kk][3] = to_tf32(2.0f * wp.ms[g + 8][8 * kk + q + 4]);
    }
    // per-row constants of the lane's two rows (accumulator rows g and g + 8)
    const float nm2_lo = -wp.ctx[g].m2, nm2_hi = -wp.ctx[g + 8].m2;
    // the rows' labels, replicated over the bytes of a word for a four-way compare
    const uint32_t msg_lo = (uint32_t)wp.ctx[g].msg * 0x01010101u, msg_hi = (uint32_t)wp.ctx[g + 8].msg * 0x01010101u;
    // ... and of the row this lane tests
    const bool tester = q < 2 && wp.ctx[my_row].row >= 0;
    const float margin = wp.ctx[my_row].margin;
    const uint32_t c1 = wp.ctx[lane & 15].c1, seq = wp.ctx[lane & 15].seq;  // for the generator calls
    int qn = 0;

    // ---- the tile, 8 groups per iteration: lanes 0-15 make the generator call of the groups
    //      l, l + 32, l + 64, l + 96 (l = 2 i) for rows 0-15, lanes 16-31 that of l + 1
#pragma unroll 1
    for (int i2 = 0; i2 < 16; ++i2) {
      uint32_t cw[4];
      philox4x32<ROUNDS>(A.rk, A.rounds, ((uint32_t)tile << 5) | (uint32_t)(2 * i2 + (lane >> 4)), c1,
                         A.pos_base, seq, cw);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int grp = 2 * i2 + h + 32 * j;  // group within the tile
          // the tester's coarse word of this group: from the lane that called for its row
          const uint32_t w = __shfl_sync(0xffffffffu, cw[j], my_row + 16 * h);
          // approximate weights of the group's 16 candidates for the lane's two rows
          float mlo = -CUDART_INF_F, mhi = -CUDART_INF_F;
          float wl[4], wh[4];  // the lane's four candidates of the group, lower and upper row
#pragma unroll
          for (int nt = 0; nt < 2; ++nt) {
            const int cbase = grp * 16 + nt * 8;
            const float4 bv = *reinterpret_cast<const float4*>(ut + (cbase + g) * kMD + 4 * q);
            float c[4] = {0.f, 0.f, 0.f, 0.f};
            mma_tf32_16x8x8(c, af[0], __float_as_uint(bv.x), __float_as_uint(bv.y));
            mma_tf32_16x8x8(c, af[1], __float_as_uint(bv.z), __float_as_uint(bv.w));
            const float2 pv = *reinterpret_cast<const float2*>(pc + cbase + 2 * q);
            wl[2 * nt] = c[0] + pv.x; wl[2 * nt + 1] = c[1] + pv.y;
            wh[2 * nt] = c[2] + pv.x; wh[2 * nt + 1] = c[3] + pv.y;
          }
          if (use_labels) {
            // labels of the lane's candidates (2 q, 2 q + 1 of each half of the group) in one word
            const uint32_t lb = (uint32_t)*reinterpret_cast<const unsigned short*>(labels + grp * 16 + 2 * q) |
                                ((uint32_t)*reinterpret_cast<const unsigned short*>(labels + grp * 16 + 8 + 2 * q) << 16);
            const uint32_t el = __vcmpeq4(lb, msg_lo), eh = __vcmpeq4(lb, msg_hi);  // 0xff per match
#pragma unroll
            for (int t = 0; t < 4; ++t) {
              if (!(el & (1u << (8 * t)))) wl[t] = -CUDART_INF_F;
              if (!(eh & (1u << (8 * t)))) wh[t] = -CUDART_INF_F;
            }
          }
          mlo = fmaxf(fmaxf(wl[0], wl[1]), fmaxf(wl[2], wl[3]));
          mhi = fmaxf(fmaxf(wh[0], wh[1]), fmaxf(wh[2], wh[3]));
          mlo += nm2_lo;
          mhi += nm2_hi;
          // maxima over the quad's four column pairs: odd q keeps the upper row, even q the lower
          const float send = (q & 1) ? mlo : mhi;
          const float got = __shfl_xor_sync(0xffffffffu, send, 1);
          float amax = fmaxf((q & 1) ? mhi : mlo, got);
          amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, 2));
          const float nms = wp.ctx[my_row].nms;
          const bool in_range = cand0 + (long long)grp * 16 < N;
          const bool pass = tester && in_range &&
                            coarse_lower(w) <= exp2_upper_from_scaled(amax + margin, kLog2e * (1.0f / 126.0f), nms);
          const unsigned bal = __ballot_sync(0xffffffffu, pass);
          if (bal != 0u) {
            if (pass) {
              const int qi = qn + __popc(bal & lt);
              if (GLS_IN_RANGE(qi, 0, kMQueue, 35u))
                wp.queue[qi] = make_uint2(w, ((uint32_t)tile * 128u + (uint32_t)grp) | ((uint32_t)my_row << 28));
            }
            qn += __popc(bal);
            while (qn >= 32) {
              __syncwarp();
              qn -= 32;
              gauss_mma_flush<ROUNDS>(A, wp, qn, 32, N, scale, half_inv_prior);
            }
          }
        }
      }
    }
    if (qn > 0) {
      __syncwarp();
      gauss_mma_flush<ROUNDS>(A, wp, 0, qn, N, scale, half_inv_prior);
    }
    // ---- one partial result per (row, tile), written only if the tile produced a candidate
    __syncwarp();
    if (lane < kMRows) {
      const Top2 m = wp.best[lane];
      const int row = wp.ctx[lane].row;
      if (row >= 0 && m.i1 >= 0) {
        Partial pr;
        pr.s1 = m.s1; pr.i1 = m.i1; pr.s2 = m.s2; pr.i2 = m.i2;
        pr.lm = kGroupLseFloor; pr.ls = 0.f; pr.pad0 = 0; pr.pad1 = 0;
        if (GLS_IN_RANGE(tile, 0, A.parts, 36u) && GLS_IN_RANGE(row, 0, A.rows, 37u))
          A.partials[(long long)row * A.parts + tile] = pr;
      }
    }
  }
  asm volatile("griddepcontrol.launch_dependents;");
}

}  // namespace gls
