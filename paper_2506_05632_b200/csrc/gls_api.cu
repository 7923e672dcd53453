// gls_api.cu -- C ABI of libgls (see include/gls.h) and the small kernels around the sweep:
// the split-vocabulary reduction with exact re-scoring of the winner, and the per-sequence
// epilogues (Algorithm 2's active-set loop; the encoder / decoder bookkeeping of Sec. 5.1).
//
// All noise is evaluated by the device functions of gls_kernels.cuh, compiled once in this
// translation unit, so the draft-side, target-side and compression entry points see bit-identical
// shared randomness (the paper's analysis assumes identical floating-point behaviour on both
// sides of the coupling, Sec. 5.3).
#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>

#include "../../include/gls.h"
#include "gls_kernels.cuh"
#include "gls_group16.cuh"
#include "gls_sweep4.cuh"
#include "gls_topm.cuh"
#include "gls_gauss.cuh"
#include "gls_gauss_mma.cuh"

namespace gls {

// Number of SMs of the current device (grids and slice plans are sized from it); looked up once
// per device.  148 on B200; that value is also the answer when no device can be queried, so that
// gls_workspace_bytes() stays callable without one.
static int num_sms() {
  constexpr int kMaxDev = 64;
  static std::atomic<int> cache[kMaxDev];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDev) {
    (void)cudaGetLastError();
    return 148;
  }
  int n = cache[dev].load(std::memory_order_relaxed);
  if (n > 0) return n;
  if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
    (void)cudaGetLastError();
    return 148;
  }
  cache[dev].store(n, std::memory_order_relaxed);
  return n;
}
constexpr int kMinChunk = 2048;
constexpr int kMaxChunk = 16384;
// Target rows of a verify call, in bytes, from which Algorithm 2 is walked in phases (measured
// break-even with the walk that races every row first: 200 MB; 100 MB for Appendix B on a row per
// draft, whose rows cost K times the noise arithmetic)
#ifndef GLS_PHASED_MIN_BYTES
#define GLS_PHASED_MIN_BYTES 192e6
#endif
#ifndef GLS_THIRD_PHASE_MIN_BYTES
#define GLS_THIRD_PHASE_MIN_BYTES 256e6
#endif
#ifndef GLS_GAUSS_MMA
#define GLS_GAUSS_MMA 1
#endif
constexpr int kMaxPhases = 4;  // phases of such a walk (two are used: position 0, the rest)

struct Plan {
  int chunk, splits, parts;
  int chunk1, splits1, chunk2, splits2;  // two sets of rows swept by one launch each
  bool two_launches;
  int per_slice;  // partial results per slice (warps per CTA)
  long long rows, n_items;
  size_t off_hints, off_partials, off_rows, total;
};

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

static void plan_layout(Plan& p) {
  p.n_items = p.rows * p.splits;
  p.off_hints = 0;
  p.off_partials = align_up((size_t)p.rows * sizeof(uint32_t), 256);
  p.off_rows = p.off_partials + align_up((size_t)p.rows * p.parts * sizeof(Partial), 256);
  p.total = p.off_rows + align_up((size_t)p.rows * sizeof(RowResult), 256);
}

// noise_spec 1 (a warp per work item).  Slice size: aim at ~8 work items per resident warp
// so that the static round-robin over warps balances, but keep slices long enough to amortise
// the per-item reduction.
static Plan make_plan1(long long rows, long long V) {
  Plan p = Plan();
  const long long target_items = 8LL * num_sms() * 32;
  long long chunk = (rows * V + target_items - 1) / target_items;
  chunk = (chunk + kWarpTokens - 1) / kWarpTokens * kWarpTokens;
  if (chunk < kMinChunk) chunk = kMinChunk;
  if (chunk > kMaxChunk) chunk = kMaxChunk;
  const long long vceil = (V + kWarpTokens - 1) / kWarpTokens * kWarpTokens;
  if (chunk > vceil) chunk = vceil;
  p.chunk = (int)chunk;
  p.splits = (int)((V + chunk - 1) / chunk);
  p.parts = p.splits;
  p.rows = rows;
  plan_layout(p);
  return p;
}

// noise_spec 4 (a CTA per work item, one partial per warp).  Every item costs a fixed set-up and
// merge, so rows are cut into as few slices as keep the static round-robin over the resident
// CTAs balanced: the fewest slices for which the last round of items wastes at most 15 % of the
// machine, or that give every CTA at least 12 items.  Slices are whole CTA steps and at least four
// of them long, except that small problems may go down to one CTA step (2048 tokens per warp).
#ifndef GLS_S4_WASTE
#define GLS_S4_WASTE 0.15
#define GLS_S4_MIN_STEPS 4
#endif
template <int SH>
static Plan make_plan4_t(long long rows, long long V) {
  Plan p = Plan();
  constexpr int kCtaTok = S4Cfg<SH>::kCtaTokens;
  constexpr int kMinChunk = GLS_S4_MIN_STEPS * kCtaTok;
  const long long grid = (long long)num_sms() * S4Cfg<SH>::kCtasPerSM;
  long long max_splits = (V + kMinChunk - 1) / kMinChunk;
  if (rows * max_splits < 2 * grid) max_splits = (V + kCtaTok - 1) / kCtaTok;
  long long splits = 1;
  for (; splits < max_splits; ++splits) {
    const long long items = rows * splits;
    if (items >= 12 * grid) break;
    const long long rounds = (items + grid - 1) / grid;
    if (items >= grid && (double)(rounds * grid - items) <= GLS_S4_WASTE * (double)(rounds * grid)) break;
  }
  long long chunk = (V + splits - 1) / splits;
  chunk = (chunk + kCtaTok - 1) / kCtaTok * kCtaTok;
  p.chunk = (int)chunk;
  p.splits = (int)((V + chunk - 1) / chunk);
  p.parts = p.splits * S4Cfg<SH>::kWarps;
  p.rows = rows;
  plan_layout(p);
  return p;
}
// the sweep's launch shape for rows of V elements (multi: the fused multi-stream race)
static int s4_shape(int dtype, long long V, bool multi) {
  if (dtype == GLS_BF16) return kS4ShapeBf16;
  return (multi || V < kS4WideMinTokens) ? kS4ShapeF32Narrow : kS4ShapeF32Wide;
}
static Plan make_plan4(long long rows, long long V, int dtype, bool multi) {
  const int sh = s4_shape(dtype, V, multi);
  return sh == kS4ShapeBf16 ? make_plan4_t<kS4ShapeBf16>(rows, V)
         : sh == kS4ShapeF32Wide ? make_plan4_t<kS4ShapeF32Wide>(rows, V)
                                 : make_plan4_t<kS4ShapeF32Narrow>(rows, V);
}

// The fused draft + verify call (noise_spec 4): one launch over both sets while the input is small
// (the launches are what a small step costs), else one launch per set, each sliced for its own
// number of rows (the kernel specialised for its set is faster where the sweep is what a step costs).
static Plan make_plan_step(long long rows1, long long rows2, long long V, int dtype) {
  Plan p = make_plan4(rows1 + rows2, V, dtype, false);
#ifndef GLS_STEP_ONE_LAUNCH_BYTES
#define GLS_STEP_ONE_LAUNCH_BYTES 128e6
#endif
  p.two_launches = (double)(rows1 + rows2) * (double)V * (dtype == GLS_BF16 ? 2.0 : 4.0) > GLS_STEP_ONE_LAUNCH_BYTES;
  p.chunk1 = p.chunk2 = p.chunk;
  p.splits1 = p.splits2 = p.splits;
  if (p.two_launches) {
    const Plan a = make_plan4(rows1, V, dtype, false), b = make_plan4(rows2, V, dtype, false);
    p.per_slice = p.parts / p.splits;  // warps per CTA
    p.chunk1 = a.chunk;
    p.splits1 = a.splits;
    p.chunk2 = b.chunk;
    p.splits2 = b.splits;
    // first set: slots = its own slicing; the slot stride serves both sets
    p.splits = a.splits;
    p.chunk = a.chunk;
    p.parts = (a.splits > b.splits ? a.splits : b.splits) * p.per_slice;
    plan_layout(p);
    p.n_items = 0;
  }
  return p;
}

// Position-by-position verification (noise_spec 4): partial-result slots for the finest slicing a
// position can get, and after the hints and partials the state of the walk (active sets, row
// lists and their lengths) in place of the per-row results.
template <int SH>
static Plan make_plan_phased_t(int B, int K, int J, long long V) {
  Plan p = Plan();
  p.rows = (long long)B * K * J;
  p.chunk = 0;
  p.splits = listed_max_splits((int)V, S4Cfg<SH>::kCtaTokens);
  p.per_slice = S4Cfg<SH>::kWarps;
  p.parts = p.splits * S4Cfg<SH>::kWarps;
  plan_layout(p);
  p.total = p.off_rows + align_up((size_t)B * sizeof(unsigned long long), 256) +
            align_up((size_t)kMaxPhases * sizeof(int), 256) + align_up((size_t)J * B * K * sizeof(int), 256);
  return p;
}
static Plan make_plan_phased(int B, int K, int J, long long V, int dtype, bool multi = false) {
  const int sh = s4_shape(dtype, V, multi);
  return sh == kS4ShapeBf16 ? make_plan_phased_t<kS4ShapeBf16>(B, K, J, V)
         : sh == kS4ShapeF32Wide ? make_plan_phased_t<kS4ShapeF32Wide>(B, K, J, V)
                                 : make_plan_phased_t<kS4ShapeF32Narrow>(B, K, J, V);
}

static Plan make_plan(long long rows, long long V, int spec, int dtype, bool multi = false) {
  return spec == 4 ? make_plan4(rows, V, dtype, multi) : make_plan1(rows, V);
}

// ------------------------------------------------------------------------------------------
// Split-V reduction: one warp per row merges the slices' partials, re-scores the leading
// candidate(s) in fp64 and merges the softmax statistics.
//   out_mode 0: write RowResult only; 1: also write tokens / scores (draft side).
// ------------------------------------------------------------------------------------------
// Warp-collective; the result is valid in lane 0.
template <int DT, int SPEC, int ROUNDS>
__device__ __forceinline__ RowResult finalize_row(const SweepArgs& A, int row, int with_lse,
                                                  uint32_t* __restrict__ dev_status,
                                                  int parts_in_use = 0) {
  const int lane = threadIdx.x & 31;
  constexpr int ES = DT == kBF16 ? 2 : 4;
  const RowLoc rl = locate_row<ES>(A, row);
  const int j = rl.j, k = rl.k, b = rl.b;
  const float inv_t = rl.inv_t;
  const float c2 = inv_t * kLog2e;

  const int used = parts_in_use > 0 ? parts_in_use : rl.second ? A.parts2 : A.parts1;
  const int n_parts = used > 0 ? used : A.parts;  // slots in use
  Top2 best;
  top2_init(best);
  float lm = kLseFloor;
  for (int s = lane; s < n_parts; s += 32) {
    const Partial p = A.partials[(long long)row * A.parts + s];
    top2_offer(best, p.s1, p.i1);
    top2_offer(best, p.s2, p.i2);
    lm = fmaxf(lm, p.lm);
  }
  top2_warp_merge(best);
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) lm = fmaxf(lm, __shfl_xor_sync(0xffffffffu, lm, d));
  double lsum = 0.0;
  if (with_lse) {
    for (int s = lane; s < n_parts; s += 32) {
      const Partial p = A.partials[(long long)row * A.parts + s];
      if (p.ls > 0.f) lsum += (double)p.ls * exp2((double)(p.lm - lm) * (double)c2);
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, d);
  }
  RowResult r;
  r.pad0 = r.pad1 = r.pad2 = 0;
  r.idx = -1;
  r.score = -CUDART_INF;
  r.lse = -CUDART_INF;
  // Three independent fp64 chains run side by side: lane 0 re-scores the leader, lane 1 the
  // runner-up if it is closer than the fp32 error bound, lane 2 takes the logarithm of the sum.
  const float window = 2.0f * 0x1p-17f * (36.0f + fabsf(best.s1));
  const int code = lane == 0 ? best.i1 : best.i2;
  const bool want = (lane == 0 && best.i1 >= 0) ||
                    (lane == 1 && best.i1 >= 0 && best.i2 >= 0 && best.s1 - best.s2 <= window);
  double ex = -CUDART_INF;
  int tok = -1;
  if (want) {
    const char* rowp = rl.rowp;
    StreamKey sk;
    sk.c1 = ((uint32_t)k & A.kmask) | (A.domain << 16);
    sk.pos = A.pos_base + (uint32_t)j;
    sk.seq = A.seq_ids ? A.seq_ids[b] : A.seq_base + (uint32_t)b;
    // In the fused multi-stream race a candidate is (token << 3) | stream; ordering by that
    // code is "lowest token, then lowest stream", the tie rule.
    tok = code;
    if (A.multi_k > 0) {
      sk.c1 = (A.domain << 16) + ((uint32_t)code & 7u);
      tok = (int)((uint32_t)code >> 3);
    }
    ex = exact_score<DT, SPEC, ROUNDS>(A, rowp, sk, tok, inv_t, b, k);
  }
  double lse = -CUDART_INF;
  if (lane == 2 && with_lse && lsum > 0.0) lse = (double)lm * (double)inv_t + log(lsum);
  lse = __shfl_sync(0xffffffffu, lse, 2);
  const double e2 = __shfl_sync(0xffffffffu, ex, 1);
  const int tok2 = __shfl_sync(0xffffffffu, tok, 1);
  const bool want2 = __shfl_sync(0xffffffffu, (int)want, 1) != 0;
  if (lane != 0) return r;
  r.lse = lse;
  if (best.i1 < 0) {
    if (dev_status) atomicOr(dev_status, GLS_DEV_EMPTY_SUPPORT);
  } else {
    r.idx = tok;
    r.score = ex;
    if (want2 && (e2 > ex || (e2 == ex && best.i2 < best.i1))) {
      r.idx = tok2;
      r.score = e2;
    }
  }
  return r;
}

template <int DT, int SPEC, int ROUNDS>
__global__ void __launch_bounds__(128)
finalize_rows_kernel(const __grid_constant__ SweepArgs A, int rows, int with_lse,
                     RowResult* __restrict__ rowres, int32_t* __restrict__ out_tokens,
                     float* __restrict__ out_scores, uint32_t* __restrict__ dev_status) {
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the sweep before this launch is complete
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= rows) return;
  const RowResult r = finalize_row<DT, SPEC, ROUNDS>(A, row, with_lse, dev_status);
  if ((threadIdx.x & 31) != 0) return;
  if (rowres) rowres[row] = r;
  if (out_tokens) out_tokens[row] = r.idx;
  if (out_scores) out_scores[row] = r.idx >= 0 ? (float)r.score : CUDART_NAN_F;
}

// ------------------------------------------------------------------------------------------
// Algorithm 2, verification phase (active-set initialisation to the end); one thread per sequence.
// rows[(b*K + k)*J + j] holds the winner of row (b,k,j) under its own noise stream.
// ------------------------------------------------------------------------------------------
// `rows` points at the K x J results of sequence b: rows[k * J + j].
__device__ void verify_sequence(const RowResult* rows, int b, int K, int L, int J, uint32_t flags,
                                bool multi_rows, const int32_t* __restrict__ draft_tokens,
                                int32_t* __restrict__ out_tokens, int32_t* __restrict__ out_num,
                                uint8_t* __restrict__ accept, float* __restrict__ out_scores,
                                uint32_t* __restrict__ dev_status) {
  unsigned long long active = K >= 64 ? ~0ull : ((1ull << K) - 1ull);
  for (int j = 0; j < J; ++j) {
    out_tokens[(long long)b * J + j] = -1;
    if (out_scores) out_scores[(long long)b * J + j] = 0.f;
  }
  for (long long t = 0; t < (long long)K * L; ++t) accept[(long long)b * K * L + t] = 0;
  int n_out = 0;
  for (int j = 0; j < J; ++j) {
    // Y_j = argmin_i min_{k in S} S_i^(j,k) / q_i^(j,k)  ==  best of the rows' winners after
    // subtracting each row's log-sum-exp; ties: lowest token, then lowest k
    double bs = 0.0;
    int bi = -1;
    // Appendix B on rows raced under all K streams at once: the target distribution of the
    // accepted prefix is the row of any draft that is still active; take the lowest such k
    const int kref = multi_rows ? __ffsll((long long)active) - 1 : -1;
    for (int k = 0; k < K; ++k) {
      if (multi_rows ? (k != kref) : (!((active >> k) & 1ull) && !(flags & GLS_COMBINE_ALL))) continue;
      const RowResult r = rows[(long long)k * J + j];
      if (r.idx < 0) continue;
      const double sc = r.score - r.lse;
      if (bi < 0 || sc > bs || (sc == bs && r.idx < bi)) {
        bs = sc;
        bi = r.idx;
      }
    }
    out_tokens[(long long)b * J + j] = bi;
    if (out_scores) out_scores[(long long)b * J + j] = bi >= 0 ? (float)bs : CUDART_NAN_F;
    if (bi < 0 && dev_status) atomicOr(dev_status, GLS_DEV_EMPTY_SUPPORT);
    n_out = j + 1;
    if (j == L) break;  // bonus token
    unsigned long long next = 0ull;
    for (int k = 0; k < K; ++k) {
      const bool ok = ((active >> k) & 1ull) && bi >= 0 &&
                      draft_tokens[((long long)b * K + k) * L + j] == bi;
      accept[((long long)b * K + k) * L + j] = ok ? 1 : 0;
      if (ok) next |= 1ull << k;
    }
    active = next;
    if (active == 0ull) break;
  }
  out_num[b] = n_out;
}

// The same loop run by one warp: lane l looks after drafts l and l + 32, so the list combine is a
// warp argmax, the pruning a ballot, and the outputs are written in parallel; only the walk over
// the positions is sequential.  `dtok` holds the sequence's draft tokens [K][L] (shared memory).
// Result identical to verify_sequence().
__device__ void verify_sequence_warp(const RowResult* rows, int b, int K, int L, int J, uint32_t flags,
                                     bool multi_rows, const int32_t* dtok,
                                     int32_t* __restrict__ out_tokens, int32_t* __restrict__ out_num,
                                     uint8_t* __restrict__ accept, float* __restrict__ out_scores,
                                     uint32_t* __restrict__ dev_status) {
  const int lane = threadIdx.x & 31;
  unsigned long long active = K >= 64 ? ~0ull : ((1ull << K) - 1ull);
  int n_out = 0;
  for (int j = 0; j < J; ++j) {
    const int kref = multi_rows ? __ffsll((long long)active) - 1 : -1;
    double bs = -CUDART_INF;
    int bi = -1;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int k = lane + 32 * h;
      if (k >= K) continue;
      if (multi_rows ? (k != kref) : (!((active >> k) & 1ull) && !(flags & GLS_COMBINE_ALL))) continue;
      const RowResult r = rows[(long long)k * J + j];
      if (r.idx < 0) continue;
      const double sc = r.score - r.lse;
      if (bi < 0 || sc > bs || (sc == bs && r.idx < bi)) {
        bs = sc;
        bi = r.idx;
      }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      const double os = __shfl_xor_sync(0xffffffffu, bs, d);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, d);
      if (oi >= 0 && (bi < 0 || os > bs || (os == bs && oi < bi))) {
        bs = os;
        bi = oi;
      }
    }
    if (lane == 0) {
      out_tokens[(long long)b * J + j] = bi;
      if (out_scores) out_scores[(long long)b * J + j] = bi >= 0 ? (float)bs : CUDART_NAN_F;
      if (bi < 0 && dev_status) atomicOr(dev_status, GLS_DEV_EMPTY_SUPPORT);
    }
    n_out = j + 1;
    if (j == L) break;  // bonus token
    unsigned long long next = 0ull;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int k = lane + 32 * h;
      const bool ok = k < K && ((active >> k) & 1ull) && bi >= 0 && dtok[k * L + j] == bi;
      if (k < K) accept[((long long)b * K + k) * L + j] = ok ? 1 : 0;
      next |= (unsigned long long)__ballot_sync(0xffffffffu, ok) << (32 * h);
    }
    active = next;
    if (active == 0ull) break;
  }
  // what lies beyond the stopping time: token -1, score 0, not accepted
  for (int j = n_out + lane; j < J; j += 32) {
    out_tokens[(long long)b * J + j] = -1;
    if (out_scores) out_scores[(long long)b * J + j] = 0.f;
  }
  for (int t = lane; t < K * L; t += 32)
    if (t % L >= n_out) accept[(long long)b * K * L + t] = 0;
  if (lane == 0) out_num[b] = n_out;
}

__global__ void verify_epilogue_kernel(const RowResult* __restrict__ rows, int B, int K, int L,
                                       int J, uint32_t flags, bool multi_rows,
                                       const int32_t* __restrict__ draft_tokens,
                                       int32_t* __restrict__ out_tokens,
                                       int32_t* __restrict__ out_num, uint8_t* __restrict__ accept,
                                       float* __restrict__ out_scores,
                                       uint32_t* __restrict__ dev_status) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  verify_sequence(rows + (long long)b * K * J, b, K, L, J, flags, multi_rows, draft_tokens, out_tokens,
                  out_num, accept, out_scores, dev_status);
}

// Split-V reduction and Algorithm 2's loop in one launch: a CTA per sequence finalises the
// sequence's K x J rows into shared memory (a warp per row), then one thread walks the positions.
struct VerifyArgs {
  int B, K, L, J;
  uint32_t flags;
  bool multi_rows;  // every row result is the best over all K noise streams (Appendix B)
  bool three_phases;  // the walk in phases: positions 1 and 2 as a phase of their own (forced)
  const int32_t* draft_tokens;
  int32_t* out_tokens;
  int32_t* out_num;
  uint8_t* accept;
  float* out_scores;
  uint32_t* dev_status;
};
constexpr int kFusedVerifyMaxWarps = 32;  // one warp per row result, up to a full CTA
constexpr size_t kFusedVerifyMaxSmem = 48 * 1024;
// a sequence's K x J row results and its K x L draft tokens
static size_t fused_verify_smem(int K, int L, int J) {
  return (size_t)K * J * sizeof(RowResult) + (size_t)K * (L > 0 ? L : 1) * sizeof(int32_t);
}
template <int DT, int SPEC, int ROUNDS>
__global__ void __launch_bounds__(kFusedVerifyMaxWarps * 32)
finalize_verify_kernel(const __grid_constant__ SweepArgs A, const VerifyArgs va) {
  RowResult* srows = reinterpret_cast<RowResult*>(gls_smem_raw);
  const int b = blockIdx.x;
  const int nrows = va.K * va.J;
  // the sequence's draft tokens, fetched while the sweep is still draining (they were written
  // by work that completed before the sweep started)
  int32_t* dtok = reinterpret_cast<int32_t*>(srows + nrows);
  for (int t = threadIdx.x; t < va.K * va.L; t += (int)blockDim.x)
    dtok[t] = va.draft_tokens[(long long)b * va.K * va.L + t];
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the sweep before this launch is complete
  for (int r = threadIdx.x >> 5; r < nrows; r += (int)(blockDim.x >> 5)) {
    const RowResult rr = finalize_row<DT, SPEC, ROUNDS>(A, b * nrows + r, 1, nullptr);
    if ((threadIdx.x & 31) == 0) srows[r] = rr;
  }
  __syncthreads();
  if (threadIdx.x < 32)
    verify_sequence_warp(srows, b, va.K, va.L, va.J, va.flags, va.multi_rows, dtok, va.out_tokens,
                         va.out_num, va.accept, va.out_scores, va.dev_status);
}

// ------------------------------------------------------------------------------------------
// Algorithm 2 in phases.  Y_j needs the target rows of the drafts that are still active at
// position j and nothing else, and nothing at all is needed past the stopping time, so the
// verification can read far fewer rows than the call is given.  The positions are cut into
// phases [j0, j1); a phase sweeps the rows (b, k, j) of its positions for the drafts k active
// when it starts (sweep4_listed_kernel over a row list in device memory), then one kernel reduces
// them, walks the phase's positions (emits Y_j, prunes the active set) and lists the rows of the
// next phase.  The first phase is position 0 alone, where every draft is active; most drafts
// are pruned there, so the second phase takes all remaining positions of the few survivors.
// State in the workspace: the active set of every sequence, a row list and its length per phase.
// ------------------------------------------------------------------------------------------
// The phases of such a walk over J positions: ends[p] = one past the last position of phase p.
static int phase_ends(int B, int J, long long V, int elt_bytes, int ends[kMaxPhases], bool three = false) {
  int n = 0;
  ends[n++] = 1;
  if (J > 3 && (three || (double)B * (J - 3) * (double)V * elt_bytes >= GLS_THIRD_PHASE_MIN_BYTES))
    ends[n++] = 3;
  if (J > 1) ends[n++] = J;
  return n;
}

struct PhasedState {
  unsigned long long* active;  // [B]
  int* counts;                 // [kMaxPhases]
  int* lists;                  // phase p at lists + B * K * (its first position): row numbers
};

__global__ void phased_init_kernel(const VerifyArgs va, const PhasedState S, int first_end,
                                   uint32_t* __restrict__ hints) {
  asm volatile("griddepcontrol.launch_dependents;");  // the first sweep may be scheduled
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long BK = (long long)va.B * va.K;
  // first phase: every draft is active at positions [0, first_end); Appendix B on a row per draft
  // reads the row of the lowest active draft only, draft 0 at position 0
  if (va.multi_rows) {
    if (t < (long long)va.B * first_end) S.lists[t] = (int)((t / first_end) * va.K * va.J + t % first_end);
  } else if (t < BK * first_end) {
    S.lists[t] = (int)((t / first_end) * va.J + t % first_end);
  }
  if (t < va.B) {
    S.active[t] = va.K >= 64 ? ~0ull : ((1ull << va.K) - 1ull);
    va.out_num[t] = 0;
  }
  if (t < kMaxPhases) S.counts[t] = t == 0 ? (int)((va.multi_rows ? va.B : BK) * first_end) : 0;
  if (hints != nullptr && t < BK * va.J) hints[t] = 0u;
  if (t < (long long)va.B * va.J) {
    va.out_tokens[t] = -1;
    if (va.out_scores) va.out_scores[t] = 0.f;
  }
  if (t < BK * va.L) va.accept[t] = 0;
}

// One warp walks positions [j0, j1) of sequence b on the row results srows[k * (j1 - j0) + j - j0]
// (valid for the drafts in `active`): emits Y_j, prunes the active set, and either lists the
// survivors' rows at the next phase's positions [j1, j2) or closes the sequence.
__device__ void phased_walk(const RowResult* srows, unsigned long long active, const VerifyArgs& va,
                            const PhasedState& S, int b, int phase, int j0, int j1, int j2) {
  const int lane = threadIdx.x & 31;
  const int K = va.K, L = va.L, J = va.J, W = j1 - j0;
  int n_out = j0;
  for (int j = j0; j < j1; ++j) {
    // Y_j: the best of the active rows' winners after subtracting each row's log-sum-exp; ties:
    // lowest token, then lowest k.  Appendix B on a row per draft: the row of the lowest active
    // draft, which was raced under all K streams.
    const int kref = va.multi_rows ? __ffsll((long long)active) - 1 : -1;
    double bs = -CUDART_INF;
    int bi = -1;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int k = lane + 32 * h;
      if (k >= K || !((active >> k) & 1ull)) continue;
      if (va.multi_rows && k != kref) continue;
      const RowResult r = srows[k * W + (j - j0)];
      if (r.idx < 0) continue;
      const double sc = r.score - r.lse;
      if (bi < 0 || sc > bs || (sc == bs && r.idx < bi)) {
        bs = sc;
        bi = r.idx;
      }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      const double os = __shfl_xor_sync(0xffffffffu, bs, d);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, d);
      if (oi >= 0 && (bi < 0 || os > bs || (os == bs && oi < bi))) {
        bs = os;
        bi = oi;
      }
    }
    if (lane == 0) {
      va.out_tokens[(long long)b * J + j] = bi;
      if (va.out_scores) va.out_scores[(long long)b * J + j] = bi >= 0 ? (float)bs : CUDART_NAN_F;
      if (bi < 0 && va.dev_status) atomicOr(va.dev_status, GLS_DEV_EMPTY_SUPPORT);
    }
    n_out = j + 1;
    if (j == L) {  // bonus token
      active = 0ull;
      break;
    }
    unsigned long long next = 0ull;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int k = lane + 32 * h;
      const bool ok = k < K && ((active >> k) & 1ull) && bi >= 0 &&
                      va.draft_tokens[((long long)b * K + k) * L + j] == bi;
      if (ok) va.accept[((long long)b * K + k) * L + j] = 1;
      next |= (unsigned long long)__ballot_sync(0xffffffffu, ok) << (32 * h);
    }
    active = next;
    if (active == 0ull) break;
  }
  if (n_out >= J) active = 0ull;
  if (active != 0ull) {  // the survivors' rows at the positions of the next phase
    const int W2 = j2 - j1;
    int base = 0;
    if (lane == 0) base = atomicAdd(&S.counts[phase + 1], __popcll(active) * W2);
    base = __shfl_sync(0xffffffffu, base, 0);
    int* list = S.lists + (long long)va.B * K * j1;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int k = lane + 32 * h;
      if (k < K && ((active >> k) & 1ull)) {
        const int rank = __popcll(active & ((1ull << k) - 1ull));
        for (int jj = 0; jj < W2; ++jj) list[base + rank * W2 + jj] = (b * K + k) * J + j1 + jj;
      }
    }
  }
  if (lane == 0) {
    S.active[b] = active;
    if (active == 0ull) va.out_num[b] = n_out;
  }
}

// Phase `phase` = positions [j0, j1) of every sequence that is still running; the next phase (if
// any) is [j1, j2).  A CTA per sequence, a warp per listed row, then one warp walks the positions.
template <int DT, int ROUNDS>
__global__ void __launch_bounds__(kFusedVerifyMaxWarps * 32)
phased_verify_kernel(const __grid_constant__ SweepArgs A, const VerifyArgs va, const PhasedState S,
                     int phase, int j0, int j1, int j2, int cta_tokens, int sweep_grid,
                     int warps_per_slice) {
  RowResult* srows = reinterpret_cast<RowResult*>(gls_smem_raw);  // [K][j1 - j0]
  const int b = blockIdx.x;
  const int lane = threadIdx.x & 31;
  unsigned long long active = S.active[b];  // written by the previous phase, complete by now
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the sweep before this launch is complete
  asm volatile("griddepcontrol.launch_dependents;");  // the next phase's sweep may be scheduled
  if (active == 0ull) return;
  const int K = va.K, J = va.J, W = j1 - j0;
  const ListedSlicing sl = listed_slicing(S.counts[phase], A.V, cta_tokens, sweep_grid);
  for (int r = threadIdx.x >> 5; r < K * W; r += (int)(blockDim.x >> 5)) {
    const int k = r / W, j = j0 + r % W;
    if (!((active >> k) & 1ull)) continue;
    if (va.multi_rows && j0 == 0 && k != 0) continue;  // the first phase listed draft 0 only
    const RowResult rr = finalize_row<DT, 4, ROUNDS>(A, (b * K + k) * J + j, 1, nullptr,
                                                     sl.splits * warps_per_slice);
    if (lane == 0) srows[r] = rr;
  }
  __syncthreads();
  if (threadIdx.x < 32) phased_walk(srows, active, va, S, b, phase, j0, j1, j2);
}

// The fused draft + verify call: a CTA per sequence finalises the sequence's K x L draft rows
// (tokens and scores go to the caller and into shared memory) and its K x J target rows, then a
// warp runs Algorithm 2's loop on them.
template <int DT, int SPEC, int ROUNDS>
__global__ void __launch_bounds__(kFusedVerifyMaxWarps * 32)
finalize_step_kernel(const __grid_constant__ SweepArgs A, const VerifyArgs va,
                     int32_t* __restrict__ out_draft_tokens, float* __restrict__ out_draft_scores) {
  asm volatile("griddepcontrol.wait;" ::: "memory");  // the sweep before this launch is complete
  RowResult* srows = reinterpret_cast<RowResult*>(gls_smem_raw);
  const int b = blockIdx.x;
  const int nd = va.K * va.L, nt = va.K * va.J;
  int32_t* dtok = reinterpret_cast<int32_t*>(srows + nt);
  for (int r = threadIdx.x >> 5; r < nd + nt; r += (int)(blockDim.x >> 5)) {
    if (r < nd) {
      const RowResult rr = finalize_row<DT, SPEC, ROUNDS>(A, b * nd + r, 0, va.dev_status);
      if ((threadIdx.x & 31) == 0) {
        dtok[r] = rr.idx;
        out_draft_tokens[(long long)b * nd + r] = rr.idx;
        if (out_draft_scores)
          out_draft_scores[(long long)b * nd + r] = rr.idx >= 0 ? (float)rr.score : CUDART_NAN_F;
      }
    } else {
      const RowResult rr = finalize_row<DT, SPEC, ROUNDS>(A, A.rows1 + b * nt + (r - nd), 1, nullptr);
      if ((threadIdx.x & 31) == 0) srows[r - nd] = rr;
    }
  }
  __syncthreads();
  if (threadIdx.x < 32)
    verify_sequence_warp(srows, b, va.K, va.L, va.J, va.flags, va.multi_rows, dtok, va.out_tokens,
                         va.out_num, va.accept, va.out_scores, va.dev_status);
}

// Sec. 5.1 encoder bookkeeping: Y = best over the K streams of the encoder row, M = l_Y.
__global__ void encoder_epilogue_kernel(const RowResult* __restrict__ rows, int B, int K,
                                        const uint8_t* __restrict__ bins, long long bins_sb,
                                        int32_t* __restrict__ enc_index,
                                        uint8_t* __restrict__ message,
                                        float* __restrict__ out_scores,
                                        uint32_t* __restrict__ dev_status, int score_stride) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  double bs = 0.0;
  int bi = -1;
  for (int k = 0; k < K; ++k) {
    const RowResult r = rows[(long long)b * K + k];
    if (r.idx < 0) continue;
    const double sc = r.score - r.lse;
    if (bi < 0 || sc > bs || (sc == bs && r.idx < bi)) {
      bs = sc;
      bi = r.idx;
    }
  }
  enc_index[b] = bi;
  message[b] = (bins && bi >= 0) ? bins[bins_sb * b + bi] : (uint8_t)0;
  if (out_scores) out_scores[(long long)b * score_stride] = bi >= 0 ? (float)bs : CUDART_NAN_F;
  if (bi < 0 && dev_status) atomicOr(dev_status, GLS_DEV_EMPTY_SUPPORT);
}

// Sec. 5.1 decoder bookkeeping: X^(k) per decoder and the match flag Y in {X^(k)}.
__global__ void decoder_epilogue_kernel(const RowResult* __restrict__ rows, int B, int K,
                                        const int32_t* __restrict__ enc_index,
                                        int32_t* __restrict__ dec_index,
                                        uint8_t* __restrict__ match,
                                        float* __restrict__ out_scores) {
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const int y = enc_index[b];
  int hit = 0;
  for (int k = 0; k < K; ++k) {
    const RowResult r = rows[(long long)b * K + k];
    dec_index[(long long)b * K + k] = r.idx;
    if (out_scores)
      out_scores[(long long)b * (1 + K) + 1 + k] = r.idx >= 0 ? (float)r.score : CUDART_NAN_F;
    if (r.idx >= 0 && r.idx == y) hit = 1;
  }
  match[b] = (uint8_t)hit;
}

// ------------------------------------------------------------------------------------------
// Sparse rows (Sec. 4.4: top-K truncation keeps M << N tokens).  A warp scores all kept tokens of
// a row directly in fp64 -- logit/T - ln(-log1p(-v)), v keyed by the token's vocabulary id -- so
// no filter, queue or workspace is involved.  Warp-collective; the result is valid in lane 0.
// ------------------------------------------------------------------------------------------
struct SparseArgs {
  const int32_t* ids;
  const float* logits;
  long long sb, sk, sj;
  int M;
};

__device__ __forceinline__ bool sparse_keep(int id, float a) {
  return id >= 0 && a < CUDART_INF_F && a > -CUDART_INF_F;  // false for NaN, +inf and masked tokens
}

template <int SPEC, int ROUNDS>
__device__ __forceinline__ RowResult sparse_row(const SweepArgs& A, const SparseArgs& S, int row,
                                                uint32_t* __restrict__ dev_status) {
  const int lane = threadIdx.x & 31;
  const int j = row % A.J;
  const int bk = row / A.J;
  const int k = bk % A.K;
  const int b = bk / A.K;
  const long long base = b * S.sb + k * S.sk + j * S.sj;
  const double inv_t = (double)A.inv_t[k];
  StreamKey sk;
  sk.c1 = ((uint32_t)k & A.kmask) | (A.domain << 16);
  sk.pos = A.pos_base + (uint32_t)j;
  sk.seq = A.seq_ids ? A.seq_ids[b] : A.seq_base + (uint32_t)b;
  double best = -CUDART_INF, amax = -CUDART_INF;
  int bid = -1;
  // multi_k > 0: the list is raced under the streams 0 .. multi_k-1 together (Appendix B); a
  // token that ties with itself under two streams is one token, so only the score matters
  const int n_streams = A.multi_k > 0 ? A.multi_k : 1;
  for (int m = lane; m < S.M; m += 32) {
    const int id = __ldg(S.ids + base + m);
    const float a = __ldg(S.logits + base + m);
    if (!sparse_keep(id, a)) continue;
    const double al = (double)a * inv_t;
    amax = fmax(amax, al);
    for (int ks = 0; ks < n_streams; ++ks) {
      if (A.multi_k > 0) sk.c1 = ((uint32_t)ks & A.kmask) | (A.domain << 16);
      const double sc = al - log(noise_exact<SPEC, ROUNDS>(A, sk, id));
      if (bid < 0 || sc > best || (sc == best && id < bid)) {
        best = sc;
        bid = id;
      }
    }
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) {
    const double ob = __shfl_xor_sync(0xffffffffu, best, d);
    const int oi = __shfl_xor_sync(0xffffffffu, bid, d);
    amax = fmax(amax, __shfl_xor_sync(0xffffffffu, amax, d));
    if (oi >= 0 && (bid < 0 || ob > best || (ob == best && oi < bid))) {
      best = ob;
      bid = oi;
    }
  }
  double sum = 0.0;
  if (bid >= 0) {
    for (int m = lane; m < S.M; m += 32) {
      const int id = __ldg(S.ids + base + m);
      const float a = __ldg(S.logits + base + m);
      if (sparse_keep(id, a)) sum += exp((double)a * inv_t - amax);
    }
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, d);
  RowResult r;
  r.pad0 = r.pad1 = r.pad2 = 0;
  r.idx = bid;
  r.score = bid >= 0 ? best : -CUDART_INF;
  r.lse = bid >= 0 ? amax + log(sum) : -CUDART_INF;
  if (bid < 0 && dev_status && lane == 0) atomicOr(dev_status, GLS_DEV_EMPTY_SUPPORT);
  return r;
}

template <int SPEC, int ROUNDS>
__global__ void __launch_bounds__(128)
sparse_draft_kernel(const __grid_constant__ SweepArgs A, const SparseArgs S, int rows,
                    int32_t* __restrict__ out_tokens, float* __restrict__ out_scores,
                    uint32_t* __restrict__ dev_status) {
  const int row = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= rows) return;
  const RowResult r = sparse_row<SPEC, ROUNDS>(A, S, row, dev_status);
  if ((threadIdx.x & 31) != 0) return;
  out_tokens[row] = r.idx;
  if (out_scores) out_scores[row] = r.idx >= 0 ? (float)r.score : CUDART_NAN_F;
}

// a CTA per sequence: a warp per row result into shared memory, then Algorithm 2's loop
template <int SPEC, int ROUNDS>
__global__ void __launch_bounds__(kFusedVerifyMaxWarps * 32)
sparse_verify_kernel(const __grid_constant__ SweepArgs A, const SparseArgs S, const VerifyArgs va) {
  RowResult* srows = reinterpret_cast<RowResult*>(gls_smem_raw);
  const int b = blockIdx.x;
  const int nrows = va.K * va.J;
  for (int r = threadIdx.x >> 5; r < nrows; r += (int)(blockDim.x >> 5)) {
    const RowResult rr = sparse_row<SPEC, ROUNDS>(A, S, b * nrows + r, nullptr);
    if ((threadIdx.x & 31) == 0) srows[r] = rr;
  }
  int32_t* dtok = reinterpret_cast<int32_t*>(srows + nrows);
  for (int t = threadIdx.x; t < va.K * va.L; t += (int)blockDim.x)
    dtok[t] = va.draft_tokens[(long long)b * va.K * va.L + t];
  __syncthreads();
  if (threadIdx.x < 32)
    verify_sequence_warp(srows, b, va.K, va.L, va.J, va.flags, va.multi_rows, dtok, va.out_tokens,
                         va.out_num, va.accept, va.out_scores, va.dev_status);
}

// Algorithm 2 in phases on sparse rows (the lists of a phase were selected just before): as
// phased_verify_kernel, with the row results computed from the lists.
template <int SPEC, int ROUNDS>
__global__ void __launch_bounds__(kFusedVerifyMaxWarps * 32)
sparse_phased_kernel(const __grid_constant__ SweepArgs A, const SparseArgs Sp, const VerifyArgs va,
                     const PhasedState S, int phase, int j0, int j1, int j2) {
  RowResult* srows = reinterpret_cast<RowResult*>(gls_smem_raw);  // [K][j1 - j0]
  const int b = blockIdx.x;
  const unsigned long long active = S.active[b];
  if (active == 0ull) return;
  const int K = va.K, J = va.J, W = j1 - j0;
  for (int r = threadIdx.x >> 5; r < K * W; r += (int)(blockDim.x >> 5)) {
    const int k = r / W, j = j0 + r % W;
    if (!((active >> k) & 1ull)) continue;
    if (va.multi_rows && j0 == 0 && k != 0) continue;  // the first phase listed draft 0 only
    const RowResult rr = sparse_row<SPEC, ROUNDS>(A, Sp, (b * K + k) * J + j, nullptr);
    if ((threadIdx.x & 31) == 0) srows[r] = rr;
  }
  __syncthreads();
  if (threadIdx.x < 32) phased_walk(srows, active, va, S, b, phase, j0, j1, j2);
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
static bool finite_pos(float x) { return std::isfinite(x) && x > 0.f; }

static int fill_noise(SweepArgs& A, const gls_noise_t* nz, uint32_t domain, int* spec_out) {
  const int rounds = nz->rounds ? (int)nz->rounds : 10;
  if (rounds < 7 || rounds > 16) return GLS_ERR_INVALID_ARG;
  const int spec = nz->noise_spec ? (int)nz->noise_spec : 4;
  if (spec < 1 || spec > 4) return GLS_ERR_INVALID_ARG;
  if (spec == 2 || spec == 3) return GLS_ERR_UNSUPPORTED;  // retired bit-splitting layouts
  if (nz->flags & ~GLS_NOISE_SHARED_ACROSS_K) return GLS_ERR_INVALID_ARG;
  uint32_t k0 = (uint32_t)(nz->seed & 0xffffffffu), k1 = (uint32_t)(nz->seed >> 32);
  for (int r = 0; r < 16; ++r) {
    A.rk[2 * r] = k0;
    A.rk[2 * r + 1] = k1;
    k0 += kPhiloxW0;
    k1 += kPhiloxW1;
  }
  A.rounds = rounds;
  A.seq_base = nz->seq_base;
  A.seq_ids = nz->seq_ids;
  A.pos_base = nz->pos_base;
  A.domain = domain;
  A.kmask = (nz->flags & GLS_NOISE_SHARED_ACROSS_K) ? 0u : 0xffffu;
  *spec_out = spec;
  return GLS_OK;
}

static int check_rows(const gls_rows_t* r) {
  if (!r || !r->data) return GLS_ERR_INVALID_ARG;
  if (r->dtype != GLS_F32 && r->dtype != GLS_BF16) return GLS_ERR_UNSUPPORTED;
  const uintptr_t es = r->dtype == GLS_F32 ? 4 : 2;
  if (((uintptr_t)r->data) % es) return GLS_ERR_MISALIGNED;
  return GLS_OK;
}

template <int DT, int ROUNDS>
static cudaError_t launch_sweep_t(const SweepArgs& A, bool lse, int grid, cudaStream_t st) {
  if (lse)
    sweep_kernel<DT, true, ROUNDS><<<grid, kSweepThreads, 0, st>>>(A);
  else
    sweep_kernel<DT, false, ROUNDS><<<grid, kSweepThreads, 0, st>>>(A);
  return cudaGetLastError();
}

// The reduction kernels are launched as programmatic dependents of the sweep before them in the
// stream: their blocks may be scheduled while the sweep drains (the sweep signals that its
// block is done), and wait at their first instruction until the whole sweep has completed and its
// writes are visible.  This hides the launch latency between the two kernels of a call.
static cudaLaunchConfig_t dependent_launch(cudaLaunchAttribute* attr, int grid, int block,
                                           size_t smem, cudaStream_t st) {
  attr->id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr->val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3((unsigned)block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cfg;
}

template <int DT, int SPEC, int ROUNDS>
static cudaError_t launch_finalize_t(const SweepArgs& A, int rows, bool lse, RowResult* rowres,
                                     int32_t* out_tokens, float* out_scores, uint32_t* status,
                                     cudaStream_t st) {
  const int wpb = 4;
  cudaLaunchAttribute attr;
  cudaLaunchConfig_t cfg = dependent_launch(&attr, (rows + wpb - 1) / wpb, wpb * 32, 0, st);
  return cudaLaunchKernelEx(&cfg, finalize_rows_kernel<DT, SPEC, ROUNDS>, A, rows, lse ? 1 : 0, rowres,
                            out_tokens, out_scores, status);
}

// sweep + split reduction of one batch of rows
// The launch size for n_items work items dealt round-robin to at most `cap` resident CTAs: the
// smallest grid that needs no more rounds than `cap` would, so that every CTA gets the same
// number of items (to within one) and no last round runs on a fraction of the machine.
static int even_grid(long long n_items, long long cap) {
  if (n_items <= cap) return (int)(n_items > 0 ? n_items : 1);
  const long long rounds = (n_items + cap - 1) / cap;
  return (int)((n_items + rounds - 1) / rounds);
}
// Measured: the eight-warp shape gains from the even deal (config 5, whole call 1.754 -> 1.714 ms);
// the one-warp shapes lose when every CTA runs the same number of items in step with all others
// (config 3, every row raced: 0.178 -> 0.200 ms) and keep one CTA per resident slot.
template <int SH>
static int sweep_grid(long long n_items, long long cap) {
  if (S4Cfg<SH>::kWarps > 1) return even_grid(n_items, cap);
  return (int)(n_items < cap ? (n_items > 0 ? n_items : 1) : cap);
}

template <int DT, int SPEC, int ROUNDS>
static cudaError_t launch_fused_verify_t(const SweepArgs& A, const VerifyArgs& va, cudaStream_t st) {
  const size_t smem = fused_verify_smem(va.K, va.L, va.J);
  const int nrows = va.K * va.J;
  const int warps = nrows < kFusedVerifyMaxWarps ? nrows : kFusedVerifyMaxWarps;
  cudaLaunchAttribute attr;
  cudaLaunchConfig_t cfg = dependent_launch(&attr, va.B, warps * 32, smem, st);
  return cudaLaunchKernelEx(&cfg, finalize_verify_kernel<DT, SPEC, ROUNDS>, A, va);
}

struct StepOut {  // the draft-side outputs of the fused draft + verify call
  int32_t* draft_tokens;
  float* draft_scores;
};
template <int DT, int SPEC, int ROUNDS>
static cudaError_t launch_step_t(const SweepArgs& A, const VerifyArgs& va, const StepOut& so,
                                 cudaStream_t st) {
  const size_t smem = fused_verify_smem(va.K, va.L, va.J);
  const int nrows = va.K * (va.L + va.J);
  const int warps = nrows < kFusedVerifyMaxWarps ? nrows : kFusedVerifyMaxWarps;
  cudaLaunchAttribute attr;
  cudaLaunchConfig_t cfg = dependent_launch(&attr, va.B, warps * 32, smem, st);
  return cudaLaunchKernelEx(&cfg, finalize_step_kernel<DT, SPEC, ROUNDS>, A, va, so.draft_tokens,
                            so.draft_scores);
}

// sweep + split reduction of one batch of rows.  With `va` (verification) and a sequence's
// K x J row results fitting in shared memory, the reduction and Algorithm 2's loop run as one
// launch and *fused is set; otherwise the rows' results are left in the workspace.
static int run_rows(SweepArgs& A, int dtype, int spec, const Plan& P, void* workspace, bool lse,
                    int32_t* out_tokens, float* out_scores, uint32_t* status, cudaStream_t st,
                    const VerifyArgs* va = nullptr, bool* fused = nullptr,
                    const StepOut* step = nullptr) {
  char* ws = (char*)workspace;
  A.chunk = P.chunk;
  A.splits = P.splits;
  A.parts = P.parts;
  A.rows = (int)P.rows;
  A.n_items = P.n_items;
  A.row_begin = 0;
  A.row_count = (int)P.rows;
  A.parts1 = P.two_launches ? P.splits1 * P.per_slice : 0;
  A.parts2 = P.two_launches ? P.splits2 * P.per_slice : 0;
  A.hints = (uint32_t*)(ws + P.off_hints);
  A.partials = (Partial*)(ws + P.off_partials);
  RowResult* rowres = (RowResult*)(ws + P.off_rows);
  // the noise_spec 4 sweep touches the hint words only when rows are cut into slices
  if ((spec != 4 || P.splits > 1 || (P.two_launches && (P.splits1 > 1 || P.splits2 > 1))) &&
      cudaMemsetAsync(A.hints, 0, (size_t)P.rows * sizeof(uint32_t), st) != cudaSuccess)
    return GLS_ERR_CUDA;
  cudaError_t err;
  const bool r10 = A.rounds == 10;
  const bool bf = dtype == GLS_BF16;
  if (spec == 4) {
    const int sh = s4_shape(dtype, A.V, A.multi_k > 0);
    // Two sets of rows: one launch with both variants of the sweep while the input is small (the
    // launches are what a small step costs), otherwise one launch per set (the kernel
    // specialised for its set is faster where the sweep itself is what a step costs).
    const bool small_step = !P.two_launches;
#define SWEEP4(SH, R)                                                                       \
  do {                                                                                      \
    const long long cap = (long long)num_sms() * S4Cfg<SH>::kCtasPerSM;                       \
    const int grid = sweep_grid<SH>(P.n_items, cap);                                        \
    const size_t smem = sizeof(S4Shared<SH>);                                               \
    if (A.multi_k > 0)                                                                      \
      sweep4_kernel<SH, 1, R, true><<<grid, S4Cfg<SH>::kWarps * 32, smem, st>>>(A);         \
    else if (A.data2 != nullptr && small_step)                                              \
      sweep4_kernel<SH, 2, R><<<grid, S4Cfg<SH>::kWarps * 32, smem, st>>>(A);               \
    else if (A.data2 != nullptr) {                                                          \
      SweepArgs A1 = A, A2 = A;                                                             \
      A1.row_count = A.rows1;                                                               \
      A1.chunk = P.chunk1;                                                                  \
      A1.splits = P.splits1;                                                                \
      A1.n_items = (long long)A.rows1 * P.splits1;                                          \
      A2.row_begin = A.rows1;                                                               \
      A2.row_count = A.rows - A.rows1;                                                      \
      A2.chunk = P.chunk2;                                                                  \
      A2.splits = P.splits2;                                                                \
      A2.n_items = (long long)A2.row_count * P.splits2;                                     \
      const int g1 = sweep_grid<SH>(A1.n_items, cap);                                       \
      const int g2 = sweep_grid<SH>(A2.n_items, cap);                                       \
      sweep4_kernel<SH, 0, R><<<g1, S4Cfg<SH>::kWarps * 32, smem, st>>>(A1);                \
      sweep4_kernel<SH, 1, R><<<g2, S4Cfg<SH>::kWarps * 32, smem, st>>>(A2);                \
    }                                                                                       \
    else if (lse)                                                                           \
      sweep4_kernel<SH, 1, R><<<grid, S4Cfg<SH>::kWarps * 32, smem, st>>>(A);               \
    else                                                                                    \
      sweep4_kernel<SH, 0, R><<<grid, S4Cfg<SH>::kWarps * 32, smem, st>>>(A);               \
  } while (0)
    if (sh == kS4ShapeBf16) { if (r10) SWEEP4(kS4ShapeBf16, 10); else SWEEP4(kS4ShapeBf16, 0); }
    else if (sh == kS4ShapeF32Wide) { if (r10) SWEEP4(kS4ShapeF32Wide, 10); else SWEEP4(kS4ShapeF32Wide, 0); }
    else { if (r10) SWEEP4(kS4ShapeF32Narrow, 10); else SWEEP4(kS4ShapeF32Narrow, 0); }
#undef SWEEP4
    err = cudaGetLastError();
  } else {
    const long long want = (P.n_items + kSweepThreads / 32 - 1) / (kSweepThreads / 32);
    const int grid = (int)(want < (long long)num_sms() * 4 ? want : (long long)num_sms() * 4);
#define SWEEP_CALL(...) launch_sweep_t<__VA_ARGS__>(A, lse, grid, st)
    if (bf) err = r10 ? SWEEP_CALL(kBF16, 10) : SWEEP_CALL(kBF16, 0);
    else err = r10 ? SWEEP_CALL(kF32, 10) : SWEEP_CALL(kF32, 0);
#undef SWEEP_CALL
  }
  if (err != cudaSuccess) return GLS_ERR_CUDA;
  const bool fuse = va != nullptr && fused_verify_smem(va->K, va->L, va->J) <= kFusedVerifyMaxSmem;
  if (fused) *fused = fuse;
  if (step != nullptr) {  // two sets of rows (noise_spec 4 only): draft results, then Algorithm 2
    if (bf) err = r10 ? launch_step_t<kBF16, 4, 10>(A, *va, *step, st) : launch_step_t<kBF16, 4, 0>(A, *va, *step, st);
    else err = r10 ? launch_step_t<kF32, 4, 10>(A, *va, *step, st) : launch_step_t<kF32, 4, 0>(A, *va, *step, st);
    return err == cudaSuccess ? GLS_OK : GLS_ERR_CUDA;
  }
#define FIN_CALL(...)                                                                          \
  (fuse ? launch_fused_verify_t<__VA_ARGS__>(A, *va, st)                                       \
        : launch_finalize_t<__VA_ARGS__>(A, (int)P.rows, lse, rowres, out_tokens, out_scores, \
                                         status, st))
  if (bf) {
    if (spec == 1) err = r10 ? FIN_CALL(kBF16, 1, 10) : FIN_CALL(kBF16, 1, 0);
    else err = r10 ? FIN_CALL(kBF16, 4, 10) : FIN_CALL(kBF16, 4, 0);
  } else {
    if (spec == 1) err = r10 ? FIN_CALL(kF32, 1, 10) : FIN_CALL(kF32, 1, 0);
    else err = r10 ? FIN_CALL(kF32, 4, 10) : FIN_CALL(kF32, 4, 0);
  }
#undef FIN_CALL
  return err == cudaSuccess ? GLS_OK : GLS_ERR_CUDA;
}

// Algorithm 2 in phases: per phase a sweep over the listed rows and the kernel that walks the
// phase's positions.
template <int SH, int ROUNDS, bool MULTI>
static int run_verify_phased_t(SweepArgs& A, const VerifyArgs& va, const Plan& P, void* workspace,
                                 cudaStream_t st, int part) {
  constexpr int DT = S4Cfg<SH>::kDT;
  char* ws = (char*)workspace;
  A.chunk = 0;
  A.splits = 0;
  A.parts = P.parts;
  A.rows = (int)P.rows;
  A.hints = (uint32_t*)(ws + P.off_hints);
  A.partials = (Partial*)(ws + P.off_partials);
  PhasedState S;
  size_t off = P.off_rows;
  S.active = (unsigned long long*)(ws + off);
  off += align_up((size_t)va.B * sizeof(unsigned long long), 256);
  S.counts = (int*)(ws + off);
  off += align_up((size_t)kMaxPhases * sizeof(int), 256);
  S.lists = (int*)(ws + off);
  const long long BK = (long long)va.B * va.K;
  // phases: position 0, then everything else; very large inputs take positions 1 and 2 before
  // the rest (most survivors of position 0 are pruned there, and a phase's fixed cost is small
  // against the rows that a sequence of B survivors would read at the remaining positions)
  int ends[kMaxPhases];
  const int n_phases = phase_ends(va.B, va.J, A.V, DT == kBF16 ? 2 : 4, ends, va.three_phases);
  // part 0: the whole walk; 1: the first phase only (the state stays in the workspace); 2: the
  // phases after the first, from that state
  const int p_begin = part == 2 ? 1 : 0, p_end = part == 1 ? 1 : n_phases;
  if (p_begin == 0) {
    const long long n = BK * va.J;  // the largest index range the initialisation covers
    phased_init_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(va, S, ends[0], A.hints);
  }
  const long long cap = (long long)num_sms() * S4Cfg<SH>::kCtasPerSM;
  const int warps = kFusedVerifyMaxWarps;
  int j0 = p_begin > 0 ? ends[p_begin - 1] : 0;
  for (int p = p_begin; p < p_end; ++p) {
    const int j1 = ends[p], j2 = p + 1 < n_phases ? ends[p + 1] : j1;
    const long long most = BK * (j1 - j0) * P.splits;  // items if every row of the phase is listed
    const int grid = (int)(most < cap ? most : cap);
    {
      // a programmatic dependent of the kernel before it (the initialisation or the previous
      // phase's walk): it waits for that kernel before it reads the list
      cudaLaunchAttribute sattr;
      cudaLaunchConfig_t scfg = dependent_launch(&sattr, grid, S4Cfg<SH>::kWarps * 32, sizeof(S4Shared<SH>), st);
      const int* list = S.lists + BK * j0;
      const int* count = S.counts + p;
      if (cudaLaunchKernelEx(&scfg, sweep4_listed_kernel<SH, ROUNDS, MULTI>, A, list, count) != cudaSuccess)
        return GLS_ERR_CUDA;
    }
    const int nrows = va.K * (j1 - j0);
    cudaLaunchAttribute attr;
    cudaLaunchConfig_t cfg = dependent_launch(&attr, va.B, (nrows < warps ? nrows : warps) * 32,
                                              (size_t)nrows * sizeof(RowResult), st);
    if (cudaLaunchKernelEx(&cfg, phased_verify_kernel<DT, ROUNDS>, A, va, S, p, j0, j1, j2,
                           (int)S4Cfg<SH>::kCtaTokens, grid, (int)S4Cfg<SH>::kWarps) != cudaSuccess)
      return GLS_ERR_CUDA;
    j0 = j1;
  }
  return cudaGetLastError() == cudaSuccess ? GLS_OK : GLS_ERR_CUDA;
}
static int run_verify_phased(SweepArgs& A, int dtype, const VerifyArgs& va, const Plan& P,
                               void* workspace, cudaStream_t st, int part) {
  const int sh = s4_shape(dtype, A.V, va.multi_rows);
  const bool r10 = A.rounds == 10;
#define PHASED(SH, M) (r10 ? run_verify_phased_t<SH, 10, M>(A, va, P, workspace, st, part) \
                             : run_verify_phased_t<SH, 0, M>(A, va, P, workspace, st, part))
  if (va.multi_rows) return sh == kS4ShapeBf16 ? PHASED(kS4ShapeBf16, true) : PHASED(kS4ShapeF32Narrow, true);
  if (sh == kS4ShapeBf16) return PHASED(kS4ShapeBf16, false);
  if (sh == kS4ShapeF32Wide) return PHASED(kS4ShapeF32Wide, false);
  return PHASED(kS4ShapeF32Narrow, false);
#undef PHASED
}

constexpr uint32_t kWalkFlags = GLS_VERIFY_ALL_ROWS | GLS_VERIFY_ACTIVE_ROWS | GLS_VERIFY_FIRST_PHASE |
                                GLS_VERIFY_REST | GLS_VERIFY_THREE_PHASES;
// known bits only, and at most one request about the walk
static bool verify_flags_ok(uint32_t flags) {
  if (flags & ~(GLS_COMBINE_ALL | GLS_NO_BONUS | kWalkFlags)) return false;
  const uint32_t w = flags & kWalkFlags;
  return (w & (w - 1u)) == 0u;
}

// How gls_target_sample_verify walks Algorithm 2: 0 = every row is raced, then the loop; 1 = in
// phases (only the rows of active drafts are read): when the walk can prune anything and the rows
// are large enough for its extra launches to pay; -1 = GLS_VERIFY_ACTIVE_ROWS asked for and
// not possible.
static int verify_walk(int dtype, bool row_per_draft, int B, int K, int L, int64_t V, int spec,
                       uint32_t flags) {
  const int J = L + ((flags & GLS_NO_BONUS) ? 0 : 1);
  const bool multi = (flags & GLS_COMBINE_ALL) && row_per_draft && K > 1;
  if (multi && (spec != 4 || K > 8 || V >= (1LL << 28))) return -1;  // the call refuses these
  const bool can = spec == 4 && (multi || !(flags & GLS_COMBINE_ALL)) && L >= 1 && J >= 2 &&
                   (size_t)K * (J - 1) * sizeof(RowResult) <= kFusedVerifyMaxSmem;
  if (flags & (GLS_VERIFY_ACTIVE_ROWS | GLS_VERIFY_FIRST_PHASE | GLS_VERIFY_REST | GLS_VERIFY_THREE_PHASES))
    return can ? 1 : -1;
  if (!can || (flags & GLS_VERIFY_ALL_ROWS)) return 0;
  const double bytes = (double)B * K * J * (double)V * (dtype == GLS_BF16 ? 2.0 : 4.0);
  return bytes >= (multi ? 0.5 : 1.0) * GLS_PHASED_MIN_BYTES ? 1 : 0;
}

static bool sizes_ok(int B, int K, int J, int64_t V) {
  if (B <= 0 || K <= 0 || K > GLS_MAX_K || J <= 0 || V <= 0) return false;
  if (V >= (1LL << 31) - 4 * kS4MaxCtaTokens) return false;
  if ((long long)B * K * J >= (1LL << 31) / 64) return false;
  return true;
}

}  // namespace gls

using namespace gls;

extern "C" {

int gls_version(void) { return 200; }

int gls_debug_bounds(uint32_t out_host[4]) {
#ifdef GLS_DEBUG_BOUNDS
  if (!out_host) return 1;
  if (cudaMemcpyFromSymbol(out_host, g_bounds_fault, 4 * sizeof(uint32_t)) != cudaSuccess) return -1;
  return 1;
#else
  if (out_host) out_host[0] = out_host[1] = out_host[2] = out_host[3] = 0u;
  return 0;
#endif
}

const char* gls_status_string(int status) {
  switch (status) {
    case GLS_OK: return "GLS_OK";
    case GLS_ERR_INVALID_ARG: return "GLS_ERR_INVALID_ARG: null pointer, size or parameter out of range";
    case GLS_ERR_UNSUPPORTED: return "GLS_ERR_UNSUPPORTED: dtype or flag combination not implemented";
    case GLS_ERR_MISALIGNED: return "GLS_ERR_MISALIGNED: base pointer not aligned to its element size";
    case GLS_ERR_WORKSPACE: return "GLS_ERR_WORKSPACE: workspace missing or smaller than gls_workspace_bytes()";
    case GLS_ERR_CUDA: return "GLS_ERR_CUDA: a CUDA runtime call failed";
    case GLS_ERR_STATIC_LIMIT:
      return "GLS_ERR_STATIC_LIMIT: the problem needs more scratch than GLS_STATIC_SCRATCH_BYTES; "
             "use the entry point that takes a workspace";
    default: return "GLS: unknown status";
  }
}

// scratch of a call that races every row it is given: the largest need over the noise layouts and
// element types (the call may use any of them)
static size_t all_rows_workspace(int B, int K, int J, int64_t V) {
  size_t need = make_plan1((long long)B * K * J, V).total;
  for (int dt = 0; dt < 2; ++dt) {
    const size_t d = make_plan4((long long)B * K * J, V, dt, false).total;
    const size_t e = make_plan4((long long)B * J, V, dt, true).total;  // fused multi-stream encoder
    const size_t f = make_plan4((long long)B * K * J, V, dt, true).total;  // Appendix B, row per draft
    if (d > need) need = d;
    if (e > need) need = e;
    if (f > need) need = f;
  }
  return need;
}

size_t gls_workspace_bytes(int B, int K, int J, int64_t V) {
  if (!sizes_ok(B, K, J, V)) return 0;
  size_t need = all_rows_workspace(B, K, J, V);
  for (int dt = 0; dt < 2; ++dt) {
    for (int multi = 0; multi < 2; ++multi) {  // verification in phases
      const size_t g = make_plan_phased(B, K, J, V, dt, multi != 0).total;
      if (g > need) need = g;
    }
  }
  return need;
}

int gls_copy_rows_to_device(void* dst_device, size_t dst_pitch, const void* src_host, size_t src_pitch,
                            size_t row_bytes, size_t n_rows, void* stream) {
  if (!dst_device || !src_host || row_bytes == 0 || dst_pitch < row_bytes || src_pitch < row_bytes)
    return GLS_ERR_INVALID_ARG;
  if (n_rows == 0) return GLS_OK;
  return cudaMemcpy2DAsync(dst_device, dst_pitch, src_host, src_pitch, row_bytes, n_rows,
                           cudaMemcpyHostToDevice, (cudaStream_t)stream) == cudaSuccess
             ? GLS_OK
             : GLS_ERR_CUDA;
}

int gls_verify_walk(int dtype, int row_per_draft, int B, int K, int L, int64_t V, int noise_spec,
                    uint32_t flags) {
  if (!verify_flags_ok(flags)) return -1;
  const int J = L + ((flags & GLS_NO_BONUS) ? 0 : 1);
  if (L < 0 || !sizes_ok(B, K, J, V) || (dtype != GLS_F32 && dtype != GLS_BF16)) return -1;
  return verify_walk(dtype, row_per_draft != 0, B, K, L, V, noise_spec, flags);
}

int gls_verify_phases(int dtype, int row_per_draft, int B, int K, int L, int64_t V, int noise_spec,
                      uint32_t flags, int ends_host[4]) {
  const int walk = gls_verify_walk(dtype, row_per_draft, B, K, L, V, noise_spec, flags);
  if (walk <= 0 || !ends_host) return walk < 0 ? -1 : 0;
  const int J = L + ((flags & GLS_NO_BONUS) ? 0 : 1);
  return phase_ends(B, J, V, dtype == GLS_BF16 ? 2 : 4, ends_host, (flags & GLS_VERIFY_THREE_PHASES) != 0);
}

size_t gls_draft_verify_workspace_bytes(int B, int K, int L, int J, int64_t V) {
  if (L < 1 || J < L || J > L + 1 || !sizes_ok(B, K, L + J, V)) return 0;
  size_t need = gls_workspace_bytes(B, K, J, V);  // large inputs: a draft call, then a verify call
  for (int dt = 0; dt < 2; ++dt) {
    const size_t t = make_plan_step((long long)B * K * L, (long long)B * K * J, V, dt).total;
    if (t > need) need = t;
  }
  return need;
}

int gls_draft_sample(const gls_rows_t* draft_logits, int B, int K, int J, int64_t V, float inv_temp,
                     const float* inv_temp_per_draft_host, const gls_noise_t* noise,
                     int32_t* out_tokens, float* out_scores, void* workspace,
                     size_t workspace_bytes, uint32_t* device_status, void* stream) {
  if (!noise || !out_tokens || !sizes_ok(B, K, J, V)) return GLS_ERR_INVALID_ARG;
  int rc = check_rows(draft_logits);
  if (rc != GLS_OK) return rc;
  SweepArgs A;
  std::memset(&A, 0, sizeof(A));
  for (int k = 0; k < K; ++k) {
    const float it = inv_temp_per_draft_host ? inv_temp_per_draft_host[k] : inv_temp;
    if (!finite_pos(it)) return GLS_ERR_INVALID_ARG;
    A.inv_t[k] = it;
  }
  int spec;
  rc = fill_noise(A, noise, 0u, &spec);
  if (rc != GLS_OK) return rc;
  const Plan P = make_plan((long long)B * K * J, V, spec, draft_logits->dtype);
  if (!workspace || workspace_bytes < P.total) return GLS_ERR_WORKSPACE;
  A.data = draft_logits->data;
  A.sb = draft_logits->stride_b;
  A.sk = draft_logits->stride_k;
  A.sj = draft_logits->stride_j;
  A.K = K;
  A.J = J;
  A.V = (int)V;
  return run_rows(A, draft_logits->dtype, spec, P, workspace, false, out_tokens, out_scores,
                  device_status, (cudaStream_t)stream);
}

int gls_target_sample_verify(const gls_rows_t* target_logits, int B, int K, int L, int64_t V,
                             float inv_temp, const int32_t* draft_tokens, const gls_noise_t* noise,
                             uint32_t flags, int32_t* out_tokens, int32_t* out_num_tokens,
                             uint8_t* out_accept, float* out_scores, void* workspace,
                             size_t workspace_bytes, uint32_t* device_status, void* stream) {
  if (!verify_flags_ok(flags)) return GLS_ERR_INVALID_ARG;
  const int J = L + ((flags & GLS_NO_BONUS) ? 0 : 1);
  if (!noise || !out_tokens || !out_num_tokens || L < 0 || !sizes_ok(B, K, J, V))
    return GLS_ERR_INVALID_ARG;
  if (L > 0 && (!draft_tokens || !out_accept)) return GLS_ERR_INVALID_ARG;
  if (!finite_pos(inv_temp)) return GLS_ERR_INVALID_ARG;
  int rc = check_rows(target_logits);
  if (rc != GLS_OK) return rc;
  SweepArgs A;
  std::memset(&A, 0, sizeof(A));
  for (int k = 0; k < K; ++k) A.inv_t[k] = inv_temp;
  int spec;
  rc = fill_noise(A, noise, 0u, &spec);
  if (rc != GLS_OK) return rc;
  // Appendix B couples every stream to the accepted prefix's distribution.  When all k share one
  // target row per position (stride_k = 0) the rows' own winners already are that race.  With a
  // row per draft, every row is raced under all K streams at once (the fused multi-stream race)
  // and the epilogue reads the row of the lowest active draft.
  const bool multi = (flags & GLS_COMBINE_ALL) && target_logits->stride_k != 0 && K > 1;
  if (multi && (spec != 4 || K > 8 || V >= (1LL << 28))) return GLS_ERR_UNSUPPORTED;
  const int walk = verify_walk(target_logits->dtype, target_logits->stride_k != 0, B, K, L, V, spec, flags);
  if (walk < 0) return GLS_ERR_UNSUPPORTED;
  const bool in_phases = walk == 1;
  const int part = (flags & GLS_VERIFY_FIRST_PHASE) ? 1 : (flags & GLS_VERIFY_REST) ? 2 : 0;
  const bool three = (flags & GLS_VERIFY_THREE_PHASES) != 0;
  flags &= ~kWalkFlags;
  const Plan P = in_phases ? make_plan_phased(B, K, J, V, target_logits->dtype, multi)
                          : make_plan((long long)B * K * J, V, spec, target_logits->dtype, multi);
  if (!workspace || workspace_bytes < P.total) return GLS_ERR_WORKSPACE;
  if (multi) A.multi_k = K;
  A.data = target_logits->data;
  A.sb = target_logits->stride_b;
  A.sk = target_logits->stride_k;
  A.sj = target_logits->stride_j;
  A.K = K;
  A.J = J;
  A.V = (int)V;
  cudaStream_t st = (cudaStream_t)stream;
  VerifyArgs va;
  va.B = B; va.K = K; va.L = L; va.J = J;
  va.flags = flags;
  va.multi_rows = multi;
  va.three_phases = three;
  va.draft_tokens = draft_tokens;
  va.out_tokens = out_tokens;
  va.out_num = out_num_tokens;
  va.accept = out_accept;
  va.out_scores = out_scores;
  va.dev_status = device_status;
  if (in_phases) return run_verify_phased(A, target_logits->dtype, va, P, workspace, st, part);
  bool fused = false;
  rc = run_rows(A, target_logits->dtype, spec, P, workspace, true, nullptr, nullptr, nullptr, st,
                &va, &fused);
  if (rc != GLS_OK) return rc;
  if (fused) return GLS_OK;
  const RowResult* rowres = (const RowResult*)((char*)workspace + P.off_rows);
  verify_epilogue_kernel<<<(B + 127) / 128, 128, 0, st>>>(rowres, B, K, L, J, flags, multi, draft_tokens,
                                                         out_tokens, out_num_tokens, out_accept,
                                                         out_scores, device_status);
  return cudaGetLastError() == cudaSuccess ? GLS_OK : GLS_ERR_CUDA;
}

int gls_draft_verify(const gls_rows_t* draft_logits, const gls_rows_t* target_logits, int B, int K,
                     int L, int64_t V, float inv_temp_draft, const float* inv_temp_per_draft_host,
                     float inv_temp_target, const gls_noise_t* noise, uint32_t flags,
                     int32_t* out_draft_tokens, float* out_draft_scores, int32_t* out_tokens,
                     int32_t* out_num_tokens, uint8_t* out_accept, float* out_scores,
                     void* workspace, size_t workspace_bytes, uint32_t* device_status,
                     void* stream) {
  if (flags & ~(GLS_COMBINE_ALL | GLS_NO_BONUS)) return GLS_ERR_INVALID_ARG;
  const int J = L + ((flags & GLS_NO_BONUS) ? 0 : 1);
  if (!noise || !out_draft_tokens || !out_tokens || !out_num_tokens || !out_accept || L < 1 ||
      !sizes_ok(B, K, L + J, V))
    return GLS_ERR_INVALID_ARG;
  if (!finite_pos(inv_temp_target)) return GLS_ERR_INVALID_ARG;
  int rc = check_rows(draft_logits);
  if (rc != GLS_OK) return rc;
  rc = check_rows(target_logits);
  if (rc != GLS_OK) return rc;
  if (draft_logits->dtype != target_logits->dtype) return GLS_ERR_UNSUPPORTED;
  SweepArgs A;
  std::memset(&A, 0, sizeof(A));
  for (int k = 0; k < K; ++k) {
    const float it = inv_temp_per_draft_host ? inv_temp_per_draft_host[k] : inv_temp_draft;
    if (!finite_pos(it)) return GLS_ERR_INVALID_ARG;
    A.inv_t[k] = it;
  }
  int spec;
  rc = fill_noise(A, noise, 0u, &spec);
  if (rc != GLS_OK) return rc;
  // one launch sweeps both sets of rows under the default noise layout; Appendix B with a target
  // row per draft and sequences whose row results exceed the epilogue's shared memory take the
  // two separate calls
  if (spec != 4) return GLS_ERR_UNSUPPORTED;
  if (fused_verify_smem(K, L, J) > kFusedVerifyMaxSmem) return GLS_ERR_UNSUPPORTED;
  const long long rows_d = (long long)B * K * L, rows_t = (long long)B * K * J;
  // Large target rows: the draft rows first, then Algorithm 2 in phases, which reads the target
  // rows of active drafts only (the draft tokens it needs are this call's own output).  Appendix
  // B on a row per draft (every row under all K streams) takes the two calls at any size.
  const bool multi = (flags & GLS_COMBINE_ALL) && target_logits->stride_k != 0 && K > 1;
  const int walk = verify_walk(target_logits->dtype, target_logits->stride_k != 0, B, K, L, V, spec, flags);
  if (walk < 0) return GLS_ERR_UNSUPPORTED;
  if (walk == 1 || multi) {
    if (!workspace || workspace_bytes < gls_draft_verify_workspace_bytes(B, K, L, J, V)) return GLS_ERR_WORKSPACE;
    rc = gls_draft_sample(draft_logits, B, K, L, V, inv_temp_draft, inv_temp_per_draft_host, noise,
                          out_draft_tokens, out_draft_scores, workspace, workspace_bytes, device_status,
                          stream);
    if (rc != GLS_OK) return rc;
    return gls_target_sample_verify(target_logits, B, K, L, V, inv_temp_target, out_draft_tokens, noise,
                                    flags, out_tokens, out_num_tokens, out_accept, out_scores,
                                    workspace, workspace_bytes, device_status, stream);
  }
  const Plan P = make_plan_step(rows_d, rows_t, V, draft_logits->dtype);
  if (!workspace || workspace_bytes < P.total) return GLS_ERR_WORKSPACE;
  A.data = draft_logits->data;
  A.sb = draft_logits->stride_b;
  A.sk = draft_logits->stride_k;
  A.sj = draft_logits->stride_j;
  A.K = K;
  A.J = L;
  A.V = (int)V;
  A.data2 = target_logits->data;
  A.sb2 = target_logits->stride_b;
  A.sk2 = target_logits->stride_k;
  A.sj2 = target_logits->stride_j;
  A.J2 = J;
  A.rows1 = (int)rows_d;
  A.inv_t2 = inv_temp_target;
  VerifyArgs va;
  va.B = B; va.K = K; va.L = L; va.J = J;
  va.flags = flags;
  va.multi_rows = false;
  va.three_phases = false;
  va.draft_tokens = nullptr;  // taken from the draft rows of this very call
  va.out_tokens = out_tokens;
  va.out_num = out_num_tokens;
  va.accept = out_accept;
  va.out_scores = out_scores;
  va.dev_status = device_status;
  StepOut so;
  so.draft_tokens = out_draft_tokens;
  so.draft_scores = out_draft_scores;
  return run_rows(A, draft_logits->dtype, spec, P, workspace, true, nullptr, nullptr, nullptr,
                  (cudaStream_t)stream, &va, nullptr, &so);
}

static int check_sparse(const gls_sparse_rows_t* r) {
  if (!r || !r->token_ids || !r->logits || r->M <= 0) return GLS_ERR_INVALID_ARG;
  if (((uintptr_t)r->token_ids) % 4 || ((uintptr_t)r->logits) % 4) return GLS_ERR_MISALIGNED;
  return GLS_OK;
}

int gls_draft_sample_sparse(const gls_sparse_rows_t* draft_rows, int B, int K, int J, float inv_temp,
                            const float* inv_temp_per_draft_host, const gls_noise_t* noise,
                            int32_t* out_tokens, float* out_scores, uint32_t* device_status,
                            void* stream) {
  if (!noise || !out_tokens || !sizes_ok(B, K, J, 1)) return GLS_ERR_INVALID_ARG;
  int rc = check_sparse(draft_rows);
  if (rc != GLS_OK) return rc;
  SweepArgs A;
  std::memset(&A, 0, sizeof(A));
  for (int k = 0; k < K; ++k) {
    const float it = inv_temp_per_draft_host ? inv_temp_per_draft_host[k] : inv_temp;
    if (!finite_pos(it)) return GLS_ERR_INVALID_ARG;
    A.inv_t[k] = it;
  }
  int spec;
  rc = fill_noise(A, noise, 0u, &spec);
  if (rc != GLS_OK) return rc;
  A.K = K;
  A.J = J;
  SparseArgs S;
  S.ids = draft_rows->token_ids;
  S.logits = draft_rows->logits;
  S.sb = draft_rows->stride_b;
  S.sk = draft_rows->stride_k;
  S.sj = draft_rows->stride_j;
  S.M = draft_rows->M;
  const int rows = B * K * J;
  cudaStream_t st = (cudaStream_t)stream;
  const int wpb = 4;
  const int grid = (rows + wpb - 1) / wpb;
#define SPARSE_DRAFT(SPEC, R) \
  sparse_draft_kernel<SPEC, R><<<grid, wpb * 32, 0, st>>>(A, S, rows, out_tokens, out_scores, device_status)
  const bool r10 = A.rounds == 10;
  if (spec == 1) { if (r10) SPARSE_DRAFT(1, 10); else SPARSE_DRAFT(1, 0); }
  else { if (r10) SPARSE_DRAFT(4, 10); else SPARSE_DRAFT(4, 0); }
#undef SPARSE_DRAFT
  return cudaGetLastError() == cudaSuccess ? GLS_OK : GLS_ERR_CUDA;
}

int gls_target_sample_verify_sparse(const gls_sparse_rows_t* target_rows, int B, int K, int L,
                                    float inv_temp, const int32_t* draft_tokens,
                                    const gls_noise_t* noise, uint32_t flags, int32_t* out_tokens,
                                    int32_t* out_num_tokens, uint8_t* out_accept, float* out_scores,
                                    uint32_t* device_status, void* stream) {
  if (flags & ~(GLS_COMBINE_ALL | GLS_NO_BONUS)) return GLS_ERR_INVALID_ARG;
  const int J = L + ((flags & GLS_NO_BONUS) ? 0 : 1);
  if (!noise || !out_tokens || !out_num_tokens || L < 0 || !sizes_ok(B, K, J, 1))
    return GLS_ERR_INVALID_ARG;
  if (L > 0 && (!draft_tokens || !out_accept)) return GLS_ERR_INVALID_ARG;
  if (!finite_pos(inv_temp)) return GLS_ERR_INVALID_ARG;
  int rc = check_sparse(target_rows);
  if (rc != GLS_OK) return rc;
  // Appendix B with a list per draft: every list is raced under all K streams (see sparse_row)
  const bool multi = (flags & GLS_COMBINE_ALL) && target_rows->stride_k != 0 && K > 1;
  const size_t smem = fused_verify_smem(K, L, J);
  if (smem > kFusedVerifyMaxSmem) return GLS_ERR_UNSUPPORTED;
  SweepArgs A;
  std::memset(&A, 0, sizeof(A));
  for (int k = 0; k < K; ++k) A.inv_t[k] = inv_temp;
  int spec;
  rc = fill_noise(A, noise, 0u, &spec);
  if (rc != GLS_OK) return rc;
  A.K = K;
  A.J = J;
  if (multi) A.multi_k = K;
  SparseArgs S;
  S.ids = target_rows->token_ids;
  S.logits = target_rows->logits;
  S.sb = target_rows->stride_b;
  S.sk = target_rows->stride_k;
  S.sj = target_rows->stride_j;
  S.M = target_rows->M;
  VerifyArgs va;
  va.B = B; va.K = K; va.L = L; va.J = J;
  va.flags = flags;
  va.multi_rows = multi;
  va.three_phases = false;
  va.draft_tokens = draft_tokens;
  va.out_tokens = out_tokens;
  va.out_num = out_num_tokens;
  va.accept = out_accept;
  va.out_scores = out_scores;
  va.dev_status = device_status;
  cudaStream_t st = (cudaStream_t)stream;
  const int nrows = K * J;
  const int warps = nrows < kFusedVerifyMaxWarps ? nrows : kFusedVerifyMaxWarps;
#define SPARSE_VERIFY(SPEC, R) sparse_verify_kernel<SPEC, R><<<B, warps * 32, smem, st>>>(A, S, va)
  const bool r10 = A.rounds == 10;
  if (spec == 1) { if (r10) SPARSE_VERIFY(1, 10); else SPARSE_VERIFY(1, 0); }
  else { if (r10) SPARSE_VERIFY(4, 10); else SPARSE_VERIFY(4, 0); }
#undef SPARSE_VERIFY
  return cudaGetLastError() == cudaSuccess ? GLS_OK : GLS_ERR_CUDA;
}

int gls_compress_select(const gls_rows_t* enc_logw, const gls_rows_t* dec_logw, const uint8_t* bins,
                        int64_t bins_stride_b, int B, int K, int64_t N, const gls_noise_t* noise,
                        int32_t* out_enc_index, uint8_t* out_message, int32_t* out_dec_index,
                        uint8_t* out_match, float* out_scores, void* workspace,
                        size_t workspace_bytes, uint32_t* device_status, void* stream) {
  if (!noise || !out_enc_index || !out_message || !sizes_ok(B, K, 1, N))
    return GLS_ERR_INVALID_ARG;
  if (bins_stride_b != 0 && bins_stride_b < N) return GLS_ERR_INVALID_ARG;
  int rc = check_rows(enc_logw);
  if (rc != GLS_OK) return rc;
  if (dec_logw) {
    rc = check_rows(dec_logw);
    if (rc != GLS_OK) return rc;
    if (!out_dec_index || !out_match) return GLS_ERR_INVALID_ARG;
  }
  SweepArgs A;
  std::memset(&A, 0, sizeof(A));
  for (int k = 0; k < K; ++k) A.inv_t[k] = 1.0f;
  int spec;
  rc = fill_noise(A, noise, 1u, &spec);
  if (rc != GLS_OK) return rc;
  const Plan P = make_plan((long long)B * K, N, spec, enc_logw->dtype);
  if (!workspace || workspace_bytes < P.total) return GLS_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  const RowResult* rowres = (const RowResult*)((char*)workspace + P.off_rows);
  A.data = enc_logw->data;
  A.sb = enc_logw->stride_b;
  A.sk = 0;
  A.sj = 0;
  A.J = 1;
  A.V = (int)N;
  // The encoder index is one race over tokens and streams, Y = argmin_{i,k} S_i^(k) / lambda_q,i.
  // With the default noise layout, up to 8 streams and N < 2^28 it runs fused: each row is read
  // and summed once and the K streams share one bound; otherwise every stream sweeps the row on
  // its own and the epilogue takes the best of the K winners.
  const bool fused_enc = spec == 4 && K <= 8 && N < (1LL << 28);
  if (fused_enc) {
    const Plan PE = make_plan((long long)B, N, spec, enc_logw->dtype, true);
    if (workspace_bytes < PE.total) return GLS_ERR_WORKSPACE;
    A.K = 1;
    A.multi_k = K;
    rc = run_rows(A, enc_logw->dtype, spec, PE, workspace, true, nullptr, nullptr, nullptr, st);
    A.multi_k = 0;
    if (rc != GLS_OK) return rc;
    const RowResult* rr = (const RowResult*)((char*)workspace + PE.off_rows);
    encoder_epilogue_kernel<<<(B + 127) / 128, 128, 0, st>>>(rr, B, 1, bins, bins_stride_b,
                                                            out_enc_index, out_message, out_scores,
                                                            device_status, 1 + K);
  } else {
    // the one row of sample b raced under each of the K streams (stride_k = 0)
    A.K = K;
    rc = run_rows(A, enc_logw->dtype, spec, P, workspace, true, nullptr, nullptr, nullptr, st);
    if (rc != GLS_OK) return rc;
    encoder_epilogue_kernel<<<(B + 127) / 128, 128, 0, st>>>(rowres, B, K, bins, bins_stride_b,
                                                            out_enc_index, out_message, out_scores,
                                                            device_status, 1 + K);
  }
  if (cudaGetLastError() != cudaSuccess) return GLS_ERR_CUDA;
  if (!dec_logw) return GLS_OK;
  A.K = K;
  // decoders: row (b,k) under stream k, restricted to candidates labelled M
  A.data = dec_logw->data;
  A.sb = dec_logw->stride_b;
  A.sk = dec_logw->stride_k;
  A.bins = bins;
  A.bins_sb = bins_stride_b;
  A.msg = out_message;
  const Plan PD = make_plan((long long)B * K, N, spec, dec_logw->dtype);
  if (workspace_bytes < PD.total) return GLS_ERR_WORKSPACE;
  rc = run_rows(A, dec_logw->dtype, spec, PD, workspace, false, nullptr, nullptr, device_status, st);
  if (rc != GLS_OK) return rc;
  const RowResult* rowres_d = (const RowResult*)((char*)workspace + PD.off_rows);
  decoder_epilogue_kernel<<<(B + 127) / 128, 128, 0, st>>>(rowres_d, B, K, out_enc_index,
                                                          out_dec_index, out_match, out_scores);
  return cudaGetLastError() == cudaSuccess ? GLS_OK : GLS_ERR_CUDA;
}

}  // extern "C"

// ------------------------------------------------------------------------------------------
// Compression from the source (Appendix C with the Gaussian model of Appendix D.3).
// ------------------------------------------------------------------------------------------
namespace gls {

// W_k = u_{X^(k)}, the MMSE reconstruction g(w, t) = (s2_zeta w + s2_eta t) / (s2_eta + s2_zeta +
// s2_eta s2_zeta) per dimension, and its mean squared error against the source; a thread per (b, k).
__global__ void gauss_recon_kernel(const float* __restrict__ u, const float* __restrict__ a,
                                   const float* __restrict__ t, const int32_t* __restrict__ dec_index,
                                   int BK, int K, int D, double s2_eta, double s2_zeta,
                                   float* __restrict__ recon, float* __restrict__ sqerr) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= BK) return;
  const int b = r / K;
  const int x = dec_index[r];
  const double den = s2_eta + s2_zeta + s2_eta * s2_zeta;
  double se = 0.0;
  for (int d = 0; d < D; ++d) {
    float g = CUDART_NAN_F;
    if (x >= 0) {
      const double w = (double)u[(long long)x * D + d];
      const double gd = (s2_zeta * w + s2_eta * (double)t[(long long)r * D + d]) / den;
      const double e = gd - (double)a[(long long)b * D + d];
      se += e * e;
      g = (float)gd;
    }
    if (recon) recon[(long long)r * D + d] = g;
  }
  if (sqerr) sqerr[r] = x >= 0 ? (float)(se / D) : CUDART_NAN_F;
}

struct GaussPlan {
  int tiles, n_ranges, rows_per_range_enc, rows_per_range_dec;
  size_t off_hints, off_partials, off_rows, total;
};
static GaussPlan make_gauss_plan(int B, int K, long long N) {
  GaussPlan p;
  p.tiles = (int)((N + kGTile - 1) / kGTile);
  // enough CTAs for several waves over the machine, each with whole blocks of rows
  long long want = (4LL * num_sms() + p.tiles - 1) / p.tiles;
  if (want < 1) want = 1;
  auto per_range = [&](long long rows) {
    long long n = want;
    const long long blocks = (rows + kGRows - 1) / kGRows;
    if (n > blocks) n = blocks;
    return (int)(((blocks + n - 1) / n) * kGRows);
  };
  p.rows_per_range_enc = per_range(B);
  p.rows_per_range_dec = per_range((long long)B * K);
  p.n_ranges = 0;  // set per pass by the caller
  const size_t rows = (size_t)B * K;
  p.off_hints = 0;
  p.off_partials = align_up(rows * sizeof(uint32_t), 256);
  p.off_rows = p.off_partials + align_up(rows * p.tiles * sizeof(Partial), 256);
  p.total = p.off_rows + align_up(rows * sizeof(RowResult), 256);
  return p;
}

}  // namespace gls

extern "C" {

size_t gls_compress_gaussian_workspace_bytes(int B, int K, int64_t N) {
  if (B <= 0 || K <= 0 || K > gls::kGMaxK || N <= 0 || N >= (1LL << 28)) return 0;
  return gls::make_gauss_plan(B, K, N).total;
}

int gls_compress_gaussian(const float* candidates, const float* source, const float* side_info,
                          const uint8_t* bins, int64_t bins_stride_b, int B, int K, int64_t N, int D,
                          double s2_eta, double s2_zeta, double s2_prior, const gls_noise_t* noise,
                          int32_t* out_enc_index, uint8_t* out_message, int32_t* out_dec_index,
                          uint8_t* out_match, float* out_scores, float* out_recon, float* out_sqerr,
                          void* workspace, size_t workspace_bytes, uint32_t* device_status,
                          void* stream) {
  if (!candidates || !source || !side_info || !noise || !out_enc_index || !out_message ||
      !out_dec_index || !out_match || B <= 0 || K <= 0 || N <= 0 || D <= 0)
    return GLS_ERR_INVALID_ARG;
  if (!(s2_eta > 0.0) || !(s2_zeta > 0.0) || !(s2_prior > 0.0) || !std::isfinite(s2_eta) ||
      !std::isfinite(s2_zeta) || !std::isfinite(s2_prior))
    return GLS_ERR_INVALID_ARG;
  if (bins_stride_b != 0 && bins_stride_b < N) return GLS_ERR_INVALID_ARG;
  if (K > kGMaxK || D > kGMaxD || N >= (1LL << 28) || (long long)B * K >= (1LL << 24))
    return GLS_ERR_UNSUPPORTED;
  if (((uintptr_t)candidates | (uintptr_t)source | (uintptr_t)side_info) % 4) return GLS_ERR_MISALIGNED;
  SweepArgs A;
  std::memset(&A, 0, sizeof(A));
  for (int k = 0; k < K; ++k) A.inv_t[k] = 1.0f;
  int spec;
  int rc = fill_noise(A, noise, 1u, &spec);
  if (rc != GLS_OK) return rc;
  if (spec != 4) return GLS_ERR_UNSUPPORTED;
  GaussPlan P = make_gauss_plan(B, K, N);
  if (!workspace || workspace_bytes < P.total) return GLS_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  char* ws = (char*)workspace;
  A.gu = candidates;
  A.ga = source;
  A.gt = side_info;
  A.gD = D;
  A.g_s2_eta = s2_eta;
  A.g_s2_zeta = s2_zeta;
  A.g_s2_prior = s2_prior;
  A.V = (int)N;
  A.J = 1;
  A.splits = 1;
  A.parts = P.tiles;
  A.hints = (uint32_t*)(ws + P.off_hints);
  A.partials = (Partial*)(ws + P.off_partials);
  RowResult* rowres = (RowResult*)(ws + P.off_rows);
  const bool r10 = A.rounds == 10;
  const double var_dec = (1.0 + s2_eta) - 1.0 / (1.0 + s2_zeta);
  // as many quads of warps per CTA as the shared memory allows (more warps per scheduler)
  constexpr size_t kSmemMax = 227 * 1024;
#define GAUSS_SWEEP(ENC, rows_, per_range_, scale_)                                              \
  do {                                                                                           \
    const int n_ranges = ((rows_) + (per_range_) - 1) / (per_range_);                            \
    const int streams = (ENC) ? K : 1;                                                           \
    int quads = kGMaxQuads;                                                                      \
    while (quads > 1 && gauss_smem_bytes(D, streams, quads) > kSmemMax) --quads;                 \
    const size_t smem = gauss_smem_bytes(D, streams, quads);                                     \
    if (smem > kSmemMax) return GLS_ERR_UNSUPPORTED;                                             \
    if (cudaMemsetAsync(A.hints, 0, (size_t)(rows_) * sizeof(uint32_t), st) != cudaSuccess ||    \
        cudaMemsetAsync(A.partials, 0xff, (size_t)(rows_) * P.tiles * sizeof(Partial), st) !=    \
            cudaSuccess)                                                                         \
      return GLS_ERR_CUDA;                                                                       \
    if (r10) {                                                                                   \
      cudaFuncSetAttribute(gauss_sweep_kernel<10, ENC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
      gauss_sweep_kernel<10, ENC><<<P.tiles * n_ranges, quads * kGWarps * 32, smem, st>>>(       \
          A, n_ranges, (per_range_), (long long)N, (float)(scale_));                             \
    } else {                                                                                     \
      cudaFuncSetAttribute(gauss_sweep_kernel<0, ENC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
      gauss_sweep_kernel<0, ENC><<<P.tiles * n_ranges, quads * kGWarps * 32, smem, st>>>(        \
          A, n_ranges, (per_range_), (long long)N, (float)(scale_));                             \
    }                                                                                            \
    if (cudaGetLastError() != cudaSuccess) return GLS_ERR_CUDA;                                  \
  } while (0)
  // encoder: one race per source sample over candidates and the K streams, with the log-sum-exp
  A.K = 1;
  A.multi_k = K;
  A.rows = B;
  A.g_dec = 0;
  GAUSS_SWEEP(true, B, P.rows_per_range_enc, 1.0 / std::sqrt(2.0 * s2_eta));
  cudaError_t err = r10 ? launch_finalize_t<kF32, 4, 10>(A, B, true, rowres, nullptr, nullptr, nullptr, st)
                        : launch_finalize_t<kF32, 4, 0>(A, B, true, rowres, nullptr, nullptr, nullptr, st);
  if (err != cudaSuccess) return GLS_ERR_CUDA;
  encoder_epilogue_kernel<<<(B + 127) / 128, 128, 0, st>>>(rowres, B, 1, bins, bins_stride_b,
                                                          out_enc_index, out_message, out_scores,
                                                          device_status, 1 + K);
  if (cudaGetLastError() != cudaSuccess) return GLS_ERR_CUDA;
  // decoders: row (b, k) under stream k, restricted to the candidates labelled M
  A.K = K;
  A.multi_k = 0;
  A.rows = B * K;
  A.g_dec = 1;
  A.bins = bins;
  A.bins_sb = bins_stride_b;
  A.msg = out_message;
  if (D == kMD && GLS_GAUSS_MMA) {
    // sixteen coordinates: the rows' dot products with the candidates on the tensor cores
    const int rows = B * K;
    long long want = (4LL * num_sms() + P.tiles - 1) / P.tiles;  // CTAs for several waves
    const long long blocks = (rows + kMRows - 1) / kMRows;
    if (want > blocks) want = blocks;
    if (want < 1) want = 1;
    const int per_range = (int)(((blocks + want - 1) / want) * kMRows);
    const int n_ranges = (rows + per_range - 1) / per_range;
    const size_t smem = gauss_mma_smem_bytes();
    if (cudaMemsetAsync(A.hints, 0, (size_t)rows * sizeof(uint32_t), st) != cudaSuccess ||
        cudaMemsetAsync(A.partials, 0xff, (size_t)rows * P.tiles * sizeof(Partial), st) != cudaSuccess)
      return GLS_ERR_CUDA;
    const float scale_dec = (float)(1.0 / std::sqrt(2.0 * var_dec));
    const bool lab = bins != nullptr && bins_stride_b == 0;
#define GAUSS_MMA(R, LAB)                                                                                  \
  do {                                                                                                     \
    cudaFuncSetAttribute(gauss_dec_mma_kernel<R, LAB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem); \
    gauss_dec_mma_kernel<R, LAB><<<P.tiles * n_ranges, kMWarps * 32, smem, st>>>(A, n_ranges, per_range,     \
                                                                                (long long)N, scale_dec);  \
  } while (0)
    if (r10) { if (lab) GAUSS_MMA(10, true); else GAUSS_MMA(10, false); }
    else { if (lab) GAUSS_MMA(0, true); else GAUSS_MMA(0, false); }
#undef GAUSS_MMA
    if (cudaGetLastError() != cudaSuccess) return GLS_ERR_CUDA;
  } else {
    GAUSS_SWEEP(false, B * K, P.rows_per_range_dec, 1.0 / std::sqrt(2.0 * var_dec));
  }
#undef GAUSS_SWEEP
  err = r10 ? launch_finalize_t<kF32, 4, 10>(A, B * K, false, rowres, nullptr, nullptr, device_status, st)
            : launch_finalize_t<kF32, 4, 0>(A, B * K, false, rowres, nullptr, nullptr, device_status, st);
  if (err != cudaSuccess) return GLS_ERR_CUDA;
  decoder_epilogue_kernel<<<(B + 127) / 128, 128, 0, st>>>(rowres, B, K, out_enc_index, out_dec_index,
                                                          out_match, out_scores);
  if (cudaGetLastError() != cudaSuccess) return GLS_ERR_CUDA;
  if (out_recon || out_sqerr) {
    gauss_recon_kernel<<<(B * K + 127) / 128, 128, 0, st>>>(candidates, source, side_info, out_dec_index,
                                                           B * K, K, D, s2_eta, s2_zeta, out_recon,
                                                           out_sqerr);
    if (cudaGetLastError() != cudaSuccess) return GLS_ERR_CUDA;
  }
  return GLS_OK;
}

}  // extern "C"

// ------------------------------------------------------------------------------------------
// Allocation-free draft sampling: scratch compiled into the library image.
// ------------------------------------------------------------------------------------------
namespace gls {

// Scratch of gls_draft_sample_static.  In host code this name is only a handle for
// cudaGetSymbolAddress; the kernels get the device address that call returns.
static __device__ __align__(256) unsigned char g_static_scratch[GLS_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
static std::mutex g_static_mutex;
static void* g_static_ptr[kMaxDevices] = {};

// Device address of the scratch on the current device, looked up once per device.
static int static_scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return GLS_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return GLS_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_mutex);
  if (g_static_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) {
      (void)cudaGetLastError();
      return GLS_ERR_CUDA;
    }
    g_static_ptr[dev] = p;
  }
  *out = g_static_ptr[dev];
  return GLS_OK;
}

}  // namespace gls

extern "C" {

size_t gls_static_scratch_bytes(void) { return (size_t)GLS_STATIC_SCRATCH_BYTES; }

// ------------------------------------------------------------------------------------------
// Dense rows truncated to their M largest logits, then the sparse-row races.
// ------------------------------------------------------------------------------------------
size_t gls_topm_workspace_bytes(int B, int K, int J, int M) {
  if (B <= 0 || K <= 0 || J <= 0 || M <= 0 || M > gls::kTopmMaxM) return 0;
  // the lists, then the state of a verification in phases (active sets, row lists, their lengths)
  return gls::align_up((size_t)B * K * J * M * sizeof(int32_t), 256) +
         gls::align_up((size_t)B * K * J * M * sizeof(float), 256) +
         gls::align_up((size_t)B * sizeof(unsigned long long), 256) +
         gls::align_up((size_t)gls::kMaxPhases * sizeof(int), 256) +
         gls::align_up((size_t)B * K * J * sizeof(int), 256);
}

}  // extern "C"

namespace gls {
// selects into the workspace and describes the result as sparse rows
// list / count: NULL, or the rows to select (device memory), at most max_listed of them
static int topm_select(const gls_rows_t* rows, int B, int K, int J, int64_t V, int M, void* workspace,
                       size_t workspace_bytes, cudaStream_t st, gls_sparse_rows_t* out,
                       const int* list = nullptr, const int* count = nullptr,
                       long long max_listed = 0) {
  if (M <= 0 || M > kTopmMaxM || !sizes_ok(B, K, J, V)) return GLS_ERR_INVALID_ARG;
  const int rc = check_rows(rows);
  if (rc != GLS_OK) return rc;
  const size_t need = gls_topm_workspace_bytes(B, K, J, M);
  if (!workspace || workspace_bytes < need) return GLS_ERR_WORKSPACE;
  TopmArgs T;
  T.data = rows->data;
  T.sb = rows->stride_b;
  T.sk = rows->stride_k;
  T.sj = rows->stride_j;
  T.K = K;
  T.J = J;
  T.V = (int)V;
  T.M = M;
  T.rows = (long long)B * K * J;
  T.ids = (int32_t*)workspace;
  T.logits = (float*)((char*)workspace + align_up((size_t)T.rows * M * sizeof(int32_t), 256));
  T.list = list;
  T.count = count;
  const long long want = ((list ? max_listed : T.rows) + kTopmWarps - 1) / kTopmWarps;
  const long long cap = (long long)num_sms() * kTopmCtasPerSM;
  const int grid = (int)(want < cap ? want : cap);
  if (rows->dtype == GLS_BF16)
    topm_select_kernel<kBF16><<<grid, kTopmWarps * 32, 0, st>>>(T);
  else
    topm_select_kernel<kF32><<<grid, kTopmWarps * 32, 0, st>>>(T);
  if (cudaGetLastError() != cudaSuccess) return GLS_ERR_CUDA;
  out->token_ids = T.ids;
  out->logits = T.logits;
  out->stride_b = (int64_t)K * J * M;
  out->stride_k = (int64_t)J * M;
  out->stride_j = M;
  out->M = M;
  return GLS_OK;
}

// The top-M verify call in phases: select + race position 0 of every draft, walk it, then select
// + race the remaining positions of the surviving drafts and finish the walk.
static int topm_verify_phased(const gls_rows_t* rows, int B, int K, int L, int J, int64_t V, int M,
                              float inv_temp, const int32_t* draft_tokens, const gls_noise_t* noise,
                              uint32_t flags, int32_t* out_tokens, int32_t* out_num_tokens,
                              uint8_t* out_accept, float* out_scores, void* workspace,
                              size_t workspace_bytes, uint32_t* device_status, cudaStream_t st) {
  if (!out_tokens || !out_num_tokens || !draft_tokens || !out_accept) return GLS_ERR_INVALID_ARG;
  if (!finite_pos(inv_temp)) return GLS_ERR_INVALID_ARG;
  if (M <= 0 || M > kTopmMaxM) return GLS_ERR_INVALID_ARG;
  if (!workspace || workspace_bytes < gls_topm_workspace_bytes(B, K, J, M)) return GLS_ERR_WORKSPACE;
  const bool multi = (flags & GLS_COMBINE_ALL) && K > 1;
  SweepArgs A;
  std::memset(&A, 0, sizeof(A));
  for (int k = 0; k < K; ++k) A.inv_t[k] = inv_temp;
  int spec;
  int rc = fill_noise(A, noise, 0u, &spec);
  if (rc != GLS_OK) return rc;
  A.K = K;
  A.J = J;
  if (multi) A.multi_k = K;
  VerifyArgs va;
  va.B = B; va.K = K; va.L = L; va.J = J;
  va.flags = flags & (GLS_COMBINE_ALL | GLS_NO_BONUS);
  va.multi_rows = multi;
  va.three_phases = (flags & GLS_VERIFY_THREE_PHASES) != 0;
  va.draft_tokens = draft_tokens;
  va.out_tokens = out_tokens;
  va.out_num = out_num_tokens;
  va.accept = out_accept;
  va.out_scores = out_scores;
  va.dev_status = device_status;
  const long long BK = (long long)B * K;
  char* ws = (char*)workspace;
  size_t off = align_up((size_t)BK * J * M * sizeof(int32_t), 256) + align_up((size_t)BK * J * M * sizeof(float), 256);
  PhasedState S;
  S.active = (unsigned long long*)(ws + off);
  off += align_up((size_t)B * sizeof(unsigned long long), 256);
  S.counts = (int*)(ws + off);
  off += align_up((size_t)kMaxPhases * sizeof(int), 256);
  S.lists = (int*)(ws + off);
  int ends[kMaxPhases];
  const int n_phases = phase_ends(B, J, V, rows->dtype == GLS_BF16 ? 2 : 4, ends, va.three_phases);
  phased_init_kernel<<<(unsigned)((BK * J + 255) / 256), 256, 0, st>>>(va, S, ends[0], nullptr);
  int j0 = 0;
  for (int p = 0; p < n_phases; ++p) {
    const int j1 = ends[p], j2 = p + 1 < n_phases ? ends[p + 1] : j1;
    gls_sparse_rows_t sp;
    rc = topm_select(rows, B, K, J, V, M, workspace, workspace_bytes, st, &sp, S.lists + BK * j0,
                     S.counts + p, BK * (j1 - j0));
    if (rc != GLS_OK) return rc;
    SparseArgs Sp;
    Sp.ids = sp.token_ids;
    Sp.logits = sp.logits;
    Sp.sb = sp.stride_b;
    Sp.sk = sp.stride_k;
    Sp.sj = sp.stride_j;
    Sp.M = sp.M;
    const int nrows = K * (j1 - j0);
    const int warps = nrows < kFusedVerifyMaxWarps ? nrows : kFusedVerifyMaxWarps;
    const size_t smem = (size_t)nrows * sizeof(RowResult);
    const bool r10 = A.rounds == 10;
#define SPARSE_PHASED(SPEC, R) \
  sparse_phased_kernel<SPEC, R><<<B, warps * 32, smem, st>>>(A, Sp, va, S, p, j0, j1, j2)
    if (spec == 1) { if (r10) SPARSE_PHASED(1, 10); else SPARSE_PHASED(1, 0); }
    else { if (r10) SPARSE_PHASED(4, 10); else SPARSE_PHASED(4, 0); }
#undef SPARSE_PHASED
    j0 = j1;
  }
  return cudaGetLastError() == cudaSuccess ? GLS_OK : GLS_ERR_CUDA;
}
}  // namespace gls

extern "C" {

int gls_draft_sample_topm(const gls_rows_t* draft_logits, int B, int K, int J, int64_t V, int M,
                          float inv_temp, const float* inv_temp_per_draft_host,
                          const gls_noise_t* noise, int32_t* out_tokens, float* out_scores,
                          void* workspace, size_t workspace_bytes, uint32_t* device_status,
                          void* stream) {
  if (!noise || !out_tokens) return GLS_ERR_INVALID_ARG;
  gls_sparse_rows_t sp;
  const int rc = gls::topm_select(draft_logits, B, K, J, V, M, workspace, workspace_bytes,
                                  (cudaStream_t)stream, &sp);
  if (rc != GLS_OK) return rc;
  return gls_draft_sample_sparse(&sp, B, K, J, inv_temp, inv_temp_per_draft_host, noise, out_tokens,
                                 out_scores, device_status, stream);
}

int gls_target_sample_verify_topm(const gls_rows_t* target_logits, int B, int K, int L, int64_t V,
                                  int M, float inv_temp, const int32_t* draft_tokens,
                                  const gls_noise_t* noise, uint32_t flags, int32_t* out_tokens,
                                  int32_t* out_num_tokens, uint8_t* out_accept, float* out_scores,
                                  void* workspace, size_t workspace_bytes, uint32_t* device_status,
                                  void* stream) {
  if (!gls::verify_flags_ok(flags) || (flags & (GLS_VERIFY_FIRST_PHASE | GLS_VERIFY_REST)))
    return GLS_ERR_INVALID_ARG;
  const uint32_t walk_flags = flags & (GLS_VERIFY_ALL_ROWS | GLS_VERIFY_ACTIVE_ROWS | GLS_VERIFY_THREE_PHASES);
  flags &= ~walk_flags;
  const int J = L + ((flags & GLS_NO_BONUS) ? 0 : 1);
  if (!noise || !out_tokens || !out_num_tokens || L < 0) return GLS_ERR_INVALID_ARG;
  if ((long long)K * J > 1536) return GLS_ERR_UNSUPPORTED;
  gls_sparse_rows_t sp;
  // rows shared by all drafts (stride_k == 0) are truncated once and stay shared
  const int ksel = (target_logits && target_logits->stride_k == 0) ? 1 : K;
  // Large inputs with a row per draft: Algorithm 2 in phases, so that only the rows it reads are
  // truncated (the selection is what the call costs).  Same rule as the dense verify call.
  int walk = 0;
  if (target_logits && noise && ksel == K && gls::sizes_ok(B, K, J, V) &&
      (target_logits->dtype == GLS_F32 || target_logits->dtype == GLS_BF16))
    walk = gls::verify_walk(target_logits->dtype, true, B, K, L, V, 4, flags | walk_flags);
  if ((walk_flags & (GLS_VERIFY_ACTIVE_ROWS | GLS_VERIFY_THREE_PHASES)) && walk != 1) return GLS_ERR_UNSUPPORTED;
  if (walk == 1)
    return gls::topm_verify_phased(target_logits, B, K, L, J, V, M, inv_temp, draft_tokens, noise,
                                   flags | (walk_flags & GLS_VERIFY_THREE_PHASES),
                                   out_tokens, out_num_tokens, out_accept, out_scores, workspace,
                                   workspace_bytes, device_status, (cudaStream_t)stream);
  const int rc = gls::topm_select(target_logits, B, ksel, J, V, M, workspace, workspace_bytes,
                                  (cudaStream_t)stream, &sp);
  if (rc != GLS_OK) return rc;
  if (ksel == 1) sp.stride_k = 0;
  return gls_target_sample_verify_sparse(&sp, B, K, L, inv_temp, draft_tokens, noise, flags,
                                         out_tokens, out_num_tokens, out_accept, out_scores,
                                         device_status, stream);
}


int gls_draft_sample_static(const gls_rows_t* draft_logits, int B, int K, int J, int64_t V,
                            float inv_temp, const float* inv_temp_per_draft_host,
                            const gls_noise_t* noise, int32_t* out_tokens, float* out_scores,
                            uint32_t* device_status, void* stream) {
  if (!gls::sizes_ok(B, K, J, V)) return GLS_ERR_INVALID_ARG;
  const size_t need = all_rows_workspace(B, K, J, V);  // what gls_draft_sample may use
  if (need == 0) return GLS_ERR_INVALID_ARG;
  if (need > (size_t)GLS_STATIC_SCRATCH_BYTES) return GLS_ERR_STATIC_LIMIT;
  void* scratch = nullptr;
  const int rc = gls::static_scratch_address(&scratch);
  if (rc != GLS_OK) return rc;
  // Same path as the workspace-taking entry point; it clears the bound hints on `stream` before
  // the sweep reads them, which is the only part of the scratch that must start at zero.
  return gls_draft_sample(draft_logits, B, K, J, V, inv_temp, inv_temp_per_draft_host, noise,
                          out_tokens, out_scores, scratch, (size_t)GLS_STATIC_SCRATCH_BYTES,
                          device_status, stream);
}

}  // extern "C"
