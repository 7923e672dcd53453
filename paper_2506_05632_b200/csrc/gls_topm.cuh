// gls_topm.cuh -- top-M truncation of dense rows in one pass (Sec. 4.4 / Appendix D.1 of arXiv
// 2506.05632: the experiments sample from the M = 50 most likely tokens).
//
// A warp owns a row.  It streams the row once (the same 2048-token steps as the noise_spec 4
// sweep: four 32-byte loads per lane, the next step's loads in flight) and keeps, in shared memory,
// the tokens whose logit exceeds a threshold thr.  thr is -inf until the buffer first overflows;
// from then on it is the M-th largest logit seen so far, so a later token can only enter the top M
// if its logit is strictly larger (ties go to the lower index, and the row is read in index
// order).  The sweep itself only compares each group's maximum with thr and queues the groups
// that exceed it; queued groups are examined 32 at a time (one per lane, their logits read again
// from L2), their tokens above thr appended to the buffer, and whenever the buffer holds more
// than M + 64 entries the warp prunes it to the M largest (an 8-bit radix select on the
// order-preserving integer code of the logits, then a stable compaction) and raises thr.  A
// token passes with probability about M / (tokens seen), so a row of 150k tokens appends a few
// hundred tokens and is pruned about ten times.  Output: per row M (token id, logit) pairs in index order, id = -1 past the number of
// finite logits.  NaN, +inf and -inf logits are never kept.
#pragma once
#include "gls_sweep4.cuh"

namespace gls {

constexpr int kTopmCap = 1024;   // buffer entries per warp: at most M + 64 kept + 512 from one batch
constexpr int kTopmMaxM = 256;
constexpr int kTopmWarps = 4;    // rows per CTA
constexpr int kTopmCtasPerSM = 4;

struct TopmArgs {
  const void* data;       // rows [B][K][J][V]
  long long sb, sk, sj;   // element strides
  int K, J, V, M;
  long long rows;
  int32_t* ids;           // [rows][M]
  float* logits;          // [rows][M]
  // NULL, or the rows to truncate: row numbers (b * K + k) * J + j in device memory and their
  // count (the verification in phases truncates only the rows it will read)
  const int* list;
  const int* count;
};

struct TopmWarpBuf {
  uint32_t key[kTopmCap];  // order-preserving code of the logit
  int idx[kTopmCap];
  uint32_t hist[256];
};

// Keeps the M largest of the n buffered entries (ties: first come, i.e. lowest index), in their
// order of arrival; returns the new count and the code of the M-th largest.  Requires n > M.
// last_pass: 0 for fp32 logits; 2 for bf16 logits, whose codes differ in their upper 16 bits only
// (the lower 16 are all zero or all one with the sign), so two of the four radix passes suffice.
__device__ __noinline__ unsigned long long topm_prune(TopmWarpBuf* wb, int n, int M, int last_pass) {
  const int lane = threadIdx.x & 31;
  const uint32_t lt = (1u << lane) - 1u;
  uint32_t prefix = 0u;
  int remaining = M;  // rank still to find among the entries that share `prefix`
#pragma unroll 1
  for (int pass = 3; pass >= last_pass; --pass) {
    for (int i = lane; i < 256; i += 32) wb->hist[i] = 0u;
    __syncwarp();
    const int shift = 8 * pass;
    for (int i = lane; i < n; i += 32) {
      const uint32_t k = wb->key[i];
      if (pass == 3 || (k >> (shift + 8)) == prefix) atomicAdd(&wb->hist[(k >> shift) & 255u], 1u);
    }
    __syncwarp();
    // lane l owns bins 255 - 8l .. 248 - 8l, scanned from the top
    uint32_t c[8];
    uint32_t mine = 0u;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      c[t] = wb->hist[255 - 8 * lane - t];
      mine += c[t];
    }
    uint32_t above = mine;  // inclusive scan over lanes, then made exclusive
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const uint32_t o = __shfl_up_sync(0xffffffffu, above, d);
      if (lane >= d) above += o;
    }
    above -= mine;
    int bin = -1, rem_new = 0;
    uint32_t run = above;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      if (bin < 0 && run + c[t] >= (uint32_t)remaining) {
        bin = 255 - 8 * lane - t;
        rem_new = remaining - (int)run;
      }
      run += c[t];
    }
    // the first lane (highest bins) whose range reaches the rank holds the answer
    const unsigned found = __ballot_sync(0xffffffffu, bin >= 0);
    const int src = __ffs(found) - 1;
    bin = __shfl_sync(0xffffffffu, bin, src);
    remaining = __shfl_sync(0xffffffffu, rem_new, src);
    prefix = (prefix << 8) | (uint32_t)bin;
    __syncwarp();
  }
  // bf16: complete the code (its lower half repeats the inverted top bit)
  const uint32_t kth = last_pass == 2 ? (prefix << 16) | ((prefix & 0x8000u) ? 0u : 0xffffu) : prefix;
  int out = 0, ties_seen = 0;
#pragma unroll 1
  for (int base = 0; base < n; base += 32) {
    const int i = base + lane;
    const bool valid = i < n;
    const uint32_t k = valid ? wb->key[i] : 0u;
    const int id = valid ? wb->idx[i] : 0;
    const bool eq = valid && k == kth;
    const unsigned eqb = __ballot_sync(0xffffffffu, eq);
    const bool keep = (valid && k > kth) || (eq && ties_seen + __popc(eqb & lt) < remaining);
    const unsigned kb = __ballot_sync(0xffffffffu, keep);
    __syncwarp();  // every lane holds its entry before anything is moved down
    if (keep) {
      const int pos = out + __popc(kb & lt);
      wb->key[pos] = k;
      wb->idx[pos] = id;
    }
    out += __popc(kb);
    ties_seen += __popc(eqb);
    __syncwarp();
  }
  return ((unsigned long long)kth << 32) | (unsigned)out;  // (code of the M-th largest, new count)
}

// Batched examination of queued groups: lane l < nb takes group queue[first + l], reads its 16
// logits again (L2 hits) and appends the tokens above the current threshold to the token buffer,
// in index order (the queue is in index order, lanes append in lane order).  Then the buffer is
// pruned if it has grown past M + 64.  Returns the new count; *thr is raised by a prune.
// Returns (threshold bits << 32) | new count; the threshold is raised by a prune.
template <int DT>
__device__ __noinline__ unsigned long long topm_expand(TopmWarpBuf* wb, const int* queue,
                                                       const char* rowp, int V, int first, int nb,
                                                       int n, int M, float thr) {
  const int lane = threadIdx.x & 31;
  float a[16];
  uint32_t m = 0u;
  int tok = 0;
  if (lane < nb) {
    tok = queue[first + lane] << 4;
#pragma unroll
    for (int t = 0; t < 16; ++t) a[t] = tok + t < V ? load_logit<DT>(rowp, tok + t) : -CUDART_INF_F;
#pragma unroll
    for (int t = 0; t < 16; ++t)
      if (a[t] > thr && a[t] < CUDART_INF_F) m |= 1u << t;  // false for NaN
  }
  const int cnt = __popc(m);
  int incl = cnt;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int o = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += o;
  }
  int pos = n + incl - cnt;
#pragma unroll
  for (int t = 0; t < 16; ++t) {
    if ((m >> t) & 1u) {
      if (GLS_IN_RANGE(pos, 0, kTopmCap, 41u)) {
        wb->key[pos] = enc_ordered(a[t] + 0.0f);  // -0 and +0 are the same logit: one code
        wb->idx[pos] = tok + t;
      }
      ++pos;
    }
  }
  n += __shfl_sync(0xffffffffu, incl, 31);
  __syncwarp();
  if (n > M + 64) {
    const unsigned long long r = topm_prune(wb, n, M, DT == kBF16 ? 2 : 0);
    n = (int)(unsigned)r;
    thr = dec_ordered((uint32_t)(r >> 32));
  }
  return ((unsigned long long)__float_as_uint(thr) << 32) | (unsigned)n;
}

template <int DT>
__global__ void __launch_bounds__(kTopmWarps * 32, kTopmCtasPerSM)
topm_select_kernel(const TopmArgs T) {
  __shared__ TopmWarpBuf bufs[kTopmWarps];
  __shared__ int queues[kTopmWarps][kS4QueueCap];  // group indices awaiting examination
  const int lane = threadIdx.x & 31;
  const int warp = threadIdx.x >> 5;
  const uint32_t lt = (1u << lane) - 1u;
  constexpr int ES = DT == kBF16 ? 2 : 4;
  typedef Group16<DT> G;
  TopmWarpBuf* const wb = &bufs[warp];
  int* const queue = queues[warp];

  const long long n_rows = T.list != nullptr ? (long long)__ldcg(T.count) : T.rows;
  for (long long it = (long long)blockIdx.x * kTopmWarps + warp; it < n_rows;
       it += (long long)gridDim.x * kTopmWarps) {
    const long long row = T.list != nullptr ? (long long)__ldcg(T.list + it) : it;
    if (!GLS_IN_RANGE(row, 0, T.rows, 42u)) continue;
    const int j = (int)(row % T.J);
    const long long bk = row / T.J;
    const int k = (int)(bk % T.K);
    const long long b = bk / T.K;
    const char* rowp = (const char*)T.data + (b * T.sb + k * T.sk + j * T.sj) * ES;
    const bool aligned = (((uintptr_t)rowp) & 31) == 0;
    const int n_steps = (T.V + kS4WarpTokens - 1) / kS4WarpTokens;
    const int n_full = aligned ? T.V / kS4WarpTokens : 0;
    const int tok0 = lane * 16;

    auto load_step = [&](G (&g)[kS4LaneGroups], int s) {
      const int tok = tok0 + s * kS4WarpTokens;
      if (s < n_full) {
        const char* p = rowp + (size_t)tok * ES;
#pragma unroll
        for (int q = 0; q < kS4LaneGroups; ++q) load16_vec(g[q], p + q * 512 * ES);
      } else {
#pragma unroll
        for (int q = 0; q < kS4LaneGroups; ++q) load16_scalar(g[q], rowp, tok + q * 512, T.V);
      }
    };

    float thr = -CUDART_INF_F;
    int n = 0, qn = 0, s = 0;
    __syncwarp();  // the previous row's output loop is done with the buffer
    G nxt[kS4LaneGroups];
    if (n_steps > 0) load_step(nxt, 0);
    for (;;) {
      // the sweep: a group whose maximum exceeds the threshold is queued (in index order); the
      // examination is called from the outer loop so that this loop carries no call
#pragma unroll 1
      for (; s < n_steps && qn < 32; ++s) {
        G g[kS4LaneGroups];
#pragma unroll
        for (int q = 0; q < kS4LaneGroups; ++q) g[q] = nxt[q];
        if (s + 1 < n_steps) load_step(nxt, s + 1);
        const int g0 = (tok0 + s * kS4WarpTokens) >> 4;
#pragma unroll
        for (int q = 0; q < kS4LaneGroups; ++q) {
          const bool hit = group16_max(g[q]) > thr;  // false for NaN
          const unsigned bal = __ballot_sync(0xffffffffu, hit);
          if (bal != 0u) {
            if (hit && GLS_IN_RANGE(qn + __popc(bal & lt), 0, kS4QueueCap, 40u)) queue[qn + __popc(bal & lt)] = g0 + 32 * q;
            qn += __popc(bal);
          }
        }
      }
      if (qn == 0 && s >= n_steps) break;
      __syncwarp();
      for (int first = 0; first < qn; first += 32) {
        const unsigned long long r = topm_expand<DT>(wb, queue, rowp, T.V, first, min(32, qn - first), n, T.M, thr);
        n = (int)(unsigned)r;
        thr = __uint_as_float((uint32_t)(r >> 32));
      }
      qn = 0;
      if (s >= n_steps) break;
    }
    if (n > T.M) n = (int)(unsigned)topm_prune(wb, n, T.M, DT == kBF16 ? 2 : 0);
    __syncwarp();
    for (int i = lane; i < T.M; i += 32) {
      T.ids[row * T.M + i] = i < n ? wb->idx[i] : -1;
      T.logits[row * T.M + i] = i < n ? dec_ordered(wb->key[i]) : -CUDART_INF_F;
    }
  }
}

}  // namespace gls
