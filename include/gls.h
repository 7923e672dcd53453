/*
 * gls.h -- C ABI of libgls: Gumbel-max list sampling (GLS) sweeps for NVIDIA B200 (sm_100a).
 *
 * The library implements the data-parallel part of "List-Level Distribution Coupling with
 * Applications to Speculative Decoding and Lossy Compression" (arXiv 2506.05632):
 *
 *   - Sec. 3, Algorithm 1: with K sets of i.i.d. Exp(1) variables S_i^(k),
 *         X^(k) = argmin_i S_i^(k) / p_i          (draft side, one race per draft k)
 *         Y     = argmin_i min_k S_i^(k) / q_i    (target side, list-combined race)
 *         accept iff Y is one of X^(1..K).
 *   - Sec. 4, Algorithm 2: the same races per position j with noise U_i^(j,k), an active set S of
 *     drafts that is pruned position by position, and a bonus token after L accepted positions.
 *   - Sec. 5.1 and Appendix C: the same races over (importance) weights, with random bin labels
 *     l_i, message M = l_Y and K decoders that only consider candidates whose label equals M.
 *
 * Everything is evaluated in the log domain:  argmin_i S_i/p_i = argmax_i (logit_i/T - ln S_i),
 * because the softmax normaliser of a row does not depend on i.  Where rows with different
 * normalisers meet (the min over k inside Y), each row's log-sum-exp is subtracted first, so the
 * quantity compared is -ln(S_i^(k) / q_i^(j,k)) with q a true probability, as Algorithm 2 writes it.
 *
 * SHARED RANDOMNESS.  The paper only asks for i.i.d. uniforms shared by both parties (Algorithm 1,
 * first step).  Here they are never stored: S = -ln U is a pure function of
 * (seed, sequence id, position id, draft index k, token index i), generated inside the kernels by
 * a counter-based generator (Philox4x32, published by Salmon et al., SC'11):
 *
 *     key     = (seed & 0xffffffff, seed >> 32)
 *     counter = (c0 = token block, c1 = k | (domain << 16), c2 = position id, c3 = sequence id)
 *     domain  = 0 decoding noise, 1 compression noise, 2 / 3 the refinement streams of 0 / 1,
 *               4 / 5 the per-token streams of 0 / 1 (noise_spec 4)
 *
 *   noise_spec 1:  block = i >> 2, w = out[i & 3],                v = (w + 0.5) * 2^-32
 *   S = -log1p(-v)   (v is strictly inside (0,1), so S is finite and positive; this is the paper's
 *                     S = -ln U with U = 1 - v)
 *
 *   noise_spec 4 builds the 16 exponentials of the tokens 16g .. 16g+15 ("group" g) from their
 *   minimum.  If E_0..E_15 are i.i.d. Exp(1), then M = min E_t is Exp(16), its position is uniform
 *   and independent of M, and the other fifteen exceed M by i.i.d. Exp(1) amounts independent of
 *   both (memorylessness).  Read backwards this is an exact sampler of 16 i.i.d. Exp(1) values:
 *                  coarse  block = ((g >> 7) << 5) | (g & 31) in `domain`: w = out[(g >> 5) & 3]
 *                          (128 consecutive groups share 32 calls; groups g, g+32, g+64, g+96 one call)
 *                  refine  block = g in `domain + 2`: r = out[0] & 0xffff, loc = (out[0] >> 16) & 15
 *                  token   block = i >> 2 in `domain + 4`: u = out[i & 3]
 *                  M   = -log1p(-v0) / 16,  v0 = (w * 2^16 + r + 0.5) * 2^-48
 *                  S_i = M                           if (i & 15) == loc
 *                  S_i = M - log1p(-(u + 0.5) 2^-32) otherwise
 *
 * A draft call and a verify call that describe the same (seed, sequence, position, k, i) therefore
 * see the same S -- that is the coupling.  Both specs are exact definitions of i.i.d. Exp(1) noise.
 * Spec 1 is the literal reading, one uniform per token.  Under spec 4 one generator call covers
 * 64 tokens, and a whole group is settled by the bound S_i >= M >= w * 2^-36 (a few dozen groups
 * per row need a closer look).  Spec 4 is the default and about three times faster: the
 * generator's 32x32->64-bit multiplies are the scarcest resource of the sweep on sm_100a.
 * (Values 2 and 3 named two intermediate layouts that split a 48-bit uniform into coarse and
 * refinement bits; they are retired and return GLS_ERR_UNSUPPORTED.)
 *
 * CONVENTIONS
 *   - Token / candidate indices are 0-based (the paper counts from 1).
 *   - All pointers are DEVICE pointers owned by the caller unless the name ends in `_host`.
 *     The library allocates no device memory, keeps no state between calls, enqueues its kernels
 *     on the caller's stream and returns without synchronising.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Rows: the token dimension is contiguous; strides are in ELEMENTS and may be 0 (broadcast).
 *     Rows whose first element is 32-byte aligned (16-byte for noise_spec 1) take the
 *     vectorised path; others are still handled (slower scalar loads).
 *   - A logit of -inf is a legal "masked" token (top-K truncation, Sec. 4.4).  NaN and +inf
 *     logits never win a race and are excluded from the log-sum-exp.
 *   - Ties (measure zero in exact arithmetic): lowest token index, then lowest k.
 *   - Errors the host can see (null pointers, sizes <= 0, K > GLS_MAX_K, V >= 2^31, bad dtype,
 *     inv_temp not finite or <= 0, workspace too small, misaligned base pointer) return a status
 *     and enqueue nothing.  A row with no finite logit yields token -1 and ORs GLS_DEV_EMPTY_SUPPORT
 *     into *device_status; nothing traps.
 *   - Scores are computed in fp64 for the handful of candidates per row that survive the filter,
 *     and returned as fp32.
 */
#ifndef GLS_H_
#define GLS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define GLS_MAX_K 64

typedef enum {
  GLS_OK = 0,
  GLS_ERR_INVALID_ARG = 1,
  GLS_ERR_UNSUPPORTED = 2,
  GLS_ERR_MISALIGNED = 3,
  GLS_ERR_WORKSPACE = 4,
  GLS_ERR_CUDA = 5,
  GLS_ERR_STATIC_LIMIT = 6 /* problem needs more scratch than the built-in static buffer holds */
} gls_status_t;

/* bits OR-ed into *device_status by the kernels */
#define GLS_DEV_EMPTY_SUPPORT 1u /* some row had no finite logit: its token is -1 */

typedef enum { GLS_F32 = 0, GLS_BF16 = 1 } gls_dtype_t;

/* A batch of rows indexed [b][k][j][i]; i (token) is contiguous. */
typedef struct {
  const void* data; /* device pointer to element [0][0][0][0]                       */
  int32_t dtype;    /* gls_dtype_t                                                  */
  int64_t stride_b; /* elements between consecutive b; 0 broadcasts                 */
  int64_t stride_k; /* elements between consecutive k; 0 = one row shared by all k  */
  int64_t stride_j; /* elements between consecutive positions j                     */
} gls_rows_t;

/* noise flags */
#define GLS_NOISE_SHARED_ACROSS_K 1u /* every k uses the noise of k = 0: the comparison scheme of
                                        Sec. 5.2 in which all decoders share one set of numbers */

/* Shared randomness: MUST be identical in the draft call and the verify call of one step. */
typedef struct {
  uint64_t seed;           /* Philox key                                                       */
  uint32_t seq_base;       /* sequence id of batch row b is seq_base + b ...                   */
  const uint32_t* seq_ids; /* ... unless this optional DEVICE array [B] is given               */
  uint32_t pos_base;       /* position id of index j is pos_base + j                           */
  uint32_t noise_spec;     /* 1 or 4 (see above); 0 selects 4                                  */
  uint32_t rounds;         /* Philox rounds, 0 selects 10; 7..16 accepted                      */
  uint32_t flags;          /* GLS_NOISE_*                                                      */
} gls_noise_t;

/* verify flags */
#define GLS_COMBINE_ACTIVE 0u /* Algorithm 2 as printed: the min over k runs over the active set */
#define GLS_COMBINE_ALL 1u    /* Appendix B, strong drafter invariance: min over all k           */
#define GLS_NO_BONUS 2u       /* target rows cover positions 0..L-1 only; no bonus token         */
/* How gls_target_sample_verify walks Algorithm 2 (same results either way; default: by size).  */
#define GLS_VERIFY_ALL_ROWS 4u    /* race every target row, then run the loop on the row results  */
#define GLS_VERIFY_ACTIVE_ROWS 8u /* in phases: only rows of active drafts are read               */
/* The walk in phases as two calls with the same arguments and the same, untouched workspace, for a
 * caller that fetches target rows on demand (e.g. from host memory).  GLS_VERIFY_FIRST_PHASE reads
 * the rows at position 0 only and writes out_tokens[:,0], out_accept[:,:,0] and out_num_tokens
 * (the emitted count for sequences that stopped, 0 for those still running).  GLS_VERIFY_REST
 * reads, of the other rows, only rows (b, k, 1..J-1) with out_accept[b,k,0] == 1 (all of them,
 * or fewer where a further phase can leave some out) and completes all outputs; rows of drafts
 * that did not survive position 0 need not hold valid data.                                      */
#define GLS_VERIFY_FIRST_PHASE 16u
#define GLS_VERIFY_REST 32u
/* The walk in phases with positions 1 and 2 as a phase of their own whatever the size (by default
 * only very large inputs take it: see gls_verify_phases).                                        */
#define GLS_VERIFY_THREE_PHASES 64u

/* Library version, major * 10000 + minor * 100 + patch. */
int gls_version(void);

/*
 * Self-check of the kernels' index arithmetic (no counterpart in the paper).  A library built with
 * -DGLS_DEBUG_BOUNDS range-checks its own shared- and global-memory indices; a violation is counted,
 * the first one recorded, and the access skipped (nothing traps).  Returns 1 and copies
 * {count, site of the first violation, its value, its limit} of the current device to the HOST
 * array (synchronising with the device) when the checks are compiled in, 0 (and zeros) when they
 * are not, -1 if the copy failed.
 */
int gls_debug_bounds(uint32_t out_host[4]);

/* Human-readable name of a status code (static storage, never NULL). */
const char* gls_status_string(int status);

/* Bytes of device workspace that any of the three entry points below needs for a problem of
 * B batch rows, K drafts (streams), J positions and V tokens (candidates).  The workspace holds
 * the per-(row, vocabulary-slice) partial results of the split reduction; its contents on entry
 * are ignored and it may be reused by the next call on the same stream. */
size_t gls_workspace_bytes(int B, int K, int J, int64_t V);

/*
 * Draft side -- Sec. 3 step 2, Algorithm 1 (third step), Algorithm 2 draft loop:
 *     X[b,k,j] = argmin_i S_i^(j,k) / p_i^(j,k) = argmax_i ( logits[b,k,j,i] * inv_temp_k - ln S )
 * with S keyed by (seed, seq(b), pos_base + j, k, i), noise domain 0.
 *
 *   draft_logits          [B,K,J,V] rows (fp32 or bf16)
 *   inv_temp              1 / temperature, used for every k unless ...
 *   inv_temp_per_draft_host  ... this HOST array [K] is non-NULL (Sec. 4.3 varies draft temperatures)
 *   out_tokens            [B,K,J] int32, -1 for a row without finite logits
 *   out_scores            NULL or [B,K,J] fp32: the winning logit*inv_temp - ln S (unnormalised)
 *   workspace, workspace_bytes  >= gls_workspace_bytes(B,K,J,V)
 *   device_status         NULL or uint32[1]; bits are OR-ed in, the caller zeroes it
 */
int gls_draft_sample(const gls_rows_t* draft_logits, int B, int K, int J, int64_t V, float inv_temp,
                     const float* inv_temp_per_draft_host, const gls_noise_t* noise,
                     int32_t* out_tokens, float* out_scores, void* workspace,
                     size_t workspace_bytes, uint32_t* device_status, void* stream);

/*
 * Compression from the source -- Appendix C (importance sampling: candidates U_i drawn from a
 * proposal, unnormalised weights p_{W|A}(U_i | a) / prop(U_i) at the encoder and
 * p_{W|T}(U_i | t_k) 1{l_i = M} / prop(U_i) at decoder k) with the Gaussian model of Sec. 5.2 /
 * Appendix D.3 applied per dimension: p_{W|A}(. | a) = N(a, s2_eta), T_k = A + N(0, s2_zeta),
 * p_{W|T}(. | t) = N(t / s2_T, s2_W - 1 / s2_T) with s2_T = 1 + s2_zeta, s2_W = 1 + s2_eta, proposal
 * N(0, s2_prior).  The log-weights
 *     encoder  sum_d -(u_id - a_bd)^2 / (2 s2_eta) + u_id^2 / (2 s2_prior)
 *     decoder  sum_d -(u_id - t_bkd / s2_T)^2 / (2 (s2_W - 1 / s2_T)) + u_id^2 / (2 s2_prior)
 * (terms common to a row dropped) are computed inside the kernels from the D coordinates of each
 * candidate -- nothing of size B x N is read or written -- and raced as in gls_compress_select,
 * whose outputs this call reproduces for those weights; the winners' weights are recomputed in
 * fp64.  Then, per decoder, W_k = U_{X^(k)}, the MMSE reconstruction
 *     g(w, t) = (s2_zeta w + s2_eta t) / (s2_eta + s2_zeta + s2_eta s2_zeta)      (Appendix D.3)
 * and its squared error against the source, averaged over the D dimensions.
 *
 *   candidates  [N,D] fp32, source [B,D] fp32, side_info [B,K,D] fp32 (all contiguous)
 *   bins        NULL, [N] (bins_stride_b = 0) or [B,N] uint8
 *   out_recon   NULL or [B,K,D] fp32;  out_sqerr NULL or [B,K] fp32;  the rest as
 *               gls_compress_select
 *   workspace   gls_compress_gaussian_workspace_bytes(B, K, N) bytes
 * Default noise layout only; D <= 16, K <= 8, N < 2^28 (GLS_ERR_UNSUPPORTED otherwise: compute
 * the weights and call gls_compress_select).
 */
size_t gls_compress_gaussian_workspace_bytes(int B, int K, int64_t N);
int gls_compress_gaussian(const float* candidates, const float* source, const float* side_info,
                          const uint8_t* bins, int64_t bins_stride_b, int B, int K, int64_t N, int D,
                          double s2_eta, double s2_zeta, double s2_prior, const gls_noise_t* noise,
                          int32_t* out_enc_index, uint8_t* out_message, int32_t* out_dec_index,
                          uint8_t* out_match, float* out_scores, float* out_recon, float* out_sqerr,
                          void* workspace, size_t workspace_bytes, uint32_t* device_status,
                          void* stream);

/*
 * Draft-side sampling for callers that cannot allocate device memory.  The paper has no counterpart
 * to this call; it exists for deployment only and computes exactly what gls_draft_sample computes.
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a step function inside a serving
 * loop that must not take cudaMalloc's device-wide synchronisation, or a plug-in whose host has
 * handed every byte of device memory to its own pool and offers no hook to borrow some.  Such a
 * caller has nowhere to get the `workspace` that gls_draft_sample asks for.  Here the scratch
 * (bound hints, per-slice partial results, per-row results) lives in a buffer of
 * GLS_STATIC_SCRATCH_BYTES that is compiled into the library image: every GPU that loads the
 * library carries it from load until the process exits.  The call itself performs no cudaMalloc,
 * no cudaFree and no allocating library routine.
 *
 * Arguments are those of gls_draft_sample without workspace / workspace_bytes; inputs and outputs
 * still belong to the caller.
 *
 * Limits and rules:
 *   - A problem whose scratch need (that of gls_draft_sample: hints, partial results and row
 *     results of the B * K * J rows; never more than gls_workspace_bytes(B, K, J, V)) exceeds
 *     GLS_STATIC_SCRATCH_BYTES is refused with GLS_ERR_STATIC_LIMIT and nothing is enqueued
 *     (gls_static_scratch_bytes() returns the limit at run time).
 *   - The first call on each device looks up the buffer's device address (one
 *     cudaGetSymbolAddress with that device current) and remembers it.  Make that first call
 *     outside any stream capture.
 *   - Every call on a device shares the one buffer, which still holds the previous call's contents;
 *     the call clears the part that must start at zero on `stream` before using it.  Two calls that
 *     can overlap on the GPU (different streams without an ordering between them) race on the
 *     buffer: order them, or use gls_draft_sample with separate workspaces.
 */
#define GLS_STATIC_SCRATCH_BYTES (4u << 20)
size_t gls_static_scratch_bytes(void);
int gls_draft_sample_static(const gls_rows_t* draft_logits, int B, int K, int J, int64_t V,
                            float inv_temp, const float* inv_temp_per_draft_host,
                            const gls_noise_t* noise, int32_t* out_tokens, float* out_scores,
                            uint32_t* device_status, void* stream);

/*
 * Target side and verification -- Sec. 3 step 1 and the verification phase of Algorithm 2 (from
 * the initialisation of the active set to the end).  With S = {0..K-1} initially, for j = 0..L-1:
 *     Y_j = i-component of argmin_{i, k in S} S_i^(j,k) / q_i^(j,k),
 *           q^(j,k) = softmax(target_logits[b,k,j,:] * inv_temp)
 *     accept[b,k,j] = (k in S and draft_tokens[b,k,j] == Y_j);  S <- {k in S : accept}
 *     if S is empty: tau = j + 1, stop.
 * If all L positions leave S non-empty, the bonus token Y_L is drawn the same way from the rows at
 * position L and tau = L + 1 (with GLS_NO_BONUS: no such rows, tau = L).
 * GLS_COMBINE_ALL is Appendix B: Y_j = argmin_i min over ALL k of S_i^(j,k) / q_i with q the target
 * distribution of the accepted prefix, while S still records the survivors.  With target rows
 * shared by all k (stride_k = 0) each stream's race over the shared row is that quantity.  With a
 * row per draft, q is the row of the lowest-numbered active draft (active drafts share the
 * accepted prefix): every row is raced under all K streams at once and the epilogue reads that
 * row; this needs the default noise layout, K <= 8 and V < 2^28 (GLS_ERR_UNSUPPORTED otherwise)
 * and costs K times the noise arithmetic of a plain call.
 * Algorithm 1 is the case L = 1 with GLS_NO_BONUS: accept iff some accept[b,k,0] is 1.
 *
 *   target_logits   [B,K,J,V] rows, J = L + 1 (J = L with GLS_NO_BONUS)
 *   draft_tokens    [B,K,L] int32 (the X of the draft phase)
 *   out_tokens      [B,J] int32, -1 at and beyond index tau
 *   out_num_tokens  [B] int32 = tau
 *   out_accept      [B,K,L] uint8
 *   out_scores      NULL or [B,J] fp32: ln(q_Y / S) of each emitted token, 0 beyond tau
 *   L = 0 is legal (bonus token only).
 */
int gls_target_sample_verify(const gls_rows_t* target_logits, int B, int K, int L, int64_t V,
                             float inv_temp, const int32_t* draft_tokens, const gls_noise_t* noise,
                             uint32_t flags, int32_t* out_tokens, int32_t* out_num_tokens,
                             uint8_t* out_accept, float* out_scores, void* workspace,
                             size_t workspace_bytes, uint32_t* device_status, void* stream);

/*
 * Which way gls_target_sample_verify would walk Algorithm 2 for these arguments (no counterpart
 * in the paper; the results do not depend on it).  0: every target row is raced, then the loop
 * runs on the row results.  1: in phases -- position 0 of every draft, then the remaining positions
 * of the drafts still active -- so that a target row is read only while Algorithm 2 can still use
 * it: B * K rows plus (J - 1) rows per draft that survives position 0, instead of B * K * J
 * (under GLS_COMBINE_ALL on a row per draft: B rows plus (J - 1) per survivor).  Chosen by size
 * unless `flags` carries GLS_VERIFY_ALL_ROWS or GLS_VERIFY_ACTIVE_ROWS; the walk in phases
 * needs the default noise layout, L >= 1 and J >= 2, and under GLS_COMBINE_ALL a row per draft.
 * row_per_draft: target rows' stride_k != 0.  Returns -1 for arguments the call would refuse.
 */
int gls_verify_walk(int dtype, int row_per_draft, int B, int K, int L, int64_t V, int noise_spec,
                    uint32_t flags);
/*
 * The phases of that walk: returns their number (0 when every row is raced, -1 for refused
 * arguments) and writes to the HOST array ends[p] = one past the last position of phase p.  Phase
 * p reads the rows (b, k, j), j in [ends[p-1], ends[p]), of the drafts k still active when it
 * starts (phase 0: every draft, position 0).  Two phases normally; very large inputs take
 * positions 1 and 2 as a phase of their own before the rest.
 */
int gls_verify_phases(int dtype, int row_per_draft, int B, int K, int L, int64_t V, int noise_spec,
                      uint32_t flags, int ends_host[4]);

/*
 * Plumbing for callers whose logits live in (pinned) host memory and who fetch only the rows a
 * call will read (no counterpart in the paper): n_rows rows of row_bytes bytes each, the rows
 * src_pitch bytes apart on the host and dst_pitch bytes apart on the device, copied host to
 * device on `stream` as one strided copy -- e.g. the position-0 rows of a [B,K,J,V] tensor
 * (pitch J * V * element size) ahead of GLS_VERIFY_FIRST_PHASE.  Asynchronous for pinned host
 * memory.  Returns GLS_OK, GLS_ERR_INVALID_ARG (null pointer, a pitch below row_bytes) or
 * GLS_ERR_CUDA.
 */
int gls_copy_rows_to_device(void* dst_device, size_t dst_pitch, const void* src_host, size_t src_pitch,
                            size_t row_bytes, size_t n_rows, void* stream);

/*
 * Draft phase and verification in one call -- Algorithm 2 from its draft loop to its end, for the
 * case where both sets of logits are resident (all L draft positions are known, e.g. a drafter
 * that is not autoregressive in the tokens sampled here, a replayed or re-scored step, or the
 * last position of an autoregressive loop together with its verification).  Equivalent to
 * gls_draft_sample(draft_logits, J = L) followed by gls_target_sample_verify(target_logits, the
 * tokens just drawn), bit for bit, but one sweep launch covers both sets of rows and one
 * reduction launch finalises the draft rows, the target rows and Algorithm 2's loop, which halves
 * the number of launches of a step (what bounds small batches).  Inputs for which
 * gls_verify_walk() answers 1 are large enough that launches do not matter: there the call runs
 * the draft rows first and then Algorithm 2 in phases on the tokens just drawn.
 *
 *   draft_logits       [B,K,L,V] rows, temperature inv_temp_draft (or per draft, host array [K])
 *   target_logits      [B,K,J,V] rows, J = L + 1 (J = L with GLS_NO_BONUS), temperature
 *                      inv_temp_target; same dtype as draft_logits
 *   out_draft_tokens   [B,K,L] int32, out_draft_scores NULL or [B,K,L] fp32 (as gls_draft_sample)
 *   out_tokens, out_num_tokens, out_accept, out_scores: as gls_target_sample_verify
 *   workspace          at least gls_draft_verify_workspace_bytes(B, K, L, J, V) bytes
 * L >= 1.  Default noise layout only; K, L such that K * (32 J + 4 L) bytes fit in 48 KB
 * (GLS_ERR_UNSUPPORTED otherwise: use the two calls).  GLS_COMBINE_ALL with a target row per draft
 * runs as the two calls internally (and has their limits: K <= 8).
 */
size_t gls_draft_verify_workspace_bytes(int B, int K, int L, int J, int64_t V);
int gls_draft_verify(const gls_rows_t* draft_logits, const gls_rows_t* target_logits, int B, int K,
                     int L, int64_t V, float inv_temp_draft, const float* inv_temp_per_draft_host,
                     float inv_temp_target, const gls_noise_t* noise, uint32_t flags,
                     int32_t* out_draft_tokens, float* out_draft_scores, int32_t* out_tokens,
                     int32_t* out_num_tokens, uint8_t* out_accept, float* out_scores,
                     void* workspace, size_t workspace_bytes, uint32_t* device_status,
                     void* stream);

/*
 * Sparse rows -- Sec. 4.4 (top-K truncation: only M << N high-probability tokens are kept) and
 * Appendix D.1 (the experiments keep the top 50 tokens).  A row is a
 * list of M kept tokens: their ids in the full vocabulary and their logits; every other token has
 * probability zero.  The races are those of the dense entry points on the row with -inf outside
 * the list, with the noise of each kept token keyed by its ORIGINAL id, so a sparse call and a
 * dense call on the correspondingly masked row return the same tokens and scores.  All kept tokens
 * are scored directly (fp64); no workspace is needed.
 *
 *   token_ids  int32 [B,K,J,M] (strides below, M contiguous); -1 marks an empty slot; the ids of
 *              one row must be distinct
 *   logits     fp32, same indexing
 *   strides    in elements, shared by both arrays; stride_k = 0 shares one list among all k
 */
typedef struct {
  const int32_t* token_ids;
  const float* logits;
  int64_t stride_b, stride_k, stride_j;
  int32_t M;
} gls_sparse_rows_t;

/* gls_draft_sample on sparse rows: out_tokens holds vocabulary ids (-1 for an empty row). */
int gls_draft_sample_sparse(const gls_sparse_rows_t* draft_rows, int B, int K, int J, float inv_temp,
                            const float* inv_temp_per_draft_host, const gls_noise_t* noise,
                            int32_t* out_tokens, float* out_scores, uint32_t* device_status,
                            void* stream);

/* gls_target_sample_verify on sparse rows (same flags, same outputs).  Each list is normalised
 * over its kept tokens, as top-K sampling does.  K * J must not exceed 1536. */
int gls_target_sample_verify_sparse(const gls_sparse_rows_t* target_rows, int B, int K, int L,
                                    float inv_temp, const int32_t* draft_tokens,
                                    const gls_noise_t* noise, uint32_t flags, int32_t* out_tokens,
                                    int32_t* out_num_tokens, uint8_t* out_accept, float* out_scores,
                                    uint32_t* device_status, void* stream);

/*
 * Top-M truncation fused in front of the sparse-row races (Sec. 4.4, Appendix D.1: the paper's
 * experiments sample from the M = 50 most likely tokens).  Every dense row [V] is reduced, in one
 * pass, to its M largest logits (ties at the M-th value: lowest token index; NaN, +inf and -inf
 * logits are never kept; a row with fewer than M finite logits keeps them all), then
 * gls_draft_sample_sparse / gls_target_sample_verify_sparse run on the lists: probabilities are
 * normalised over the kept tokens and the noise of a kept token is that of its vocabulary id.
 * 1 <= M <= 256.  `workspace` (device, gls_topm_workspace_bytes) receives the lists: int32 ids
 * [B,K,J,M] followed, 256-byte aligned, by fp32 logits [B,K,J,M], in index order, id -1 past the
 * kept count; the caller may read them after the call.  Errors as for the dense entry points;
 * K * (L + 1) must not exceed 1536 for the verify call.  The verify call on a row per draft walks
 * Algorithm 2 in phases when gls_verify_walk() says so for the dense rows (or `flags` carries
 * GLS_VERIFY_ACTIVE_ROWS; GLS_VERIFY_ALL_ROWS forbids it): the selection, which is what the call
 * costs, then runs only over the rows the walk reads -- position 0 of every draft, then the
 * remaining positions of the drafts that survived it -- and the lists of the other rows are left
 * unwritten.  After the lists the workspace holds the state of that walk.
 */
size_t gls_topm_workspace_bytes(int B, int K, int J, int M);
int gls_draft_sample_topm(const gls_rows_t* draft_logits, int B, int K, int J, int64_t V, int M,
                          float inv_temp, const float* inv_temp_per_draft_host,
                          const gls_noise_t* noise, int32_t* out_tokens, float* out_scores,
                          void* workspace, size_t workspace_bytes, uint32_t* device_status,
                          void* stream);
int gls_target_sample_verify_topm(const gls_rows_t* target_logits, int B, int K, int L, int64_t V,
                                  int M, float inv_temp, const int32_t* draft_tokens,
                                  const gls_noise_t* noise, uint32_t flags, int32_t* out_tokens,
                                  int32_t* out_num_tokens, uint8_t* out_accept, float* out_scores,
                                  void* workspace, size_t workspace_bytes, uint32_t* device_status,
                                  void* stream);

/*
 * Compression -- Sec. 5.1 and Appendix C.  Per batch row b (one source sample):
 *     encoder:   Y = argmin_i min_k S_i^(k) / lambda_q,i          lambda_q = softmax(enc_logw[b,:])
 *                M = bins[Y]                                      (the log2(L_max)-bit message)
 *     decoder k: X^(k) = argmin_{i : bins[i] == M} S_i^(k) / lambda_p,i^(k)
 *                                                                 from dec_logw[b,k,:]
 *     match = (Y is one of X^(1..K))
 * Noise is keyed by (seed, seq(b), pos_base, k, i) in domain 1.  Normalising the weights cannot
 * change a per-row argmin; it only enters the reported encoder score through the log-sum-exp.
 *
 *   enc_logw      rows [B,1,1,N]: stride_b (or 0) is used, stride_k / stride_j are ignored
 *   dec_logw      rows [B,K,1,N]; NULL skips the decoders (out_dec_index / out_match then unused)
 *   bins          NULL (every label equal, L_max = 1) or uint8 labels [N] (bins_stride_b = 0) or
 *                 [B,N] (bins_stride_b = N)
 *   out_enc_index [B] int32, out_message [B] uint8, out_dec_index [B,K] int32, out_match [B] uint8
 *   out_scores    NULL or [B,1+K] fp32: encoder ln(lambda_q,Y / S), then each decoder's
 *                 unnormalised winning logw - ln S
 *   workspace     >= gls_workspace_bytes(B, K, 1, N)  (the encoder and decoder phases reuse it)
 */
int gls_compress_select(const gls_rows_t* enc_logw, const gls_rows_t* dec_logw, const uint8_t* bins,
                        int64_t bins_stride_b, int B, int K, int64_t N, const gls_noise_t* noise,
                        int32_t* out_enc_index, uint8_t* out_message, int32_t* out_dec_index,
                        uint8_t* out_match, float* out_scores, void* workspace,
                        size_t workspace_bytes, uint32_t* device_status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* GLS_H_ */
