/*
 * avsa -- protected sparse video attention for joint audio-video diffusion transformers, sm_100a.
 *
 * C ABI of libavsa.so.  Three calls make one layer-step of the path:
 *
 *   avsa_cross_attn_scores   audio->video cross-attention (Eq. 1) that also emits the per-video-token
 *                            cross-modal response scores (Eq. 2, with the blend of Eq. 4 folded in)
 *   avsa_build_block_mask    protected token set (Eq. 3 / Eq. 8), block-importance top-k, and the
 *                            protected block mask (Eq. 9) as ascending per-row column lists
 *   avsa_sparse_self_attn    video self-attention under that mask (Eq. 10 / Eq. 11)
 *
 * Conventions for every call
 *   - All data pointers are DEVICE pointers unless a parameter says "host".  The caller owns every
 *     buffer.  The library allocates no device memory, never synchronises the stream (except
 *     avsa_read_status) and enqueues work on the given stream only.
 *   - Tensors are bf16 with the head dimension contiguous, described by element strides (avsa_bf16_4d),
 *     so both [B,H,N,d] and [B,N,H,d] storage work.  Base pointers must be 16-byte aligned and strides
 *     multiples of 8 elements.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).  No call reads device
 *     data on the host, so the calls may be recorded into a CUDA graph by stream capture (not on the legacy
 *     default stream) and replayed; pointers, sizes and counts are fixed at capture time.
 *   - `ws` is scratch of at least the matching *_workspace_bytes().  Its first AVSA_STATUS_BYTES (256) bytes
 *     are reserved for a 24-byte status record of six int32: code (avsa_status), where, item, aux -- filled
 *     when a device-side check fails (a wait that ran out of time, or a malformed column list) -- then at
 *     byte 16 the count of recomputed work items (see below) and at byte 20 the head of the persistent
 *     kernels' work queue.  Calls on the same workspace must not overlap on the GPU.
 *   - The attention calls (cross-attention pass 1, sparse self-attention, protected rows) run a kernel that
 *     normalises each row by the maximum of its first key tile instead of a running maximum (softmax is
 *     invariant to that shift), and behind it an exact-rescaling kernel for the work items whose rows
 *     outgrew that reference (a row whose sum of exp(logit - reference) ends above 2^64 or not finite;
 *     values of v are assumed to stay below 2^60 in magnitude).  Results do not depend on which kernel
 *     produced them beyond rounding; the int32 at byte 16 of ws counts the recomputed items (diagnostic).
 *   - Errors detectable on the host return at once with nothing enqueued.  Return values are
 *     avsa_status codes.
 *   - Supported shapes: (blk, d) in {(128,128), (64,64)}; any N >= 1 (the last block may be partial:
 *     pooled means divide by the valid count, invalid keys are masked, rows >= N are not written).
 */
#ifndef AVSA_H_
#define AVSA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define AVSA_API __attribute__((visibility("default")))
#else
#define AVSA_API
#endif

typedef enum {
  AVSA_OK = 0,
  AVSA_ERR_INVALID_ARG = 1,  /* null pointer, bad size, bad alignment or stride */
  AVSA_ERR_UNSUPPORTED = 2,  /* (blk, d) combination or device not supported */
  AVSA_ERR_WORKSPACE = 3,    /* ws is NULL or smaller than *_workspace_bytes() */
  AVSA_ERR_CUDA = 4,         /* a CUDA runtime / driver call failed */
  AVSA_ERR_TIMEOUT = 5,      /* device: a bounded wait expired (read with avsa_read_status) */
  AVSA_ERR_BAD_MASK = 6      /* device: a column list entry was out of range or not ascending */
} avsa_status;

/* Size of the status record area at the start of every workspace. */
#define AVSA_STATUS_BYTES 256

/* bf16 tensor [B,H,N,d], d contiguous; strides in elements. */
typedef struct {
  const void* ptr;
  int64_t stride_b, stride_h, stride_n;
} avsa_bf16_4d;

/* flags of avsa_build_block_mask */
#define AVSA_PROTECT_ROWS 1u            /* Eq. 9: a protected query block keeps every key block */
#define AVSA_PROTECT_COLS 2u            /* opt-in superset: protected key blocks visible to all rows */
#define AVSA_USE_GIVEN_BLOCK_SCORES 4u  /* block_scores is an input; q and k are not read */
#define AVSA_PROTECT_TOKENS 8u          /* lists carry the base pattern only (no block is made dense); the
                                           protected rows are restored by avsa_protected_rows_attn */

#define AVSA_PROTECT_BLOCK_SUM 16u      /* not in the paper: n_protect counts BLOCKS (0..NB); the protected blocks are
                                           those with the largest summed response (fp64 sum of the block's scores
                                           rounded to fp32, ties to the lowest block index); prot_tok flags every
                                           token of a protected block.  Combines with ROWS / COLS / TOKENS. */

/* Optional, ORed into flags: a block counts as protected only if it holds at least n (1..blk) protected tokens.
 * Not in the paper: in raster order a compact region straddles many blocks, and n > 1 trades the protection of
 * stray tokens for fewer dense blocks.  n = 0 or 1 is the block lift of Eq. 9 (any protected token). */
#define AVSA_MIN_TOKENS_PER_BLOCK(n) (((unsigned)(n) & 0xffu) << 8)

/*
 * (1) Cross-attention with response scores -- Eq. 1, Eq. 2 (and the running blend of Eq. 4).
 *
 *   A[b,h,j,i] = softmax_i(q[b,h,j,:] . k[b,h,i,:] * softmax_scale)            (queries j, keys i)
 *   o[b,h,j,:] = sum_i A[b,h,j,i] v[b,h,i,:]                  -> o   bf16, same strides as q's tensor
 *   lse[b,h,j] = natural-log log-sum-exp of row j              -> lse fp32 [B,H,Nq]
 *   scores[b,i] = score_beta * scores[b,i] + score_gamma * sum_h sum_j A[b,h,j,i]   fp32 [B,Nk]
 *
 * For the audio->video direction q holds the audio queries and k, v the video keys/values.  The
 * paper's Norm is any scalar: score_gamma = 1/(H*Nq*layers) makes the scores sum to 1; score_beta = 1
 * accumulates layers; score_beta = alpha with score_gamma = (1-alpha)/(H*Nq) is Eq. 4.
 * With score_beta == 0 the previous contents of scores are ignored (may be uninitialised).
 * o, lse and scores may each be NULL to skip that output (scores == NULL skips the second pass).
 * softmax_scale == 0 means 1/sqrt(d).  When scores are requested min(Nq, Nk) <= 512 (the score pass keeps the
 * shorter axis of a head on chip: the audio queries, or, in the reverse video->audio direction of the
 * bidirectional pair, the audio keys); without scores any Nq and Nk.  The head sum is taken in a fixed order, so
 * results reproduce bit for bit.  `o` has strides (o_stride_b, o_stride_h, o_stride_n) = q's.
 */
AVSA_API int avsa_cross_attn_scores(int B, int H, int Nq, int Nk, int d, avsa_bf16_4d q, avsa_bf16_4d k, avsa_bf16_4d v,
                           void* o_bf16, float* lse, float* scores, float score_beta, float score_gamma,
                           float softmax_scale, void* ws, size_t ws_bytes, void* stream);
AVSA_API size_t avsa_cross_attn_scores_workspace_bytes(int B, int H, int Nq, int Nk, int d);

/*
 * (2) Mask construction -- Eq. 3 / Eq. 8 (protected set), Eq. 9 (protected mask), and the base
 * sparse pattern the paper leaves open, here: block mean-pooling of q and k, block scores
 * Bs[b,h,qb,kb] = mean(q block qb) . mean(k block kb) * softmax_scale, per (head, query block)
 * top-k_keep over kb.
 *
 *   scores       fp32 [B,N] token saliency; may be NULL iff n_protect == 0
 *   n_protect    size of the protected token set, 0 <= n_protect <= N (= ceil(rho N), host integer)
 *   k_keep       kept key blocks per unprotected row, 1 <= k_keep <= NB, NB = ceil(N / blk)
 *   block_scores fp32 [B,H,NB,NB]: output, or input with AVSA_USE_GIVEN_BLOCK_SCORES (never NULL)
 *   col_idx      int32 [B,H,NB,NB]: kept key blocks of each row, ascending, unused slots = -1
 *   col_cnt      int32 [B,H,NB]
 *   prot_tok     uint8 [B,N]  1 = token in the protected set (optional, may be NULL)
 *   prot_blk     uint8 [B,NB] 1 = block holds a protected token (optional, may be NULL)
 *
 * Every top-k orders by (value larger, then index smaller); NaN ranks as -inf; -0 equals +0.
 * Given the same fp32 scores / block_scores the outputs are exactly determined (integer results).
 * Without any AVSA_PROTECT_* flag AVSA_PROTECT_ROWS is assumed.  NB <= 2048.
 */
AVSA_API int avsa_build_block_mask(int B, int H, int N, int d, int blk, avsa_bf16_4d q, avsa_bf16_4d k, const float* scores,
                          int n_protect, int k_keep, unsigned flags, float softmax_scale, float* block_scores,
                          int32_t* col_idx, int32_t* col_cnt, uint8_t* prot_tok, uint8_t* prot_blk, void* ws,
                          size_t ws_bytes, void* stream);
AVSA_API size_t avsa_build_block_mask_workspace_bytes(int B, int H, int N, int d, int blk);

/*
 * (3) Block-sparse self-attention -- Eq. 10 (Eq. 5 when every list is full).
 *
 *   o[b,h,i,:] = softmax_j(q_i . k_j * softmax_scale  restricted to keys j of the listed blocks) v
 *
 * For query block qb of head h the kept key blocks are col_idx[b,h,qb,0 .. col_cnt[b,h,qb]-1]
 * (row stride NB, ascending, each in [0,NB)).  Every list needs at least one entry; a malformed
 * entry sets AVSA_ERR_BAD_MASK in the status record and that block is skipped without any
 * out-of-range access.  o is bf16 with the strides of q; lse (optional) is fp32 [B,H,N] natural log.
 *
 * After the call the int32 at byte 16 of ws is the number of work items the exact kernel recomputed (see
 * the conventions above), and their indices ((b*H + h)*NB + query block, in no particular order) follow
 * as int32 behind the first AVSA_STATUS_BYTES bytes (diagnostic; results do not depend on it).
 */
AVSA_API int avsa_sparse_self_attn(int B, int H, int N, int d, int blk, avsa_bf16_4d q, avsa_bf16_4d k, avsa_bf16_4d v,
                          const int32_t* col_idx, const int32_t* col_cnt, void* o_bf16, float* lse,
                          float softmax_scale, void* ws, size_t ws_bytes, void* stream);
AVSA_API size_t avsa_sparse_self_attn_workspace_bytes(int B, int H, int N, int d, int blk);

/*
 * (4) Token-exact protection -- Eq. 9 applied to tokens, i.e. the row-wise form of Eq. 11: the rows of
 * the protected tokens are dense attention rows ("dense-row recomputation" in the paper's notes).
 *
 * Use with lists built under AVSA_PROTECT_TOKENS: run avsa_sparse_self_attn first, then this call, which
 * recomputes o[b,h,i,:] (and lse[b,h,i], if given) for every token i with prot_tok[b,i] != 0 as dense
 * attention over all N keys and overwrites those rows in place.  The cost is n_protect * N per head
 * (Eq. 16's rho N^2 term) instead of a whole block row per touched block.
 *   prot_tok   uint8 [B,N] as written by avsa_build_block_mask; exactly n_protect flags per batch item,
 *              otherwise AVSA_ERR_BAD_MASK is recorded and that batch item is left untouched
 *   o_bf16     in/out, bf16 with the strides of q;  lse in/out fp32 [B,H,N] or NULL
 * n_protect == 0 is a no-op.  The workspace also depends on n_protect.
 */
AVSA_API int avsa_protected_rows_attn(int B, int H, int N, int d, int blk, avsa_bf16_4d q, avsa_bf16_4d k,
                                      avsa_bf16_4d v, const uint8_t* prot_tok, int n_protect, void* o_bf16,
                                      float* lse, float softmax_scale, void* ws, size_t ws_bytes, void* stream);
AVSA_API size_t avsa_protected_rows_attn_workspace_bytes(int B, int H, int N, int d, int blk, int n_protect);

/*
 * (5) Cache-reuse indicators -- Eq. 12 (stream-wise feature change), Eq. 13 (change over the protected video
 * tokens), Eq. 14 (saliency drift) and Eq. 15 (their maximum against the threshold).
 *
 *   y_v, yhat_v  bf16 [B,Nv,C] contiguous: current and cached block outputs of the video stream
 *   y_a, yhat_a  bf16 [B,Na,C] contiguous: the same for the audio stream
 *   prot_tok     uint8 [B,Nv] protected-token flags (NULL: no protected set, dp = 0)
 *   s_cur, s_anchor  fp32 [B,Nv] current and anchor saliency maps (both NULL: ds = 0)
 *   out          fp32 [B,8]: dv, da, dp, ds, dsync = max(dv, da, lambda_p*dp, lambda_s*ds), reuse (1.0 iff
 *                dsync < tau), two unused slots
 *   dv = sum|y - yhat| / (sum|y| + eps), likewise da and dp; ds = 1 - <s,s^>/(|s||s^| + eps).
 * C must be a multiple of 8.  Sums are taken in a fixed order (bit-reproducible).  The paper's settings are
 * lambda_p = 0.5, lambda_s = 0.1, tau = 0.2.
 */
AVSA_API int avsa_cache_indicators(int B, int Nv, int Na, int C, const void* y_v, const void* yhat_v, const void* y_a,
                                   const void* yhat_a, const uint8_t* prot_tok, const float* s_cur,
                                   const float* s_anchor, float lambda_p, float lambda_s, float tau, float eps,
                                   float* out, void* ws, size_t ws_bytes, void* stream);
AVSA_API size_t avsa_cache_indicators_workspace_bytes(int B, int Nv, int Na, int C);

/*
 * Allocation-free variant of avsa_build_block_mask.  The paper has no counterpart; this is a
 * convenience of the library for callers that have no device allocator to draw a workspace from:
 * code that runs after its host application has frozen its memory budget, extensions loaded into
 * a runtime that owns all device memory and hands none out, and latency-critical loops in which a
 * synchronising allocation is not acceptable.
 *
 * Same arguments and results as avsa_build_block_mask, without `ws`: the scratch (pooled block means,
 * fallback flag buffers and the status record) lives in a fixed array of AVSA_STATIC_SCRATCH_BYTES
 * inside the library, which every GPU that loads libavsa.so holds until the process exits.
 *   - Shapes whose avsa_build_block_mask_workspace_bytes() exceeds AVSA_STATIC_SCRATCH_BYTES are
 *     refused with AVSA_ERR_WORKSPACE and nothing is enqueued.
 *   - The first call on each device looks up the array's device address (with that device current).
 *     Make that first call before starting any stream capture.
 *   - The call allocates nothing: no cudaMalloc/cudaFree, no allocating library routine.
 *   - All calls on a device share the one array, and it keeps the previous call's contents; what must
 *     start from zero (the status record) is cleared by the call itself.  Two such calls that overlap
 *     on the GPU (different streams) race on the array: serialise them.
 *   - The mask kernels have no device-side failure mode (no waits, no list input), so there is no
 *     status record to read after this call.
 *   - Call it from one host thread at a time per device.  The looked-up address belongs to the current
 *     context: after cudaDeviceReset() it is stale, and the library must be reloaded before the next call.
 */
#define AVSA_STATIC_SCRATCH_BYTES (16u << 20)
AVSA_API int avsa_build_block_mask_static(int B, int H, int N, int d, int blk, avsa_bf16_4d q, avsa_bf16_4d k,
                                          const float* scores, int n_protect, int k_keep, unsigned flags,
                                          float softmax_scale, float* block_scores, int32_t* col_idx,
                                          int32_t* col_cnt, uint8_t* prot_tok, uint8_t* prot_blk, void* stream);

/* Host integer ceil(pct/100 * n): the count forms of rho and kappa (Eq. 8's ceiling). */
AVSA_API int avsa_count_from_percent(int pct, int n);

/* Synchronises `stream`, copies the status record of `ws` to the host and returns its code
 * (AVSA_OK, AVSA_ERR_TIMEOUT or AVSA_ERR_BAD_MASK).  detail (host, optional) receives 3 ints that
 * say where the check failed.  For tests and debugging; the hot path never calls it. */
AVSA_API int avsa_read_status(const void* ws, void* stream, int* detail);

/* Self-test of the device-side time limit (tests only): enqueues one warp that waits on a barrier nothing
 * ever signals, gives up after `limit_cycles` SM clock cycles (0 .. 2e9, i.e. about a second at most), records
 * AVSA_ERR_TIMEOUT in the status record at `ws` (>= AVSA_STATUS_BYTES; detail = {99, 0, cycles waited / 1024})
 * and returns; the context stays usable.  The tile kernels bound every one of their waits the same way. */
AVSA_API int avsa_selftest_bounded_wait(void* ws, size_t ws_bytes, long long limit_cycles, void* stream);

AVSA_API const char* avsa_status_string(int status);
AVSA_API int avsa_version(void);

#ifdef __cplusplus
}
#endif
#endif /* AVSA_H_ */
