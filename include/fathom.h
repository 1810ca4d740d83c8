/*
 * fathom.h — C ABI of the B200 (sm_100a) implementation of Fathom's decode-step hot path:
 * bit-plane key store, per-query depth allocation, variable-depth bit-plane scan, top-k
 * selection and exact attention over the selected rows.
 *
 * Conventions shared by every call
 * --------------------------------
 *  - Shapes: Hkv KV heads, Hq query heads, G = Hq / Hkv query heads per KV head (query head h
 *    reads KV head h / G), d = 128 channels, n tokens, nb = ceil(n / 64) blocks of 64 tokens.
 *  - Every data pointer is a DEVICE pointer unless the argument says otherwise.  `planes` and
 *    `scales` may instead point to pinned host memory that the device can address (the paper's
 *    host-resident store, Sec. 3.6): the scan then reads it directly over the host link.
 *  - All buffers are allocated and owned by the caller.  The library allocates only the scratch
 *    arena and one status word when a context is created, and frees them when it is destroyed.
 *  - The five data-path calls only ENQUEUE work on `stream` (a cudaStream_t passed as void*;
 *    NULL = the legacy default stream).  None of them synchronises; results (`depth`, `scores`,
 *    `idx`) stay on the device and feed the next call, so a decode step needs no host round trip
 *    (Sec. 3.6 and Sec. 6, ablation A6: fixed-size plan, no host synchronisation).
 *  - Return value: FATHOM_OK (0) or a negative fathom_status.  Arguments that can be checked on
 *    the host (null pointers, d != 128, strides too small or misaligned, k out of range, scratch
 *    too small) are rejected before anything is launched and leave all outputs untouched.
 *    Conditions only the device can see are recorded in a status word read back with
 *    fathom_device_status(); kernels never trap, assert or wait without a bound.
 *  - Determinism: the same inputs give the same bytes in `planes`, `scales`, `depth`, `idx`,
 *    `scores` and `out` on every run (no floating-point atomics anywhere).
 *  - Inputs must be finite; |k| must stay below 8 * 65504 so that a block scale fits fp16.
 *  - One context may be used by one host thread at a time; calls on different streams that use
 *    the same context share its scratch arena and must not overlap on the device.
 */
#ifndef FATHOM_H_
#define FATHOM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  FATHOM_OK = 0,
  FATHOM_ERR_INVALID_ARG = -1,      /* null pointer, non-positive size, k or budget out of range */
  FATHOM_ERR_UNSUPPORTED = -2,      /* d != 128, heads_per_plan not in {1,2,4,8}, unknown mode/dtype */
  FATHOM_ERR_ALIGNMENT = -3,        /* pointer or stride not aligned as the layout requires */
  FATHOM_ERR_SCRATCH_TOO_SMALL = -4,/* context scratch smaller than fathom_scratch_bytes() for this call */
  FATHOM_ERR_CUDA = -5,             /* a CUDA runtime call failed (see fathom_last_cuda_error) */
  FATHOM_ERR_STATIC_LIMIT = -6      /* problem larger than the built-in scratch of an allocation-free entry point */
} fathom_status;

typedef enum { FATHOM_F32 = 0, FATHOM_BF16 = 1 } fathom_dtype;

typedef enum {
  FATHOM_DEPTH_WATERFILL = 0,       /* reverse water-filling of `budget` bits (Sec. 3.3, Eq. 3-4) */
  FATHOM_DEPTH_FIXED_TOP_R = 1,     /* `budget` = r channels with the largest sum_h |q_j| at depth 4 (Sec. 2, SparQ's grouped rule) */
  FATHOM_DEPTH_UNIFORM = 2          /* every channel at depth `budget` in 0..4 (Sec. 2, thumbnail scans) */
} fathom_depth_mode;

/* Bits of the device status word (fathom_device_status). */
#define FATHOM_DEV_TOPK_SHORT     0x1u  /* top-k found fewer than k eligible tokens (non-finite scores) */
#define FATHOM_DEV_WAIT_EXPIRED   0x2u  /* a bounded device-side wait gave up */

/* One session's store for one layer.  Strides are in elements of the respective array. */
typedef struct {
  int32_t n_kv_heads;          /* Hkv >= 1 */
  int32_t n_q_heads;           /* Hq, a multiple of Hkv */
  int32_t d;                   /* channels per head; must be 128 */
  int32_t reserved;            /* set to 0 */
  int64_t n;                   /* tokens, n >= 1 */
  int64_t plane_stride_words;  /* uint64 words per (KV head, channel, plane) row; >= nb, multiple of 2 (16 B), < 2^24 */
  int64_t scale_stride;        /* fp16 elements per (KV head, channel) row; >= nb, multiple of 8 (16 B), < 2^32 */
  int64_t score_stride;        /* floats per query-head score row; >= n, multiple of 4 (16 B) */
} fathom_layout;

/* Strides that are multiples of 128 bytes (16 words, 64 scales, 32 scores) make every row start on a memory-line boundary;
 * the scan of a host-resident store reaches its best link rate only then (a 128-byte run that straddles two lines costs two
 * requests on the link). */

typedef struct fathom_ctx fathom_ctx;   /* opaque: device id, scratch arena, status word */

/* ---- context ------------------------------------------------------------------------------
 * fathom_create allocates `scratch_bytes` of device memory on `device` (plus a status word) and
 * returns a context in *ctx (host pointer).  fathom_destroy frees both; passing NULL is a no-op.
 * fathom_scratch_bytes returns the scratch a context needs so that every call with this layout
 * and this k succeeds (top-k: histograms, candidate and winner lists; attention: split partials).
 * The paper has no counterpart of these three; they exist so that the data path never allocates. */
int fathom_create(fathom_ctx** ctx, int device, size_t scratch_bytes);
int fathom_destroy(fathom_ctx* ctx);
size_t fathom_scratch_bytes(const fathom_layout* layout, int k);

/* Human-readable text for a fathom_status (static string, never NULL). */
const char* fathom_strerror(int status);
/* Text of the last CUDA error seen by this context (static or context-owned string). */
const char* fathom_last_cuda_error(const fathom_ctx* ctx);
/* Copies the device status word to *status (host pointer) and clears it.  Synchronises `stream`. */
int fathom_device_status(fathom_ctx* ctx, void* stream, uint32_t* status);
/* Self-test of the bounded device-side waits (the paper has no counterpart): enqueues a one-warp kernel in which one
 * thread polls, at most `tries` (1 .. 4096) times, a barrier that nothing will ever complete - no copy or tensor-core
 * operation is outstanding - then sets FATHOM_DEV_WAIT_EXPIRED in the status word and returns.  The kernels that wait
 * on copies or tensor-core work take the same path when a wait runs out; the context stays usable afterwards. */
int fathom_selftest_wait_expiry(fathom_ctx* ctx, int tries, void* stream);
/* Library version, major * 100 + minor. */
int fathom_version(void);

/* ---- (1) plane builder — Sec. 3.2, Eq. 2 and the paragraph that follows it ----------------
 * For every KV head, 64-token block beta and channel j:  a = max_{i in beta, i < n} |k_ij|, the stored
 * scale is s = fp16_round_nearest(a / 8) and the code is c = clip(floor(k / s), -8, 7) + 8 taken with
 * the stored scale (s == 0 gives c = 8).  Bit p (0 = most significant = sign) of the 64 codes is packed
 * into one 64-bit word, token i at bit (i mod 64), absent tail tokens as 0.
 *   K       in   [Hkv][n][d], token-major, k_dtype FATHOM_F32 or FATHOM_BF16, 16-byte aligned
 *   planes  out  [Hkv][d][4][plane_stride_words] uint64; words beta >= nb of a row are not written
 *   scales  out  [Hkv][d][scale_stride] fp16 bit patterns; elements beta >= nb are not written
 * A prefix of t planes of a channel is its t-bit mid-rise quantiser with the same block scale.
 * Appending keys (the paper does not cover it): new tokens can raise the maximum of the last, partly filled
 * block, so that block must be re-quantised; earlier blocks never change.  Call this function on the tail only:
 * per KV head, pass K, planes and scales advanced to block b0 = 8 * (old_block_count / 8) (a multiple of 8 keeps
 * all three pointers 16-byte aligned), n = new_n - 64 * b0, n_kv_heads = 1 and the store's own strides. */
int fathom_build_planes(fathom_ctx* ctx, const fathom_layout* layout, const void* K, int k_dtype,
                        uint64_t* planes, uint16_t* scales, void* stream);

/* ---- (2) depth allocator — Sec. 3.3, Eq. 3 and Eq. 4; Appendix A -------------------------
 * One plan per `heads_per_plan` consecutive query heads (G = the paper's group-shared plan; 1 = one
 * plan per query head).  WATERFILL: g_j = (sum_h q_hj^2) * var_j in fp64; the 4d candidate planes
 * (j, m = 1..4) are ranked by g_j 4^-m (ties: lower channel, then lower plane) and the first
 * min(budget, 4d) are granted; depth_j = planes granted to channel j.  This is Eq. 4 at the smallest
 * water line whose depths fit the budget, evaluated exactly, so sum_j depth_j == min(budget, 4d).
 *   q      in   [Hq][d] fp32          var  in  [Hkv][d] fp32 (unused by the other two modes)
 *   depth  out  [Hq / heads_per_plan][d] uint8, values 0..4 */
int fathom_alloc_depth(fathom_ctx* ctx, const fathom_layout* layout, const float* q, const float* var,
                       int mode, int budget, int heads_per_plan, uint8_t* depth, void* stream);

/* ---- (3) scan — Sec. 3.2 (prefix dequantiser), Sec. 3.3 (inactive channels are skipped) ---
 * For every plan, every query head h of it and every token i < n:
 *   scores[h][i] = sum_{j : depth_j > 0} q_hj * (c_ij >> (4 - t_j) + 1/2 - 2^(t_j - 1)) * (8 s_{beta(i), j}) / 2^(t_j - 1)
 * reading only planes p < t_j and the scales of the active channels; fp32 accumulation; no 1/sqrt(d)
 * factor.  The accumulate runs on the tensor cores: the plane bit becomes the sign of the stored fp16 scale (exact), the
 * query factors are split into two fp16 parts (the precision of an fp32 weight), products are exact in fp32 accumulators
 * and summed in an order that the plan alone fixes, so scores do not depend on the launch geometry.
 * `planes` / `scales` may be device memory or device-addressable pinned host memory (the call asks the
 * runtime which it is: planes in device memory are scanned by persistent CTAs that fetch their next tile ahead, planes
 * in host memory by one CTA per tile in block order, which keeps the requests on the host link sequential).
 * Depth values above 4 are read as 4.
 * Environment: FATHOM_SCAN_PATH=simt (read once per process) selects the earlier CUDA-core kernel (one predicated fp32
 * add per plane bit and head) for every scan; both meet the same tolerance.
 *   scores  out  [Hq][score_stride] fp32; elements i >= n of a row are not written
 * heads_per_plan must be 1, 2, 4 or 8 and divide G. */
int fathom_scan(fathom_ctx* ctx, const fathom_layout* layout, const uint64_t* planes,
                const uint16_t* scales, const float* q, const uint8_t* depth, int heads_per_plan,
                float* scores, void* stream);

/* ---- (3b) the scans of several sessions in one launch — Sec. 4 "Offload harness" (many concurrent sessions) ------
 * Equivalent to one fathom_scan per item (same arguments, bit-identical scores), but all items' tiles form one grid,
 * so that short sessions do not each pay a launch, a ramp-up and a tail - which is what keeps a host link busy when
 * the planes live in pinned host memory.  Every item has its own layout (its n and strides); all items must have
 * the same n_kv_heads and n_q_heads.  items is a HOST array (read during the call); the pointers inside follow the
 * rules of fathom_scan. */
typedef struct fathom_scan_item {
  fathom_layout layout;
  const uint64_t* planes;
  const uint16_t* scales;
  const float* q;
  const uint8_t* depth;
  float* scores;
} fathom_scan_item;
int fathom_scan_batch(fathom_ctx* ctx, const fathom_scan_item* items, int n_items, int heads_per_plan, void* stream);
/* Tuning and test knob, process-wide, no GPU work (the paper has no counterpart): a positive `ctas` fixes the number of
 * CTAs that share a plan's tiles in every later scan launch (each then walks several tiles, also across the sessions of
 * a batch); 0 restores the automatic choice.  Scores never depend on it.  Always returns FATHOM_OK. */
int fathom_scan_set_ctas_per_plan(int ctas);

/* ---- (4) top-k — Sec. 2 "Top-k decoding" ---------------------------------------------------
 * Per query head: the first n_sink and the last n_local tokens are always selected; the remaining
 * k - |forced| are the tokens with the highest scores among the others, ties to the lower token
 * index, -0 equal to +0.  Requires 1 <= k <= n, forced count <= k, k <= FATHOM_MAX_K.
 *   scores  in   [Hq][score_stride] fp32 (finite)
 *   idx     out  [Hq][k] int32, ascending token indices
 * Uses the context scratch (fathom_scratch_bytes).
 * Long rows (at least 64 chunks of 1024 scores, k - forced >= 256) are read once: a histogram of every 16th chunk
 * gives an estimated threshold bin (and a bound: the bin of the sample's own k-th largest score), one pass collects
 * the tokens above the estimate, and the exact selection runs among them, head by head.  A head that collected fewer
 * than it needs is served instead by a second launch, enqueued behind the first, in which the head's CTA collects
 * above the bound and selects; the decision is taken on the device and the result is the same either way.  Shorter
 * rows take two passes (histogram of all scores, filter).
 * Environment: FATHOM_TOPK_PATH=two_pass (read once) always takes the two-pass selection. */
#define FATHOM_MAX_K 16384
int fathom_topk(fathom_ctx* ctx, const fathom_layout* layout, const float* scores, int k,
                int n_sink, int n_local, int32_t* idx, void* stream);
/* How many times fathom_topk reads the scores for these arguments (host only, no GPU work): 1 or 2, or a negative
 * status for arguments fathom_topk would reject. */
int fathom_topk_passes(const fathom_layout* layout, int k, int n_sink, int n_local);

/* ---- (3+4) fused scan and top-k, scores never materialised — Sec. 9 Conclusion (fusing the scan with what follows it) ------
 * Gives exactly the idx that fathom_topk would give on the scores of fathom_scan (same arguments), without writing
 * or re-reading the n * Hq scores: (a) every 16th 1024-token tile is scanned and histogrammed per head (12 leading
 * score-key bits); (b) the full scan keeps only the (score, token) pairs that reach a threshold bin's lower edge;
 * (c) the exact selection (ties to the lower token) runs on those candidates and writes idx.  Two thresholds come
 * from the sample: a BOUND (the bin of the sample's k-th largest score: at least k tokens reach it, so no winner lies
 * below) and an ESTIMATE (the bin of the rank that k tokens of the whole sequence are expected to reach, plus four
 * standard deviations: ~6 times fewer candidates).  The scan runs with the estimate; if any head then holds fewer
 * candidates than it needs, a second scan with the bound, enqueued behind the first, does the work instead - the
 * decision is taken on the device, and the result never depends on how representative the sample is.
 * Sequences too short to sample (fewer than 16 tiles or fewer than 2 k sampled tokens) are scanned into scratch
 * and selected densely.  Uses the context scratch (fathom_scratch_bytes). */
int fathom_scan_topk(fathom_ctx* ctx, const fathom_layout* layout, const uint64_t* planes, const uint16_t* scales,
                     const float* q, const uint8_t* depth, int heads_per_plan, int k, int n_sink, int n_local,
                     int32_t* idx, void* stream);

/* ---- (5) gather + exact attention — Sec. 2 "Top-k decoding" --------------------------------
 * Per query head h with KV head h / G:  out[h] = softmax_i(softmax_scale * q_h . K[idx[h][i]]) . V[idx[h][i]]
 * over its own k selected rows (fp32 arithmetic on rows of `row_dtype`).
 *   Krows, Vrows  in  [Hkv][n][d] FATHOM_BF16 or FATHOM_F32, 16-byte aligned
 *   idx           in  [Hq][k] int32, each in [0, n)        out  [Hq][d] fp32
 * Uses the context scratch (fathom_scratch_bytes). */
int fathom_sparse_attend(fathom_ctx* ctx, const fathom_layout* layout, const float* q,
                         const void* Krows, const void* Vrows, int row_dtype, const int32_t* idx,
                         int k, float softmax_scale, float* out, void* stream);

/* ---- (6) union of a group's winners, fetched once — Sec. 1 and Sec. 4 "Offload harness" ---------
 * The G query heads of a KV head mostly pick overlapping tokens; the offloaded decode step fetches the
 * distinct rows of each KV head once (at most G * k of them) and runs attention on the fetched copy.
 * For every KV head this call forms the ascending list of distinct tokens in idx[kv*G .. kv*G+G-1][*],
 * copies their K and V rows into the staging buffers in that order, and rewrites every pick as its position
 * in the staged rows.  Attention over (K_stage, V_stage, idx_local) with a layout whose n is G * k gives
 * bit for bit what attention over (Krows, Vrows, idx) gives.
 *   idx          in   [Hq][k] int32 (each list without repeats, e.g. from fathom_topk)
 *   Krows, Vrows in   [Hkv][n][d] FATHOM_BF16 or FATHOM_F32, device memory or device-addressable pinned host
 *                     memory (then each distinct row crosses the host link exactly once), 16-byte aligned
 *   K_stage, V_stage out [Hkv][G * k][d] same dtype, device; rows beyond union_count[kv] are not written
 *   idx_local    out  [Hq][k] int32, positions in [0, union_count[kv])
 *   union_count  out  [Hkv] int32
 * Uses the context scratch (fathom_scratch_bytes). */
int fathom_gather_union(fathom_ctx* ctx, const fathom_layout* layout, const int32_t* idx, int k,
                        const void* Krows, const void* Vrows, int row_dtype, void* K_stage, void* V_stage,
                        int32_t* idx_local, int32_t* union_count, void* stream);

/* ---- (7) KLT-rotated store and session calibration — Sec. 3.5 "Basis rule", Appendix B5 --------------
 * On models without QK-norm the paper stores planes of the rotated keys (k - mu) V, V the eigenbasis of the
 * key covariance of the KV head, and ranks channels by g_j = sum_h ((q_h V)_j)^2 lambda_j; nothing else changes
 * (q . k = (q V) . ((k - mu) V) + q . mu, and the last term is the same for every key).  With these three calls
 * the rest of the path is used as is: build planes from K_rot, pass q_rot to fathom_alloc_depth (with the
 * eigenvalues as `var`) and to fathom_scan, and run attention on the original rows.
 *   fathom_calibrate:    mean [Hkv][d] and unbiased covariance cov [Hkv][d][d] (fp32) of the session's own keys in ONE
 *                        read of the keys: the keys are centred on a shift (the mean of 64 keys spread over the sequence),
 *                        sum (x - shift)(x - shift)^T is accumulated on the tensor cores (tf32 operands split in head
 *                        and tail, fp32 accumulation per CTA) together with the per-channel sums S, and a reduction
 *                        in fp64 gives mean = shift + S / n, cov = (sum - S S^T / n) / (n - 1); fixed order throughout.
 *                        fathom_klt_basis turns the covariances into bases and eigenvalues.
 *                        Uses the context scratch.  FATHOM_CALIBRATE_PATH=simt: two passes in plain fp32 FMAs.
 *   fathom_rotate_keys:  K_rot [Hkv][n][d] fp32 = (K - mean) basis, basis [Hkv][d][d] row-major with the
 *                        directions in its columns; tensor cores, tf32 operands split in head and tail (three
 *                        products, fp32 accumulation, fixed order); FATHOM_ROTATE_PATH=simt: plain fp32 FMAs.
 *   fathom_rotate_query: q_rot [Hq][d] = q basis[h / G].
 * K is [Hkv][n][d], FATHOM_F32 or FATHOM_BF16, 16-byte aligned, like basis, cov and K_rot. */
int fathom_calibrate(fathom_ctx* ctx, const fathom_layout* layout, const void* K, int k_dtype, float* mean,
                     float* cov, void* stream);
/*   fathom_klt_basis:    basis [Hkv][d][d] (fp32, row-major, directions in its columns) and eigenvalues [Hkv][d] (fp32,
 *                        descending) of cov [Hkv][d][d] (its symmetric part is used): two-sided cyclic Jacobi in fp64, one
 *                        CTA per KV head, rotations accumulated in fp32, fixed order (bit-reproducible); every direction is
 *                        signed so that its largest component is positive.  About 6 ms for 8 KV heads, once per session.  The eigenvalues
 *                        are the `var` of fathom_alloc_depth for the rotated store. */
int fathom_klt_basis(fathom_ctx* ctx, const fathom_layout* layout, const float* cov, float* basis, float* eigenvalues,
                     void* stream);
int fathom_rotate_keys(fathom_ctx* ctx, const fathom_layout* layout, const void* K, int k_dtype,
                       const float* mean, const float* basis, float* K_rot, void* stream);
int fathom_rotate_query(fathom_ctx* ctx, const fathom_layout* layout, const float* q, const float* basis,
                        float* q_rot, void* stream);
/* The rotated store in one call: planes and scales (layout and meaning as fathom_build_planes) of the rotated keys
 * (K - mean) basis, bit for bit what fathom_rotate_keys (tensor-core path) followed by fathom_build_planes produce,
 * without the [Hkv][n][d] fp32 array of rotated keys in between: the accumulator of the rotation is quantised in the
 * kernel's epilogue (block maximum, fp16 scale, plane bits by comparison with multiples of the stored scale, plane
 * words by warp ballots), 256 tokens = one 32-byte sector of every (channel, plane) row at a time.  It trades time
 * for memory: the warp-collective quantiser in the epilogue makes it slower than the two calls (4.2 ms against
 * 1.8 + 0.8 ms at n = 1M, 8 KV heads), but n * Hkv * 512 bytes of intermediate storage are not needed.  Arguments as
 * fathom_rotate_keys and fathom_build_planes; uses the context scratch. */
int fathom_build_planes_rotated(fathom_ctx* ctx, const fathom_layout* layout, const void* K, int k_dtype,
                                const float* mean, const float* basis, uint64_t* planes, uint16_t* scales, void* stream);

/* ---- (8) per-channel key statistics — Sec. 3.3 (the Var(k_j) of g_j), Appendix B5 (from the session's own keys)
 * mean [Hkv][d] and var [Hkv][d] (device, fp32): mean and unbiased (n - 1) sample variance of every channel of
 * K [Hkv][n][d] (device, FATHOM_F32 or FATHOM_BF16, 16-byte aligned).  One pass over the keys; per 1024-token
 * tile fp32 sums of the keys shifted by the tile's middle key, merged across tiles in fp64 in tile order
 * (deterministic).  var feeds fathom_alloc_depth for the raw store.  n = 1 gives var = 0.  Uses the context scratch
 * (FATHOM_ERR_SCRATCH_TOO_SMALL if the context was created for a smaller layout). */
int fathom_channel_variance(fathom_ctx* ctx, const fathom_layout* layout, const void* K, int k_dtype, float* mean,
                            float* var, void* stream);

/* ---- (9) per-layer budgets — Sec. 3.4 "Per-layer budgets" --------------------------------------------------
 * HOST function, no GPU work: the greedy plan that assigns each of n_layers layers one of n_levels budgets
 * (levels[], strictly ascending bits, e.g. 24 .. 128) at a target mean.  err [n_layers][n_levels] (host, row-major)
 * is the caller's measured error of layer l at budget levels[i].  Every layer starts at levels[0]; each step raises
 * one layer by one level, the layer with the largest error drop per added bit (ties: lower layer), while the sum of
 * budgets stays <= target_mean * n_layers.  level_index [n_layers] (host) receives the chosen level per layer; pass
 * levels[level_index[l]] as `budget` to fathom_alloc_depth for layer l.  The paper fixes neither start nor step size;
 * this is the reading taken.  FATHOM_ERR_INVALID_ARG on NULL, non-ascending levels or NaN errors. */
int fathom_plan_layer_budgets(const double* err, int n_layers, int n_levels, const int* levels, double target_mean,
                              int* level_index);

/* ---- (5b) gather + exact attention without any allocation — the paper has no counterpart ------
 * Same computation, arguments and results as fathom_sparse_attend, for callers that cannot obtain device
 * memory of their own: a plug-in that is only handed buffers by its host application, a serving process
 * whose memory pool already owns the whole GPU (cudaMalloc would fail there), or a decode loop that must
 * not pay the device-wide synchronisation an allocation or a free can imply.  It needs no fathom_ctx and
 * calls neither cudaMalloc nor cudaFree nor any allocating library routine: the per-chunk softmax partials
 * live in an array that is compiled into the library (about 1 MB of device memory on every GPU that loads
 * the library, held until the process exits).
 *   Limit: n_q_heads * ceil(k / 128) <= FATHOM_ATTEND_STATIC_MAX_CHUNKS, otherwise FATHOM_ERR_STATIC_LIMIT
 *   is returned and nothing is launched (32 query heads allow k <= 8192).
 *   First use on a device: the call looks up the device address of the built-in array once per device
 *   (cudaGetSymbolAddress, with the stream's device current — make it current before calling).  Make this
 *   first call before any stream capture begins; later calls on that device only enqueue one kernel.
 *   Sharing: every call on a device uses the same array, which keeps the previous call's contents.  Each
 *   call overwrites every element it later reads and re-arms its ticket counters, so nothing needs clearing, but two calls that may overlap
 *   on the device (different streams, no dependency) race on it and must be ordered by the caller. */
#define FATHOM_ATTEND_STATIC_MAX_CHUNKS 2048
int fathom_sparse_attend_static(const fathom_layout* layout, const float* q, const void* Krows,
                                const void* Vrows, int row_dtype, const int32_t* idx, int k,
                                float softmax_scale, float* out, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* FATHOM_H_ */
