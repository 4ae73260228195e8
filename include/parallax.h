/*
 * parallax.h -- C ABI of the B200 (sm_100a) Parallax decode-forward library.
 *
 * What it computes (Sec. 3.1, Eq. "parallax_forward"; streamed as in Sec. 3.3,
 * Eq. "parallax_expand" and Algorithm 1): for every sequence b and query head hq,
 * with p_j = softmax_j(scale * q.k_j) over the first seqlens[b] cached keys of KV
 * head hkv = hq / (Hq/Hkv), t_j = r.k_j (NOT scaled) and tbar = sum_j p_j t_j,
 *
 *     out[b,hq,:] = sum_j p_j (1 + tbar - t_j) v_j
 *                 = (sum p v)(1 + sum p t) - sum (p t) v .
 *
 * The context is read once.  Long or few contexts are cut into key chunks
 * ("splits"); each split leaves an unnormalised partial state and a combine
 * kernel merges them (App. "Kernel Optimization Details", items 2 and 3).
 *
 * Conventions for every entry point
 *   - Pointers named *_host are HOST pointers; all other data pointers are DEVICE
 *     pointers owned by the caller.  The library never allocates or frees device
 *     memory and never synchronises, except where an entry point says otherwise.
 *   - Work is enqueued on `stream` (a cudaStream_t passed as an opaque pointer;
 *     NULL = the legacy default stream) and the call returns at once.
 *   - Return value: PLX_OK (0) or a negative PLX_ERR_* code; on error nothing has
 *     been launched.
 *   - Layouts are row-major and contiguous:
 *         q, r              bf16 [B, Hq, D]          one query token per sequence;
 *                                                    r is the probe rho, already
 *                                                    normalised/rotated upstream
 *         k_cache, v_cache  bf16 [B, Hkv, T_max, D]
 *         seqlens           int32 [B], valid keys per sequence (clamped to
 *                           [0, T_max]); NULL means T_max for every sequence.
 *                           K/V rows at positions >= seqlens[b] are never read into
 *                           the result and may hold anything, NaN included.
 *         out               [B, Hq, D], bf16 (round-to-nearest-even) or fp32
 *     seqlens[b] == 0 gives a row of zeros.  The new token's own key and value are
 *     expected to be in the cache already and counted by seqlens.
 *   - Supported shapes: D in {64, 128}; Hq a multiple of Hkv with group size
 *     Hq/Hkv from 1 to 64 (up to eight query heads of a KV head are served by one CTA;
 *     larger groups by several CTAs per KV head, or -- parallax_decode_fwd_ex,
 *     parallax_decode_fwd_paged and parallax_decode_step route them by measured crossover,
 *     at D = 128 from five heads per KV head on -- by the tensor-core kernels,
 *     see parallax_decode_fwd_multi, which also lifts the limit of 64); q, r, out 4-byte
 *     aligned; k_cache, v_cache 16-byte aligned; workspace 16-byte aligned.
 *   - Launch ordering: the decode kernels are launched with the programmatic stream
 *     serialisation attribute (they wait, before they touch memory, for the kernel
 *     before them in the stream) and signal their own dependents early, so that
 *     back-to-back decode calls overlap a call's launch with its predecessor's tail.
 *     For a kernel launched the ordinary way after a call nothing changes: it starts
 *     when the call's kernels have completed.  A kernel that the CALLER launches as
 *     a programmatic dependent after a decode call may be scheduled before that
 *     call has completed and has to execute cudaGridDependencySynchronize() before
 *     it touches the call's output, as that launch mode requires of any kernel.
 *   - Thread safety: entry points may be called from several host threads;
 *     parallax_set_layout / parallax_decode_fwd share one process-wide default.
 */
#ifndef PARALLAX_H_
#define PARALLAX_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define PLX_OK 0
#define PLX_ERR_NULL_POINTER (-1)
#define PLX_ERR_BAD_SHAPE (-2)
#define PLX_ERR_UNSUPPORTED (-3)
#define PLX_ERR_ALIGNMENT (-4)
#define PLX_ERR_WORKSPACE (-5)
#define PLX_ERR_NEED_LAYOUT (-6)
#define PLX_ERR_CUDA (-7)
#define PLX_ERR_DEVICE_TIMEOUT (-8)
#define PLX_ERR_STATIC_SCRATCH (-9)
#define PLX_ERR_DEVICE_CHECK (-10) /* debug build only (PLX_DEBUG_CHECKS): a kernel refused an out-of-range index */

#define PLX_OUT_BF16 0
#define PLX_OUT_F32 1

/* Precision of the softmax weights P1, P2 on their way into the value product (prefill entry point). */
#define PLX_P_BF16_RESIDUAL 0 /* bf16 plus its bf16 rounding residual: fp32-class result (default) */
#define PLX_P_BF16 1          /* plain bf16: faster, relative error ~2^-9 * sqrt(D) on rows with few keys */
/* residuals only in the 128-row tiles in which some row sees fewer than PLX_P_ADAPTIVE_MIN_KEYS keys, plain
 * bf16 weights elsewhere: the few-key rows (where the two branches' cancellation amplifies the weights'
 * rounding) keep the fp32-class result, rows that average over a thousand keys or more get the precision of a
 * bf16 tensor-core attention kernel (relative RMS error ~1.6e-3, the level of a bf16 output's own rounding),
 * and a long prefill executes about 1.03 instead of 1.5 times its algorithmic tensor work */
#define PLX_P_BF16_ADAPTIVE 2
#define PLX_P_ADAPTIVE_MIN_KEYS 1024

/* Largest split count any entry point accepts. */
#define PLX_MAX_SPLITS 1024

/* Library version as major*10000 + minor*100 + patch. */
int parallax_version(void);

/* Static, human-readable text for a status code. */
const char* parallax_status_string(int status);

/*
 * Partial-state record format (App. "Kernel Optimization Details", item 3: the
 * unnormalised partials (m, d1, d2, O1, O2) kept in a small fp32 workspace).
 * One record per (b, hq, split), `parallax_partial_stride(D)` = 2*D + 4 floats:
 *     [0] m   reference exponent in natural-log units of scale*q.k; every other
 *             field is relative to it (m is at most the split's true maximum logit
 *             and within 8*ln2 of it); -inf marks an empty split
 *     [1] d1 = sum_j exp(s_j - m)          [2] d2 = sum_j exp(s_j - m) t_j
 *     [3] unused
 *     [4 .. 4+D)      O1 = sum_j exp(s_j - m) v_j
 *     [4+D .. 4+2D)   O2 = sum_j exp(s_j - m) t_j v_j
 * Records are stored as [B, Hq, num_splits, stride].
 */
int parallax_partial_stride(int D);

/*
 * Bytes of workspace that parallax_decode_fwd_ex / _host need for up to
 * `max_splits` splits: a 256-byte header (device status word), one arrival counter
 * per (b, hq), staging for q, r and out (host-buffer entry point) and the partial
 * records.  Pure host function.  Returns 0 on invalid arguments.
 */
size_t parallax_decode_workspace_bytes(int B, int Hq, int D, int max_splits);

/*
 * The split plan the library would choose (App. "Kernel Optimization Details",
 * item 2: splits sized to the device's wave).  Pure host function: depends only
 * on the shape, `num_sms` and whether a seqlens array will be passed (never on
 * its contents, which live on the device; with unequal contexts finer chunks
 * balance better).
 * chunk_len is a multiple of 64 keys; num_splits = ceil(T_max / chunk_len).
 */
int parallax_decode_plan(int B, int Hq, int Hkv, int D, int T_max, int num_sms, int has_seqlens,
                         int* chunk_len, int* num_splits);

/*
 * Full decode forward with every option explicit (Algorithm 1 with one query row
 * per head, plus split and merge).
 *   T_max            cache stride in keys (second-to-last dimension of the caches)
 *   out_dtype        PLX_OUT_BF16 or PLX_OUT_F32
 *   workspace        device memory of at least
 *                    parallax_decode_workspace_bytes(B, Hq, D, splits used);
 *                    may be NULL only when the call resolves to one split.
 *                    Zero it once before first use (cudaMemset); every call leaves
 *                    the words it relies on (status, the item ticket of the
 *                    multi-token kernel, arrival counters) zero again.
 *                    Zero it again after a call that failed on the device.  Calls
 *                    that overlap on the GPU must not share a workspace.
 *   num_splits       0 = let the library plan; otherwise the number of key chunks
 *                    (1..PLX_MAX_SPLITS); the chunk length is T_max/num_splits
 *                    rounded up to a multiple of 64 keys.
 * One launch: with several splits every CTA leaves its partial record in the
 * workspace and the last CTA of a (sequence, KV head) to arrive merges them in
 * split order (App. "Kernel Optimization Details", item 3), so the result does
 * not depend on the arrival order.
 */
int parallax_decode_fwd_ex(const void* q, const void* r, const void* k_cache, const void* v_cache,
                           const int32_t* seqlens, void* out, int B, int Hq, int Hkv, int D,
                           int T_max, float scale, int out_dtype, void* workspace,
                           size_t workspace_bytes, int num_splits, void* stream);

/*
 * Decode forward over a PAGED KV cache (serving layout; the paper does not fix a cache layout).
 * Same computation, options and workspace rules as parallax_decode_fwd_ex, but the keys and
 * values of sequence b live in pages:
 *     k_pages, v_pages  bf16 [num_pages, Hkv, page_size, D]  (the page pools)
 *     block_table       int32 [B, max_pages_per_seq]: page id of logical page i of sequence b;
 *                       entries past ceil(seqlens[b] / page_size) are never read
 * Key j of sequence b is row j % page_size of page block_table[b][j / page_size].
 * page_size must be a multiple of 16 (64 or more keeps the page lookup off the load path);
 * seqlens[b] <= max_pages_per_seq * page_size (NULL = that maximum for every sequence).
 */
int parallax_decode_fwd_paged(const void* q, const void* r, const void* k_pages, const void* v_pages,
                              const int32_t* block_table, const int32_t* seqlens, void* out, int B,
                              int Hq, int Hkv, int D, int num_pages, int page_size,
                              int max_pages_per_seq, float scale, int out_dtype, void* workspace,
                              size_t workspace_bytes, int num_splits, void* stream);

/*
 * Process-wide defaults for the short form below: cache stride, output type and
 * workspace.  Host-only; returns PLX_ERR_* on invalid values.
 */
int parallax_set_layout(int T_max, int out_dtype, void* workspace, size_t workspace_bytes);

/*
 * Short form: same as parallax_decode_fwd_ex with T_max, out_dtype and workspace
 * taken from parallax_set_layout and num_splits = 0 (planned).  Returns
 * PLX_ERR_NEED_LAYOUT if no layout has been set.
 */
int parallax_decode_fwd(const void* q, const void* r, const void* k_cache, const void* v_cache,
                        const int32_t* seqlens, void* out, int B, int Hq, int Hkv, int D,
                        float scale, void* stream);

/*
 * Split-KV main kernel alone: stops after writing the partial state of every
 * (b, hq, split) to `partials` ([B, Hq, num_splits, stride] fp32, device).  Splits
 * that start at or beyond seqlens[b] get an empty record (m = -inf, rest zero).
 * Key chunk `split` covers keys [split*chunk_len, (split+1)*chunk_len); chunk_len
 * must be a positive multiple of 16 and num_splits*chunk_len >= T_max.
 * `status` is an optional device int32 that the kernel sets non-zero if one of its
 * bounded waits ran out (NULL = not recorded).
 */
int parallax_decode_splitkv_partial(const void* q, const void* r, const void* k_cache,
                                    const void* v_cache, const int32_t* seqlens, float* partials,
                                    int B, int Hq, int Hkv, int D, int T_max, float scale,
                                    int chunk_len, int num_splits, int32_t* status, void* stream);

/*
 * Split-KV combine (App. "Kernel Optimization Details", item 3: log-sum-exp
 * rescaling of the partials, then Algorithm 1's final line
 * O1/d1 * (1 + d2/d1) - O2/d1).  Merges, for every (b, hq), the first
 * split_counts[b] records (all num_splits when split_counts is NULL; device
 * int32 [B]) in split order, skipping records whose m is -inf.  A row with no
 * non-empty record is written as zeros.  The merge order is fixed, so results are
 * bitwise repeatable.  Also usable to merge partial states gathered from several
 * GPUs that each hold a slice of one context.
 */
int parallax_decode_combine(const float* partials, const int32_t* split_counts, void* out, int B,
                            int Hq, int D, int num_splits, int out_dtype, void* stream);

/*
 * Combine for a context whose keys are sharded over several GPUs (one exchange step: every rank
 * runs parallax_decode_splitkv_partial on its slice of each sequence, the records are all-gathered,
 * then every rank merges locally; App. "Kernel Optimization Details", item 3 applied across devices).
 * `partials` is the gathered buffer [num_ranks, B, Hq, num_splits, stride] in THIS GPU's memory
 * (exactly what an all-gather of the per-rank [B, Hq, num_splits, stride] buffers produces); all
 * num_ranks * num_splits (<= PLX_MAX_SPLITS) records of a row are merged in rank-major order, empty
 * records (m = -inf) are skipped, a row with none gives zeros.
 */
int parallax_decode_combine_gathered(const float* partials, void* out, int B, int Hq, int D,
                                     int num_ranks, int num_splits, int out_dtype, void* stream);

/*
 * End-to-end step with HOST buffers for the per-step tensors: copies q_host and
 * r_host (bf16 [B,Hq,D], ideally pinned) to staging inside `workspace`, runs
 * parallax_decode_fwd_ex on the device-resident caches, copies the result to
 * out_host, and SYNCHRONISES `stream` before returning.  The KV cache and seqlens
 * stay device pointers: the cache is resident state of a decode step, not a
 * per-step input.  Page-locked (device-mapped) host memory takes a shorter route:
 * the attention kernel reads q_host and r_host itself (16-byte aligned buffers:
 * every CTA fetches its own rows over the host link into shared memory, so the
 * transfer of later CTAs' rows overlaps the streaming of the earlier ones) and
 * writes out_host itself, so the step is ONE launch with no copy command at all;
 * pageable memory is staged with copy commands.  The result is the same bits
 * either way.
 */
int parallax_decode_fwd_host(const void* q_host, const void* r_host, const void* k_cache,
                             const void* v_cache, const int32_t* seqlens, void* out_host, int B,
                             int Hq, int Hkv, int D, int T_max, float scale, int out_dtype,
                             void* workspace, size_t workspace_bytes, int num_splits, void* stream);

/*
 * Reads the device status word in the workspace header into *status_host
 * (0 = no device-side wait ever ran out).  Synchronises `stream`.
 */
int parallax_workspace_status(const void* workspace, int32_t* status_host, void* stream);

/*
 * Multi-token causal forward: Algorithm 1 with a tile of query rows (prefill, chunked
 * prefill, or several new tokens per decode step).  q, r and out are [B, Hq, Lq, D];
 * the Lq tokens of sequence b are the LAST Lq positions of its context of
 * seqlens[b] keys (NULL = T_max), whose keys and values are already in the caches.
 * Token i attends to keys 0 .. seqlens[b] - Lq + i (the sum over j <= i of
 * Eq. "parallax_forward"); a token with no visible key gives a row of zeros.
 * Lq = 1 computes what parallax_decode_fwd_ex computes.
 * Supported: D in {64, 128}, any Hq multiple of Hkv; all tensors 16-byte aligned.
 * p_precision: PLX_P_BF16_RESIDUAL keeps the decode path's accuracy (the weights reach the value
 * product as bf16 plus residual, at the price of two extra MMAs per tile); PLX_P_BF16 sends plain
 * bf16 weights, the precision of a conventional bf16 attention kernel; PLX_P_BF16_ADAPTIVE keeps the
 * residual products only in the row tiles in which some row sees fewer than PLX_P_ADAPTIVE_MIN_KEYS keys
 * (two launches: the plain build and the residual build, each over its own tiles).
 * `status` is an optional device int32 set non-zero if a bounded device-side wait
 * ran out (NULL = not recorded).  One launch, no workspace.
 */
int parallax_prefill_fwd(const void* q, const void* r, const void* k_cache, const void* v_cache,
                         const int32_t* seqlens, void* out, int B, int Hq, int Hkv, int D, int Lq,
                         int T_max, float scale, int out_dtype, int p_precision, int32_t* status,
                         void* stream);

/*
 * Decode forward over an fp8 (e4m3) KV cache, a serving variant that halves the bytes the step has
 * to read (the paper's kernels use 16-bit caches; the arithmetic of Algorithm 1 is unchanged).
 * k_cache, v_cache: e4m3 bytes [B, Hkv, T_max, D] holding k / k_scale and v / v_scale (one positive
 * scale per tensor); q, r, out, seqlens, workspace, num_splits as in parallax_decode_fwd_ex.  The
 * result is the Parallax output for the dequantised cache (k_scale * k8, v_scale * v8): e4m3 converts
 * exactly to fp16, the products run as fp16 x fp16 -> fp32 MMAs (q and r are converted bf16 -> fp16:
 * exact for magnitudes in [6.1e-5, 65504]), the weights reach the value product as fp16 plus fp16
 * residual.  D in {64, 128} (at D = 64 the rows are 64 bytes: the compute-matched shape of Sec. 3.3
 * "Profiling Result"); up to eight heads per KV head are served by one CTA, as with a 16-bit cache.
 * PLX_ERR_BAD_SHAPE if a scale is not a
 * positive finite number.
 */
int parallax_decode_fwd_fp8(const void* q, const void* r, const void* k_cache, const void* v_cache,
                            const int32_t* seqlens, void* out, int B, int Hq, int Hkv, int D, int T_max,
                            float scale, float k_scale, float v_scale, int out_dtype, void* workspace,
                            size_t workspace_bytes, int num_splits, void* stream);

/*
 * parallax_prefill_fwd with split-KV, for short chunks on few sequences (chunked prefill or a draft of
 * a few dozen tokens at batch 1..8, where one CTA per 128-row tile would leave most SMs idle): the key
 * tiles of every row tile are divided among num_splits CTAs (0 = planned: about one CTA per SM, at
 * least 512 keys per split, one split when the tiles alone fill the device), each writes its rows'
 * unnormalised state (m, d1, d2, O1, O2: the record format of parallax_decode_splitkv_partial) to
 * `workspace`, and the merge kernel of the decode path finishes the rows (a second launch, only when
 * there is more than one split).  workspace: caller-owned device memory, 16-byte aligned, of
 * parallax_prefill_workspace_bytes(B, Hq, D, Lq, max_splits) bytes = B*Hq*Lq*max_splits*(2D+4)*4; a
 * smaller one lowers the split count, NULL means one split.  Everything else as parallax_prefill_fwd.
 */
size_t parallax_prefill_workspace_bytes(int B, int Hq, int D, int Lq, int max_splits);
int parallax_prefill_fwd_ex(const void* q, const void* r, const void* k_cache, const void* v_cache,
                            const int32_t* seqlens, void* out, int B, int Hq, int Hkv, int D, int Lq,
                            int T_max, float scale, int out_dtype, int p_precision, void* workspace,
                            size_t workspace_bytes, int num_splits, int32_t* status, void* stream);

/*
 * parallax_prefill_fwd over a PAGED cache (chunked prefill in a serving engine): k_pages, v_pages
 * bf16 [num_pages, Hkv, page_size, D]; block_table int32 [B, max_pages_per_seq] device array whose
 * entry (b, i) is the page holding keys i*page_size .. of sequence b (only the pages below
 * ceil(seqlens[b] / page_size) are read).  page_size must be a multiple of 64 (a 64-key tile never
 * straddles a page); the context capacity is page_size * max_pages_per_seq; seqlens is required in
 * practice (NULL = every sequence fills its capacity).  Everything else as parallax_prefill_fwd.
 */
int parallax_prefill_fwd_paged(const void* q, const void* r, const void* k_pages, const void* v_pages,
                               const int32_t* block_table, const int32_t* seqlens, void* out, int B,
                               int Hq, int Hkv, int D, int Lq, int num_pages, int page_size,
                               int max_pages_per_seq, float scale, int out_dtype, int p_precision,
                               int32_t* status, void* stream);

/*
 * parallax_prefill_fwd_paged with the split-KV of parallax_prefill_fwd_ex (a short chunk of few
 * sequences over a paged cache, the common shape of chunked prefill in a serving engine): arguments of
 * the former, then workspace, workspace_bytes and num_splits as in the latter.
 */
int parallax_prefill_fwd_paged_ex(const void* q, const void* r, const void* k_pages, const void* v_pages,
                                  const int32_t* block_table, const int32_t* seqlens, void* out, int B,
                                  int Hq, int Hkv, int D, int Lq, int num_pages, int page_size,
                                  int max_pages_per_seq, float scale, int out_dtype, int p_precision,
                                  void* workspace, size_t workspace_bytes, int num_splits,
                                  int32_t* status, void* stream);

/*
 * parallax_decode_fwd_fp8 over a PAGED e4m3 cache: k_pages, v_pages e4m3 bytes
 * [num_pages, Hkv, page_size, D] with the block table of parallax_decode_fwd_paged (page_size a
 * multiple of 16) and the per-tensor scales of parallax_decode_fwd_fp8.  D must be 128.
 */
int parallax_decode_fwd_paged_fp8(const void* q, const void* r, const void* k_pages, const void* v_pages,
                                  const int32_t* block_table, const int32_t* seqlens, void* out, int B,
                                  int Hq, int Hkv, int D, int num_pages, int page_size,
                                  int max_pages_per_seq, float scale, float k_scale, float v_scale,
                                  int out_dtype, void* workspace, size_t workspace_bytes, int num_splits,
                                  void* stream);

/*
 * Decode step with SEVERAL new tokens per sequence (speculative decoding, multi-token prediction,
 * a short chunk of a chunked prefill): what parallax_prefill_fwd computes, on the decode kernel.
 * q, r and out are [B, Hq, Lq, D]; the Lq tokens of sequence b are the LAST Lq positions of its
 * context of seqlens[b] keys (NULL = T_max), already in the caches; token i attends to keys
 * 0 .. seqlens[b] - Lq + i, a token with no visible key gives a row of zeros.  The Lq tokens of a
 * query head are handled like Lq more query heads of its KV head (split-KV, fused merge and the
 * bandwidth-bound streaming of the decode kernel apply), so the call is HBM-bound where the
 * tensor-core multi-token kernel would compute a 128-row tile for a handful of rows.  That holds up
 * to eight rows per KV head (Lq * Hq / Hkv <= 8, one CTA per KV head; four at D = 128).  Nine (five) to 64 rows run
 * on the tensor-core kernel of parallax_decode_fwd_rows (keys on the accumulator lanes; 33 to 64 rows at D = 64
 * only for contexts of at least 4096 keys on many sequences), larger steps
 * on parallax_prefill_fwd_ex (residual weights); both keep their split records in the same
 * workspace, so the call accepts any Lq.  (Steps of 9..64 rows whose q, r or out is not 16-byte
 * aligned stay on the decode kernel; parallax_decode_fwd_args always does.)  Workspace as parallax_decode_fwd_ex for Hq * Lq
 * query heads (parallax_decode_workspace_bytes(B, Hq * Lq, D, max_splits)); everything else as there.
 * With a workspace, a step on that kernel with more (sequence, KV head, split) items
 * than SMs runs one CTA per SM that draws its items from a word of the workspace's header (zero
 * between calls, like the status word); without one it runs one CTA per item.
 */
int parallax_decode_fwd_multi(const void* q, const void* r, const void* k_cache, const void* v_cache,
                              const int32_t* seqlens, void* out, int B, int Hq, int Hkv, int D, int Lq,
                              int T_max, float scale, int out_dtype, void* workspace,
                              size_t workspace_bytes, int num_splits, void* stream);

/*
 * The same step on the tensor-core kernel that keeps the KEYS on the accumulator lanes (Algorithm 1 with
 * S^T = K_c [Q; R]^T per 128-key tile and O^T += V_c^T P^T, so the tensor work follows the rows present):
 * up to 64 rows per KV head (Lq * Hq / Hkv <= 64; more than 32 are worked as two halves that share their K/V
 * through L2), D = 64 or 128, bf16 caches, contiguous layout; q, r, k_cache,
 * v_cache, out 16-byte aligned.  Split-KV like parallax_prefill_fwd_ex: `workspace` holds split records only
 * (parallax_prefill_workspace_bytes(B, Hq, D, Lq, max_splits) bytes, 16-byte aligned; NULL = one split),
 * num_splits 0 = planned (fewer items than SMs: about one CTA per SM, at least four 128-key tiles per split; more:
 * the count a model of the step's time prefers, often 1), records merged by the decode path's merge kernels on
 * the same stream.  `status` (device int32, may be NULL) receives
 * PLX_ERR_DEVICE_TIMEOUT if a bounded device-side wait runs out.  PLX_ERR_UNSUPPORTED for other shapes.
 * parallax_decode_fwd_multi chooses this kernel by itself (parallax_decode_fwd_multi_paged too, over paged
 * caches); this entry forces it.  Arguments, token order and causal rule as parallax_decode_fwd_multi.  One or
 * two launches on `stream`; argument errors are returned before anything is launched.
 */
int parallax_decode_fwd_rows(const void* q, const void* r, const void* k_cache, const void* v_cache,
                             const int32_t* seqlens, void* out, int B, int Hq, int Hkv, int D, int Lq,
                             int T_max, float scale, int out_dtype, void* workspace, size_t workspace_bytes,
                             int num_splits, int32_t* status, void* stream);

/*
 * Which kernel parallax_decode_fwd_multi (page_size = 0) or parallax_decode_fwd_multi_paged would run for a step
 * of this shape, given 16-byte aligned tensors and a workspace with room for split records, and, for the
 * keys-on-lanes kernel, the split count it would plan for num_splits = 0 (1 = no merge launch; 0 is reported for
 * the other kernels).  Host only: nothing is launched, no pointer is needed.  For callers that account for
 * launches or want to log the route; the numbers follow the device the calling thread has current.
 */
#define PLX_MULTI_KERNEL_DECODE 0    /* the decode kernel: up to eight rows per KV head (four at D = 128) */
#define PLX_MULTI_KERNEL_ROWS 1      /* the keys-on-lanes tensor-core kernel: up to 64 rows per KV head */
#define PLX_MULTI_KERNEL_ROW_MAJOR 2 /* the row-major split-KV tensor-core kernel */
int parallax_decode_multi_plan(int B, int Hq, int Hkv, int D, int Lq, int T_max, int page_size, int* kernel,
                               int* num_splits);

/* parallax_decode_fwd_multi over the paged cache of parallax_decode_fwd_paged (q, r, out [B, Hq, Lq, D]);
 * the hand-over to the keys-on-lanes kernel needs a page_size that divides 128 or is a multiple of it,
 * the hand-over to the row-major tensor-core kernel a multiple of 64. */
int parallax_decode_fwd_multi_paged(const void* q, const void* r, const void* k_pages, const void* v_pages,
                                    const int32_t* block_table, const int32_t* seqlens, void* out, int B,
                                    int Hq, int Hkv, int D, int Lq, int num_pages, int page_size,
                                    int max_pages_per_seq, float scale, int out_dtype, void* workspace,
                                    size_t workspace_bytes, int num_splits, void* stream);

/*
 * Every option of the decode forward in one call, for combinations the entry points above do not name
 * (e.g. several new tokens over a paged e4m3 cache with per-head scales).  Fill a parallax_decode_args
 * with zeros, set struct_bytes = sizeof(parallax_decode_args) (a library built from a later header
 * accepts a shorter struct and treats the missing tail as zeros) and the fields that apply:
 *   q, r, out          [B, Hq, D], or [B, Hq, Lq, D] when Lq > 1 (Lq = 0 or 1: one token)
 *   k_cache, v_cache   contiguous [B, Hkv, T_max, D] (block_table NULL), or page pools
 *                      [num_pages, Hkv, page_size, D] with block_table [B, max_pages_per_seq]
 *                      (then T_max is ignored: the capacity is page_size * max_pages_per_seq)
 *   kv_dtype           PLX_KV_BF16 or PLX_KV_E4M3; for e4m3 either the scalars k_scale,
 *                      v_scale or the device arrays k_scales, v_scales [Hkv] (both non-NULL)
 *   seqlens, scale, out_dtype, workspace, workspace_bytes, num_splits, stream: as parallax_decode_fwd_ex
 *                      (workspace sized for Hq * Lq query heads)
 * Same kernel, same results, same error codes as the specific entry points; PLX_ERR_BAD_SHAPE for a
 * struct_bytes the library cannot read.
 */
#define PLX_KV_BF16 0
#define PLX_KV_E4M3 1
typedef struct parallax_decode_args {
    size_t struct_bytes;
    const void* q;
    const void* r;
    const void* k_cache;
    const void* v_cache;
    const int32_t* seqlens;
    void* out;
    int B, Hq, Hkv, D, Lq, T_max;
    float scale;
    int out_dtype;
    int kv_dtype;
    float k_scale, v_scale;
    const float* k_scales;
    const float* v_scales;
    const int32_t* block_table;
    int num_pages, page_size, max_pages_per_seq;
    int num_splits;
    void* workspace;
    size_t workspace_bytes;
    void* stream;
} parallax_decode_args;
int parallax_decode_fwd_args(const parallax_decode_args* args);

/*
 * The two e4m3 entry points with one scale PER KV HEAD (the usual granularity of a serving engine's
 * quantised cache): head h of the cache holds k / k_scales[h] and v / v_scales[h].  k_scales and
 * v_scales are DEVICE arrays of Hkv fp32 values, positive and finite (not checked: they are read by
 * the kernel, one pair per CTA); everything else as parallax_decode_fwd_fp8 /
 * parallax_decode_fwd_paged_fp8.  The scales never touch the tiles: k_scales[h] multiplies the two
 * score rows of head h, v_scales[h] its two accumulators once, before the split records are written.
 */
int parallax_decode_fwd_fp8_per_head(const void* q, const void* r, const void* k_cache,
                                     const void* v_cache, const int32_t* seqlens, void* out, int B,
                                     int Hq, int Hkv, int D, int T_max, float scale,
                                     const float* k_scales, const float* v_scales, int out_dtype,
                                     void* workspace, size_t workspace_bytes, int num_splits,
                                     void* stream);
int parallax_decode_fwd_paged_fp8_per_head(const void* q, const void* r, const void* k_pages,
                                           const void* v_pages, const int32_t* block_table,
                                           const int32_t* seqlens, void* out, int B, int Hq, int Hkv,
                                           int D, int num_pages, int page_size, int max_pages_per_seq,
                                           float scale, const float* k_scales, const float* v_scales,
                                           int out_dtype, void* workspace, size_t workspace_bytes,
                                           int num_splits, void* stream);

/*
 * Training forward: parallax_prefill_fwd that also writes the per-row state the backward needs
 * (App. "Parallax Backward": the forward caches o, vbar, tbar, omega and m per row):
 *     lse  [B, Hq, Lq] fp32   m_i + log(omega_i), natural-log units; +inf for a row that sees no key
 *     tbar [B, Hq, Lq] fp32   softmax-weighted mean of the probe scores rho_i . k_j (0 without keys)
 *     vbar [B, Hq, Lq, D]     softmax-weighted mean of the values, in out's dtype (0 without keys)
 * All three are required (non-NULL, vbar 16-byte aligned).  Same launch as parallax_prefill_fwd.
 */
int parallax_prefill_fwd_save(const void* q, const void* r, const void* k_cache, const void* v_cache,
                              const int32_t* seqlens, void* out, float* lse, float* tbar, void* vbar,
                              int B, int Hq, int Hkv, int D, int Lq, int T_max, float scale,
                              int out_dtype, int p_precision, int32_t* status, void* stream);

/* Bytes of device workspace parallax_prefill_bwd needs: one 16-byte record per query row plus 64. */
size_t parallax_prefill_bwd_workspace_bytes(int B, int Hq, int Lq);

/*
 * Backward of parallax_prefill_fwd_save (App. "Parallax Backward", Eq. "bwd_projections",
 * "bwd_dq", "bwd_dr", "bwd_dk", "bwd_dv").  With p_ij the softmax weight, t_ij = rho_i . k_j,
 *     tau_i = dO_i . o_i, beta_i = dO_i . vbar_i, a_ij = dO_i . v_j, delta_ij = a_ij - beta_i,
 *     g1_ij = p_ij [a_ij - tau_i + (tbar_i - t_ij) delta_ij],   g2_ij = -p_ij delta_ij,
 *     dq_i = scale sum_j g1_ij k_j              dr_i = sum_j g2_ij k_j
 *     dk_j = scale sum_i g1_ij q_i + sum_i g2_ij rho_i      dv_j = sum_i p_ij (1 + tbar_i - t_ij) dO_i
 * (i over the rows that see key j, of every query head that shares the KV head).
 * Inputs: q, r, dout bf16 [B,Hq,Lq,D]; k_cache, v_cache bf16 [B,Hkv,T_max,D]; out, vbar
 * [B,Hq,Lq,D] in io_dtype (PLX_OUT_*), lse, tbar fp32 [B,Hq,Lq] as written by the forward; seqlens
 * as in the forward.  Outputs in grad_dtype: dq, dr [B,Hq,Lq,D]; dk, dv [B,Hkv,T_max,D], every row
 * written (zeros past a context, for rows without keys and for keys no row sees).
 * Three launches on `stream`: the projections tau, beta into `workspace` (caller-owned device
 * memory, parallax_prefill_bwd_workspace_bytes, 16-byte aligned), the row-tile pass (dq, dr) and
 * the column-tile pass (dk, dv).  The weights reach the tensor cores as bf16.  D in {64, 128};
 * all tensors 16-byte aligned.  `status` as in the forward.  Nothing is allocated.
 */
int parallax_prefill_bwd(const void* q, const void* r, const void* k_cache, const void* v_cache,
                         const void* dout, const void* out, const float* lse, const float* tbar,
                         const void* vbar, const int32_t* seqlens, void* dq, void* dr, void* dk,
                         void* dv, int B, int Hq, int Hkv, int D, int Lq, int T_max, float scale,
                         int io_dtype, int grad_dtype, void* workspace, size_t workspace_bytes,
                         int32_t* status, void* stream);

/*
 * Upstream step of a decode call (Sec. 4.2 and App. "Backbone Architecture": RMSNorm on q, k and
 * rho; RoPE with base theta on q and k, optionally on rho): for every sequence b with
 * pos = seqlens[b] - 1 (the new token is already counted; NULL = T_max - 1),
 *     q_out[b,h]       = rope(rmsnorm(q_raw[b,h]) * q_weight, pos)
 *     r_out[b,h]       = rmsnorm(r_raw[b,h]) * r_weight        (rotated too if rope_on_r != 0)
 *     k_cache[b,h,pos] = rope(rmsnorm(k_raw[b,h]) * k_weight, pos)
 *     v_cache[b,h,pos] = v_raw[b,h]
 * with rmsnorm(x) = x / sqrt(mean(x^2) + eps) over the head dimension and rope the "rotate half"
 * rotary embedding (element i paired with i + D/2, angle pos * theta^(-2i/D)).  All tensors bf16:
 * q_raw, r_raw, q_out, r_out [B,Hq,D]; k_raw, v_raw [B,Hkv,D]; caches [B,Hkv,T_max,D]; weights
 * [D] or NULL (= ones).  Sequences with seqlens[b] <= 0 are left untouched.  q_out / r_out may
 * alias q_raw / r_raw.  D in {64, 128}.  One launch; its outputs feed parallax_decode_fwd_ex.
 */
int parallax_decode_prepare(const void* q_raw, const void* r_raw, const void* k_raw, const void* v_raw,
                            const void* q_weight, const void* r_weight, const void* k_weight,
                            const int32_t* seqlens, void* q_out, void* r_out, void* k_cache,
                            void* v_cache, int B, int Hq, int Hkv, int D, int T_max, float eps,
                            float rope_theta, int rope_on_r, void* stream);

/*
 * One decode step in one call: parallax_decode_prepare followed by parallax_decode_fwd_ex on its
 * outputs (q_out, r_out are caller-owned bf16 [B,Hq,D] buffers that receive the prepared query and
 * probe; they may alias q_raw / r_raw).  The attention kernel is launched as a programmatic dependent
 * of the upstream-step kernel: its CTAs are scheduled while that kernel still runs and wait, as their
 * first instruction, for its completion, so the second launch's latency is hidden (measured on small
 * batches: 2 to 5 us per step with stream launches, about 0.5 us per step inside a CUDA graph).  Arguments as in the two calls.  Nothing is launched if the attention call's
 * arguments are invalid.
 */
int parallax_decode_step(const void* q_raw, const void* r_raw, const void* k_raw, const void* v_raw,
                         const void* q_weight, const void* r_weight, const void* k_weight,
                         const int32_t* seqlens, void* q_out, void* r_out, void* k_cache, void* v_cache,
                         void* out, int B, int Hq, int Hkv, int D, int T_max, float eps, float rope_theta,
                         int rope_on_r, float scale, int out_dtype, void* workspace,
                         size_t workspace_bytes, int num_splits, void* stream);

/* Size of the built-in scratch array used by parallax_decode_fwd_static (8 MiB per device). */
#define PLX_STATIC_SCRATCH_BYTES (8u * 1024u * 1024u)

/*
 * Decode forward that allocates nothing and needs no workspace (the paper has no
 * counterpart; this is a convenience of this library).  It is for callers that
 * cannot obtain device memory where they decode: code inside a region where
 * cudaMalloc is not allowed, plug-ins that must not allocate behind their host
 * framework's memory pool, latency-critical loops that must stay off the
 * allocator.  Same arguments and result as parallax_decode_fwd_ex minus the
 * workspace; the caller still owns and passes every input and the output.
 *
 * The split-KV partial records go to a fixed PLX_STATIC_SCRATCH_BYTES array that
 * is part of the library image: every GPU that loads the library holds it until
 * the process exits.  Consequences:
 *   - Size limit: B * Hq * splits * (2*D + 4) * 4 bytes must fit.  With
 *     num_splits = 0 the library plans within the limit (down to one split, which
 *     needs no scratch); an explicit num_splits that does not fit is rejected
 *     with PLX_ERR_STATIC_SCRATCH and nothing is launched.
 *   - The first call on each device looks up the array's device address (with
 *     that device current) and caches it; make that first call outside any
 *     stream capture.
 *   - All calls on a device share the one array, and it keeps the previous
 *     call's records.  Nothing in it needs clearing between calls (each call
 *     writes every record it later reads), but two calls that overlap on the GPU
 *     (different streams, or several host threads) race on it: serialise them.
 *   - No device status word is kept: a bounded wait that runs out is not reported.
 * The call itself uses no cudaMalloc, cudaFree or allocating library routine.
 */
int parallax_decode_fwd_static(const void* q, const void* r, const void* k_cache, const void* v_cache,
                               const int32_t* seqlens, void* out, int B, int Hq, int Hkv, int D,
                               int T_max, float scale, int out_dtype, int num_splits, void* stream);

/*
 * Read-only streaming probe (a measurement aid; the paper has no counterpart).  The decode forward
 * only reads the K/V stream (Sec. 3.3: the KV stream is the cost), so its bandwidth ceiling is the
 * rate at which a kernel can read HBM and keep nothing, not the rate of a copy.  This call reads
 * `bytes` bytes at `src` (device, 16-byte aligned; bytes a multiple of 8192) exactly once:
 *   mode PLX_PROBE_VECTOR_LOADS  16-byte L1-bypassing loads, eight independent loads per thread;
 *   mode PLX_PROBE_BULK_COPIES   bulk asynchronous copies of 8 KiB into warp-private three-slot
 *                                shared-memory rings, two CTAs per SM (the staging geometry of
 *                                the decode kernel at D = 128 with the arithmetic removed).
 * `ctas` = number of CTAs, each reading one contiguous range (0 = eight per SM for vector loads,
 * two per SM for bulk copies).  `sink` (device, 16-byte aligned, PLX_PROBE_SINK_BYTES bytes) receives
 * one 16-byte store per CTA (per warp in bulk mode) so that the loads are live; its contents mean
 * nothing.  `status` (device int32, may be NULL) receives PLX_ERR_DEVICE_TIMEOUT if a bounded wait of
 * the bulk mode runs out.  One launch on `stream`; nothing is allocated.  Time it with events:
 * bandwidth = bytes / elapsed.
 */
#define PLX_PROBE_VECTOR_LOADS 0
#define PLX_PROBE_BULK_COPIES 1
#define PLX_PROBE_SINK_BYTES 65536
int parallax_read_probe(const void* src, size_t bytes, void* sink, int mode, int ctas, int32_t* status,
                        void* stream);

#ifdef __cplusplus
}
#endif
#endif /* PARALLAX_H_ */
