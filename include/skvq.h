/*
 * skvq.h -- C ABI of the B200-native SKVQ hot path (sliding-window KV-cache
 * quantization, arXiv 2405.06219): append tokens to a cache whose older part is
 * 2/4-bit group-quantized, and run decode attention directly on that cache.
 *
 * General rules
 *   - Every pointer is a DEVICE pointer owned by the caller unless its comment
 *     says "host".  The library allocates nothing, frees nothing and keeps no
 *     pointer after a call returns.
 *   - Every device buffer must be 16-byte aligned.
 *   - Calls only enqueue work on `cuda_stream` (a cudaStream_t passed as void*,
 *     NULL = the default stream); they never synchronise.  Lengths are read on
 *     the device.
 *   - Return value: SKVQ_OK or a negative SKVQ_ERR_* code.  On an error nothing
 *     is launched.  Conditions only the device can see (a sequence that would
 *     exceed its capacity) leave that sequence untouched and OR a bit into
 *     skvq_cache::status.
 *   - Kernels of one call, and of consecutive calls on a stream, are chained with programmatic
 *     dependent launches: a kernel may be scheduled while its predecessor on the stream drains
 *     and waits on the device before it touches that predecessor's results.  Nothing changes for
 *     the caller: stream order is kept.
 *   - Compiled for sm_100a only; there is no CPU path.
 *
 * Notation: B sequences, Hq query heads, Hkv KV heads (Hq % Hkv == 0, query head
 * hq reads KV head hq / (Hq/Hkv)), D = head_dim, W = window, G = group size,
 * ng = D/G groups per row, L_b = lengths[b], Lq_b = max(L_b - W, 0) tokens of
 * sequence b that have left the window; of those, positions below n_sink (attention
 * sinks) stay fp16 and the rest are quantized.
 */
#ifndef SKVQ_H_
#define SKVQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SKVQ_OK 0
#define SKVQ_ERR_INVALID_ARG (-1) /* NULL where a buffer is required, negative size, ... */
#define SKVQ_ERR_UNSUPPORTED (-2) /* head_dim != 128, k_bits not in {2,3,4}, v_bits not in {2,3,4,15}, G not in {32,64,128}, Hq % Hkv != 0, Hq/Hkv > 8 */
#define SKVQ_ERR_MISALIGNED (-3)  /* a device buffer is not 16-byte aligned */
#define SKVQ_ERR_CAPACITY (-4)    /* host-visible overflow: n_new or max_len_hint beyond max_tokens */
#define SKVQ_ERR_WORKSPACE (-5)   /* workspace missing or smaller than skvq_workspace_size() */
#define SKVQ_ERR_CUDA (-6)        /* the CUDA runtime reported an error at launch */
#define SKVQ_ERR_SCRATCH_LIMIT (-7) /* skvq_decode_attention_noalloc: the split partials of this shape need more
                                     than SKVQ_NOALLOC_SCRATCH_BYTES */

#define SKVQ_STATUS_OVERFLOW 1    /* bit set in *status when a sequence would have exceeded max_tokens */
#define SKVQ_STATUS_COPY_TIMEOUT 2 /* bit set when a shared-memory copy inside decode attention never completed (bounded
                                     wait ran out); the affected tokens contribute nothing to the result */
#define SKVQ_STATUS_BOUNDS 4       /* only from a library built with -DSKVQ_CHECKED (a debugging build): a kernel was about to
                                     use a row, slot or partial index outside its buffer; the access was skipped */

/* Rows of the quantized segment are allocated in multiples of this many tokens so
 * that a kernel may stage whole tiles; see skvq_quant_capacity(). */
#define SKVQ_TOKEN_ALIGN 64

/* Group boundaries (skvq_cache::group_bounds_*) are multiples of this many channels. */
#define SKVQ_GROUP_GRANULE 32

/* v_bits value of the "1.5-bit" setting for values (abstract; Sec. 4.2: keys at 2 bits, values at 1.5 bits): three
 * levels per code (2^1.5 = 2.83 rounds to 3), five codes per byte in base 3.  The paper gives neither the levels nor the
 * storage of that setting; this is the library's reading of it. */
#define SKVQ_BITS_TERNARY 15

/* Shape and quantization settings (host struct). */
typedef struct skvq_config {
    int32_t batch;       /* B >= 1 */
    int32_t n_q_heads;   /* Hq */
    int32_t n_kv_heads;  /* Hkv */
    int32_t head_dim;    /* D, must be 128 */
    int32_t k_bits;      /* 2, 3 or 4 (3: the 3-bit setting of the paper's comparison with KVQuant, Sec. 4.3) */
    int32_t v_bits;      /* 2, 3, 4 or SKVQ_BITS_TERNARY (three-level codes, 1.625 bits per element stored) */
    int32_t group_size;  /* G: 32, 64 or 128; a row has ng = D/G groups that share scale/zero: equal runs of G consecutive
                            (reordered) channels, or, with skvq_cache::group_bounds_*, ng runs of unequal width whose
                            AVERAGE width is G (Sec. 4.2: the number of groups is kept, not their size) */
    int32_t window;      /* W >= 0 latest tokens kept in fp16 (Sec. 3.2); 0 quantizes everything */
    int32_t max_tokens;  /* per-sequence capacity (quantized segment + window) */
    int32_t n_sink;      /* 0..64: the first n_sink positions of a sequence are never quantized (Sec. 3.2, filter
                            rules; the paper's experiments keep 5); 0 = none */
    int32_t meta_fp8;    /* 0: scale and zero point stored in fp16; 1: in FP8 E4M3 (Sec. 4.1 "Quantization"; 2.5
                            instead of 3 bits per element at 2 bits and group 32).  The codes are computed
                            against the stored, rounded parameters either way. */
} skvq_config;

/*
 * The cache (host struct of device pointers).  cap = skvq_quant_capacity(cfg).
 * Layouts are row-major:
 *   k_codes/v_codes  uint8   [B][Hkv][cap][D*bits/8]  a row is a little-endian bit stream: code j = bits [j*bits, (j+1)*bits)
 *                                                     of the row, j counted in reordered order (2- and 4-bit codes never
 *                                                     cross a byte; a 3-bit code may: 8 codes per 3 bytes, 48-byte rows).
 *                                                     v_bits = SKVQ_BITS_TERNARY: (D+4)/5 = 26 bytes per row, code j is
 *                                                     base-3 digit j % 5 (weight 3^(j % 5)) of byte j / 5; the two unused
 *                                                     digits of the last byte are 0
 *   k_meta/v_meta    half2   [B][Hkv][cap][ng]        {scale h, zero z}; dequantized x^ = h*code + z.  With meta_fp8:
 *                    uint8   [B][Hkv][cap][ng][2]     {E4M3 byte of h, E4M3 byte of z} (1 sign, 4 exponent bits with
 *                                                     bias 7, 3 mantissa bits, no infinities, largest finite 448;
 *                                                     rounded to nearest even from fp32, saturating)
 *   k_win/v_win      half    [B][Hkv][W][D]           ring; token t sits in slot t % W, reordered order
 *   lengths          int32   [B]                      tokens appended so far (start at 0)
 *   reorder_k/_v     int32   [Hkv][D]                 gather index: stored[j] = source[idx[j]]; each
 *                                                     row must be a permutation of 0..D-1 (Eq. 1)
 *   alpha_k/_v       float   [Hkv][ng]                clip factor per group in (0,1] (Eq. 2)
 *   status           int32   [1]                      optional (may be NULL); SKVQ_STATUS_* bits are OR-ed in
 *   k_sink/v_sink    half    [B][Hkv][n_sink][D]      position t < n_sink once it has left the window, reordered
 *                                                     order; may be NULL when n_sink == 0
 *   group_bounds_k/_v int32  [Hkv][ng+1]              optional (NULL = equal groups): group g of KV head h covers reordered
 *                                                     channels [bounds[h][g], bounds[h][g+1]); bounds[h][0] = 0,
 *                                                     bounds[h][ng] = D, strictly increasing, every entry a multiple of
 *                                                     SKVQ_GROUP_GRANULE (Sec. 3.1: channels of similar range share a
 *                                                     group; split_groups(X, group_indices) of Algorithm 1).  The arrays
 *                                                     live on the device, so the library cannot check them: validate the
 *                                                     host copy with skvq_check_group_bounds() before uploading it.
 * Rows at or beyond Lq_b, and rows below n_sink, of the quantized buffers hold unspecified bytes.  The buffers fully describe the state:
 * copying them is a checkpoint.
 */
typedef struct skvq_cache {
    void *k_codes, *v_codes;
    void *k_meta, *v_meta;
    void *k_win, *v_win;
    int32_t *lengths;
    const int32_t *reorder_k, *reorder_v;
    const float *alpha_k, *alpha_v;
    int32_t *status;
    void *k_sink, *v_sink;
    const int32_t *group_bounds_k, *group_bounds_v;
} skvq_cache;

/* Options of one decode-attention call (host struct). */
typedef struct skvq_attn_args {
    float sm_scale;         /* softmax scale, e.g. 1/sqrt(D) */
    int32_t max_len_hint;   /* host upper bound on lengths[] (sizes the grid); <= max_tokens */
    int32_t n_splits;       /* 0 = library chooses (one CTA per resident slot of the GPU, all with the same share of
                               the batch's quantized tokens); n > 0 asks for about n pieces per (sequence, KV head) */
    void *workspace;        /* device scratch for the split partials, >= skvq_workspace_size() bytes */
    size_t workspace_bytes;
    void *ev_begin, *ev_end;/* optional cudaEvent_t (else NULL) recorded on the stream immediately
                               before / after the partition kernel, for profiling; events keep the merge kernel from
                               overlapping the partition kernel's tail, so leave them NULL in production */
} skvq_attn_args;

/* Library version (major*100 + minor). */
int skvq_version(void);

/* Static text for a return code. */
const char *skvq_strerror(int code);

/* Number of CUDA kernels this library has launched in this process (monotonic). */
uint64_t skvq_launch_count(void);

/* Validate cfg (host only).  Returns SKVQ_OK or the error a call with it would return. */
int skvq_check_config(const skvq_config *cfg);

/* Validate group boundaries on the host: bounds is int32 [n_kv_heads][ng+1] with ng = head_dim / group_size.  Returns
 * SKVQ_OK, or SKVQ_ERR_INVALID_ARG when a row does not start at 0, end at head_dim, increase strictly, or holds an entry
 * that is not a multiple of SKVQ_GROUP_GRANULE. */
int skvq_check_group_bounds(const skvq_config *cfg, const int32_t *bounds_host);

/* Rows per (sequence, KV head) in the quantized segment:
 * round_up(max(max_tokens - W, 0), SKVQ_TOKEN_ALIGN), at least SKVQ_TOKEN_ALIGN.  Negative on a bad cfg. */
int32_t skvq_quant_capacity(const skvq_config *cfg);

/* Bytes of k_codes, v_codes, k_meta, v_meta, k_win, v_win (in that order) for cfg.  Host only. */
int skvq_cache_sizes(const skvq_config *cfg, size_t bytes_out[6]);

/* Bytes of k_sink (= v_sink) for cfg; 0 when n_sink == 0 or on a bad cfg.  Host only. */
size_t skvq_sink_bytes(const skvq_config *cfg);

/*
 * Append tokens (Sec. 3.2, Algorithm 1 body, clipping_quant; Eq. 2).
 * Sequence b receives n_b = n_new_per_seq ? n_new_per_seq[b] : n_new tokens (0 <= n_b <= n_new).
 * With L0 = lengths[b], L1 = L0 + n_b: every token in [max(L0-W,0), max(L1-W,0)) is reordered
 * (stored[j] = x[idx[j]]), split into groups of G channels and quantized per group:
 *   lo = alpha*min, hi = alpha*max, h = fp16((hi-lo)/qmax), z = fp16(lo),
 *   code = clamp(rint((x - z)/h), 0, qmax)   (fp32, IEEE division, ties to even; h == 0 -> code 0;
 *                                             qmax = 2^bits-1, or 2 for the three-level codes)
 * (min, max and alpha are those of the channel's group: equal runs of G channels, or the runs given by group_bounds_*)
 * the last min(L1, W) tokens are kept in fp16 in the ring, and lengths[b] becomes L1.
 * Exception (Sec. 3.2, the filter mask of Algorithm 1): a token at a position below n_sink is copied, reordered,
 * to k_sink/v_sink when it leaves the window instead of being quantized.
 * One bulk call equals the same tokens appended one at a time.
 *   k, v           half [B][n_new][Hkv][D], original channel order (rows beyond n_b are ignored)
 *   n_new_per_seq  device int32 [B] or NULL
 * If L1 > max_tokens the sequence is left unchanged and SKVQ_STATUS_OVERFLOW is set in *status.
 * NaN/Inf inputs give unspecified codes.
 */
int skvq_quantize_append(const skvq_config *cfg, const skvq_cache *cache, const void *k, const void *v,
                         const int32_t *n_new_per_seq, int32_t n_new, void *cuda_stream);

/* Scratch bytes skvq_decode_attention needs for lengths up to max_len_hint and the given n_splits
 * (0 = the library's choice for that hint; the choice depends on the GPU's SM count, so ask on the
 * machine that will run the call).  0 on a bad cfg. */
size_t skvq_workspace_size(const skvq_config *cfg, int32_t max_len_hint, int32_t n_splits);

/*
 * Decode attention of one query per sequence over [quantized prefix || fp16 window]
 * (Eq. 1 and the first lines of Algorithm 1; softmax and its scale written out):
 *   q' = q[reorder_k],  s_t = sm_scale * sum_j q'_j K~[t][j],  p = softmax_t(s),
 *   o'_j = sum_t p_t V~[t][j],  out[reorder_v[j]] = o'_j,
 * where K~/V~ are h*code+z for t < Lq_b (the sink row for t < n_sink) and the ring value for Lq_b <= t < L_b.  Dequantization
 * happens in registers; no dequantized cache is written.  A sequence of length 0 yields zeros.
 * Tokens beyond max_len_hint (a sequence longer than the hint) are not looked at.
 *   q    half [B][Hq][D]      out  half [B][Hq][D]
 * The workspace contents are overwritten; calls sharing a workspace must be stream-ordered.
 */
int skvq_decode_attention(const skvq_config *cfg, const skvq_cache *cache, const void *q, void *out,
                          const skvq_attn_args *args, void *cuda_stream);

/*
 * One decode step driven from HOST buffers: copies k_new, v_new (half [B][1][Hkv][D]) and q
 * (half [B][Hq][D]) from host memory into `staging`, appends the token, runs decode attention and
 * copies out (half [B][Hq][D]) back to host memory, all enqueued on the stream (the caller
 * synchronises before reading out_host).  Pinned host memory keeps the copies asynchronous; when k_new, v_new
 * and q lie back to back in host memory in that order they travel in one copy instead of three.
 *   staging  device scratch of at least skvq_step_staging_size(cfg) bytes
 */
size_t skvq_step_staging_size(const skvq_config *cfg);
int skvq_decode_step_host(const skvq_config *cfg, const skvq_cache *cache, const void *k_new_host,
                          const void *v_new_host, const void *q_host, void *out_host, void *staging,
                          const skvq_attn_args *args, void *cuda_stream);

/*
 * Decode attention for callers that have no device memory left to lend and must not allocate.
 * (The paper has no counterpart: this is a packaging variant of skvq_decode_attention, same result.)
 *
 * Who needs it: a serving engine usually sizes its KV cache to swallow whatever HBM remains after the
 * weights, so by the time the decode loop runs there is no spare buffer to pass as `workspace`, and a
 * cudaMalloc inside that loop would either fail or stall every stream on the device while it runs.  The
 * same holds for code that runs as a plug-in inside somebody else's memory pool and may not call the
 * allocator at all.  For them the split partials go into an array that is part of the library image:
 * SKVQ_NOALLOC_SCRATCH_BYTES of device memory on every GPU that loads the library, held until exit.
 * The call itself allocates and frees nothing (no cudaMalloc/cudaFree, no allocating library routine).
 *
 * Arguments are those of skvq_decode_attention with the fields of skvq_attn_args passed directly; q, out and
 * the cache are still the caller's.  Limits and rules:
 *   - Shapes whose partials need more than SKVQ_NOALLOC_SCRATCH_BYTES (that is,
 *     skvq_workspace_size(cfg, max_len_hint, n_splits) > SKVQ_NOALLOC_SCRATCH_BYTES) are refused with
 *     SKVQ_ERR_SCRATCH_LIMIT before anything is launched; ask for fewer splits or use the workspace variant.
 *   - The first call on each device looks up the array's device address (with that device current).  The CUDA
 *     runtime loads a library's device image lazily, so this first lookup is also the moment the image, and the
 *     array in it, is placed in that device's memory: on a device that is already full it fails with
 *     SKVQ_ERR_CUDA.  Make the first call on every device at start-up -- before the engine sizes its KV cache to
 *     the remaining memory, and outside any stream capture; later calls only launch kernels.
 *   - The looked-up address is kept until the process exits.  cudaDeviceReset() (or anything else that destroys
 *     the device's primary context) invalidates it; this entry point must not be used on that device afterwards.
 *   - All calls on a device share the one array, and it keeps whatever the last call left there.  Nothing
 *     needs clearing (a call writes every partial before it reads it), but two calls that overlap on the GPU
 *     -- different streams, no ordering between them -- race on it.  Keep them stream-ordered.
 */
#define SKVQ_NOALLOC_SCRATCH_BYTES (8u << 20)
int skvq_decode_attention_noalloc(const skvq_config *cfg, const skvq_cache *cache, const void *q, void *out,
                                  float sm_scale, int32_t max_len_hint, int32_t n_splits, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* SKVQ_H_ */
