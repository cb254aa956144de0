/*
 * gqla.h -- C ABI of the GQLA decode hot path for NVIDIA B200 (sm_100a).
 *
 * GQLA (Group-Query Latent Attention) weights expose two algebraically
 * equivalent decoding paths (paper Sec. 3.1, "Two equivalent decoding paths"):
 *
 *   MQA-absorb path, Eq. (mqa):  all h_q heads attend the shared latent
 *       k_hat_s = [c_s^KV ; k_s^R]  (r_kv + d_r wide),  v_hat_s = c_s^KV,
 *       with W^UK folded into the query and W^UV applied to the output.
 *   GQA path, Eq. (mha):  head i attends its group's expanded cache
 *       k_{s,i} = [k^C_{s,j(i)} ; k_s^R],  v_{s,i} = v^C_{s,j(i)},
 *       j(i) = ceil(i / (h_q/g)).
 *
 * General conventions
 *   - Every data pointer is a DEVICE pointer owned by the caller.  The library
 *     allocates nothing, frees nothing, and never synchronises; each call
 *     enqueues its kernels on `stream` (a cudaStream_t passed as void*, NULL =
 *     the legacy default stream) and returns.
 *   - Tensors are row-major with the innermost dimension contiguous.  Base
 *     pointers and row strides must be 16-byte aligned (GQLA_ERR_ALIGN).
 *   - `dtype` is the storage type of q, cache and weights: GQLA_BF16 or
 *     GQLA_F32.  Accumulation, softmax statistics, split partials and LSE are
 *     always fp32.  With GQLA_BF16 the softmax probabilities are rounded to
 *     bf16 before the P.V contraction on the tensor-core kernels.
 *   - Weights W^UK, W^UV are stored [g, r_kv, d_h]: W[j][r][d] is entry (d, r)
 *     of the paper's group-j slice W_j in R^{d_h x r_kv}.
 *   - Sequence b owns cache rows seq_start[b] .. seq_start[b]+seqlens[b]-1.
 *     seqlens[b] already counts the s_q tokens of this step (their rows are
 *     appended before the call).  Query p (0 <= p < s_q) sits at position
 *     seqlens[b]-s_q+p and attends rows [0, seqlens[b]-(s_q-1-p)): the causal
 *     sum  sum_{s=1..t}  of Eqs. (mha)/(mqa).  A query with no visible row
 *     yields o = 0 and lse = -inf.
 *   - Split-KV: split k of S covers rows [k*chunk, min((k+1)*chunk, T)) with
 *     chunk = ceil(ceil(T/S)/64)*64; a split may be empty (o = 0, lse = -inf).
 *     Each partial is normalised within its split; lse is the natural-log
 *     sum-exp of the scaled scores.
 *   - Balanced split-KV: a decode call given num_splits = -S (S >= 2) lets the library cut the batch
 *     itself.  The 128-row tiles of all sequences are laid end to end (sequence 0 first) and divided
 *     into equal shares, one per resident worker (a CTA, or a CTA pair on the absorb path), so that
 *     every SM gets the same amount of cache to read however ragged the batch is:  tile n belongs to
 *     worker n / share,  share = max(ceil(total/W), ceil(max_b tiles_b/(S-1)), 1).  The pieces of a
 *     sequence are numbered in row order; o_part / lse_part still have S slots per sequence, unused
 *     slots get lse = -inf and their o_part is left unwritten (gqla_combine_splits never reads it).
 *     W depends on the GPU and the shape: gqla_balanced_workers reports it, gqla_balanced_plan lists
 *     the row ranges.  Where no kernel with this scheduler covers the call (gqla_balanced_workers
 *     returns 0) the fixed plan with S splits is used instead -- also a valid set of partials.
 *   - Weights (w_uk, w_uv) are constants of a decode loop, and the projection kernels treat them so: their tiles
 *     are requested before the kernel waits for the preceding work of the stream.  Write or update weights, then
 *     synchronise the stream once, before the first call that reads them; never produce a weight tensor with a
 *     kernel that may still be running when a call of this library is enqueued behind it.  Every other input
 *     (queries, caches, lengths, partials) is read only after the preceding work of the stream has completed.
 *   - Errors: argument violations return a code before anything is launched.
 *     A launch failure returns GQLA_ERR_CUDA.  Device-side waits are bounded;
 *     if one expires the kernel writes a non-zero code to *status_word (device
 *     int32, may be NULL) and exits -- the call itself stays asynchronous.
 */
#ifndef GQLA_H_
#define GQLA_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* The (h_q, g, d_h, r_kv, d_h^R) tuple of Sec. 4.2; canonical (128, 8, 128, 512, 64).
 * The value dimension equals d_h. */
typedef struct {
    int32_t h_q;  /* query heads                      */
    int32_t g;    /* K/V groups, h_q % g == 0          */
    int32_t d_h;  /* per-head dim                      */
    int32_t r_kv; /* latent rank                       */
    int32_t d_r;  /* decoupled-RoPE dim d_h^R          */
} gqla_dims;

typedef enum {
    GQLA_OK = 0,
    GQLA_ERR_NULL = 1,        /* a required pointer is NULL                     */
    GQLA_ERR_SHAPE = 2,       /* a dimension / count is out of range            */
    GQLA_ERR_ALIGN = 3,       /* pointer or stride not 16-byte aligned          */
    GQLA_ERR_DTYPE = 4,       /* unknown dtype                                  */
    GQLA_ERR_UNSUPPORTED = 5, /* valid but no kernel covers it                  */
    GQLA_ERR_CUDA = 6,        /* a CUDA runtime / driver call failed            */
    GQLA_ERR_TIMEOUT = 7,     /* value written to *status_word by a bounded wait */
    GQLA_ERR_CAPACITY = 8,    /* the call needs more built-in scratch than the library holds */
    GQLA_ERR_DEBUG_CHECK = 9  /* value written to *status_word by an index check of a -DGQLA_DEBUG build */
} gqla_status;

typedef enum { GQLA_BF16 = 0, GQLA_F32 = 1 } gqla_dtype;

/* Kernel policy (process-wide): AUTO picks the tensor-core (tcgen05) kernels
 * when the shape is covered and the generic SIMT kernels otherwise; GENERIC
 * forces the SIMT kernels (used by tests to cross-check the two). */
typedef enum { GQLA_POLICY_AUTO = 0, GQLA_POLICY_GENERIC = 1 } gqla_policy;
void gqla_set_policy(gqla_policy p);
int32_t gqla_get_policy(void);

/* Status word of the calls that have no status_word argument (gqla_absorb_q, gqla_up_proj,
 * gqla_expand_cache, gqla_append_expand, gqla_combine_up_proj; not in the paper: error reporting only).
 * Their tensor-core kernels bound every device-side wait like the decode kernels do; with a word registered
 * here (a device int32 the caller owns and has set to 0, process-wide, NULL = none, the default) an expired
 * wait leaves GQLA_ERR_TIMEOUT | (place << 8) in it instead of going unnoticed.  The word must stay valid
 * while any such call is in flight; it is read and written by kernels only, never by the host side of
 * the library.  gqla_get_status_word returns what was registered. */
void gqla_set_status_word(int32_t* device_word);
int32_t* gqla_get_status_word(void);

/* Eq. (mqa), line 2:  q_hat_i = [ (W^UK_{j(i)})^T q_i^C ; q_i^R ].
 *   q_c   [B, s_q, h_q, d_h]   q_r [B, s_q, h_q, d_r]   w_uk [g, r_kv, d_h]
 *   q_hat [B, s_q, h_q, r_kv + d_r]  (out, same dtype) */
gqla_status gqla_absorb_q(const gqla_dims* dims, gqla_dtype dtype, int32_t B, int32_t s_q,
                          const void* q_c, const void* q_r, const void* w_uk, void* q_hat, void* stream);

/* Eq. (mqa), lines 3-5: split-KV attention of every head over the shared latent rows.
 *   q_hat [B, s_q, h_q, r_kv+d_r];  cache [N, r_kv+d_r] with row stride
 *   cache_row_stride (elements) and cache_rows = N rows in total (rows >= N are never read; rows
 *   < N outside a sequence may be fetched by a tile and must hold finite values -- they get
 *   zero weight);  seq_start int64 [B], seqlens int32 [B] (device).
 *   o_part   [B, S, s_q, h_q, r_kv] fp32 (out),  lse_part [B, S, s_q, h_q] fp32 (out).
 *   S = num_splits >= 1.  Cache bytes are read once per step whatever s_q is (Sec. 4.2.1). */
gqla_status gqla_decode_absorb(const gqla_dims* dims, gqla_dtype dtype, int32_t B, int32_t s_q, float scale,
                               int32_t num_splits, const void* q_hat, const void* cache,
                               int64_t cache_row_stride, int64_t cache_rows, const int64_t* seq_start,
                               const int32_t* seqlens, float* o_part, float* lse_part, int32_t* status_word,
                               void* stream);

/* Eq. (mqa), lines 3-5, for a whole sequence in one piece (no split-KV): the same attention as
 * gqla_decode_absorb with num_splits = 1, but the normalised latent output is written once, in the
 * storage dtype, instead of as an fp32 partial that a merge would only copy:
 *   o_hat [B, s_q, h_q, r_kv] (out, same dtype as q_hat);  lse [B, s_q, h_q] fp32 (out) or NULL.
 * It feeds gqla_up_proj directly.  Other arguments as for gqla_decode_absorb. */
gqla_status gqla_decode_absorb_final(const gqla_dims* dims, gqla_dtype dtype, int32_t B, int32_t s_q, float scale,
                                     const void* q_hat, const void* cache, int64_t cache_row_stride,
                                     int64_t cache_rows, const int64_t* seq_start, const int32_t* seqlens,
                                     void* o_hat, float* lse, int32_t* status_word, void* stream);

/* Sec. 3.1: k^C = W^UK c^KV, v^C = W^UV c^KV per group, k^R carried over -- the one-shot
 * cache expansion that switches from the absorb path to the GQA path.
 *   cache [N, r_kv+d_r] (row stride cache_row_stride);  w_uk, w_uv [g, r_kv, d_h]
 *   k_c [N, g, d_h], v [N, g, d_h], k_r [N, d_r]  (out, same dtype; 2 g d_h + d_r per token).
 *   k_r may be NULL to skip the copy (the GQA path can read k^R from the latent cache's tail). */
gqla_status gqla_expand_cache(const gqla_dims* dims, gqla_dtype dtype, int64_t N, const void* cache,
                              int64_t cache_row_stride, const void* w_uk, const void* w_uv, void* k_c, void* v,
                              void* k_r, void* stream);

/* Sec. 3.1 again, for the rows a decode step appends: the expansion is a per-token linear map, so a
 * cache that was expanded once stays current if every step expands only its new rows.  For each
 * sequence b and p < s_q with seqlens[b] - s_q + p >= 0, row n = seq_start[b] + seqlens[b] - s_q + p of
 * k_c, v (and k_r unless NULL) is computed from row n of the latent cache; seqlens already counts the
 * new tokens, whose latent rows the caller has written.  No other row is touched.  Layouts as for
 * gqla_expand_cache; seq_start int64 [B] and seqlens int32 [B] are device arrays. */
gqla_status gqla_append_expand(const gqla_dims* dims, gqla_dtype dtype, int32_t B, int32_t s_q, const void* cache,
                               int64_t cache_row_stride, const int64_t* seq_start, const int32_t* seqlens,
                               const void* w_uk, const void* w_uv, void* k_c, void* v, void* k_r, void* stream);

/* Eq. (mha): split-KV attention of each head over its group's K_C, V plus the shared k^R.
 *   q [B, s_q, h_q, d_h+d_r] (= [q^C ; q^R]);  k_c, v [N, g, d_h];  k_r [N, .] with row stride
 *   k_r_row_stride (elements; d_r for a dense plane, r_kv+d_r when aliasing the latent cache);
 *   n_rows = N, the row count of the three planes (same reading rule as cache_rows above).
 *   o_part [B, S, s_q, h_q, d_h] fp32 (out),  lse_part [B, S, s_q, h_q] fp32 (out). */
gqla_status gqla_decode_gqa(const gqla_dims* dims, gqla_dtype dtype, int32_t B, int32_t s_q, float scale,
                            int32_t num_splits, const void* q, const void* k_c, const void* v, const void* k_r,
                            int64_t k_r_row_stride, int64_t n_rows, const int64_t* seq_start,
                            const int32_t* seqlens, float* o_part, float* lse_part, int32_t* status_word,
                            void* stream);

/* The same GQA-path step as gqla_decode_gqa followed by gqla_combine_splits, for callers that cannot
 * supply the split partials.  (The paper has no counterpart: it concerns who owns memory, not what is
 * computed.)  Meant for hosts that may not allocate on the device while decoding: a server whose memory
 * manager claimed the whole GPU at start-up, a loop that cannot afford the device-wide synchronisation of
 * cudaMalloc/cudaFree, or a C caller with no allocator of its own.  The partials are kept in an array built
 * into the library's device image, so the call allocates and frees nothing.
 *   Inputs as for gqla_decode_gqa, except that num_splits must be >= 1 (the fixed split plan; the balanced
 *   plan, num_splits <= -2, returns GQLA_ERR_SHAPE here).  out [B, s_q, h_q, d_h] of `dtype` (device,
 *   16-byte aligned), lse [B, s_q, h_q] fp32 (device) or NULL.
 *   Limits: B*num_splits*s_q*h_q <= 65536 rows and rows*d_h <= 4194304 floats (16 MiB + 256 KiB in all);
 *   anything larger returns GQLA_ERR_CAPACITY before any launch -- use gqla_decode_gqa with your own
 *   buffers then.  Each GPU that runs this entry point holds the array until the process exits.
 *   The first call on a device looks up the array's device address (one runtime query, remembered per
 *   device; the device must be current, as for every call).  That query is also the moment the CUDA
 *   runtime loads this part of the library onto the device and reserves the array there.  So make one
 *   call per device at start-up -- B = 0 is enough: it performs the query and launches nothing -- before
 *   any stream capture and, on a host whose memory manager takes the whole GPU, before it does so; if
 *   the array cannot be placed any more the call returns GQLA_ERR_CUDA.
 *   All calls on one GPU share the array and it keeps the previous call's contents.  Nothing needs
 *   clearing (every partial is rewritten before it is read), but two calls that may run concurrently on
 *   the same GPU race on it: issue them on one stream or order them yourself. */
gqla_status gqla_decode_gqa_noalloc(const gqla_dims* dims, gqla_dtype dtype, int32_t B, int32_t s_q, float scale,
                                    int32_t num_splits, const void* q, const void* k_c, const void* v,
                                    const void* k_r, int64_t k_r_row_stride, int64_t n_rows,
                                    const int64_t* seq_start, const int32_t* seqlens, void* out, float* lse,
                                    int32_t* status_word, void* stream);

/* The two decode calls over a PAGED cache (paging is not in the paper, which names KV paging among the effects
 * its model omits, Sec. 5.1 "Limitations"; it changes where a row is fetched from and nothing else).  The cache
 * (or, on the GQA path, each of k_c, v, k_r) is cut into pages of page_size rows; row t of sequence b is row
 *   block_table[b * max_pages + t / page_size] * page_size + t % page_size
 * with block_table an int32 [B, max_pages] device array whose entries below ceil(seqlens[b] / page_size)
 * must name pages inside the cache (page * page_size + page_size <= cache_rows / n_rows); later entries
 * are never read.  Everything else is as for gqla_decode_absorb / gqla_decode_gqa, and the outputs are
 * the same as for the packed cache holding the same rows.  The tensor-core kernels take page sizes that
 * are multiples of 128 rows with num_splits == 1 or the balanced plan (num_splits <= -2); other
 * combinations run on the generic kernels. */
gqla_status gqla_decode_absorb_paged(const gqla_dims* dims, gqla_dtype dtype, int32_t B, int32_t s_q, float scale,
                                     int32_t num_splits, const void* q_hat, const void* cache,
                                     int64_t cache_row_stride, int64_t cache_rows, const int32_t* block_table,
                                     int32_t max_pages, int32_t page_size, const int32_t* seqlens, float* o_part,
                                     float* lse_part, int32_t* status_word, void* stream);
gqla_status gqla_decode_gqa_paged(const gqla_dims* dims, gqla_dtype dtype, int32_t B, int32_t s_q, float scale,
                                  int32_t num_splits, const void* q, const void* k_c, const void* v, const void* k_r,
                                  int64_t k_r_row_stride, int64_t n_rows, const int32_t* block_table,
                                  int32_t max_pages, int32_t page_size, const int32_t* seqlens, float* o_part,
                                  float* lse_part, int32_t* status_word, void* stream);

/* FP8 (E4M3) KV cache.  The paper names KV-cache quantisation among the effects its model leaves out (Sec. 5.1
 * "Limitations", item (i)); what follows is this library's reading.  Elements are E4M3 codes (8-bit float: 4
 * exponent bits with bias 7, 3 mantissa bits, no infinities, largest finite value 448, NaN = S.1111.111), one
 * byte each: 576 B per token on the absorb path, 2112 B on the GQA path.  Scales are fp32, one per tensor
 * plane (latent part, RoPE part; K_C, V, k^R), chosen by the caller (e.g. max|x| / 448 from calibration):
 * a stored value is  code * scale.  Queries are quantised per row, with the planes' scales folded in, so a
 * score needs one factor per row and an output one factor per call:
 *     x_s = scale * q_scale[row] * sum_c dec(q8[row, c]) dec(k8[s, c]),      o = v_scale * softmax(x) . dec(v8).
 * The softmax probabilities are rounded to E4M3 before the P.V contraction on the tensor-core kernels (to fp32
 * nothing on the generic ones), the counterpart of the bf16 rounding of the bf16 path.
 *
 * gqla_quantize_cols_e4m3: dst[r, c] = encode(float(src[r, c]) * (1 / scale)), scale = scale_a for columns
 *   c < split and scale_b for the others (the latent cache: split = r_kv, scale_a = latent scale, scale_b = RoPE
 *   scale; a single plane: split = width).  src [rows, width] of src_dtype with row stride src_row_stride
 *   (elements); dst [rows, width] bytes, dense.  encode rounds to the nearest code, ties to the even mantissa,
 *   saturating at +-448; the multiplication and the reciprocal are fp32 operations with IEEE rounding.
 * gqla_quantize_rows_e4m3: per row  y = float(src) * pre  (pre_a for c < split, pre_b for the others: the
 *   scales of the key planes the row will meet),  s = max|y| / 448  (1 for an all-zero row),
 *   dst = encode(y * (1 / s)),  row_scale[row] = s.  src [rows, width] dense.  Use it on q_hat (absorb path:
 *   split = r_kv) or on [q^C ; q^R] (GQA path: split = d_h). */
gqla_status gqla_quantize_cols_e4m3(gqla_dtype src_dtype, int64_t rows, int32_t width, int32_t split, float scale_a,
                                    float scale_b, const void* src, int64_t src_row_stride, uint8_t* dst, void* stream);
gqla_status gqla_quantize_rows_e4m3(gqla_dtype src_dtype, int64_t rows, int32_t width, int32_t split, float pre_a,
                                    float pre_b, const void* src, uint8_t* dst, float* row_scale, void* stream);
/* Eq. (mqa), lines 3-5, over an E4M3 latent cache:  q8 [B, s_q, h_q, r_kv+d_r] codes, q_scale [B, s_q, h_q] fp32,
 * cache8 [N, r_kv+d_r] codes with row stride cache_row_stride (bytes), v_scale = the latent plane's scale.
 * num_splits as for gqla_decode_absorb (>= 1 fixed plan, <= -2 balanced).  Outputs and the other arguments as
 * for gqla_decode_absorb. */
gqla_status gqla_decode_absorb_fp8(const gqla_dims* dims, int32_t B, int32_t s_q, float scale, int32_t num_splits,
                                   const uint8_t* q8, const float* q_scale, const uint8_t* cache8,
                                   int64_t cache_row_stride, int64_t cache_rows, float v_scale, const int64_t* seq_start,
                                   const int32_t* seqlens, float* o_part, float* lse_part, int32_t* status_word,
                                   void* stream);
/* The whole-sequence form (no split-KV), the FP8 counterpart of gqla_decode_absorb_final: the normalised latent
 * output goes out once, as bf16 o_hat [B, s_q, h_q, r_kv] (lse [B, s_q, h_q] fp32 or NULL), ready for gqla_up_proj.
 * Tensor-core shapes only (r_kv = 512, d_r = 64, AUTO policy): GQLA_ERR_UNSUPPORTED otherwise -- use
 * gqla_decode_absorb_fp8 with one split and gqla_combine_splits there. */
gqla_status gqla_decode_absorb_fp8_final(const gqla_dims* dims, int32_t B, int32_t s_q, float scale, const uint8_t* q8,
                                         const float* q_scale, const uint8_t* cache8, int64_t cache_row_stride,
                                         int64_t cache_rows, float v_scale, const int64_t* seq_start,
                                         const int32_t* seqlens, void* o_hat, float* lse, int32_t* status_word,
                                         void* stream);
/* Eq. (mha) over E4M3 planes:  q8 [B, s_q, h_q, d_h+d_r], q_scale [B, s_q, h_q];  k_c8, v8 [N, g, d_h];
 * k_r8 [N, .] with row stride k_r_row_stride (bytes);  v_scale = the V plane's scale.  num_splits as for
 * gqla_decode_gqa.  Outputs and the other arguments as for gqla_decode_gqa. */
gqla_status gqla_decode_gqa_fp8(const gqla_dims* dims, int32_t B, int32_t s_q, float scale, int32_t num_splits,
                                const uint8_t* q8, const float* q_scale, const uint8_t* k_c8, const uint8_t* v8,
                                const uint8_t* k_r8, int64_t k_r_row_stride, int64_t n_rows, float v_scale,
                                const int64_t* seq_start, const int32_t* seqlens, float* o_part, float* lse_part,
                                int32_t* status_word, void* stream);

/* Log-sum-exp merge of split partials (split-KV is not in the paper; it is the flash-decoding
 * reduction of the same softmax):  M = max_k lse_k, w_k = exp(lse_k - M),
 *   out = sum_k w_k o_k / sum_k w_k,   lse = M + ln sum_k w_k;  all splits empty -> out = 0, lse = -inf.
 *   o_part [B, S, rows_per_seq, d_out] fp32, lse_part [B, S, rows_per_seq] fp32 (rows_per_seq = s_q*h_q)
 *   out [B, rows_per_seq, d_out] of out_dtype;  lse [B, rows_per_seq] fp32 or NULL. */
gqla_status gqla_combine_splits(int32_t B, int32_t rows_per_seq, int32_t num_splits, int32_t d_out,
                                gqla_dtype out_dtype, const float* o_part, const float* lse_part, void* out,
                                float* lse, void* stream);

/* Eq. (mqa), line 6:  o_i = W^UV_{j(i)} o_hat_i.
 *   o_hat [B, s_q, h_q, r_kv]   w_uv [g, r_kv, d_h]   o [B, s_q, h_q, d_h] (out, same dtype) */
gqla_status gqla_up_proj(const gqla_dims* dims, gqla_dtype dtype, int32_t B, int32_t s_q, const void* o_hat,
                         const void* w_uv, void* o, void* stream);

/* The three calls a value head dimension of its own touches.  Sec. 3.1 gives W^UV the shape of W^UK, and
 * gqla_dims says so (d_v == d_h); the MLA -> GQLA factorisation of Sec. 3.2 ("From MLA to GQLA") carries a
 * separate d_h^V:  W~^UKV in R^{g (d_h + d_h^V) x r_kv}  (e.g. d_h = 192, d_h^V = 256).  These variants
 * take it as `d_v` (>= 1); everything else is as for the call without the suffix:
 *   gqla_expand_cache_dv   w_uv [g, r_kv, d_v]  ->  v [N, g, d_v]        (k_c stays [N, g, d_h])
 *   gqla_decode_gqa_dv     v [N, g, d_v]        ->  o_part [B, S, s_q, h_q, d_v]
 *   gqla_up_proj_dv        w_uv [g, r_kv, d_v]  ->  o [B, s_q, h_q, d_v]
 * The absorb path needs nothing else (its attention runs in the latent space), and gqla_combine_splits
 * takes the output width as d_out already.  With d_v == d_h they are the calls without the suffix.
 * gqla_decode_gqa_dv runs on the tensor-core kernel when d_h = 128, d_r = 64 and d_v is a multiple of 128 up to
 * 512 (one CTA per 128-column block of V; the blocks of a group share its K tiles through L2), on the generic
 * kernel otherwise (d_v <= 512); the other two run on the generic kernels whenever d_v != d_h. */
gqla_status gqla_expand_cache_dv(const gqla_dims* dims, int32_t d_v, gqla_dtype dtype, int64_t N, const void* cache,
                                 int64_t cache_row_stride, const void* w_uk, const void* w_uv, void* k_c, void* v,
                                 void* k_r, void* stream);
gqla_status gqla_decode_gqa_dv(const gqla_dims* dims, int32_t d_v, gqla_dtype dtype, int32_t B, int32_t s_q, float scale,
                               int32_t num_splits, const void* q, const void* k_c, const void* v, const void* k_r,
                               int64_t k_r_row_stride, int64_t n_rows, const int64_t* seq_start, const int32_t* seqlens,
                               float* o_part, float* lse_part, int32_t* status_word, void* stream);
gqla_status gqla_up_proj_dv(const gqla_dims* dims, int32_t d_v, gqla_dtype dtype, int32_t B, int32_t s_q,
                            const void* o_hat, const void* w_uv, void* o, void* stream);

/* gqla_combine_splits followed by gqla_up_proj in one kernel (Eq. (mqa), line 6, applied to the merged
 * latent output): the merged o_hat never goes to memory.  Same arguments as the two calls:
 *   o_part [B, S, s_q, h_q, r_kv] fp32, lse_part [B, S, s_q, h_q] fp32, w_uv [g, r_kv, d_h]
 *   o [B, s_q, h_q, d_h] (out, `dtype`),  lse [B, s_q, h_q] fp32 (out) or NULL.
 * With GQLA_BF16 the tensor-core kernel rounds the merged o_hat to bf16 before the contraction, as
 * gqla_up_proj's input is; the generic kernel keeps it in fp32. */
gqla_status gqla_combine_up_proj(const gqla_dims* dims, gqla_dtype dtype, int32_t B, int32_t s_q, int32_t num_splits,
                                 const float* o_part, const float* lse_part, const void* w_uv, void* o, float* lse,
                                 void* stream);

/* Integer bookkeeping, exported so it can be compared exactly with an independent statement.
 * HOST pointers. */
/* Split ranges of a sequence of `seqlen` rows: begin[k], end[k] for k < num_splits. */
gqla_status gqla_split_plan(int32_t seqlen, int32_t num_splits, int32_t* begin, int32_t* end);
/* Balanced plan (see the conventions above) of a batch, on the host: begin/end [B * S] receive the row
 * range of every (sequence, slot), (0, 0) for an unused slot; worker [B * S] (may be NULL) the worker
 * that produces it, -1 for an unused slot.  s_cap = S >= 2, workers = W >= 1.  HOST pointers. */
gqla_status gqla_balanced_plan(const int32_t* seqlens, int32_t B, int32_t s_cap, int32_t workers, int32_t* begin,
                               int32_t* end, int32_t* worker);
/* Number of workers W a balanced decode call of this shape is cut for on the CURRENT device
 * (path: 0 = absorb, 1 = GQA); 0 if such a call falls back to the fixed plan; -1 on error.  The figure is that of
 * the bf16 / f32 calls; gqla_decode_absorb_fp8 always runs on CTA pairs and cuts for half the SMs per 128 query
 * rows, where the bf16 call of a shape with at most 64 query rows cuts for one worker per SM. */
int32_t gqla_balanced_workers(const gqla_dims* dims, gqla_dtype dtype, int32_t s_q, int32_t path);
/* Rows visible to query p of an s_q-token step: max(0, seqlen - (s_q-1-p)). */
int32_t gqla_visible_limit(int32_t seqlen, int32_t s_q, int32_t p);
/* 0-indexed group of 0-indexed head: the paper's j(i) = ceil(i/(h_q/g)); -1 on bad input. */
int32_t gqla_group_of_head(const gqla_dims* dims, int32_t head);
/* Name of the kernel family the current policy selects ("tcgen05" or "generic") for a decode call
 * (path: 0 = absorb, 1 = GQA) or for the grouped projections gqla_absorb_q, gqla_up_proj and
 * gqla_combine_up_proj (path: 2; s_q is ignored). */
const char* gqla_kernel_for(const gqla_dims* dims, gqla_dtype dtype, int32_t s_q, int32_t path);
const char* gqla_status_str(gqla_status s);

#ifdef __cplusplus
}
#endif
#endif /* GQLA_H_ */
