// C-ABI entry points of the GQLA decode library: argument validation, kernel selection, launch.
#include "../../include/gqla.h"

#include <atomic>

#include "common.cuh"
#include "generic_kernels.cuh"
#include "sched.cuh"
#include "tc_dispatch.cuh"

using namespace gqla;

namespace {

std::atomic<int> g_policy{GQLA_POLICY_AUTO};

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

gqla_status check_dims(const gqla_dims* d) {
    if (d == nullptr) return GQLA_ERR_NULL;
    if (d->h_q <= 0 || d->g <= 0 || d->d_h <= 0 || d->r_kv <= 0 || d->d_r < 0) return GQLA_ERR_SHAPE;
    if (d->h_q % d->g != 0) return GQLA_ERR_SHAPE;
    return GQLA_OK;
}
gqla_status check_dtype(gqla_dtype t) { return (t == GQLA_BF16 || t == GQLA_F32) ? GQLA_OK : GQLA_ERR_DTYPE; }

gqla_status launch_status() { return cudaGetLastError() == cudaSuccess ? GQLA_OK : GQLA_ERR_CUDA; }

gqla_status launch_decode_generic(gqla_dtype dtype, const DecodeArgs& a, cudaStream_t st) {
    if (a.dv > 32 * kGenericMaxV) return GQLA_ERR_UNSUPPORTED;
    const int64_t nrows = (int64_t)a.B * a.S * a.s_q * a.h_q;
    if (nrows == 0) return GQLA_OK;
    const int warps = 4;
    const int64_t blocks = (nrows + warps - 1) / warps;
    if (blocks > 0x7fffffffLL) return GQLA_ERR_SHAPE;
    if (dtype == GQLA_BF16)
        decode_generic_kernel<__nv_bfloat16><<<(unsigned)blocks, warps * 32, 0, st>>>(a);
    else
        decode_generic_kernel<float><<<(unsigned)blocks, warps * 32, 0, st>>>(a);
    return launch_status();
}

gqla_status launch_decode_generic_fp8(const DecodeArgs& a, cudaStream_t st) {
    if (a.dv > 32 * kGenericMaxV) return GQLA_ERR_UNSUPPORTED;
    const int64_t nrows = (int64_t)a.B * a.S * a.s_q * a.h_q;
    if (nrows == 0) return GQLA_OK;
    const int warps = 4;
    const int64_t blocks = (nrows + warps - 1) / warps;
    if (blocks > 0x7fffffffLL) return GQLA_ERR_SHAPE;
    decode_generic_kernel<e4m3><<<(unsigned)blocks, warps * 32, 0, st>>>(a);
    return launch_status();
}

}  // namespace

extern "C" {

void gqla_set_policy(gqla_policy p) { g_policy.store(p == GQLA_POLICY_GENERIC ? GQLA_POLICY_GENERIC : GQLA_POLICY_AUTO); }
int32_t gqla_get_policy(void) { return g_policy.load(); }

void gqla_set_status_word(int32_t* device_word) { projection_status_word() = device_word; }
int32_t* gqla_get_status_word(void) { return projection_status_word(); }

const char* gqla_status_str(gqla_status s) {
    switch (s) {
        case GQLA_OK: return "ok";
        case GQLA_ERR_NULL: return "null pointer";
        case GQLA_ERR_SHAPE: return "bad shape";
        case GQLA_ERR_ALIGN: return "pointer or stride not 16-byte aligned";
        case GQLA_ERR_DTYPE: return "unknown dtype";
        case GQLA_ERR_UNSUPPORTED: return "unsupported configuration";
        case GQLA_ERR_CUDA: return "CUDA error";
        case GQLA_ERR_TIMEOUT: return "device wait timed out";
        case GQLA_ERR_CAPACITY: return "call exceeds the library's built-in scratch capacity";
        case GQLA_ERR_DEBUG_CHECK: return "index check of a debug build failed";
    }
    return "unknown status";
}

gqla_status gqla_split_plan(int32_t seqlen, int32_t num_splits, int32_t* begin, int32_t* end) {
    if (begin == nullptr || end == nullptr) return GQLA_ERR_NULL;
    if (seqlen < 0 || num_splits < 1) return GQLA_ERR_SHAPE;
    for (int32_t k = 0; k < num_splits; ++k) split_range(seqlen, num_splits, k, &begin[k], &end[k]);
    return GQLA_OK;
}

int32_t gqla_visible_limit(int32_t seqlen, int32_t s_q, int32_t p) { return visible_limit(seqlen, s_q, p); }

gqla_status gqla_balanced_plan(const int32_t* seqlens, int32_t B, int32_t s_cap, int32_t workers, int32_t* begin,
                               int32_t* end, int32_t* worker) {
    if (seqlens == nullptr || begin == nullptr || end == nullptr) return GQLA_ERR_NULL;
    if (B < 0 || s_cap < 2 || workers < 1) return GQLA_ERR_SHAPE;
    for (int32_t b = 0; b < B; ++b)
        if (seqlens[b] < 0) return GQLA_ERR_SHAPE;
    const int64_t n = (int64_t)B * s_cap;
    for (int64_t i = 0; i < n; ++i) {
        begin[i] = end[i] = -1;  // "not written yet"
        if (worker != nullptr) worker[i] = -1;
    }
    // every worker walks its share exactly as the kernels' roles do
    for (int32_t w = 0; w < workers; ++w) {
        Walker wk;
        wk.init_balanced(seqlens, B, s_cap, w, workers, balanced_start_serial(seqlens, B, s_cap, w, workers));
        Piece pc;
        while (wk.next(pc)) {
            if (pc.n_tiles > 0) {
                const int64_t i = (int64_t)pc.b * s_cap + pc.k;
                if (pc.k < 0 || pc.k >= s_cap || begin[i] != -1) return GQLA_ERR_UNSUPPORTED;  // would be a bug
                begin[i] = pc.tok_begin;
                end[i] = pc.tok_end;
                if (worker != nullptr) worker[i] = w;
            }
            for (int32_t k = pc.fill_begin; k < pc.fill_end; ++k) {
                const int64_t i = (int64_t)pc.b * s_cap + k;
                if (begin[i] != -1) return GQLA_ERR_UNSUPPORTED;
                begin[i] = end[i] = 0;
            }
        }
    }
    for (int64_t i = 0; i < n; ++i)
        if (begin[i] == -1) return GQLA_ERR_UNSUPPORTED;  // a slot nobody owns: would be a bug
    return GQLA_OK;
}

int32_t gqla_balanced_workers(const gqla_dims* d, gqla_dtype dtype, int32_t s_q, int32_t path) {
    if (check_dims(d) != GQLA_OK) return -1;
    if (g_policy.load() != GQLA_POLICY_AUTO || !tc_covers(*d, dtype, s_q, path)) return 0;
    return tc_balanced_workers(*d, s_q, path);
}

int32_t gqla_group_of_head(const gqla_dims* d, int32_t head) {
    if (check_dims(d) != GQLA_OK || head < 0 || head >= d->h_q) return -1;
    return head / (d->h_q / d->g);
}

const char* gqla_kernel_for(const gqla_dims* d, gqla_dtype dtype, int32_t s_q, int32_t path) {
    if (check_dims(d) != GQLA_OK) return "invalid";
    if (g_policy.load() != GQLA_POLICY_AUTO) return "generic";
    if (path == 2) return tc_gemm_covers(*d, dtype) ? "tcgen05" : "generic";
    return tc_covers(*d, dtype, s_q, path) ? "tcgen05" : "generic";
}

gqla_status gqla_absorb_q(const gqla_dims* d, gqla_dtype dtype, int32_t B, int32_t s_q, const void* q_c,
                          const void* q_r, const void* w_uk, void* q_hat, void* stream) {
    gqla_status s;
    if ((s = check_dims(d)) != GQLA_OK) return s;
    if ((s = check_dtype(dtype)) != GQLA_OK) return s;
    if (B < 0 || s_q < 1) return GQLA_ERR_SHAPE;
    if (q_c == nullptr || w_uk == nullptr || q_hat == nullptr || (d->d_r > 0 && q_r == nullptr)) return GQLA_ERR_NULL;
    if (!aligned16(q_c) || !aligned16(q_r) || !aligned16(w_uk) || !aligned16(q_hat)) return GQLA_ERR_ALIGN;
    const int64_t rows = (int64_t)B * s_q * d->h_q;
    if (rows == 0) return GQLA_OK;
    if (rows > 0x7fffffffLL) return GQLA_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    if (g_policy.load() == GQLA_POLICY_AUTO) {
        s = tc_absorb_q(*d, dtype, B, s_q, q_c, q_r, w_uk, q_hat, st);
        if (s != GQLA_ERR_UNSUPPORTED) return s;
    }
    const int hpg = d->h_q / d->g;
    const size_t smem = (size_t)d->d_h * sizeof(float);
    if (smem > 48 * 1024) return GQLA_ERR_UNSUPPORTED;
    if (dtype == GQLA_BF16)
        absorb_q_generic_kernel<__nv_bfloat16><<<(unsigned)rows, 128, smem, st>>>(
            d->h_q, hpg, d->d_h, d->r_kv, d->d_r, (const __nv_bfloat16*)q_c, (const __nv_bfloat16*)q_r,
            (const __nv_bfloat16*)w_uk, (__nv_bfloat16*)q_hat);
    else
        absorb_q_generic_kernel<float><<<(unsigned)rows, 128, smem, st>>>(
            d->h_q, hpg, d->d_h, d->r_kv, d->d_r, (const float*)q_c, (const float*)q_r, (const float*)w_uk,
            (float*)q_hat);
    return launch_status();
}

gqla_status gqla_up_proj(const gqla_dims* d, gqla_dtype dtype, int32_t B, int32_t s_q, const void* o_hat,
                         const void* w_uv, void* o, void* stream) {
    return gqla_up_proj_dv(d, d == nullptr ? 0 : d->d_h, dtype, B, s_q, o_hat, w_uv, o, stream);
}

gqla_status gqla_up_proj_dv(const gqla_dims* d, int32_t d_v, gqla_dtype dtype, int32_t B, int32_t s_q,
                            const void* o_hat, const void* w_uv, void* o, void* stream) {
    gqla_status s;
    if ((s = check_dims(d)) != GQLA_OK) return s;
    if ((s = check_dtype(dtype)) != GQLA_OK) return s;
    if (B < 0 || s_q < 1 || d_v < 1) return GQLA_ERR_SHAPE;
    if (o_hat == nullptr || w_uv == nullptr || o == nullptr) return GQLA_ERR_NULL;
    if (!aligned16(o_hat) || !aligned16(w_uv) || !aligned16(o)) return GQLA_ERR_ALIGN;
    const int64_t rows = (int64_t)B * s_q * d->h_q;
    if (rows == 0) return GQLA_OK;
    if (rows > 0x7fffffffLL) return GQLA_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    if (g_policy.load() == GQLA_POLICY_AUTO && d_v == d->d_h) {
        s = tc_up_proj(*d, dtype, B, s_q, o_hat, w_uv, o, st);
        if (s != GQLA_ERR_UNSUPPORTED) return s;
    }
    const int hpg = d->h_q / d->g;
    const size_t smem = (size_t)d->r_kv * sizeof(float);
    if (smem > 48 * 1024) return GQLA_ERR_UNSUPPORTED;
    if (dtype == GQLA_BF16)
        up_proj_generic_kernel<__nv_bfloat16><<<(unsigned)rows, 128, smem, st>>>(
            d->h_q, hpg, d_v, d->r_kv, (const __nv_bfloat16*)o_hat, (const __nv_bfloat16*)w_uv, (__nv_bfloat16*)o);
    else
        up_proj_generic_kernel<float><<<(unsigned)rows, 128, smem, st>>>(d->h_q, hpg, d_v, d->r_kv,
                                                                        (const float*)o_hat, (const float*)w_uv,
                                                                        (float*)o);
    return launch_status();
}

gqla_status gqla_combine_up_proj(const gqla_dims* d, gqla_dtype dtype, int32_t B, int32_t s_q, int32_t num_splits,
                                 const float* o_part, const float* lse_part, const void* w_uv, void* o, float* lse,
                                 void* stream) {
    gqla_status s;
    if ((s = check_dims(d)) != GQLA_OK) return s;
    if ((s = check_dtype(dtype)) != GQLA_OK) return s;
    if (B < 0 || s_q < 1 || num_splits < 1) return GQLA_ERR_SHAPE;
    if (o_part == nullptr || lse_part == nullptr || w_uv == nullptr || o == nullptr) return GQLA_ERR_NULL;
    if (!aligned16(o_part) || !aligned16(w_uv) || !aligned16(o)) return GQLA_ERR_ALIGN;
    const int64_t rows = (int64_t)B * s_q * d->h_q;
    if (rows == 0) return GQLA_OK;
    if (rows > 0x7fffffffLL) return GQLA_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    if (g_policy.load() == GQLA_POLICY_AUTO) {
        s = tc_combine_up_proj(*d, dtype, B, s_q, num_splits, o_part, lse_part, w_uv, o, lse, st);
        if (s != GQLA_ERR_UNSUPPORTED) return s;
    }
    const size_t smem = (size_t)d->r_kv * sizeof(float);
    if (smem > 48 * 1024) return GQLA_ERR_UNSUPPORTED;
    const int hpg = d->h_q / d->g;
    if (dtype == GQLA_BF16)
        combine_up_generic_kernel<__nv_bfloat16><<<(unsigned)rows, 128, smem, st>>>(
            d->h_q, hpg, d->d_h, d->r_kv, s_q * d->h_q, num_splits, o_part, lse_part, (const __nv_bfloat16*)w_uv,
            (__nv_bfloat16*)o, lse);
    else
        combine_up_generic_kernel<float><<<(unsigned)rows, 128, smem, st>>>(d->h_q, hpg, d->d_h, d->r_kv, s_q * d->h_q,
                                                                           num_splits, o_part, lse_part,
                                                                           (const float*)w_uv, (float*)o, lse);
    return launch_status();
}

gqla_status gqla_expand_cache(const gqla_dims* d, gqla_dtype dtype, int64_t N, const void* cache,
                              int64_t cache_row_stride, const void* w_uk, const void* w_uv, void* k_c, void* v,
                              void* k_r, void* stream) {
    return gqla_expand_cache_dv(d, d == nullptr ? 0 : d->d_h, dtype, N, cache, cache_row_stride, w_uk, w_uv, k_c, v, k_r,
                                stream);
}

gqla_status gqla_expand_cache_dv(const gqla_dims* d, int32_t d_v, gqla_dtype dtype, int64_t N, const void* cache,
                                 int64_t cache_row_stride, const void* w_uk, const void* w_uv, void* k_c, void* v,
                                 void* k_r, void* stream) {
    gqla_status s;
    if ((s = check_dims(d)) != GQLA_OK) return s;
    if ((s = check_dtype(dtype)) != GQLA_OK) return s;
    if (N < 0 || cache_row_stride < d->r_kv + d->d_r || d_v < 1) return GQLA_ERR_SHAPE;
    if (N == 0) return GQLA_OK;
    if (cache == nullptr || w_uk == nullptr || w_uv == nullptr || k_c == nullptr || v == nullptr) return GQLA_ERR_NULL;
    if (!aligned16(cache) || !aligned16(w_uk) || !aligned16(w_uv) || !aligned16(k_c) || !aligned16(v) ||
        !aligned16(k_r))
        return GQLA_ERR_ALIGN;
    cudaStream_t st = (cudaStream_t)stream;
    if (g_policy.load() == GQLA_POLICY_AUTO && d_v == d->d_h) {
        s = tc_expand_cache(*d, dtype, N, cache, cache_row_stride, w_uk, w_uv, k_c, v, k_r, st);
        if (s != GQLA_ERR_UNSUPPORTED) return s;
    }
    const size_t smem = (size_t)kExpandRows * d->r_kv * sizeof(float);
    if (smem > 48 * 1024) return GQLA_ERR_UNSUPPORTED;
    const int64_t blocks = (N + kExpandRows - 1) / kExpandRows;
    if (blocks > 0x7fffffffLL) return GQLA_ERR_SHAPE;
    if (dtype == GQLA_BF16)
        expand_cache_generic_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, smem, st>>>(
            N, d->g, d->d_h, d_v, d->r_kv, d->d_r, (const __nv_bfloat16*)cache, cache_row_stride,
            (const __nv_bfloat16*)w_uk, (const __nv_bfloat16*)w_uv, (__nv_bfloat16*)k_c, (__nv_bfloat16*)v,
            (__nv_bfloat16*)k_r);
    else
        expand_cache_generic_kernel<float><<<(unsigned)blocks, 256, smem, st>>>(
            N, d->g, d->d_h, d_v, d->r_kv, d->d_r, (const float*)cache, cache_row_stride, (const float*)w_uk,
            (const float*)w_uv, (float*)k_c, (float*)v, (float*)k_r);
    return launch_status();
}

gqla_status gqla_append_expand(const gqla_dims* d, gqla_dtype dtype, int32_t B, int32_t s_q, const void* cache,
                               int64_t cache_row_stride, const int64_t* seq_start, const int32_t* seqlens,
                               const void* w_uk, const void* w_uv, void* k_c, void* v, void* k_r, void* stream) {
    gqla_status s;
    if ((s = check_dims(d)) != GQLA_OK) return s;
    if ((s = check_dtype(dtype)) != GQLA_OK) return s;
    if (B < 0 || s_q < 1 || cache_row_stride < d->r_kv + d->d_r) return GQLA_ERR_SHAPE;
    if (B == 0) return GQLA_OK;
    if (cache == nullptr || seq_start == nullptr || seqlens == nullptr || w_uk == nullptr || w_uv == nullptr ||
        k_c == nullptr || v == nullptr)
        return GQLA_ERR_NULL;
    if (!aligned16(cache) || !aligned16(w_uk) || !aligned16(w_uv) || !aligned16(k_c) || !aligned16(v) ||
        !aligned16(k_r))
        return GQLA_ERR_ALIGN;
    if (g_policy.load() == GQLA_POLICY_AUTO) {
        s = tc_append_expand(*d, dtype, B, s_q, cache, cache_row_stride, seq_start, seqlens, w_uk, w_uv, k_c, v, k_r,
                             (cudaStream_t)stream);
        if (s != GQLA_ERR_UNSUPPORTED) return s;
    }
    const size_t smem = ((size_t)kExpandRows * d->r_kv + (size_t)kAppendKSplit * kExpandRows * kAppendCols) * sizeof(float);
    if (smem > 48 * 1024 || 2 * d->g > 65535) return GQLA_ERR_UNSUPPORTED;
    const int64_t blocks = ((int64_t)B * s_q + kExpandRows - 1) / kExpandRows;
    if (blocks > 0x7fffffffLL) return GQLA_ERR_SHAPE;
    const dim3 grid((unsigned)blocks, (unsigned)(2 * d->g));
    cudaStream_t st = (cudaStream_t)stream;
    if (dtype == GQLA_BF16)
        append_expand_kernel<__nv_bfloat16><<<grid, kAppendThreads, smem, st>>>(
            B, s_q, d->g, d->d_h, d->r_kv, d->d_r, (const __nv_bfloat16*)cache, cache_row_stride, seq_start, seqlens,
            (const __nv_bfloat16*)w_uk, (const __nv_bfloat16*)w_uv, (__nv_bfloat16*)k_c, (__nv_bfloat16*)v,
            (__nv_bfloat16*)k_r);
    else
        append_expand_kernel<float><<<grid, kAppendThreads, smem, st>>>(B, s_q, d->g, d->d_h, d->r_kv, d->d_r, (const float*)cache,
                                                             cache_row_stride, seq_start, seqlens, (const float*)w_uk,
                                                             (const float*)w_uv, (float*)k_c, (float*)v, (float*)k_r);
    return launch_status();
}

static gqla_status check_decode_common(const gqla_dims* d, gqla_dtype dtype, int32_t B, int32_t s_q, int32_t S,
                                       const RowMap& rows, const int32_t* seqlens, const float* o_part,
                                       const float* lse_part) {
    gqla_status s;
    if ((s = check_dims(d)) != GQLA_OK) return s;
    if ((s = check_dtype(dtype)) != GQLA_OK) return s;
    if (B < 0 || s_q < 1 || S == 0 || S == -1) return GQLA_ERR_SHAPE;  // S <= -2: balanced plan, -S slots
    if (rows.block_table != nullptr && (rows.page_size < 1 || rows.max_pages < 1)) return GQLA_ERR_SHAPE;
    if (B == 0) return GQLA_OK;
    if ((rows.seq_start == nullptr && rows.block_table == nullptr) || seqlens == nullptr || o_part == nullptr ||
        lse_part == nullptr)
        return GQLA_ERR_NULL;
    if (!aligned16(o_part)) return GQLA_ERR_ALIGN;
    return GQLA_OK;
}

static RowMap packed_rows(const int64_t* seq_start) { return RowMap{seq_start, nullptr, 0, 0}; }
static RowMap paged_rows(const int32_t* block_table, int32_t max_pages, int32_t page_size) {
    return RowMap{nullptr, block_table, max_pages, page_size};
}

static gqla_status decode_absorb_any(const gqla_dims* d, gqla_dtype dtype, int32_t B, int32_t s_q, float scale,
                                     int32_t num_splits, const void* q_hat, const void* cache, int64_t cache_row_stride,
                                     int64_t cache_rows, const RowMap& rows, const int32_t* seqlens, float* o_part,
                                     float* lse_part, int32_t* status_word, void* stream) {
    gqla_status s = check_decode_common(d, dtype, B, s_q, num_splits, rows, seqlens, o_part, lse_part);
    if (s != GQLA_OK) return s;
    if (B == 0) return GQLA_OK;
    if (q_hat == nullptr || cache == nullptr) return GQLA_ERR_NULL;
    if (!aligned16(q_hat) || !aligned16(cache)) return GQLA_ERR_ALIGN;
    if (cache_row_stride < d->r_kv + d->d_r || cache_rows < 0) return GQLA_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    if (g_policy.load() == GQLA_POLICY_AUTO && tc_covers(*d, dtype, s_q, 0)) {
        s = tc_decode_absorb(*d, B, s_q, scale, num_splits, q_hat, cache, cache_row_stride, cache_rows, rows, seqlens,
                             o_part, lse_part, status_word, st);
        if (s != GQLA_ERR_UNSUPPORTED) return s;
    }
    DecodeArgs a{};
    a.q = q_hat;
    a.kA = cache; a.kA_stride = cache_row_stride; a.kA_gstride = 0; a.dA = d->r_kv + d->d_r;
    a.kB = nullptr; a.kB_stride = 0; a.dB = 0;
    a.v = cache; a.v_stride = cache_row_stride; a.v_gstride = 0; a.dv = d->r_kv;
    a.rows = rows; a.seqlens = seqlens;
    a.B = B; a.S = num_splits < 0 ? -num_splits : num_splits; a.s_q = s_q; a.h_q = d->h_q; a.hpg = d->h_q / d->g;
    a.scale = scale; a.o_part = o_part; a.lse_part = lse_part;
    return launch_decode_generic(dtype, a, st);
}

gqla_status gqla_decode_absorb(const gqla_dims* d, gqla_dtype dtype, int32_t B, int32_t s_q, float scale,
                               int32_t num_splits, const void* q_hat, const void* cache, int64_t cache_row_stride,
                               int64_t cache_rows, const int64_t* seq_start, const int32_t* seqlens, float* o_part,
                               float* lse_part, int32_t* status_word, void* stream) {
    return decode_absorb_any(d, dtype, B, s_q, scale, num_splits, q_hat, cache, cache_row_stride, cache_rows,
                             packed_rows(seq_start), seqlens, o_part, lse_part, status_word, stream);
}

gqla_status gqla_decode_absorb_final(const gqla_dims* d, gqla_dtype dtype, int32_t B, int32_t s_q, float scale,
                                     const void* q_hat, const void* cache, int64_t cache_row_stride, int64_t cache_rows,
                                     const int64_t* seq_start, const int32_t* seqlens, void* o_hat, float* lse,
                                     int32_t* status_word, void* stream) {
    gqla_status s;
    if ((s = check_dims(d)) != GQLA_OK) return s;
    if ((s = check_dtype(dtype)) != GQLA_OK) return s;
    if (B < 0 || s_q < 1) return GQLA_ERR_SHAPE;
    if (B == 0) return GQLA_OK;
    if (q_hat == nullptr || cache == nullptr || seq_start == nullptr || seqlens == nullptr || o_hat == nullptr)
        return GQLA_ERR_NULL;
    if (!aligned16(q_hat) || !aligned16(cache) || !aligned16(o_hat)) return GQLA_ERR_ALIGN;
    if (cache_row_stride < d->r_kv + d->d_r || cache_rows < 0) return GQLA_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    const RowMap rows = packed_rows(seq_start);
    if (g_policy.load() == GQLA_POLICY_AUTO && tc_covers(*d, dtype, s_q, 0)) {
        s = tc_decode_absorb(*d, B, s_q, scale, 1, q_hat, cache, cache_row_stride, cache_rows, rows, seqlens, nullptr, lse,
                             status_word, st, o_hat);
        if (s != GQLA_ERR_UNSUPPORTED) return s;
    }
    DecodeArgs a{};
    a.q = q_hat;
    a.kA = cache; a.kA_stride = cache_row_stride; a.kA_gstride = 0; a.dA = d->r_kv + d->d_r;
    a.kB = nullptr; a.kB_stride = 0; a.dB = 0;
    a.v = cache; a.v_stride = cache_row_stride; a.v_gstride = 0; a.dv = d->r_kv;
    a.rows = rows; a.seqlens = seqlens;
    a.B = B; a.S = 1; a.s_q = s_q; a.h_q = d->h_q; a.hpg = d->h_q / d->g;
    a.scale = scale; a.o_part = nullptr; a.lse_part = lse; a.o_final = o_hat;
    return launch_decode_generic(dtype, a, st);
}

gqla_status gqla_decode_absorb_paged(const gqla_dims* d, gqla_dtype dtype, int32_t B, int32_t s_q, float scale,
                                     int32_t num_splits, const void* q_hat, const void* cache, int64_t cache_row_stride,
                                     int64_t cache_rows, const int32_t* block_table, int32_t max_pages,
                                     int32_t page_size, const int32_t* seqlens, float* o_part, float* lse_part,
                                     int32_t* status_word, void* stream) {
    return decode_absorb_any(d, dtype, B, s_q, scale, num_splits, q_hat, cache, cache_row_stride, cache_rows,
                             paged_rows(block_table, max_pages, page_size), seqlens, o_part, lse_part, status_word, stream);
}

static gqla_status decode_gqa_any(const gqla_dims* d, int32_t d_v, gqla_dtype dtype, int32_t B, int32_t s_q, float scale,
                                  int32_t num_splits, const void* q, const void* k_c, const void* v, const void* k_r,
                                  int64_t k_r_row_stride, int64_t n_rows, const RowMap& rows, const int32_t* seqlens,
                                  float* o_part, float* lse_part, int32_t* status_word, void* stream) {
    gqla_status s = check_decode_common(d, dtype, B, s_q, num_splits, rows, seqlens, o_part, lse_part);
    if (s != GQLA_OK) return s;
    if (B == 0) return GQLA_OK;
    if (q == nullptr || k_c == nullptr || v == nullptr || (d->d_r > 0 && k_r == nullptr)) return GQLA_ERR_NULL;
    if (!aligned16(q) || !aligned16(k_c) || !aligned16(v) || !aligned16(k_r)) return GQLA_ERR_ALIGN;
    if ((d->d_r > 0 && k_r_row_stride < d->d_r) || n_rows < 0 || d_v < 1) return GQLA_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    if (g_policy.load() == GQLA_POLICY_AUTO && tc_covers(*d, dtype, s_q, 1)) {
        s = tc_decode_gqa(*d, B, s_q, scale, num_splits, q, k_c, v, k_r, k_r_row_stride, n_rows, rows, seqlens, o_part,
                          lse_part, status_word, st, d_v);
        if (s != GQLA_ERR_UNSUPPORTED) return s;
    }
    DecodeArgs a{};
    a.q = q;
    a.kA = k_c; a.kA_stride = (int64_t)d->g * d->d_h; a.kA_gstride = d->d_h; a.dA = d->d_h;
    a.kB = k_r; a.kB_stride = k_r_row_stride; a.dB = d->d_r;
    a.v = v; a.v_stride = (int64_t)d->g * d_v; a.v_gstride = d_v; a.dv = d_v;
    a.rows = rows; a.seqlens = seqlens;
    a.B = B; a.S = num_splits < 0 ? -num_splits : num_splits; a.s_q = s_q; a.h_q = d->h_q; a.hpg = d->h_q / d->g;
    a.scale = scale; a.o_part = o_part; a.lse_part = lse_part;
    return launch_decode_generic(dtype, a, st);
}

gqla_status gqla_decode_gqa_dv(const gqla_dims* d, int32_t d_v, gqla_dtype dtype, int32_t B, int32_t s_q, float scale,
                               int32_t num_splits, const void* q, const void* k_c, const void* v, const void* k_r,
                               int64_t k_r_row_stride, int64_t n_rows, const int64_t* seq_start, const int32_t* seqlens,
                               float* o_part, float* lse_part, int32_t* status_word, void* stream) {
    return decode_gqa_any(d, d_v, dtype, B, s_q, scale, num_splits, q, k_c, v, k_r, k_r_row_stride, n_rows,
                          packed_rows(seq_start), seqlens, o_part, lse_part, status_word, stream);
}

gqla_status gqla_decode_gqa(const gqla_dims* d, gqla_dtype dtype, int32_t B, int32_t s_q, float scale,
                            int32_t num_splits, const void* q, const void* k_c, const void* v, const void* k_r,
                            int64_t k_r_row_stride, int64_t n_rows, const int64_t* seq_start, const int32_t* seqlens,
                            float* o_part, float* lse_part, int32_t* status_word, void* stream) {
    return decode_gqa_any(d, d == nullptr ? 0 : d->d_h, dtype, B, s_q, scale, num_splits, q, k_c, v, k_r, k_r_row_stride,
                          n_rows, packed_rows(seq_start), seqlens, o_part, lse_part, status_word, stream);
}

gqla_status gqla_decode_gqa_paged(const gqla_dims* d, gqla_dtype dtype, int32_t B, int32_t s_q, float scale,
                                  int32_t num_splits, const void* q, const void* k_c, const void* v, const void* k_r,
                                  int64_t k_r_row_stride, int64_t n_rows, const int32_t* block_table, int32_t max_pages,
                                  int32_t page_size, const int32_t* seqlens, float* o_part, float* lse_part,
                                  int32_t* status_word, void* stream) {
    return decode_gqa_any(d, d == nullptr ? 0 : d->d_h, dtype, B, s_q, scale, num_splits, q, k_c, v, k_r, k_r_row_stride,
                          n_rows, paged_rows(block_table, max_pages, page_size), seqlens, o_part, lse_part, status_word,
                          stream);
}

gqla_status gqla_combine_splits(int32_t B, int32_t rows_per_seq, int32_t num_splits, int32_t d_out,
                                gqla_dtype out_dtype, const float* o_part, const float* lse_part, void* out,
                                float* lse, void* stream) {
    gqla_status s;
    if ((s = check_dtype(out_dtype)) != GQLA_OK) return s;
    if (B < 0 || rows_per_seq < 1 || num_splits < 1 || d_out < 1) return GQLA_ERR_SHAPE;
    if (B == 0) return GQLA_OK;
    if (o_part == nullptr || lse_part == nullptr || out == nullptr) return GQLA_ERR_NULL;
    if (!aligned16(o_part) || !aligned16(out)) return GQLA_ERR_ALIGN;
    const int64_t rows = (int64_t)B * rows_per_seq;
    if (rows > 0x7fffffffLL) return GQLA_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    if (d_out % 4 == 0) {
        const int vec = d_out % 16 == 0 ? 16 : (d_out % 8 == 0 ? 8 : 4);  // output columns per thread
        const int64_t items = rows * (d_out / vec);
        const int64_t nblk = (items + 255) / 256;
        if (nblk > 0x7fffffffLL) return GQLA_ERR_SHAPE;
        const dim3 blocks((unsigned)nblk), threads(256);
        const bool bf = out_dtype == GQLA_BF16;
        cudaError_t e;
#define GQLA_COMBINE(TO, V)                                                                                              \
    e = tc::launch_pdl(combine_vec_kernel<TO, V>, blocks, threads, 0, st, rows, rows_per_seq, num_splits, d_out, o_part, \
                       lse_part, (TO*)out, lse)
        if (vec == 16) { if (bf) GQLA_COMBINE(__nv_bfloat16, 16); else GQLA_COMBINE(float, 16); }
        else if (vec == 8) { if (bf) GQLA_COMBINE(__nv_bfloat16, 8); else GQLA_COMBINE(float, 8); }
        else { if (bf) GQLA_COMBINE(__nv_bfloat16, 4); else GQLA_COMBINE(float, 4); }
#undef GQLA_COMBINE
        return e == cudaSuccess ? GQLA_OK : GQLA_ERR_CUDA;
    }
    const size_t smem = (size_t)num_splits * sizeof(float);
    if (smem > 48 * 1024) return GQLA_ERR_UNSUPPORTED;
    if (out_dtype == GQLA_BF16)
        combine_generic_kernel<__nv_bfloat16><<<(unsigned)rows, 128, smem, st>>>(B, rows_per_seq, num_splits, d_out,
                                                                                 o_part, lse_part,
                                                                                 (__nv_bfloat16*)out, lse);
    else
        combine_generic_kernel<float><<<(unsigned)rows, 128, smem, st>>>(B, rows_per_seq, num_splits, d_out, o_part,
                                                                         lse_part, (float*)out, lse);
    return launch_status();
}

// ------------------------------------------------------------------------------------------------ FP8 (E4M3) cache

gqla_status gqla_quantize_cols_e4m3(gqla_dtype src_dtype, int64_t rows, int32_t width, int32_t split, float scale_a,
                                    float scale_b, const void* src, int64_t src_row_stride, uint8_t* dst, void* stream) {
    gqla_status s;
    if ((s = check_dtype(src_dtype)) != GQLA_OK) return s;
    if (rows < 0 || width < 1 || split < 0 || split > width || src_row_stride < width) return GQLA_ERR_SHAPE;
    if (!(scale_a > 0.f) || !(scale_b > 0.f)) return GQLA_ERR_SHAPE;
    if (rows == 0) return GQLA_OK;
    if (src == nullptr || dst == nullptr) return GQLA_ERR_NULL;
    const int64_t items = rows * ((width + 1) / 2);
    const int64_t blocks = (items + 255) / 256;
    if (blocks > 0x7fffffffLL) return GQLA_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    if (src_dtype == GQLA_BF16)
        quantize_cols_kernel<__nv_bfloat16><<<(unsigned)blocks, 256, 0, st>>>(rows, width, split, scale_a, scale_b,
                                                                              (const __nv_bfloat16*)src, src_row_stride, dst);
    else
        quantize_cols_kernel<float><<<(unsigned)blocks, 256, 0, st>>>(rows, width, split, scale_a, scale_b,
                                                                      (const float*)src, src_row_stride, dst);
    return launch_status();
}

gqla_status gqla_quantize_rows_e4m3(gqla_dtype src_dtype, int64_t rows, int32_t width, int32_t split, float pre_a,
                                    float pre_b, const void* src, uint8_t* dst, float* row_scale, void* stream) {
    gqla_status s;
    if ((s = check_dtype(src_dtype)) != GQLA_OK) return s;
    if (rows < 0 || width < 1 || split < 0 || split > width) return GQLA_ERR_SHAPE;
    if (rows == 0) return GQLA_OK;
    if (src == nullptr || dst == nullptr || row_scale == nullptr) return GQLA_ERR_NULL;
    const int64_t blocks = (rows + 3) / 4;
    if (blocks > 0x7fffffffLL) return GQLA_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    cudaError_t e;
    if (src_dtype == GQLA_BF16 && width % 8 == 0 && split % 8 == 0 && width <= 8 * 32 * kQuantChunksPerLane && aligned16(src) &&
        (reinterpret_cast<uintptr_t>(dst) & 7u) == 0)
        e = tc::launch_pdl(quantize_rows_bf16_vec_kernel, dim3((unsigned)blocks), dim3(128), 0, st, rows, width, split, pre_a,
                           pre_b, (const __nv_bfloat16*)src, dst, row_scale);
    else if (src_dtype == GQLA_BF16)
        e = tc::launch_pdl(quantize_rows_kernel<__nv_bfloat16>, dim3((unsigned)blocks), dim3(128), 0, st, rows, width, split,
                           pre_a, pre_b, (const __nv_bfloat16*)src, dst, row_scale);
    else
        e = tc::launch_pdl(quantize_rows_kernel<float>, dim3((unsigned)blocks), dim3(128), 0, st, rows, width, split, pre_a,
                           pre_b, (const float*)src, dst, row_scale);
    return e == cudaSuccess ? GQLA_OK : GQLA_ERR_CUDA;
}

// S >= 1: fixed split plan;  S <= -2: balanced plan with -S slots (tensor-core kernels; the generic ones run the
// fixed plan with -S splits, also a valid set of partials)
static gqla_status check_fp8_common(const gqla_dims* d, int32_t B, int32_t s_q, int32_t S, const void* q8,
                                    const float* q_scale, float v_scale, const int64_t* seq_start, const int32_t* seqlens,
                                    const float* o_part, const float* lse_part) {
    gqla_status s;
    if ((s = check_dims(d)) != GQLA_OK) return s;
    if (B < 0 || s_q < 1 || S == 0 || S == -1 || !(v_scale > 0.f)) return GQLA_ERR_SHAPE;
    if (B == 0) return GQLA_OK;
    if (q8 == nullptr || q_scale == nullptr || seq_start == nullptr || seqlens == nullptr || o_part == nullptr ||
        lse_part == nullptr)
        return GQLA_ERR_NULL;
    if (!aligned16(q8) || !aligned16(o_part)) return GQLA_ERR_ALIGN;
    return GQLA_OK;
}

gqla_status gqla_decode_absorb_fp8(const gqla_dims* d, int32_t B, int32_t s_q, float scale, int32_t num_splits,
                                   const uint8_t* q8, const float* q_scale, const uint8_t* cache8, int64_t cache_row_stride,
                                   int64_t cache_rows, float v_scale, const int64_t* seq_start, const int32_t* seqlens,
                                   float* o_part, float* lse_part, int32_t* status_word, void* stream) {
    gqla_status s = check_fp8_common(d, B, s_q, num_splits, q8, q_scale, v_scale, seq_start, seqlens, o_part, lse_part);
    if (s != GQLA_OK) return s;
    if (B == 0) return GQLA_OK;
    if (cache8 == nullptr) return GQLA_ERR_NULL;
    if (!aligned16(cache8)) return GQLA_ERR_ALIGN;
    if (cache_row_stride < d->r_kv + d->d_r || cache_rows < 0) return GQLA_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    if (g_policy.load() == GQLA_POLICY_AUTO) {
        s = tc_decode_absorb_fp8(*d, B, s_q, scale, num_splits, q8, q_scale, cache8, cache_row_stride, cache_rows, v_scale,
                                 packed_rows(seq_start), seqlens, o_part, lse_part, status_word, st);
        if (s != GQLA_ERR_UNSUPPORTED) return s;
    }
    DecodeArgs a{};
    a.q = q8;
    a.kA = cache8; a.kA_stride = cache_row_stride; a.kA_gstride = 0; a.dA = d->r_kv + d->d_r;
    a.kB = nullptr; a.kB_stride = 0; a.dB = 0;
    a.v = cache8; a.v_stride = cache_row_stride; a.v_gstride = 0; a.dv = d->r_kv;
    a.rows = packed_rows(seq_start); a.seqlens = seqlens;
    a.B = B; a.S = num_splits < 0 ? -num_splits : num_splits; a.s_q = s_q; a.h_q = d->h_q; a.hpg = d->h_q / d->g;
    a.scale = scale; a.o_part = o_part; a.lse_part = lse_part; a.q_row_scale = q_scale; a.v_scale = v_scale;
    return launch_decode_generic_fp8(a, st);
}

gqla_status gqla_decode_absorb_fp8_final(const gqla_dims* d, int32_t B, int32_t s_q, float scale, const uint8_t* q8,
                                         const float* q_scale, const uint8_t* cache8, int64_t cache_row_stride,
                                         int64_t cache_rows, float v_scale, const int64_t* seq_start, const int32_t* seqlens,
                                         void* o_hat, float* lse, int32_t* status_word, void* stream) {
    gqla_status s;
    if ((s = check_dims(d)) != GQLA_OK) return s;
    if (B < 0 || s_q < 1 || !(v_scale > 0.f)) return GQLA_ERR_SHAPE;
    if (B == 0) return GQLA_OK;
    if (q8 == nullptr || q_scale == nullptr || cache8 == nullptr || seq_start == nullptr || seqlens == nullptr ||
        o_hat == nullptr)
        return GQLA_ERR_NULL;
    if (!aligned16(q8) || !aligned16(cache8) || !aligned16(o_hat)) return GQLA_ERR_ALIGN;
    if (cache_row_stride < d->r_kv + d->d_r || cache_rows < 0) return GQLA_ERR_SHAPE;
    if (g_policy.load() != GQLA_POLICY_AUTO) return GQLA_ERR_UNSUPPORTED;
    return tc_decode_absorb_fp8(*d, B, s_q, scale, 1, q8, q_scale, cache8, cache_row_stride, cache_rows, v_scale,
                                packed_rows(seq_start), seqlens, nullptr, lse, status_word, (cudaStream_t)stream, o_hat);
}

gqla_status gqla_decode_gqa_fp8(const gqla_dims* d, int32_t B, int32_t s_q, float scale, int32_t num_splits,
                                const uint8_t* q8, const float* q_scale, const uint8_t* k_c8, const uint8_t* v8,
                                const uint8_t* k_r8, int64_t k_r_row_stride, int64_t n_rows, float v_scale,
                                const int64_t* seq_start, const int32_t* seqlens, float* o_part, float* lse_part,
                                int32_t* status_word, void* stream) {
    gqla_status s = check_fp8_common(d, B, s_q, num_splits, q8, q_scale, v_scale, seq_start, seqlens, o_part, lse_part);
    if (s != GQLA_OK) return s;
    if (B == 0) return GQLA_OK;
    if (k_c8 == nullptr || v8 == nullptr || (d->d_r > 0 && k_r8 == nullptr)) return GQLA_ERR_NULL;
    if (!aligned16(k_c8) || !aligned16(v8) || !aligned16(k_r8)) return GQLA_ERR_ALIGN;
    if ((d->d_r > 0 && k_r_row_stride < d->d_r) || n_rows < 0) return GQLA_ERR_SHAPE;
    cudaStream_t st = (cudaStream_t)stream;
    if (g_policy.load() == GQLA_POLICY_AUTO) {
        s = tc_decode_gqa_fp8(*d, B, s_q, scale, num_splits, q8, q_scale, k_c8, v8, k_r8, k_r_row_stride, n_rows, v_scale,
                              packed_rows(seq_start), seqlens, o_part, lse_part, status_word, st);
        if (s != GQLA_ERR_UNSUPPORTED) return s;
    }
    DecodeArgs a{};
    a.q = q8;
    a.kA = k_c8; a.kA_stride = (int64_t)d->g * d->d_h; a.kA_gstride = d->d_h; a.dA = d->d_h;
    a.kB = k_r8; a.kB_stride = k_r_row_stride; a.dB = d->d_r;
    a.v = v8; a.v_stride = (int64_t)d->g * d->d_h; a.v_gstride = d->d_h; a.dv = d->d_h;
    a.rows = packed_rows(seq_start); a.seqlens = seqlens;
    a.B = B; a.S = num_splits < 0 ? -num_splits : num_splits; a.s_q = s_q; a.h_q = d->h_q; a.hpg = d->h_q / d->g;
    a.scale = scale; a.o_part = o_part; a.lse_part = lse_part; a.q_row_scale = q_scale; a.v_scale = v_scale;
    return launch_decode_generic_fp8(a, st);
}

}  // extern "C"
