// Host-side dispatch to the tensor-core (tcgen05) kernels.  Each function returns
// GQLA_ERR_UNSUPPORTED when the shape is outside what those kernels cover, in which case
// the caller falls through to the generic SIMT kernels.
#pragma once
#include <stdlib.h>

#include "../../include/gqla.h"
#include "common.cuh"
#include "tc_decode_absorb.cuh"
#include "tc_decode_absorb_t.cuh"
#include "tc_decode_gqa.cuh"
#include "tc_decode_gqa_t.cuh"
#include "tc_decode_gqa_fp8.cuh"
#include "tc_decode_absorb_fp8.cuh"
#include "tc_append.cuh"
#include "tc_combine_up.cuh"
#include "tc_expand.cuh"
#include "tc_gemm.cuh"

// Largest (padded) query-row count per group served by the tokens-on-M GQA kernel when the environment does not
// say otherwise; beyond it the row-replicating kernel runs (its replication factor 128/R is then 2 or 1).
#ifndef GQLA_GQA_TOKENS_MAX_ROWS
#define GQLA_GQA_TOKENS_MAX_ROWS 32
#endif
// Likewise for the absorb path: largest (padded) h_q * s_q served by its tokens-on-M kernel by default.
#ifndef GQLA_ABSORB_TOKENS_MAX_ROWS
#define GQLA_ABSORB_TOKENS_MAX_ROWS 64
#endif

namespace gqla {

// Status word of the calls whose C signature has none (gqla_absorb_q, gqla_up_proj, gqla_expand_cache,
// gqla_append_expand, gqla_combine_up_proj): registered once per process with gqla_set_status_word.
inline int32_t*& projection_status_word() {
    static int32_t* word = nullptr;
    return word;
}

inline bool stride_ok(int64_t elems) { return (elems * 2) % 16 == 0; }
inline int next_pow2(int x) {
    int p = 1;
    while (p < x) p <<= 1;
    return p;
}

// Shapes the grouped tcgen05 GEMMs cover: bf16, d_h = 128, r_kv a multiple of 256, d_r a multiple
// of 8, at most 128 heads per group (padded to a power of two of head slots per query position).
inline bool tc_gemm_covers(const gqla_dims& d, gqla_dtype dtype) {
    const int hpg = d.h_q / d.g;
    return dtype == GQLA_BF16 && d.d_h == 128 && d.r_kv % 256 == 0 && d.r_kv <= 4096 && d.d_r % 8 == 0 && hpg <= 128;
}

// Rows of the GQA kernel's query block: heads per group and query positions are each padded to a power
// of two (the padding rows are computed and dropped), at least 8 rows in all.
inline int gqa_rows(const gqla_dims& d, int32_t s_q, int* hpg_box, int* sq_box) {
    const int sb = next_pow2(s_q);
    int hb = next_pow2(d.h_q / d.g);
    if (hb * sb < 8) hb = 8 / sb;
    if (hpg_box != nullptr) *hpg_box = hb;
    if (sq_box != nullptr) *sq_box = sb;
    return hb * sb;
}
inline bool is_pow2(int x) { return x > 0 && (x & (x - 1)) == 0; }

inline bool tc_covers(const gqla_dims& d, gqla_dtype dtype, int32_t s_q, int32_t path) {
    if (dtype != GQLA_BF16) return false;
    if (path == 1) {
        // the group's (h_q/g) * s_q rows, padded to R, are replicated 128/R times down the MMA tile
        if (d.d_h != 128 || d.d_r != 64 || s_q < 1 || s_q > 8) return false;
        return gqa_rows(d, s_q, nullptr, nullptr) <= 128;
    }
    // absorb path: the pair kernel is specialised for the 512 + 64 latent row
    return d.r_kv == 512 && d.d_r == 64 && s_q >= 1 && s_q <= 8;
}

// SMs of the current device (cached per device ordinal); 0 on failure.
inline int sm_count() {
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
        cached[dev] = n;
    }
    return cached[dev];
}

inline int absorb_resident_pairs();

// Query rows of the absorb path's tokens-on-M kernel (tc_decode_absorb_t.cuh): h_q * s_q padded to 16, 32 or 64.
inline int absorb_rows_t(const gqla_dims& d, int32_t s_q) {
    const int r = next_pow2(d.h_q * s_q);
    return r < 16 ? 16 : r;
}
// Which absorb kernel serves a shape: the tokens-on-M kernel up to 64 query rows (half the pair kernel's tile), the
// pair kernel beyond.  GQLA_ABSORB_KERNEL=rows|tokens overrides the choice for the shapes both cover, h_q * s_q <= 64
// (read once per process; a tuning aid).
inline bool absorb_prefers_tokens(const gqla_dims& d, int32_t s_q) {
    static const int forced = []() {
        const char* e = getenv("GQLA_ABSORB_KERNEL");
        if (e == nullptr) return 0;
        return e[0] == 't' ? 1 : (e[0] == 'r' ? 2 : 0);
    }();
    const int rows_t = absorb_rows_t(d, s_q);
    if (rows_t > 64) return false;
    if (forced != 0) return forced == 1;
    return rows_t <= GQLA_ABSORB_TOKENS_MAX_ROWS;
}

// Workers of the balanced plan on the absorb path's CTA-pair kernels (bf16 and E4M3): pairs resident at once per
// block of 128 query rows.
inline int32_t pair_balanced_workers(const gqla_dims& d, int32_t s_q) {
    const int row_blocks = (s_q * d.h_q + 127) / 128;
    const int pairs = absorb_resident_pairs();
    return pairs / row_blocks > 0 ? pairs / row_blocks : 0;
}

// Workers of the balanced plan: the GQA path runs one CTA per SM and keeps the cut points of all g
// groups identical (so the CTAs of the g groups read one k_R tile together): W = SMs / g workers per
// group.  The absorb path runs one CTA pair per two SMs: W = (SMs / 2) / row_blocks per row block.
// 0 when the device cannot be queried (or has no GPU): the fixed plan is used then.
inline int32_t tc_balanced_workers(const gqla_dims& d, int32_t s_q, int32_t path) {
    const int sms = sm_count();
    if (sms <= 0) return 0;
    if (path == 1) return sms / d.g > 0 ? sms / d.g : 0;
    if (absorb_prefers_tokens(d, s_q)) return sms;  // one persistent CTA per SM
    return pair_balanced_workers(d, s_q);
}

inline gqla_status tc_expand_cache(const gqla_dims& d, gqla_dtype dtype, int64_t N, const void* cache,
                                   int64_t cache_row_stride, const void* w_uk, const void* w_uv, void* k_c, void* v,
                                   void* k_r, cudaStream_t st) {
    if (!tc_gemm_covers(d, dtype) || !stride_ok(cache_row_stride)) return GQLA_ERR_UNSUPPORTED;
    const int64_t m_tiles = (N + 127) / 128;
    if (m_tiles * 2 * d.g > 0x7fffffffLL) return GQLA_ERR_UNSUPPORTED;
    CUtensorMap tmA, tmK, tmV;
    {
        const uint64_t dims[2] = {(uint64_t)d.r_kv, (uint64_t)N};
        const uint64_t str[1] = {(uint64_t)cache_row_stride * 2};
        const uint32_t box[2] = {64, 128};
        if (!tc::make_tmap_bf16(&tmA, cache, 2, dims, str, box)) return GQLA_ERR_CUDA;
    }
    {
        const uint64_t dims[2] = {(uint64_t)d.d_h, (uint64_t)d.g * d.r_kv};
        const uint64_t str[1] = {(uint64_t)d.d_h * 2};
        const uint32_t box[2] = {64, 64};
        if (!tc::make_tmap_bf16(&tmK, w_uk, 2, dims, str, box)) return GQLA_ERR_CUDA;
        if (!tc::make_tmap_bf16(&tmV, w_uv, 2, dims, str, box)) return GQLA_ERR_CUDA;
    }
    // the canonical shape (r_kv = 512, even g) runs on CTA pairs that keep their latent rows resident
    if (d.r_kv == 64 * tc::ExpandSmem::kKBlocks && d.g % 2 == 0 && (N + 255) / 256 * 2 <= 0x7fffffffLL) {
        tc::ExpandParams ep{};
        ep.n_rows = N; ep.g = d.g; ep.r_kv = d.r_kv; ep.d_r = d.d_r;
        ep.k_c = k_c; ep.v = v; ep.cache = cache; ep.k_r = k_r; ep.cache_stride = cache_row_stride; ep.status = projection_status_word();
        auto kern = tc::expand_tc_kernel;
        static bool attr_set[64] = {};
        int dev = 0;
        cudaGetDevice(&dev);
        if (dev < 0 || dev >= 64 || !attr_set[dev]) {
            if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::ExpandSmem::kTotal) != cudaSuccess)
                return GQLA_ERR_CUDA;
            if (dev >= 0 && dev < 64) attr_set[dev] = true;
        }
        // output planes as [N, g * 128] matrices; stores of 64 columns x 128 rows, clipped at row N
        CUtensorMap tmOK, tmOV;
        {
            const uint64_t odims[2] = {(uint64_t)d.g * 128, (uint64_t)N};
            const uint64_t ostr[1] = {(uint64_t)d.g * 128 * 2};
            const uint32_t obox[2] = {64, 128};
            if (!tc::make_tmap_bf16(&tmOK, k_c, 2, odims, ostr, obox)) return GQLA_ERR_CUDA;
            if (!tc::make_tmap_bf16(&tmOV, v, 2, odims, ostr, obox)) return GQLA_ERR_CUDA;
        }
        const unsigned pairs = (unsigned)((N + 255) / 256);
        return tc::launch_pdl(kern, dim3(2 * pairs), dim3(tc::ExpandSmem::kThreads), tc::ExpandSmem::kTotal, st, ep, tmA, tmK,
                              tmV, tmOK, tmOV) == cudaSuccess
                   ? GQLA_OK
                   : GQLA_ERR_CUDA;
    }
    tc::GemmParams p{};
    p.k_blocks = d.r_kv / 64;
    p.m_total = N;
    p.h_q = d.h_q; p.g = d.g; p.hpg = d.h_q / d.g; p.d_h = d.d_h; p.r_kv = d.r_kv; p.d_r = d.d_r;
    p.out0 = k_c; p.out1 = v; p.aux_in = cache; p.aux_out = k_r; p.aux_stride = cache_row_stride;
    p.status = projection_status_word();
    // 128 x 256 output tiles (two adjacent groups) when g is even: the 128-row latent tile is then re-read
    // through L2 by g CTAs instead of 2g
    cudaError_t e = (d.g % 2 == 0)
                        ? tc::gemm_launch<tc::kGemmExpand, 256, true>(p, tmA, tmK, tmV, dim3((unsigned)(m_tiles * d.g)), st)
                        : tc::gemm_launch<tc::kGemmExpand, 128, true>(p, tmA, tmK, tmV, dim3((unsigned)(m_tiles * 2 * d.g)),
                                                                      st);
    return e == cudaSuccess ? GQLA_OK : GQLA_ERR_CUDA;
}

// 4-D view of a [B*s_q, h_q, feat] activation: (feat, head-in-group, group, position).
inline bool make_grouped_act_map(CUtensorMap* m, const void* base, const gqla_dims& d, int feat, int64_t positions,
                                 int tile_rows = 128) {
    const int hpg = d.h_q / d.g, hpb = next_pow2(hpg);
    const uint64_t dims[4] = {(uint64_t)feat, (uint64_t)hpg, (uint64_t)d.g, (uint64_t)positions};
    const uint64_t str[3] = {(uint64_t)feat * 2, (uint64_t)hpg * feat * 2, (uint64_t)d.h_q * feat * 2};
    const uint32_t box[4] = {64, (uint32_t)hpb, 1, (uint32_t)(tile_rows / hpb)};  // beyond the hpg heads: zero fill
    return tc::make_tmap_bf16(m, base, 4, dims, str, box);
}

inline gqla_status tc_absorb_q(const gqla_dims& d, gqla_dtype dtype, int32_t B, int32_t s_q, const void* q_c,
                               const void* q_r, const void* w_uk, void* q_hat, cudaStream_t st) {
    if (!tc_gemm_covers(d, dtype)) return GQLA_ERR_UNSUPPORTED;
    const int hpg = d.h_q / d.g, hpb = next_pow2(hpg);
    const int64_t positions = (int64_t)B * s_q;
    const int64_t m_tiles = (positions + 128 / hpb - 1) / (128 / hpb);
    if (m_tiles > 0x7fffffffLL) return GQLA_ERR_UNSUPPORTED;
    CUtensorMap tmA, tmB;
    if (!make_grouped_act_map(&tmA, q_c, d, d.d_h, positions)) return GQLA_ERR_CUDA;
    {
        // W_UK[j] as a K-major B operand: rows = (j, r), columns = d (contraction)
        const uint64_t dims[2] = {(uint64_t)d.d_h, (uint64_t)d.g * d.r_kv};
        const uint64_t str[1] = {(uint64_t)d.d_h * 2};
        const uint32_t box[2] = {64, 256};
        if (!tc::make_tmap_bf16(&tmB, w_uk, 2, dims, str, box)) return GQLA_ERR_CUDA;
    }
    tc::GemmParams p{};
    p.k_blocks = d.d_h / 64;
    p.m_total = positions;
    p.h_q = d.h_q; p.g = d.g; p.hpg = hpg; p.hpb = hpb; p.d_h = d.d_h; p.r_kv = d.r_kv; p.d_r = d.d_r;
    p.out0 = q_hat; p.aux_in = q_r; p.status = projection_status_word();
    cudaError_t e = tc::gemm_launch<tc::kGemmAbsorbQ, 256, false>(
        p, tmA, tmB, tmB, dim3((unsigned)m_tiles, (unsigned)d.g, (unsigned)(d.r_kv / 256)), st);
    return e == cudaSuccess ? GQLA_OK : GQLA_ERR_CUDA;
}

inline gqla_status tc_up_proj(const gqla_dims& d, gqla_dtype dtype, int32_t B, int32_t s_q, const void* o_hat,
                              const void* w_uv, void* o, cudaStream_t st) {
    if (!tc_gemm_covers(d, dtype)) return GQLA_ERR_UNSUPPORTED;
    const int hpg = d.h_q / d.g, hpb = next_pow2(hpg);
    const int64_t positions = (int64_t)B * s_q;
    // 64-row tiles where a group's head slots allow: this kernel is bound by what one CTA pulls of o_hat (r_kv columns
    // per row), and the 128-row tiling leaves more than half of the SMs idle at the shapes of a decode step
    const int bm = hpb <= 64 ? 64 : 128;
    const int64_t m_tiles = (positions + bm / hpb - 1) / (bm / hpb);
    if (m_tiles > 0x7fffffffLL) return GQLA_ERR_UNSUPPORTED;
    CUtensorMap tmA, tmB;
    if (!make_grouped_act_map(&tmA, o_hat, d, d.r_kv, positions, bm)) return GQLA_ERR_CUDA;
    {
        // W_UV[j] as an MN-major B operand: rows = (j, r) (contraction), columns = d (output)
        const uint64_t dims[2] = {(uint64_t)d.d_h, (uint64_t)d.g * d.r_kv};
        const uint64_t str[1] = {(uint64_t)d.d_h * 2};
        const uint32_t box[2] = {64, 64};
        if (!tc::make_tmap_bf16(&tmB, w_uv, 2, dims, str, box)) return GQLA_ERR_CUDA;
    }
    tc::GemmParams p{};
    p.k_blocks = d.r_kv / 64;
    p.m_total = positions;
    p.h_q = d.h_q; p.g = d.g; p.hpg = hpg; p.hpb = hpb; p.d_h = d.d_h; p.r_kv = d.r_kv; p.d_r = d.d_r;
    p.out0 = o; p.status = projection_status_word();
    const dim3 grid((unsigned)m_tiles, (unsigned)d.g, 1);
    cudaError_t e = bm == 64 ? tc::gemm_launch<tc::kGemmUpProj, 128, true, 64>(p, tmA, tmB, tmB, grid, st)
                             : tc::gemm_launch<tc::kGemmUpProj, 128, true, 128>(p, tmA, tmB, tmB, grid, st);
    return e == cudaSuccess ? GQLA_OK : GQLA_ERR_CUDA;
}

// Expansion of the step's new rows; covers bf16, d_h = 128, r_kv a multiple of 128 up to 512, d_r a multiple of 8.
inline gqla_status tc_append_expand(const gqla_dims& d, gqla_dtype dtype, int32_t B, int32_t s_q, const void* cache,
                                    int64_t cache_row_stride, const int64_t* seq_start, const int32_t* seqlens,
                                    const void* w_uk, const void* w_uv, void* k_c, void* v, void* k_r, cudaStream_t st) {
    if (dtype != GQLA_BF16 || d.d_h != 128 || d.r_kv % tc::AppendSmem::kChunkK != 0 ||
        d.r_kv > tc::AppendSmem::kMaxChunks * tc::AppendSmem::kChunkK || d.d_r % 8 != 0 || d.d_r > 256 ||
        !stride_ok(cache_row_stride) || 2 * d.g > 65535)
        return GQLA_ERR_UNSUPPORTED;
    const int64_t m_tiles = ((int64_t)B * s_q + tc::AppendSmem::kRows - 1) / tc::AppendSmem::kRows;
    if (m_tiles > 0x7fffffffLL) return GQLA_ERR_UNSUPPORTED;
    CUtensorMap tmK, tmV;
    {
        // W[j] as an MN-major B operand: rows = (j, r) (contraction), columns = d (output)
        const uint64_t dims[2] = {(uint64_t)d.d_h, (uint64_t)d.g * d.r_kv};
        const uint64_t str[1] = {(uint64_t)d.d_h * 2};
        const uint32_t box[2] = {64, 64};
        if (!tc::make_tmap_bf16(&tmK, w_uk, 2, dims, str, box)) return GQLA_ERR_CUDA;
        if (!tc::make_tmap_bf16(&tmV, w_uv, 2, dims, str, box)) return GQLA_ERR_CUDA;
    }
    tc::AppendParams p{};
    p.B = B; p.s_q = s_q; p.g = d.g; p.r_kv = d.r_kv; p.d_r = d.d_r;
    p.cache = (const __nv_bfloat16*)cache; p.cache_stride = cache_row_stride;
    p.seq_start = seq_start; p.seqlens = seqlens;
    p.k_c = (__nv_bfloat16*)k_c; p.v = (__nv_bfloat16*)v; p.k_r = (__nv_bfloat16*)k_r; p.status = projection_status_word();
    auto kern = tc::append_expand_tc_kernel;
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::AppendSmem::kTotal) != cudaSuccess)
            return GQLA_ERR_CUDA;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    return tc::launch_pdl(kern, dim3((unsigned)m_tiles, (unsigned)(2 * d.g), 1), dim3(tc::AppendSmem::kThreads),
                          tc::AppendSmem::kTotal, st, p, tmK, tmV) == cudaSuccess
               ? GQLA_OK
               : GQLA_ERR_CUDA;
}

// Fused split merge + up-projection; covers what tc_up_proj covers with d_h = 128 and r_kv % 128 == 0.
inline gqla_status tc_combine_up_proj(const gqla_dims& d, gqla_dtype dtype, int32_t B, int32_t s_q, int32_t S,
                                      const float* o_part, const float* lse_part, const void* w_uv, void* o, float* lse,
                                      cudaStream_t st) {
    const int hpg = d.h_q / d.g, hpb = next_pow2(hpg);
    if (!tc_gemm_covers(d, dtype) || S > tc::CombineUpSmem::kMaxS || hpb > 64 ||
        d.r_kv > tc::CombineUpSmem::kMaxChunks * tc::CombineUpSmem::kChunkK)
        return GQLA_ERR_UNSUPPORTED;
    const int64_t positions = (int64_t)B * s_q;
    const int64_t m_tiles = (positions + 64 / hpb - 1) / (64 / hpb);
    if (m_tiles > 0x7fffffffLL) return GQLA_ERR_UNSUPPORTED;
    CUtensorMap tmB;
    {
        const uint64_t dims[2] = {(uint64_t)d.d_h, (uint64_t)d.g * d.r_kv};
        const uint64_t str[1] = {(uint64_t)d.d_h * 2};
        const uint32_t box[2] = {64, 64};
        if (!tc::make_tmap_bf16(&tmB, w_uv, 2, dims, str, box)) return GQLA_ERR_CUDA;
    }
    tc::CombineUpParams p{};
    p.S = S; p.s_q = s_q; p.h_q = d.h_q; p.g = d.g; p.hpg = hpg; p.hpb = hpb; p.r_kv = d.r_kv;
    p.positions = positions; p.o_part = o_part; p.lse_part = lse_part; p.out = o; p.lse = lse; p.status = projection_status_word();
    auto kern = tc::combine_up_tc_kernel;
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::CombineUpSmem::kTotal) != cudaSuccess)
            return GQLA_ERR_CUDA;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    return tc::launch_pdl(kern, dim3((unsigned)m_tiles, (unsigned)d.g, 1), dim3(tc::CombineUpSmem::kThreads),
                          tc::CombineUpSmem::kTotal, st, p, tmB) == cudaSuccess
               ? GQLA_OK
               : GQLA_ERR_CUDA;
}

template <int R>
inline cudaError_t absorb_t_launch(const tc::AbsorbParams& p, const CUtensorMap& q, const CUtensorMap& c, unsigned grid,
                                   cudaStream_t st) {
    auto kern = tc::decode_absorb_t_kernel<R>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::AbsorbTSmem<R>::kTotal);
    if (e != cudaSuccess) return e;
    return tc::launch_pdl(kern, dim3(grid), dim3(tc::AbsorbTSmem<R>::kThreads), tc::AbsorbTSmem<R>::kTotal, st, p, q, c);
}

inline gqla_status tc_decode_absorb(const gqla_dims& d, int32_t B, int32_t s_q, float scale, int32_t S,
                                    const void* q_hat, const void* cache, int64_t cache_row_stride,
                                    int64_t cache_rows, const RowMap& rows, const int32_t* seqlens,
                                    float* o_part, float* lse_part, int32_t* status, cudaStream_t st,
                                    void* o_final = nullptr) {
    if (!tc_covers(d, GQLA_BF16, s_q, 0) || !stride_ok(cache_row_stride) || cache_rows > 0x7fffffffLL ||
        cache_rows < 1)
        return GQLA_ERR_UNSUPPORTED;
    if (rows.paged() && rows.page_size % kTileRows != 0) return GQLA_ERR_UNSUPPORTED;  // a tile must not straddle pages
    const int rows_total = s_q * d.h_q;
    const int row_blocks = (rows_total + 127) / 128;
    // S < 0: balanced plan with -S slots per sequence, W persistent pairs per row block
    const int32_t workers = S < 0 ? tc_balanced_workers(d, s_q, 0) : 0;
    const bool balanced = S < 0 && workers > 0;
    if (S < 0) S = -S;
    // paged: pieces must start on tile boundaries, which the fixed plan's 64-row granule does not give for S > 1
    if (rows.paged() && !balanced && S != 1) return GQLA_ERR_UNSUPPORTED;
    const int64_t pairs = balanced ? (int64_t)workers * row_blocks : (int64_t)B * S * row_blocks;
    if (2 * pairs > 0x7fffffffLL) return GQLA_ERR_UNSUPPORTED;
    const bool tokens_on_m = absorb_prefers_tokens(d, s_q);
    const int rows_t = absorb_rows_t(d, s_q);
    CUtensorMap tmQ, tmC;
    {
        const uint64_t dims[2] = {(uint64_t)(d.r_kv + d.d_r), (uint64_t)B * rows_total};
        const uint64_t str[1] = {(uint64_t)(d.r_kv + d.d_r) * 2};
        const uint32_t box[2] = {64, tokens_on_m ? (uint32_t)rows_t : 64u};  // beyond the last row: zero fill
        if (!tc::make_tmap_bf16(&tmQ, q_hat, 2, dims, str, box)) return GQLA_ERR_CUDA;
    }
    {
        const uint64_t dims[2] = {(uint64_t)(d.r_kv + d.d_r), (uint64_t)cache_rows};
        const uint64_t str[1] = {(uint64_t)cache_row_stride * 2};
        const uint32_t box[2] = {64, 64};
        if (!tc::make_tmap_bf16(&tmC, cache, 2, dims, str, box)) return GQLA_ERR_CUDA;
    }
    tc::AbsorbParams p{};
    p.B = B; p.S = S; p.s_q = s_q; p.h_q = d.h_q; p.rows_total = rows_total; p.row_blocks = row_blocks;
    p.balanced = balanced ? 1 : 0; p.W = workers;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.rows = rows; p.seqlens = seqlens; p.o_part = o_part; p.lse_part = lse_part; p.status = status;
    p.o_final = (__nv_bfloat16*)o_final;
    if (o_final != nullptr && (balanced || S != 1)) return GQLA_ERR_UNSUPPORTED;
    if (tokens_on_m) {
        const unsigned grid = (unsigned)(balanced ? workers : B * S);  // single CTAs: W of them, or one per piece
        const cudaError_t e = rows_t == 16   ? absorb_t_launch<16>(p, tmQ, tmC, grid, st)
                              : rows_t == 32 ? absorb_t_launch<32>(p, tmQ, tmC, grid, st)
                                             : absorb_t_launch<64>(p, tmQ, tmC, grid, st);
        return e == cudaSuccess ? GQLA_OK : GQLA_ERR_CUDA;
    }
    auto kern = tc::decode_absorb_tc_kernel<0>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::AbsorbSmem::kTotal) != cudaSuccess)
        return GQLA_ERR_CUDA;
    return tc::launch_pdl(kern, dim3((unsigned)(2 * pairs)), dim3(tc::AbsorbSmem::kThreads), tc::AbsorbSmem::kTotal, st, p,
                          tmQ, tmC) == cudaSuccess
               ? GQLA_OK
               : GQLA_ERR_CUDA;
}

// CTA pairs of the absorb kernel that can be resident at once on the current device (cached).
inline int absorb_resident_pairs() {
    static int cached[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
    if (cached[dev] == 0) {
        auto kern = tc::decode_absorb_tc_kernel<0>;
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::AbsorbSmem::kTotal) != cudaSuccess) {
            (void)cudaGetLastError();
            return 0;
        }
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(2 * 148, 1, 1);
        cfg.blockDim = dim3(tc::AbsorbSmem::kThreads, 1, 1);
        cfg.dynamicSmemBytes = tc::AbsorbSmem::kTotal;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, kern, &cfg) != cudaSuccess || n <= 0) {
            (void)cudaGetLastError();
            const int sms = sm_count();
            n = sms / 2;
        }
        cached[dev] = n;
    }
    return cached[dev];
}

// Rows of the tokens-on-M GQA kernel's query block: heads per group and query positions each padded to a power of
// two, at least 16 rows in all (the smallest N of an M = 128 MMA).
inline int gqa_rows_t(const gqla_dims& d, int32_t s_q, int* hpg_box, int* sq_box) {
    const int sb = next_pow2(s_q);
    int hb = next_pow2(d.h_q / d.g);
    if (hb * sb < 16) hb = 16 / sb;
    if (hpg_box != nullptr) *hpg_box = hb;
    if (sq_box != nullptr) *sq_box = sb;
    return hb * sb;
}

// Which GQA kernel serves a shape both cover: the tokens-on-M kernel (tc_decode_gqa_t.cuh) for few query rows per
// group, the row-replicating one beyond.  GQLA_GQA_KERNEL=rows|tokens in the environment overrides the choice for
// shapes both cover (read once per process; a tuning aid).
inline bool gqa_prefers_tokens(int rows_t) {
    static const int forced = []() {
        const char* e = getenv("GQLA_GQA_KERNEL");
        if (e == nullptr) return 0;
        return e[0] == 't' ? 1 : (e[0] == 'r' ? 2 : 0);
    }();
    if (rows_t > 64) return false;
    if (forced != 0) return forced == 1;
    return rows_t <= GQLA_GQA_TOKENS_MAX_ROWS;
}

template <int R>
inline cudaError_t gqa_t_launch(const tc::GqaParams& p, const CUtensorMap& q, const CUtensorMap& k, const CUtensorMap& r,
                                const CUtensorMap& v, unsigned grid, cudaStream_t st) {
    auto kern = tc::decode_gqa_t_kernel<R>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::GqaTSmem<R>::kTotal);
    if (e != cudaSuccess) return e;
    return tc::launch_pdl(kern, dim3(grid), dim3(tc::GqaTSmem<R>::kThreads), tc::GqaTSmem<R>::kTotal, st, p, q, k, r, v);
}

template <int R>
inline cudaError_t gqa_launch(const tc::GqaParams& p, const CUtensorMap& q, const CUtensorMap& k, const CUtensorMap& r,
                              const CUtensorMap& v, unsigned grid, cudaStream_t st) {
    auto kern = tc::decode_gqa_tc_kernel<R>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::GqaSmem::kTotal);
    if (e != cudaSuccess) return e;
    return tc::launch_pdl(kern, dim3(grid), dim3(tc::GqaSmem::kThreads), tc::GqaSmem::kTotal, st, p, q, k, r, v);
}

// d_v: value head dim, a multiple of 128 up to 512 (d_h when the shapes of Sec. 3.1 apply).  With d_v > 128 every
// (rows, group) unit is served by d_v / 128 CTAs, one per 128-column block of V and of the output; each of them
// computes the scores itself (the K tiles are shared through L2), which is the price of keeping one kernel.
inline gqla_status tc_decode_gqa(const gqla_dims& d, int32_t B, int32_t s_q, float scale, int32_t S, const void* q,
                                 const void* k_c, const void* v, const void* k_r, int64_t k_r_row_stride,
                                 int64_t n_rows, const RowMap& rows, const int32_t* seqlens, float* o_part,
                                 float* lse_part, int32_t* status, cudaStream_t st, int32_t d_v = 128) {
    if (!tc_covers(d, GQLA_BF16, s_q, 1) || !stride_ok(k_r_row_stride) || n_rows > 0x7fffffffLL || n_rows < 1 ||
        d_v % 128 != 0 || d_v < 128 || d_v > 512)
        return GQLA_ERR_UNSUPPORTED;
    const int v_blocks = d_v / 128;
    if (rows.paged() && rows.page_size % kTileRows != 0) return GQLA_ERR_UNSUPPORTED;  // a tile must not straddle pages
    // S < 0: balanced plan with -S slots per sequence, W persistent CTAs per (group, value block)
    const int32_t workers = S < 0 ? tc_balanced_workers(d, s_q, 1) / v_blocks : 0;
    const bool balanced = S < 0 && workers > 0;
    if (S < 0) S = -S;
    if (rows.paged() && !balanced && S != 1) return GQLA_ERR_UNSUPPORTED;  // see tc_decode_absorb
    const int64_t units = (balanced ? (int64_t)workers * d.g : (int64_t)B * S * d.g) * v_blocks;
    if (units > 0x7fffffffLL) return GQLA_ERR_UNSUPPORTED;
    const int hpg = d.h_q / d.g;
    int hpg_box = 0, sq_box = 0;
    int R = gqa_rows(d, s_q, &hpg_box, &sq_box);
    const bool tokens_on_m = gqa_prefers_tokens(gqa_rows_t(d, s_q, nullptr, nullptr));
    if (tokens_on_m) R = gqa_rows_t(d, s_q, &hpg_box, &sq_box);
    CUtensorMap tmQ, tmK, tmR, tmV;
    {
        const int feat = d.d_h + d.d_r;
        const uint64_t dims[4] = {(uint64_t)feat, (uint64_t)hpg, (uint64_t)d.g, (uint64_t)B * s_q};
        const uint64_t str[3] = {(uint64_t)feat * 2, (uint64_t)hpg * feat * 2, (uint64_t)d.h_q * feat * 2};
        const uint32_t box[4] = {64, (uint32_t)hpg_box, 1, (uint32_t)sq_box};  // beyond a dimension: zero fill
        if (!tc::make_tmap_bf16(&tmQ, q, 4, dims, str, box)) return GQLA_ERR_CUDA;
    }
    {
        const uint64_t dims[3] = {(uint64_t)d.d_h, (uint64_t)d.g, (uint64_t)n_rows};
        const uint64_t str[2] = {(uint64_t)d.d_h * 2, (uint64_t)d.g * d.d_h * 2};
        const uint64_t vdims[3] = {(uint64_t)d_v, (uint64_t)d.g, (uint64_t)n_rows};
        const uint64_t vstr[2] = {(uint64_t)d_v * 2, (uint64_t)d.g * d_v * 2};
        const uint32_t box[3] = {64, 1, 128};
        if (!tc::make_tmap_bf16(&tmK, k_c, 3, dims, str, box)) return GQLA_ERR_CUDA;
        if (!tc::make_tmap_bf16(&tmV, v, 3, vdims, vstr, box)) return GQLA_ERR_CUDA;
    }
    {
        const uint64_t dims[2] = {(uint64_t)d.d_r, (uint64_t)n_rows};
        const uint64_t str[1] = {(uint64_t)k_r_row_stride * 2};
        const uint32_t box[2] = {64, 128};
        if (!tc::make_tmap_bf16(&tmR, k_r, 2, dims, str, box)) return GQLA_ERR_CUDA;
    }
    tc::GqaParams p{};
    p.v_blocks = v_blocks; p.d_v = d_v;
    p.B = B; p.S = S; p.s_q = s_q; p.h_q = d.h_q; p.g = d.g; p.hpg = hpg; p.hpg_box = hpg_box;
    p.balanced = balanced ? 1 : 0; p.W = workers;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.rows = rows; p.seqlens = seqlens; p.o_part = o_part; p.lse_part = lse_part; p.status = status;
    cudaError_t e;
    if (tokens_on_m) {
        switch (R) {
            case 16: e = gqa_t_launch<16>(p, tmQ, tmK, tmR, tmV, (unsigned)units, st); break;
            case 32: e = gqa_t_launch<32>(p, tmQ, tmK, tmR, tmV, (unsigned)units, st); break;
            case 64: e = gqa_t_launch<64>(p, tmQ, tmK, tmR, tmV, (unsigned)units, st); break;
            default: return GQLA_ERR_UNSUPPORTED;
        }
        return e == cudaSuccess ? GQLA_OK : GQLA_ERR_CUDA;
    }
    switch (R) {
        case 8: e = gqa_launch<8>(p, tmQ, tmK, tmR, tmV, (unsigned)units, st); break;
        case 16: e = gqa_launch<16>(p, tmQ, tmK, tmR, tmV, (unsigned)units, st); break;
        case 32: e = gqa_launch<32>(p, tmQ, tmK, tmR, tmV, (unsigned)units, st); break;
        case 64: e = gqa_launch<64>(p, tmQ, tmK, tmR, tmV, (unsigned)units, st); break;
        case 128: e = gqa_launch<128>(p, tmQ, tmK, tmR, tmV, (unsigned)units, st); break;
        default: return GQLA_ERR_UNSUPPORTED;
    }
    return e == cudaSuccess ? GQLA_OK : GQLA_ERR_CUDA;
}

// Absorb path over an E4M3 latent cache; covers what the bf16 pair kernel covers (r_kv = 512, d_r = 64).
inline gqla_status tc_decode_absorb_fp8(const gqla_dims& d, int32_t B, int32_t s_q, float scale, int32_t S, const uint8_t* q8,
                                        const float* q_scale, const uint8_t* cache8, int64_t cache_row_stride,
                                        int64_t cache_rows, float v_scale, const RowMap& rows, const int32_t* seqlens,
                                        float* o_part, float* lse_part, int32_t* status, cudaStream_t st,
                                        void* o_final = nullptr) {
    if (!tc_covers(d, GQLA_BF16, s_q, 0) || cache_row_stride % 16 != 0 || cache_rows > 0x7fffffffLL || cache_rows < 1)
        return GQLA_ERR_UNSUPPORTED;
    const int rows_total = s_q * d.h_q;
    const int row_blocks = (rows_total + 127) / 128;
    const int32_t workers = S < 0 ? pair_balanced_workers(d, s_q) : 0;
    const bool balanced = S < 0 && workers > 0;
    if (S < 0) S = -S;
    const int64_t pairs = balanced ? (int64_t)workers * row_blocks : (int64_t)B * S * row_blocks;
    if (2 * pairs > 0x7fffffffLL) return GQLA_ERR_UNSUPPORTED;
    CUtensorMap tmQ, tmQr, tmC, tmCr;
    {
        const uint64_t dims[2] = {(uint64_t)(d.r_kv + d.d_r), (uint64_t)B * rows_total};
        const uint64_t str[1] = {(uint64_t)(d.r_kv + d.d_r)};
        const uint32_t box[2] = {128, 64}, box_r[2] = {64, 64};
        if (!tc::make_tmap_u8(&tmQ, q8, 2, dims, str, box, CU_TENSOR_MAP_SWIZZLE_128B)) return GQLA_ERR_CUDA;
        if (!tc::make_tmap_u8(&tmQr, q8, 2, dims, str, box_r, CU_TENSOR_MAP_SWIZZLE_64B)) return GQLA_ERR_CUDA;
    }
    {
        const uint64_t dims[2] = {(uint64_t)(d.r_kv + d.d_r), (uint64_t)cache_rows};
        const uint64_t str[1] = {(uint64_t)cache_row_stride};
        const uint32_t box[2] = {128, 64}, box_r[2] = {64, 64};
        if (!tc::make_tmap_u8(&tmC, cache8, 2, dims, str, box, CU_TENSOR_MAP_SWIZZLE_128B)) return GQLA_ERR_CUDA;
        if (!tc::make_tmap_u8(&tmCr, cache8, 2, dims, str, box_r, CU_TENSOR_MAP_SWIZZLE_64B)) return GQLA_ERR_CUDA;
    }
    tc::AbsorbFp8Params p{};
    p.B = B; p.S = S; p.s_q = s_q; p.h_q = d.h_q; p.rows_total = rows_total; p.row_blocks = row_blocks;
    p.balanced = balanced ? 1 : 0; p.W = workers;
    p.scale_log2 = scale * 1.4426950408889634f; p.v_scale = v_scale; p.q_scale = q_scale;
    p.rows = rows; p.seqlens = seqlens; p.o_part = o_part; p.lse_part = lse_part; p.status = status;
    p.o_final = (__nv_bfloat16*)o_final;
    if (o_final != nullptr && (balanced || S != 1)) return GQLA_ERR_UNSUPPORTED;
    auto kern = tc::decode_absorb_fp8_tc_kernel<0>;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::AbsorbFp8Smem::kTotal) != cudaSuccess)
        return GQLA_ERR_CUDA;
    return tc::launch_pdl(kern, dim3((unsigned)(2 * pairs)), dim3(tc::AbsorbFp8Smem::kThreads), tc::AbsorbFp8Smem::kTotal, st,
                          p, tmQ, tmQr, tmC, tmCr) == cudaSuccess
               ? GQLA_OK
               : GQLA_ERR_CUDA;
}

template <int R>
inline cudaError_t gqa_fp8_launch(const tc::GqaFp8Params& p, const CUtensorMap& qc, const CUtensorMap& qr, const CUtensorMap& k,
                                  const CUtensorMap& r, const CUtensorMap& v, unsigned grid, cudaStream_t st) {
    auto kern = tc::decode_gqa_fp8_tc_kernel<R>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::GqaFp8Smem::kTotal);
    if (e != cudaSuccess) return e;
    return tc::launch_pdl(kern, dim3(grid), dim3(tc::GqaFp8Smem::kThreads), tc::GqaFp8Smem::kTotal, st, p, qc, qr, k, r, v);
}

// GQA path over E4M3 planes; covers what the bf16 tensor-core kernel covers (d_h = 128, d_r = 64, at most 128 rows
// per group).  Strides are in bytes here (one byte per element) and must be multiples of 16.
inline gqla_status tc_decode_gqa_fp8(const gqla_dims& d, int32_t B, int32_t s_q, float scale, int32_t S, const uint8_t* q8,
                                     const float* q_scale, const uint8_t* k_c8, const uint8_t* v8, const uint8_t* k_r8,
                                     int64_t k_r_row_stride, int64_t n_rows, float v_scale, const RowMap& rows,
                                     const int32_t* seqlens, float* o_part, float* lse_part, int32_t* status,
                                     cudaStream_t st) {
    if (!tc_covers(d, GQLA_BF16, s_q, 1) || k_r_row_stride % 16 != 0 || n_rows > 0x7fffffffLL || n_rows < 1)
        return GQLA_ERR_UNSUPPORTED;
    const int32_t workers = S < 0 ? tc_balanced_workers(d, s_q, 1) : 0;
    const bool balanced = S < 0 && workers > 0;
    if (S < 0) S = -S;
    const int64_t units = balanced ? (int64_t)workers * d.g : (int64_t)B * S * d.g;
    if (units > 0x7fffffffLL) return GQLA_ERR_UNSUPPORTED;
    const int hpg = d.h_q / d.g;
    int hpg_box = 0, sq_box = 0;
    const int R = gqa_rows(d, s_q, &hpg_box, &sq_box);
    CUtensorMap tmQc, tmQr, tmK, tmR, tmV;
    {
        const int feat = d.d_h + d.d_r;
        const uint64_t dims[4] = {(uint64_t)feat, (uint64_t)hpg, (uint64_t)d.g, (uint64_t)B * s_q};
        const uint64_t str[3] = {(uint64_t)feat, (uint64_t)hpg * feat, (uint64_t)d.h_q * feat};
        const uint32_t box_c[4] = {128, (uint32_t)hpg_box, 1, (uint32_t)sq_box};
        const uint32_t box_r[4] = {64, (uint32_t)hpg_box, 1, (uint32_t)sq_box};
        if (!tc::make_tmap_u8(&tmQc, q8, 4, dims, str, box_c, CU_TENSOR_MAP_SWIZZLE_128B)) return GQLA_ERR_CUDA;
        if (!tc::make_tmap_u8(&tmQr, q8, 4, dims, str, box_r, CU_TENSOR_MAP_SWIZZLE_64B)) return GQLA_ERR_CUDA;
    }
    {
        const uint64_t dims[3] = {(uint64_t)d.d_h, (uint64_t)d.g, (uint64_t)n_rows};
        const uint64_t str[2] = {(uint64_t)d.d_h, (uint64_t)d.g * d.d_h};
        const uint32_t box[3] = {128, 1, 128};
        if (!tc::make_tmap_u8(&tmK, k_c8, 3, dims, str, box, CU_TENSOR_MAP_SWIZZLE_128B)) return GQLA_ERR_CUDA;
        if (!tc::make_tmap_u8(&tmV, v8, 3, dims, str, box, CU_TENSOR_MAP_SWIZZLE_128B)) return GQLA_ERR_CUDA;
    }
    {
        const uint64_t dims[2] = {(uint64_t)d.d_r, (uint64_t)n_rows};
        const uint64_t str[1] = {(uint64_t)k_r_row_stride};
        const uint32_t box[2] = {64, 128};
        if (!tc::make_tmap_u8(&tmR, k_r8, 2, dims, str, box, CU_TENSOR_MAP_SWIZZLE_64B)) return GQLA_ERR_CUDA;
    }
    tc::GqaFp8Params p{};
    p.B = B; p.S = S; p.s_q = s_q; p.h_q = d.h_q; p.g = d.g; p.hpg = hpg; p.hpg_box = hpg_box;
    p.balanced = balanced ? 1 : 0; p.W = workers;
    p.scale_log2 = scale * 1.4426950408889634f; p.v_scale = v_scale; p.q_scale = q_scale;
    p.rows = rows; p.seqlens = seqlens; p.o_part = o_part; p.lse_part = lse_part; p.status = status;
    cudaError_t e;
    switch (R) {
        case 8: e = gqa_fp8_launch<8>(p, tmQc, tmQr, tmK, tmR, tmV, (unsigned)units, st); break;
        case 16: e = gqa_fp8_launch<16>(p, tmQc, tmQr, tmK, tmR, tmV, (unsigned)units, st); break;
        case 32: e = gqa_fp8_launch<32>(p, tmQc, tmQr, tmK, tmR, tmV, (unsigned)units, st); break;
        case 64: e = gqa_fp8_launch<64>(p, tmQc, tmQr, tmK, tmR, tmV, (unsigned)units, st); break;
        case 128: e = gqa_fp8_launch<128>(p, tmQc, tmQr, tmK, tmR, tmV, (unsigned)units, st); break;
        default: return GQLA_ERR_UNSUPPORTED;
    }
    return e == cudaSuccess ? GQLA_OK : GQLA_ERR_CUDA;
}

}  // namespace gqla
