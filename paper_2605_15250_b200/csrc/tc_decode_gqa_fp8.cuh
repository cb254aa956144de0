// GQA-path split-KV flash decoding over an FP8 (E4M3) expanded cache on tcgen05 (Eq. (mha); KV-cache
// quantisation is among the effects the paper's model leaves out, Sec. 5.1 "Limitations").  Same structure as
// the bf16 kernel of tc_decode_gqa.cuh -- one CTA per group, R query rows replicated F = 128/R times down the
// 128-row MMA tile, replica f keeping the scores of tokens [f*R, (f+1)*R) of every 128-token tile, P handed
// to the P.V MMA through tensor memory -- with what one byte per element changes:
//
//   * MMAs are kind::f8f6f4 (E4M3 x E4M3 -> fp32), K = 32 elements per instruction: S = Q K^T takes 4 MMAs over
//     the 128-wide K_C part and 2 over the 64-wide k_R part, O += P V takes 4.
//   * A tile stage is 40 KB (K_C 16 KB, k_R 8 KB, V 16 KB), so the ring holds four tiles instead of two: twice
//     the tiles in flight for the same bytes, which is what a memory-bound kernel wants when every tile is
//     half as large.  The 64-byte rows of the k_R and q^R tiles use the 64-byte swizzle, everything else the
//     128-byte one.
//   * Scores are scaled per query row (q_scale folds the key planes' scales in), outputs by v_scale.
//   * P is rounded to E4M3 (4 significant bits; smallest positive value 2^-9, largest 448).  A replica's softmax
//     reference is put kF8Bias = 6 binades BELOW the tile maximum that raised it and raised again when a tile's
//     maximum exceeds it by more than 8.75: P <= 430, and terms down to 2^-15 of the largest one count right after a
//     raise (2^-17.75 before the next).  A raise rescales O and has to wait for the previous tile's P.V, so it is
//     kept rare; following the maximum within one binade rescaled on a large share of the tiles.
#pragma once
#include "common.cuh"
#include "sched.cuh"
#include "tc_common.cuh"

namespace gqla {
namespace tc {

struct GqaFp8Params {
    int32_t B, S, s_q, h_q, g, hpg, hpg_box;
    int32_t balanced, W;
    float scale_log2, v_scale;
    const float* q_scale;  // [B, s_q, h_q]
    RowMap rows;
    const int32_t* seqlens;
    float* o_part;    // [B, S, s_q, h_q, 128]
    float* lse_part;  // [B, S, s_q, h_q]
    int32_t* status;
};

struct GqaFp8Smem {
    static constexpr int kQcBytes = 16384;                   // 128 rows x 128 E4M3 (K_C part), 128-byte swizzle
    static constexpr int kQrBytes = 8192;                    // 128 rows x 64 E4M3 (RoPE part), 64-byte swizzle
    static constexpr int kQBytes = kQcBytes + kQrBytes;
    static constexpr int kKcBytes = 16384;                   // 128 tokens x 128
    static constexpr int kKrBytes = 8192;                    // 128 tokens x 64
    static constexpr int kVBytes = 16384;                    // 128 tokens x 128
    static constexpr int kStageBytes = kKcBytes + kKrBytes + kVBytes;
    static constexpr int kStages = 4;
    static constexpr int kMergePitch = 36;
    static constexpr int kMergeBytes = 128 * kMergePitch * 4;
    static constexpr int kOffMerge = kQBytes + kStages * kStageBytes;
    static constexpr int kTileBytes = kOffMerge + kMergeBytes;
    // q_full q_empty o_free kfull[4] vfull[4] kempty[4] vempty[4] s_full[2] p_ready[2] pv_done[2]
    static constexpr int kNumBars = 3 + 4 * kStages + 6;
    static constexpr int kThreads = 192;
    static constexpr int kTotal = kTileBytes + kNumBars * 8 + 16;
    static_assert(kMergeBytes >= (kThreads + 4) * 4, "plan scratch must fit in the merge buffer");
    static_assert(kTotal <= 232448, "shared memory budget of one CTA");
    static_assert(OneCtaPerSM<kTotal>::value, "");
};

constexpr uint32_t kF8ColS = 0;    // two 128-column score buffers
constexpr uint32_t kF8ColP = 256;  // two 32-column E4M3 probability buffers (four per 32-bit column)
constexpr uint32_t kF8ColO = 384;  // 128-column output accumulator
constexpr float kF8Bias = 6.0f;    // log2 units a raised softmax reference sits below the maximum that raised it
constexpr float kF8Grow = 8.75f;   // a score this far above its reference raises it (2^8.75 = 430 < 448)

// K-major operand tile with 64-byte swizzle: rows of 64 bytes, 8-row groups 512 B apart.
__device__ __forceinline__ uint64_t desc_kmajor_sw64(uint32_t smem_addr) {
    return (1ull << 46) | (4ull << 61) | (uint64_t)((smem_addr & 0x3FFFF) >> 4) | (1ull << 16) | ((uint64_t)(512 >> 4) << 32);
}
// Instruction descriptor for kind::f8f6f4 with E4M3 operands (format code 0) and fp32 accumulation.
__host__ __device__ constexpr uint32_t idesc_e4m3(uint32_t M, uint32_t N, uint32_t a_mn_major, uint32_t b_mn_major) {
    return (1u << 4) | (a_mn_major << 15) | (b_mn_major << 16) | ((N >> 3) << 17) | ((M >> 4) << 24);
}
__device__ __forceinline__ void umma_f8_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                           uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// A from tensor memory: one row per lane, four E4M3 per 32-bit column (K = 32 -> 8 columns).
__device__ __forceinline__ void umma_f8_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                           uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Four probabilities -> one 32-bit column (byte k = element k).
__device__ __forceinline__ uint32_t pack_e4m3x4(float e0, float e1, float e2, float e3) {
    return (uint32_t)float2_to_e4m3x2(e0, e1) | ((uint32_t)float2_to_e4m3x2(e2, e3) << 16);
}

template <int R>
__global__ void __launch_bounds__(GqaFp8Smem::kThreads, 1)
decode_gqa_fp8_tc_kernel(const GqaFp8Params p, const __grid_constant__ CUtensorMap tmQc,
                         const __grid_constant__ CUtensorMap tmQr, const __grid_constant__ CUtensorMap tmK,
                         const __grid_constant__ CUtensorMap tmR, const __grid_constant__ CUtensorMap tmV) {
    using L = GqaFp8Smem;
    constexpr int F = 128 / R;
    constexpr int W = R < 32 ? 32 : R;   // columns of S a warp reads per tile
    constexpr int CH = 32;
    constexpr int NCH = W / CH;
    constexpr int NS = L::kStages;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* tiles = smem_raw;
    if ((smem_u32(tiles) & 1023u) != 0) {  // swizzled tiles need 1 KB alignment
        if (threadIdx.x == 0 && p.status != nullptr) atomicCAS(p.status, 0, kStatusTimeout | (15 << 8));
        return;
    }
    uint8_t* qc_smem = tiles;
    uint8_t* qr_smem = tiles + L::kQcBytes;
    uint8_t* stage0 = tiles + L::kQBytes;
    float* merge = reinterpret_cast<float*>(tiles + L::kOffMerge);
    uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + L::kTileBytes);
    uint64_t* q_full = bars + 0;
    uint64_t* q_empty = bars + 1;
    uint64_t* o_free = bars + 2;
    uint64_t* kfull = bars + 3;
    uint64_t* vfull = kfull + NS;
    uint64_t* kempty = vfull + NS;
    uint64_t* vempty = kempty + NS;
    uint64_t* s_full = vempty + NS;   // [2]
    uint64_t* p_ready = s_full + 2;   // [2]
    uint64_t* pv_done = p_ready + 2;  // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + L::kNumBars);
    volatile int32_t* abort_flag = reinterpret_cast<volatile int32_t*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const Abort ab{abort_flag, p.status};

    if (threadIdx.x == 0) {
        for (int i = 0; i < L::kNumBars; ++i) {
            const bool per_warp = (&bars[i] == o_free) || (&bars[i] == &p_ready[0]) || (&bars[i] == &p_ready[1]);
            mbar_init(&bars[i], per_warp ? 4 : 1);
        }
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }

    pdl_launch_dependents();
    pdl_wait();
    const int j = blockIdx.x % p.g;
    Walker walk;
    if (p.balanced) {
        const BalancedStart st = balanced_prepass(p.seqlens, p.B, p.S, blockIdx.x / p.g, p.W,
                                                  reinterpret_cast<int32_t*>(merge), L::kThreads);
        walk.init_balanced(p.seqlens, p.B, p.S, blockIdx.x / p.g, p.W, st);
    } else {
        const int unit = blockIdx.x / p.g;
        walk.init_fixed(p.seqlens, p.B, p.S, unit / p.S, unit % p.S);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    Piece pc;
    int gt = 0;  // tiles walked so far: ring slot = gt % NS, ring phase = (gt / NS) & 1; S/P buffer = gt & 1
    int pi = 0;  // non-empty pieces walked so far

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (elect_one()) {
            tma_prefetch_desc(&tmQc);
            tma_prefetch_desc(&tmQr);
            tma_prefetch_desc(&tmK);
            tma_prefetch_desc(&tmR);
            tma_prefetch_desc(&tmV);
            bool ok = true;
            while (ok && walk.next(pc)) {
                if (pc.n_tiles == 0) continue;
                if (pi > 0 && !(ok = mbar_wait(q_empty, (pi - 1) & 1, ab, 13))) break;
                mbar_expect_tx(q_full, L::kQBytes);
                for (int f = 0; f < F; ++f) {
                    asm volatile(
                        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], "
                        "[%1, {%3, %4, %5, %6}], [%2];" ::"r"(smem_u32(qc_smem + f * R * 128)),
                        "l"(reinterpret_cast<uint64_t>(&tmQc)), "r"(smem_u32(q_full)), "r"(0), "r"(0), "r"(j),
                        "r"(pc.b * p.s_q)
                        : "memory");
                    asm volatile(
                        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], "
                        "[%1, {%3, %4, %5, %6}], [%2];" ::"r"(smem_u32(qr_smem + f * R * 64)),
                        "l"(reinterpret_cast<uint64_t>(&tmQr)), "r"(smem_u32(q_full)), "r"(128), "r"(0), "r"(j),
                        "r"(pc.b * p.s_q)
                        : "memory");
                }
                int64_t tile_row = p.rows.row(pc.b, pc.tok_begin);
                for (int t = 0; t < pc.n_tiles; ++t, ++gt) {
                    const int s = gt % NS;
                    const uint32_t ph = (gt / NS) & 1;
                    uint8_t* st = stage0 + s * L::kStageBytes;
                    const int32_t row = (int32_t)tile_row;
                    if (t + 1 < pc.n_tiles)
                        tile_row = p.rows.paged() ? p.rows.row(pc.b, pc.tok_begin + (t + 1) * 128) : tile_row + 128;
                    if (!(ok = mbar_wait(&kempty[s], ph ^ 1, ab, 1))) break;
                    mbar_expect_tx(&kfull[s], L::kKcBytes + L::kKrBytes);
                    tma_load_3d(st, &tmK, 0, j, row, &kfull[s]);
                    tma_load_2d(st + L::kKcBytes, &tmR, 0, row, &kfull[s]);
                    if (!(ok = mbar_wait(&vempty[s], ph ^ 1, ab, 2))) break;
                    mbar_expect_tx(&vfull[s], L::kVBytes);
                    tma_load_3d(st + L::kKcBytes + L::kKrBytes, &tmV, 0, j, row, &vfull[s]);
                }
                ++pi;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (elect_one()) {
            constexpr uint32_t idesc_qk = idesc_e4m3(128, 128, 0, 0);
            constexpr uint32_t idesc_pv = idesc_e4m3(128, 128, 0, 1);
            const uint32_t qc_addr = smem_u32(qc_smem), qr_addr = smem_u32(qr_smem);
            auto issue_qk = [&](int n) -> bool {
                const int s = n % NS;
                if (!mbar_wait(&kfull[s], (n / NS) & 1, ab, 3)) return false;
                tc_fence_after();
                const uint32_t st = smem_u32(stage0 + s * L::kStageBytes);
                const uint32_t d = tmem_base + kF8ColS + (uint32_t)(n & 1) * 128;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)  // K_C part: 128 elements = 4 x 32
                    umma_f8_ss(d, desc_kmajor_sw128(qc_addr + ks * 32), desc_kmajor_sw128(st + ks * 32), idesc_qk, ks != 0);
#pragma unroll
                for (int ks = 0; ks < 2; ++ks)  // k_R part: 64 elements = 2 x 32
                    umma_f8_ss(d, desc_kmajor_sw64(qr_addr + ks * 32), desc_kmajor_sw64(st + L::kKcBytes + ks * 32), idesc_qk, 1);
                umma_commit(&s_full[n & 1]);
                umma_commit(&kempty[s]);
                return true;
            };
            bool ok = true;
            while (ok && walk.next(pc)) {
                if (pc.n_tiles == 0) continue;
                if (!(ok = mbar_wait(q_full, pi & 1, ab, 4))) break;
                tc_fence_after();
                if (!(ok = issue_qk(gt))) break;
                for (int t = 0; t < pc.n_tiles && ok; ++t) {
                    const int n = gt + t;
                    const int s = n % NS;
                    if (t + 1 < pc.n_tiles) {
                        if (!(ok = issue_qk(n + 1))) break;
                    } else {
                        umma_commit(q_empty);
                    }
                    if (!(ok = mbar_wait(&p_ready[n & 1], (n >> 1) & 1, ab, 5))) break;
                    if (t == 0 && pi > 0 && !(ok = mbar_wait(o_free, (pi - 1) & 1, ab, 14))) break;
                    if (!(ok = mbar_wait(&vfull[s], (n / NS) & 1, ab, 6))) break;
                    tc_fence_after();
                    const uint32_t v_addr = smem_u32(stage0 + s * L::kStageBytes + L::kKcBytes + L::kKrBytes);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)  // 128 tokens = 4 x 32; a k-step is 32 rows of 128 bytes
                        umma_f8_ts(tmem_base + kF8ColO, tmem_base + kF8ColP + (uint32_t)(n & 1) * 32 + ks * 8,
                                   desc_mnmajor_sw128(v_addr + ks * 4096, 16384), idesc_pv, (t | ks) != 0);
                    umma_commit(&vempty[s]);
                    umma_commit(&pv_done[n & 1]);
                }
                gt += pc.n_tiles;
                ++pi;
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax: one TMEM lane per thread
        const int q = warp & 3;
        const int Lr = q * 32 + lane;
        const int r = Lr % R;
        const int f = Lr / R;
        const int pq = r / p.hpg_box;
        const int il = r % p.hpg_box;
        const bool row_valid = il < p.hpg && pq < p.s_q;
        const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
        const int col0 = R < 32 ? q * 32 : f * R;
        const int sub = R < 32 ? lane / R : 0;
        auto owns = [&](int c) -> bool { return R >= 32 || (c / R) == sub; };
        const int mcg = Lr & 7, mrow0 = Lr >> 3;

        {   // a thread only ever writes its own columns of P; everything else stays zero for good
            uint32_t z[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) z[i] = 0u;
            tmem_st32(lane_base + kF8ColP, z);
            tmem_st32(lane_base + kF8ColP + 32, z);
            tmem_wait_st();
        }

        while (walk.next(pc)) {
            GQLA_DEBUG_CHECK(pc.b >= 0 && pc.b < p.B, p.status, 32);  // a piece names a sequence of the batch
            const int32_t T = p.seqlens[pc.b];
            const int64_t slot0 = (int64_t)pc.b * p.S;
            GQLA_DEBUG_CHECK(pc.n_tiles == 0 || (pc.k >= 0 && pc.k < p.S), p.status, 33);  // ... and one of its S slots
            GQLA_DEBUG_CHECK(pc.tok_begin >= 0 && pc.tok_begin <= pc.tok_end && pc.tok_end <= (T > 0 ? T : 0), p.status, 34);
            GQLA_DEBUG_CHECK(pc.n_tiles == (pc.tok_end > pc.tok_begin ? (pc.tok_end - pc.tok_begin + 127) / 128 : 0), p.status, 35);
            GQLA_DEBUG_CHECK(!p.balanced || pc.tok_begin % 128 == 0, p.status, 36);  // balanced pieces start on tile boundaries
            GQLA_DEBUG_CHECK(pc.fill_begin >= 0 && pc.fill_begin <= pc.fill_end && pc.fill_end <= p.S || pc.fill_end == 0, p.status, 37);
            if (f == 0 && row_valid)
                for (int kk = pc.fill_begin; kk < pc.fill_end; ++kk)
                    p.lse_part[((slot0 + kk) * p.s_q + pq) * p.h_q + (int64_t)j * p.hpg + il] = -INFINITY;
            if (pc.n_tiles == 0 && p.balanced) continue;
            int32_t lim = visible_limit(T, p.s_q, pq);
            if (lim > pc.tok_end) lim = pc.tok_end;
            lim -= pc.tok_begin;
            // the row's score scale: softmax scale x log2(e) x the query row's quantisation scale
            const float sl2 =
                p.scale_log2 * (row_valid ? p.q_scale[((int64_t)pc.b * p.s_q + pq) * p.h_q + (int64_t)j * p.hpg + il] : 1.f);
            float m_used = -INFINITY, l = 0.f;
            bool ok = true;

            for (int t = 0; t < pc.n_tiles && ok; ++t) {
                const int n = gt + t;
                const int sb = n & 1;
                ok = __all_sync(0xffffffffu, mbar_wait_fast(&s_full[sb], (n >> 1) & 1, ab, 7));
                if (!ok) break;
                tc_fence_after();
                const uint32_t s_addr = lane_base + kF8ColS + (uint32_t)sb * 128 + col0;
                const int tok0 = t * 128 + col0;
                uint32_t x[CH];
                float mx = -INFINITY;
#pragma unroll
                for (int ch = 0; ch < NCH; ++ch) {
                    tmem_ld<CH>(s_addr + ch * CH, x);
                    tmem_wait_ld();
#pragma unroll
                    for (int c = 0; c < CH; ++c)
                        if (owns(c) && tok0 + ch * CH + c < lim) mx = fmaxf(mx, __uint_as_float(x[c]));
                }
                // m_used is the replica's softmax REFERENCE: raised to kF8Bias below the tile maximum that exceeded it by
                // more than kF8Grow (a raise rescales O and has to wait for the previous tile's P.V: it is made rare)
                const float m_t = mx * sl2;
                const bool need = m_t > m_used + kF8Grow;
                const float m_new = m_t - kF8Bias;
                const float factor = need ? ex2(m_used - m_new) : 1.f;
                if (__any_sync(0xffffffffu, need) && t > 0) {
                    ok = __all_sync(0xffffffffu, mbar_wait_fast(&pv_done[(n - 1) & 1], ((n - 1) >> 1) & 1, ab, 8));
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll 1
                    for (int c = 0; c < 128; c += 32) {
                        uint32_t o[32];
                        tmem_ld32(lane_base + kF8ColO + c, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * factor);
                        tmem_st32(lane_base + kF8ColO + c, o);
                    }
                    tmem_wait_st();
                }
                if (need) {
                    l *= factor;
                    m_used = m_new;
                }
                const float m_sub = m_used == -INFINITY ? 0.f : m_used;
                const uint32_t p_addr = lane_base + kF8ColP + (uint32_t)sb * 32 + col0 / 4;
#pragma unroll
                for (int ch = 0; ch < NCH; ++ch) {
                    if (NCH > 1) {
                        tmem_ld<CH>(s_addr + ch * CH, x);
                        tmem_wait_ld();
                    }
                    uint32_t pk[CH / 4];
#pragma unroll
                    for (int c = 0; c < CH; c += 4) {
                        const int tok = tok0 + ch * CH + c;
                        const bool mine = owns(c);  // R is a multiple of 8, so four neighbours share an owner
                        float e[4];
#pragma unroll
                        for (int i = 0; i < 4; ++i) {
                            e[i] = (mine && tok + i < lim) ? ex2(fmaf(__uint_as_float(x[c + i]), sl2, -m_sub)) : 0.f;
                            l += e[i];
                        }
                        pk[c / 4] = pack_e4m3x4(e[0], e[1], e[2], e[3]);
                    }
                    tmem_st<CH / 4>(p_addr + ch * (CH / 4), pk);
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&p_ready[sb]);
            }

            // -------------------------------------------------------------- merge the F replicas of each row
            const int n_last = gt + pc.n_tiles - 1;
            if (pc.n_tiles > 0 && ok)
                ok = __all_sync(0xffffffffu, mbar_wait(&pv_done[n_last & 1], (n_last >> 1) & 1, ab, 9));
            tc_fence_after();
            const float m_eff = m_used;  // the reference the replica's sums are relative to (-inf: nothing seen)
            merge[Lr * L::kMergePitch + 32] = m_eff;
            merge[Lr * L::kMergePitch + 33] = l;
            named_bar_sync(1, 128);
            float M = -INFINITY;
#pragma unroll
            for (int ff = 0; ff < F; ++ff) M = fmaxf(M, merge[(ff * R + r) * L::kMergePitch + 32]);
            float Lt = 0.f;
#pragma unroll
            for (int ff = 0; ff < F; ++ff) {
                const float mf = merge[(ff * R + r) * L::kMergePitch + 32];
                if (mf > -INFINITY) Lt += merge[(ff * R + r) * L::kMergePitch + 33] * ex2(mf - M);
            }
            const bool live = ok && pc.n_tiles > 0 && Lt > 0.f;
            const float w = (live && m_used > -INFINITY) ? ex2(m_eff - M) / Lt * p.v_scale : 0.f;
            const int64_t out_row0 = ((slot0 + pc.k) * p.s_q) * p.h_q + (int64_t)j * p.hpg;
#pragma unroll 1
            for (int c4 = 0; c4 < 4; ++c4) {
                uint32_t o[32];
                if (pc.n_tiles > 0 && ok) {  // warp-uniform
                    tmem_ld32(lane_base + kF8ColO + c4 * 32, o);
                    tmem_wait_ld();
                }
                float4* mrow = reinterpret_cast<float4*>(merge + Lr * L::kMergePitch);
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    mrow[i] = w == 0.f ? make_float4(0.f, 0.f, 0.f, 0.f)
                                       : make_float4(__uint_as_float(o[4 * i]) * w, __uint_as_float(o[4 * i + 1]) * w,
                                                     __uint_as_float(o[4 * i + 2]) * w, __uint_as_float(o[4 * i + 3]) * w);
                if (c4 == 3) {
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(o_free);
                }
                named_bar_sync(1, 128);
                for (int rr = mrow0; rr < R; rr += 16) {
                    const int pp = rr / p.hpg_box, ii = rr % p.hpg_box;
                    if (ii >= p.hpg || pp >= p.s_q) continue;
                    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                    for (int ff = 0; ff < F; ++ff) {
                        const float4 xx = *reinterpret_cast<const float4*>(merge + (ff * R + rr) * L::kMergePitch + 4 * mcg);
                        acc.x += xx.x; acc.y += xx.y; acc.z += xx.z; acc.w += xx.w;
                    }
                    *reinterpret_cast<float4*>(p.o_part + (out_row0 + (int64_t)pp * p.h_q + ii) * 128 + c4 * 32 + 4 * mcg) = acc;
                }
                named_bar_sync(1, 128);
            }
            if (f == 0 && row_valid)
                p.lse_part[out_row0 + (int64_t)pq * p.h_q + il] = live ? (M + log2f(Lt)) * 0.6931471805599453f : -INFINITY;
            gt += pc.n_tiles;
            if (pc.n_tiles > 0) ++pi;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, 512);
}

}  // namespace tc
}  // namespace gqla
