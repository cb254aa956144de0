// Absorb-path split-KV flash decoding on tcgen05 (Eq. (mqa), lines 3-5): a PAIR of CTAs (one
// 2-CTA cluster, cta_group::2 MMAs) per (sequence, split, block of 128 query rows).
//
//   S = Qh Kh^T    Qh: 128 rows (head, query) x 576,  Kh = [c ; k_R] rows of the latent cache
//   O = P  V       V = the first 512 columns of the same cache rows
//
// Why a pair: O for 128 rows x 512 fp32 columns is all 256 KB of one SM's tensor memory, leaving no
// room for S.  With a 2-CTA MMA of M = 128 each CTA holds 64 rows; its accumulators use all 128 TMEM
// lanes for half as many columns (lanes 0-63: columns [0, N/2), lanes 64-127: columns [N/2, N) of
// the same 64 rows), so O takes 256 columns and S (128 tokens) 64.  Each CTA also supplies half of
// every B operand from its own shared memory: 64 of the tile's 128 cache rows for S = Qh Kh^T, and
// 128 of every 256 latent columns for O = P V.  The cache is fetched from HBM once; the two operand
// shapes are staged separately through L2 ([64 rows x 64 columns] 8 KB boxes, 128-byte swizzle).
//
// Warp roles per CTA: warp 0 TMA producer, warp 1 TMEM owner (+ MMA issuer in the leader CTA),
// warps 2-5 softmax: thread = TMEM lane = (row, token half); the two threads of a row share the
// running max through shared memory and keep separate partial sums.
#pragma once
#include "common.cuh"
#include "tc_common.cuh"

namespace gqla {
namespace tc {

struct AbsorbParams {
    int32_t B, S, s_q, h_q, rows_total /* s_q*h_q */, row_blocks /* ceil(rows_total/128) */;
    float scale_log2;
    const int64_t* seq_start;
    const int32_t* seqlens;
    float* o_part;    // [B, S, s_q*h_q, 512]
    float* lse_part;  // [B, S, s_q*h_q]
    int32_t* status;
};

struct AbsorbSmem {
    static constexpr int kBox = 8192;              // 64 rows x 64 bf16, 128-byte swizzle
    static constexpr int kQBytes = 9 * kBox;       // 64 query rows x 576
    static constexpr int kPBytes = 2 * kBox;       // 64 rows x 128 tokens (two 64-token k-blocks)
    static constexpr int kNK = 6;                  // ring of K boxes (Qh Kh^T operand)
    static constexpr int kNV = 4;                  // ring of V box PAIRS (P V operand: 64 tokens x 128 columns)
    static constexpr int kOffP = kQBytes;
    static constexpr int kOffK = kOffP + 2 * kPBytes;
    static constexpr int kOffV = kOffK + kNK * kBox;
    static constexpr int kTileBytes = kOffV + kNV * 2 * kBox;
    // barriers: kfull[kNK] kempty[kNK] vfull[kNV] vempty[kNV] q_full s_full[2] p_ready[2] pv_done[2] xch[2] fin
    static constexpr int kNumBars = 2 * kNK + 2 * kNV + 10;
    static constexpr int kBarPReady = 2 * kNK + 2 * kNV + 3;  // index of p_ready[0]
    static constexpr int kBarXch = 2 * kNK + 2 * kNV + 7;     // index of xch[0]
    static constexpr int kTotal = 1024 + kTileBytes + kNumBars * 8 + 16 + 3 * 128 * 4 + 2 * 128 * 4;
};

constexpr uint32_t kAColO = 0;    // O: MMA m (latent columns [256m, 256m+256)) at TMEM columns [128m, 128m+128)
constexpr uint32_t kAColS = 256;  // two 64-column score buffers

template <int DUMMY>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(192, 1)
decode_absorb_tc_kernel(const AbsorbParams p, const __grid_constant__ CUtensorMap tmQ,
                        const __grid_constant__ CUtensorMap tmC) {
    using L = AbsorbSmem;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + L::kTileBytes);
    uint64_t* kfull = bars;
    uint64_t* kempty = kfull + L::kNK;
    uint64_t* vfull = kempty + L::kNK;
    uint64_t* vempty = vfull + L::kNV;
    uint64_t* q_full = vempty + L::kNV;
    uint64_t* s_full = q_full + 1;   // [2]
    uint64_t* p_ready = s_full + 2;  // [2] leader only, 256 arrivals
    uint64_t* pv_done = p_ready + 2; // [2]
    uint64_t* xch = pv_done + 2;     // [2] softmax threads of this CTA: per-tile max exchange (128 arrivals)
    uint64_t* fin = xch + 2;         //     and the final partial-sum exchange
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + L::kNumBars);
    volatile int32_t* abort_flag = reinterpret_cast<volatile int32_t*>(tmem_slot + 1);
    float* sm_l = reinterpret_cast<float*>(tmem_slot + 4);  // [128] final partial sums
    float* sm_max = sm_l + 128;                              // [2][128] per-tile local maxima

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta = cluster_ctarank();  // 0 = leader
    const Abort ab{abort_flag, p.status};

    // work unit of the pair
    const int pair = blockIdx.x >> 1;
    const int rb = pair % p.row_blocks;
    const int k = (pair / p.row_blocks) % p.S;
    const int b = pair / (p.row_blocks * p.S);
    const int32_t T = p.seqlens[b];
    int32_t begin, end;
    split_range(T, p.S, k, &begin, &end);
    const int n_tiles = end > begin ? (end - begin + 127) >> 7 : 0;
    const int64_t row0 = p.seq_start[b] + begin;
    const int rho0 = rb * 128 + (int)cta * 64;  // first (query, head) row of this CTA

    if (threadIdx.x == 0) {
        for (int i = 0; i < L::kNumBars; ++i) {
            const bool pr = i == L::kBarPReady || i == L::kBarPReady + 1;
            mbar_init(&bars[i], pr ? 256 : (i >= L::kBarXch ? 128 : 1));
        }
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc2(tmem_slot, 512);
        tmem_relinquish2();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();  // both CTAs' barriers exist before any remote arrival
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (n_tiles > 0 && elect_one()) {
            tma_prefetch_desc(&tmQ);
            tma_prefetch_desc(&tmC);
            // every "full" barrier lives in the leader and counts the bytes of BOTH CTAs
            const uint32_t q_full_l = mapa(smem_u32(q_full), 0);
            if (cta == 0) mbar_expect_tx(q_full, 2 * L::kQBytes);
            for (int kb = 0; kb < 9; ++kb)
                tma_load_2d_pair(tiles + kb * L::kBox, &tmQ, kb * 64, b * p.rows_total + rho0, q_full_l);
            int ik = 0, iv = 0;  // running box / pair counters
            auto load_k = [&](int t) -> bool {
                const int32_t row = (int32_t)(row0 + (int64_t)t * 128 + cta * 64);
                for (int kb = 0; kb < 9; ++kb, ++ik) {
                    const int s = ik % L::kNK;
                    if (!mbar_wait(&kempty[s], ((ik / L::kNK) & 1) ^ 1, ab, 1)) return false;
                    if (cta == 0) mbar_expect_tx(&kfull[s], 2 * L::kBox);
                    tma_load_2d_pair(tiles + L::kOffK + s * L::kBox, &tmC, kb * 64, row, mapa(smem_u32(&kfull[s]), 0));
                }
                return true;
            };
            auto load_v = [&](int t) -> bool {
                // order: token half h, then MMA m; this CTA supplies latent columns [256m + 128cta, +128)
                for (int h = 0; h < 2; ++h)
                    for (int m = 0; m < 2; ++m, ++iv) {
                        const int s = iv % L::kNV;
                        if (!mbar_wait(&vempty[s], ((iv / L::kNV) & 1) ^ 1, ab, 2)) return false;
                        if (cta == 0) mbar_expect_tx(&vfull[s], 4 * L::kBox);
                        const int32_t row = (int32_t)(row0 + (int64_t)t * 128 + h * 64);
                        const uint32_t bar = mapa(smem_u32(&vfull[s]), 0);
                        uint8_t* dst = tiles + L::kOffV + s * 2 * L::kBox;
                        tma_load_2d_pair(dst, &tmC, 256 * m + 128 * (int)cta, row, bar);
                        tma_load_2d_pair(dst + L::kBox, &tmC, 256 * m + 128 * (int)cta + 64, row, bar);
                    }
                return true;
            };
            bool ok = load_k(0);
            for (int t = 0; t < n_tiles && ok; ++t) {
                if (t + 1 < n_tiles) ok = load_k(t + 1);
                if (ok) ok = load_v(t);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (cta == 0 && n_tiles > 0 && elect_one()) {
            constexpr uint32_t idesc_qk = idesc_bf16(128, 128, 0, 0);
            constexpr uint32_t idesc_pv = idesc_bf16(128, 256, 0, 1);
            const uint32_t q_addr = smem_u32(tiles);
            int ik = 0, iv = 0;
            auto issue_qk = [&](int t) -> bool {
                const uint32_t d = tmem_base + kAColS + (uint32_t)(t & 1) * 64;
                for (int kb = 0; kb < 9; ++kb, ++ik) {
                    const int s = ik % L::kNK;
                    if (!mbar_wait(&kfull[s], (ik / L::kNK) & 1, ab, 3)) return false;
                    tc_fence_after();
                    const uint32_t k_addr = smem_u32(tiles + L::kOffK + s * L::kBox);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        umma_ss2(d, desc_kmajor_sw128(q_addr + kb * L::kBox + ks * 32),
                                 desc_kmajor_sw128(k_addr + ks * 32), idesc_qk, (kb | ks) != 0);
                    umma_commit2(&kempty[s], 3);
                }
                umma_commit2(&s_full[t & 1], 3);
                return true;
            };
            bool ok = mbar_wait(q_full, 0, ab, 4);
            if (ok) ok = issue_qk(0);
            for (int t = 0; t < n_tiles && ok; ++t) {
                if (t + 1 < n_tiles) ok = issue_qk(t + 1);
                if (!ok) break;
                if (!(ok = mbar_wait(&p_ready[t & 1], (t >> 1) & 1, ab, 5))) break;
                const uint32_t p_addr = smem_u32(tiles + L::kOffP + (t & 1) * L::kPBytes);
                for (int h = 0; h < 2 && ok; ++h)
                    for (int m = 0; m < 2; ++m, ++iv) {
                        const int s = iv % L::kNV;
                        if (!(ok = mbar_wait(&vfull[s], (iv / L::kNV) & 1, ab, 6))) break;
                        tc_fence_after();
                        const uint32_t v_addr = smem_u32(tiles + L::kOffV + s * 2 * L::kBox);
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            umma_ss2(tmem_base + kAColO + (uint32_t)m * 128,
                                     desc_kmajor_sw128(p_addr + h * L::kBox + ks * 32),
                                     desc_mnmajor_sw128(v_addr + ks * 2048, L::kBox), idesc_pv, (t | h | ks) != 0);
                        umma_commit2(&vempty[s], 3);
                    }
                if (ok) umma_commit2(&pv_done[t & 1], 3);
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax: thread = TMEM lane
        const int q = warp & 3;
        const int Lr = q * 32 + lane;  // TMEM lane
        const int r = Lr & 63;         // row within this CTA
        const int hf = Lr >> 6;        // token half of each 128-token tile / column half of each O block
        const int rho = rho0 + r;      // (query, head) row of the sequence
        const bool row_valid = rho < p.rows_total;
        const int pq = row_valid ? rho / p.h_q : 0;
        int32_t lim = visible_limit(T, p.s_q, pq);
        if (lim > end) lim = end;
        lim -= begin;
        if (!row_valid) lim = 0;
        const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t p_ready_l[2] = {mapa(smem_u32(&p_ready[0]), 0), mapa(smem_u32(&p_ready[1]), 0)};
        float m_used = -INFINITY, l = 0.f;
        bool ok = true;

        for (int t = 0; t < n_tiles && ok; ++t) {
            const int sb = t & 1;
            ok = __all_sync(0xffffffffu, mbar_wait(&s_full[sb], (t >> 1) & 1, ab, 7));
            if (!ok) break;
            tc_fence_after();
            const uint32_t s_addr = lane_base + kAColS + (uint32_t)sb * 64;
            const int tok0 = t * 128 + hf * 64;
            uint32_t x[64];
            tmem_ld32(s_addr, x);
            tmem_ld32(s_addr + 32, x + 32);
            tmem_wait_ld();
            float mx = -INFINITY;
#pragma unroll
            for (int c = 0; c < 64; ++c)
                if (tok0 + c < lim) mx = fmaxf(mx, __uint_as_float(x[c]));
            // the other token half of this row lives in lane Lr ^ 64
            sm_max[sb * 128 + Lr] = mx;
            mbar_arrive(&xch[sb]);
            ok = __all_sync(0xffffffffu, mbar_wait(&xch[sb], (t >> 1) & 1, ab, 10));
            if (!ok) break;
            mx = fmaxf(mx, sm_max[sb * 128 + (Lr ^ 64)]);
            const float m_t = mx * p.scale_log2;
            const bool need = m_t > m_used + 8.0f;
            const float factor = need ? ex2(m_used - m_t) : 1.f;
            if (__any_sync(0xffffffffu, need) && t > 0) {
                ok = __all_sync(0xffffffffu, mbar_wait(&pv_done[(t - 1) & 1], ((t - 1) >> 1) & 1, ab, 8));
                if (!ok) break;
                tc_fence_after();
#pragma unroll 1
                for (int c = 0; c < 256; c += 32) {
                    uint32_t o[32];
                    tmem_ld32(lane_base + kAColO + c, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * factor);
                    tmem_st32(lane_base + kAColO + c, o);
                }
                tmem_wait_st();
            }
            if (need) {
                l *= factor;
                m_used = m_t;
            }
            const float m_sub = m_used == -INFINITY ? 0.f : m_used;
            // P row r, k-block hf: 128 bytes = 8 chunks of 8 bf16, chunk index XORed with (r & 7)
            uint8_t* prow = tiles + L::kOffP + sb * L::kPBytes + hf * L::kBox + r * 128;
#pragma unroll
            for (int ch = 0; ch < 8; ++ch) {
                uint32_t pk[4];
#pragma unroll
                for (int c = 0; c < 8; c += 2) {
                    const int tok = tok0 + ch * 8 + c;
                    const float e0 = tok < lim ? ex2(fmaf(__uint_as_float(x[ch * 8 + c]), p.scale_log2, -m_sub)) : 0.f;
                    const float e1 =
                        tok + 1 < lim ? ex2(fmaf(__uint_as_float(x[ch * 8 + c + 1]), p.scale_log2, -m_sub)) : 0.f;
                    l += e0 + e1;
                    pk[c / 2] = pack_bf16(e0, e1);
                }
                *reinterpret_cast<uint4*>(prow + ((ch ^ (r & 7)) << 4)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
            }
            fence_proxy_async_smem();  // generic-proxy writes of P -> visible to the tensor core
            tc_fence_before();
            mbar_arrive_cluster(p_ready_l[sb]);
        }

        // ------------------------------------------------------------------ epilogue: normalise and store
        if (n_tiles > 0 && ok)
            ok = __all_sync(0xffffffffu, mbar_wait(&pv_done[(n_tiles - 1) & 1], ((n_tiles - 1) >> 1) & 1, ab, 9));
        tc_fence_after();
        sm_l[Lr] = l;
        mbar_arrive(fin);
        if (!__all_sync(0xffffffffu, mbar_wait(fin, 0, ab, 11))) ok = false;
        const float Lt = l + sm_l[Lr ^ 64];
        const bool live = ok && n_tiles > 0 && Lt > 0.f && m_used > -INFINITY;
        const float inv = live ? 1.f / Lt : 0.f;
        float* orow = p.o_part + ((int64_t)(b * p.S + k) * p.rows_total + (row_valid ? rho : 0)) * 512;
        for (int m = 0; m < 2; ++m) {
            float4* dst = reinterpret_cast<float4*>(orow + 256 * m + 128 * hf);
#pragma unroll 1
            for (int c = 0; c < 128; c += 32) {
                uint32_t o[32];
                tmem_ld32(lane_base + kAColO + m * 128 + c, o);  // warp-collective: never under a per-thread branch
                tmem_wait_ld();
                if (row_valid) {
#pragma unroll
                    for (int i = 0; i < 8; ++i)
                        dst[c / 4 + i] =
                            live ? make_float4(__uint_as_float(o[4 * i]) * inv, __uint_as_float(o[4 * i + 1]) * inv,
                                               __uint_as_float(o[4 * i + 2]) * inv, __uint_as_float(o[4 * i + 3]) * inv)
                                 : make_float4(0.f, 0.f, 0.f, 0.f);
                }
            }
        }
        if (row_valid && hf == 0)
            p.lse_part[(int64_t)(b * p.S + k) * p.rows_total + rho] =
                live ? (m_used + log2f(Lt)) * 0.6931471805599453f : -INFINITY;
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();  // neither CTA leaves while the other may still signal its barriers
    if (warp == 1) tmem_dealloc2(tmem_base, 512);
}

}  // namespace tc
}  // namespace gqla
