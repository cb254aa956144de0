// Absorb-path split-KV flash decoding on tcgen05 with the TOKENS on the MMA's M axis (Eq. (mqa)), for models whose
// h_q * s_q <= 64 query rows fill at most half of a 128-row MMA tile (the LLaMA-shaped setup of Sec. 5: h_q = 32).
//
// tc_decode_absorb.cuh pads the query rows to 128, so at h_q = 32 three quarters of its tensor work is padding and
// the kernel runs at the pace of its MMAs, not of the cache stream.  Here both products are transposed, as in
// tc_decode_gqa_t.cuh:
//
//   S^T = C Qh^T     M = 64 tokens of the tile, N = R query rows, K = 576      (A = cache tile, B = Qh, both K-major)
//   O^T = C_v^T P^T  M = 128 latent columns (x 4 blocks), N = R, K = 64 tokens  (A = the SAME tile read MN-major)
//
// A tile of 64 cache rows (9 boxes of [64 rows x 64 columns], 72 KB) is fetched ONCE and serves as the K operand of
// the first product and, its first eight boxes, as the V operand of the second: every cache byte enters shared memory
// once.  Two tile stages; a stage is released when the tile's P.V has completed.  M = 64 keeps two tiles resident
// beside Qh (with 128-token tiles one stage alone takes 144 KB); its accumulator sits in TMEM lanes 0-15 of each of
// the four lane quadrants (row i of the tile -> lane 32 * (i / 16) + i % 16); the softmax warps read it with
// tcgen05.ld.16x256b, which spreads those 16 lanes over all 32 threads (two tokens x two query rows per thread and
// eight-column load).  The softmax follows tc_decode_gqa_t.cuh: references shared by all threads,
// one barrier.red.or per tile, true row maxima only when a score outgrows its reference by 2^8, row sums met once
// per piece.  O^T has four blocks of R TMEM columns (latent columns [128 m, 128 m + 128) in the lanes); every row
// leaves as 4 x 128 consecutive values, as fp32 partials or, for a whole-sequence call, as the final bf16 row.
//
// Shared memory holds two tiles and one of them is always held by the softmax (a tile fetched once has to stay from its
// first product until its second), so the producer also asks a later tile into L2 when it issues a load, and the held time
// is kept short: the issuer polls instead of blocking, the softmax uses every lane.  Measured (h_q = 32, s_q = 1, 128
// sequences of 8-32 K tokens, balanced plan, one GPU): 437 us in a burst against 541 us for the pair kernel; launched
// back to back for seconds under the power cap, a quarter of the tensor work leaves the clocks at 1.70 GHz where the pair
// kernel's drop to 1.21 GHz: 505 us against 633 us per launch.  With 64 rows (sixteen per softmax warp, one P^T buffer):
// 502 against 554 us in a burst.
#pragma once
#include "common.cuh"
#include "sched.cuh"
#include "tc_common.cuh"
#include "tc_decode_absorb.cuh"  // AbsorbParams
#include "tc_decode_gqa_t.cuh"   // bar_or, warp_max_redux, desc_mnmajor_rows, tmem_ld_n / tmem_st_n

namespace gqla {
namespace tc {

template <int R>
struct AbsorbTSmem {
    static constexpr int kTile = 64;                          // tokens per tile
    static constexpr int kQBlock = R * 128;                   // one k-block of Qh: R rows x 64 bf16
    static constexpr int kQBytes = 9 * kQBlock;               // R rows x 576
    static constexpr int kBox = 8192;                         // 64 tokens x 64 bf16, 128-byte swizzle
    static constexpr int kStageBytes = 9 * kBox;              // 64 tokens x 576
    static constexpr int kStages = 2;
    static constexpr int kPRow = 2 * R;                       // one token's R probabilities (bf16)
    static constexpr int kPSwzBits = R == 64 ? 3 : (R == 32 ? 2 : 1);  // swizzle span = row length (128 / 64 / 32 bytes)
    static constexpr int kPBuf = (kTile * kPRow + 1023) / 1024 * 1024;
    static constexpr int kPBufs = R == 64 ? 1 : 2;            // P^T buffers (one where Qh takes 72 KB: P(n) waits for P.V(n-1))
    static constexpr int kGroup = 3 * kBox;                   // boxes land in groups of three, one barrier each
    static constexpr int kOffStage = kQBytes;
    static constexpr int kOffP = kOffStage + kStages * kStageBytes;
    static constexpr int kOffRed = kOffP + kPBufs * kPBuf;    // [4 quadrants][R] floats; also the plan scratch
    static constexpr int kRowsPerWarp = R == 64 ? 16 : 8;    // query rows (score columns) a softmax warp takes of its 16 tokens
    static constexpr int kSoftmaxWarps = 4 * (R / kRowsPerWarp);
    static constexpr int kThreads = 64 + 32 * kSoftmaxWarps;
    static constexpr int kRedBytes = 4 * R * 4 > (kThreads + 4) * 4 ? 4 * R * 4 : (kThreads + 4) * 4;
    static constexpr int kTileBytes = kOffRed + (kRedBytes + 15) / 16 * 16;
    // q_full q_empty o_free full[2][3] empty[2] s_full[2] p_ready[2] pv_done[2]
    static constexpr int kNumBars = 17;
    static constexpr int kTotal = kTileBytes + kNumBars * 8 + 16;
    static_assert(R == 16 || R == 32 || R == 64, "query rows are padded to 16, 32 or 64");
    static_assert(kQBytes % 1024 == 0, "swizzled tiles start on 1 KB boundaries");
    static_assert(kTotal <= 232448, "shared memory budget of one CTA");
    static_assert(OneCtaPerSM<kTotal>::value, "");
};

#ifndef GQLA_ABSORB_T_PREFETCH
#define GQLA_ABSORB_T_PREFETCH 2
#endif
constexpr int kPrefetchAhead = GQLA_ABSORB_T_PREFETCH;  // tiles between a load and the L2 prefetch issued with it
constexpr uint32_t kPollSpins = 1u << 25;  // polls of the MMA issuer without progress before it gives up

template <int R>
__global__ void __launch_bounds__(AbsorbTSmem<R>::kThreads, 1)
decode_absorb_t_kernel(const AbsorbParams p, const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmC) {
    using L = AbsorbTSmem<R>;
    constexpr int RW = L::kRowsPerWarp;
    constexpr int NJ = RW / 4;  // query rows per softmax thread
    constexpr int kSmT = 32 * L::kSoftmaxWarps;
    constexpr int TK = L::kTile;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* tiles = smem_raw;
    if ((smem_u32(tiles) & 1023u) != 0) {
        if (threadIdx.x == 0 && p.status != nullptr) atomicCAS(p.status, 0, kStatusTimeout | (15 << 8));
        return;
    }
    uint8_t* q_smem = tiles;
    uint8_t* stage0 = tiles + L::kOffStage;
    uint8_t* p_smem = tiles + L::kOffP;
    float* red = reinterpret_cast<float*>(tiles + L::kOffRed);
    uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + L::kTileBytes);
    uint64_t* q_full = bars + 0;
    uint64_t* q_empty = bars + 1;
    uint64_t* o_free = bars + 2;
    uint64_t* full = bars + 3;      // [2][3] a group of three boxes of the tile has landed
    uint64_t* empty = bars + 9;     // [2] the tile's P.V has completed
    uint64_t* s_full = bars + 11;   // [2]
    uint64_t* p_ready = bars + 13;  // [2]
    uint64_t* pv_done = bars + 15;  // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + L::kNumBars);
    volatile int32_t* abort_flag = reinterpret_cast<volatile int32_t*>(tmem_slot + 1);

    // TMEM columns: two score buffers of R columns, then four output blocks of R columns
    constexpr uint32_t kColS = 0, kColO = 2 * R;
    constexpr uint32_t kTmemCols = 6 * R <= 128 ? 128 : (6 * R <= 256 ? 256 : 512);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const Abort ab{abort_flag, p.status};

    if (threadIdx.x == 0) {
        for (int i = 0; i < L::kNumBars; ++i) mbar_init(&bars[i], (i == 2 || i == 13 || i == 14) ? L::kSoftmaxWarps : 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }

    pdl_launch_dependents();
    pdl_wait();
    const int unit = blockIdx.x;
    Walker walk;
    if (p.balanced) {
        const BalancedStart st = balanced_prepass(p.seqlens, p.B, p.S, unit, p.W, reinterpret_cast<int32_t*>(red), L::kThreads);
        walk.init_balanced(p.seqlens, p.B, p.S, unit, p.W, st);
    } else {
        walk.init_fixed(p.seqlens, p.B, p.S, unit / p.S, unit % p.S);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    Piece pc;
    int gt = 0;  // 64-token tiles walked so far: stage = gt & 1, barrier phase = (gt >> 1) & 1
    int pi = 0;  // non-empty pieces walked so far

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (elect_one()) {
            tma_prefetch_desc(&tmQ);
            tma_prefetch_desc(&tmC);
            bool ok = true;
            while (ok && walk.next(pc)) {
                if (pc.n_tiles == 0) continue;
                const int nt = (pc.tok_end - pc.tok_begin + TK - 1) / TK;
                if (pi > 0 && !(ok = mbar_wait(q_empty, (pi - 1) & 1, ab, 13))) break;
                mbar_expect_tx(q_full, L::kQBytes);
                for (int kb = 0; kb < 9; ++kb)
                    tma_load_2d(q_smem + kb * L::kQBlock, &tmQ, kb * 64, pc.b * p.rows_total, q_full);
                for (int t = 0; t < nt; ++t, ++gt) {
                    const int s = gt & 1;
                    uint8_t* st = stage0 + s * L::kStageBytes;
                    // a page holds a multiple of 128 rows and pieces start on multiples of 64: no tile straddles pages
                    const int32_t row = (int32_t)p.rows.row(pc.b, pc.tok_begin + t * TK);
                    if (!(ok = mbar_wait(&empty[s], ((gt >> 1) & 1) ^ 1, ab, 1))) break;
#pragma unroll
                    for (int g = 0; g < 3; ++g) {
                        mbar_expect_tx(&full[s * 3 + g], L::kGroup);
#pragma unroll
                        for (int kb = 3 * g; kb < 3 * g + 3; ++kb)
                            tma_load_2d(st + kb * L::kBox, &tmC, kb * 64, row, &full[s * 3 + g]);
                    }
                    // Shared memory holds two tiles and one of them is held by the softmax: what can be in flight from
                    // HBM is extended through L2 -- the tile after the next is asked into L2 now, so that its load,
                    // issued when a stage frees, finds it there.
                    if (t + kPrefetchAhead < nt) {
                        const int32_t prow = (int32_t)p.rows.row(pc.b, pc.tok_begin + (t + kPrefetchAhead) * TK);
#pragma unroll
                        for (int kb = 0; kb < 9; ++kb) tma_prefetch_l2_2d(&tmC, kb * 64, prow);
                    }
                }
                ++pi;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (elect_one()) {
            constexpr uint32_t idesc_qk = idesc_bf16(64, R, 0, 0);   // S^T: A = cache tile (K-major), B = Qh (K-major)
            constexpr uint32_t idesc_pv = idesc_bf16(128, R, 1, 1);  // O^T: A = the tile read MN-major, B = P^T rows
            const uint32_t q_addr = smem_u32(q_smem), p_addr0 = smem_u32(p_smem);
            bool ok = true;
            while (ok && walk.next(pc)) {
                if (pc.n_tiles == 0) continue;
                const int nt = (pc.tok_end - pc.tok_begin + TK - 1) / TK;
                // The issuer never blocks on one of its two jobs while the other could run: it polls for the next
                // group of boxes (-> twelve MMAs of S^T) and for the next P^T (-> P.V, which releases a tile stage
                // and so keeps the loads flowing).  S^T(n) goes to score buffer n & 1, free once P.V(n-2) was issued.
                int s_tile = 0, s_grp = 0, pv_tile = 0;
                bool q_ok = false, o_ok = pi == 0;
                uint32_t idle = 0;
                while (pv_tile < nt) {
                    bool did = false;
                    if (pv_tile < s_tile) {
                        const int n = gt + pv_tile, s = n & 1;
                        if (mbar_test_wait(&p_ready[s], (n >> 1) & 1)) {
                            if (!o_ok) o_ok = mbar_test_wait(o_free, (pi - 1) & 1);  // O^T of the previous piece was read
                            if (o_ok) {
                                tc_fence_after();
                                const uint32_t v_addr = smem_u32(stage0 + s * L::kStageBytes);
                                const uint32_t pb = p_addr0 + (n % L::kPBufs) * L::kPBuf;
                                // descriptors stepped through their low words (the high words are constants): the
                                // issuer's instructions per MMA are part of the time a tile stays held
                                const uint64_t vd = desc_mnmajor_sw128(v_addr, L::kBox), pd = desc_mnmajor_rows(pb, L::kPRow);
                                const uint32_t v_lo = (uint32_t)vd, v_hi = (uint32_t)(vd >> 32);
                                const uint32_t p_lo = (uint32_t)pd, p_hi = (uint32_t)(pd >> 32);
#pragma unroll
                                for (int m = 0; m < 4; ++m)      // latent columns [128 m, +128): boxes 2m and 2m + 1
#pragma unroll
                                    for (int ks = 0; ks < 4; ++ks)  // 16 tokens per step
                                        umma_ss_lo(tmem_base + kColO + m * R, v_lo + ((2 * m * L::kBox + ks * 2048) >> 4), v_hi,
                                                   p_lo + ((ks * 16 * L::kPRow) >> 4), p_hi, idesc_pv, (pv_tile | ks) != 0);
                                umma_commit(&empty[s]);
                                umma_commit(&pv_done[s]);
                                ++pv_tile;
                                did = true;
                            }
                        }
                    }
                    if (s_tile < nt && s_tile <= pv_tile + 1) {
                        const int n = gt + s_tile, s = n & 1;
                        if (!q_ok) q_ok = mbar_test_wait(q_full, pi & 1);
                        if (q_ok && mbar_test_wait(&full[s * 3 + s_grp], (n >> 1) & 1)) {
                            tc_fence_after();
                            const uint32_t st = smem_u32(stage0 + s * L::kStageBytes);
                            const uint32_t d = tmem_base + kColS + (uint32_t)s * R;
                            const uint32_t k_lo = desc_lo(desc_kmajor_sw128(st + 3 * s_grp * L::kBox));
                            const uint32_t q_lo = desc_lo(desc_kmajor_sw128(q_addr + 3 * s_grp * L::kQBlock));
#pragma unroll
                            for (int kk = 0; kk < 3; ++kk)
#pragma unroll
                                for (int ks = 0; ks < 4; ++ks)
                                    umma_ss_lo(d, k_lo + ((kk * L::kBox + ks * 32) >> 4), kDescHiSw128,
                                               q_lo + ((kk * L::kQBlock + ks * 32) >> 4), kDescHiSw128, idesc_qk,
                                               (uint32_t)(s_grp | kk | ks));
                            if (++s_grp == 3) {
                                umma_commit(&s_full[s]);
                                s_grp = 0;
                                if (++s_tile == nt) umma_commit(q_empty);
                            }
                            did = true;
                        }
                    }
                    if (did) {
                        idle = 0;
                    } else if (++idle > kPollSpins) {
                        ab.raise(5);
                        ok = false;
                        break;
                    } else if ((idle & 255u) == 255u && ab.raised()) {
                        ok = false;
                        break;
                    }
                }
                gt += nt;
                ++pi;
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax
        // An M = 64 accumulator occupies lanes 0-15 of each TMEM lane quadrant.  tcgen05.ld.16x256b hands those 16 lanes
        // x 8 columns to all 32 threads of the warp: thread t gets the scores of tokens t/4 and t/4 + 8 of its quadrant
        // for the query rows 2 (t % 4), 2 (t % 4) + 1 of the warp's eight (and, with sixteen rows per warp, the same two of
        // the second eight) -- every lane works.
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;    // the warp's rows: [half * RW, +RW) of the R query rows
        const int r0 = half * RW;
        const int c2 = 2 * (lane & 3);       // the thread's rows: r0 + rj(j), rj(j) = c2 + (j & 1) + 8 (j >> 1)
        const int tl = q * 32 + lane;        // TMEM lane == latent column within a block in the epilogue
        const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
        float m_ref[NJ], l[NJ];
        auto rj = [&](int j) -> int { return c2 + (j & 1) + 8 * (j >> 1); };

        while (walk.next(pc)) {
            const int32_t T = p.seqlens[pc.b];
            const int64_t slot0 = (int64_t)pc.b * p.S;
            GQLA_DEBUG_CHECK(pc.b >= 0 && pc.b < p.B, p.status, 32);
            GQLA_DEBUG_CHECK(pc.n_tiles == 0 || (pc.k >= 0 && pc.k < p.S), p.status, 33);
            if (half == 0 && tl < p.rows_total && p.lse_part != nullptr)  // thread tl speaks for row tl
                for (int kk = pc.fill_begin; kk < pc.fill_end; ++kk) p.lse_part[(slot0 + kk) * p.rows_total + tl] = -INFINITY;
            if (pc.n_tiles == 0 && p.balanced) continue;
            const int nt = pc.n_tiles == 0 ? 0 : (pc.tok_end - pc.tok_begin + TK - 1) / TK;
#pragma unroll
            for (int j = 0; j < NJ; ++j) { m_ref[j] = -INFINITY; l[j] = 0.f; }
            bool ok = true;

            for (int t = 0; t < nt && ok; ++t) {
                const int n = gt + t;
                const int s = n & 1;
                // a failed wait raises the CTA's abort flag; the warps agree on leaving at the barrier below
                bool okl = __all_sync(0xffffffffu, mbar_wait_fast(&s_full[s], (n >> 1) & 1, ab, 7));
                tc_fence_after();
                // (the P^T buffer was last read by P.V(n-2), which the issuer queued before S^T(n): MMAs complete in
                // issue order, so S^T(n) having landed means that P.V(n-2) has read it)
                uint32_t x[2 * NJ];  // x[4 (j >> 1) + 2 h + (j & 1)]: token h (0: t/4, 1: t/4 + 8), row j of the thread
                if (okl) {
                    if (NJ == 2) tmem_ld_16x256b(lane_base + kColS + (uint32_t)s * R + r0, x);
                    else tmem_ld_16x256b_x2(lane_base + kColS + (uint32_t)s * R + r0, x);
                    tmem_wait_ld();
                }
                // query row r = pq * h_q + head; position pq sees the tokens below T - (s_q - 1 - pq)
                float xs[2 * NJ];  // same order
                bool grow = false;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const int ta = pc.tok_begin + t * TK + q * 16 + (lane >> 2) + 8 * h;
                    const int pq_min = p.s_q - (T - ta) > 0 ? p.s_q - (T - ta) : 0;
                    const int r_lo = ta < pc.tok_end ? pq_min * p.h_q : R;
#pragma unroll
                    for (int j = 0; j < NJ; ++j) {
                        const int r = r0 + rj(j), i = 4 * (j >> 1) + 2 * h + (j & 1);
                        const bool vis = okl && r >= r_lo && r < p.rows_total;
                        xs[i] = vis ? __uint_as_float(x[i]) * p.scale_log2 : -INFINITY;
                        grow |= xs[i] > m_ref[j] + kTRescaleThreshold;
                    }
                }
                if (bar_or(grow || !okl, kSmT)) {
                    if (ab.raised()) { ok = false; break; }  // same answer in every thread: the flag was set before the barrier
                    float factor[NJ];
                    bool any = false;
#pragma unroll
                    for (int j = 0; j < NJ; ++j) {  // the row's maximum over the warp's 16 tokens: lanes with equal t % 4
                        float mx = fmaxf(xs[4 * (j >> 1) + (j & 1)], xs[4 * (j >> 1) + 2 + (j & 1)]);
                        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 4));
                        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 8));
                        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
                        if (lane < 4) red[q * R + r0 + rj(j)] = mx;
                    }
                    named_bar_sync(1, kSmT);
#pragma unroll
                    for (int j = 0; j < NJ; ++j) {
                        const int r = r0 + rj(j);
                        const float tm = fmaxf(fmaxf(red[r], red[R + r]), fmaxf(red[2 * R + r], red[3 * R + r]));
                        const float mn = fmaxf(m_ref[j], tm);
                        factor[j] = mn > m_ref[j] ? ex2(m_ref[j] - mn) : 1.f;  // ex2(-inf) = 0 on first use
                        any |= mn > m_ref[j];
                        l[j] *= factor[j];
                        m_ref[j] = mn;
                    }
                    named_bar_sync(1, kSmT);  // red may be rewritten by the next tile
                    if (__any_sync(0xffffffffu, any) && t > 0) {
                        // O^T may be rescaled only between P.V(n-1) completing and P.V(n) being issued
                        if (!__all_sync(0xffffffffu, mbar_wait(&pv_done[(n - 1) & 1], ((n - 1) >> 1) & 1, ab, 8))) {
                            okl = false;  // noticed by everybody at the next barrier
                        } else {
                            tc_fence_after();
#pragma unroll
                            for (int cc = 0; cc < RW; cc += 8) {  // eight rows at a time
                                float f8[8];  // row cc + c is row (c & 1) + 2 (cc >> 3) of the lanes with t % 4 == c / 2
#pragma unroll
                                for (int c = 0; c < 8; ++c) f8[c] = __shfl_sync(0xffffffffu, factor[(c & 1) + 2 * (cc >> 3)], c >> 1);
#pragma unroll
                                for (int m = 0; m < 4; ++m) {
                                    uint32_t o[8];
                                    tmem_ld8(lane_base + kColO + m * R + r0 + cc, o);
                                    tmem_wait_ld();
#pragma unroll
                                    for (int c = 0; c < 8; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * f8[c]);
                                    tmem_st8(lane_base + kColO + m * R + r0 + cc, o);
                                }
                            }
                            tmem_wait_st();
                        }
                    }
                }
                // probabilities: a bf16 pair (the thread's two rows) into each of its two tokens' rows of P^T
                const int pbi = n % L::kPBufs;
                uint32_t pk[NJ];  // [2 h + pair]: the bf16 pair of token h for the thread's row pair
#pragma unroll
                for (int h = 0; h < 2; ++h)
#pragma unroll
                    for (int jp = 0; jp < NJ; jp += 2) {
                        const int i = 4 * (jp >> 1) + 2 * h;
                        const float e0 = xs[i] > -INFINITY ? ex2(xs[i] - m_ref[jp]) : 0.f;
                        const float e1 = xs[i + 1] > -INFINITY ? ex2(xs[i + 1] - m_ref[jp + 1]) : 0.f;
                        l[jp] += e0;
                        l[jp + 1] += e1;
                        pk[(NJ / 2) * h + (jp >> 1)] = pack_bf16(e0, e1);
                    }
                // a single P^T buffer is still being read by P.V(n-1)
                if (L::kPBufs == 1 && t > 0 && okl)
                    okl = __all_sync(0xffffffffu, mbar_wait(&pv_done[(n - 1) & 1], ((n - 1) >> 1) & 1, ab, 8));
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint32_t off = (uint32_t)(q * 16 + (lane >> 2) + 8 * h) * L::kPRow;  // the token's row of P^T
                    const uint32_t pswz = (off >> 7) & ((1u << L::kPSwzBits) - 1);             // XOR of its 16-byte chunks
#pragma unroll
                    for (int jp = 0; jp < NJ; jp += 2) {
                        const uint32_t col = (uint32_t)(r0 + rj(jp)) * 2;                      // byte of that row pair in it
                        *reinterpret_cast<uint32_t*>(p_smem + pbi * L::kPBuf + off + (((col >> 4) ^ pswz) << 4) + (col & 15)) =
                            pk[(NJ / 2) * h + (jp >> 1)];
                    }
                }
                fence_proxy_async_smem();  // generic-proxy writes of P^T -> visible to the tensor core
                tc_fence_before();
                __syncwarp();
                if (lane == 0 && okl) mbar_arrive(&p_ready[s]);
            }

            // -------------------------------------------------------------- row sums across the tokens, then the output
            const int n_last = gt + nt - 1;
            if (nt > 0 && ok) ok = __all_sync(0xffffffffu, mbar_wait(&pv_done[n_last & 1], (n_last >> 1) & 1, ab, 9));
            tc_fence_after();
#pragma unroll
            for (int j = 0; j < NJ; ++j) {  // the row's sum over the warp's tokens: lanes with equal t % 4
                float ws = l[j];
                ws += __shfl_xor_sync(0xffffffffu, ws, 4);
                ws += __shfl_xor_sync(0xffffffffu, ws, 8);
                ws += __shfl_xor_sync(0xffffffffu, ws, 16);
                if (lane < 4) red[q * R + r0 + rj(j)] = ws;
            }
            named_bar_sync(1, kSmT);
            const int64_t out_row0 = (p.o_final != nullptr ? (int64_t)pc.b : slot0 + pc.k) * p.rows_total;
            if (q == 0 && lane < 4 && p.lse_part != nullptr) {
#pragma unroll
                for (int j = 0; j < NJ; ++j) {
                    const int r = r0 + rj(j);
                    const float Lt = (red[r] + red[R + r]) + (red[2 * R + r] + red[3 * R + r]);
                    const bool live = ok && nt > 0 && Lt > 0.f && m_ref[j] > -INFINITY;
                    if (r < p.rows_total) p.lse_part[out_row0 + r] = live ? (m_ref[j] + log2f(Lt)) * 0.6931471805599453f : -INFINITY;
                }
            }
#pragma unroll
            for (int cc = 0; cc < RW; cc += 8) {  // eight rows at a time (a lane is a latent column of all of them)
                float inv[8];
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const int r = r0 + cc + c;
                    const float Lt = (red[r] + red[R + r]) + (red[2 * R + r] + red[3 * R + r]);
                    inv[c] = (ok && nt > 0 && Lt > 0.f) ? 1.f / Lt : 0.f;
                }
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    uint32_t o[8];
                    if (nt > 0 && ok) {  // warp-uniform
                        tmem_ld8(lane_base + kColO + m * R + r0 + cc, o);
                        tmem_wait_ld();
                    }
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        const int r = r0 + cc + c;
                        if (r >= p.rows_total) continue;  // padding rows are computed and dropped
                        const float val = inv[c] > 0.f ? __uint_as_float(o[c]) * inv[c] : 0.f;
                        // lane tl holds latent column 128 m + tl of every row: 128 consecutive values per row and block
                        if (p.o_final != nullptr) p.o_final[(out_row0 + r) * 512 + m * 128 + tl] = __float2bfloat16(val);
                        else p.o_part[(out_row0 + r) * 512 + m * 128 + tl] = val;
                    }
                }
            }
            named_bar_sync(1, kSmT);  // red is rewritten by the next piece
            // O^T has been read: the next piece's first P.V may overwrite it
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(o_free);
            gt += nt;
            if (nt > 0) ++pi;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace tc
}  // namespace gqla
