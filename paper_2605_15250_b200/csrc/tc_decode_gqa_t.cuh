// GQA-path split-KV flash decoding on tcgen05 with the TOKENS on the MMA's M axis (Eq. (mha)).
//
// A group has only R = (h_q/g) * s_q query rows (32 at the canonical shape with s_q = 2, 8-16 for small models)
// against an MMA tile of 128 rows.  tc_decode_gqa.cuh fills the tile by replicating the rows, which issues
// 128/R times the tensor work the method needs.  Here the products are transposed instead:
//
//   S^T = K Q^T     M = 128 tokens of the tile, N = R query rows, K = 192     (A = K tile, B = Q, both K-major)
//   O^T = V^T P^T   M = 128 value columns,      N = R,            K = 128 tokens (A = V tile read MN-major, B = P^T)
//
// so the tensor core does exactly the method's FLOPs (N = R instead of 128).  The price is in the softmax: a
// TMEM lane is now a TOKEN and holds one score of every query row, so a row's maximum and sum live across the
// 128 softmax threads.  They are kept out of the loop:
//   * R/8 softmax warps per TMEM lane quadrant (8 or 16 in all): a thread owns one token of the tile and eight of
//     the query rows, so the softmax of a tile is spread over up to 512 threads.  Every thread holds the same reference m_ref[r] for its rows and checks its own token's scores against
//     it; a bar.red.or tells the warps whether any score outgrew its reference by more than 2^8.  Only
//     then (and on a piece's first tile) are the true row maxima of the tile reduced (redux over a warp, shared
//     memory across warps), the references raised and O^T rescaled column by column;
//   * every thread sums the probabilities of ITS tokens per row; the 128 partial sums of a row meet once per
//     piece.
// P^T goes to shared memory as the B operand of the second product in its MN-major form -- one row of R
// probabilities (2R bytes) per token, which is exactly what a thread holds, so it leaves as 16-byte stores; the rows
// use the swizzle whose span equals their length (128 / 64 / 32 bytes for R = 64 / 32 / 16).  Double-buffered so
// that writing P(n) only waits for P.V(n-2).  O^T has one value column per lane and one query row per TMEM column, so the epilogue needs no
// replica merge: for every row the 128 lanes store 128 consecutive floats.
#pragma once
#include "common.cuh"
#include "sched.cuh"
#include "tc_common.cuh"
#include "tc_decode_gqa.cuh"  // GqaParams

namespace gqla {
namespace tc {

template <int R>
struct GqaTSmem {
    static constexpr int kQBlock = R * 128;                  // one k-block of Q: R rows x 64 bf16
    static constexpr int kQBytes = 3 * kQBlock;              // rounded up to 1 KB below
    static constexpr int kQRegion = (kQBytes + 1023) / 1024 * 1024;
    static constexpr int kKcBytes = 2 * 16384;               // 128 tokens x 128
    static constexpr int kKrBytes = 16384;                   // 128 tokens x 64
    static constexpr int kVBytes = 2 * 16384;                // 128 tokens x 128
    static constexpr int kStageBytes = kKcBytes + kKrBytes + kVBytes;
    static constexpr int kStages = 2;
    static constexpr int kPRow = 2 * R;                      // one token's R probabilities (bf16)
    static constexpr int kPSwzBits = R == 64 ? 3 : (R == 32 ? 2 : 1);  // swizzle span = row length: 128 / 64 / 32 bytes
    static constexpr int kPBuf = (128 * kPRow + 1023) / 1024 * 1024;   // 128 tokens, 1 KB aligned
    static constexpr int kOffStage = kQRegion;
    static constexpr int kOffP = kOffStage + kStages * kStageBytes;
    static constexpr int kOffRed = kOffP + 2 * kPBuf;        // [4 warps][R] floats: row maxima / sums across warps
    static constexpr int kRedBytes = 4 * R * 4;
    static constexpr int kTileBytes = kOffRed + (kRedBytes > 3072 ? kRedBytes : 3072);  // also the plan scratch
    // q_full q_empty o_free kfull[2] vfull[2] kempty[2] vempty[2] s_full[2] p_ready[2] pv_done[2]
    static constexpr int kNumBars = 17;
    static constexpr int kRowsPerThread = R <= 32 ? 8 : 16;           // query rows a softmax thread takes of its token
    static constexpr int kSoftmaxWarps = 4 * (R / kRowsPerThread);  // R / kRowsPerThread warps per TMEM lane quadrant
    static constexpr int kThreads = 64 + 32 * kSoftmaxWarps;
    static constexpr int kTotal = kTileBytes + kNumBars * 8 + 16;
    static_assert(R == 16 || R == 32 || R == 64, "query rows are padded to a power of two in [16, 64]");
    static_assert(kTileBytes >= kOffRed + (kThreads + 4) * 4, "plan scratch must fit in the reduction buffer");
    static_assert(kTotal <= 232448, "shared memory budget of one CTA");
    static_assert(OneCtaPerSM<kTotal>::value, "");
};

// MN-major operand whose rows (one per k index) are `row_bytes` = 128 / 64 / 32 bytes long and swizzled over that span:
// 8-row groups are 8 * row_bytes apart (SBO); the MN extent fits one row, so LBO is unused.
__device__ __forceinline__ uint64_t desc_mnmajor_rows(uint32_t smem_addr, uint32_t row_bytes) {
    const uint64_t mode = row_bytes == 128 ? 2ull : (row_bytes == 64 ? 4ull : 6ull);
    return (1ull << 46) | (mode << 61) | (uint64_t)((smem_addr & 0x3FFFF) >> 4) | (1ull << 16) |
           ((uint64_t)((8 * row_bytes) >> 4) << 32);
}

constexpr float kTRescaleThreshold = 8.0f;  // log2 units: P may grow to 2^8 before the references are raised

// Maximum of a float over the warp with one redux: floats are mapped to integers of the same order.
__device__ __forceinline__ float warp_max_redux(float x) {
    int i = __float_as_int(x);
    i ^= (i >> 31) & 0x7fffffff;
    i = __reduce_max_sync(0xffffffffu, i);
    i ^= (i >> 31) & 0x7fffffff;
    return __int_as_float(i);
}
__device__ __forceinline__ void tmem_ld_n(uint32_t taddr, uint32_t* r, int n) {  // n in {8, 16}
    if (n == 8) tmem_ld8(taddr, r);
    else tmem_ld16(taddr, r);
}
__device__ __forceinline__ void tmem_st_n(uint32_t taddr, const uint32_t* r, int n) {
    if (n == 8) tmem_st8(taddr, r);
    else tmem_st16(taddr, r);
}

template <int R>
__global__ void __launch_bounds__(GqaTSmem<R>::kThreads, 1)
decode_gqa_t_kernel(const GqaParams p, const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmR, const __grid_constant__ CUtensorMap tmV) {
    using L = GqaTSmem<R>;
    constexpr int RW = L::kRowsPerThread;    // query rows per softmax thread (the others belong to its partner warps)
    constexpr int CH = RW;                   // rows handled per pass (TMEM columns per load)
    constexpr int NCH = RW / CH;
    constexpr int kSmT = 32 * L::kSoftmaxWarps;  // softmax threads
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* tiles = smem_raw;
    if ((smem_u32(tiles) & 1023u) != 0) {  // swizzled tiles need 1 KB alignment
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
    uint64_t* kfull = bars + 3;    // [2]
    uint64_t* vfull = bars + 5;    // [2]
    uint64_t* kempty = bars + 7;   // [2]
    uint64_t* vempty = bars + 9;   // [2]
    uint64_t* s_full = bars + 11;  // [2]
    uint64_t* p_ready = bars + 13; // [2]
    uint64_t* pv_done = bars + 15; // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + L::kNumBars);
    volatile int32_t* abort_flag = reinterpret_cast<volatile int32_t*>(tmem_slot + 1);

    // TMEM columns: two score buffers of R columns, then the R-column output accumulator
    constexpr uint32_t kColS = 0, kColO = 2 * R;
    constexpr uint32_t kTmemCols = 3 * R <= 64 ? 64 : (3 * R <= 128 ? 128 : (3 * R <= 256 ? 256 : 512));

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
    const int vb = blockIdx.x % p.v_blocks;
    const int j = (blockIdx.x / p.v_blocks) % p.g;
    const int unit = blockIdx.x / (p.v_blocks * p.g);
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
    int gt = 0;  // tiles walked so far: ring slot = gt & 1, barrier phase = (gt >> 1) & 1
    int pi = 0;  // non-empty pieces walked so far

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (elect_one()) {
            tma_prefetch_desc(&tmQ);
            tma_prefetch_desc(&tmK);
            tma_prefetch_desc(&tmR);
            tma_prefetch_desc(&tmV);
            bool ok = true;
            while (ok && walk.next(pc)) {
                if (pc.n_tiles == 0) continue;
                if (pi > 0 && !(ok = mbar_wait(q_empty, (pi - 1) & 1, ab, 13))) break;
                mbar_expect_tx(q_full, L::kQBytes);
                for (int kb = 0; kb < 3; ++kb)
                    asm volatile(
                        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], "
                        "[%1, {%3, %4, %5, %6}], [%2];" ::"r"(smem_u32(q_smem + kb * L::kQBlock)),
                        "l"(reinterpret_cast<uint64_t>(&tmQ)), "r"(smem_u32(q_full)), "r"(kb * 64), "r"(0), "r"(j),
                        "r"(pc.b * p.s_q)
                        : "memory");
                int64_t tile_row = p.rows.row(pc.b, pc.tok_begin);
                for (int t = 0; t < pc.n_tiles; ++t, ++gt) {
                    const int s = gt & 1;
                    const uint32_t ph = (gt >> 1) & 1;
                    uint8_t* st = stage0 + s * L::kStageBytes;
                    const int32_t row = (int32_t)tile_row;
                    if (t + 1 < pc.n_tiles)
                        tile_row = p.rows.paged() ? p.rows.row(pc.b, pc.tok_begin + (t + 1) * 128) : tile_row + 128;
                    if (!(ok = mbar_wait(&kempty[s], ph ^ 1, ab, 1))) break;
                    mbar_expect_tx(&kfull[s], L::kKcBytes + L::kKrBytes);
                    tma_load_3d(st, &tmK, 0, j, row, &kfull[s]);
                    tma_load_3d(st + 16384, &tmK, 64, j, row, &kfull[s]);
                    tma_load_2d(st + L::kKcBytes, &tmR, 0, row, &kfull[s]);
                    if (!(ok = mbar_wait(&vempty[s], ph ^ 1, ab, 2))) break;
                    mbar_expect_tx(&vfull[s], L::kVBytes);
                    tma_load_3d(st + L::kKcBytes + L::kKrBytes, &tmV, vb * 128, j, row, &vfull[s]);
                    tma_load_3d(st + L::kKcBytes + L::kKrBytes + 16384, &tmV, vb * 128 + 64, j, row, &vfull[s]);
                }
                ++pi;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (elect_one()) {
            constexpr uint32_t idesc_qk = idesc_bf16(128, R, 0, 0);  // S^T: A = K tile (K-major), B = Q (K-major)
            constexpr uint32_t idesc_pv = idesc_bf16(128, R, 1, 1);  // O^T: A = V tile read MN-major, B = P^T rows (MN-major)
            const uint32_t q_addr = smem_u32(q_smem), p_addr0 = smem_u32(p_smem);
            auto issue_qk = [&](int n) -> bool {
                const int s = n & 1;
                if (!mbar_wait(&kfull[s], (n >> 1) & 1, ab, 3)) return false;
                tc_fence_after();
                const uint32_t st = smem_u32(stage0 + s * L::kStageBytes);
                const uint32_t d = tmem_base + kColS + (uint32_t)s * R;
                // descriptors stepped through their low words (the high words are constants): fewer instructions per MMA
                const uint32_t k_lo = desc_lo(desc_kmajor_sw128(st)), q_lo = desc_lo(desc_kmajor_sw128(q_addr));
#pragma unroll
                for (int kb = 0; kb < 3; ++kb)
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        umma_ss_lo(d, k_lo + ((kb * 16384 + ks * 32) >> 4), kDescHiSw128, q_lo + ((kb * L::kQBlock + ks * 32) >> 4),
                                   kDescHiSw128, idesc_qk, (uint32_t)(kb | ks));
                umma_commit(&s_full[s]);
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
                    const int s = n & 1;
                    const uint32_t ph = (n >> 1) & 1;
                    if (t + 1 < pc.n_tiles) {
                        if (!(ok = issue_qk(n + 1))) break;
                    } else {
                        umma_commit(q_empty);
                    }
                    if (!(ok = mbar_wait(&p_ready[s], ph, ab, 5))) break;
                    if (t == 0 && pi > 0 && !(ok = mbar_wait(o_free, (pi - 1) & 1, ab, 14))) break;
                    if (!(ok = mbar_wait(&vfull[s], ph, ab, 6))) break;
                    tc_fence_after();
                    const uint32_t v_addr = smem_u32(stage0 + s * L::kStageBytes + L::kKcBytes + L::kKrBytes);
                    const uint32_t pb = p_addr0 + s * L::kPBuf;
                    const uint64_t vd = desc_mnmajor_sw128(v_addr, 16384), pd = desc_mnmajor_rows(pb, L::kPRow);
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)  // 16 tokens per step: rows [16 ks, +16) of the V boxes and of P^T
                        umma_ss_lo(tmem_base + kColO, (uint32_t)vd + ((ks * 2048) >> 4), (uint32_t)(vd >> 32),
                                   (uint32_t)pd + ((ks * 16 * L::kPRow) >> 4), (uint32_t)(pd >> 32), idesc_pv, (uint32_t)(t | ks));
                    umma_commit(&vempty[s]);
                    umma_commit(&pv_done[s]);
                }
                gt += pc.n_tiles;
                ++pi;
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax: one TMEM lane = one token per thread
        const int q = warp & 3;
        const int half = (warp - 2) >> 2;  // which part of the query rows this warp takes: rows [half * RW, +RW)
        const int r0 = half * RW;
        const int tl = q * 32 + lane;  // token within the tile == TMEM lane (and value column in the epilogue)
        const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
        // query row r = pq * hpg_box + il (the Q box is hpg_box heads x sq_box positions; beyond them: zero rows)
        float m_ref[RW], l[RW];  // of rows r0 .. r0 + RW - 1

        while (walk.next(pc)) {
            const int32_t T = p.seqlens[pc.b];
            const int64_t slot0 = (int64_t)pc.b * p.S;
            GQLA_DEBUG_CHECK(pc.b >= 0 && pc.b < p.B, p.status, 32);
            GQLA_DEBUG_CHECK(pc.n_tiles == 0 || (pc.k >= 0 && pc.k < p.S), p.status, 33);
            if (vb == 0 && half == 0 && tl < R) {  // split slots this worker marks empty (thread tl speaks for row tl)
                const int pq = tl / p.hpg_box, il = tl % p.hpg_box;
                if (il < p.hpg && pq < p.s_q)
                    for (int kk = pc.fill_begin; kk < pc.fill_end; ++kk)
                        p.lse_part[((slot0 + kk) * p.s_q + pq) * p.h_q + (int64_t)j * p.hpg + il] = -INFINITY;
            }
            if (pc.n_tiles == 0 && p.balanced) continue;
#pragma unroll
            for (int r = 0; r < RW; ++r) { m_ref[r] = -INFINITY; l[r] = 0.f; }
            const int hshift = __ffs(p.hpg_box) - 1;  // hpg_box is a power of two: pq = r >> hshift
            bool ok = true;

            for (int t = 0; t < pc.n_tiles && ok; ++t) {
                const int n = gt + t;
                const int s = n & 1;
                // A wait that fails raises the CTA's abort flag; the warps agree on leaving at the next barrier below
                // (a warp that left the loop on its own would strand the others in that barrier).
                bool okl = __all_sync(0xffffffffu, mbar_wait(&s_full[s], (n >> 1) & 1, ab, 7));
                tc_fence_after();
                // P^T buffer s was last read by P.V(n-2)
                if (okl && t > 1) okl = __all_sync(0xffffffffu, mbar_wait(&pv_done[s], ((n - 2) >> 1) & 1, ab, 8));
                // rows this thread's token is visible to: query position pq sees tokens below T - (s_q-1-pq), so the
                // token at absolute position ta is seen by positions pq >= s_q - (T - ta); padding positions see nothing
                const int ta = pc.tok_begin + t * 128 + tl;
                const int pq_min = p.s_q - (T - ta) > 0 ? p.s_q - (T - ta) : 0;
                const int r_lo = ta < pc.tok_end ? (pq_min << hshift) : R;
                const int r_hi = p.s_q << hshift;
                uint8_t* prow = p_smem + s * L::kPBuf + tl * L::kPRow;  // this token's row of P^T
                const uint32_t pswz = ((uint32_t)(tl * L::kPRow) >> 7) & ((1u << L::kPSwzBits) - 1);  // XOR of its 16-byte chunks
#pragma unroll
                for (int ch = 0; ch < NCH; ++ch) {
                    uint32_t x[CH];
                    float xs[CH];
                    bool grow = false;
                    if (okl) {
                        tmem_ld_n(lane_base + kColS + (uint32_t)s * R + r0 + ch * CH, x, CH);
                        tmem_wait_ld();
                    }
                    // does any visible score of this token outgrow its row's reference?
#pragma unroll
                    for (int c = 0; c < CH; ++c) {
                        const int rl = ch * CH + c, r = r0 + rl;  // local and global row
                        const bool vis = okl && r >= r_lo && r < r_hi;
                        xs[c] = vis ? __uint_as_float(x[c]) * p.scale_log2 : -INFINITY;
                        grow |= xs[c] > m_ref[rl] + kTRescaleThreshold;
                    }
                    if (bar_or(grow || !okl, kSmT)) {
                        if (ab.raised()) { ok = false; break; }  // same answer in every thread: the flag was set before the barrier
                        // raise the references of this chunk's rows to the tile's true maxima and rescale O^T
                        float* redw = red + q * R + r0 + ch * CH;
#pragma unroll
                        for (int c = 0; c < CH; ++c) {
                            const float wm = warp_max_redux(xs[c]);
                            if (lane == 0) redw[c] = wm;
                        }
                        named_bar_sync(1, kSmT);
                        float factor[CH];
                        bool any = false;
#pragma unroll
                        for (int c = 0; c < CH; ++c) {
                            const int rl = ch * CH + c, r = r0 + rl;
                            const float tm = fmaxf(fmaxf(red[r], red[R + r]), fmaxf(red[2 * R + r], red[3 * R + r]));
                            const float mn = fmaxf(m_ref[rl], tm);
                            factor[c] = mn > m_ref[rl] ? ex2(m_ref[rl] - mn) : 1.f;  // ex2(-inf) = 0 on first use
                            any |= mn > m_ref[rl];
                            l[rl] *= factor[c];
                            m_ref[rl] = mn;
                        }
                        named_bar_sync(1, kSmT);  // red may be rewritten by the next chunk / tile
                        // (`any` is the same in the threads of a warp -- they hold the same rows -- but not across the two
                        // halves, which rescale their own columns of O^T; no barrier follows inside this branch)
                        if (any && t > 0) {
                            // O^T may be rescaled only between P.V(n-1) completing and P.V(n) being issued
                            if (!__all_sync(0xffffffffu, mbar_wait(&pv_done[(n - 1) & 1], ((n - 1) >> 1) & 1, ab, 8))) {
                                okl = false;  // noticed by everybody at the next barrier
                            } else {
                                tc_fence_after();
                                uint32_t o[CH];
                                tmem_ld_n(lane_base + kColO + r0 + ch * CH, o, CH);
                                tmem_wait_ld();
#pragma unroll
                                for (int c = 0; c < CH; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * factor[c]);
                                tmem_st_n(lane_base + kColO + r0 + ch * CH, o, CH);
                                tmem_wait_st();
                            }
                        }
                    }
                    // probabilities of this token for the chunk's rows -> its row of P^T, eight rows per 16-byte store
                    uint32_t pk[CH / 2];
#pragma unroll
                    for (int c = 0; c < CH; c += 2) {
                        const int rl = ch * CH + c;
                        const float e0 = xs[c] > -INFINITY ? ex2(xs[c] - m_ref[rl]) : 0.f;
                        const float e1 = xs[c + 1] > -INFINITY ? ex2(xs[c + 1] - m_ref[rl + 1]) : 0.f;
                        l[rl] += e0;
                        l[rl + 1] += e1;
                        pk[c / 2] = pack_bf16(e0, e1);
                    }
#pragma unroll
                    for (int i = 0; i < CH / 8; ++i)
                        *reinterpret_cast<uint4*>(prow + ((((uint32_t)((r0 + ch * CH) / 8 + i)) ^ pswz) << 4)) =
                            make_uint4(pk[4 * i], pk[4 * i + 1], pk[4 * i + 2], pk[4 * i + 3]);
                }
                if (!ok) break;
                fence_proxy_async_smem();  // generic-proxy writes of P^T -> visible to the tensor core
                tc_fence_before();
                __syncwarp();
                if (lane == 0 && okl) mbar_arrive(&p_ready[s]);
            }

            // -------------------------------------------------------------- row sums across the 128 tokens, then the output
            const int n_last = gt + pc.n_tiles - 1;
            if (pc.n_tiles > 0 && ok)
                ok = __all_sync(0xffffffffu, mbar_wait(&pv_done[n_last & 1], (n_last >> 1) & 1, ab, 9));
            tc_fence_after();
            const int64_t out_row0 = ((slot0 + pc.k) * p.s_q) * p.h_q + (int64_t)j * p.hpg;
#pragma unroll
            for (int ch = 0; ch < NCH; ++ch) {  // unrolled: l and m_ref must stay in registers
                float* redw = red + q * R + r0 + ch * CH;
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    const float ws = warp_sum(l[ch * CH + c]);
                    if (lane == 0) redw[c] = ws;
                }
                named_bar_sync(1, kSmT);
                uint32_t o[CH];
                if (pc.n_tiles > 0 && ok) {  // warp-uniform
                    tmem_ld_n(lane_base + kColO + r0 + ch * CH, o, CH);
                    tmem_wait_ld();
                }
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    const int rl = ch * CH + c, r = r0 + rl;
                    const int pq = r / p.hpg_box, il = r % p.hpg_box;
                    if (il >= p.hpg || pq >= p.s_q) continue;  // padding rows are computed and dropped
                    const float Lt = (red[r] + red[R + r]) + (red[2 * R + r] + red[3 * R + r]);
                    const bool live = ok && pc.n_tiles > 0 && Lt > 0.f && m_ref[rl] > -INFINITY;
                    const int64_t orow = out_row0 + (int64_t)pq * p.h_q + il;
                    // lane tl holds value column tl of every row: 128 consecutive floats per row
                    p.o_part[orow * p.d_v + vb * 128 + tl] = live ? __uint_as_float(o[c]) / Lt : 0.f;
                    if (vb == 0 && tl == 0) p.lse_part[orow] = live ? (m_ref[rl] + log2f(Lt)) * 0.6931471805599453f : -INFINITY;
                }
                named_bar_sync(1, kSmT);
            }
            // O^T has been read: the next piece's first P.V may overwrite it
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(o_free);
            gt += pc.n_tiles;
            if (pc.n_tiles > 0) ++pi;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

}  // namespace tc
}  // namespace gqla
