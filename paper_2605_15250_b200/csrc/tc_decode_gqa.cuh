// GQA-path split-KV flash decoding on tcgen05 (Eq. (mha)).  A CTA works for one group j and walks
// the (sequence, split) pieces its plan gives it (sched.cuh): exactly one piece under the fixed
// plan, an equal share of the batch's 128-row tiles under the balanced plan (persistent CTA).
//
//   S = Q K^T   Q: the group's h_q/g heads x s_q queries (R rows), K = [K_C[:, j] ; k_R]  (192 wide)
//   O = P V     P = exp2(S * scale*log2e - m),  V = V[:, j]                                (128 wide)
//
// The MMA tile is 128 rows, the group only has (h_q/g)*s_q <= 128 of them.  Heads per group and query
// positions are each padded to a power of two (R rows in all; padding rows hold zeros or the next
// sequence's queries and are dropped at the store), and the R query rows
// are replicated F = 128/R times down the tile and replica f only keeps the scores of tokens
// [f*R, (f+1)*R) of each 128-token tile (its other probabilities are zero).  Every TMEM lane thus
// runs an independent online softmax over a disjoint token subset -- no cross-thread reduction in
// the main loop -- and the F partial (m, l, O) triples of a row are merged once per piece.
//
// Warp roles: warp 0 TMA producer, warp 1 MMA issuer (+ TMEM owner), warps 2-5 softmax (one TMEM
// lane per thread).  P goes back to TMEM as bf16 and is the A operand of the P.V MMA.  The three
// roles walk the same plan independently; ring slots and barrier phases follow a tile counter that
// runs across pieces, so the producer streams the next piece's tiles while the softmax warps still
// merge and store the previous one.
#pragma once
#include "common.cuh"
#include "sched.cuh"
#include "tc_common.cuh"

namespace gqla {
namespace tc {

struct GqaParams {
    int32_t B, S, s_q, h_q, g, hpg, hpg_box;
    int32_t balanced, W;  // balanced plan: W workers per (group, value block), grid = W * g * v_blocks
    int32_t v_blocks, d_v;  // value head dim d_v = 128 * v_blocks: a CTA computes one 128-column block of the output
                            // (v_blocks = 1 unless the value head dim differs from d_h, Sec. 3.2)
    float scale_log2;
    RowMap rows;  // packed or paged (pages a multiple of 128 rows, pieces starting on tile boundaries)
    const int32_t* seqlens;
    float* o_part;    // [B, S, s_q, h_q, d_v]
    float* lse_part;  // [B, S, s_q, h_q]
    int32_t* status;
};

struct GqaSmem {
    static constexpr int kQBytes = 3 * 16384;                // 128 rows x 192 bf16, three 64-wide k-blocks
    static constexpr int kKcBytes = 2 * 16384;               // 128 tokens x 128
    static constexpr int kKrBytes = 16384;                   // 128 tokens x 64
    static constexpr int kVBytes = 2 * 16384;                // 128 tokens x 128
    static constexpr int kStageBytes = kKcBytes + kKrBytes + kVBytes;
    static constexpr int kStages = 2;
    // floats per lane row of the merge buffer: 32 output columns + the row's (m, l) + 2 spare; a pitch of
    // 36 words keeps 16-byte accesses of a quarter warp on distinct banks
    static constexpr int kMergePitch = 36;
    static constexpr int kMergeBytes = 128 * kMergePitch * 4;
    static constexpr int kOffMerge = kQBytes + kStages * kStageBytes;
    static constexpr int kTileBytes = kOffMerge + kMergeBytes;
    // q_full q_empty o_free kfull[2] vfull[2] kempty[2] vempty[2] s_full[2] p_ready[2] pv_done[2]
    static constexpr int kNumBars = 17;
    static constexpr int kThreads = 192;
    // behind the barriers: tmem slot + abort flag (16 B).  The merge buffer doubles as the plan scratch.
    static constexpr int kTotal = kTileBytes + kNumBars * 8 + 16;
    static_assert(kMergeBytes >= (kThreads + 4) * 4, "plan scratch must fit in the merge buffer");
    static_assert(kTotal <= 232448, "shared memory budget of one CTA");
    static_assert(OneCtaPerSM<kTotal>::value, "");
};

// TMEM columns (all 512 are used, so one CTA per SM)
constexpr uint32_t kColS = 0;    // two 128-column score buffers
constexpr uint32_t kColP = 256;  // two 64-column bf16 probability buffers
constexpr uint32_t kColO = 384;  // 128-column output accumulator
constexpr float kRescaleThreshold = 8.0f;  // log2 units: P may grow to 2^8 before O is rescaled

template <int R>
__global__ void __launch_bounds__(GqaSmem::kThreads, 1)
decode_gqa_tc_kernel(const GqaParams p, const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                     const __grid_constant__ CUtensorMap tmR, const __grid_constant__ CUtensorMap tmV) {
    using L = GqaSmem;
    constexpr int F = 128 / R;
    // TMEM loads/stores take one address per warp.  A warp's 32 lanes cover 32/R replicas when R < 32, so
    // the warp reads the 32-column window of its lanes' sub-blocks and each thread keeps its own R columns.
    constexpr int W = R < 32 ? 32 : R;   // columns of S a warp reads per tile
    constexpr int CH = 32;
    constexpr int NCH = W / CH;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* tiles = smem_raw;
    if ((smem_u32(tiles) & 1023u) != 0) {  // swizzled tiles need 1 KB alignment
        if (threadIdx.x == 0 && p.status != nullptr) atomicCAS(p.status, 0, kStatusTimeout | (15 << 8));
        return;
    }
    uint8_t* q_smem = tiles;
    uint8_t* stage0 = tiles + L::kQBytes;
    float* merge = reinterpret_cast<float*>(tiles + L::kOffMerge);
    uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + L::kTileBytes);
    uint64_t* q_full = bars + 0;
    uint64_t* q_empty = bars + 1;  // the last Q K^T of a piece has completed: Q may be overwritten
    uint64_t* o_free = bars + 2;   // the softmax warps have read O of a piece: P.V may overwrite it
    uint64_t* kfull = bars + 3;    // [2]
    uint64_t* vfull = bars + 5;    // [2]
    uint64_t* kempty = bars + 7;   // [2]
    uint64_t* vempty = bars + 9;   // [2]
    uint64_t* s_full = bars + 11;  // [2]
    uint64_t* p_ready = bars + 13; // [2]
    uint64_t* pv_done = bars + 15; // [2]: P.V of tile n arrives on pv_done[n & 1]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + L::kNumBars);
    volatile int32_t* abort_flag = reinterpret_cast<volatile int32_t*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const Abort ab{abort_flag, p.status};

    if (threadIdx.x == 0) {
        // o_free and p_ready[2] take one arrival per softmax warp
        for (int i = 0; i < L::kNumBars; ++i) mbar_init(&bars[i], (i == 2 || i == 13 || i == 14) ? 4 : 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 512);
        tmem_relinquish();
    }

    pdl_launch_dependents();
    pdl_wait();  // barriers and TMEM are set up; everything below reads the caller's tensors
    // the plan of this CTA: group j, and either one (sequence, split) piece or worker w's share
    // consecutive CTAs: the value blocks of a group, then the groups of the same rows (they share k_R and K_C tiles
    // through L2)
    const int vb = blockIdx.x % p.v_blocks;
    const int j = (blockIdx.x / p.v_blocks) % p.g;
    const int unit = blockIdx.x / (p.v_blocks * p.g);
    Walker walk;
    if (p.balanced) {
        const BalancedStart st = balanced_prepass(p.seqlens, p.B, p.S, unit, p.W, reinterpret_cast<int32_t*>(merge), L::kThreads);
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
                // Q of this piece's sequence; the previous piece's Q K^T must all have completed
                if (pi > 0 && !(ok = mbar_wait(q_empty, (pi - 1) & 1, ab, 13))) break;
                mbar_expect_tx(q_full, L::kQBytes);
                for (int kb = 0; kb < 3; ++kb)
                    for (int f = 0; f < F; ++f)
                        asm volatile(
                            "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], "
                            "[%1, {%3, %4, %5, %6}], [%2];" ::"r"(smem_u32(q_smem + kb * 16384 + f * R * 128)),
                            "l"(reinterpret_cast<uint64_t>(&tmQ)), "r"(smem_u32(q_full)), "r"(kb * 64), "r"(0), "r"(j),
                            "r"(pc.b * p.s_q)
                            : "memory");
                int64_t tile_row = p.rows.row(pc.b, pc.tok_begin);
                for (int t = 0; t < pc.n_tiles; ++t, ++gt) {
                    const int s = gt & 1;
                    const uint32_t ph = (gt >> 1) & 1;
                    uint8_t* st = stage0 + s * L::kStageBytes;
                    const int32_t row = (int32_t)tile_row;
                    // the next tile's row is fetched while this tile's slots are waited for; a tile never straddles a page
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
            constexpr uint32_t idesc_qk = idesc_bf16(128, 128, 0, 0);
            constexpr uint32_t idesc_pv = idesc_bf16(128, 128, 0, 1);
            const uint32_t q_addr = smem_u32(q_smem);
            auto issue_qk = [&](int n) -> bool {  // n: running tile number
                const int s = n & 1;
                if (!mbar_wait(&kfull[s], (n >> 1) & 1, ab, 3)) return false;
                tc_fence_after();
                const uint32_t st = smem_u32(stage0 + s * L::kStageBytes);
                const uint32_t d = tmem_base + kColS + (uint32_t)s * 128;
#pragma unroll
                for (int kb = 0; kb < 3; ++kb)
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        umma_ss(d, desc_kmajor_sw128(q_addr + kb * 16384 + ks * 32),
                                desc_kmajor_sw128(st + kb * 16384 + ks * 32), idesc_qk, (kb | ks) != 0);
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
                        umma_commit(q_empty);  // every Q K^T of this piece has been issued
                    }
                    if (!(ok = mbar_wait(&p_ready[s], ph, ab, 5))) break;
                    // the first P.V of a piece overwrites O: the previous piece's O must have been read
                    if (t == 0 && pi > 0 && !(ok = mbar_wait(o_free, (pi - 1) & 1, ab, 14))) break;
                    if (!(ok = mbar_wait(&vfull[s], ph, ab, 6))) break;
                    tc_fence_after();
                    const uint32_t v_addr = smem_u32(stage0 + s * L::kStageBytes + L::kKcBytes + L::kKrBytes);
#pragma unroll
                    for (int ks = 0; ks < 8; ++ks)
                        umma_ts(tmem_base + kColO, tmem_base + kColP + (uint32_t)s * 64 + ks * 8,
                                desc_mnmajor_sw128(v_addr + ks * 2048, 16384), idesc_pv, (t | ks) != 0);
                    umma_commit(&vempty[s]);
                    umma_commit(&pv_done[s]);
                }
                gt += pc.n_tiles;
                ++pi;
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax: one TMEM lane per thread
        const int q = warp & 3;
        const int Lr = q * 32 + lane;        // TMEM lane == tile row
        const int r = Lr % R;                // logical query row
        const int f = Lr / R;                // replica: token sub-block of every tile
        const int pq = r / p.hpg_box;        // query position within the step
        const int il = r % p.hpg_box;        // head within the group
        const bool row_valid = il < p.hpg && pq < p.s_q;  // padding rows are computed and dropped
        const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
        const int col0 = R < 32 ? q * 32 : f * R;  // first column of the warp's window (warp-uniform)
        const int sub = R < 32 ? lane / R : 0;     // which R-column sub-block of the window is this thread's
        auto owns = [&](int c) -> bool { return R >= 32 || (c / R) == sub; };
        const int mcg = Lr & 7, mrow0 = Lr >> 3;  // merge: group of four output columns and first row of this thread

        {   // a thread only ever writes its own columns of P; everything else stays zero for good
            uint32_t z[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) z[i] = 0u;
#pragma unroll
            for (int c = 0; c < 128; c += 32) tmem_st32(lane_base + kColP + c, z);
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
            // split slots this worker marks empty
            if (f == 0 && row_valid && vb == 0)
                for (int kk = pc.fill_begin; kk < pc.fill_end; ++kk)
                    p.lse_part[((slot0 + kk) * p.s_q + pq) * p.h_q + (int64_t)j * p.hpg + il] = -INFINITY;
            if (pc.n_tiles == 0 && p.balanced) continue;  // an empty sequence: its slots were marked above
            int32_t lim = visible_limit(T, p.s_q, pq);
            if (lim > pc.tok_end) lim = pc.tok_end;
            lim -= pc.tok_begin;                 // visible tokens of this piece, relative to its first row
            float m_used = -INFINITY, l = 0.f;
            bool ok = true;

            for (int t = 0; t < pc.n_tiles && ok; ++t) {
                const int n = gt + t;
                const int s = n & 1;
                ok = __all_sync(0xffffffffu, mbar_wait(&s_full[s], (n >> 1) & 1, ab, 7));
                if (!ok) break;
                tc_fence_after();
                const uint32_t s_addr = lane_base + kColS + (uint32_t)s * 128 + col0;
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
                const float m_t = mx * p.scale_log2;  // -inf when nothing is visible
                const bool need = m_t > m_used + kRescaleThreshold;
                const float factor = need ? ex2(m_used - m_t) : 1.f;  // ex2(-inf) = 0 on first use
                if (__any_sync(0xffffffffu, need) && t > 0) {
                    // O is only touched between P.V(n-1) completing and P.V(n) being issued.  A warp may run one
                    // tile ahead of the others, so completions are counted on two alternating barriers: with a
                    // single one, parity alone could not tell "P.V(n-1) done" from "P.V(n-3) done".
                    ok = __all_sync(0xffffffffu, mbar_wait(&pv_done[(n - 1) & 1], ((n - 1) >> 1) & 1, ab, 8));
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll 1
                    for (int c = 0; c < 128; c += 32) {
                        uint32_t o[32];
                        tmem_ld32(lane_base + kColO + c, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * factor);
                        tmem_st32(lane_base + kColO + c, o);
                    }
                    tmem_wait_st();
                }
                if (need) {
                    l *= factor;
                    m_used = m_t;
                }
                const float m_sub = m_used == -INFINITY ? 0.f : m_used;
                const uint32_t p_addr = lane_base + kColP + (uint32_t)s * 64 + col0 / 2;
#pragma unroll
                for (int ch = 0; ch < NCH; ++ch) {
                    if (NCH > 1) {
                        tmem_ld<CH>(s_addr + ch * CH, x);
                        tmem_wait_ld();
                    }
                    uint32_t pk[CH / 2];
#pragma unroll
                    for (int c = 0; c < CH; c += 2) {
                        const int tok = tok0 + ch * CH + c;
                        const bool mine = owns(c);  // R is even, so c and c+1 share an owner
                        const float e0 = (mine && tok < lim) ? ex2(fmaf(__uint_as_float(x[c]), p.scale_log2, -m_sub)) : 0.f;
                        const float e1 =
                            (mine && tok + 1 < lim) ? ex2(fmaf(__uint_as_float(x[c + 1]), p.scale_log2, -m_sub)) : 0.f;
                        l += e0 + e1;
                        pk[c / 2] = pack_bf16(e0, e1);
                    }
                    tmem_st<CH / 2>(p_addr + ch * (CH / 2), pk);
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&p_ready[s]);
            }

            // -------------------------------------------------------------- merge the F replicas of each row
            const int n_last = gt + pc.n_tiles - 1;
            if (pc.n_tiles > 0 && ok)
                ok = __all_sync(0xffffffffu, mbar_wait(&pv_done[n_last & 1], (n_last >> 1) & 1, ab, 9));
            tc_fence_after();
            merge[Lr * L::kMergePitch + 32] = m_used;
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
            const float w = (live && m_used > -INFINITY) ? ex2(m_used - M) / Lt : 0.f;
            const int64_t out_row0 = ((slot0 + pc.k) * p.s_q) * p.h_q + (int64_t)j * p.hpg;
            // 32 output columns at a time through the merge buffer: lane rows in (16-byte stores), sums of the
            // F replicas out (thread = four columns of every 16th row; 16-byte loads and global stores)
#pragma unroll 1
            for (int c4 = 0; c4 < 4; ++c4) {
                uint32_t o[32];
                if (pc.n_tiles > 0 && ok) {  // warp-uniform
                    tmem_ld32(lane_base + kColO + c4 * 32, o);
                    tmem_wait_ld();
                }
                float4* mrow = reinterpret_cast<float4*>(merge + Lr * L::kMergePitch);
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    mrow[i] = w == 0.f ? make_float4(0.f, 0.f, 0.f, 0.f)
                                       : make_float4(__uint_as_float(o[4 * i]) * w, __uint_as_float(o[4 * i + 1]) * w,
                                                     __uint_as_float(o[4 * i + 2]) * w, __uint_as_float(o[4 * i + 3]) * w);
                if (c4 == 3) {  // O has been read: the next piece's first P.V may overwrite it
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
                        const float4 x = *reinterpret_cast<const float4*>(merge + (ff * R + rr) * L::kMergePitch + 4 * mcg);
                        acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
                    }
                    *reinterpret_cast<float4*>(p.o_part + (out_row0 + (int64_t)pp * p.h_q + ii) * p.d_v + vb * 128 + c4 * 32 +
                                               4 * mcg) = acc;
                }
                named_bar_sync(1, 128);
            }
            if (f == 0 && row_valid && vb == 0)
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
