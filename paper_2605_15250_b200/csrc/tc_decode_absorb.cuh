// Absorb-path split-KV flash decoding on tcgen05 (Eq. (mqa), lines 3-5): a PAIR of CTAs (one
// 2-CTA cluster, cta_group::2 MMAs) works for one block of 128 query rows and walks the
// (sequence, split) pieces its plan gives it (sched.cuh): exactly one piece under the fixed plan,
// an equal share of the batch's 128-row tiles under the balanced plan (persistent pair).
//
//   S = Qh Kh^T    Qh: 128 rows (head, query) x 576,  Kh = [c ; k_R] rows of the latent cache
//   O = P  V       V = the first 512 columns of the same cache rows
//
// Why a pair: O for 128 rows x 512 fp32 columns is all 256 KB of one SM's tensor memory, leaving no
// room for S.  With a 2-CTA MMA of M = 128 each CTA holds 64 rows; its accumulators use all 128 TMEM
// lanes for half as many columns (lanes 0-63: columns [0, N/2), lanes 64-127: columns [N/2, N) of
// the same 64 rows), so O takes 256 columns and S (128 tokens) 64.  Each CTA also supplies half of
// every B operand from its own shared memory: 64 of the tile's 128 cache rows for S = Qh Kh^T, and
// 128 of every 256 latent columns for O = P V.  The cache is fetched from HBM once; the second
// operand shape comes out of L2 ([64 rows x 64 columns] 8 KB boxes, 128-byte swizzle).
//
// Staging: two rings per CTA, one of K groups (three 8 KB boxes = 192 columns of 64 rows) and one of
// V groups (two box pairs = one token half of a tile), each one tile deep, each filled by a producer
// thread of its own (a thread issues a tensor load only every few hundred cycles, and a tile needs 17);
// the loads of tile t+1 are in flight while the MMAs of tile t run, and the K loads of the next piece
// while this piece is stored.
// Barriers are per group, not per box: every barrier operation of the issuing threads costs on the
// order of 100 cycles next to tensor-core operand traffic, and one MMA of this shape is only 32-64
// cycles of tensor work.
//
// Warp roles per CTA: warp 0 TMA producer of Q and K, warp 1 TMEM owner (+ MMA issuer in the leader CTA),
// warps 2-9 softmax, warp 10 TMA producer of V.  A softmax thread owns one TMEM lane = (row, token half)
// and one half of that lane's 64 score columns, so a row's 128 scores of a tile sit in four threads of
// four different warps; they share the tile maximum through shared memory and keep separate partial sums.
#pragma once
#include "common.cuh"
#include "sched.cuh"
#include "tc_common.cuh"

namespace gqla {
namespace tc {

struct AbsorbParams {
    int32_t B, S, s_q, h_q, rows_total /* s_q*h_q */, row_blocks /* ceil(rows_total/128) */;
    int32_t balanced, W;  // balanced plan: W pairs per row block, grid = 2 * W * row_blocks
    float scale_log2;
    RowMap rows;      // packed or paged (pages a multiple of 128 rows, pieces starting on tile boundaries)
    const int32_t* seqlens;
    float* o_part;    // [B, S, s_q*h_q, 512]
    float* lse_part;  // [B, S, s_q*h_q]
    __nv_bfloat16* o_final;  // not null: S = 1, fixed plan; the normalised output goes here as bf16 [B, s_q*h_q, 512]
                             // (o_part unused, lse_part may be null)
    int32_t* status;
};

struct AbsorbSmem {
    static constexpr int kBox = 8192;              // 64 rows x 64 bf16, 128-byte swizzle
    static constexpr int kQBytes = 9 * kBox;       // 64 query rows x 576
    static constexpr int kPBytes = 2 * kBox;       // 64 rows x 128 tokens (two 64-token k-blocks)
    static constexpr int kKGroup = 3 * kBox;       // three column blocks of this CTA's 64 rows of a tile
    static constexpr int kVGroup = 4 * kBox;       // 64 tokens x this CTA's 2 x 128 latent columns
    static constexpr int kNK = 3;                  // ring of K groups (Qh Kh^T operand): one tile
    static constexpr int kNV = 2;                  // ring of V groups (P V operand): one tile
    static constexpr int kOffK = kQBytes;
    static constexpr int kOffP = kOffK + kNK * kKGroup;
    static constexpr int kOffV = kOffP + kPBytes;
    static constexpr int kTileBytes = kOffV + kNV * kVGroup;
    // kfull[kNK] kempty[kNK] vfull[kNV] vempty[kNV] q_full q_empty o_free epi_done s_full[2] p_ready[2]
    // pv_done[2] xch[2] fin epi
    static constexpr int kNumBars = 2 * kNK + 2 * kNV + 14;
    static constexpr int kSoftmaxWarps = 8;
    static constexpr int kVProducerWarp = 2 + kSoftmaxWarps;  // behind the softmax warps
    static constexpr int kThreads = 96 + 32 * kSoftmaxWarps;
    // output staging for the epilogue (P and the V ring, idle once the last P.V of a piece has completed):
    // 64 rows x 256 fp32 (the columns of one MMA m) per pass, padded pitch
    static constexpr int kOutPitch = 256 * 4 + 16;
    static_assert(64 * kOutPitch <= kPBytes + kNV * kVGroup, "output staging must fit in P + V ring");
    // behind the barriers: tmem slot + abort flag (16 B), sm_max [2][4][64] (sm_l [4][64] and the plan
    // scratch reuse it).  No slack for re-aligning the base: the kernel checks the 1 KB alignment.
    static constexpr int kTotal = kTileBytes + kNumBars * 8 + 16 + 2 * 4 * 64 * 4;
    static_assert(2 * 4 * 64 >= kThreads + 4, "plan scratch must fit in sm_max");
    static_assert(kTotal <= 232448, "shared memory budget of one CTA");
    static_assert(OneCtaPerSM<kTotal>::value, "");
};

constexpr uint32_t kAColO = 0;    // O: MMA m (latent columns [256m, 256m+256)) at TMEM columns [128m, 128m+128)
constexpr uint32_t kAColS = 256;  // two 64-column score buffers

template <int DUMMY>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(AbsorbSmem::kThreads, 1)
decode_absorb_tc_kernel(const AbsorbParams p, const __grid_constant__ CUtensorMap tmQ,
                        const __grid_constant__ CUtensorMap tmC) {
    using L = AbsorbSmem;
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* tiles = smem_raw;
    if ((smem_u32(tiles) & 1023u) != 0) {  // swizzled tiles need 1 KB alignment; same answer in both CTAs
        if (threadIdx.x == 0 && p.status != nullptr) atomicCAS(p.status, 0, kStatusTimeout | (15 << 8));
        return;
    }
    uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + L::kTileBytes);
    uint64_t* kfull = bars;
    uint64_t* kempty = kfull + L::kNK;
    uint64_t* vfull = kempty + L::kNK;
    uint64_t* vempty = vfull + L::kNV;
    uint64_t* q_full = vempty + L::kNV;
    uint64_t* q_empty = q_full + 1;    // every Qh Kh^T of a piece has completed: Q may be overwritten
    uint64_t* o_free = q_empty + 1;    // leader only: both CTAs' softmax warps have read O of a piece
    uint64_t* epi_done = o_free + 1;   // this CTA's output staging (P + V ring) is free again
    uint64_t* s_full = epi_done + 1;   // [2]
    uint64_t* p_ready = s_full + 2;    // [2] leader only: one arrival per softmax warp of the pair
    uint64_t* pv_done = p_ready + 2;   // [2]
    uint64_t* xch = pv_done + 2;       // [2] softmax warps of this CTA: per-tile max exchange
    uint64_t* fin = xch + 2;           //     the final partial-sum exchange of a piece
    uint64_t* epi = fin + 1;           //     and the steps of the output staging
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + L::kNumBars);
    volatile int32_t* abort_flag = reinterpret_cast<volatile int32_t*>(tmem_slot + 1);
    float* sm_max = reinterpret_cast<float*>(tmem_slot + 4);  // [2][4][64] per-tile partial maxima
    // [4][64] final partial sums; written only after the last P.V of a piece, i.e. after every warp has
    // arrived on p_ready of its last tile and hence finished reading sm_max
    float* sm_l = sm_max;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta = cluster_ctarank();  // 0 = leader
    const Abort ab{abort_flag, p.status};

    if (threadIdx.x == 0) {
        for (int i = 0; i < L::kNumBars; ++i) {
            uint64_t* bar = &bars[i];
            const bool pair_wide = bar == &p_ready[0] || bar == &p_ready[1] || bar == o_free;
            const bool cta_wide = bar == &xch[0] || bar == &xch[1] || bar == fin || bar == epi || bar == epi_done;
            mbar_init(bar, pair_wide ? 2 * L::kSoftmaxWarps : (cta_wide ? L::kSoftmaxWarps : 1));
        }
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc2(tmem_slot, 512);
        tmem_relinquish2();
    }

    pdl_launch_dependents();
    pdl_wait();  // barriers and TMEM are set up; everything below reads the caller's tensors
    // the plan of this pair: row block rb, and either one (sequence, split) piece or worker w's share
    const int pair = blockIdx.x >> 1;
    const int rb = pair % p.row_blocks;
    Walker walk;
    if (p.balanced) {
        const BalancedStart st = balanced_prepass(p.seqlens, p.B, p.S, pair / p.row_blocks, p.W,
                                                  reinterpret_cast<int32_t*>(sm_max), L::kThreads);
        walk.init_balanced(p.seqlens, p.B, p.S, pair / p.row_blocks, p.W, st);
    } else {
        const int unit = pair / p.row_blocks;
        walk.init_fixed(p.seqlens, p.B, p.S, unit / p.S, unit % p.S);
    }
    const int rho0 = rb * 128 + (int)cta * 64;  // first (query, head) row of this CTA
    tc_fence_before();
    __syncthreads();
    cluster_sync();  // both CTAs' barriers exist before any remote arrival
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    Piece pc;
    int pi = 0;  // non-empty pieces walked so far (phase of the per-piece barriers)

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer of Q and the K ring
        // (both CTAs).  Every "full" barrier lives in the leader and counts the bytes of BOTH CTAs.
        if (elect_one()) {
            tma_prefetch_desc(&tmQ);
            tma_prefetch_desc(&tmC);
            const uint32_t q_full_l = mapa(smem_u32(q_full), 0);
            int ks = 0;
            uint32_t kph = 1;  // parity that means "slot is free"
            bool ok = true;
            while (ok && walk.next(pc)) {
                if (pc.n_tiles == 0) continue;
                // Q rows of this piece's sequence; the previous piece's Qh Kh^T must all have completed
                if (pi > 0 && !(ok = mbar_wait(q_empty, (pi - 1) & 1, ab, 13))) break;
                if (cta == 0) mbar_expect_tx(q_full, 2 * L::kQBytes);
                for (int kb = 0; kb < 9; ++kb)
                    tma_load_2d_pair(tiles + kb * L::kBox, &tmQ, kb * 64, pc.b * p.rows_total + rho0, q_full_l);
                // K groups in the order (tile, column third); a tile never straddles a page
                int64_t tile_row = p.rows.row(pc.b, pc.tok_begin);
                for (int kt = 0; kt < pc.n_tiles && ok; ++kt) {
                    const int32_t row = (int32_t)(tile_row + cta * 64);
                    // the next tile's row is fetched while this tile's slots are waited for
                    if (kt + 1 < pc.n_tiles)
                        tile_row = p.rows.paged() ? p.rows.row(pc.b, pc.tok_begin + (kt + 1) * 128) : tile_row + 128;
#pragma unroll 1
                    for (int kg = 0; kg < 3; ++kg) {
                        if (!(ok = mbar_wait(&kempty[ks], kph, ab, 1))) break;
                        if (cta == 0) mbar_expect_tx(&kfull[ks], 2 * L::kKGroup);
                        const uint32_t bar = mapa(smem_u32(&kfull[ks]), 0);
                        uint8_t* dst = tiles + L::kOffK + ks * L::kKGroup;
#pragma unroll
                        for (int i = 0; i < 3; ++i) tma_load_2d_pair(dst + i * L::kBox, &tmC, (3 * kg + i) * 64, row, bar);
                        if (++ks == L::kNK) { ks = 0; kph ^= 1; }
                    }
                }
                ++pi;
            }
        }
    } else if (warp == L::kVProducerWarp) {
        // ------------------------------------------------------------------ TMA producer of the V ring (both
        // CTAs).  A thread issues a tensor load only every few hundred cycles, and a tile needs 17 of them:
        // the two rings are fed by two threads.  V groups in the order (tile, token half); a V slot is free
        // only after P.V of the previous tile, i.e. after Qh Kh^T of this tile has read the same cache rows
        // as K boxes, so the V boxes come out of L2.
        if (elect_one()) {
            int vs = 0;
            uint32_t vph = 1;
            bool ok = true;
            while (ok && walk.next(pc)) {
                if (pc.n_tiles == 0) continue;
                // the V ring doubles as the output staging of the previous piece
                if (pi > 0 && !(ok = mbar_wait(epi_done, (pi - 1) & 1, ab, 16))) break;
                int64_t tile_row = p.rows.row(pc.b, pc.tok_begin);
                for (int vt = 0; vt < pc.n_tiles && ok; ++vt) {
                    const int64_t row0 = tile_row;
                    if (vt + 1 < pc.n_tiles)
                        tile_row = p.rows.paged() ? p.rows.row(pc.b, pc.tok_begin + (vt + 1) * 128) : tile_row + 128;
#pragma unroll 1
                    for (int vh = 0; vh < 2; ++vh) {
                        if (!(ok = mbar_wait(&vempty[vs], vph, ab, 2))) break;
                        if (cta == 0) mbar_expect_tx(&vfull[vs], 2 * L::kVGroup);
                        const int32_t row = (int32_t)(row0 + vh * 64);
                        const uint32_t bar = mapa(smem_u32(&vfull[vs]), 0);
                        uint8_t* dst = tiles + L::kOffV + vs * L::kVGroup;
                        // box (m, i): latent columns [256m + 128cta + 64i, +64) -- this CTA's half of MMA m's N
#pragma unroll
                        for (int mi = 0; mi < 4; ++mi)
                            tma_load_2d_pair(dst + mi * L::kBox, &tmC, 256 * (mi >> 1) + 128 * (int)cta + 64 * (mi & 1), row,
                                             bar);
                        if (++vs == L::kNV) { vs = 0; vph ^= 1; }
                    }
                }
                ++pi;
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (cta == 0 && elect_one()) {
            constexpr uint32_t idesc_qk = idesc_bf16(128, 128, 0, 0);
            constexpr uint32_t idesc_pv = idesc_bf16(128, 256, 0, 1);
            const uint64_t q_desc = desc_kmajor_sw128(smem_u32(tiles));
            const uint64_t p_desc = desc_kmajor_sw128(smem_u32(tiles + L::kOffP));
            int ks = 0, vs = 0;
            uint32_t kph = 0, vph = 0;
            int gt = 0;  // tiles issued so far: score buffer = gt & 1, phase = (gt >> 1) & 1
            auto issue_qk = [&](int n) -> bool {
                const uint32_t d = tmem_base + kAColS + (uint32_t)(n & 1) * 64;
#pragma unroll 1
                for (int g3 = 0; g3 < 3; ++g3) {
                    if (!mbar_wait_fast(&kfull[ks], kph, ab, 3)) return false;
                    tc_fence_after();
                    // descriptors as low words: the high word is a constant, stepping is one 32-bit add
                    const uint32_t kd = desc_lo(desc_kmajor_sw128(smem_u32(tiles + L::kOffK + ks * L::kKGroup)));
                    const uint32_t qd = desc_lo(q_desc) + ((g3 * 3 * L::kBox) >> 4);
                    if (g3 == 0)
                        umma_ss2_lo<false>(d, qd, kd, idesc_qk);  // the tile's first MMA overwrites S
                    else
                        umma_ss2_lo<true>(d, qd, kd, idesc_qk);
#pragma unroll
                    for (int i = 0; i < 3; ++i)
#pragma unroll
                        for (int kk = 0; kk < 4; ++kk)
                            if ((i | kk) != 0)
                                umma_ss2_lo<true>(d, qd + ((i * L::kBox + kk * 32) >> 4), kd + ((i * L::kBox + kk * 32) >> 4),
                                                  idesc_qk);
                    umma_commit2(&kempty[ks], 3);
                    if (++ks == L::kNK) { ks = 0; kph ^= 1; }
                }
                umma_commit2(&s_full[n & 1], 3);
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
                    if (t + 1 < pc.n_tiles) {
                        if (!(ok = issue_qk(n + 1))) break;
                    } else {
                        umma_commit2(q_empty, 3);  // every Qh Kh^T of this piece has been issued
                    }
                    if (!(ok = mbar_wait_fast(&p_ready[n & 1], (n >> 1) & 1, ab, 5))) break;
                    // the first P.V of a piece overwrites O: the previous piece's O must have been read
                    if (t == 0 && pi > 0 && !(ok = mbar_wait(o_free, (pi - 1) & 1, ab, 14))) break;
                    tc_fence_after();
#pragma unroll 1
                    for (int h = 0; h < 2; ++h) {
                        if (!(ok = mbar_wait_fast(&vfull[vs], vph, ab, 6))) break;
                        tc_fence_after();
                        const uint32_t vd = desc_lo(desc_mnmajor_sw128(smem_u32(tiles + L::kOffV + vs * L::kVGroup), L::kBox));
                        const uint32_t pd = desc_lo(p_desc) + ((h * L::kBox) >> 4);
#pragma unroll
                        for (int m = 0; m < 2; ++m) {
                            const uint32_t dm = tmem_base + kAColO + (uint32_t)m * 128;
                            if ((t | h) == 0)
                                umma_ss2_lo<false>(dm, pd, vd + ((m * 2 * L::kBox) >> 4), idesc_pv);  // first P.V of a piece
                            else
                                umma_ss2_lo<true>(dm, pd, vd + ((m * 2 * L::kBox) >> 4), idesc_pv);
#pragma unroll
                            for (int kk = 1; kk < 4; ++kk)
                                umma_ss2_lo<true>(dm, pd + ((kk * 32) >> 4), vd + ((m * 2 * L::kBox + kk * 2048) >> 4), idesc_pv);
                        }
                        umma_commit2(&vempty[vs], 3);
                        if (++vs == L::kNV) { vs = 0; vph ^= 1; }
                    }
                    if (ok) umma_commit2(&pv_done[n & 1], 3);
                }
                gt += pc.n_tiles;
                ++pi;
            }
        }
    } else {
        // ------------------------------------------------------------------ softmax
        const int q = warp & 3;              // TMEM lane quadrant this warp may access
        const int ch = (warp - 2) >> 2;      // which 32 of the lane's 64 score columns
        const int Lr = q * 32 + lane;        // TMEM lane
        const int r = Lr & 63;               // row within this CTA
        const int hf = Lr >> 6;              // token half of each 128-token tile / column half of each O block
        const int part = hf * 2 + ch;        // one of the four threads of row r
        const int rho = rho0 + r;            // (query, head) row of the sequence
        const bool row_valid = rho < p.rows_total;
        const int pq = row_valid ? rho / p.h_q : 0;
        const uint32_t lane_base = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t p_ready_l[2] = {mapa(smem_u32(&p_ready[0]), 0), mapa(smem_u32(&p_ready[1]), 0)};
        const uint32_t o_free_l = mapa(smem_u32(o_free), 0);
        int gt = 0;  // tiles walked so far
        int ec = 0;  // completed phases of the `epi` barrier

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
            if (part == 0 && row_valid && p.lse_part != nullptr)
                for (int kk = pc.fill_begin; kk < pc.fill_end; ++kk) p.lse_part[(slot0 + kk) * p.rows_total + rho] = -INFINITY;
            if (pc.n_tiles == 0 && p.balanced) continue;  // an empty sequence: its slots were marked above
            int32_t lim = visible_limit(T, p.s_q, pq);
            if (lim > pc.tok_end) lim = pc.tok_end;
            lim -= pc.tok_begin;
            if (!row_valid) lim = 0;
            float m_used = -INFINITY, l = 0.f;
            bool ok = true;

            for (int t = 0; t < pc.n_tiles && ok; ++t) {
                const int n = gt + t;
                const int sb = n & 1;
                const uint32_t nph = (n >> 1) & 1;
                ok = __all_sync(0xffffffffu, mbar_wait(&s_full[sb], nph, ab, 7));
                if (!ok) break;
                tc_fence_after();
                const int tok0 = t * 128 + hf * 64 + ch * 32;
                uint32_t x[32];
                tmem_ld32(lane_base + kAColS + (uint32_t)sb * 64 + ch * 32, x);
                tmem_wait_ld();
                const bool full = tok0 + 32 <= lim;  // every score of this thread is visible
                float mx = -INFINITY;
                if (full) {
#pragma unroll
                    for (int c = 0; c < 32; ++c) mx = fmaxf(mx, __uint_as_float(x[c]));
                } else {
#pragma unroll
                    for (int c = 0; c < 32; ++c)
                        if (tok0 + c < lim) mx = fmaxf(mx, __uint_as_float(x[c]));
                }
                // the other three parts of this row live in other warps
                float* mxs = sm_max + sb * 256;
                mxs[part * 64 + r] = mx;
                __syncwarp();
                if (lane == 0) mbar_arrive(&xch[sb]);
                ok = __all_sync(0xffffffffu, mbar_wait(&xch[sb], nph, ab, 10));
                if (!ok) break;
                mx = fmaxf(fmaxf(mxs[r], mxs[64 + r]), fmaxf(mxs[128 + r], mxs[192 + r]));
                const float m_t = mx * p.scale_log2;
                const bool need = m_t > m_used + 8.0f;
                const float factor = need ? ex2(m_used - m_t) : 1.f;
                if (need) {
                    l *= factor;
                    m_used = m_t;
                }
                const float m_sub = m_used == -INFINITY ? 0.f : m_used;
                uint32_t pk[16];
                if (full) {
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        const float e0 = ex2(fmaf(__uint_as_float(x[c]), p.scale_log2, -m_sub));
                        const float e1 = ex2(fmaf(__uint_as_float(x[c + 1]), p.scale_log2, -m_sub));
                        l += e0 + e1;
                        pk[c / 2] = pack_bf16(e0, e1);
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 32; c += 2) {
                        const float e0 = tok0 + c < lim ? ex2(fmaf(__uint_as_float(x[c]), p.scale_log2, -m_sub)) : 0.f;
                        const float e1 =
                            tok0 + c + 1 < lim ? ex2(fmaf(__uint_as_float(x[c + 1]), p.scale_log2, -m_sub)) : 0.f;
                        l += e0 + e1;
                        pk[c / 2] = pack_bf16(e0, e1);
                    }
                }
                // O may be rescaled, and the P buffer rewritten, only once P.V(n-1) has completed
                if (t > 0) {
                    ok = __all_sync(0xffffffffu, mbar_wait(&pv_done[(n - 1) & 1], ((n - 1) >> 1) & 1, ab, 8));
                    if (!ok) break;
                    tc_fence_after();
                }
                if (__any_sync(0xffffffffu, need) && t > 0) {
                    // this thread's share of the lane's O: columns [128m + 64ch, +64) for m = 0, 1
#pragma unroll 1
                    for (int c = 0; c < 4; ++c) {
                        const uint32_t col = kAColO + (uint32_t)(c >> 1) * 128 + ch * 64 + (c & 1) * 32;
                        uint32_t o[32];
                        tmem_ld32(lane_base + col, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * factor);
                        tmem_st32(lane_base + col, o);
                    }
                    tmem_wait_st();
                }
                // P row r, k-block hf: 128 bytes = 8 chunks of 8 bf16, chunk index XORed with (r & 7)
                uint8_t* prow = tiles + L::kOffP + hf * L::kBox + r * 128;
#pragma unroll
                for (int c4 = 0; c4 < 4; ++c4)
                    *reinterpret_cast<uint4*>(prow + (((ch * 4 + c4) ^ (r & 7)) << 4)) =
                        make_uint4(pk[4 * c4], pk[4 * c4 + 1], pk[4 * c4 + 2], pk[4 * c4 + 3]);
                fence_proxy_async_smem();  // generic-proxy writes of P -> visible to the tensor core
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(p_ready_l[sb]);
            }

            // -------------------------------------------------------------- epilogue: normalise and store
            const int n_last = gt + pc.n_tiles - 1;
            if (pc.n_tiles > 0 && ok)
                ok = __all_sync(0xffffffffu, mbar_wait(&pv_done[n_last & 1], (n_last >> 1) & 1, ab, 9));
            tc_fence_after();
            sm_l[part * 64 + r] = l;
            __syncwarp();
            if (lane == 0) mbar_arrive(fin);
            if (!__all_sync(0xffffffffu, mbar_wait(fin, pi & 1, ab, 11))) ok = false;
            const float Lt = (sm_l[r] + sm_l[64 + r]) + (sm_l[128 + r] + sm_l[192 + r]);
            const bool live = ok && pc.n_tiles > 0 && Lt > 0.f && m_used > -INFINITY;
            const float inv = live ? 1.f / Lt : 0.f;
            // The CTA's 64 output rows leave through shared memory (P and the V ring are idle now: the last
            // P.V has completed) as 1 KB bulk stores, the 256 columns of MMA m = 0 first, then those of m = 1.
            // The padded pitch keeps the 16-byte stores of a quarter warp on distinct banks.
            uint8_t* stage = tiles + L::kOffP;
            if (p.o_final != nullptr) {
                // whole-sequence call: the final bf16 rows (1 KB each) fit the staging at once -- one pass
                uint4* dst = reinterpret_cast<uint4*>(stage + r * L::kOutPitch + (128 * hf + 64 * ch) * 2);
#pragma unroll 1
                for (int mc = 0; mc < 4; ++mc) {  // (m, 32-column half) of this thread's 64 columns of each m
                    const int m = mc >> 1, c = (mc & 1) * 32;
                    uint32_t o[32];
                    if (pc.n_tiles > 0 && ok) {  // warp-uniform
                        tmem_ld32(lane_base + kAColO + m * 128 + ch * 64 + c, o);
                        tmem_wait_ld();
                    }
                    auto pk = [&](int e) -> uint32_t {  // columns e, e + 1 of this chunk, normalised (0 for a dead row)
                        return live ? pack_bf16(__uint_as_float(o[e]) * inv, __uint_as_float(o[e + 1]) * inv) : 0u;
                    };
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        dst[(256 * m + c) * 2 / 16 + i] = make_uint4(pk(8 * i), pk(8 * i + 2), pk(8 * i + 4), pk(8 * i + 6));
                }
                fence_proxy_async_smem();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive_cluster(o_free_l);
                if (lane == 0) mbar_arrive(epi);
                if (!__all_sync(0xffffffffu, mbar_wait(epi, ec & 1, ab, 12))) ok = false;
                ++ec;
                if (ok && lane < 8) {
                    const int rr = (warp - 2) * 8 + lane;
                    if (rho0 + rr < p.rows_total) {
                        bulk_store(p.o_final + ((int64_t)pc.b * p.rows_total + rho0 + rr) * 512, stage + rr * L::kOutPitch,
                                   512 * 2);
                        bulk_commit();
                        bulk_wait_read();
                    }
                }
            } else {
                float* gbase = p.o_part + ((slot0 + pc.k) * p.rows_total + rho0) * 512;
#pragma unroll 1
                for (int m = 0; m < 2; ++m) {
                    float4* dst = reinterpret_cast<float4*>(stage + r * L::kOutPitch + (128 * hf + 64 * ch) * 4);
#pragma unroll 1
                    for (int c = 0; c < 64; c += 32) {
                        uint32_t o[32];
                        if (pc.n_tiles > 0 && ok) {  // warp-uniform
                            tmem_ld32(lane_base + kAColO + m * 128 + ch * 64 + c, o);
                            tmem_wait_ld();
                        }
#pragma unroll
                        for (int i = 0; i < 8; ++i)
                            dst[c / 4 + i] =
                                live ? make_float4(__uint_as_float(o[4 * i]) * inv, __uint_as_float(o[4 * i + 1]) * inv,
                                                   __uint_as_float(o[4 * i + 2]) * inv, __uint_as_float(o[4 * i + 3]) * inv)
                                     : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                    fence_proxy_async_smem();  // staged rows -> visible to the bulk-copy engine
                    if (m == 1) {              // O has been read: the next piece's first P.V may overwrite it
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive_cluster(o_free_l);
                    }
                    __syncwarp();
                    if (lane == 0) mbar_arrive(epi);
                    if (!__all_sync(0xffffffffu, mbar_wait(epi, ec & 1, ab, 12))) ok = false;
                    ++ec;
                    if (ok && lane < 8) {
                        const int rr = (warp - 2) * 8 + lane;  // each softmax warp ships eight rows
                        if (rho0 + rr < p.rows_total) {
                            bulk_store(gbase + (int64_t)rr * 512 + 256 * m, stage + rr * L::kOutPitch, 256 * 4);
                            bulk_commit();
                            bulk_wait_read();
                        }
                    }
                    if (m == 0) {  // the staging is rewritten next: every warp's stores must have read it
                        __syncwarp();
                        if (lane == 0) mbar_arrive(epi);
                        if (!__all_sync(0xffffffffu, mbar_wait(epi, ec & 1, ab, 12))) ok = false;
                        ++ec;
                    }
                }
            }
            // staging (and with it P and the V ring) is free again once every warp's stores have read it
            __syncwarp();
            if (lane == 0) mbar_arrive(epi_done);
            if (!__all_sync(0xffffffffu, mbar_wait(epi_done, pi & 1, ab, 12))) ok = false;
            if (row_valid && part == 0 && p.lse_part != nullptr)
                p.lse_part[(slot0 + pc.k) * p.rows_total + rho] =
                    live ? (m_used + log2f(Lt)) * 0.6931471805599453f : -INFINITY;
            gt += pc.n_tiles;
            ++pi;
        }
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();  // neither CTA leaves while the other may still signal its barriers
    if (warp == 1) tmem_dealloc2(tmem_base, 512);
}

}  // namespace tc
}  // namespace gqla
