// Split merge fused with the latent up-projection (Eq. (mqa), line 6, applied to the log-sum-exp merge
// of the split partials):   o_i = W^UV_{j(i)} ( sum_k w_k o_hat_{i,k} ),  w_k = exp(lse_k - M) / sum exp.
// The merged latent output never goes to HBM: four builder warps read the fp32 partials (one warp per
// row, 512 contiguous bytes per load), weight and sum them, and write the bf16 A operand straight into
// shared memory in the 128-byte-swizzled K-major layout; warp 0 fetches W^UV[j] with TMA, warp 1 issues
// tcgen05.mma into a TMEM accumulator; the builder warps then store the 64 x 128 output tile.  Both
// operands are resident in full (r_kv <= 512), so every load of the CTA is in flight at once.
// One CTA = 64 rows = 64/hpg query positions x hpg heads of one group (M = 64 MMAs: twice as many CTAs as
// with 128-row tiles, and this kernel is bound by the latency of its loads, not by the tensor core);
// K = r_kv in chunks of 128.  With M = 64 the accumulator row m sits in TMEM lane (m % 16) + 32 (m / 16).
#pragma once
#include "tc_common.cuh"

namespace gqla {
namespace tc {

struct CombineUpParams {
    int32_t S, s_q, h_q, g, hpg, r_kv;
    int32_t hpb;            // heads per group padded to a power of two (head slots of a tile)
    int64_t positions;      // B * s_q
    const float* o_part;    // [B, S, s_q*h_q, r_kv]
    const float* lse_part;  // [B, S, s_q*h_q]
    void* out;              // [B, s_q, h_q, 128] bf16
    float* lse;             // [B, s_q, h_q] or null
    int32_t* status;
};

struct CombineUpSmem {
    static constexpr int kChunkK = 128;
    static constexpr int kRows = 64;
    static constexpr int kABytes = 2 * 8192;    // 64 rows x 128 k, two 64-wide k-blocks
    static constexpr int kBBytes = 4 * 8192;    // 128 k x 128 n: (k-block, n-block) boxes of 64 x 64
    static constexpr int kMaxChunks = 4;        // r_kv <= 512: the whole A and B operands are resident at once
    static constexpr int kTileBytes = kMaxChunks * (kABytes + kBBytes);
    static constexpr int kNumBars = 3;          // a_ready b_full acc_full
    static constexpr int kThreads = 192;
    static constexpr int kMaxS = 64;            // split slots the kernel takes (their lse is staged per row)
    static constexpr int kTotal = 1024 + kTileBytes + kNumBars * 8 + 16 + 2 * kRows * 4 + kRows * kMaxS * 4 + kRows * 8;
    static_assert(OneCtaPerSM<kTotal>::value, "");
};

__global__ void __launch_bounds__(CombineUpSmem::kThreads, 1)
combine_up_tc_kernel(const CombineUpParams p, const __grid_constant__ CUtensorMap tmB) {
    using L = CombineUpSmem;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* a_smem = tiles;
    uint8_t* b_smem = tiles + L::kMaxChunks * L::kABytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + L::kTileBytes);
    uint64_t* a_ready = bars;       // the four builder warps have written A
    uint64_t* b_full = bars + 1;
    uint64_t* acc_full = bars + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + L::kNumBars);
    volatile int32_t* abort_flag = reinterpret_cast<volatile int32_t*>(tmem_slot + 1);
    float* sm_M = reinterpret_cast<float*>(tmem_slot + 4);  // [64] row maximum of lse
    float* sm_inv = sm_M + L::kRows;                         // [64] 1 / sum_k exp(lse_k - M), 0 for a dead row
    float* sm_lse = sm_inv + L::kRows;                       // [64][kMaxS] lse of every split of every tile row
    // [64] first partial row of every tile row (-1: padding row); the index arithmetic has 64-bit divisions,
    // so it is done once per row, not once per load
    int64_t* sm_pr = reinterpret_cast<int64_t*>(sm_lse + L::kRows * L::kMaxS);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const Abort ab{abort_flag, p.status};
    const int m_tile = blockIdx.x, j = blockIdx.y;
    const int n_chunks = p.r_kv / L::kChunkK;
    const int rows_per_seq = p.s_q * p.h_q;
    pdl_launch_dependents();

    if (threadIdx.x == 0) {
        for (int i = 0; i < L::kNumBars; ++i) mbar_init(&bars[i], i == 0 ? 4 : 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, 128);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();  // set-up done; the partials come from the previous kernel of the stream

    if (warp == 0) {
        // ------------------------------------------------------------------ W^UV chunks (MN-major B operand)
        if (elect_one()) {
            tma_prefetch_desc(&tmB);
            mbar_expect_tx(b_full, n_chunks * L::kBBytes);
            for (int c = 0; c < n_chunks; ++c)
                for (int kb = 0; kb < 2; ++kb)
                    for (int nb = 0; nb < 2; ++nb)
                        tma_load_2d(b_smem + c * L::kBBytes + (kb * 2 + nb) * 8192, &tmB, nb * 64,
                                    j * p.r_kv + c * L::kChunkK + kb * 64, b_full);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (elect_one()) {
            constexpr uint32_t idesc = idesc_bf16(64, 128, 0, 1);
            bool ok = mbar_wait(b_full, 0, ab, 2);
            if (ok) ok = mbar_wait(a_ready, 0, ab, 3);
            tc_fence_after();
            for (int c = 0; c < n_chunks && ok; ++c) {
                const uint32_t a_addr = smem_u32(a_smem + c * L::kABytes);
                const uint32_t b_addr = smem_u32(b_smem + c * L::kBBytes);
#pragma unroll
                for (int kb = 0; kb < 2; ++kb)
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        umma_ss(tmem_base, desc_kmajor_sw128(a_addr + kb * 8192 + ks * 32),
                                desc_mnmajor_sw128(b_addr + kb * 16384 + ks * 2048, 8192), idesc, (c | kb | ks) != 0);
            }
            if (ok) umma_commit(acc_full);
        }
    } else {
        // ------------------------------------------------------------------ builders, then epilogue
        const int q = warp & 3;  // TMEM lane quadrant of this warp; it holds tile rows [16q, 16q + 16)
        // global row of tile row tr: position m_tile * (64/hpb) + tr / hpb, head j * hpg + tr % hpb (head
        // slots beyond the group's hpg heads stay empty)
        auto row_of = [&](int tr, int64_t* part_row, int64_t* out_row) -> bool {
            const int64_t pos = (int64_t)m_tile * (L::kRows / p.hpb) + tr / p.hpb;
            if (pos >= p.positions || tr % p.hpb >= p.hpg) return false;
            const int i = j * p.hpg + tr % p.hpb;
            const int64_t b = pos / p.s_q;
            const int pq = (int)(pos % p.s_q);
            *part_row = b * p.S * rows_per_seq + (int64_t)pq * p.h_q + i;  // split 0; + k * rows_per_seq
            *out_row = pos * p.h_q + i;
            return true;
        };
        // per-row softmax statistics over the S splits: lanes 0-15 = the warp's rows
        if (lane < 16) {
            const int tr = q * 16 + lane;
            int64_t pr = 0, orow = 0;
            float M = -INFINITY, inv = 0.f;
            if (row_of(tr, &pr, &orow)) {
                for (int k = 0; k < p.S; ++k) {
                    const float v = __ldg(p.lse_part + pr + (int64_t)k * rows_per_seq);
                    sm_lse[tr * L::kMaxS + k] = v;
                    M = fmaxf(M, v);
                }
                float den = 0.f;
                if (M > -INFINITY)
                    for (int k = 0; k < p.S; ++k) den += expf(sm_lse[tr * L::kMaxS + k] - M);
                inv = den > 0.f ? 1.f / den : 0.f;
                if (p.lse != nullptr) p.lse[orow] = den > 0.f ? M + logf(den) : -INFINITY;
            }
            sm_M[tr] = M;
            sm_inv[tr] = inv;
            sm_pr[tr] = row_of(tr, &pr, &orow) ? pr : -1;
        }
        __syncwarp();
        bool ok = true;
        {
            const int chunk16 = (lane & 15) >> 1, half = lane & 1;
            uint8_t* a_lane = a_smem + (lane >> 4) * 8192;  // k-block (within a chunk) of this lane's 4 columns
#pragma unroll 1
            for (int r0 = 0; r0 < 16; r0 += 4) {
                // 4 rows x all K chunks at a time: every load of a split slot is issued before any is used.
                // Within a fetched slot the loads are unconditional (the partial of a row for which the slot is
                // empty may hold anything: it is masked after the load).
                float4 acc[4][L::kMaxChunks];
                const float* src[4];
                float rM[4], rinv[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int tr = q * 16 + r0 + u;
                    const int64_t pr = sm_pr[tr];
                    const bool valid = pr >= 0;
                    rinv[u] = valid ? sm_inv[tr] : 0.f;
                    rM[u] = sm_M[tr];
                    src[u] = p.o_part + (valid ? pr : 0) * p.r_kv + 4 * lane;
#pragma unroll
                    for (int c = 0; c < L::kMaxChunks; ++c) acc[u][c] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
                for (int k = 0; k < p.S; ++k) {
                    float4 x[4][L::kMaxChunks];
                    float wk[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int tr = q * 16 + r0 + u;
                        wk[u] = rinv[u] == 0.f ? 0.f : expf(sm_lse[tr * L::kMaxS + k] - rM[u]) * rinv[u];
                    }
                    // a slot that is empty for all four rows (the usual case under the balanced plan, whose
                    // rows of one pass belong to one sequence) is not fetched at all; warp-uniform branch
                    if (wk[0] == 0.f && wk[1] == 0.f && wk[2] == 0.f && wk[3] == 0.f) continue;
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
#pragma unroll
                        for (int c = 0; c < L::kMaxChunks; ++c)
                            if (c < n_chunks)
                                x[u][c] = *reinterpret_cast<const float4*>(src[u] + (int64_t)k * rows_per_seq * p.r_kv +
                                                                           c * L::kChunkK);
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const bool use = wk[u] != 0.f;
#pragma unroll
                        for (int c = 0; c < L::kMaxChunks; ++c)
                            if (c < n_chunks) {
                                acc[u][c].x = fmaf(wk[u], use ? x[u][c].x : 0.f, acc[u][c].x);
                                acc[u][c].y = fmaf(wk[u], use ? x[u][c].y : 0.f, acc[u][c].y);
                                acc[u][c].z = fmaf(wk[u], use ? x[u][c].z : 0.f, acc[u][c].z);
                                acc[u][c].w = fmaf(wk[u], use ? x[u][c].w : 0.f, acc[u][c].w);
                            }
                    }
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int tr = q * 16 + r0 + u;
#pragma unroll
                    for (int c = 0; c < L::kMaxChunks; ++c)
                        if (c < n_chunks) {
                            uint2 v;
                            v.x = pack_bf16(acc[u][c].x, acc[u][c].y);
                            v.y = pack_bf16(acc[u][c].z, acc[u][c].w);
                            *reinterpret_cast<uint2*>(a_lane + c * L::kABytes + tr * 128 + ((chunk16 ^ (tr & 7)) << 4) +
                                                      half * 8) = v;
                        }
                }
            }
            fence_proxy_async_smem();  // generic-proxy writes of A -> visible to the tensor core
            __syncwarp();
            if (lane == 0) mbar_arrive(a_ready);
        }
        // epilogue: TMEM lane = tile row
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait(acc_full, 0, ab, 5));
        tc_fence_after();
        const int tr = q * 16 + (lane & 15);
        int64_t pr = 0, orow = 0;
        const bool valid = lane < 16 && row_of(tr, &pr, &orow);  // lanes 16-31 of a quadrant hold no row
        __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(p.out) + orow * 128;
        if (ok) {
#pragma unroll 1
            for (int c0 = 0; c0 < 128; c0 += 32) {
                uint32_t v[32];
                tmem_ld32(tmem_addr(tmem_base, q * 32, c0), v);
                tmem_wait_ld();
                if (valid) {
                    uint4* d4 = reinterpret_cast<uint4*>(dst + c0);
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        uint4 o;
                        o.x = pack_bf16(__uint_as_float(v[8 * t + 0]), __uint_as_float(v[8 * t + 1]));
                        o.y = pack_bf16(__uint_as_float(v[8 * t + 2]), __uint_as_float(v[8 * t + 3]));
                        o.z = pack_bf16(__uint_as_float(v[8 * t + 4]), __uint_as_float(v[8 * t + 5]));
                        o.w = pack_bf16(__uint_as_float(v[8 * t + 6]), __uint_as_float(v[8 * t + 7]));
                        d4[t] = o;
                    }
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, 128);
}

}  // namespace tc
}  // namespace gqla
