// tcgen05 GEMM kernels for the three plain contractions of the path:
//   expand_cache :  K_C / V [n, j, :] = sum_r c[n, r] W[j][r][:]          (Sec. 3.1)
//   absorb_q     :  q_hat[row, r]     = sum_d q_c[row, d] W_UK[j][r][d]   (Eq. (mqa), line 2)
//   up_proj      :  o[row, d]         = sum_r o_hat[row, r] W_UV[j][r][d] (Eq. (mqa), line 6)
// One CTA computes a 128 x BN output tile: warp 0 streams A/B tiles with TMA through a ring of
// shared-memory stages, warp 1 issues tcgen05.mma into a TMEM accumulator, warps 2-5 read the
// accumulator back (tcgen05.ld), stage their bf16 rows in the idle stage ring and ship each row as one bulk store.
#pragma once
#include "tc_common.cuh"

namespace gqla {
namespace tc {

enum GemmMode { kGemmExpand = 0, kGemmAbsorbQ = 1, kGemmUpProj = 2 };

struct GemmParams {
    int32_t k_blocks;   // K / 64
    int64_t m_total;    // expand: cache rows N;  others: B * s_q (query positions)
    int32_t h_q, g, hpg, d_h, r_kv, d_r;
    int32_t hpb;        // heads per group padded to a power of two: a tile is BM/hpb positions x hpb head slots
    void* out0;         // expand: k_c;  absorb_q: q_hat;  up_proj: o
    void* out1;         // expand: v
    const void* aux_in; // absorb_q: q_r (copied into q_hat's tail);  expand: cache (for the k_R copy)
    void* aux_out;      // expand: k_r plane or null
    int64_t aux_stride; // expand: cache row stride (elements)
    int32_t* status;
};

template <int BN, bool B_MN, int BM = 128>
struct GemmSmem {
    static constexpr int kABytes = BM * 128;   // BM rows x 64 bf16
    static constexpr int kStages = 196608 / (kABytes + BN * 128);  // 192 KB of tiles in flight: 4, 6 or 8 stages
    static constexpr int kBBytes = BN * 128;   // K-major: BN rows x 64 k;  MN-major: (BN/64) boxes of 64 k-rows x 64 n
    static constexpr int kStageBytes = kABytes + kBBytes;
    static constexpr int kOutPitch = BN * 2 + 16;  // output staging of the epilogue (reuses the stage ring)
    static_assert(BM * kOutPitch <= kStages * kStageBytes, "output staging must fit in the stage ring");
    static_assert(BM == 64 || BM == 128, "an MMA tile has 64 or 128 rows");
    static_assert(2 * kStages + 1 <= 24, "barriers must fit in the 256 bytes behind the tiles");
    static constexpr int kTotal = kStages * kStageBytes + 1024 /*align slack*/ + 256 /*barriers*/;
    static_assert(OneCtaPerSM<kTotal>::value, "");
};

template <int MODE, int BN, bool B_MN, int BM = 128>
__global__ void __launch_bounds__(192, 1)
gemm_tc_kernel(const GemmParams p, const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
               const __grid_constant__ CUtensorMap tmB1) {
    using L = GemmSmem<BN, B_MN, BM>;
    static_assert(BM == 128 || MODE != kGemmExpand, "the expansion uses 128-row tiles");
    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + L::kStages * L::kStageBytes);
    uint64_t* full = bars;
    uint64_t* empty = bars + L::kStages;
    uint64_t* acc_full = bars + 2 * L::kStages;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * L::kStages + 1);
    volatile int32_t* abort_flag = reinterpret_cast<volatile int32_t*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const Abort ab{abort_flag, p.status};
    pdl_launch_dependents();

    // tile coordinates
    // expand: linear grid, (plane, group) fastest so that the CTAs sharing a tile of cache rows run together
    // (expand: a CTA covers BN / d_h adjacent groups of one plane; grp counts in units of that many groups)
    constexpr int kGroupsPerCta = (MODE == kGemmExpand) ? BN / 128 : 1;
    const int grp_slots = (MODE == kGemmExpand) ? 2 * p.g / kGroupsPerCta : 1;
    const int m_tile = (MODE == kGemmExpand) ? (int)(blockIdx.x / grp_slots) : (int)blockIdx.x;
    const int grp = (MODE == kGemmExpand) ? (int)(blockIdx.x % grp_slots) * kGroupsPerCta
                                          : (int)blockIdx.y;  // plane * g + first group j, or j
    const int n_tile = (MODE == kGemmExpand) ? 0 : (int)blockIdx.z;

    if (threadIdx.x == 0) {
        for (int s = 0; s < L::kStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], 1);
        }
        mbar_init(acc_full, 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, BN);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const CUtensorMap* tmB = (MODE == kGemmExpand && grp >= p.g) ? &tmB1 : &tmB0;
    const int j = (MODE == kGemmExpand) ? grp % p.g : grp;

    // The projection weights are constants of the model, never outputs of the previous kernel of the stream: their
    // tiles for the first ring stages are requested BEFORE the wait on that kernel and travel while it drains.
    // (The activations, which it may have written, are requested after the wait.)
    const int n_pre = (MODE == kGemmExpand) ? 0 : (p.k_blocks < L::kStages ? p.k_blocks : L::kStages);
    auto load_b = [&](int kb, int s) {
        uint8_t* b_dst = tiles + s * L::kStageBytes + L::kABytes;
        if (B_MN && MODE == kGemmExpand) {
            // rows = j * K + k, columns = d; one 64x64 box per 64 output columns, two per group
#pragma unroll
            for (int nb = 0; nb < BN / 64; ++nb)
                tma_load_2d(b_dst + nb * 8192, tmB, (nb & 1) * 64, (j + (nb >> 1)) * p.k_blocks * 64 + kb * 64, &full[s]);
        } else if (B_MN) {
            // rows = j * K + k, columns = output feature; one 64x64 box per 64 output columns
#pragma unroll
            for (int nb = 0; nb < BN / 64; ++nb)
                tma_load_2d(b_dst + nb * 8192, tmB, n_tile * BN + nb * 64, j * p.k_blocks * 64 + kb * 64, &full[s]);
        } else {
            // rows = j * r_kv + output feature, columns = k
            tma_load_2d(b_dst, tmB, kb * 64, j * p.r_kv + n_tile * BN, &full[s]);
        }
    };
    if (warp == 0 && n_pre > 0) {
        if (elect_one()) {
            tma_prefetch_desc(tmB);
            for (int kb = 0; kb < n_pre; ++kb) {  // the ring is empty: no wait needed for its first round
                mbar_expect_tx(&full[kb], L::kStageBytes);
                load_b(kb, kb);
            }
        }
        __syncwarp();
    }
    pdl_wait();  // set-up done; the activations may come from the previous kernel of the stream

    if (warp == 0) {
        if (elect_one()) {
            tma_prefetch_desc(&tmA);
            tma_prefetch_desc(tmB);
            for (int kb = 0; kb < p.k_blocks; ++kb) {
                const int s = kb % L::kStages;
                const uint32_t ph = (kb / L::kStages) & 1;
                if (!mbar_wait(&empty[s], ph ^ 1, ab, 1)) break;
                uint8_t* a_dst = tiles + s * L::kStageBytes;
                if (kb >= n_pre) mbar_expect_tx(&full[s], L::kStageBytes);  // stages [0, n_pre) were armed before the wait
                if (MODE == kGemmExpand) {
                    tma_load_2d(a_dst, &tmA, kb * 64, m_tile * 128, &full[s]);
                } else {
                    // 4-D view (feature, head-in-group, group, query position): 128/hpb positions x hpb head
                    // slots (slots beyond the group's hpg heads read zeros and are not stored)
                    asm volatile(
                        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], "
                        "[%1, {%3, %4, %5, %6}], [%2];" ::"r"(smem_u32(a_dst)),
                        "l"(reinterpret_cast<uint64_t>(&tmA)), "r"(smem_u32(&full[s])), "r"(kb * 64), "r"(0), "r"(j),
                        "r"(m_tile * (BM / p.hpb))
                        : "memory");
                }
                if (kb >= n_pre) load_b(kb, s);
            }
        }
    } else if (warp == 1) {
        if (elect_one()) {
            constexpr uint32_t idesc = idesc_bf16(BM, BN, 0, B_MN ? 1 : 0);
            bool ok = true;
            for (int kb = 0; kb < p.k_blocks && ok; ++kb) {
                const int s = kb % L::kStages;
                const uint32_t ph = (kb / L::kStages) & 1;
                ok = mbar_wait(&full[s], ph, ab, 2);
                if (!ok) break;
                tc_fence_after();
                const uint32_t a_addr = smem_u32(tiles + s * L::kStageBytes);
                const uint32_t b_addr = a_addr + L::kABytes;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    const uint64_t a_desc = desc_kmajor_sw128(a_addr + ks * 32);
                    const uint64_t b_desc = B_MN ? desc_mnmajor_sw128(b_addr + ks * 2048, 8192)
                                                 : desc_kmajor_sw128(b_addr + ks * 32);
                    umma_ss(tmem_base, a_desc, b_desc, idesc, (kb | ks) != 0);
                }
                umma_commit(&empty[s]);
            }
            if (ok) umma_commit(acc_full);
        }
    } else {
        // epilogue: warp w may touch TMEM lanes [32 * (w % 4), +32)
        const int q = warp & 3;
        // row of the tile: the TMEM lane for 128-row tiles; a 64-row accumulator sits in lanes 0-15 of each quadrant
        const int row = BM == 128 ? q * 32 + lane : q * 16 + (lane & 15);
        const bool has_row = BM == 128 || lane < 16;
        // (output addresses and the side copies first: they overlap the main loop instead of following it)
        __nv_bfloat16* dst = nullptr;
        if (MODE == kGemmExpand) {
            const int64_t n = (int64_t)m_tile * 128 + row;
            if (n < p.m_total) {
                __nv_bfloat16* plane = reinterpret_cast<__nv_bfloat16*>(grp >= p.g ? p.out1 : p.out0);
                dst = plane + n * ((int64_t)p.g * p.d_h) + (int64_t)j * p.d_h + n_tile * BN;
                if (grp == 0 && n_tile == 0 && p.aux_out != nullptr) {
                    const uint4* src = reinterpret_cast<const uint4*>(
                        reinterpret_cast<const __nv_bfloat16*>(p.aux_in) + n * p.aux_stride + p.r_kv);
                    uint4* kr = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.aux_out) + n * p.d_r);
                    for (int c = 0; c < p.d_r / 8; ++c) kr[c] = src[c];
                }
            }
        } else {
            const int64_t bp = (int64_t)m_tile * (BM / p.hpb) + row / p.hpb;
            const int il = row % p.hpb;
            const int i = j * p.hpg + il;
            if (has_row && bp < p.m_total && il < p.hpg) {
                const int64_t r = bp * p.h_q + i;
                if (MODE == kGemmAbsorbQ) {
                    __nv_bfloat16* orow = reinterpret_cast<__nv_bfloat16*>(p.out0) + r * (p.r_kv + p.d_r);
                    dst = orow + n_tile * BN;
                    if (n_tile == 0) {
                        const uint4* src =
                            reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.aux_in) + r * p.d_r);
                        uint4* tail = reinterpret_cast<uint4*>(orow + p.r_kv);
                        for (int c = 0; c < p.d_r / 8; ++c) tail[c] = src[c];
                    }
                } else {
                    dst = reinterpret_cast<__nv_bfloat16*>(p.out0) + r * p.d_h + n_tile * BN;
                }
            }
        }
        const bool ok = mbar_wait(acc_full, 0, ab, 3);
        tc_fence_after();
        if (ok) {
            // The thread's output row leaves through shared memory as ONE bulk store (BN * 2 contiguous bytes): 16-byte
            // stores of 32 threads to 32 different rows made the epilogue the longest part of these kernels.  The
            // stage ring is idle here (the accumulator is complete, so every load has landed and been multiplied);
            // the padded pitch keeps the 16-byte stores of a quarter warp on distinct banks.  A thread stages and
            // ships only its own row, so no barrier is needed in between.
            uint8_t* srow = tiles + row * L::kOutPitch;
#pragma unroll 1
            for (int c0 = 0; c0 < BN; c0 += 64) {  // two loads in flight per wait
                uint32_t v[64];
                tmem_ld32(tmem_addr(tmem_base, q * 32, c0), v);
                tmem_ld32(tmem_addr(tmem_base, q * 32, c0 + 32), v + 32);
                tmem_wait_ld();
                uint4* d4 = reinterpret_cast<uint4*>(srow + c0 * 2);
                if (has_row)  // (lanes 16-31 of a 64-row accumulator hold nothing)
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    uint4 o;
                    o.x = pack_bf16(__uint_as_float(v[8 * t + 0]), __uint_as_float(v[8 * t + 1]));
                    o.y = pack_bf16(__uint_as_float(v[8 * t + 2]), __uint_as_float(v[8 * t + 3]));
                    o.z = pack_bf16(__uint_as_float(v[8 * t + 4]), __uint_as_float(v[8 * t + 5]));
                    o.w = pack_bf16(__uint_as_float(v[8 * t + 6]), __uint_as_float(v[8 * t + 7]));
                    d4[t] = o;
                }
            }
            fence_proxy_async_smem();  // staged row -> visible to the bulk-copy engine
            if (dst != nullptr) {
                bulk_store(dst, srow, BN * 2);
                bulk_commit();
                bulk_wait_read();  // shared memory must outlive the copy's reads
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) tmem_dealloc(tmem_base, BN);
}

// ----------------------------------------------------------------------------- host launchers

template <int MODE, int BN, bool B_MN, int BM = 128>
inline cudaError_t gemm_launch(const GemmParams& p, const CUtensorMap& a, const CUtensorMap& b0, const CUtensorMap& b1,
                               dim3 grid, cudaStream_t st) {
    using L = GemmSmem<BN, B_MN, BM>;
    auto kern = gemm_tc_kernel<MODE, BN, B_MN, BM>;
    static bool attr_set[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev < 0 || dev >= 64 || !attr_set[dev]) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, L::kTotal);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) attr_set[dev] = true;
    }
    return launch_pdl(kern, grid, dim3(192), L::kTotal, st, p, a, b0, b1);
}

}  // namespace tc
}  // namespace gqla
