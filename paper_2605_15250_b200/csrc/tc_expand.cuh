// One-shot cache expansion on CTA pairs (Sec. 3.1: k^C = W^UK c, v^C = W^UV c per group):
//   [K_C | V][n, :] = c[n, 0:r_kv] . [W^UK ; W^UV]      a plain GEMM  N x r_kv x (2 g d_h).
// A pair owns 256 cache rows (128 per CTA).  Its latent rows are loaded ONCE and stay in shared memory
// while the pair walks all 2 g d_h / 256 column tiles; the weights stream through a ring, each CTA
// fetching half of every B tile (cta_group::2 MMAs of 256 x 256 x 16 read B from both CTAs), so the
// weights cross L2 -> SM once per 256 rows instead of once per 128.  Two 256-column accumulators in
// TMEM: the epilogue warps store tile t while the MMAs of tile t + 1 run.  The output leaves through a
// swizzled shared-memory staging box and TMA stores (64 columns x 128 rows at a time): one thread per row
// writing its row straight to global memory costs more store instructions than the MMAs give it time for.
// Warp roles per CTA: warp 0 TMA producer, warp 1 TMEM owner (+ MMA issuer in the leader), warps 2-5
// epilogue (TMEM lane = row).
#pragma once
#include "tc_common.cuh"


namespace gqla {
namespace tc {

struct ExpandParams {
    int64_t n_rows;          // cache rows N
    int32_t g, r_kv, d_r;    // d_h = 128
    void* k_c;               // [N, g, 128]
    void* v;                 // [N, g, 128]
    const void* cache;       // for the k_R copy
    void* k_r;               // [N, d_r] or null
    int64_t cache_stride;    // elements
    int32_t* status;
};

struct ExpandSmem {
    static constexpr int kKBlocks = 8;                   // r_kv = 512
    static constexpr int kABytes = kKBlocks * 16384;     // 128 rows x 512, eight 64-wide k-blocks
    static constexpr int kBStage = 2 * 8192;             // 64 k x 128 n: this CTA's half of a 256-column tile
    // ring of B stages: measured on the C2 cache, 4 stages 0.498 ms, 5 stages 0.464 ms (the weights come out of
    // L2 and every k-block is only 512 cycles of tensor work)
    static constexpr int kStages = 5;
    static constexpr int kOutBytes = 16384;              // output staging box: 128 rows x 64 bf16, 128-byte swizzle
    static constexpr int kTileBytes = kABytes + kStages * kBStage + kOutBytes;  // one staging box (a second one measured slower: 0.524 vs 0.498 ms)
    static constexpr int kNumBars = 1 + 2 * kStages + 4;  // a_full, b_full[], b_empty[], acc_full[2], acc_empty[2]
    static constexpr int kThreads = 192;
    static constexpr int kTotal = 1024 + kTileBytes + kNumBars * 8 + 16;
    static_assert(kTotal <= 232448, "shared memory budget of one CTA");
    static_assert(OneCtaPerSM<kTotal>::value, "");
};

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(ExpandSmem::kThreads, 1)
expand_tc_kernel(const ExpandParams p, const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmK,
                 const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmOK,
                 const __grid_constant__ CUtensorMap tmOV) {
    using L = ExpandSmem;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* a_smem = tiles;
    uint8_t* b_smem = tiles + L::kABytes;
    uint8_t* out_smem = b_smem + L::kStages * L::kBStage;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + L::kTileBytes);
    uint64_t* a_full = bars;                       // leader: both CTAs' latent rows have landed
    uint64_t* b_full = bars + 1;                   // [kStages] leader: both halves of a B stage have landed
    uint64_t* b_empty = b_full + L::kStages;       // [kStages] per CTA
    uint64_t* acc_full = b_empty + L::kStages;     // [2] per CTA (multicast commit)
    uint64_t* acc_empty = acc_full + 2;            // [2] leader: the epilogue warps of both CTAs have read the tile
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + L::kNumBars);
    volatile int32_t* abort_flag = reinterpret_cast<volatile int32_t*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta = cluster_ctarank();
    const Abort ab{abort_flag, p.status};
    const int pair = blockIdx.x >> 1;
    const int64_t row_base = (int64_t)pair * 256 + cta * 128;  // first cache row of this CTA
    const int n_tiles = 2 * p.g * 128 / 256;                    // column tiles of 256: g of them (K_C first, then V)

    if (threadIdx.x == 0) {
        for (int i = 0; i < L::kNumBars; ++i) mbar_init(&bars[i], (&bars[i] == &acc_empty[0] || &bars[i] == &acc_empty[1]) ? 8 : 1);
        *abort_flag = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc2(tmem_slot, 512);
        tmem_relinquish2();
    }
    pdl_launch_dependents();
    tc_fence_before();
    __syncthreads();
    cluster_sync();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    pdl_wait();

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer (both CTAs)
        if (elect_one()) {
            tma_prefetch_desc(&tmA);
            tma_prefetch_desc(&tmK);
            tma_prefetch_desc(&tmV);
            const uint32_t a_full_l = mapa(smem_u32(a_full), 0);
            if (cta == 0) mbar_expect_tx(a_full, 2 * L::kABytes);
            for (int kb = 0; kb < L::kKBlocks; ++kb)
                tma_load_2d_pair(a_smem + kb * 16384, &tmA, kb * 64, (int32_t)row_base, a_full_l);
            int s = 0;
            uint32_t ph = 1;  // parity that means "stage is free"
            bool ok = true;
            for (int t = 0; t < n_tiles && ok; ++t) {
                // this CTA supplies columns [128 cta, +128) of the tile: one whole group of one plane
                const int jj = (2 * t) % p.g + (int)cta;
                const CUtensorMap* tmB = 2 * t >= p.g ? &tmV : &tmK;
                for (int kb = 0; kb < L::kKBlocks; ++kb) {
                    if (!(ok = mbar_wait(&b_empty[s], ph, ab, 1))) break;
                    if (cta == 0) mbar_expect_tx(&b_full[s], 2 * L::kBStage);
                    const uint32_t bar = mapa(smem_u32(&b_full[s]), 0);
                    uint8_t* dst = b_smem + s * L::kBStage;
                    tma_load_2d_pair(dst, tmB, 0, jj * p.r_kv + kb * 64, bar);
                    tma_load_2d_pair(dst + 8192, tmB, 64, jj * p.r_kv + kb * 64, bar);
                    if (++s == L::kStages) { s = 0; ph ^= 1; }
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer (leader CTA only)
        if (cta == 0 && elect_one()) {
            constexpr uint32_t idesc = idesc_bf16(256, 256, 0, 1);
            const uint32_t a_lo = desc_lo(desc_kmajor_sw128(smem_u32(a_smem)));
            int s = 0;
            uint32_t ph = 0;
            bool ok = mbar_wait(a_full, 0, ab, 2);
            tc_fence_after();
            for (int t = 0; t < n_tiles && ok; ++t) {
                const int buf = t & 1;
                if (!(ok = mbar_wait(&acc_empty[buf], ((t >> 1) & 1) ^ 1, ab, 3))) break;
                tc_fence_after();
                const uint32_t d = tmem_base + (uint32_t)buf * 256;
                for (int kb = 0; kb < L::kKBlocks; ++kb) {
                    if (!(ok = mbar_wait(&b_full[s], ph, ab, 4))) break;
                    tc_fence_after();
                    const uint32_t b_lo = desc_lo(desc_mnmajor_sw128(smem_u32(b_smem + s * L::kBStage), 8192));
                    if (kb == 0)
                        umma_ss2_lo<false>(d, a_lo, b_lo, idesc);
                    else
                        umma_ss2_lo<true>(d, a_lo + ((kb * 16384) >> 4), b_lo, idesc);
#pragma unroll
                    for (int ks = 1; ks < 4; ++ks)
                        umma_ss2_lo<true>(d, a_lo + ((kb * 16384 + ks * 32) >> 4), b_lo + ((ks * 2048) >> 4), idesc);
                    umma_commit2(&b_empty[s], 3);
                    if (++s == L::kStages) { s = 0; ph ^= 1; }
                }
                if (ok) umma_commit2(&acc_full[buf], 3);
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue: TMEM lane = row
        const int q = warp & 3;
        const int64_t n = row_base + q * 32 + lane;
        const bool valid = n < p.n_rows;
        const uint32_t acc_empty_l[2] = {mapa(smem_u32(&acc_empty[0]), 0), mapa(smem_u32(&acc_empty[1]), 0)};
        if (valid && p.k_r != nullptr) {  // k^R is carried over unchanged
            const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(p.cache) +
                                                              n * p.cache_stride + p.r_kv);
            uint4* kr = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(p.k_r) + n * p.d_r);
            for (int c = 0; c < p.d_r / 8; ++c) kr[c] = src[c];
        }
        bool ok = true;
        for (int t = 0; t < n_tiles && ok; ++t) {
            const int buf = t & 1;
            ok = __all_sync(0xffffffffu, mbar_wait(&acc_full[buf], (t >> 1) & 1, ab, 5));
            if (!ok) break;
            tc_fence_after();
            const CUtensorMap* tmO = 2 * t >= p.g ? &tmOV : &tmOK;
            const int col_base = ((2 * t) % p.g) * 128;  // first column of the tile in its plane's [N, g * 128] rows
            const int r = q * 32 + lane;                 // row of this thread within the CTA's 128
#pragma unroll 1
            for (int cb = 0; cb < 4; ++cb) {
                uint32_t v[64];
                tmem_ld32(tmem_addr(tmem_base, q * 32, buf * 256 + cb * 64), v);
                tmem_ld32(tmem_addr(tmem_base, q * 32, buf * 256 + cb * 64 + 32), v + 32);
                tmem_wait_ld();
                // the staging box is rewritten: the store that last read it must have finished reading
                uint8_t* box = out_smem;
                if (threadIdx.x == 64) bulk_wait_read();
                named_bar_sync(1, 128);
#pragma unroll
                for (int c = 0; c < 8; ++c) {  // 8 chunks of 8 bf16; chunk index XORed with (row & 7)
                    uint4 o;
                    o.x = pack_bf16(__uint_as_float(v[8 * c + 0]), __uint_as_float(v[8 * c + 1]));
                    o.y = pack_bf16(__uint_as_float(v[8 * c + 2]), __uint_as_float(v[8 * c + 3]));
                    o.z = pack_bf16(__uint_as_float(v[8 * c + 4]), __uint_as_float(v[8 * c + 5]));
                    o.w = pack_bf16(__uint_as_float(v[8 * c + 6]), __uint_as_float(v[8 * c + 7]));
                    *reinterpret_cast<uint4*>(box + r * 128 + ((c ^ (r & 7)) << 4)) = o;
                }
                fence_proxy_async_smem();
                named_bar_sync(1, 128);
                if (threadIdx.x == 64 && row_base < p.n_rows) {  // a CTA wholly behind the last row stores nothing
                    tma_store_2d(tmO, box, col_base + cb * 64, (int32_t)row_base);
                    bulk_commit();
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(acc_empty_l[buf]);
        }
        if (threadIdx.x == 64) bulk_wait_read();  // the last store still reads the staging box
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();
    if (warp == 1) tmem_dealloc2(tmem_base, 512);
}

}  // namespace tc
}  // namespace gqla
