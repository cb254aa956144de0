// Expansion of the rows a decode step appends (Sec. 3.1: k^C = W^UK c^KV, v^C = W^UV c^KV per group, a
// per-token map) on tcgen05.  One CTA = 64 new rows x one (plane, group): four builder warps gather the
// latent rows (one per (sequence, new token); they are not contiguous in the cache) into the
// 128-byte-swizzled K-major A operand, warp 0 fetches W[j] with TMA as an MN-major B operand, warp 1 issues
// M = 64 MMAs into a TMEM accumulator (row m in TMEM lane (m % 16) + 32 (m / 16)), and the builder warps
// store the 64 x 128 bf16 tile to the rows' places in the plane.  Both operands are resident in full
// (r_kv <= 512), so every load of the CTA is in flight at once.
#pragma once
#include "tc_common.cuh"

namespace gqla {
namespace tc {

struct AppendParams {
    int32_t B, s_q, g, r_kv, d_r;
    const __nv_bfloat16* cache;  // [N, >= r_kv + d_r]
    int64_t cache_stride;
    const int64_t* seq_start;
    const int32_t* seqlens;
    __nv_bfloat16* k_c;          // [N, g, 128]
    __nv_bfloat16* v;            // [N, g, 128]
    __nv_bfloat16* k_r;          // [N, d_r] or null
    int32_t* status;
};

struct AppendSmem {
    static constexpr int kChunkK = 128;
    static constexpr int kRows = 64;
    static constexpr int kABytes = 2 * 8192;  // 64 rows x 128 k, two 64-wide k-blocks
    static constexpr int kBBytes = 4 * 8192;  // 128 k x 128 n: (k-block, n-block) boxes of 64 x 64
    static constexpr int kMaxChunks = 4;
    static constexpr int kTileBytes = kMaxChunks * (kABytes + kBBytes);
    static constexpr int kNumBars = 3;  // a_ready b_full acc_full
    static constexpr int kThreads = 192;
    static constexpr int kTotal = 1024 + kTileBytes + kNumBars * 8 + 16 + kRows * 8;
    static_assert(OneCtaPerSM<kTotal>::value, "");
};

__global__ void __launch_bounds__(AppendSmem::kThreads, 1)
append_expand_tc_kernel(const AppendParams p, const __grid_constant__ CUtensorMap tmK,
                        const __grid_constant__ CUtensorMap tmV) {
    using L = AppendSmem;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint8_t* a_smem = tiles;
    uint8_t* b_smem = tiles + L::kMaxChunks * L::kABytes;
    uint64_t* bars = reinterpret_cast<uint64_t*>(tiles + L::kTileBytes);
    uint64_t* a_ready = bars;  // the four builder warps have written A
    uint64_t* b_full = bars + 1;
    uint64_t* acc_full = bars + 2;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + L::kNumBars);
    volatile int32_t* abort_flag = reinterpret_cast<volatile int32_t*>(tmem_slot + 1);
    int64_t* sm_row = reinterpret_cast<int64_t*>(tmem_slot + 4);  // [64] cache row of every tile row, -1: none

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const Abort ab{abort_flag, p.status};
    const int m_tile = blockIdx.x;
    const int plane = blockIdx.y / p.g, j = blockIdx.y % p.g;
    const CUtensorMap* tmB = plane == 0 ? &tmK : &tmV;
    const int n_chunks = p.r_kv / L::kChunkK;
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
    pdl_wait();  // set-up done; lengths and latent rows may come from the previous kernel of the stream
    if (threadIdx.x < L::kRows) {
        const int64_t u = (int64_t)m_tile * L::kRows + threadIdx.x;  // (sequence, new token) unit
        int64_t n = -1;
        if (u < (int64_t)p.B * p.s_q) {
            const int32_t b = (int32_t)(u / p.s_q), pq = (int32_t)(u % p.s_q);
            const int32_t pos = p.seqlens[b] - p.s_q + pq;
            if (pos >= 0) n = p.seq_start[b] + pos;
        }
        sm_row[threadIdx.x] = n;
    }
    __syncthreads();

    if (warp == 0) {
        // ------------------------------------------------------------------ W[j] chunks (MN-major B operand)
        if (elect_one()) {
            tma_prefetch_desc(tmB);
            mbar_expect_tx(b_full, n_chunks * L::kBBytes);
            for (int c = 0; c < n_chunks; ++c)
                for (int kb = 0; kb < 2; ++kb)
                    for (int nb = 0; nb < 2; ++nb)
                        tma_load_2d(b_smem + c * L::kBBytes + (kb * 2 + nb) * 8192, tmB, nb * 64,
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
        const int n16 = p.r_kv / 8;  // 16-byte pieces of a latent row
        // a row is n16 pieces; lane l copies pieces l and l + 32: piece cc is k-block cc / 8, 16-byte column
        // cc % 8 of that block's 128-byte row, XORed with the row's low three bits (the 128-byte swizzle)
        // every load of the warp's 16 rows is issued before the first is used (the rows are cold in L2)
        uint4 x[16][2], kr[16];
#pragma unroll
        for (int r = 0; r < 16; ++r) {
            const int64_t n = sm_row[q * 16 + r];
            const uint4* src = reinterpret_cast<const uint4*>(p.cache + (n >= 0 ? n : 0) * p.cache_stride);
#pragma unroll
            for (int h = 0; h < 2; ++h)
                x[r][h] = (n >= 0 && lane + 32 * h < n16) ? __ldg(src + lane + 32 * h) : make_uint4(0u, 0u, 0u, 0u);
            // the shared RoPE key travels unchanged (one (plane, group) slice does it)
            kr[r] = (p.k_r != nullptr && blockIdx.y == 0 && n >= 0 && lane < p.d_r / 8) ? __ldg(src + n16 + lane)
                                                                                     : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int r = 0; r < 16; ++r) {
            const int tr = q * 16 + r;
            const int64_t n = sm_row[tr];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const int cc = lane + 32 * h;
                if (cc < n16)
                    *reinterpret_cast<uint4*>(a_smem + (cc >> 3) * 8192 + tr * 128 + (((cc & 7) ^ (tr & 7)) << 4)) = x[r][h];
            }
            if (p.k_r != nullptr && blockIdx.y == 0 && n >= 0 && lane < p.d_r / 8)
                reinterpret_cast<uint4*>(p.k_r + n * p.d_r)[lane] = kr[r];
        }
        fence_proxy_async_smem();  // generic-proxy writes of A -> visible to the tensor core
        __syncwarp();
        if (lane == 0) mbar_arrive(a_ready);
        // epilogue: TMEM lane = tile row
        const bool ok = __all_sync(0xffffffffu, mbar_wait(acc_full, 0, ab, 5));
        tc_fence_after();
        const int tr = q * 16 + (lane & 15);
        const int64_t n = sm_row[tr];
        const bool valid = lane < 16 && n >= 0;  // lanes 16-31 of a quadrant hold no row
        __nv_bfloat16* dst = (plane == 0 ? p.k_c : p.v) + ((n >= 0 ? n : 0) * p.g + j) * 128;
        if (ok) {
#pragma unroll 1
            for (int c0 = 0; c0 < 128; c0 += 32) {
                uint32_t x[32];
                tmem_ld32(tmem_addr(tmem_base, q * 32, c0), x);
                tmem_wait_ld();
                if (valid) {
                    uint4* d4 = reinterpret_cast<uint4*>(dst + c0);
#pragma unroll
                    for (int t = 0; t < 4; ++t) {
                        uint4 o;
                        o.x = pack_bf16(__uint_as_float(x[8 * t + 0]), __uint_as_float(x[8 * t + 1]));
                        o.y = pack_bf16(__uint_as_float(x[8 * t + 2]), __uint_as_float(x[8 * t + 3]));
                        o.z = pack_bf16(__uint_as_float(x[8 * t + 4]), __uint_as_float(x[8 * t + 5]));
                        o.w = pack_bf16(__uint_as_float(x[8 * t + 6]), __uint_as_float(x[8 * t + 7]));
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
