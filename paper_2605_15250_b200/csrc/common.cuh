// Shared device/host helpers for the GQLA kernels (integer bookkeeping, type loads).
#pragma once
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace gqla {

constexpr int kSplitGranule = 64;

// Split-KV partition: chunk = ceil(ceil(T/S)/64)*64 rows per split.
__host__ __device__ inline void split_range(int32_t T, int32_t S, int32_t k, int32_t* begin, int32_t* end) {
    int64_t per = ((int64_t)T + S - 1) / S;
    int64_t chunk = ((per + kSplitGranule - 1) / kSplitGranule) * kSplitGranule;
    int64_t b = (int64_t)k * chunk, e = (int64_t)(k + 1) * chunk;
    *begin = (int32_t)(b < T ? b : T);
    *end = (int32_t)(e < T ? e : T);
}

// Rows visible to query p of an s_q-token step (causal sum over s = 1..t, Eqs. (mha)/(mqa)).
__host__ __device__ inline int32_t visible_limit(int32_t T, int32_t s_q, int32_t p) {
    int32_t lim = T - (s_q - 1 - p);
    return lim > 0 ? lim : 0;
}

// Where the cache rows of a sequence live.  Packed: row t of sequence b is seq_start[b] + t.  Paged: the
// cache is cut into pages of page_size rows and block_table[b * max_pages + t / page_size] names the page of
// row t (paging is not in the paper; it only changes where a row is fetched from).
struct RowMap {
    const int64_t* seq_start;    // packed layout (null when paged)
    const int32_t* block_table;  // paged layout (null when packed)
    int32_t max_pages, page_size;
    __host__ __device__ bool paged() const { return block_table != nullptr; }
    __device__ __forceinline__ int64_t row(int32_t b, int32_t t) const {
        if (block_table == nullptr) return seq_start[b] + t;
        return (int64_t)block_table[(int64_t)b * max_pages + t / page_size] * page_size + t % page_size;
    }
};

// FP8 E4M3 storage (4 exponent bits, bias 7; 3 mantissa bits; no infinity; largest finite value 448).
struct e4m3 {
    uint8_t code;
};
// One code -> fp32 (exact: every E4M3 value is an fp16 value).
__device__ __forceinline__ float e4m3_to_float(uint8_t code) {
    uint32_t h2;
    asm("{\n\t.reg .b16 c;\n\tcvt.u16.u32 c, %1;\n\tcvt.rn.f16x2.e4m3x2 %0, c;\n\t}" : "=r"(h2) : "r"((uint32_t)code));
    return __half2float(__ushort_as_half((unsigned short)(h2 & 0xffffu)));
}
// Two fp32 -> two codes (low byte = lo): round to nearest even, magnitudes beyond 448 saturate, NaN -> 0x7F.
__device__ __forceinline__ uint16_t float2_to_e4m3x2(float lo, float hi) {
    uint16_t r;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(r) : "f"(hi), "f"(lo));
    return r;
}
__device__ __forceinline__ float ldf(const e4m3* p) { return e4m3_to_float(p->code); }
__device__ __forceinline__ float ldf(const float* p) { return *p; }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void stf(float* p, float v) { *p = v; }
__device__ __forceinline__ void stf(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

}  // namespace gqla
