// gqla_decode_gqa_noalloc: the GQA-path decode step for callers that have no device memory to
// spare for split partials and no way to get any.
//
// Who that is.  The split-KV decode needs room for one partial output and one partial
// log-sum-exp per (sequence, split, query, head) between the attention kernel and the merge.
// gqla_decode_gqa leaves that room to the caller.  Some callers cannot provide it:
//   * a serving process whose memory manager took the whole GPU for weights and KV-cache blocks at
//     start-up, so that a later cudaMalloc fails or evicts somebody else's pages;
//   * a decode loop that must not stall: cudaMalloc and cudaFree synchronise the whole device, so
//     calling them between steps serialises every stream the process runs;
//   * a plain-C or other-language host that links this library without any allocator layer of its
//     own (no torch, no pool) and only holds the buffers it was handed.
// For them the partials live in a fixed array that is part of this library's device image.
//
// What that costs.  Every GPU on which the library's kernels get loaded carries the array
// (kScratchFloats floats, a little over 16 MiB) until the process exits, used or not.  There is one array
// per GPU and every call on that GPU writes into it, so two calls whose kernels may overlap on the
// device (different streams, no ordering between them) corrupt each other: keep such calls on one
// stream or order them with events.  The array keeps whatever the previous call left there; this
// is harmless because the attention kernel rewrites every partial of the current call, empty
// splits included, before the merge reads it -- nothing in it has to start at zero.
//
// When the array comes into being.  The CUDA runtime loads a module lazily: the array is reserved on a
// GPU when this file's device code is first needed there, which is the first call of the entry point on
// that GPU (the address query below, also for a call with B = 0).  A host whose memory manager is going
// to claim the whole GPU must therefore make one call per device -- B = 0 is enough, it launches nothing
// -- at start-up, BEFORE it claims the memory; later calls allocate nothing.
#include <cuda_runtime.h>
#include <math.h>

#include <mutex>

#include "../../include/gqla.h"
#include "common.cuh"

namespace {

// Capacity: partial outputs first, partial log-sum-exps behind them.
constexpr int64_t kMaxPartialFloats = 4ll << 20;  // rows * d_h      <= 4 Mi floats (16 MiB)
constexpr int64_t kMaxPartialRows = 64ll << 10;   // B*S*s_q*h_q     <= 64 Ki rows  (256 KiB)
constexpr int64_t kScratchFloats = kMaxPartialFloats + kMaxPartialRows;  // 16 MiB + 256 KiB of floats

// In host code this name is only a handle for the runtime's symbol table.  It is NOT a device
// address: handing `g_split_scratch` itself to a kernel launch would give the kernel a host pointer.
// Host code must translate it with cudaGetSymbolAddress (below); device code may name it directly.
static __device__ __align__(256) float g_split_scratch[kScratchFloats];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
float* g_scratch_on_device[kMaxDevices] = {};  // device address of the array, per device ordinal

// Returns the device address of the array on the CURRENT device, asking the runtime the first
// time this device is seen.  nullptr on failure.
float* scratch_for_current_device() {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (g_scratch_on_device[dev] == nullptr) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_split_scratch) != cudaSuccess || p == nullptr) {
            (void)cudaGetLastError();
            return nullptr;
        }
        g_scratch_on_device[dev] = static_cast<float*>(p);
    }
    return g_scratch_on_device[dev];
}

// Merge of the split partials held in the array (named directly: this is device code).
// One block per (sequence, query, head) row; thread d owns output columns d, d + 128, ...
//   M = max_k lse_k,  w_k = exp(lse_k - M),  out = sum_k w_k o_k / sum_k w_k,  lse = M + ln sum_k w_k.
template <typename T>
__global__ void __launch_bounds__(128)
merge_from_scratch_kernel(int32_t rows_per_seq, int32_t S, int32_t d_out, T* __restrict__ out, float* __restrict__ lse) {
    const float* o_part = g_split_scratch;
    const float* lse_part = g_split_scratch + kMaxPartialFloats;
    const int64_t r = blockIdx.x;
    const int64_t b = r / rows_per_seq;
    const int rr = (int)(r % rows_per_seq);
    const float* lp = lse_part + b * S * rows_per_seq + rr;
    float m = -INFINITY;
    for (int k = 0; k < S; ++k) m = fmaxf(m, lp[(int64_t)k * rows_per_seq]);
    const bool dead = !(m > -INFINITY);
    float den = 0.f;
    for (int k = 0; k < S; ++k) den += dead ? 0.f : expf(lp[(int64_t)k * rows_per_seq] - m);
    const float inv = den > 0.f ? 1.f / den : 0.f;
    const float* op = o_part + (b * S * rows_per_seq + rr) * d_out;
    for (int d = threadIdx.x; d < d_out; d += blockDim.x) {
        float acc = 0.f;
        for (int k = 0; k < S; ++k) {
            const float wk = dead ? 0.f : expf(lp[(int64_t)k * rows_per_seq] - m);
            if (wk != 0.f) acc = fmaf(wk, op[(int64_t)k * rows_per_seq * d_out + d], acc);
        }
        gqla::stf(out + r * d_out + d, acc * inv);
    }
    if (lse != nullptr && threadIdx.x == 0) lse[r] = dead ? -INFINITY : m + logf(den);
}

}  // namespace

extern "C" gqla_status gqla_decode_gqa_noalloc(const gqla_dims* dims, gqla_dtype dtype, int32_t B, int32_t s_q,
                                               float scale, int32_t num_splits, const void* q, const void* k_c,
                                               const void* v, const void* k_r, int64_t k_r_row_stride,
                                               int64_t n_rows, const int64_t* seq_start, const int32_t* seqlens,
                                               void* out, float* lse, int32_t* status_word, void* stream) {
    if (dims == nullptr || out == nullptr) return GQLA_ERR_NULL;
    if (dtype != GQLA_BF16 && dtype != GQLA_F32) return GQLA_ERR_DTYPE;
    if (dims->h_q <= 0 || dims->d_h <= 0 || B < 0 || s_q < 1 || num_splits < 1) return GQLA_ERR_SHAPE;
    if ((reinterpret_cast<uintptr_t>(out) & 15u) != 0) return GQLA_ERR_ALIGN;
    // Capacity check before anything touches the device: the partials of this call must fit the array.
    const int64_t rows = (int64_t)B * num_splits * s_q * dims->h_q;
    if (rows > kMaxPartialRows || rows * dims->d_h > kMaxPartialFloats) return GQLA_ERR_CAPACITY;
    // The address query comes before the B == 0 return on purpose: an empty call is the documented way to
    // make the runtime load this module (and reserve the array) on the current device at start-up.
    float* scratch = scratch_for_current_device();
    if (scratch == nullptr) return GQLA_ERR_CUDA;
    if (B == 0) return GQLA_OK;
    float* o_part = scratch;
    float* lse_part = scratch + kMaxPartialFloats;
    // The attention kernel is the library's ordinary one; it gets the translated device address.
    gqla_status s = gqla_decode_gqa(dims, dtype, B, s_q, scale, num_splits, q, k_c, v, k_r, k_r_row_stride, n_rows,
                                    seq_start, seqlens, o_part, lse_part, status_word, stream);
    if (s != GQLA_OK) return s;
    const int32_t rows_per_seq = s_q * dims->h_q;
    const unsigned blocks = (unsigned)((int64_t)B * rows_per_seq);
    cudaStream_t st = (cudaStream_t)stream;
    if (dtype == GQLA_BF16)
        merge_from_scratch_kernel<__nv_bfloat16>
            <<<blocks, 128, 0, st>>>(rows_per_seq, num_splits, dims->d_h, (__nv_bfloat16*)out, lse);
    else
        merge_from_scratch_kernel<float><<<blocks, 128, 0, st>>>(rows_per_seq, num_splits, dims->d_h, (float*)out, lse);
    return cudaGetLastError() == cudaSuccess ? GQLA_OK : GQLA_ERR_CUDA;
}
