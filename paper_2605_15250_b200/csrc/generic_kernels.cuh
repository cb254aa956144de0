// Generic SIMT kernels: any (h_q, g, d_h, r_kv, d_r), bf16 or fp32 storage, any s_q.
// They are the correctness floor for shapes the tensor-core kernels do not cover, and an
// on-device cross-check for the ones they do.  fp32 arithmetic throughout.
#pragma once
#include <type_traits>

#include "common.cuh"

namespace gqla {

struct DecodeArgs {
    // score(s) = scale * ( q[0:dA] . kA[s] + q[dA:dA+dB] . kB[s] ),  value(s) = v[s][0:dv]
    const void* q;       // [B, s_q, h_q, dA+dB]
    const void* kA;      // first key part; row stride kA_stride, + group * kA_gstride
    const void* kB;      // second key part (shared by all groups); may be null when dB == 0
    const void* v;       // values; row stride v_stride, + group * v_gstride
    int64_t kA_stride, kA_gstride, kB_stride, v_stride, v_gstride;
    int32_t dA, dB, dv;
    RowMap rows;
    const int32_t* seqlens;
    int32_t B, S, s_q, h_q, hpg;
    float scale;
    float* o_part;    // [B, S, s_q, h_q, dv]
    float* lse_part;  // [B, S, s_q, h_q]
    void* o_final;    // not null (S == 1 only): the output goes here in the storage type, o_part unused, lse_part may be null
    // FP8 cache: scores are multiplied by q_row_scale[(b, p, i)] (null = 1) and outputs by v_scale (0 = 1)
    const float* q_row_scale;
    float v_scale;
};

constexpr int kGenericMaxV = 16;  // value columns per lane: dv <= 512

// One warp per (b, split, p, head) row.  Lanes stride over the feature dimension; the
// online-softmax state (m, l) is warp-uniform; each lane owns dv/32 output columns.
template <typename E>
__global__ void __launch_bounds__(128) decode_generic_kernel(DecodeArgs a) {
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    const int64_t nrows = (int64_t)a.B * a.S * a.s_q * a.h_q;
    if (row >= nrows) return;
    const int i = (int)(row % a.h_q);
    const int p = (int)((row / a.h_q) % a.s_q);
    const int k = (int)((row / ((int64_t)a.h_q * a.s_q)) % a.S);
    const int b = (int)(row / ((int64_t)a.h_q * a.s_q * a.S));
    const int j = i / a.hpg;  // 0-indexed form of j(i) = ceil(i/(h_q/g))

    const int32_t T = a.seqlens[b];
    int32_t begin, end;
    split_range(T, a.S, k, &begin, &end);
    const int32_t lim = visible_limit(T, a.s_q, p);
    if (end > lim) end = lim;

    const E* q = (const E*)a.q + ((int64_t)(b * a.s_q + p) * a.h_q + i) * (a.dA + a.dB);
    const E* kA = (const E*)a.kA + (int64_t)j * a.kA_gstride;
    const E* kB = (const E*)a.kB;
    const E* vv = (const E*)a.v + (int64_t)j * a.v_gstride;

    float acc[kGenericMaxV];
#pragma unroll
    for (int c = 0; c < kGenericMaxV; ++c) acc[c] = 0.f;
    float m = -INFINITY, l = 0.f;
    const float x_scale = a.scale * (a.q_row_scale != nullptr ? a.q_row_scale[(int64_t)(b * a.s_q + p) * a.h_q + i] : 1.f);

    for (int32_t s = begin; s < end; ++s) {
        const int64_t n = a.rows.row(b, s);
        const E* ka = kA + n * a.kA_stride;
        float dot = 0.f;
        for (int d = lane; d < a.dA; d += 32) dot = fmaf(ldf(q + d), ldf(ka + d), dot);
        if (a.dB > 0) {
            const E* kb = kB + n * a.kB_stride;
            for (int d = lane; d < a.dB; d += 32) dot = fmaf(ldf(q + a.dA + d), ldf(kb + d), dot);
        }
        const float x = warp_sum(dot) * x_scale;
        const float m_new = fmaxf(m, x);
        const float corr = expf(m - m_new);  // exp(-inf) = 0 on the first row
        const float e = expf(x - m_new);
        l = l * corr + e;
        const E* vr = vv + n * a.v_stride;
#pragma unroll
        for (int c = 0; c < kGenericMaxV; ++c) {
            const int d = lane + 32 * c;
            if (d < a.dv) acc[c] = fmaf(e, ldf(vr + d), acc[c] * corr);
        }
        m = m_new;
    }

    const float inv = (l > 0.f ? 1.f / l : 0.f) * (a.v_scale != 0.f ? a.v_scale : 1.f);
#pragma unroll
    for (int c = 0; c < kGenericMaxV; ++c) {
        const int d = lane + 32 * c;
        if (d < a.dv) {
            if constexpr (!std::is_same<E, e4m3>::value) {
                if (a.o_final != nullptr) {
                    stf((E*)a.o_final + row * a.dv + d, acc[c] * inv);
                    continue;
                }
            }
            {
                a.o_part[row * a.dv + d] = acc[c] * inv;
            }
        }
    }
    if (lane == 0 && a.lse_part != nullptr) a.lse_part[row] = l > 0.f ? m + logf(l) : -INFINITY;
}

// Log-sum-exp merge: one block per (b, row).  Weights staged in shared memory.
template <typename TO>
__global__ void __launch_bounds__(128) combine_generic_kernel(int32_t B, int32_t rows_per_seq, int32_t S, int32_t d_out,
                                                              const float* __restrict__ o_part,
                                                              const float* __restrict__ lse_part, TO* __restrict__ out,
                                                              float* __restrict__ lse) {
    extern __shared__ float w[];  // [S]
    __shared__ float red[4];
    const int64_t r = blockIdx.x;  // b * rows_per_seq + row
    const int b = (int)(r / rows_per_seq);
    const int rr = (int)(r % rows_per_seq);
    const float* lp = lse_part + ((int64_t)b * S) * rows_per_seq + rr;
    float mx = -INFINITY;
    for (int k = threadIdx.x; k < S; k += blockDim.x) mx = fmaxf(mx, lp[(int64_t)k * rows_per_seq]);
    mx = warp_max(mx);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
    __syncthreads();
    mx = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
    __syncthreads();
    const bool dead = !(mx > -INFINITY);
    float den = 0.f;
    for (int k = threadIdx.x; k < S; k += blockDim.x) {
        const float wk = dead ? 0.f : expf(lp[(int64_t)k * rows_per_seq] - mx);
        w[k] = wk;
        den += wk;
    }
    den = warp_sum(den);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = den;
    __syncthreads();
    den = red[0] + red[1] + red[2] + red[3];
    const float inv = den > 0.f ? 1.f / den : 0.f;
    const float* op = o_part + (((int64_t)b * S) * rows_per_seq + rr) * d_out;
    for (int d = threadIdx.x; d < d_out; d += blockDim.x) {
        float acc = 0.f;
        for (int k = 0; k < S; ++k) {
            const float wk = w[k];
            if (wk != 0.f) acc = fmaf(wk, op[(int64_t)k * rows_per_seq * d_out + d], acc);
        }
        stf(out + r * d_out + d, acc * inv);
    }
    if (lse != nullptr && threadIdx.x == 0) lse[r] = dead ? -INFINITY : mx + logf(den);
}

// Vectorised log-sum-exp merge for d_out % 4 == 0: one thread per (row, four output columns).  Every
// thread of a row recomputes the row's S weights from lse_part (a handful of cached, broadcast loads),
// so there is no cross-thread step and all its 16-byte loads of the partials are independent and in
// flight together; consecutive threads read consecutive float4, i.e. whole rows are streamed.
__device__ __forceinline__ void store4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ void store4(__nv_bfloat16* p, float4 v) {
    __nv_bfloat162 lo = __floats2bfloat162_rn(v.x, v.y), hi = __floats2bfloat162_rn(v.z, v.w);
    uint2 u;
    u.x = *reinterpret_cast<uint32_t*>(&lo);
    u.y = *reinterpret_cast<uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(p) = u;
}
__device__ __forceinline__ float4 ld_stream4(const float* p) {  // read once: do not keep in L1
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0, %1, %2, %3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w)
                 : "l"(p));
    return v;
}
// V = 4, 8 or 16 output columns per thread (as many as d_out allows: the kernel's CTAs wait, resident beside those of
// the decode kernel, for it to finish, and only a grid small enough to be resident as a whole runs as one wave;
// 16-byte stores of bf16).
template <typename TO, int V>
__global__ void __launch_bounds__(256) combine_vec_kernel(int64_t rows, int32_t rows_per_seq, int32_t S, int32_t d_out,
                                                          const float* __restrict__ o_part,
                                                          const float* __restrict__ lse_part, TO* __restrict__ out,
                                                          float* __restrict__ lse) {
    // (dependent-launch instructions; no-ops when the kernel is launched the ordinary way)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int32_t vec_per_row = d_out / V;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const int64_t r = idx / vec_per_row;
    if (r >= rows) return;
    const int c = (int)(idx % vec_per_row) * V;
    const int64_t b = r / rows_per_seq;
    const int rr = (int)(r % rows_per_seq);
    const float* lp = lse_part + b * S * rows_per_seq + rr;
    float mx = -INFINITY;
    for (int k = 0; k < S; ++k) mx = fmaxf(mx, __ldg(lp + (int64_t)k * rows_per_seq));
    const bool dead = !(mx > -INFINITY);
    const float* op = o_part + (b * S * rows_per_seq + rr) * d_out + c;
    const int64_t kstride = (int64_t)rows_per_seq * d_out;
    float4 acc[V / 4];
#pragma unroll
    for (int u = 0; u < V / 4; ++u) acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
    float den = 0.f;
    for (int k = 0; k < S; ++k) {
        const float wk = dead ? 0.f : expf(__ldg(lp + (int64_t)k * rows_per_seq) - mx);
        den += wk;
        if (wk == 0.f) continue;  // an empty split's partial is never read
#pragma unroll
        for (int u = 0; u < V / 4; ++u) {
            const float4 x = ld_stream4(op + k * kstride + 4 * u);
            acc[u].x = fmaf(wk, x.x, acc[u].x);
            acc[u].y = fmaf(wk, x.y, acc[u].y);
            acc[u].z = fmaf(wk, x.z, acc[u].z);
            acc[u].w = fmaf(wk, x.w, acc[u].w);
        }
    }
    const float inv = den > 0.f ? 1.f / den : 0.f;
#pragma unroll
    for (int u = 0; u < V / 4; ++u) {
        acc[u].x *= inv; acc[u].y *= inv; acc[u].z *= inv; acc[u].w *= inv;
    }
    if constexpr (V >= 8 && sizeof(TO) == 2) {  // eight bf16 per 16-byte store
#pragma unroll
        for (int u = 0; u < V / 8; ++u) {
            __nv_bfloat162 h0 = __floats2bfloat162_rn(acc[2 * u].x, acc[2 * u].y), h1 = __floats2bfloat162_rn(acc[2 * u].z, acc[2 * u].w);
            __nv_bfloat162 h2 = __floats2bfloat162_rn(acc[2 * u + 1].x, acc[2 * u + 1].y),
                           h3 = __floats2bfloat162_rn(acc[2 * u + 1].z, acc[2 * u + 1].w);
            uint4 u4;
            u4.x = *reinterpret_cast<uint32_t*>(&h0);
            u4.y = *reinterpret_cast<uint32_t*>(&h1);
            u4.z = *reinterpret_cast<uint32_t*>(&h2);
            u4.w = *reinterpret_cast<uint32_t*>(&h3);
            *reinterpret_cast<uint4*>(out + r * d_out + c + 8 * u) = u4;
        }
    } else {
#pragma unroll
        for (int u = 0; u < V / 4; ++u) store4(out + r * d_out + c + 4 * u, acc[u]);
    }
    if (lse != nullptr && c == 0) lse[r] = dead ? -INFINITY : mx + logf(den);
}

// q_hat[row, r] = sum_d W_UK[j][r][d] * q_c[row, d]  (r < r_kv);  q_hat[row, r_kv + d] = q_r[row, d].
// One block per row (b, p, i); the q_c row is staged in shared memory.
template <typename T>
__global__ void __launch_bounds__(128) absorb_q_generic_kernel(int32_t h_q, int32_t hpg, int32_t d_h, int32_t r_kv,
                                                               int32_t d_r, const T* __restrict__ q_c,
                                                               const T* __restrict__ q_r, const T* __restrict__ w_uk,
                                                               T* __restrict__ q_hat) {
    extern __shared__ float qs[];  // [d_h]
    const int64_t row = blockIdx.x;
    const int i = (int)(row % h_q);
    const int j = i / hpg;
    for (int d = threadIdx.x; d < d_h; d += blockDim.x) qs[d] = ldf(q_c + row * d_h + d);
    __syncthreads();
    const T* W = w_uk + (int64_t)j * r_kv * d_h;
    T* out = q_hat + row * (r_kv + d_r);
    for (int r = threadIdx.x; r < r_kv; r += blockDim.x) {
        const T* wr = W + (int64_t)r * d_h;
        float acc = 0.f;
        for (int d = 0; d < d_h; ++d) acc = fmaf(ldf(wr + d), qs[d], acc);
        stf(out + r, acc);
    }
    for (int d = threadIdx.x; d < d_r; d += blockDim.x) out[r_kv + d] = q_r[row * d_r + d];
}

// o[row, d] = sum_r W_UV[j][r][d] * o_hat[row, r].  One block per row; o_hat row staged in smem.
// d_h here is the width of W_UV's rows and of the output (the value head dim d_h^V when it differs from d_h).
template <typename T>
__global__ void __launch_bounds__(128) up_proj_generic_kernel(int32_t h_q, int32_t hpg, int32_t d_h, int32_t r_kv,
                                                              const T* __restrict__ o_hat, const T* __restrict__ w_uv,
                                                              T* __restrict__ o) {
    extern __shared__ float os[];  // [r_kv]
    const int64_t row = blockIdx.x;
    const int i = (int)(row % h_q);
    const int j = i / hpg;
    for (int r = threadIdx.x; r < r_kv; r += blockDim.x) os[r] = ldf(o_hat + row * r_kv + r);
    __syncthreads();
    const T* W = w_uv + (int64_t)j * r_kv * d_h;
    for (int d = threadIdx.x; d < d_h; d += blockDim.x) {
        float acc = 0.f;
        for (int r = 0; r < r_kv; ++r) acc = fmaf(ldf(W + (int64_t)r * d_h + d), os[r], acc);
        stf(o + row * d_h + d, acc);
    }
}

// Split merge fused with the up-projection: o[row, d] = sum_r W_UV[j][r][d] * (sum_k w_k o_part[row, k, r]).
// One block per row; the merged latent row lives in shared memory only.
template <typename T>
__global__ void __launch_bounds__(128) combine_up_generic_kernel(int32_t h_q, int32_t hpg, int32_t d_h, int32_t r_kv,
                                                                 int32_t rows_per_seq, int32_t S,
                                                                 const float* __restrict__ o_part,
                                                                 const float* __restrict__ lse_part,
                                                                 const T* __restrict__ w_uv, T* __restrict__ o,
                                                                 float* __restrict__ lse) {
    extern __shared__ float os[];  // [r_kv]
    const int64_t row = blockIdx.x;  // (b, p, i)
    const int i = (int)(row % h_q);
    const int j = i / hpg;
    const int64_t b = row / rows_per_seq;
    const int rr = (int)(row % rows_per_seq);
    const float* lp = lse_part + b * S * rows_per_seq + rr;
    float mx = -INFINITY;
    for (int k = 0; k < S; ++k) mx = fmaxf(mx, lp[(int64_t)k * rows_per_seq]);
    const bool dead = !(mx > -INFINITY);
    float den = 0.f;
    for (int k = 0; k < S; ++k) den += dead ? 0.f : expf(lp[(int64_t)k * rows_per_seq] - mx);
    const float inv = den > 0.f ? 1.f / den : 0.f;
    const float* op = o_part + (b * S * rows_per_seq + rr) * r_kv;
    for (int r = threadIdx.x; r < r_kv; r += blockDim.x) {
        float acc = 0.f;
        for (int k = 0; k < S; ++k) {
            const float wk = dead ? 0.f : expf(lp[(int64_t)k * rows_per_seq] - mx);
            if (wk != 0.f) acc = fmaf(wk, op[(int64_t)k * rows_per_seq * r_kv + r], acc);
        }
        os[r] = acc * inv;
    }
    __syncthreads();
    const T* W = w_uv + (int64_t)j * r_kv * d_h;
    for (int d = threadIdx.x; d < d_h; d += blockDim.x) {
        float acc = 0.f;
        for (int r = 0; r < r_kv; ++r) acc = fmaf(ldf(W + (int64_t)r * d_h + d), os[r], acc);
        stf(o + row * d_h + d, acc);
    }
    if (lse != nullptr && threadIdx.x == 0) lse[row] = dead ? -INFINITY : mx + logf(den);
}

// K_C[n, j, d] = sum_r W_UK[j][r][d] c[n][r],  V likewise with W_UV,  k_R[n] = cache[n, r_kv:].
// One block per kRows cache rows; the latent rows are staged in shared memory and every thread
// owns one (j, d) output column of both planes for all staged rows.
constexpr int kExpandRows = 8;
template <typename T>
__global__ void __launch_bounds__(256) expand_cache_generic_kernel(int64_t N, int32_t g, int32_t d_h, int32_t d_v,
                                                                   int32_t r_kv, int32_t d_r, const T* __restrict__ cache,
                                                                   int64_t cache_stride, const T* __restrict__ w_uk,
                                                                   const T* __restrict__ w_uv, T* __restrict__ k_c,
                                                                   T* __restrict__ v, T* __restrict__ k_r) {
    extern __shared__ float cs[];  // [kExpandRows][r_kv]
    const int64_t n0 = (int64_t)blockIdx.x * kExpandRows;
    const int nr = (int)((N - n0) < kExpandRows ? (N - n0) : kExpandRows);
    for (int t = threadIdx.x; t < nr * r_kv; t += blockDim.x) {
        const int rr = t / r_kv, c = t % r_kv;
        cs[rr * r_kv + c] = ldf(cache + (n0 + rr) * cache_stride + c);
    }
    __syncthreads();
    // plane 0: K_C with W_UK [g, r_kv, d_h];  plane 1: V with W_UV [g, r_kv, d_v]
    for (int plane = 0; plane < 2; ++plane) {
        const int dd = plane == 0 ? d_h : d_v;
        const T* wbase = plane == 0 ? w_uk : w_uv;
        T* out = plane == 0 ? k_c : v;
        const int cols = g * dd;
        for (int col = threadIdx.x; col < cols; col += blockDim.x) {
            const int j = col / dd, d = col % dd;
            const T* w = wbase + (int64_t)j * r_kv * dd + d;
            float acc[kExpandRows];
#pragma unroll
            for (int rr = 0; rr < kExpandRows; ++rr) acc[rr] = 0.f;
            for (int r = 0; r < r_kv; ++r) {
                const float a = ldf(w + (int64_t)r * dd);
#pragma unroll
                for (int rr = 0; rr < kExpandRows; ++rr) acc[rr] = fmaf(a, cs[rr * r_kv + r], acc[rr]);
            }
#pragma unroll
            for (int rr = 0; rr < kExpandRows; ++rr)
                if (rr < nr) stf(out + (n0 + rr) * cols + col, acc[rr]);
        }
    }
    if (k_r != nullptr)
        for (int t = threadIdx.x; t < nr * d_r; t += blockDim.x) {
            const int rr = t / d_r, c = t % d_r;
            k_r[(n0 + rr) * d_r + c] = cache[(n0 + rr) * cache_stride + r_kv + c];
        }
}

// The same expansion for the rows appended by the current decode step only: the last s_q rows of every
// sequence (positions seqlens[b] - s_q + p >= 0).  One block stages kExpandRows such rows and computes one
// (plane, group) slice of them, so a weight slice is read once per block.  Thread (d, q) sums a quarter
// of the latent index for output column d of all staged rows (the weight loads of a warp are coalesced
// and several are in flight); the four quarters meet in shared memory.
constexpr int kAppendThreads = 512, kAppendKSplit = 4, kAppendCols = kAppendThreads / kAppendKSplit;
template <typename T>
__global__ void __launch_bounds__(kAppendThreads)
append_expand_kernel(int32_t B, int32_t s_q, int32_t g, int32_t d_h, int32_t r_kv, int32_t d_r,
                     const T* __restrict__ cache, int64_t cache_stride, const int64_t* __restrict__ seq_start,
                     const int32_t* __restrict__ seqlens, const T* __restrict__ w_uk, const T* __restrict__ w_uv,
                     T* __restrict__ k_c, T* __restrict__ v, T* __restrict__ k_r) {
    extern __shared__ float cs[];                 // [kExpandRows][r_kv] latent rows
    float* red = cs + kExpandRows * r_kv;         // [kAppendKSplit][kExpandRows][kAppendCols] partial sums
    __shared__ int64_t rows[kExpandRows];
    const int64_t u0 = (int64_t)blockIdx.x * kExpandRows;  // first (sequence, new token) unit of this block
    if (threadIdx.x < kExpandRows) {
        const int64_t u = u0 + threadIdx.x;
        int64_t n = -1;
        if (u < (int64_t)B * s_q) {
            const int32_t b = (int32_t)(u / s_q), pq = (int32_t)(u % s_q);
            const int32_t pos = seqlens[b] - s_q + pq;
            if (pos >= 0) n = seq_start[b] + pos;
        }
        rows[threadIdx.x] = n;
    }
    __syncthreads();
    for (int t = threadIdx.x; t < kExpandRows * r_kv; t += blockDim.x) {
        const int rr = t / r_kv, c = t % r_kv;
        cs[t] = rows[rr] >= 0 ? ldf(cache + rows[rr] * cache_stride + c) : 0.f;
    }
    __syncthreads();
    const int plane = blockIdx.y / g, j = blockIdx.y % g;
    const T* w = (plane == 0 ? w_uk : w_uv) + (int64_t)j * r_kv * d_h;
    T* out = plane == 0 ? k_c : v;
    const int dl = threadIdx.x % kAppendCols, kq = threadIdx.x / kAppendCols;
    const int r_lo = (int)((int64_t)r_kv * kq / kAppendKSplit), r_hi = (int)((int64_t)r_kv * (kq + 1) / kAppendKSplit);
    for (int d0 = 0; d0 < d_h; d0 += kAppendCols) {
        const int d = d0 + dl;
        float acc[kExpandRows];
#pragma unroll
        for (int rr = 0; rr < kExpandRows; ++rr) acc[rr] = 0.f;
        if (d < d_h) {
#pragma unroll 8
            for (int r = r_lo; r < r_hi; ++r) {
                const float a = ldf(w + (int64_t)r * d_h + d);
#pragma unroll
                for (int rr = 0; rr < kExpandRows; ++rr) acc[rr] = fmaf(a, cs[rr * r_kv + r], acc[rr]);
            }
        }
#pragma unroll
        for (int rr = 0; rr < kExpandRows; ++rr) red[(kq * kExpandRows + rr) * kAppendCols + dl] = acc[rr];
        __syncthreads();
        // thread (dl, kq) finishes rows kq and kq + kAppendKSplit
        if (d < d_h)
            for (int rr = kq; rr < kExpandRows; rr += kAppendKSplit) {
                float sum = 0.f;
#pragma unroll
                for (int q = 0; q < kAppendKSplit; ++q) sum += red[(q * kExpandRows + rr) * kAppendCols + dl];
                if (rows[rr] >= 0) stf(out + (rows[rr] * g + j) * d_h + d, sum);
            }
        __syncthreads();
    }
    if (k_r != nullptr && blockIdx.y == 0)
        for (int t = threadIdx.x; t < kExpandRows * d_r; t += blockDim.x) {
            const int rr = t / d_r, c = t % d_r;
            if (rows[rr] >= 0) k_r[rows[rr] * d_r + c] = cache[rows[rr] * cache_stride + r_kv + c];
        }
}


// ------------------------------------------------------------------------------------------------ FP8 (E4M3)
// Quantisers.  Every step is an fp32 operation with IEEE rounding (division included), so the code a value
// gets is a pure function of its stored bits and the scales.

// dst[r, c] = encode( float(src[r, c]) * (1 / scale) ),  scale = scale_a for c < split, scale_b otherwise.
template <typename T>
__global__ void __launch_bounds__(256) quantize_cols_kernel(int64_t rows, int32_t width, int32_t split, float scale_a,
                                                            float scale_b, const T* __restrict__ src, int64_t src_stride,
                                                            uint8_t* __restrict__ dst) {
    const float inv_a = __fdiv_rn(1.f, scale_a), inv_b = __fdiv_rn(1.f, scale_b);
    const int64_t pairs_per_row = (width + 1) / 2;
    const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= rows * pairs_per_row) return;
    const int64_t r = idx / pairs_per_row;
    const int c = (int)(idx % pairs_per_row) * 2;
    const float x0 = __fmul_rn(ldf(src + r * src_stride + c), c < split ? inv_a : inv_b);
    if (c + 1 < width) {
        const float x1 = __fmul_rn(ldf(src + r * src_stride + c + 1), c + 1 < split ? inv_a : inv_b);
        const uint16_t pk = float2_to_e4m3x2(x0, x1);
        dst[r * width + c] = (uint8_t)(pk & 0xff);
        dst[r * width + c + 1] = (uint8_t)(pk >> 8);
    } else {
        dst[r * width + c] = (uint8_t)(float2_to_e4m3x2(x0, 0.f) & 0xff);
    }
}

// Per row: y = float(src) * pre (pre_a for c < split, pre_b otherwise), s = max|y| / 448 (1 for a zero row),
// dst = encode(y * (1 / s)), row_scale = s.  One warp per row.
template <typename T>
__global__ void __launch_bounds__(128) quantize_rows_kernel(int64_t rows, int32_t width, int32_t split, float pre_a,
                                                            float pre_b, const T* __restrict__ src,
                                                            uint8_t* __restrict__ dst, float* __restrict__ row_scale) {
    // (dependent-launch instructions; no-ops when the kernel is launched the ordinary way)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int lane = threadIdx.x & 31;
    const int64_t r = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (r >= rows) return;
    const T* x = src + r * width;
    float amax = 0.f;
    for (int c = lane; c < width; c += 32) amax = fmaxf(amax, fabsf(__fmul_rn(ldf(x + c), c < split ? pre_a : pre_b)));
    amax = warp_max(amax);
    const float s = amax > 0.f ? __fdiv_rn(amax, 448.f) : 1.f;
    const float inv = __fdiv_rn(1.f, s);
    for (int c = lane; c < width; c += 32) {
        const float y = __fmul_rn(__fmul_rn(ldf(x + c), c < split ? pre_a : pre_b), inv);
        dst[r * width + c] = (uint8_t)(float2_to_e4m3x2(y, 0.f) & 0xff);
    }
    if (lane == 0) row_scale[r] = s;
}

// The same for bf16 rows whose width and split are multiples of 8 and whose width is at most 1024: every lane keeps
// its 16-byte chunks (8 values each) of the row in registers, so the row is read once and written as 8-byte
// chunks.  Same fp32 operations in the same order per element: the codes are identical to the kernel above.
constexpr int kQuantChunksPerLane = 4;
__global__ void __launch_bounds__(128) quantize_rows_bf16_vec_kernel(int64_t rows, int32_t width, int32_t split, float pre_a,
                                                                     float pre_b, const __nv_bfloat16* __restrict__ src,
                                                                     uint8_t* __restrict__ dst, float* __restrict__ row_scale) {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const int lane = threadIdx.x & 31;
    const int64_t r = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (r >= rows) return;
    const uint4* x = reinterpret_cast<const uint4*>(src + r * width);
    const int chunks = width >> 3;
    float y[kQuantChunksPerLane][8];
    float amax = 0.f;
#pragma unroll
    for (int k = 0; k < kQuantChunksPerLane; ++k) {
        const int ci = lane + 32 * k;
        if (ci < chunks) {
            const uint4 u = x[ci];
            const float pre = ci * 8 < split ? pre_a : pre_b;
            const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                y[k][2 * i] = __fmul_rn(__uint_as_float(w[i] << 16), pre);           // bf16 -> fp32 is a shift
                y[k][2 * i + 1] = __fmul_rn(__uint_as_float(w[i] & 0xffff0000u), pre);
                amax = fmaxf(amax, fmaxf(fabsf(y[k][2 * i]), fabsf(y[k][2 * i + 1])));
            }
        }
    }
    amax = warp_max(amax);
    const float s = amax > 0.f ? __fdiv_rn(amax, 448.f) : 1.f;
    const float inv = __fdiv_rn(1.f, s);
    uint2* out = reinterpret_cast<uint2*>(dst + r * width);
#pragma unroll
    for (int k = 0; k < kQuantChunksPerLane; ++k) {
        const int ci = lane + 32 * k;
        if (ci < chunks) {
            uint32_t lo = (uint32_t)float2_to_e4m3x2(__fmul_rn(y[k][0], inv), __fmul_rn(y[k][1], inv)) |
                          ((uint32_t)float2_to_e4m3x2(__fmul_rn(y[k][2], inv), __fmul_rn(y[k][3], inv)) << 16);
            uint32_t hi = (uint32_t)float2_to_e4m3x2(__fmul_rn(y[k][4], inv), __fmul_rn(y[k][5], inv)) |
                          ((uint32_t)float2_to_e4m3x2(__fmul_rn(y[k][6], inv), __fmul_rn(y[k][7], inv)) << 16);
            out[ci] = make_uint2(lo, hi);
        }
    }
    if (lane == 0) row_scale[r] = s;
}

}  // namespace gqla
