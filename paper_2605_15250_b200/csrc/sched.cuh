// Work scheduling of the split-KV decode kernels: which (sequence, split) pieces a CTA (or CTA pair)
// processes, and in which order.  Split-KV is not in the paper; two plans are offered.
//
//   fixed:     split k of S of a sequence of T rows covers [k*chunk, min((k+1)*chunk, T)),
//              chunk = ceil(ceil(T/S)/64)*64.  One piece per launched worker.
//   balanced:  the 128-row tiles of all sequences are laid end to end (sequence 0 first) and cut into
//              equal shares of `share` tiles, one share per worker w of W:  worker w owns the global
//              tiles [w*share, (w+1)*share).  share = max(ceil(total/W), ceil(max_b tiles_b/(S-1))), so
//              no sequence is cut into more than S pieces (S >= 2).  The pieces of sequence b are
//              numbered k = 0, 1, .. in row order; slots k >= n_pieces(b) are marked empty (lse = -inf)
//              by the worker that owns piece 0 (for an empty sequence: by the worker whose share contains
//              its position off_b, or by the last worker when it lies behind every tile).
//
// Both are pure integer functions of (seqlens, S, W), evaluated identically by every role of a worker
// and, on the host, by gqla_balanced_plan for comparison with an independent statement of the rule.
#pragma once
#include <stdint.h>

#include "common.cuh"

namespace gqla {

constexpr int kTileRows = 128;

struct Piece {
    int32_t b, k;                  // sequence and split slot
    int32_t tok_begin, tok_end;    // rows of the sequence covered (tok_begin is a multiple of 128 when balanced)
    int32_t n_tiles;               // ceil((tok_end - tok_begin)/128); 0 for an empty piece
    int32_t fill_begin, fill_end;  // split slots [fill_begin, fill_end) of b this worker marks empty
};

// Everything a worker needs to start walking a balanced plan.
struct BalancedStart {
    int32_t share, my_begin, my_end, b0, off_b0, total;
};

__host__ __device__ inline int32_t ceil_div_i32(int64_t a, int64_t b) { return (int32_t)((a + b - 1) / b); }
__host__ __device__ inline int32_t tiles_of(int32_t T) { return T > 0 ? (T + kTileRows - 1) / kTileRows : 0; }

// share from the batch totals (see the header comment).
__host__ __device__ inline int32_t balanced_share(int64_t total_tiles, int32_t max_tiles, int32_t S, int32_t W) {
    int32_t share = ceil_div_i32(total_tiles, W);
    const int32_t min_share = ceil_div_i32(max_tiles, S - 1);
    if (share < min_share) share = min_share;
    return share < 1 ? 1 : share;
}

struct Walker {
    const int32_t* seqlens;
    int32_t B, S;
    bool balanced;
    // fixed plan: exactly one piece
    int32_t fb, fk;
    bool fixed_done;
    // balanced plan
    int32_t w, W, share, my_begin, my_end, b, off, total;

    __host__ __device__ void init_fixed(const int32_t* sl, int32_t B_, int32_t S_, int32_t b_, int32_t k_) {
        seqlens = sl; B = B_; S = S_; balanced = false; fb = b_; fk = k_; fixed_done = false;
        w = W = share = my_begin = my_end = b = off = total = 0;
    }
    __host__ __device__ void init_balanced(const int32_t* sl, int32_t B_, int32_t S_, int32_t w_, int32_t W_,
                                          const BalancedStart& st) {
        seqlens = sl; B = B_; S = S_; balanced = true; fb = fk = 0; fixed_done = true;
        w = w_; W = W_; share = st.share; my_begin = st.my_begin; my_end = st.my_end;
        b = st.b0; off = st.off_b0; total = st.total;
    }

    __host__ __device__ bool next(Piece& pc) {
        if (!balanced) {
            if (fixed_done) return false;
            fixed_done = true;
            const int32_t T = seqlens[fb];
            pc.b = fb; pc.k = fk;
            split_range(T, S, fk, &pc.tok_begin, &pc.tok_end);
            pc.n_tiles = pc.tok_end > pc.tok_begin ? tiles_of(pc.tok_end - pc.tok_begin) : 0;
            pc.fill_begin = pc.fill_end = 0;
            return true;
        }
        while (b < B) {
            // past this worker's share (an empty sequence exactly on the boundary belongs to w + 1);
            // the last worker walks on to pick up empty sequences behind the last tile
            if (off >= my_end && w != W - 1) return false;
            const int32_t T = seqlens[b];
            const int32_t tiles = tiles_of(T);
            const int32_t cur_b = b, cur_off = off;
            ++b;
            off += tiles;
            if (tiles == 0) {
                const int32_t owner = cur_off >= total ? W - 1 : cur_off / share;
                if (owner != w) continue;
                pc.b = cur_b; pc.k = 0; pc.tok_begin = pc.tok_end = 0; pc.n_tiles = 0;
                pc.fill_begin = 0; pc.fill_end = S;
                return true;
            }
            const int32_t g0 = cur_off > my_begin ? cur_off : my_begin;
            const int32_t g1 = cur_off + tiles < my_end ? cur_off + tiles : my_end;
            if (g0 >= g1) continue;
            pc.b = cur_b;
            pc.k = g0 == cur_off ? 0 : w - cur_off / share;
            pc.tok_begin = (g0 - cur_off) * kTileRows;
            const int32_t te = (g1 - cur_off) * kTileRows;
            pc.tok_end = te < T ? te : T;
            pc.n_tiles = g1 - g0;
            if (pc.k == 0) {
                pc.fill_begin = (cur_off + tiles - 1) / share - cur_off / share + 1;
                pc.fill_end = S;
            } else {
                pc.fill_begin = pc.fill_end = 0;
            }
            return true;
        }
        return false;
    }
};

// Single-thread evaluation of the start record of worker w (host helper; the kernels compute the same
// values cooperatively with balanced_prepass below).
__host__ __device__ inline BalancedStart balanced_start_serial(const int32_t* seqlens, int32_t B, int32_t S, int32_t w,
                                                               int32_t W) {
    int64_t total = 0;
    int32_t mx = 0;
    for (int32_t i = 0; i < B; ++i) {
        const int32_t t = tiles_of(seqlens[i]);
        total += t;
        if (t > mx) mx = t;
    }
    BalancedStart st;
    st.share = balanced_share(total, mx, S, W);
    const int64_t mb = (int64_t)w * st.share;
    st.my_begin = (int32_t)(mb < total ? mb : total);
    const int64_t me = (int64_t)st.my_begin + st.share;
    st.my_end = (int32_t)(me < total ? me : total);
    st.total = (int32_t)total;
    st.b0 = B;
    st.off_b0 = (int32_t)total;
    int32_t off = 0;
    for (int32_t i = 0; i < B; ++i) {
        const int32_t t = tiles_of(seqlens[i]);
        if (off + (t > 0 ? t : 1) > st.my_begin) {
            st.b0 = i;
            st.off_b0 = off;
            break;
        }
        off += t;
    }
    return st;
}

#ifdef __CUDACC__
// Cooperative evaluation by all `nthreads` threads of a CTA (a multiple of 32, at most 1024).  `scratch` is
// shared memory of at least 3 * 32 + 4 int32.  Same result as balanced_start_serial.  Contains __syncthreads.
// Thread t owns the contiguous chunk [t * chunk, (t + 1) * chunk) of the sequences; chunk sums are scanned
// with warp shuffles and one shared-memory hop across warps.
__device__ inline BalancedStart balanced_prepass(const int32_t* seqlens, int32_t B, int32_t S, int32_t w, int32_t W,
                                                 int32_t* scratch, int nthreads) {
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nwarps = nthreads >> 5;
    const int32_t chunk = (B + nthreads - 1) / nthreads;
    const int32_t lo = tid * chunk < B ? tid * chunk : B, hi = lo + chunk < B ? lo + chunk : B;
    int32_t sum = 0, mx = 0;
    for (int32_t i = lo; i < hi; ++i) {
        const int32_t t = tiles_of(seqlens[i]);
        sum += t;
        if (t > mx) mx = t;
    }
    // inclusive scan of the chunk sums and maximum within the warp
    int32_t incl = sum;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int32_t up = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += up;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    int32_t* wsum = scratch;       // [32] warp totals
    int32_t* wmax = scratch + 32;  // [32] warp maxima
    int32_t* wfound = scratch + 64;  // [32] first matching sequence of each warp (B: none)
    int32_t* res = scratch + 96;   // [0] off_b0
    if (lane == 31) wsum[wid] = incl;
    if (lane == 0) wmax[wid] = mx;
    __syncthreads();
    int64_t total = 0;
    int32_t base = 0, gmax = 0;
    for (int i = 0; i < nwarps; ++i) {
        const int32_t c = wsum[i];
        if (i < wid) base += c;
        total += c;
        gmax = max(gmax, wmax[i]);
    }
    BalancedStart st;
    st.share = balanced_share(total, gmax, S, W);
    const int64_t mb = (int64_t)w * st.share;
    st.my_begin = (int32_t)(mb < total ? mb : total);
    const int64_t me = (int64_t)st.my_begin + st.share;
    st.my_end = (int32_t)(me < total ? me : total);
    st.total = (int32_t)total;
    // first sequence whose tiles (an empty one counts as a point) end beyond my_begin
    int32_t off = base + incl - sum, found = B, found_off = 0;
    for (int32_t i = lo; i < hi; ++i) {
        const int32_t t = tiles_of(seqlens[i]);
        if (off + (t > 0 ? t : 1) > st.my_begin) { found = i; found_off = off; break; }
        off += t;
    }
    int32_t wf = found;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) wf = min(wf, __shfl_xor_sync(0xffffffffu, wf, o));
    if (lane == 0) wfound[wid] = wf;
    __syncthreads();
    int32_t b0 = B;
    for (int i = 0; i < nwarps; ++i) b0 = min(b0, wfound[i]);
    if (found < B && found == b0) res[0] = found_off;
    __syncthreads();
    st.b0 = b0;
    st.off_b0 = b0 < B ? res[0] : (int32_t)total;
    __syncthreads();  // scratch may be reused by the caller
    return st;
}
#endif

}  // namespace gqla
