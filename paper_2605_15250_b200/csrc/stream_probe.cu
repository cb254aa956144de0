// Bandwidth probe of the absorb kernel's K stream: CTAs pull [64 rows x 64 columns] bf16 TMA boxes of a latent
// cache [N, 576] through a ring of three-box groups exactly as the decode kernel's K producer does, and nothing
// consumes them (a second thread hands every landed group straight back).  It answers one question: how fast can
// this access pattern be fed from HBM (or from L2) with a given number of bytes in flight per CTA?
// A measurement tool beside the sweep; not part of the decode path.  Every wait is bounded.
#include "tc_common.cuh"

using namespace gqla::tc;

namespace {

constexpr int kGroupBytes = 3 * 8192;

struct ProbeParams {
    int32_t tiles, rows_per_seq, depth, l2_resident;
    int32_t* status;
};

__global__ void __launch_bounds__(64, 1) stream_probe_kernel(const ProbeParams p, const __grid_constant__ CUtensorMap tm) {
    extern __shared__ __align__(1024) uint8_t smem[];
    uint64_t* full = reinterpret_cast<uint64_t*>(smem + p.depth * kGroupBytes);
    uint64_t* empty = full + p.depth;
    volatile int32_t* flag = reinterpret_cast<volatile int32_t*>(empty + p.depth);
    if (threadIdx.x == 0) {
        for (int i = 0; i < p.depth; ++i) {
            mbar_init(&full[i], 1);
            mbar_init(&empty[i], 1);
        }
        *flag = 0;
        fence_mbar_init();
    }
    __syncthreads();
    const Abort ab{flag, p.status};
    const int b = blockIdx.x >> 1, half = blockIdx.x & 1;  // a CTA pair shares a sequence: 64 of every 128 rows each
    const int groups = p.tiles * 3;
    if (threadIdx.x == 0) {
        int s = 0;
        uint32_t ph = 1;
        for (int gi = 0; gi < groups; ++gi) {
            const int t = gi / 3, kg = gi % 3;
            if (!mbar_wait(&empty[s], ph, ab, 1)) break;
            mbar_expect_tx(&full[s], kGroupBytes);
            const int row = b * p.rows_per_seq + (p.l2_resident ? 0 : t * 128) + half * 64;
            for (int i = 0; i < 3; ++i) tma_load_2d(smem + s * kGroupBytes + i * 8192, &tm, (3 * kg + i) * 64, row, &full[s]);
            if (++s == p.depth) { s = 0; ph ^= 1; }
        }
    } else if (threadIdx.x == 32) {
        int s = 0;
        uint32_t ph = 0;
        for (int gi = 0; gi < groups; ++gi) {
            if (!mbar_wait(&full[s], ph, ab, 2)) break;
            mbar_arrive(&empty[s]);
            if (++s == p.depth) { s = 0; ph ^= 1; }
        }
    }
}

}  // namespace

// cache: device pointer to bf16 [n_rows, 576] (dense); n_ctas CTAs (two per sequence) stream `tiles` 128-row tiles each
// through a ring of `depth` groups (24 KB each, depth <= 9).  l2_resident != 0: every tile re-reads the sequence's
// first tile.  Returns 0, or 1 (bad argument), 2 (tensor map), 3 (launch).
extern "C" int gqla_stream_probe(const void* cache, long long n_rows, int n_ctas, int tiles, int rows_per_seq, int depth,
                                 int l2_resident, int32_t* status, void* stream) {
    if (cache == nullptr || depth < 1 || depth > 9 || n_ctas < 1 || tiles < 1 ||
        (long long)((n_ctas + 1) / 2 - 1) * rows_per_seq + (long long)tiles * 128 > n_rows)
        return 1;
    CUtensorMap tm;
    const uint64_t dims[2] = {576, (uint64_t)n_rows};
    const uint64_t str[1] = {576 * 2};
    const uint32_t box[2] = {64, 64};
    if (!make_tmap_bf16(&tm, cache, 2, dims, str, box)) return 2;
    ProbeParams p{tiles, rows_per_seq, depth, l2_resident, status};
    const int smem = depth * kGroupBytes + depth * 16 + 16;
    if (cudaFuncSetAttribute(stream_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return 3;
    stream_probe_kernel<<<n_ctas, 64, smem, (cudaStream_t)stream>>>(p, tm);
    return cudaGetLastError() == cudaSuccess ? 0 : 3;
}
