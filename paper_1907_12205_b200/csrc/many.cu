// Filtering and A_0 = mean for very many nodes with short vectors: the regime of the synthetic mean-estimation
// experiment (Section 5.3, "Mean estimation on synthetic data": p = 220,000 nodes, r = 11, d <= 100), where the
// group table no longer fits kernel parameters and a whole group (r rows of d values) is a few KB.
//
//   vote_many_kernel       one warp per node group: the lanes walk the columns, compare the r rows pairwise on their
//                          bit patterns and OR the "differs" bits over the warp; lane 0 finds the class with more
//                          than r/2 members and writes its lowest worker id (or -1).
//   hier_mean_many_kernel  one CTA per vote set and 32 columns: its warps add runs of the set's votes (the winners'
//                          rows; a group without a majority counts as a zero row) in fp64, the runs are added in
//                          order, and the mean is written.
// Vote sets are runs of consecutive groups (the group table is already a random partition).
#include "common.cuh"

namespace detox {

namespace {

constexpr int kManyWarps = 8;   // groups per CTA

struct OffsetTable {
    int32_t offset[DETOX_MAX_ROWS + 1];
};

__host__ __device__ constexpr int many_pair_index(int r, int a, int b) { return a * (2 * r - a - 1) / 2 + (b - a - 1); }

template <int R>
__global__ void __launch_bounds__(kManyWarps * 32)
vote_many_kernel(const float* __restrict__ X, int64_t ld, int64_t n, int d, const int32_t* __restrict__ members, int64_t G,
                 int32_t* __restrict__ winner) {
    constexpr int kPairs = R * (R - 1) / 2;
    constexpr int kWords = kPairs == 0 ? 1 : (kPairs + 31) / 32;
    const int lane = threadIdx.x & 31;
    const int64_t g = (int64_t)blockIdx.x * kManyWarps + (threadIdx.x >> 5);
    if (g >= G) return;
    int32_t id[R];
    bool valid = true;
#pragma unroll
    for (int a = 0; a < R; ++a) {
        id[a] = members[g * R + a];
        valid &= id[a] >= 0 && id[a] < n;
    }
    if (!valid) {                       // an id outside 0..n-1: the group has no vote
        if (lane == 0) winner[g] = -1;
        return;
    }
    uint32_t diff[kWords];
#pragma unroll
    for (int w = 0; w < kWords; ++w) diff[w] = 0u;
    for (int c = lane; c < d; c += 32) {
        uint32_t v[R];
#pragma unroll
        for (int a = 0; a < R; ++a) v[a] = ld_stream_u1(X + (int64_t)id[a] * ld + c);
#pragma unroll
        for (int a = 0; a < R; ++a)
#pragma unroll
            for (int b = a + 1; b < R; ++b) {
                const int p = many_pair_index(R, a, b);
                if (v[a] != v[b]) diff[p >> 5] |= 1u << (p & 31);
            }
    }
#pragma unroll
    for (int w = 0; w < kWords; ++w) diff[w] = __reduce_or_sync(0xffffffffu, diff[w]);
    if (lane != 0) return;
    int win = -1;
#pragma unroll
    for (int a = 0; a < R; ++a) {
        if (win >= 0) continue;
        int agree = 1;
        int lowest = id[a];
#pragma unroll
        for (int b = 0; b < R; ++b) {
            if (b == a) continue;
            const int p = a < b ? many_pair_index(R, a, b) : many_pair_index(R, b, a);
            if (((diff[p >> 5] >> (p & 31)) & 1u) == 0u) {
                ++agree;
                lowest = id[b] < lowest ? id[b] : lowest;
            }
        }
        if (2 * agree > R) win = lowest;
    }
    winner[g] = win;
}

// grid (column tiles of 32, S); 32 warps: warp w adds a run of consecutive groups of the set (lane = column), the
// runs' fp64 sums are then added in run order, so the result does not depend on timing.
constexpr int kMeanManyWarps = 32;
__global__ void __launch_bounds__(kMeanManyWarps * 32)
hier_mean_many_kernel(const float* __restrict__ X, int64_t ld, int d, const int32_t* __restrict__ winner,
                      const __grid_constant__ OffsetTable sets, float* __restrict__ M, int64_t ldm) {
    __shared__ double part[kMeanManyWarps][32];
    const int s = blockIdx.y;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int c = blockIdx.x * 32 + lane;
    const int b = sets.offset[s], e = sets.offset[s + 1];
    const int run = (e - b + kMeanManyWarps - 1) / kMeanManyWarps;
    const int g0 = b + warp * run, g1 = g0 + run < e ? g0 + run : e;
    double acc = 0.0;
    if (c < d) {
        int g = g0;
        for (; g + 8 <= g1; g += 8) {          // eight loads in flight, added in group order
            float v[8];
#pragma unroll
            for (int k = 0; k < 8; ++k) {
                const int w = winner[g + k];
                v[k] = w >= 0 ? X[(int64_t)w * ld + c] : 0.f;
            }
#pragma unroll
            for (int k = 0; k < 8; ++k) acc += (double)v[k];
        }
        for (; g < g1; ++g) {
            const int w = winner[g];
            acc += w >= 0 ? (double)X[(int64_t)w * ld + c] : 0.0;
        }
    }
    part[warp][lane] = acc;
    __syncthreads();
    if (warp == 0 && c < d) {
        double tot = 0.0;
#pragma unroll 8
        for (int w = 0; w < kMeanManyWarps; ++w) tot += part[w][lane];
        M[(int64_t)s * ldm + c] = (float)(tot / (double)(e - b));
    }
}

}  // namespace

}  // namespace detox

using namespace detox;

extern "C" detox_status detox_vote_hier_mean_many(const float* X, int64_t ld, int64_t n, int r, int d,
                                                  const int32_t* members, const int32_t* set_offsets, int S, float* M,
                                                  int64_t ldm, int32_t* winner, void* stream) {
    if (!X || !members || !winner || n < 1 || n > ((int64_t)1 << 30) || d < 1 || ld < d) return DETOX_ERR_BAD_ARG;
    if (r < 1 || (r & 1) == 0 || n % r != 0) return DETOX_ERR_BAD_ARG;
    if (r > kMaxR || d > DETOX_MANY_MAX_D) return DETOX_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(X) & 3u) != 0) return DETOX_ERR_BAD_ARG;
    const int64_t G = n / r;
    OffsetTable tab;
    if (M) {
        if (!set_offsets || S < 1 || S > kMaxRows || ldm < d || (reinterpret_cast<uintptr_t>(M) & 3u) != 0)
            return S > kMaxRows ? DETOX_ERR_UNSUPPORTED : DETOX_ERR_BAD_ARG;
        if (set_offsets[0] != 0 || set_offsets[S] != G) return DETOX_ERR_BAD_ARG;
        for (int s = 0; s < S; ++s) {
            if (set_offsets[s + 1] <= set_offsets[s]) return DETOX_ERR_BAD_ARG;
            tab.offset[s] = set_offsets[s];
        }
        tab.offset[S] = set_offsets[S];
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const unsigned blocks = (unsigned)ceil_div(G, (int64_t)kManyWarps);
    switch (r) {
#define DETOX_CASE(R) \
    case R: vote_many_kernel<R><<<blocks, kManyWarps * 32, 0, st>>>(X, ld, n, d, members, G, winner); break;
        DETOX_CASE(1) DETOX_CASE(3) DETOX_CASE(5) DETOX_CASE(7) DETOX_CASE(9) DETOX_CASE(11) DETOX_CASE(13) DETOX_CASE(15)
#undef DETOX_CASE
        default: return DETOX_ERR_UNSUPPORTED;
    }
    detox_status rc = launch_status();
    if (rc != DETOX_OK || !M) return rc;
    hier_mean_many_kernel<<<dim3((unsigned)ceil_div((int64_t)d, 32), (unsigned)S), kMeanManyWarps * 32, 0, st>>>(X, ld, d, winner, tab, M, ldm);
    return launch_status();
}
