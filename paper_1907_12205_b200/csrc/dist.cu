// Pairwise squared distances between m rows (the O(p^2 d) part of Krum-type aggregators, Section 4,
// "Improved speed").  Output: D, m x m fp64, symmetric, zero diagonal.
//
//   m <= 16 : differences are formed directly, (x_i - x_j)^2, with one fp32 accumulator per pair in
//             registers; HBM-bound (m*d*4 bytes read once).
//   16 < m <= 256 with 16-byte aligned rows: the tensor-core Gram of gram_tc.cu.
//   otherwise : CUDA-core Gram tiles G = X X^T over K-slabs, D_ij = G_ii + G_jj - 2 G_ij.
// Both write per-CTA partial sums that a second kernel adds in a fixed order in fp64, so results
// are deterministic and bitwise-equal rows get bitwise-equal distances.
#include "common.cuh"

namespace detox {

namespace {

// ------------------------------------------------------------------ m <= 16: direct differences

constexpr int kDirThreads = 256;
constexpr int kDirWarps = kDirThreads / 32;

// VEC = columns per thread and step (4: 16-byte loads; 2: 8-byte; 1: scalar).  Columns past the last
// multiple of VEC are added by one thread.
template <int M, int VEC>
__global__ void __launch_bounds__(kDirThreads)
sqdist_direct_kernel(const float* __restrict__ X, int64_t ld, int64_t d, const int32_t* __restrict__ rows,
                     double* __restrict__ partial) {
    constexpr int NP = M * (M - 1) / 2;
    float acc[NP];
#pragma unroll
    for (int p = 0; p < NP; ++p) acc[p] = 0.f;
    // rows (optional): the M rows are X[rows[i]]; a negative entry stands for a zero row
    const float* rowp[M];
    float keep[M];
#pragma unroll
    for (int i = 0; i < M; ++i) {
        const int r = rows ? rows[i] : i;
        rowp[i] = X + (int64_t)(r < 0 ? 0 : r) * ld;
        keep[i] = r < 0 ? 0.f : 1.f;
    }

    const int64_t stride = (int64_t)gridDim.x * kDirThreads;
    const int64_t nv = d / VEC;
    for (int64_t c = (int64_t)blockIdx.x * kDirThreads + threadIdx.x; c < nv; c += stride) {
        float v[M][VEC];
#pragma unroll
        for (int i = 0; i < M; ++i) {
            if (VEC == 4) {
                const float4 t = ld_stream_f4(rowp[i] + c * 4);
                v[i][0] = t.x; v[i][1 % VEC] = t.y; v[i][2 % VEC] = t.z; v[i][3 % VEC] = t.w;
            } else if (VEC == 2) {
                const float2 t = __ldcs(reinterpret_cast<const float2*>(rowp[i]) + c);
                v[i][0] = t.x; v[i][1 % VEC] = t.y;
            } else {
                v[i][0] = __ldcs(rowp[i] + c);
            }
#pragma unroll
            for (int e = 0; e < VEC; ++e) v[i][e] = keep[i] == 0.f ? 0.f : v[i][e];
        }
        int p = 0;
#pragma unroll
        for (int i = 0; i < M; ++i)
#pragma unroll
            for (int j = i + 1; j < M; ++j, ++p) {
#pragma unroll
                for (int e = 0; e < VEC; ++e) {
                    const float a = v[i][e] - v[j][e];
                    acc[p] = fmaf(a, a, acc[p]);
                }
            }
    }
    if (VEC > 1 && blockIdx.x == 0 && threadIdx.x == 0) {
        for (int64_t c = nv * VEC; c < d; ++c) {
            int p = 0;
#pragma unroll
            for (int i = 0; i < M; ++i)
#pragma unroll
                for (int j = i + 1; j < M; ++j, ++p) {
                    const float a = (keep[i] == 0.f ? 0.f : rowp[i][c]) - (keep[j] == 0.f ? 0.f : rowp[j][c]);
                    acc[p] = fmaf(a, a, acc[p]);
                }
        }
    }

    // block reduction in fp64, fixed order
    __shared__ double red[kDirWarps][NP > 0 ? NP : 1];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int p = 0; p < NP; ++p) {
        double v = (double)acc[p];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
        if (lane == 0) red[warp][p] = v;
    }
    __syncthreads();
    for (int p = threadIdx.x; p < NP; p += kDirThreads) {
        double v = 0.0;
#pragma unroll
        for (int w = 0; w < kDirWarps; ++w) v += red[w][p];
        partial[(int64_t)blockIdx.x * NP + p] = v;
    }
}

// D from the per-CTA pair partials of the direct kernel: one warp per pair, lanes take the partials
// round-robin (independent loads), then a fixed shuffle tree.
__global__ void sqdist_direct_reduce_kernel(const double* __restrict__ partial, int nblocks, int m,
                                            double* __restrict__ D) {
    const int np = m * (m - 1) / 2;
    const int lane = threadIdx.x & 31;
    const int warps = (gridDim.x * blockDim.x) >> 5;
    for (int p = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; p < np; p += warps) {
        double v = 0.0;
        for (int b = lane; b < nblocks; b += 32) v += partial[(int64_t)b * np + p];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
        if (lane == 0) {
            int i = 0, rem = p;
            while (rem >= m - 1 - i) { rem -= m - 1 - i; ++i; }
            const int j = i + 1 + rem;
            D[i * m + j] = v;
            D[j * m + i] = v;
        }
    }
    if (blockIdx.x == 0)
        for (int i = threadIdx.x; i < m; i += blockDim.x) D[i * m + i] = 0.0;
}

// ------------------------------------------------------------------ m > 16: CUDA-core Gram tiles

constexpr int kGT = 64;          // output tile edge
constexpr int kGK = 32;          // columns per shared-memory step
constexpr int kGramThreads = 256;  // 16 x 16 threads, 4 x 4 outputs each

__global__ void __launch_bounds__(kGramThreads)
gram_simt_kernel(const float* __restrict__ X, int64_t ld, int m, int64_t d, int ntile, int nslab,
                 int64_t slab_cols, double* __restrict__ partial) {
    __shared__ float As[kGT][kGK + 1];
    __shared__ float Bs[kGT][kGK + 1];

    // item -> (tile pair bi <= bj, slab)
    const int pair = blockIdx.x / nslab;
    const int slab = blockIdx.x - pair * nslab;
    int bi = 0, rem = pair;
    while (rem >= ntile - bi) { rem -= ntile - bi; ++bi; }
    const int bj = bi + rem;

    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    double acc[4][4];
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) acc[a][b] = 0.0;

    const int64_t c_begin = (int64_t)slab * slab_cols;
    const int64_t c_end = c_begin + slab_cols < d ? c_begin + slab_cols : d;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    for (int64_t c0 = c_begin; c0 < c_end; c0 += kGK) {
        // each warp loads 8 rows of each tile; a row is 32 consecutive floats
#pragma unroll
        for (int rr = 0; rr < kGT / 8; ++rr) {
            const int r = warp * (kGT / 8) + rr;
            const int64_t c = c0 + lane;
            const int ra = bi * kGT + r, rb = bj * kGT + r;
            As[r][lane] = (ra < m && c < c_end) ? __ldg(X + (int64_t)ra * ld + c) : 0.f;
            Bs[r][lane] = (rb < m && c < c_end) ? __ldg(X + (int64_t)rb * ld + c) : 0.f;
        }
        __syncthreads();
        float part[4][4];
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) part[a][b] = 0.f;
#pragma unroll
        for (int k = 0; k < kGK; ++k) {
            float av[4], bv[4];
#pragma unroll
            for (int a = 0; a < 4; ++a) av[a] = As[ty + 16 * a][k];
#pragma unroll
            for (int b = 0; b < 4; ++b) bv[b] = Bs[tx + 16 * b][k];
#pragma unroll
            for (int a = 0; a < 4; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) part[a][b] = fmaf(av[a], bv[b], part[a][b]);
        }
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int b = 0; b < 4; ++b) acc[a][b] += (double)part[a][b];
        __syncthreads();
    }

    double* out = partial + (int64_t)blockIdx.x * (kGT * kGT);
#pragma unroll
    for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) out[(ty + 16 * a) * kGT + (tx + 16 * b)] = acc[a][b];
}

// Gram entry (i <= j) = sum over slabs of the tile partials, in slab order
__global__ void gram_reduce_kernel(const double* __restrict__ partial, int m, int ntile, int nslab,
                                   double* __restrict__ gram) {
    const int64_t total = (int64_t)m * m;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int i = (int)(e / m), j = (int)(e - (int64_t)i * m);
        if (i > j) continue;
        const int bi = i / kGT, bj = j / kGT;
        const int pair = bi * ntile - bi * (bi - 1) / 2 + (bj - bi);
        const double* p = partial + (int64_t)pair * nslab * (kGT * kGT) + (i % kGT) * kGT + (j % kGT);
        double v = 0.0;
#pragma unroll 8
        for (int s = 0; s < nslab; ++s) v += p[(int64_t)s * (kGT * kGT)];
        gram[e] = v;
    }
}

// D_ij = G_ii + G_jj - 2 G_ij from the upper triangle; never negative; exact zero on the diagonal
__global__ void dist_from_gram_kernel(const double* __restrict__ gram, int m, double* __restrict__ D) {
    const int64_t total = (int64_t)m * m;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int i = (int)(e / m), j = (int)(e - (int64_t)i * m);
        if (i == j) { D[e] = 0.0; continue; }
        const int a = i < j ? i : j, b = i < j ? j : i;
        const double v = gram[(int64_t)a * m + a] + gram[(int64_t)b * m + b] - 2.0 * gram[(int64_t)a * m + b];
        D[e] = v > 0.0 ? v : 0.0;
    }
}

struct GramPlan {
    int ntile, npair, nslab;
    int64_t slab_cols;
};

GramPlan gram_plan(int m, int64_t d) {
    GramPlan g;
    g.ntile = (m + kGT - 1) / kGT;
    g.npair = g.ntile * (g.ntile + 1) / 2;
    int64_t want = (4 * kSMs + g.npair - 1) / g.npair;  // about 4 CTAs per SM in total
    int64_t max_slabs = ceil_div(d, kGK);
    g.nslab = (int)(want < max_slabs ? want : max_slabs);
    if (g.nslab < 1) g.nslab = 1;
    g.slab_cols = ceil_div(ceil_div(d, g.nslab), kGK) * kGK;
    g.nslab = (int)ceil_div(d, g.slab_cols);
    return g;
}

int direct_blocks(int64_t d) {
    int64_t b = ceil_div(d, (int64_t)kDirThreads * 2 * 8);  // at least ~8 column pairs per thread
    if (b > 4 * kSMs) b = 4 * kSMs;
    return (int)(b < 1 ? 1 : b);
}

template <int M>
detox_status launch_direct_partials(const float* X, int64_t ld, int64_t d, const int32_t* rows, double* partial,
                                    cudaStream_t s) {
    const int nb = direct_blocks(d);
    const uintptr_t addr = reinterpret_cast<uintptr_t>(X);
    if ((addr & 15u) == 0 && ld % 4 == 0) sqdist_direct_kernel<M, 4><<<nb, kDirThreads, 0, s>>>(X, ld, d, rows, partial);
    else if ((addr & 7u) == 0 && ld % 2 == 0) sqdist_direct_kernel<M, 2><<<nb, kDirThreads, 0, s>>>(X, ld, d, rows, partial);
    else sqdist_direct_kernel<M, 1><<<nb, kDirThreads, 0, s>>>(X, ld, d, rows, partial);
    return launch_status();
}

template <int M>
detox_status launch_direct(const float* X, int64_t ld, int64_t d, const int32_t* rows, double* D, double* partial,
                           cudaStream_t s) {
    const int nb = direct_blocks(d);
    detox_status st = launch_direct_partials<M>(X, ld, d, rows, partial, s);
    if (st != DETOX_OK) return st;
    sqdist_direct_reduce_kernel<<<(M * (M - 1) / 2 + 3) / 4, 128, 0, s>>>(partial, nb, M, D);
    return launch_status();
}

}  // namespace

size_t dist_ws_bytes(int m, int64_t d) {
    if (m <= 16) return align_up((size_t)direct_blocks(d) * (size_t)(m * (m - 1) / 2 + 1) * sizeof(double));
    GramPlan g = gram_plan(m, d);
    size_t simt = align_up((size_t)g.npair * g.nslab * kGT * kGT * sizeof(double)) + align_up((size_t)m * m * sizeof(double));
    size_t tc = m <= 256 ? tc_ws_bytes(m, d) : 0;
    return simt > tc ? simt : tc;
}

// 2 <= m <= 16: only the per-CTA pair partials (ws: [nblocks][m (m-1) / 2] fp64, pairs in row-major order of
// i < j); *nblocks says how many there are.
detox_status launch_sqdist_partials(const float* X, int64_t ld, int m, int64_t d, const int32_t* rows, void* ws,
                                    int* nblocks, cudaStream_t s) {
    double* partial = static_cast<double*>(ws);
    *nblocks = direct_blocks(d);
    switch (m) {
#define DETOX_CASE(M) \
    case M: return launch_direct_partials<M>(X, ld, d, rows, partial, s);
        DETOX_CASE(2) DETOX_CASE(3) DETOX_CASE(4) DETOX_CASE(5) DETOX_CASE(6) DETOX_CASE(7) DETOX_CASE(8)
        DETOX_CASE(9) DETOX_CASE(10) DETOX_CASE(11) DETOX_CASE(12) DETOX_CASE(13) DETOX_CASE(14) DETOX_CASE(15)
        DETOX_CASE(16)
#undef DETOX_CASE
        default: return DETOX_ERR_UNSUPPORTED;
    }
}

detox_status launch_sqdist(const float* X, int64_t ld, int m, int64_t d, const int32_t* rows, double* D, void* ws,
                           int* status, cudaStream_t s) {
    double* partial = static_cast<double*>(ws);
    if (rows && m > 16) return DETOX_ERR_UNSUPPORTED;   // only the direct kernel takes a row list
    switch (m) {
        case 1:
            return cudaMemsetAsync(D, 0, sizeof(double), s) == cudaSuccess ? DETOX_OK : DETOX_ERR_CUDA;
#define DETOX_CASE(M) \
    case M: return launch_direct<M>(X, ld, d, rows, D, partial, s);
        DETOX_CASE(2) DETOX_CASE(3) DETOX_CASE(4) DETOX_CASE(5) DETOX_CASE(6) DETOX_CASE(7) DETOX_CASE(8)
        DETOX_CASE(9) DETOX_CASE(10) DETOX_CASE(11) DETOX_CASE(12) DETOX_CASE(13) DETOX_CASE(14) DETOX_CASE(15)
        DETOX_CASE(16)
#undef DETOX_CASE
        default: break;
    }
    if (tc_supported(X, ld, m, d)) return launch_sqdist_tc(X, ld, m, d, D, ws, status, s);
    GramPlan g = gram_plan(m, d);
    double* gram = reinterpret_cast<double*>(static_cast<char*>(ws) +
                                             align_up((size_t)g.npair * g.nslab * kGT * kGT * sizeof(double)));
    gram_simt_kernel<<<g.npair * g.nslab, kGramThreads, 0, s>>>(X, ld, m, d, g.ntile, g.nslab, g.slab_cols, partial);
    detox_status st = launch_status();
    if (st != DETOX_OK) return st;
    gram_reduce_kernel<<<64, 256, 0, s>>>(partial, m, g.ntile, g.nslab, gram);
    if ((st = launch_status()) != DETOX_OK) return st;
    dist_from_gram_kernel<<<64, 256, 0, s>>>(gram, m, D);
    return launch_status();
}

}  // namespace detox
