// Pairwise squared distances between m rows (the O(p^2 d) part of Krum-type aggregators, Section 4,
// "Improved speed").  Output: D, m x m fp64, symmetric, zero diagonal.
//
//   m <= 16 : differences are formed directly, (x_i - x_j)^2, with one fp32 accumulator per pair in
//             registers; HBM-bound (m*d*4 bytes read once).  From 9 rows on, long 16-byte aligned rows are
//             streamed through shared memory with bulk copies so that the copies overlap the arithmetic.
//   16 < m <= 256 with 16-byte aligned rows: the tensor-core Gram of gram_tc.cu.
//   otherwise : CUDA-core tiles of squared differences over K-slabs (rows that are not 16-byte aligned, more than
//             256 rows).
// All write per-CTA partial sums that a second kernel adds in a fixed order in fp64, so results
// are deterministic and bitwise-equal rows get bitwise-equal distances.
#include "common.cuh"
#include "mbarrier.cuh"

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

// ------------------------------------------------------------------ 9 <= m <= 16, long rows: staged differences
//
// With 36 to 120 pair accumulators a thread has no registers left to keep the next columns in flight, and the
// kernel above waits out the memory latency between its steps.  Here tiles of 1024 columns of all rows stream
// into a ring of shared-memory stages with bulk copies (one per row and tile, issued by the first warp a few tiles
// ahead of the arithmetic) while all eight warps form the differences from the stage that has landed.  One
// persistent CTA per SM; eight warps, so that a thread may keep up to 255 registers.
constexpr int kStgWarps = 8;
constexpr int kStgThreads = kStgWarps * 32;
constexpr int kStgPieces = kStgThreads;                   // 16-byte pieces per row and tile: one per thread
constexpr int64_t kStgMinCols = (int64_t)kSMs * kStgPieces * 4 * 4;   // at least four tiles per CTA

__host__ __device__ constexpr int stg_stages(int M) { return M <= 12 ? 4 : 3; }   // 16 rows x 4 KB x 3 = 192 KB

// Two fp32 differences in one instruction (same rounding as the scalar subtraction).
__device__ __forceinline__ uint64_t sub_f32x2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

__device__ __forceinline__ void bulk_copy_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// Rows must be 16-byte aligned (base and pitch).  `status` is cleared by the first CTA (if clear_status) and set to
// DETOX_ERR_TIMEOUT when a bounded wait runs out; the partials of that CTA are then NaN.
template <int M>
__global__ void __launch_bounds__(kStgThreads, 1)
sqdist_staged_kernel(const float* __restrict__ X, int64_t ld, int64_t d, const int32_t* __restrict__ rows,
                     double* __restrict__ partial, int* __restrict__ status, int clear_status) {
    constexpr int NP = M * (M - 1) / 2;
    constexpr int kStages = stg_stages(M), kAhead = kStages - 1;
    extern __shared__ __align__(128) uint8_t stage_mem[];      // [kStages][M][kStgPieces] pieces of 16 bytes
    __shared__ uint64_t full[kStages], empty[kStages];
    __shared__ int64_t roff[M];                                // element offset of row i, -1 for a zero row
    __shared__ int abort_word;
    __shared__ double red[kStgWarps][NP];
    volatile int* abort_flag = &abort_word;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&full[s], 1);
            mbar_init(&empty[s], kStgWarps);
        }
        abort_word = 0;
        mbar_fence_init();
        if (blockIdx.x == 0 && clear_status) *status = 0;
    }
    if (tid < M) {
        const int r = rows ? rows[tid] : tid;      // a negative entry of the row list stands for a zero row
        roff[tid] = r < 0 ? -1 : (int64_t)r * ld;
    }
    __syncthreads();
    uint32_t zero_rows = 0;                         // bit i: row i is a zero row
#pragma unroll
    for (int i = 0; i < M; ++i) zero_rows |= roff[i] < 0 ? 1u << i : 0u;
    const int nreal = M - __popc(zero_rows);

    const int64_t npiece_all = d / 4;              // whole 16-byte pieces per row; the last d % 4 columns come below
    const int64_t ntiles = (npiece_all + kStgPieces - 1) / kStgPieces;
    // this CTA's tiles: b, b + G, ...; `it` counts them; tile `it` goes through stage it % kStages
    const int64_t my_tiles = ntiles > blockIdx.x ? (ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    constexpr uint32_t kRowBytes = kStgPieces * 16u, kStageBytes = M * kRowBytes;

    // first warp: copy this CTA's tile number `it` (lane i takes row i) once its stage has been read
    auto issue = [&](int64_t it) -> bool {
        const int s = (int)(it % kStages);
        const uint32_t ph = (uint32_t)(it / kStages) & 1u;
        int ok = 1;
        if (lane == 0) ok = mbar_wait(&empty[s], ph ^ 1u, abort_flag, status) ? 1 : 0;
        if (!__shfl_sync(0xffffffffu, ok, 0)) return false;
        const int64_t t = blockIdx.x + it * gridDim.x;
        const int64_t left = npiece_all - t * kStgPieces;
        const uint32_t bytes = (uint32_t)(left < kStgPieces ? left : kStgPieces) * 16u;
        if (lane == 0) mbar_expect_tx(&full[s], bytes * (uint32_t)nreal);
        __syncwarp();
        if (lane < M && roff[lane] >= 0)
            bulk_copy_g2s(stage_mem + (size_t)s * kStageBytes + (size_t)lane * kRowBytes,
                          X + roff[lane] + t * (int64_t)(kStgPieces * 4), bytes, &full[s]);
        return true;
    };

    float acc[NP];
#pragma unroll
    for (int p = 0; p < NP; ++p) acc[p] = 0.f;

    bool alive = true;
    if (warp == 0)
        for (int64_t it = 0; it < kAhead && it < my_tiles && alive; ++it) alive = issue(it);
    int s = 0;
    uint32_t ph = 0;
    for (int64_t it = 0; it < my_tiles && alive; ++it) {
        if (warp == 0 && it + kAhead < my_tiles) alive = issue(it + kAhead);
        if (!alive || !mbar_wait(&full[s], ph, abort_flag, status)) break;
        const int64_t t = blockIdx.x + it * gridDim.x;
        if (t * kStgPieces + tid < npiece_all) {
            const uint8_t* src = stage_mem + (size_t)s * kStageBytes + (size_t)tid * 16u;
            ulonglong2 v[M];                        // four columns of every row as two packed pairs
#pragma unroll
            for (int i = 0; i < M; ++i) {
                v[i] = make_ulonglong2(0ull, 0ull);
                if (!((zero_rows >> i) & 1u)) v[i] = *reinterpret_cast<const ulonglong2*>(src + (size_t)i * kRowBytes);
            }
            int p = 0;
#pragma unroll
            for (int i = 0; i < M; ++i)
#pragma unroll
                for (int j = i + 1; j < M; ++j, ++p) {
                    const uint64_t d01 = sub_f32x2(v[i].x, v[j].x), d23 = sub_f32x2(v[i].y, v[j].y);
                    const float a0 = __uint_as_float((uint32_t)d01), a1 = __uint_as_float((uint32_t)(d01 >> 32));
                    const float a2 = __uint_as_float((uint32_t)d23), a3 = __uint_as_float((uint32_t)(d23 >> 32));
                    acc[p] = fmaf(a3, a3, fmaf(a2, a2, fmaf(a1, a1, fmaf(a0, a0, acc[p]))));
                }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[s]);   // one arrival per warp: the stage may be refilled
        if (++s == kStages) { s = 0; ph ^= 1u; }
    }
    if (blockIdx.x == 0 && tid == 0) {
        for (int64_t c = npiece_all * 4; c < d; ++c) {
            int p = 0;
#pragma unroll
            for (int i = 0; i < M; ++i)
#pragma unroll
                for (int j = i + 1; j < M; ++j, ++p) {
                    const float a = (roff[i] < 0 ? 0.f : X[roff[i] + c]) - (roff[j] < 0 ? 0.f : X[roff[j] + c]);
                    acc[p] = fmaf(a, a, acc[p]);
                }
        }
    }
    // block reduction in fp64, fixed order
#pragma unroll
    for (int p = 0; p < NP; ++p) {
        double v = (double)acc[p];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
        if (lane == 0) red[warp][p] = v;
    }
    __syncthreads();
    const bool bad = *abort_flag != 0;
    // a CTA that gave up may still have copies in flight: give them a bounded time to land before it goes away
    if (bad) {
        for (int i = 0; i < 64; ++i) __nanosleep(2000);
        __syncthreads();
    }
    for (int p = tid; p < NP; p += kStgThreads) {
        double v = 0.0;
#pragma unroll
        for (int w = 0; w < kStgWarps; ++w) v += red[w][p];
        partial[(int64_t)blockIdx.x * NP + p] = bad ? __longlong_as_double(0x7ff8000000000000LL) : v;
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
            D[i * m + j] = v;   // may be NaN (two rows with non-finite entries); the ranking kernels take NaN as +Inf
            D[j * m + i] = v;
        }
    }
    if (blockIdx.x == 0)
        for (int i = threadIdx.x; i < m; i += blockDim.x) D[i * m + i] = 0.0;
}

// ------------------------------------------------------------------ m > 16: CUDA-core tiles of squared differences
//
// Differences are formed before squaring, as in the small kernels: nothing cancels when the rows share a large
// common vector, and bitwise-equal rows are at distance exactly zero.

constexpr int kGT = 64;          // output tile edge
constexpr int kGK = 32;          // columns per shared-memory step
constexpr int kGramThreads = 256;  // 16 x 16 threads, 4 x 4 outputs each

__global__ void __launch_bounds__(kGramThreads)
sqdist_simt_kernel(const float* __restrict__ X, int64_t ld, int m, int64_t d, int ntile, int nslab,
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
                for (int b = 0; b < 4; ++b) {
                    const float t = av[a] - bv[b];
                    part[a][b] = fmaf(t, t, part[a][b]);
                }
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

// D_ij (i < j) = sum over slabs of the tile partials, in slab order; mirrored; zero diagonal
__global__ void sqdist_simt_reduce_kernel(const double* __restrict__ partial, int m, int ntile, int nslab,
                                          double* __restrict__ D) {
    const int64_t total = (int64_t)m * m;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int i = (int)(e / m), j = (int)(e - (int64_t)i * m);
        if (i > j) continue;
        if (i == j) { D[e] = 0.0; continue; }
        const int bi = i / kGT, bj = j / kGT;
        const int pair = bi * ntile - bi * (bi - 1) / 2 + (bj - bi);
        const double* p = partial + (int64_t)pair * nslab * (kGT * kGT) + (i % kGT) * kGT + (j % kGT);
        double v = 0.0;
#pragma unroll 8
        for (int s = 0; s < nslab; ++s) v += p[(int64_t)s * (kGT * kGT)];
        D[e] = v;   // may be NaN (two rows with non-finite entries); the ranking kernels take NaN as +Inf
        D[(int64_t)j * m + i] = v;
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

// 9 to 16 rows that are 16-byte aligned and long enough take the staged kernel (one CTA per SM).
bool use_staged(int m, const float* X, int64_t ld, int64_t d) {
    return m >= 9 && m <= 16 && aligned16(X) && ld % 4 == 0 && d >= kStgMinCols;
}

// Launches the pair-partial kernel for M rows; *nblocks = how many partial vectors it writes.  `status` (device)
// is cleared and used by the staged kernel only.
template <int M>
detox_status launch_direct_partials(const float* X, int64_t ld, int64_t d, const int32_t* rows, double* partial,
                                    int* status, bool clear_status, int* nblocks, cudaStream_t s) {
    if constexpr (M >= 9) {
        if (use_staged(M, X, ld, d)) {
            constexpr size_t smem = (size_t)stg_stages(M) * M * kStgPieces * 16;
            if (cudaFuncSetAttribute(sqdist_staged_kernel<M>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
                cudaSuccess)
                return DETOX_ERR_CUDA;
            *nblocks = kSMs;
            sqdist_staged_kernel<M><<<kSMs, kStgThreads, smem, s>>>(X, ld, d, rows, partial, status, clear_status ? 1 : 0);
            return launch_status();
        }
    }
    const int nb = direct_blocks(d);
    *nblocks = nb;
    const uintptr_t addr = reinterpret_cast<uintptr_t>(X);
    if ((addr & 15u) == 0 && ld % 4 == 0) sqdist_direct_kernel<M, 4><<<nb, kDirThreads, 0, s>>>(X, ld, d, rows, partial);
    else if ((addr & 7u) == 0 && ld % 2 == 0) sqdist_direct_kernel<M, 2><<<nb, kDirThreads, 0, s>>>(X, ld, d, rows, partial);
    else sqdist_direct_kernel<M, 1><<<nb, kDirThreads, 0, s>>>(X, ld, d, rows, partial);
    return launch_status();
}

template <int M>
detox_status launch_direct(const float* X, int64_t ld, int64_t d, const int32_t* rows, double* D, double* partial,
                           int* status, cudaStream_t s) {
    int nb = 0;
    detox_status st = launch_direct_partials<M>(X, ld, d, rows, partial, status, false, &nb, s);   // the caller cleared it
    if (st != DETOX_OK) return st;
    sqdist_direct_reduce_kernel<<<(M * (M - 1) / 2 + 3) / 4, 128, 0, s>>>(partial, nb, M, D);
    return launch_status();
}

}  // namespace

size_t dist_ws_bytes(int m, int64_t d) {
    if (m <= 16) return align_up((size_t)direct_blocks(d) * (size_t)(m * (m - 1) / 2 + 1) * sizeof(double));
    GramPlan g = gram_plan(m, d);
    size_t simt = align_up((size_t)g.npair * g.nslab * kGT * kGT * sizeof(double));
    size_t tc = m <= 256 ? tc_ws_bytes(m, d) : 0;
    return simt > tc ? simt : tc;
}

bool sqdist_partials_use_status(int m, const float* X, int64_t ld, int64_t d) { return use_staged(m, X, ld, d); }

// 2 <= m <= 16: only the per-CTA pair partials (ws: [nblocks][m (m-1) / 2] fp64, pairs in row-major order of
// i < j); *nblocks says how many there are.  When sqdist_partials_use_status() holds, the kernel clears the device
// status word itself and sets it to DETOX_ERR_TIMEOUT if a bounded wait runs out (its partials are then NaN).
detox_status launch_sqdist_partials(const float* X, int64_t ld, int m, int64_t d, const int32_t* rows, void* ws,
                                    int* status, bool clear_status, int* nblocks, cudaStream_t s) {
    double* partial = static_cast<double*>(ws);
    switch (m) {
#define DETOX_CASE(M) \
    case M: return launch_direct_partials<M>(X, ld, d, rows, partial, status, clear_status, nblocks, s);
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
    case M: return launch_direct<M>(X, ld, d, rows, D, partial, status, s);
        DETOX_CASE(2) DETOX_CASE(3) DETOX_CASE(4) DETOX_CASE(5) DETOX_CASE(6) DETOX_CASE(7) DETOX_CASE(8)
        DETOX_CASE(9) DETOX_CASE(10) DETOX_CASE(11) DETOX_CASE(12) DETOX_CASE(13) DETOX_CASE(14) DETOX_CASE(15)
        DETOX_CASE(16)
#undef DETOX_CASE
        default: break;
    }
    if (tc_supported(X, ld, m, d)) return launch_sqdist_tc(X, ld, m, d, D, ws, status, s);
    GramPlan g = gram_plan(m, d);
    sqdist_simt_kernel<<<g.npair * g.nslab, kGramThreads, 0, s>>>(X, ld, m, d, g.ntile, g.nslab, g.slab_cols, partial);
    detox_status st = launch_status();
    if (st != DETOX_OK) return st;
    sqdist_simt_reduce_kernel<<<64, 256, 0, s>>>(partial, m, g.ntile, g.nslab, D);
    return launch_status();
}

}  // namespace detox
