// Choice of the centring rows for the tensor-core distance pass.
//
// The tensor-core path forms D_ij = |a_i|^2 + |a_j|^2 - 2 a_i.a_j from inner products, which loses accuracy when the
// rows share a large common vector (honest gradients of one loss at one model do): the three terms are then much
// larger than their difference, and the tensor cores' fp32 accumulation loses most on long sums of one sign.
// Distances do not change when one vector is subtracted from every row, so the pass may work on a_i = x_i - c with c
// in the middle of the rows; it forms c, column by column, as the mean of a few rows that are listed here.  The rows
// are found on a sample of the columns: squared distances between all rows over a few evenly spaced column blocks
// (formed as differences, so they are accurate whatever the rows share), then for every row the median of its
// distances to the others; the rows are ranked by that median and every s-th of the more central half is taken (so
// that a group of colluding rows that sit in the very middle cannot fill the list).  Centring is switched on only
// when the most central row is closer to the typical row than the origin is by a clear margin; rows that hover around
// zero are left as they are.
//
// Everything is deterministic: per-block partial sums are added in a fixed order and ties go to the lower index.
#include <math_constants.h>

#include "common.cuh"

namespace detox {

namespace {

constexpr int kPickThreads = 256;
constexpr int kMaxCentreRows = 16;   // as in the distance kernels

struct CentrePlan {
    int cols;      // columns per sampled block
    int nblk;      // sampled blocks
    int nsplit;    // CTAs per block (they share the pairs)
};

CentrePlan centre_plan(int m, int64_t d) {
    CentrePlan p;
    p.cols = 64;           // (the tensor-core path, the only user, has at most 256 rows: a tile is at most 66.5 KB)
    const int64_t avail = ceil_div(d, (int64_t)p.cols);
    p.nblk = 32;
    if (p.nblk > avail) p.nblk = (int)avail;
    const int64_t want = ceil_div((int64_t)m * m, 4 * kPickThreads);
    int64_t ns = (2 * kSMs) / p.nblk;
    if (ns > want) ns = want;
    p.nsplit = (int)(ns < 1 ? 1 : ns);
    return p;
}

struct CentreWs {
    float* part;        // [nblk][m*m]: entry i*m+j (i < j) = squared distance over the block; i*m+i = squared norm
    float* key;         // [m] median sample distance of row i to the others
    float* nrm;         // [m] sample squared norm
    unsigned* counter;  // [2] CTAs of the pick kernel / of the check kernel that have finished; behind them one float:
                        // the typical squared norm of a row as the sample predicts it for all d columns
};

CentreWs centre_carve(void* ws, int m, int nblk) {
    CentreWs w;
    char* p = static_cast<char*>(ws);
    w.part = reinterpret_cast<float*>(p);
    p += align_up((size_t)nblk * m * m * sizeof(float));
    w.key = reinterpret_cast<float*>(p);
    p += align_up((size_t)m * sizeof(float));
    w.nrm = reinterpret_cast<float*>(p);
    p += align_up((size_t)m * sizeof(float));
    w.counter = reinterpret_cast<unsigned*>(p);
    return w;
}

__device__ __forceinline__ float nan_to_inf(float v) { return v != v ? CUDART_INF_F : v; }

// grid (nblk, nsplit): block b covers columns [c0, c0 + cols), the blocks evenly spaced over d
__global__ void __launch_bounds__(kPickThreads)
centre_sample_kernel(const float* __restrict__ X, int64_t ld, int m, int64_t d, int cols, float* __restrict__ part,
                     unsigned* __restrict__ counter) {
    extern __shared__ float tile[];   // [m][cols + 1]
    const int b = blockIdx.x, nblk = gridDim.x;
    const int64_t nb_all = (d + cols - 1) / cols;
    const int64_t c0 = (nb_all * b / nblk) * cols;
    const int pitch = cols + 1;
    if (b == 0 && blockIdx.y == 0 && threadIdx.x == 0) counter[0] = counter[1] = 0u;   // for the kernels that follow
    for (int e = threadIdx.x; e < m * cols; e += kPickThreads) {
        const int r = e / cols, c = e - r * cols;
        const int64_t col = c0 + c;
        tile[r * pitch + c] = col < d ? X[(int64_t)r * ld + col] : 0.f;
    }
    __syncthreads();
    float* out = part + (int64_t)b * m * m;
    const int total = m * m;
    for (int e = blockIdx.y * kPickThreads + threadIdx.x; e < total; e += gridDim.y * kPickThreads) {
        const int i = e / m, j = e - i * m;
        if (j < i) continue;
        const float* ti = tile + i * pitch;
        const float* tj = tile + j * pitch;
        float s = 0.f;
        if (i == j) {
            for (int c = 0; c < cols; ++c) s = fmaf(ti[c], ti[c], s);
        } else {
            for (int c = 0; c < cols; ++c) {
                const float t = ti[c] - tj[c];
                s = fmaf(t, t, s);
            }
        }
        out[e] = s;
    }
}

// One CTA per row: the median of the row's sample distances to the other rows and its sample norm; the CTA that
// finishes last picks the row with the smallest median and decides whether centring pays.
__global__ void __launch_bounds__(kPickThreads)
centre_pick_kernel(const float* __restrict__ part, int nblk, int m, float scale, float* __restrict__ key,
                   float* __restrict__ nrm, unsigned* __restrict__ counter, int* __restrict__ centre) {
    extern __shared__ float rowv[];   // [m]
    __shared__ float s_val[kPickThreads];
    __shared__ int s_idx[kPickThreads];
    __shared__ bool s_last;
    const int i = blockIdx.x;
    const int64_t mm = (int64_t)m * m;
    for (int j = threadIdx.x; j < m; j += kPickThreads) {
        const int a = i < j ? i : j, b2 = i < j ? j : i;
        float v = 0.f;
        for (int b = 0; b < nblk; ++b) v += part[(int64_t)b * mm + (int64_t)a * m + b2];
        v = nan_to_inf(v);
        if (j == i) nrm[i] = v;
        rowv[j] = j == i ? CUDART_INF_F : v;
    }
    __syncthreads();
    const int h = (m - 2) / 2;   // middle of the m - 1 distances to the other rows
    for (int j = threadIdx.x; j < m; j += kPickThreads) {
        if (j == i) continue;
        const float v = rowv[j];
        int rank = 0;
        for (int k = 0; k < m; ++k) {
            if (k == i) continue;
            const float u = rowv[k];
            rank += (u < v || (u == v && k < j)) ? 1 : 0;
        }
        if (rank == h) key[i] = v;
    }
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_last = atomicAdd(counter, 1u) == (unsigned)(m - 1);
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // smallest key, ties to the lower row
    float best = CUDART_INF_F;
    int arg = 0x7fffffff;
    for (int r = threadIdx.x; r < m; r += kPickThreads) {
        const float v = __ldcg(key + r);
        if (v < best || (v == best && r < arg)) { best = v; arg = r; }
    }
    s_val[threadIdx.x] = best;
    s_idx[threadIdx.x] = arg;
    __syncthreads();
    for (int o = kPickThreads / 2; o > 0; o >>= 1) {
        if (threadIdx.x < o) {
            const float v = s_val[threadIdx.x + o];
            const int r = s_idx[threadIdx.x + o];
            if (v < s_val[threadIdx.x] || (v == s_val[threadIdx.x] && r < s_idx[threadIdx.x])) {
                s_val[threadIdx.x] = v;
                s_idx[threadIdx.x] = r;
            }
        }
        __syncthreads();
    }
    const float best_key = s_val[0];
    __syncthreads();
    // median of the sample norms (rank counting again; rowv is free now)
    for (int r = threadIdx.x; r < m; r += kPickThreads) rowv[r] = __ldcg(nrm + r);
    __syncthreads();
    const int hm = (m - 1) / 2;
    for (int r = threadIdx.x; r < m; r += kPickThreads) {
        const float v = rowv[r];
        int rank = 0;
        for (int k = 0; k < m; ++k) {
            const float u = rowv[k];
            rank += (u < v || (u == v && k < r)) ? 1 : 0;
        }
        if (rank == hm) s_val[0] = v;
    }
    __syncthreads();
    // on when the most central row's typical distance to the others is clearly below what two rows that hover around
    // zero have (twice the typical squared norm)
    const int want = m / 2 < kMaxCentreRows ? m / 2 : kMaxCentreRows;
    const bool on = best_key < 1.5f * s_val[0] && want >= 1;
    // the rows at ranks 0, s, 2s, ... of the ordering by median distance, inside its more central half
    const int stride = (m / 2) / (want > 0 ? want : 1) > 1 ? (m / 2) / want : 1;
    for (int r = threadIdx.x; r < m; r += kPickThreads) rowv[r] = __ldcg(key + r);
    __syncthreads();
    for (int r = threadIdx.x; r < m; r += kPickThreads) {
        const float v = rowv[r];
        int rank = 0;
        for (int k = 0; k < m; ++k) {
            const float u = rowv[k];
            rank += (u < v || (u == v && k < r)) ? 1 : 0;
        }
        if (rank % stride == 0 && rank / stride < want) centre[2 + rank / stride] = r;
    }
    if (threadIdx.x == 0) {
        centre[0] = on ? want : 0;
        *reinterpret_cast<float*>(counter + 2) = s_val[0] * scale;   // for the check after the pass
    }
}

// After the distance pass: did the subtraction leave the rows small?  The listed rows were chosen on a sample of the
// columns; a row that is central there and holds huge values elsewhere would, once subtracted, swamp the differences
// between the other rows.  `norms` holds, per output slot and group of transform warps, every row's exact squared
// norm after the subtraction.  One CTA per row adds its shares up; the last one takes the median over the rows and
// compares it with what the sample predicted for the rows as they came.  If the typical row is more than 16 times
// larger than that, the centring is withdrawn (centre[0] = 0) and *redo = 1 asks for the pass to be repeated without it.
constexpr float kCentreSlack = 16.f;
__global__ void __launch_bounds__(128)
centre_check_kernel(const float* __restrict__ norms, int nshares, int m, float* __restrict__ na,
                    unsigned* __restrict__ counter, int* __restrict__ centre, int* __restrict__ redo) {
    __shared__ double red[4];
    __shared__ bool s_last;
    const int i = blockIdx.x;
    if (*centre <= 0) {
        if (i == 0 && threadIdx.x == 0) *redo = 0;
        return;
    }
    double a = 0.0;
    for (int s = threadIdx.x; s < nshares; s += 128) a += (double)norms[(int64_t)s * m + i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = a;
    __syncthreads();
    if (threadIdx.x == 0) {
        na[i] = nan_to_inf((float)(red[0] + red[1] + red[2] + red[3]));
        __threadfence();
        s_last = atomicAdd(counter + 1, 1u) == (unsigned)(m - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    // median by rank counting (m <= 256 on this path: two rows per thread at most)
    const int hm = (m - 1) / 2;
    const float ref = *reinterpret_cast<const float*>(counter + 2);
    for (int r = threadIdx.x; r < m; r += 128) {
        const float mine = __ldcg(na + r);
        int rank = 0;
        for (int k = 0; k < m; ++k) {
            const float u = __ldcg(na + k);
            rank += (u < mine || (u == mine && k < r)) ? 1 : 0;
        }
        if (rank == hm) {
            const bool keep = mine <= kCentreSlack * ref;
            *redo = keep ? 0 : 1;
            if (!keep) *centre = 0;
            counter[1] = 0u;
        }
    }
}

}  // namespace

size_t centre_ws_bytes(int m, int64_t d) {
    const CentrePlan p = centre_plan(m, d);
    return align_up((size_t)p.nblk * m * m * sizeof(float)) + 2 * align_up((size_t)m * sizeof(float)) + 256;   // counters, float
}

detox_status launch_pick_centre(const float* X, int64_t ld, int m, int64_t d, void* ws, int* centre, cudaStream_t s) {
    const CentrePlan p = centre_plan(m, d);
    CentreWs w = centre_carve(ws, m, p.nblk);
    const size_t smem = (size_t)m * (p.cols + 1) * sizeof(float);
    if (cudaFuncSetAttribute(centre_sample_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return DETOX_ERR_CUDA;
    centre_sample_kernel<<<dim3((unsigned)p.nblk, (unsigned)p.nsplit), kPickThreads, smem, s>>>(X, ld, m, d, p.cols, w.part,
                                                                                          w.counter);
    detox_status st = launch_status();
    if (st != DETOX_OK) return st;
    // the sample's squared norms are scaled up to all d columns for the check after the pass
    const int64_t sampled = (int64_t)p.nblk * p.cols < d ? (int64_t)p.nblk * p.cols : d;
    const float scale = (float)((double)d / (double)sampled);
    centre_pick_kernel<<<m, kPickThreads, (size_t)m * sizeof(float), s>>>(w.part, p.nblk, m, scale, w.key, w.nrm, w.counter,
                                                                         centre);
    return launch_status();
}

detox_status launch_check_centre(const float* norms, int nshares, int m, void* ws, int64_t d, int* centre, int* redo,
                                 cudaStream_t s) {
    const CentrePlan p = centre_plan(m, d);
    CentreWs w = centre_carve(ws, m, p.nblk);
    // the pick kernel is done with `key`: it holds the exact norms now; the second counter word was cleared by the
    // sample kernel
    centre_check_kernel<<<m, 128, 0, s>>>(norms, nshares, m, w.key, w.counter, centre, redo);
    return launch_status();
}

}  // namespace detox
