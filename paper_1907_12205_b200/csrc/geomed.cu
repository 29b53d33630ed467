// Geometric median of m <= 32 rows by Weiszfeld's iteration (one of the A_1 choices analysed in Section 4,
// Theorem 4): y <- sum_j w_j x_j / sum_j w_j with w_j = 1 / max(||x_j - y||, eps), started at the mean.
//
// One streaming pass per iteration: a thread forms y_new on its 16-byte piece from the current weights,
// writes it, and at once adds its share of ||x_j - y_new||^2 for the next weights (the rows are
// re-read from L1).  Per-CTA partial sums are added in fp64 in a fixed order by one small kernel,
// so the iteration is deterministic.  HBM-bound: (m + 1) * d * 4 bytes per iteration.
#include "common.cuh"

namespace detox {

namespace {

constexpr int kGmMaxRows = 32;
constexpr int kGmThreads = 256;

struct GmWs {
    double* partial;   // [blocks][32]
    float* weight;     // [32] normalised weights w_j / sum w
    size_t total;
};

GmWs gm_ws(void* ws, int64_t d) {
    GmWs w;
    char* p = static_cast<char*>(ws);
    const size_t blocks = (size_t)ceil_div(d, kGmThreads);   // upper bound (scalar path)
    w.partial = reinterpret_cast<double*>(p);
    w.weight = reinterpret_cast<float*>(p + align_up(blocks * kGmMaxRows * sizeof(double)));
    w.total = align_up(blocks * kGmMaxRows * sizeof(double)) + 256;
    return w;
}

__global__ void gm_unit_weights_kernel(int m, float* __restrict__ weight) {
    if (threadIdx.x < kGmMaxRows) weight[threadIdx.x] = threadIdx.x < m ? 1.0f / (float)m : 0.f;
}

template <int VEC>
__global__ void __launch_bounds__(kGmThreads)
gm_step_kernel(const float* __restrict__ X, int64_t ld, int m, int64_t d, const float* __restrict__ weight,
               float* __restrict__ y, double* __restrict__ partial) {
    __shared__ float w[kGmMaxRows];
    __shared__ double red[kGmThreads / 32][kGmMaxRows];
    if (threadIdx.x < kGmMaxRows) w[threadIdx.x] = weight[threadIdx.x];
    __syncthreads();

    const int64_t col = ((int64_t)blockIdx.x * kGmThreads + threadIdx.x) * VEC;
    const int64_t left = d - col;
    const int valid = left >= VEC ? VEC : (left > 0 ? (int)left : 0);
    float yv[VEC];
#pragma unroll
    for (int c = 0; c < VEC; ++c) yv[c] = 0.f;
    float dist[kGmMaxRows];
#pragma unroll
    for (int j = 0; j < kGmMaxRows; ++j) dist[j] = 0.f;

    if (valid > 0) {
        for (int j = 0; j < m; ++j) {
            const float* p = X + (int64_t)j * ld + col;
            if (VEC == 4 && valid == 4) {
                const float4 x = __ldg(reinterpret_cast<const float4*>(p));
                yv[0] = fmaf(w[j], x.x, yv[0]); yv[1 % VEC] = fmaf(w[j], x.y, yv[1 % VEC]);
                yv[2 % VEC] = fmaf(w[j], x.z, yv[2 % VEC]); yv[3 % VEC] = fmaf(w[j], x.w, yv[3 % VEC]);
            } else {
#pragma unroll
                for (int c = 0; c < VEC; ++c)
                    if (c < valid) yv[c] = fmaf(w[j], __ldg(p + c), yv[c]);
            }
        }
#pragma unroll
        for (int c = 0; c < VEC; ++c)
            if (c < valid) y[col + c] = yv[c];
#pragma unroll
        for (int j = 0; j < kGmMaxRows; ++j) {
            if (j < m) {
                const float* p = X + (int64_t)j * ld + col;
                float acc = 0.f;
#pragma unroll
                for (int c = 0; c < VEC; ++c)
                    if (c < valid) {
                        const float t = __ldg(p + c) - yv[c];
                        acc = fmaf(t, t, acc);
                    }
                dist[j] = acc;
            }
        }
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int j = 0; j < kGmMaxRows; ++j) {
        double v = (double)dist[j];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
        if (lane == 0) red[warp][j] = v;
    }
    __syncthreads();
    if (threadIdx.x < kGmMaxRows) {
        double v = 0.0;
#pragma unroll
        for (int k = 0; k < kGmThreads / 32; ++k) v += red[k][threadIdx.x];
        partial[(int64_t)blockIdx.x * kGmMaxRows + threadIdx.x] = v;
    }
}

// One warp per row: squared distance = sum of the CTA partials (fixed order); then the Weiszfeld weights.
__global__ void __launch_bounds__(kGmMaxRows * 32)
gm_weights_kernel(const double* __restrict__ partial, int nblocks, int m, float eps, float* __restrict__ weight) {
    __shared__ double wj[kGmMaxRows];
    const int j = threadIdx.x >> 5, lane = threadIdx.x & 31;
    double v = 0.0;
    if (j < m)
        for (int b = lane; b < nblocks; b += 32) v += partial[(int64_t)b * kGmMaxRows + j];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
    if (lane == 0) {
        const double dist = sqrt(v);
        wj[j] = j < m ? 1.0 / (dist > (double)eps ? dist : (double)eps) : 0.0;
    }
    __syncthreads();
    if (threadIdx.x < kGmMaxRows) {
        double tot = 0.0;
        for (int k = 0; k < m; ++k) tot += wj[k];
        weight[threadIdx.x] = (float)(wj[threadIdx.x] / tot);
    }
}

}  // namespace

size_t geomed_ws_bytes(int64_t d) { return gm_ws(nullptr, d).total; }

detox_status launch_geometric_median(const float* X, int64_t ld, int m, int64_t d, int iters, float eps, float* out,
                                     void* ws, cudaStream_t s) {
    if (m > kGmMaxRows) return DETOX_ERR_UNSUPPORTED;
    GmWs w = gm_ws(ws, d);
    const bool vec = aligned16(X) && aligned16(out) && ld % 4 == 0;
    const int nblocks = (int)ceil_div(d, (int64_t)kGmThreads * (vec ? 4 : 1));
    gm_unit_weights_kernel<<<1, 32, 0, s>>>(m, w.weight);
    detox_status st = launch_status();
    for (int t = 0; t <= iters && st == DETOX_OK; ++t) {     // step 0 gives the mean and the distances to it
        if (vec) gm_step_kernel<4><<<nblocks, kGmThreads, 0, s>>>(X, ld, m, d, w.weight, out, w.partial);
        else gm_step_kernel<1><<<nblocks, kGmThreads, 0, s>>>(X, ld, m, d, w.weight, out, w.partial);
        if ((st = launch_status()) != DETOX_OK) break;
        if (t < iters) {
            gm_weights_kernel<<<1, kGmMaxRows * 32, 0, s>>>(w.partial, nblocks, m, eps, w.weight);
            st = launch_status();
        }
    }
    return st;
}

}  // namespace detox
