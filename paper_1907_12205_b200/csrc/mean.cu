// Streaming means: A_0 = mean over each vote group (Algorithm 2, step 3) and the average of the rows
// selected by Multi-Krum.  One pass: k*d*4 bytes read, d*4 bytes written per output row.
// The same kernels, with SIGN set, give the coordinate-wise sign majority used with signSGD
// (Section 5.2, setup 4): sign(sum_i sign(x_i)), in {-1, 0, +1}.
#include "common.cuh"

namespace detox {

namespace {

constexpr int kMeanThreads = 256;

template <int VEC>
struct Acc;
template <>
struct Acc<4> {
    float4 a;
    __device__ __forceinline__ void zero() { a = make_float4(0.f, 0.f, 0.f, 0.f); }
    __device__ __forceinline__ void add(const float4& v) { a.x += v.x; a.y += v.y; a.z += v.z; a.w += v.w; }
    __device__ __forceinline__ void div(float k) { a.x /= k; a.y /= k; a.z /= k; a.w /= k; }
};

// Row r of X at column `col`; a negative r stands for a zero row.
__device__ __forceinline__ const float* row_ptr(const float* X, int64_t ld, int r, int64_t col) {
    return X + (int64_t)(r < 0 ? 0 : r) * ld + col;
}
__device__ __forceinline__ float4 mask_piece(float4 v, int r) {
    return r < 0 ? make_float4(0.f, 0.f, 0.f, 0.f) : v;
}

__device__ __forceinline__ float4 load_piece(const float* p, int valid) {
    if (valid >= 4) return ld_stream_f4(p);
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (valid > 0) v.x = __ldcs(p);
    if (valid > 1) v.y = __ldcs(p + 1);
    if (valid > 2) v.z = __ldcs(p + 2);
    return v;
}
__device__ __forceinline__ void store_piece(float* p, const float4& v, int valid) {
    if (valid >= 4) { st_stream_f4(p, v); return; }
    if (valid > 0) p[0] = v.x;
    if (valid > 1) p[1] = v.y;
    if (valid > 2) p[2] = v.z;
}

__device__ __forceinline__ float sgn(float v) { return (float)((v > 0.f) - (v < 0.f)); }   // sgn(NaN) = 0
__device__ __forceinline__ float4 sgn4(const float4& v) { return make_float4(sgn(v.x), sgn(v.y), sgn(v.z), sgn(v.w)); }

// Rows are added in list order, four loads in flight at a time.
template <int VEC, bool SIGN, typename RowOf>
__device__ __forceinline__ void mean_columns(const float* __restrict__ X, int64_t ld, int64_t d, int k,
                                             RowOf row_of, float* __restrict__ out) {
    const int64_t col = ((int64_t)blockIdx.x * kMeanThreads + threadIdx.x) * VEC;
    if (col >= d) return;
    if (VEC == 4) {
        const int64_t left = d - col;
        const int valid = left >= 4 ? 4 : (int)left;
        Acc<4> acc;
        acc.zero();
        int t = 0;
        for (; t + 4 <= k; t += 4) {
            const int r0 = row_of(t), r1 = row_of(t + 1), r2 = row_of(t + 2), r3 = row_of(t + 3);
            float4 v0 = load_piece(row_ptr(X, ld, r0, col), valid);
            float4 v1 = load_piece(row_ptr(X, ld, r1, col), valid);
            float4 v2 = load_piece(row_ptr(X, ld, r2, col), valid);
            float4 v3 = load_piece(row_ptr(X, ld, r3, col), valid);
            v0 = mask_piece(v0, r0); v1 = mask_piece(v1, r1); v2 = mask_piece(v2, r2); v3 = mask_piece(v3, r3);
            if (SIGN) { v0 = sgn4(v0); v1 = sgn4(v1); v2 = sgn4(v2); v3 = sgn4(v3); }
            acc.add(v0); acc.add(v1); acc.add(v2); acc.add(v3);
        }
        for (; t < k; ++t) {
            const int r = row_of(t);
            float4 v = mask_piece(load_piece(row_ptr(X, ld, r, col), valid), r);
            if (SIGN) v = sgn4(v);
            acc.add(v);
        }
        if (SIGN) acc.a = sgn4(acc.a);
        else acc.div((float)k);
        store_piece(out + col, acc.a, valid);
    } else {
        float acc = 0.f;
        for (int t = 0; t < k; ++t) {
            const int r = row_of(t);
            float v = __ldcs(row_ptr(X, ld, r, col));
            v = r < 0 ? 0.f : v;
            acc += SIGN ? sgn(v) : v;
        }
        out[col] = SIGN ? sgn(acc) : acc / (float)k;
    }
}

template <int VEC, bool SIGN>
__global__ void __launch_bounds__(kMeanThreads)
hier_mean_kernel(const float* __restrict__ Z, int64_t ldz, int64_t d, const __grid_constant__ SetTable sets,
                 float* __restrict__ M, int64_t ldm) {
    const int s = blockIdx.y;
    const int b = sets.offset[s];
    const int k = sets.offset[s + 1] - b;
    mean_columns<VEC, SIGN>(Z, ldz, d, k, [&](int t) { return (int)sets.member[b + t]; }, M + (int64_t)s * ldm);
}

template <int VEC, bool SIGN>
__global__ void __launch_bounds__(kMeanThreads)
mean_rows_kernel(const float* __restrict__ X, int64_t ld, int64_t d, const int32_t* __restrict__ rows, int k,
                 float* __restrict__ out) {
    if (rows)
        mean_columns<VEC, SIGN>(X, ld, d, k, [&](int t) { return rows[t]; }, out);
    else
        mean_columns<VEC, SIGN>(X, ld, d, k, [](int t) { return t; }, out);
}

}  // namespace

detox_status launch_hier_mean(const float* Z, int64_t ldz, int64_t d, const SetTable& sets, int S, float* M,
                              int64_t ldm, cudaStream_t s, bool sign) {
    const bool vec = aligned16(Z) && aligned16(M) && ldz % 4 == 0 && ldm % 4 == 0;
    const int vecw = vec ? 4 : 1;
    int64_t bx = ceil_div(d, (int64_t)kMeanThreads * vecw);
    if (bx > 0x7fffffffLL || S > 65535) return DETOX_ERR_UNSUPPORTED;
    dim3 grid((unsigned)bx, (unsigned)S);
    if (vec && sign) hier_mean_kernel<4, true><<<grid, kMeanThreads, 0, s>>>(Z, ldz, d, sets, M, ldm);
    else if (vec) hier_mean_kernel<4, false><<<grid, kMeanThreads, 0, s>>>(Z, ldz, d, sets, M, ldm);
    else if (sign) hier_mean_kernel<1, true><<<grid, kMeanThreads, 0, s>>>(Z, ldz, d, sets, M, ldm);
    else hier_mean_kernel<1, false><<<grid, kMeanThreads, 0, s>>>(Z, ldz, d, sets, M, ldm);
    return launch_status();
}

detox_status launch_mean_rows(const float* X, int64_t ld, int64_t d, const int32_t* rows_dev, int k, float* out,
                              cudaStream_t s, bool sign) {
    const bool vec = aligned16(X) && aligned16(out) && ld % 4 == 0;
    const int vecw = vec ? 4 : 1;
    int64_t bx = ceil_div(d, (int64_t)kMeanThreads * vecw);
    if (bx > 0x7fffffffLL) return DETOX_ERR_UNSUPPORTED;
    if (vec && sign) mean_rows_kernel<4, true><<<(unsigned)bx, kMeanThreads, 0, s>>>(X, ld, d, rows_dev, k, out);
    else if (vec) mean_rows_kernel<4, false><<<(unsigned)bx, kMeanThreads, 0, s>>>(X, ld, d, rows_dev, k, out);
    else if (sign) mean_rows_kernel<1, true><<<(unsigned)bx, kMeanThreads, 0, s>>>(X, ld, d, rows_dev, k, out);
    else mean_rows_kernel<1, false><<<(unsigned)bx, kMeanThreads, 0, s>>>(X, ld, d, rows_dev, k, out);
    return launch_status();
}

}  // namespace detox
