// Per-coordinate order statistics over m rows: the coordinate-wise median (Section 4; Appendix B.1)
// and the second stage of Bulyan (mean of the beta values closest to the median).
//
// m <= 32: one thread owns 1, 2 or 4 coordinates and sorts their m values in registers with a
//          fixed network; the median needs only part of it.
// m  > 32: a CTA stages a 32-coordinate tile as integer keys in shared memory and its 8 warps run
//          the layers of a merge-exchange network over it (warp = one comparator at a time for 32
//          coordinates, so shared-memory accesses are conflict-free and control flow is uniform).
#include "common.cuh"
#include "sortnet.cuh"

namespace detox {

namespace {

constexpr int kRegThreads = 128;

// Start of the window of `beta` consecutive sorted values that are closest to the median `med`.
// dist(i) = |v_i - med| in fp32 falls, then rises, along the sorted order.  The window [L, L+beta) is
// right when the value just above it is not strictly closer than its lowest value; on equal distance
// the lower value stays.  The predicate below is true exactly for the starts that are too far left.
template <typename KeyAt>
__device__ __forceinline__ int window_start(int theta, int beta, float med, KeyAt key_at) {
    const int h_lo = (theta - 1) >> 1;
    int L = 0;
    for (int s = 0; s < theta - beta; ++s) {
        bool move_right;
        if (s + beta <= h_lo) {
            move_right = true;  // the window must reach the middle element
        } else {
            const float lo = float_of_key(key_at(s));
            const float up = float_of_key(key_at(s + beta));
            move_right = fabsf(up - med) < fabsf(lo - med);
        }
        L += move_right ? 1 : 0;
    }
    return L;
}

template <int M, int C, bool TRIM>
__global__ void __launch_bounds__(kRegThreads)
colselect_reg_kernel(const float* __restrict__ X, int64_t ld, int64_t d, const int32_t* __restrict__ rows,
                     int beta, float* __restrict__ out) {
    const int64_t col0 = ((int64_t)blockIdx.x * kRegThreads + threadIdx.x) * C;
    if (col0 >= d) return;
    const int64_t left = d - col0;
    const int valid = left >= C ? C : (int)left;

    int32_t key[C][M];
#pragma unroll
    for (int i = 0; i < M; ++i) {
        const float* p = X + (int64_t)(rows ? rows[i] : i) * ld + col0;
        if (C == 4 && valid == 4) {
            uint4 v = ld_stream_u4(p);
            key[0][i] = key_of_bits(v.x);
            key[1 % C][i] = key_of_bits(v.y);
            key[2 % C][i] = key_of_bits(v.z);
            key[3 % C][i] = key_of_bits(v.w);
        } else if (C == 2 && valid == 2) {
            uint2 v = __ldcs(reinterpret_cast<const uint2*>(p));
            key[0][i] = key_of_bits(v.x);
            key[1 % C][i] = key_of_bits(v.y);
        } else {
#pragma unroll
            for (int c = 0; c < C; ++c) key[c][i] = c < valid ? key_of_bits(ld_stream_u1(p + c)) : 0;
        }
    }

    __shared__ int32_t sorted[TRIM ? M * C * kRegThreads : 1];
    float res[C];
#pragma unroll
    for (int c = 0; c < C; ++c) {
        sort_registers<M>(key[c]);
        float med;
        if (M & 1) med = float_of_key(key[c][M / 2]);
        else med = (float_of_key(key[c][M / 2 > 0 ? M / 2 - 1 : 0]) + float_of_key(key[c][M / 2])) * 0.5f;
        if (!TRIM) {
            res[c] = med;
        } else {
            int32_t* mine = sorted + (size_t)c * M * kRegThreads + threadIdx.x;
#pragma unroll
            for (int i = 0; i < M; ++i) mine[i * kRegThreads] = key[c][i];
            const int L = window_start(M, beta, med, [&](int i) { return mine[i * kRegThreads]; });
            float acc = 0.f;
#pragma unroll
            for (int i = 0; i < M; ++i)
                if (i >= L && i < L + beta) acc += float_of_key(key[c][i]);
            res[c] = acc / (float)beta;
        }
    }
    if (C == 4 && valid == 4) {
        st_stream_f4(out + col0, make_float4(res[0], res[1 % C], res[2 % C], res[3 % C]));
    } else if (C == 2 && valid == 2) {
        __stcs(reinterpret_cast<float2*>(out + col0), make_float2(res[0], res[1 % C]));
    } else {
#pragma unroll
        for (int c = 0; c < C; ++c)
            if (c < valid) out[col0 + c] = res[c];
    }
}

// ------------------------------------------------------------------------------- m > 32

constexpr int kTileCols = 32;
constexpr int kBigWarps = 8;
constexpr int kBigThreads = kTileCols * kBigWarps;

__global__ void __launch_bounds__(kBigThreads)
colselect_smem_kernel(const float* __restrict__ X, int64_t ld, int m, int64_t d,
                      const int32_t* __restrict__ rows, int beta, float* __restrict__ out) {
    extern __shared__ int32_t keys[];  // [m][kTileCols]
    const int c = threadIdx.x & (kTileCols - 1);
    const int w = threadIdx.x >> 5;
    const int64_t col = (int64_t)blockIdx.x * kTileCols + c;
    const bool live = col < d;

    for (int i = w; i < m; i += kBigWarps) {
        const int64_t r = rows ? rows[i] : i;
        keys[i * kTileCols + c] = live ? key_of_bits(ld_stream_u1(X + r * ld + col)) : 0;
    }
    __syncthreads();

    // merge exchange: every (p, k) layer holds disjoint comparators
    for (int p = 1; p < m; p <<= 1) {
        for (int k = p; k >= 1; k >>= 1) {
            const int j0 = k % p;
            const int span = m - 1 - k - j0;  // j runs j0, j0+2k, ... while j <= m-1-k
            if (span >= 0) {
                const int nj = span / (2 * k) + 1;
                const int total = nj * k;
                for (int idx = w; idx < total; idx += kBigWarps) {
                    const int jj = idx / k;
                    const int i = idx - jj * k;
                    const int a = j0 + jj * 2 * k + i;
                    const int b = a + k;
                    if (b < m && (a / (2 * p)) == (b / (2 * p))) {
                        const int32_t x = keys[a * kTileCols + c];
                        const int32_t y = keys[b * kTileCols + c];
                        keys[a * kTileCols + c] = min(x, y);
                        keys[b * kTileCols + c] = max(x, y);
                    }
                }
            }
            __syncthreads();
        }
    }

    if (w == 0 && live) {
        float med;
        if (m & 1) med = float_of_key(keys[(m / 2) * kTileCols + c]);
        else med = (float_of_key(keys[(m / 2 - 1) * kTileCols + c]) + float_of_key(keys[(m / 2) * kTileCols + c])) * 0.5f;
        if (beta == 0) {
            out[col] = med;
        } else {
            const int L = window_start(m, beta, med, [&](int i) { return keys[i * kTileCols + c]; });
            // compensated fp32 sum over up to 1024 values
            float acc = 0.f, comp = 0.f;
            for (int i = L; i < L + beta; ++i) {
                const float y = float_of_key(keys[i * kTileCols + c]) - comp;
                const float t = acc + y;
                comp = (t - acc) - y;
                acc = t;
            }
            out[col] = acc / (float)beta;
        }
    }
}

template <int M, int C>
detox_status launch_reg(const float* X, int64_t ld, int64_t d, const int32_t* rows, int beta, float* out,
                        cudaStream_t s) {
    int64_t bx = ceil_div(d, (int64_t)kRegThreads * C);
    if (bx > 0x7fffffffLL) return DETOX_ERR_UNSUPPORTED;
    if (beta == 0) colselect_reg_kernel<M, C, false><<<(unsigned)bx, kRegThreads, 0, s>>>(X, ld, d, rows, beta, out);
    else colselect_reg_kernel<M, C, true><<<(unsigned)bx, kRegThreads, 0, s>>>(X, ld, d, rows, beta, out);
    return launch_status();
}

template <int M>
detox_status launch_reg_m(const float* X, int64_t ld, int64_t d, const int32_t* rows, int beta, float* out,
                          bool vec, cudaStream_t s) {
    constexpr int C = M <= 8 ? 4 : (M <= 16 ? 2 : 1);
    if (vec && C > 1) return launch_reg<M, C>(X, ld, d, rows, beta, out, s);
    return launch_reg<M, 1>(X, ld, d, rows, beta, out, s);
}

}  // namespace

detox_status launch_coord_select(const float* X, int64_t ld, int m, int64_t d, const int32_t* rows_dev, int beta,
                                 float* out, cudaStream_t s) {
    const bool vec = aligned16(X) && aligned16(out) && ld % 4 == 0;
    switch (m) {
#define DETOX_CASE(M) \
    case M: return launch_reg_m<M>(X, ld, d, rows_dev, beta, out, vec, s);
        DETOX_CASE(1) DETOX_CASE(2) DETOX_CASE(3) DETOX_CASE(4) DETOX_CASE(5) DETOX_CASE(6) DETOX_CASE(7)
        DETOX_CASE(8) DETOX_CASE(9) DETOX_CASE(10) DETOX_CASE(11) DETOX_CASE(12) DETOX_CASE(13) DETOX_CASE(14)
        DETOX_CASE(15) DETOX_CASE(16) DETOX_CASE(17) DETOX_CASE(18) DETOX_CASE(19) DETOX_CASE(20) DETOX_CASE(21)
        DETOX_CASE(22) DETOX_CASE(23) DETOX_CASE(24) DETOX_CASE(25) DETOX_CASE(26) DETOX_CASE(27) DETOX_CASE(28)
        DETOX_CASE(29) DETOX_CASE(30) DETOX_CASE(31) DETOX_CASE(32)
#undef DETOX_CASE
        default: break;
    }
    const size_t smem = (size_t)m * kTileCols * sizeof(int32_t);
    if (cudaFuncSetAttribute(colselect_smem_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess)
        return DETOX_ERR_CUDA;
    int64_t bx = ceil_div(d, kTileCols);
    if (bx > 0x7fffffffLL) return DETOX_ERR_UNSUPPORTED;
    colselect_smem_kernel<<<(unsigned)bx, kBigThreads, smem, s>>>(X, ld, m, d, rows_dev, beta, out);
    return launch_status();
}

}  // namespace detox
