// Register-resident per-coordinate order statistics (shared by the translation units that
// instantiate the network sizes; see median.cu for the overview).
#pragma once

#include "common.cuh"
#include "sortnet.cuh"

namespace detox {
namespace regselect {

constexpr int kRegThreads = 128;

// Start of the window of `beta` consecutive sorted values that are closest to the median `med`.
// dist(i) = |v_i - med| in fp32 falls, then rises, along the sorted order.  The window [L, L+beta) is
// right when the value just above it is not strictly closer than its lowest value; on equal distance
// the lower value stays.  The predicate below is true exactly for the starts that are too far left
// (true for s < L, false from L on), so L is found by bisection over s in [0, theta - beta].
template <typename KeyAt>
__device__ __forceinline__ int window_start(int theta, int beta, float med, KeyAt key_at) {
    const int h_lo = (theta - 1) >> 1;
    int lo = 0, hi = theta - beta;
    while (lo < hi) {
        const int s = (lo + hi) >> 1;
        bool move_right;
        if (s + beta <= h_lo) {
            move_right = true;  // the window must reach the middle element
        } else {
            const float below = float_of_key(key_at(s));
            const float above = float_of_key(key_at(s + beta));
            move_right = fabsf(above - med) < fabsf(below - med);
        }
        if (move_right) lo = s + 1;
        else hi = s;
    }
    return lo;
}

__host__ __device__ constexpr int reg_threads(int M, int C, bool trim) {
    // the TRIM variant keeps M * C keys per thread in (static) shared memory, next to a staged row list
    return (trim && M * C * kRegThreads * 4 + M * 8 > 48 * 1024) ? kRegThreads / 2 : kRegThreads;
}

// M = network size, m = rows actually present (M - m even; the gap is filled with lowest / highest keys)
template <int M, int C, bool TRIM>
__global__ void __launch_bounds__(reg_threads(M, C, TRIM))
colselect_reg_kernel(const float* __restrict__ X, int64_t ld, int m, int64_t d, const int32_t* __restrict__ rows,
                     int beta, float* __restrict__ out) {
    constexpr int kThreads = reg_threads(M, C, TRIM);
    // a row list is staged in shared memory once per CTA, as element offsets of the rows (-1 for a negative entry,
    // which stands for a zero row): read from global memory it would put an index load and a 64-bit multiply in
    // front of every data load
    __shared__ int64_t soff[M];
    bool any_zero_row = false;
    if (rows) {
        int neg = 0;
        for (int i = threadIdx.x; i < m; i += kThreads) {
            const int rr = rows[i];
            soff[i] = rr < 0 ? -1 : (int64_t)rr * ld;
            neg |= rr < 0;
        }
        any_zero_row = __syncthreads_or(neg) != 0;
    }
    const int64_t col0 = ((int64_t)blockIdx.x * kThreads + threadIdx.x) * C;
    if (col0 >= d) return;
    const int64_t left = d - col0;
    const int valid = left >= C ? C : (int)left;

    // Network sizes up to 32 are used with m == M; larger ones may carry padding: at most kMaxGap slots, the top ones
    // (the dispatcher rounds m up to the next network size, 8 apart up to 64 and 16 apart above).  Only those slots
    // pay for the clamped row index and the padding test; the others have a compile-time row.
    constexpr bool kPadded = M > 32;
    constexpr int kMaxGap = !kPadded ? 0 : (M <= 64 ? 7 : 15);
    constexpr int kSure = M - kMaxGap;            // slots below this always hold a row
    const int pad = kPadded ? (M - m) >> 1 : 0;   // lowest keys added (and as many highest)
    int32_t key[C][M];
    const uint32_t col32 = (uint32_t)col0;        // the launcher keeps d below 2^31 per launch
    auto load_piece = [&](const float* p, uint32_t keep, int i) {
        if (C == 4 && valid == 4) {
            uint4 v = ld_stream_u4(p);
            key[0][i] = (int32_t)(v.x & keep);
            key[1 % C][i] = (int32_t)(v.y & keep);
            key[2 % C][i] = (int32_t)(v.z & keep);
            key[3 % C][i] = (int32_t)(v.w & keep);
        } else if (C == 2 && valid == 2) {
            uint2 v = __ldcs(reinterpret_cast<const uint2*>(p));
            key[0][i] = (int32_t)(v.x & keep);
            key[1 % C][i] = (int32_t)(v.y & keep);
        } else {
#pragma unroll
            for (int c = 0; c < C; ++c) key[c][i] = c < valid ? (int32_t)(ld_stream_u1(p + c) & keep) : 0;
        }
    };
    // All loads first, with no branch in between, so that they are in flight together; slots beyond m
    // re-read the last row and are replaced by padding keys afterwards.  The test for a row list is
    // taken once, outside the loads: a per-load test would serialise them.
    if (rows) {
        const float* base = X + col0;
        if (!any_zero_row) {
#pragma unroll
            for (int i = 0; i < M; ++i) load_piece(base + soff[i < kSure ? i : (i < m ? i : m - 1)], 0xFFFFFFFFu, i);
        } else {
#pragma unroll
            for (int i = 0; i < M; ++i) {
                const int64_t off = soff[i < kSure ? i : (i < m ? i : m - 1)];
                load_piece(base + (off < 0 ? 0 : off), off < 0 ? 0u : 0xFFFFFFFFu, i);
            }
        }
    } else {
        // row pointer (the same for the whole warp) + 4 * column: one 32 x 32 + 64 bit multiply-add per value
#pragma unroll
        for (int i = 0; i < M; ++i) {
            const float* rowp = X + (int64_t)(i < kSure ? i : (i < m ? i : m - 1)) * ld;
            load_piece(reinterpret_cast<const float*>(reinterpret_cast<const char*>(rowp) + (uint64_t)col32 * 4u), 0xFFFFFFFFu, i);
        }
    }
#pragma unroll
    for (int i = 0; i < M; ++i) {
#pragma unroll
        for (int c = 0; c < C; ++c) {
            int32_t k = key_of_bits((uint32_t)key[c][i]);
            if (i >= kSure && i >= m) k = (i - m < pad) ? (int32_t)0x80000000 : 0x7fffffff;
            key[c][i] = k;
        }
    }

    __shared__ int32_t sorted[TRIM ? M * C * kThreads : 1];
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
            // the m real values sit at sorted positions pad .. pad+m-1
            int32_t* mine = sorted + (size_t)c * M * kThreads + threadIdx.x;
#pragma unroll
            for (int i = 0; i < M; ++i) mine[i * kThreads] = key[c][i];
            // beta > 0: the beta values closest to the median; beta < 0: the middle -beta values (trimmed mean)
            const int cnt = beta < 0 ? -beta : beta;
            const int L = pad + (beta < 0 ? (m - cnt) >> 1
                                          : window_start(m, beta, med, [&](int i) { return mine[(i + pad) * kThreads]; }));
            // the window is read back from the sorted keys in shared memory (a masked sum over all M registers costs
            // more than that as soon as the window is short); four interleaved partial sums
            const int32_t* win = mine + (size_t)L * kThreads;
            float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
            int i = 0;
            for (; i + 3 < cnt; i += 4) {
                a0 += float_of_key(win[(i + 0) * kThreads]);
                a1 += float_of_key(win[(i + 1) * kThreads]);
                a2 += float_of_key(win[(i + 2) * kThreads]);
                a3 += float_of_key(win[(i + 3) * kThreads]);
            }
            for (; i < cnt; ++i) a0 += float_of_key(win[i * kThreads]);
            res[c] = ((a0 + a1) + (a2 + a3)) / (float)cnt;
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

template <int M, int C>
detox_status launch_reg(const float* X, int64_t ld, int m, int64_t d, const int32_t* rows, int beta, float* out,
                        cudaStream_t s) {
    // the kernel works with 32-bit column offsets: wider matrices go in pieces of 2^30 columns
    constexpr int64_t kMaxCols = (int64_t)1 << 30;
    for (int64_t c0 = 0; c0 < d; c0 += kMaxCols) {
        const int64_t dc = d - c0 < kMaxCols ? d - c0 : kMaxCols;
        if (beta == 0) {
            constexpr int T = reg_threads(M, C, false);
            colselect_reg_kernel<M, C, false><<<(unsigned)ceil_div(dc, (int64_t)T * C), T, 0, s>>>(X + c0, ld, m, dc, rows, beta,
                                                                                              out + c0);
        } else {
            constexpr int T = reg_threads(M, C, true);
            colselect_reg_kernel<M, C, true><<<(unsigned)ceil_div(dc, (int64_t)T * C), T, 0, s>>>(X + c0, ld, m, dc, rows, beta,
                                                                                             out + c0);
        }
        const detox_status st = launch_status();
        if (st != DETOX_OK) return st;
    }
    return DETOX_OK;
}

template <int M>
detox_status launch_reg_m(const float* X, int64_t ld, int m, int64_t d, const int32_t* rows, int beta, float* out,
                          bool vec, cudaStream_t s) {
    constexpr int C = M <= 12 ? 4 : (M <= 28 ? 2 : 1);
    if (vec && C > 1) return launch_reg<M, C>(X, ld, m, d, rows, beta, out, s);
    return launch_reg<M, 1>(X, ld, m, d, rows, beta, out, s);
}

}  // namespace regselect

// Instantiated in median_m64.cu / median_m96.cu / median_m128.cu: network sizes 39..64, 79..96, 111..128.
detox_status launch_reg_upto64(int M, const float* X, int64_t ld, int m, int64_t d, const int32_t* rows, int beta,
                               float* out, bool vec, cudaStream_t s);
detox_status launch_reg_upto96(int M, const float* X, int64_t ld, int m, int64_t d, const int32_t* rows, int beta,
                               float* out, bool vec, cudaStream_t s);
detox_status launch_reg_upto128(int M, const float* X, int64_t ld, int m, int64_t d, const int32_t* rows, int beta,
                                float* out, bool vec, cudaStream_t s);

// median_pair.cu: 128 < m <= 256, two lanes per coordinate
detox_status launch_pair_select(const float* X, int64_t ld, int m, int64_t d, const int32_t* rows, int beta,
                                float* out, cudaStream_t s);

}  // namespace detox
