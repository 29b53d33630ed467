// Per-coordinate order statistics over m rows: the coordinate-wise median (Section 4; Appendix B.1)
// and the second stage of Bulyan (mean of the beta values closest to the median).
//
// m <= 128: one thread owns 1, 2 or 4 coordinates and sorts their values in registers with a fixed
//           network; the median needs only part of it.  Sizes above 32 are served by a few network
//           sizes: the m values are padded with equally many lowest and highest keys, which leaves
//           the median (and the values around it) where they were.
// 128 < m <= 256: two lanes per coordinate, up to 128 registers of keys each (median_pair.cu).
// m  > 256: a CTA stages a 32-coordinate tile as integer keys in shared memory and its 8 warps run
//          the layers of a merge-exchange network over it (warp = one comparator at a time for 32
//          coordinates, so shared-memory accesses are conflict-free and control flow is uniform).
#include "median_impl.cuh"

namespace detox {

namespace {

using namespace regselect;

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
        const int64_t r = rows ? rows[i] : i;     // a negative entry of the row list stands for a zero row
        keys[i * kTileCols + c] = (live && r >= 0) ? key_of_bits(ld_stream_u1(X + r * ld + col)) : key_of_bits(0u);
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
            const int cnt = beta < 0 ? -beta : beta;   // beta < 0: the middle -beta values (trimmed mean)
            const int L = beta < 0 ? (m - cnt) >> 1
                                   : window_start(m, beta, med, [&](int i) { return keys[i * kTileCols + c]; });
            // compensated fp32 sum over up to 1024 values
            float acc = 0.f, comp = 0.f;
            for (int i = L; i < L + cnt; ++i) {
                const float y = float_of_key(keys[i * kTileCols + c]) - comp;
                const float t = acc + y;
                comp = (t - acc) - y;
                acc = t;
            }
            out[col] = acc / (float)cnt;
        }
    }
}

}  // namespace

detox_status launch_coord_select(const float* X, int64_t ld, int m, int64_t d, const int32_t* rows_dev, int beta,
                                 float* out, cudaStream_t s) {
    const bool vec = aligned16(X) && aligned16(out) && ld % 4 == 0;
    switch (m) {
#define DETOX_CASE(M) \
    case M: return launch_reg_m<M>(X, ld, m, d, rows_dev, beta, out, vec, s);
        DETOX_CASE(1) DETOX_CASE(2) DETOX_CASE(3) DETOX_CASE(4) DETOX_CASE(5) DETOX_CASE(6) DETOX_CASE(7)
        DETOX_CASE(8) DETOX_CASE(9) DETOX_CASE(10) DETOX_CASE(11) DETOX_CASE(12) DETOX_CASE(13) DETOX_CASE(14)
        DETOX_CASE(15) DETOX_CASE(16) DETOX_CASE(17) DETOX_CASE(18) DETOX_CASE(19) DETOX_CASE(20) DETOX_CASE(21)
        DETOX_CASE(22) DETOX_CASE(23) DETOX_CASE(24) DETOX_CASE(25) DETOX_CASE(26) DETOX_CASE(27) DETOX_CASE(28)
        DETOX_CASE(29) DETOX_CASE(30) DETOX_CASE(31) DETOX_CASE(32)
#undef DETOX_CASE
        default: break;
    }
    if (m <= 128) {
        // network sizes above 32: every 8th size up to 64, every 16th up to 128, in either parity
        // (M - m must be even so that as many lowest as highest keys are added)
        const int step = m <= 64 ? 8 : 16;
        int M = ((m + step - 1) / step) * step;
        if ((M - m) & 1) M -= 1;
        if (M <= 64) return launch_reg_upto64(M, X, ld, m, d, rows_dev, beta, out, vec, s);
        if (M <= 96) return launch_reg_upto96(M, X, ld, m, d, rows_dev, beta, out, vec, s);
        return launch_reg_upto128(M, X, ld, m, d, rows_dev, beta, out, vec, s);
    }
    if (m <= 256) return launch_pair_select(X, ld, m, d, rows_dev, beta, out, s);
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
