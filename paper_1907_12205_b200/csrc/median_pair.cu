// Per-coordinate order statistics with two adjacent lanes per coordinate (128 < m <= 256 rows).
//
// Each lane sorts H keys in registers (lane 0: rows 0..H-1; lane 1: the other rows plus padding
// keys, lowest and highest, placed so that the wanted median lands on sorted position H-1 of the
// 2H).  One bitonic split across the lane pair (min / max against the partner's reversed run)
// leaves the H smallest keys in lane 0 and the H largest in lane 1; the median is then the
// maximum of lane 0's keys (for an even count, averaged with the minimum of lane 1's).  Sorting
// two halves and splitting costs about half the comparators of one network over all m values.
// For Bulyan's second stage both halves are sorted with a bitonic merge (sortnet.cuh: any H) and
// laid out in shared memory for the data-dependent window search.
#include "median_impl.cuh"

namespace detox {

namespace {

constexpr int kPairThreads = 128;              // 64 coordinates per CTA
constexpr int kPairCols = kPairThreads / 2;

template <int kHalf, bool TRIM>
__global__ void __launch_bounds__(kPairThreads)
colselect_pair_kernel(const float* __restrict__ X, int64_t ld, int m, int64_t d, const int32_t* __restrict__ rows,
                      int beta, float* __restrict__ out) {
    extern __shared__ int32_t sorted[];        // TRIM only: [2 * kHalf][kPairCols]
    // a row list is staged in shared memory once per CTA, as element offsets of the rows (-1 for a negative entry,
    // which stands for a zero row): read from global memory it would put an index load and a 64-bit multiply in
    // front of every data load
    __shared__ int64_t soff[2 * kHalf];
    if (rows) {
        for (int i = threadIdx.x; i < m; i += kPairThreads) {
            const int rr = rows[i];
            soff[i] = rr < 0 ? -1 : (int64_t)rr * ld;
        }
        __syncthreads();
    }
    const int hsel = threadIdx.x & 1;
    const int cidx = threadIdx.x >> 1;
    const int64_t col_raw = (int64_t)blockIdx.x * kPairCols + cidx;
    const bool live = col_raw < d;
    const int64_t col = live ? col_raw : d - 1;   // dead pairs recompute the last coordinate and do not store

    const int pad_lo = (kHalf - 1) - ((m - 1) >> 1);   // lowest keys added: puts the (lower) median on position 127
    const int extra = m - kHalf;                        // real rows held by lane 1

    int32_t key[kHalf];
    // Lane 0 always holds kHalf rows.  Lane 1 holds `extra` rows, at least kSure of them when the median picks
    // kHalf (half of m rounded up to 8), so only its top slots pay for the clamped row and the padding test.
    constexpr int kSure = kHalf - 16;
    // the test for a row list is taken once, outside the loads: a per-load test would serialise them
    if (rows) {
#pragma unroll
        for (int i = 0; i < kHalf; ++i) {
            int ri = hsel ? kHalf + i : i;
            if (i >= kSure) ri = ri < m ? ri : m - 1;
            const int64_t off = soff[ri];
            const uint32_t v = ld_stream_u1(X + col + (off < 0 ? 0 : off));
            key[i] = (int32_t)(off < 0 ? 0u : v);
        }
    } else {
        // this lane's first row at its column; row i of the lane is i * ld further (the same step for all lanes)
        const float* base = X + (int64_t)(hsel ? kHalf : 0) * ld + col;
        const int last = (hsel ? extra : kHalf) - 1;
#pragma unroll
        for (int i = 0; i < kHalf; ++i) key[i] = (int32_t)ld_stream_u1(base + (int64_t)(i < kSure ? i : (i < last ? i : last)) * ld);
    }
#pragma unroll
    for (int i = 0; i < kHalf; ++i) {
        int32_t k = key_of_bits((uint32_t)key[i]);
        if (i >= kSure && hsel && i >= extra) k = (i - extra < pad_lo) ? (int32_t)0x80000000 : 0x7fffffff;
        key[i] = k;
    }
    sort_registers<kHalf>(key);

    // bitonic split with the partner lane: lane 0 keeps the minima, lane 1 the maxima
#pragma unroll
    for (int i = 0; i < kHalf / 2; ++i) {
        const int j = kHalf - 1 - i;
        const int32_t from_j = __shfl_xor_sync(0xffffffffu, key[j], 1);
        const int32_t from_i = __shfl_xor_sync(0xffffffffu, key[i], 1);
        key[i] = hsel ? max(key[i], from_j) : min(key[i], from_j);
        key[j] = hsel ? max(key[j], from_i) : min(key[j], from_i);
    }

    if (!TRIM) {
        int32_t ext = key[0];
#pragma unroll
        for (int i = 1; i < kHalf; ++i) ext = hsel ? min(ext, key[i]) : max(ext, key[i]);
        const int32_t up_min = __shfl_xor_sync(0xffffffffu, ext, 1);   // lane 0 receives lane 1's minimum
        if (hsel == 0 && live) {
            const float lo = float_of_key(ext);
            out[col] = (m & 1) ? lo : (lo + float_of_key(up_min)) * 0.5f;
        }
        return;
    }

    // Lane 0's keys now rise and then fall, lane 1's fall and then rise.  Lane 1 complements its keys, which
    // turns its sequence into a rise-then-fall one as well, so both lanes run the same merge network; lane 1's
    // keys come out in descending order of the real values.
    const int32_t flip = hsel ? -1 : 0;
#pragma unroll
    for (int i = 0; i < kHalf; ++i) key[i] ^= flip;
    bitonic_merge_registers<kHalf>(key);
    // position p of the 2 kHalf sorted keys -> sorted[p * kPairCols + slot]; the slot is rotated by 16 for the
    // upper half so that the two lanes of a pair never hit the same bank
    {
        constexpr BitonicMergeNet<kHalf> net{};
        const int slot = (cidx + hsel * 16) & (kPairCols - 1);
#pragma unroll
        for (int i = 0; i < kHalf; ++i) {
            const int p = hsel ? 2 * kHalf - 1 - net.pos[i] : net.pos[i];
            sorted[p * kPairCols + slot] = key[i] ^ flip;
        }
    }
    __syncwarp();
    auto at = [&](int p) { return sorted[p * kPairCols + ((cidx + (p >= kHalf ? 16 : 0)) & (kPairCols - 1))]; };
    float med = float_of_key(at(kHalf - 1));
    if ((m & 1) == 0) med = (med + float_of_key(at(kHalf))) * 0.5f;
    const int cnt = beta < 0 ? -beta : beta;   // beta < 0: the middle -beta values (trimmed mean)
    // both lanes of the pair find the same window
    const int L = pad_lo + (beta < 0 ? (m - cnt) >> 1
                                     : regselect::window_start(m, beta, med, [&](int i) { return at(i + pad_lo); }));
    // each lane adds the part of the window that lies in its own half of the sorted positions, read back from
    // shared memory (cheaper than a masked sum over all of its registers); four interleaved partial sums
    const int lo_p = hsel * kHalf, hi_p = lo_p + kHalf;
    const int p0 = L > lo_p ? L : lo_p, p1 = L + cnt < hi_p ? L + cnt : hi_p;
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
    int p = p0;
    for (; p + 3 < p1; p += 4) {
        a0 += float_of_key(at(p));
        a1 += float_of_key(at(p + 1));
        a2 += float_of_key(at(p + 2));
        a3 += float_of_key(at(p + 3));
    }
    for (; p < p1; ++p) a0 += float_of_key(at(p));
    float sum = (a0 + a1) + (a2 + a3);
    sum += __shfl_xor_sync(0xffffffffu, sum, 1);
    if (hsel == 0 && live) out[col] = sum / (float)cnt;
}


template <int H>
detox_status launch_pair(const float* X, int64_t ld, int m, int64_t d, const int32_t* rows, int beta, float* out,
                         cudaStream_t s) {
    int64_t bx = ceil_div(d, kPairCols);
    if (bx > 0x7fffffffLL) return DETOX_ERR_UNSUPPORTED;
    if (beta == 0) {
        colselect_pair_kernel<H, false><<<(unsigned)bx, kPairThreads, 0, s>>>(X, ld, m, d, rows, beta, out);
    } else {
        const size_t smem = (size_t)2 * H * kPairCols * sizeof(int32_t);
        if (cudaFuncSetAttribute(colselect_pair_kernel<H, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)smem) != cudaSuccess)
            return DETOX_ERR_CUDA;
        colselect_pair_kernel<H, true><<<(unsigned)bx, kPairThreads, smem, s>>>(X, ld, m, d, rows, beta, out);
    }
    return launch_status();
}

}  // namespace

// 128 < m <= 256.  H = half of m rounded up to 8.
detox_status launch_pair_select(const float* X, int64_t ld, int m, int64_t d, const int32_t* rows, int beta,
                                float* out, cudaStream_t s) {
    const int H = ((m + 1) / 2 + 7) / 8 * 8;
    switch (H) {
#define DETOX_CASE(HH) \
    case HH: return launch_pair<HH>(X, ld, m, d, rows, beta, out, s);
        DETOX_CASE(72) DETOX_CASE(80) DETOX_CASE(88) DETOX_CASE(96) DETOX_CASE(104) DETOX_CASE(112) DETOX_CASE(120) DETOX_CASE(128)
#undef DETOX_CASE
        default: return DETOX_ERR_UNSUPPORTED;
    }
}

}  // namespace detox
