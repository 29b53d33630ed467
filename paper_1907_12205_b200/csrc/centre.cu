// Choice of the centring rows for the tensor-core distance pass.
//
// The tensor-core path forms D_ij = |a_i|^2 + |a_j|^2 - 2 a_i.a_j from inner products, which loses accuracy when the
// rows share a large common vector (honest gradients of one loss at one model do): the three terms are then much
// larger than their difference, and the tensor cores' fp32 accumulation loses most on long sums of one sign.
// Distances do not change when one vector is subtracted from every row, so the pass may work on a_i = x_i - c with c
// in the middle of the rows; it forms c, column by column, as the mean of a few rows that are listed here.
//
// The rows are found on a sample of the columns (16 evenly spaced blocks of 64), at a cost linear in the number of
// rows: per column the median of seven rows at fixed, evenly spaced positions gives a first centre that a minority of
// outlying rows cannot move; every row's squared distance to it and squared norm are added up over the sample; the
// rows are ranked by that distance and every s-th of the closer half is listed (so that a group of colluding rows
// that sit in the very middle cannot fill the list).  Centring is switched on only when the typical row is clearly
// closer to the first centre than to the origin; rows that hover around zero are left as they are.
//
// Everything is deterministic: per-block partial sums are added in a fixed order and ties go to the lower index.
#include <math_constants.h>

#include "common.cuh"
#include "gram_tc.cuh"

namespace detox {

namespace {

constexpr int kPickThreads = 256;
constexpr int kSampleCols = 64;      // columns per sampled block
constexpr int kSampleBlocks = 16;
constexpr int kFirstRows = 7;        // rows whose column-wise median is the first centre

int sample_blocks(int64_t d) {
    const int64_t avail = ceil_div(d, (int64_t)kSampleCols);
    return (int)(avail < kSampleBlocks ? avail : kSampleBlocks);
}

struct CentreWs {
    float* part;        // [nblk][2][m]: per block, every row's squared distance to the first centre, then its squared norm
    int* agree;         // [nblk][m] votes formed on the fly: which members of the group gave the block's sampled pieces
    float* key;         // [m] scratch of the check after the pass
    unsigned* counter;  // [2] "a row failed the check" / CTAs of the check kernel that have finished; behind them one
                        // float: the typical squared norm of a centred row as the sample predicts it for all d columns
};

CentreWs centre_carve(void* ws, int m) {
    CentreWs w;
    char* p = static_cast<char*>(ws);
    w.part = reinterpret_cast<float*>(p);
    p += align_up((size_t)kSampleBlocks * 2 * m * sizeof(float));
    w.agree = reinterpret_cast<int*>(p);
    p += align_up((size_t)kSampleBlocks * m * sizeof(int));
    w.key = reinterpret_cast<float*>(p);
    p += align_up((size_t)m * sizeof(float));
    w.counter = reinterpret_cast<unsigned*>(p);
    return w;
}

__device__ __forceinline__ float nan_to_inf(float v) { return v != v ? CUDART_INF_F : v; }
__device__ __forceinline__ float finite_or_zero(float v) {
    return (__float_as_uint(v) & 0x7f800000u) != 0x7f800000u ? v : 0.f;
}
__device__ __forceinline__ void order2(float& a, float& b) {
    const float lo = fminf(a, b), hi = fmaxf(a, b);
    a = lo;
    b = hi;
}

// One CTA per sampled block of 64 columns (evenly spaced over d).
//
// VOTE: row g of the sample is the vote of the three rows members.id[3g .. 3g + 2] of X, formed piece by piece (four
// columns) as the distance pass will form it: the value two members agree on bitwise, zeros when all differ.
// agree[b][g] gets one bit per member: it gave every sampled piece of this block (the pass that follows subtracts
// rows of X, so the rows listed for centring are handed on as such a member's row).
template <bool VOTE>
__global__ void __launch_bounds__(kPickThreads)
centre_sample_kernel(const float* __restrict__ X, int64_t ld, int m, int64_t d, float* __restrict__ part,
                     unsigned* __restrict__ counter, const __grid_constant__ VoteMembers members,
                     int* __restrict__ agree) {
    extern __shared__ float tile[];   // [m][kSampleCols + 1], then the first centre [kSampleCols], then (VOTE) agree bits [m]
    constexpr int pitch = kSampleCols + 1;
    float* first = tile + (size_t)m * pitch;
    const int b = blockIdx.x, nblk = gridDim.x;
    const int64_t nb_all = (d + kSampleCols - 1) / kSampleCols;
    const int64_t c0 = (nb_all * b / nblk) * kSampleCols;
    if (b == 0 && threadIdx.x == 0) counter[0] = counter[1] = 0u;   // for the kernels that follow
    if (VOTE) {
        int* ok = reinterpret_cast<int*>(first + kSampleCols);
        for (int r = threadIdx.x; r < m; r += kPickThreads) ok[r] = 7;
        __syncthreads();
        for (int e = threadIdx.x; e < m * (kSampleCols / 4); e += kPickThreads) {
            const int r = e / (kSampleCols / 4), c = (e - r * (kSampleCols / 4)) * 4;
            uint32_t v[3][4];
#pragma unroll
            for (int k = 0; k < 3; ++k) {
                const float* row = X + (int64_t)members.id[3 * r + k] * ld;
#pragma unroll
                for (int i = 0; i < 4; ++i) v[k][i] = c0 + c + i < d ? __float_as_uint(row[c0 + c + i]) : 0u;
            }
            bool ne[3];   // pairs (0,1), (0,2), (1,2)
#pragma unroll
            for (int pr = 0; pr < 3; ++pr) {
                const int a = pr == 2 ? 1 : 0, bb = pr == 0 ? 1 : 2;
                ne[pr] = ((v[a][0] ^ v[bb][0]) | (v[a][1] ^ v[bb][1]) | (v[a][2] ^ v[bb][2]) | (v[a][3] ^ v[bb][3])) != 0u;
            }
            const bool first_wins = !ne[0] || !ne[1], other_wins = !ne[2];
            int mask = 0;
            if (first_wins) mask = 1 | (ne[0] ? 0 : 2) | (ne[1] ? 0 : 4);
            else if (other_wins) mask = 6;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const uint32_t u = first_wins ? v[0][i] : (other_wins ? v[1][i] : 0u);
                tile[r * pitch + c + i] = finite_or_zero(__uint_as_float(u));
            }
            if (mask != 7) atomicAnd(&ok[r], mask);
        }
        __syncthreads();
        for (int r = threadIdx.x; r < m; r += kPickThreads) agree[(size_t)b * m + r] = ok[r];
    } else {
        for (int e = threadIdx.x; e < m * kSampleCols; e += kPickThreads) {
            const int r = e / kSampleCols, c = e - r * kSampleCols;
            const int64_t col = c0 + c;
            tile[r * pitch + c] = col < d ? finite_or_zero(X[(int64_t)r * ld + col]) : 0.f;
        }
    }
    __syncthreads();
    if (threadIdx.x < kSampleCols) {
        // median of the rows at positions (2k + 1) m / 14, k = 0..6: the 16-comparator sorting network on seven values
        const int c = threadIdx.x;
        float v[kFirstRows];
#pragma unroll
        for (int k = 0; k < kFirstRows; ++k) v[k] = tile[(((2 * k + 1) * m) / (2 * kFirstRows)) * pitch + c];
        order2(v[0], v[6]); order2(v[2], v[3]); order2(v[4], v[5]);
        order2(v[0], v[2]); order2(v[1], v[4]); order2(v[3], v[6]);
        order2(v[0], v[1]); order2(v[2], v[5]); order2(v[3], v[4]);
        order2(v[1], v[2]); order2(v[4], v[6]);
        order2(v[2], v[3]); order2(v[4], v[5]);
        order2(v[1], v[2]); order2(v[3], v[4]); order2(v[5], v[6]);
        first[c] = v[3];
    }
    __syncthreads();
    float* out = part + (size_t)b * 2 * m;
    for (int r = threadIdx.x; r < m; r += kPickThreads) {
        const float* row = tile + r * pitch;
        float dist = 0.f, nrm = 0.f;
#pragma unroll 8
        for (int c = 0; c < kSampleCols; ++c) {
            const float x = row[c], t = x - first[c];
            dist = fmaf(t, t, dist);
            nrm = fmaf(x, x, nrm);
        }
        out[r] = dist;
        out[m + r] = nrm;
    }
}

// One CTA: adds the blocks' partial sums, ranks the rows by their distance to the first centre, lists the centring
// rows, decides whether centring pays, and gives every row its power-of-two scale for the split-fp16 pass:
// expo[r] = kTargetRmsLog2 - floor(log2(rms of row r's sampled entries after the subtraction)), so that 2^expo[r] times
// the row has its typical entry in [2^6, 2^7).  A row whose sample is zero or not finite takes the typical row's scale.
__global__ void __launch_bounds__(kPickThreads)
centre_pick_kernel(const float* __restrict__ part, int nblk, int m, float scale, float inv_sampled,
                   unsigned* __restrict__ counter, int* __restrict__ centre, int* __restrict__ expo,
                   const __grid_constant__ VoteMembers members, const int* __restrict__ agree) {
    extern __shared__ float sh[];   // dist [m], norm [m]
    float* dist = sh;
    float* nrm = sh + m;
    __shared__ float med[2];
    __shared__ int centring_on;
    for (int r = threadIdx.x; r < m; r += kPickThreads) {
        float a = 0.f, n = 0.f;
        for (int b = 0; b < nblk; ++b) {
            a += part[(size_t)b * 2 * m + r];
            n += part[(size_t)b * 2 * m + m + r];
        }
        dist[r] = nan_to_inf(a);
        nrm[r] = nan_to_inf(n);
    }
    __syncthreads();
    const int want = m / 2 < kMaxCentreRows ? m / 2 : kMaxCentreRows;
    // the rows at ranks 0, s, 2s, ... of the ordering by distance, inside its closer half
    const int stride = (m / 2) / (want > 0 ? want : 1) > 1 ? (m / 2) / want : 1;
    const int hm = (m - 1) / 2;
    for (int r = threadIdx.x; r < m; r += kPickThreads) {
        const float v = dist[r], w = nrm[r];
        int rank = 0, rank_n = 0;
        for (int k = 0; k < m; ++k) {
            const float u = dist[k], un = nrm[k];
            rank += (u < v || (u == v && k < r)) ? 1 : 0;
            rank_n += (un < w || (un == w && k < r)) ? 1 : 0;
        }
        if (rank % stride == 0 && rank / stride < want) centre[2 + rank / stride] = r;
        if (rank == hm) med[0] = v;
        if (rank_n == hm) med[1] = w;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        // on when the typical row is clearly closer to the first centre than to the origin.  Rows that hover around
        // zero have a ratio of squared distances of 0.8 .. 1.2 (the seven rows behind the first centre are a little
        // closer to it than the others) and gain nothing; rows that share a vector as long as their individual parts
        // have 0.6, and their sums of products, all of one sign, already lose to the tensor cores' truncation.
        centring_on = (want >= 1 && med[0] < 0.7f * med[1]) ? 1 : 0;
        centre[0] = centring_on ? want : 0;
        // for the check after the pass: the typical squared norm the sample predicts for the centred rows
        *reinterpret_cast<float*>(counter + 2) = med[0] * scale;
    }
    __syncthreads();
    if (agree != nullptr && threadIdx.x < want) {
        // votes formed on the fly: listed vote g is handed on as the row of X of a member that gave every sampled piece
        // (the first member when none did: whatever is subtracted, it is the same for all rows)
        const int g = centre[2 + threadIdx.x];
        int mask = 7;
        for (int b = 0; b < nblk; ++b) mask &= agree[(size_t)b * m + g];
        const int k = (mask & 1) ? 0 : ((mask & 2) ? 1 : ((mask & 4) ? 2 : 0));
        centre[2 + kMaxCentreRows + threadIdx.x] = (int)members.id[3 * g + k];
    }
    const float typical = (centring_on ? med[0] : med[1]) * inv_sampled;
    for (int r = threadIdx.x; r < m; r += kPickThreads) {
        float v = (centring_on ? dist[r] : nrm[r]) * inv_sampled;   // mean square of the sampled entries
        if (!(v > 0.f && v < CUDART_INF_F)) v = typical;
        int e = 0;
        if (v > 0.f && v < CUDART_INF_F) e = kTargetRmsLog2 - (ilogbf(v) >> 1);
        expo[r] = e < -100 ? -100 : (e > 100 ? 100 : e);
    }
}

// After the distance pass, two questions.
//
// Did the subtraction leave the rows small?  The listed rows were chosen on a sample of the columns; a row that is
// central there and holds huge values elsewhere would, once subtracted, swamp the differences between the other rows.
// `norms` holds, per output slot and group of transform warps, every row's exact squared norm after the subtraction
// (and after the row's scale 2^expo, when the split-fp16 pass ran).  One CTA per row adds its shares up; the last one
// takes the median over the rows and compares it with what the sample predicted for the centred rows.  If the
// typical row is more than 4 times larger than that, the centring is withdrawn (centre[0] = 0): a listed row with
// one large entry outside the sample is enough to put that entry into every row, and the distances would then be
// small differences of large norms.
//
// Did the split-fp16 pass (expo != null) see every entry?  In every slot the tensor cores' own squared norm of the
// row, the diagonal entry of the slot's partial, must be finite and within 1/256 of the exact one (an fp16 overflow
// makes it Inf or NaN), and the scaled row as a whole must not have come out far below the range its scale aimed at
// (its entries would have lost their low bits).  A row whose exact norm is not finite also sends the call to the other
// pass, which sees the row unscaled.
//
// *redo = 1 asks for the split-TF32 pass (with the centring that is left) when either answer is no.
constexpr float kCentreSlack = 4.f;
__device__ unsigned long long g_repeated_passes;   // calls whose check asked for the pass to be repeated (a diagnostic)
__global__ void __launch_bounds__(128)
centre_check_kernel(const float* __restrict__ norms, const float* __restrict__ partial, int nitems, int groups, int m,
                    int ncol, float min_scaled_norm, const int* __restrict__ expo, float* __restrict__ na,
                    unsigned* __restrict__ counter, int* __restrict__ centre, int* __restrict__ redo) {
    __shared__ double red[4];
    __shared__ int red_bad[4];
    __shared__ bool s_last;
    __shared__ int s_keep;
    const int i = blockIdx.x;
    const bool fast = expo != nullptr;
    const int ncentre = *centre;
    if (!fast && ncentre <= 0) {
        if (i == 0 && threadIdx.x == 0) *redo = 0;
        return;
    }
    double a = 0.0;
    int bad = 0;
    for (int it = threadIdx.x; it < nitems; it += 128) {
        float n = 0.f;
        for (int g = 0; g < groups; ++g) n += norms[((int64_t)it * groups + g) * m + i];
        a += (double)n;
        if (fast) {
            if (!(n < CUDART_INF_F)) {
                bad = 1;   // Inf or NaN: an entry of the row itself, or one that its scale pushed out of fp32
            } else if (n > 0.f) {
                const float t = partial[((int64_t)it * m + i) * ncol + i];
                if (!(fabsf(n - t) <= n * (1.f / 256.f))) bad = 1;
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        a += __shfl_xor_sync(0xffffffffu, a, o);
        bad |= __shfl_xor_sync(0xffffffffu, bad, o);
    }
    if ((threadIdx.x & 31) == 0) { red[threadIdx.x >> 5] = a; red_bad[threadIdx.x >> 5] = bad; }
    if (threadIdx.x == 0) s_keep = 1;
    __syncthreads();
    if (threadIdx.x == 0) {
        float total = nan_to_inf((float)(red[0] + red[1] + red[2] + red[3]));
        bad = red_bad[0] | red_bad[1] | red_bad[2] | red_bad[3];
        if (fast) {
            if (total > 0.f && total < min_scaled_norm) bad = 1;
            total = total < CUDART_INF_F ? ldexpf(total, -2 * expo[i]) : total;   // back to the row's own units
        }
        na[i] = total;
        if (bad) atomicOr(counter, 1u);
        __threadfence();
        s_last = atomicAdd(counter + 1, 1u) == (unsigned)(m - 1);
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    if (ncentre > 0) {
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
            if (rank == hm && !(mine <= kCentreSlack * ref)) s_keep = 0;
        }
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        const bool any_bad = __ldcg(counter) != 0u;
        *redo = (!s_keep || any_bad) ? 1 : 0;
        if (!s_keep || any_bad) atomicAdd(&g_repeated_passes, 1ull);
        if (!s_keep) *centre = 0;
        counter[0] = counter[1] = 0u;
    }
}

}  // namespace

size_t centre_ws_bytes(int m, int64_t d) {
    (void)d;
    return align_up((size_t)kSampleBlocks * 2 * m * sizeof(float)) + align_up((size_t)kSampleBlocks * m * sizeof(int)) +
           align_up((size_t)m * sizeof(float)) + 256;   // counters, float
}

// members != null: the m rows are the votes of the groups of three rows of X listed there.
detox_status launch_pick_centre(const float* X, int64_t ld, int m, int64_t d, void* ws, int* centre, int* expo,
                                cudaStream_t s, const VoteMembers* members) {
    CentreWs w = centre_carve(ws, m);
    const int nblk = sample_blocks(d);
    const size_t smem = ((size_t)m * (kSampleCols + 1) + kSampleCols + (members ? m : 0)) * sizeof(float);
    const VoteMembers none{};
    if (members) {
        if (cudaFuncSetAttribute(centre_sample_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return DETOX_ERR_CUDA;
        centre_sample_kernel<true><<<nblk, kPickThreads, smem, s>>>(X, ld, m, d, w.part, w.counter, *members, w.agree);
    } else {
        if (cudaFuncSetAttribute(centre_sample_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return DETOX_ERR_CUDA;
        centre_sample_kernel<false><<<nblk, kPickThreads, smem, s>>>(X, ld, m, d, w.part, w.counter, none, nullptr);
    }
    detox_status st = launch_status();
    if (st != DETOX_OK) return st;
    // the sample's squared norms are scaled up to all d columns for the check after the pass
    const int64_t sampled = (int64_t)nblk * kSampleCols < d ? (int64_t)nblk * kSampleCols : d;
    const float scale = (float)((double)d / (double)sampled);
    centre_pick_kernel<<<1, kPickThreads, (size_t)2 * m * sizeof(float), s>>>(w.part, nblk, m, scale, 1.f / (float)sampled,
                                                                            w.counter, centre, expo, members ? *members : none,
                                                                            members ? w.agree : nullptr);
    return launch_status();
}

detox_status launch_check_centre(const float* norms, const float* partial, int nitems, int groups, int m, int ncol,
                                 void* ws, int64_t d, int* centre, int* redo, const int* expo, cudaStream_t s) {
    CentreWs w = centre_carve(ws, m);
    // a scaled row aims at a typical entry of 2^6 or more; below 2^2 its scale was far off
    const float min_scaled_norm = (float)((double)d * 16.0);
    // both counter words were cleared by the sample kernel
    centre_check_kernel<<<m, 128, 0, s>>>(norms, partial, nitems, groups, m, ncol, min_scaled_norm, expo, w.key, w.counter,
                                          centre, redo);
    return launch_status();
}

unsigned long long tc_repeated_passes() {
    unsigned long long v = 0;
    if (cudaMemcpyFromSymbol(&v, g_repeated_passes, sizeof(v)) != cudaSuccess) return ~0ull;
    return v;
}

}  // namespace detox
