// Krum scoring and index selection on the m x m distance matrix (Multi-Krum; Bulyan stage 1).
// All of this is O(m^2 log m) work on at most a few MB: latency-bound, a handful of small kernels.
//
// Step 1 (rank_rows): every row's distances are ranked once (ties: lower column index first) and
//   stored in ascending order together with their column indices.
// Multi-Krum: score_i = sum of the first nb entries of row i's ascending list, added in that order;
//   the m_sel smallest scores win (ties: lower index).
// Bulyan: theta rounds in one CTA, one thread per row.  A row's score is the sum of its nb closest
//   remaining rows, i.e. of the remaining entries of its ascending list up to a pointer.  Removing the
//   round's winner changes every other row's sum by one entry at most (the winner's distance leaves
//   if it was counted; the farthest counted entry leaves when nb shrinks), so each round costs O(1)
//   per row instead of a walk over the list (the last few rounds, with at most 8 neighbours, re-add
//   them from scratch so that exact ties stay exact).  Bitwise-equal rows see the same values in the same
//   order, so their scores stay bitwise equal and ties keep going to the lower index.
#include <math_constants.h>

#include "common.cuh"

namespace detox {

namespace {

constexpr int kFreshSumBelow = 8;   // Bulyan rounds with at most this many neighbours re-add them from scratch

// NaN compares false with everything, which would break the ranking below: it is ranked as +Inf.
__device__ __forceinline__ double nan_to_inf(double v) { return v != v ? CUDART_INF : v; }

struct SelectWs {
    double* sorted_d;    // m x m, row i ascending, self at the end (+inf)
    int32_t* sorted_j;   // m x m, matching column indices
    int32_t* pos_t;      // m x m, pos_t[j][i] = position of column j in row i's list
    double* score;       // m
};

SelectWs carve(void* ws, int m) {
    SelectWs w;
    char* p = static_cast<char*>(ws);
    w.sorted_d = reinterpret_cast<double*>(p);
    p += align_up((size_t)m * m * sizeof(double));
    w.sorted_j = reinterpret_cast<int32_t*>(p);
    p += align_up((size_t)m * m * sizeof(int32_t));
    w.pos_t = reinterpret_cast<int32_t*>(p);
    p += align_up((size_t)m * m * sizeof(int32_t));
    w.score = reinterpret_cast<double*>(p);
    return w;
}

__global__ void __launch_bounds__(256)
rank_rows_kernel(const double* __restrict__ D, int m, double* __restrict__ sorted_d, int32_t* __restrict__ sorted_j,
                 int32_t* __restrict__ pos_t) {
    extern __shared__ double rowv[];  // m
    const int i = blockIdx.x;
    // a NaN distance (a row with non-finite entries, or a distance pass that gave up) counts as +Inf, so that the
    // ranks below are always a permutation of 0..m-1 and every slot of the lists is written
    for (int j = threadIdx.x; j < m; j += blockDim.x) rowv[j] = (j == i) ? CUDART_INF : nan_to_inf(D[(int64_t)i * m + j]);
    __syncthreads();
    for (int j = threadIdx.x; j < m; j += blockDim.x) {
        int rank;
        if (j == i) {
            rank = m - 1;
        } else {
            const double v = rowv[j];
            rank = 0;
            for (int k = 0; k < m; ++k) {
                if (k == i) continue;
                const double u = rowv[k];
                rank += (u < v || (u == v && k < j)) ? 1 : 0;
            }
        }
        sorted_d[(int64_t)i * m + rank] = rowv[j];
        sorted_j[(int64_t)i * m + rank] = j;
        pos_t[(int64_t)j * m + i] = rank;
    }
}

__device__ __forceinline__ int krum_neighbours(int alive, int f) {
    int nb = alive - f - 2;
    nb = nb < 1 ? 1 : nb;
    nb = nb > alive - 1 ? alive - 1 : nb;
    return nb;
}

// One thread per row; the lists may live in global or in shared memory.  ONE_WARP: m <= 32 and only the first
// warp of the CTA is inside (it synchronises by itself); otherwise the whole CTA is (m <= blockDim.x).
template <bool ONE_WARP>
__device__ __forceinline__ void group_sync() {
    if (ONE_WARP) __syncwarp();
    else __syncthreads();
}

template <bool ONE_WARP>
__device__ __forceinline__ void multikrum_select_body(const double* sorted_d, int m, int f, int m_sel, int32_t* sel,
                                                      double* scores_out) {
    __shared__ double score[kMaxRows];
    __shared__ int chosen[kMaxRows];
    const int i = threadIdx.x;
    const int nb = krum_neighbours(m, f);
    if (i < m) {
        double s = 0.0;
        for (int k = 0; k < nb; ++k) s += sorted_d[(int64_t)i * m + k];
        score[i] = s;
        if (scores_out) scores_out[i] = s;
    }
    group_sync<ONE_WARP>();
    if (i < m) {
        int rank = 0;
        const double s = score[i];
        for (int k = 0; k < m; ++k) rank += (score[k] < s || (score[k] == s && k < i)) ? 1 : 0;
        chosen[i] = rank < m_sel ? 1 : 0;
    }
    group_sync<ONE_WARP>();
    if (i < m && chosen[i] && sel) {
        int pos = 0;
        for (int k = 0; k < i; ++k) pos += chosen[k];
        sel[pos] = i;
    }
}

// Idx: the type the column and position tables are held in (int32 in global memory; uint8 when cached in shared memory)
template <bool ONE_WARP, typename Idx>
__device__ __forceinline__ void bulyan_select_body(const double* sorted_d, const Idx* sorted_j, const Idx* pos_t,
                                                   int m, int f, int32_t* sel) {
    __shared__ unsigned char alive[kMaxRows];
    __shared__ double best_s[32];
    __shared__ int best_i[32];
    __shared__ int picked;
    const int i = threadIdx.x;
    const int lane = i & 31, warp = i >> 5;
    const int nwarps = ONE_WARP ? 1 : (int)(blockDim.x >> 5);
    const bool mine = i < m;
    if (i < kMaxRows) alive[i] = mine ? 1 : 0;
    const double* dist = sorted_d + (int64_t)i * m;   // row i's other rows, closest first (self last)
    const Idx* col = sorted_j + (int64_t)i * m;

    // round 0: the nb closest rows, added in ascending order
    int nb = krum_neighbours(m, f);
    int last = nb - 1;        // position of the farthest counted entry; every remaining entry up to it is counted
    int counted = nb;
    double sum = 0.0;
    if (mine)
        for (int k = 0; k < nb; ++k) sum += dist[k];
    group_sync<ONE_WARP>();

    const int theta = m - 2 * f;
    for (int round = 0; round < theta; ++round) {
        // argmin over (score, index) among the remaining rows
        // (Inf - Inf from a non-finite row gives a NaN sum: it competes as +Inf, so the winner is always a remaining row)
        double s = (mine && alive[i]) ? nan_to_inf(sum) : CUDART_INF;
        int idx = (mine && alive[i]) ? i : 0x7fffffff;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const double s2 = __shfl_down_sync(0xffffffffu, s, o);
            const int i2 = __shfl_down_sync(0xffffffffu, idx, o);
            if (s2 < s || (s2 == s && i2 < idx)) { s = s2; idx = i2; }
        }
        if (lane == 0) { best_s[warp] = s; best_i[warp] = idx; }
        group_sync<ONE_WARP>();
        if (warp == 0) {
            s = lane < nwarps ? best_s[lane] : CUDART_INF;
            idx = lane < nwarps ? best_i[lane] : 0x7fffffff;
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) {
                const double s2 = __shfl_down_sync(0xffffffffu, s, o);
                const int i2 = __shfl_down_sync(0xffffffffu, idx, o);
                if (s2 < s || (s2 == s && i2 < idx)) { s = s2; idx = i2; }
            }
            if (lane == 0) {
                picked = idx;
                sel[round] = idx;
                alive[idx] = 0;
            }
        }
        group_sync<ONE_WARP>();
        const int gone = picked;
        const int remaining = m - round - 1;
        const int nb_next = remaining >= 1 ? krum_neighbours(remaining, f) : 0;
        if (mine && alive[i] && remaining >= 1) {
            // the removed row leaves the sum if it was counted
            const int q = pos_t[(int64_t)gone * m + i];
            double left_q = 0.0, left_far = 0.0;
            if (q <= last) {
                left_q = dist[q];
                --counted;
                if (q == last) {
                    do { --last; } while (last >= 0 && !alive[col[last]]);
                }
            }
            // then the count follows nb: drop the farthest counted entry, or take the next remaining one.  The first
            // such step (the usual one: nb shrinks by one a round) is taken before either distance is used, so that
            // the two loads travel together; the subtractions keep their order.
            if (counted > nb_next) {
                left_far = dist[last];
                --counted;
                do { --last; } while (last >= 0 && !alive[col[last]]);
            }
            sum -= left_q;
            sum -= left_far;
            while (counted > nb_next) {
                sum -= dist[last];
                --counted;
                do { --last; } while (last >= 0 && !alive[col[last]]);
            }
            while (counted < nb_next) {
                do { ++last; } while (last < m - 1 && !alive[col[last]]);
                sum += dist[last];
                ++counted;
            }
            if (counted == 0) sum = 0.0;
            // Few neighbours left: add them afresh in ascending order.  With one neighbour two mutually
            // closest rows must tie exactly (their score is the same distance), which running
            // subtractions would blur in the last bit.
            if (nb_next <= kFreshSumBelow) {
                sum = 0.0;
                int seen = 0;
                for (int k = 0; seen < nb_next && k < m - 1; ++k) {
                    if (alive[col[k]]) {
                        sum += dist[k];
                        ++seen;
                    }
                }
            }
        }
        nb = nb_next;
        group_sync<ONE_WARP>();
    }
    (void)nb;
}

__global__ void __launch_bounds__(1024)
multikrum_select_kernel(const double* __restrict__ sorted_d, int m, int f, int m_sel, int32_t* __restrict__ sel,
                        double* __restrict__ scores_out) {
    multikrum_select_body<false>(sorted_d, m, f, m_sel, sel, scores_out);
}

__global__ void __launch_bounds__(1024)
bulyan_select_kernel(const double* __restrict__ sorted_d, const int32_t* __restrict__ sorted_j,
                     const int32_t* __restrict__ pos_t, int m, int f, int32_t* __restrict__ sel) {
    bulyan_select_body<false>(sorted_d, sorted_j, pos_t, m, f, sel);
}

// Up to 256 rows the two index tables fit in shared memory as bytes (2 m^2 <= 128 KB), and up to 128 rows the ranked
// distances do as well (8 m^2 <= 128 KB).  A round is a chain of dependent look-ups (which position did the removed
// row have in my list? which is my next remaining neighbour? what is that distance?); from shared memory each costs
// tens of cycles instead of a trip to L2 (measured per call: 165 -> 148 microseconds at 75 rows with everything
// cached, 360 -> 340 at 225 rows with the tables alone: the three CTA-wide barriers of a round remain).
constexpr int kCachedSelectRows = 256;
constexpr int kCachedDistRows = 128;
__global__ void __launch_bounds__(kCachedSelectRows)
bulyan_select_cached_kernel(const double* __restrict__ sorted_d, const int32_t* __restrict__ sorted_j,
                            const int32_t* __restrict__ pos_t, int m, int f, int32_t* __restrict__ sel) {
    extern __shared__ __align__(8) uint8_t tables[];   // [m*m] distances (m <= 128 only), [m*m] columns, [m*m] positions
    const bool with_dist = m <= kCachedDistRows;
    double* dist_s = reinterpret_cast<double*>(tables);
    uint8_t* col8 = tables + (with_dist ? (size_t)m * m * sizeof(double) : 0);
    uint8_t* pos8 = col8 + m * m;
    for (int e = threadIdx.x; e < m * m; e += blockDim.x) {
        col8[e] = (uint8_t)sorted_j[e];
        pos8[e] = (uint8_t)pos_t[e];
        if (with_dist) dist_s[e] = sorted_d[e];
    }
    __syncthreads();
    bulyan_select_body<false>(with_dist ? dist_s : sorted_d, col8, pos8, m, f, sel);
}

// m <= 16: everything between the distance pass and the final mean / order statistics in one CTA:
// the per-CTA pair partials of the direct distance kernel are added up (one warp per pair, lanes
// round-robin over the partials, then a fixed shuffle tree), every row's distances are ranked, the
// selection runs on the lists in shared memory, and the chosen indices are mapped through the row
// list when there is one.  The device status word is cleared on the way (unless `status` is null).
constexpr int kSmallRows = 16;
constexpr int kSmallThreads = 1024;
constexpr int kSmallPartialsPerLane = 19;   // covers the direct distance kernel's 4 CTAs per SM

template <bool BULYAN>
__global__ void __launch_bounds__(kSmallThreads)
krum_small_kernel(const double* __restrict__ partial, int nblocks, int m, int f, int m_sel,
                  const int32_t* __restrict__ rows, int32_t* __restrict__ sel, int32_t* __restrict__ mapped,
                  double* __restrict__ scores_out, int* __restrict__ status) {
    __shared__ double dmat[kSmallRows][kSmallRows];
    __shared__ double s_sorted_d[kSmallRows * kSmallRows];
    __shared__ int32_t s_sorted_j[kSmallRows * kSmallRows];
    __shared__ int32_t s_pos_t[kSmallRows * kSmallRows];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid == 0 && status) *status = 0;   // null: the distance kernel before this one owns the status word

    const int np = m * (m - 1) / 2;
    for (int p = warp; p < np; p += kSmallThreads / 32) {
        // all of a lane's partials are requested before the first is added (the order of the additions stays)
        double part[kSmallPartialsPerLane];
#pragma unroll
        for (int k = 0; k < kSmallPartialsPerLane; ++k) {
            const int b = lane + 32 * k;
            part[k] = b < nblocks ? partial[(int64_t)b * np + p] : 0.0;
        }
        double v = 0.0;
#pragma unroll
        for (int k = 0; k < kSmallPartialsPerLane; ++k)
            if (lane + 32 * k < nblocks) v += part[k];
        for (int b = lane + 32 * kSmallPartialsPerLane; b < nblocks; b += 32) v += partial[(int64_t)b * np + p];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) v += __shfl_down_sync(0xffffffffu, v, o);
        if (lane == 0) {
            int i = 0, rem = p;
            while (rem >= m - 1 - i) { rem -= m - 1 - i; ++i; }
            const int j = i + 1 + rem;
            dmat[i][j] = nan_to_inf(v);   // non-finite rows: Inf - Inf between two of them is as far as it gets
            dmat[j][i] = nan_to_inf(v);
        }
    }
    if (tid < m) dmat[tid][tid] = CUDART_INF;   // a row never counts itself: it goes to the end of its own list
    __syncthreads();

    if (tid < m * m) {
        const int i = tid / m, j = tid - i * m;
        int rank;
        if (j == i) {
            rank = m - 1;
        } else {
            const double v = dmat[i][j];
            rank = 0;
            for (int k = 0; k < m; ++k) {
                if (k == i) continue;
                const double u = dmat[i][k];
                rank += (u < v || (u == v && k < j)) ? 1 : 0;
            }
        }
        s_sorted_d[i * m + rank] = dmat[i][j];
        s_sorted_j[i * m + rank] = j;
        s_pos_t[j * m + i] = rank;
    }
    __syncthreads();

    // m <= 16 rows: the selection runs in the first warp alone
    const int count = BULYAN ? m - 2 * f : m_sel;
    if (warp == 0) {
        if (BULYAN) bulyan_select_body<true>(s_sorted_d, s_sorted_j, s_pos_t, m, f, sel);
        else multikrum_select_body<true>(s_sorted_d, m, f, m_sel, sel, scores_out);
    }
    if (rows && mapped) {
        __syncthreads();
        if (tid < count) mapped[tid] = rows[sel[tid]];
    }
}

__global__ void map_indices_kernel(const int32_t* __restrict__ idx, const int32_t* __restrict__ map, int cnt,
                                   int32_t* __restrict__ out) {
    int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k < cnt) out[k] = map[idx[k]];
}

// dst[member[k]] = src[k] for the G votes (votes were produced in set order; give them back in group order)
__global__ void scatter_by_set_order_kernel(const int32_t* __restrict__ src, const __grid_constant__ SetTable sets,
                                            int G, int32_t* __restrict__ dst) {
    int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k < G) dst[sets.member[k]] = src[k];
}

// Rows chosen inside one vote set (local indices) -> vote indices and worker ids
__global__ void map_set_selection_kernel(const int32_t* __restrict__ local, int cnt,
                                         const __grid_constant__ SetTable sets, int set_begin,
                                         const int32_t* __restrict__ winner_in_set_order,
                                         int32_t* __restrict__ sel_votes, int32_t* __restrict__ sel_workers) {
    int k = blockIdx.x * blockDim.x + threadIdx.x;
    if (k >= cnt) return;
    const int pos = set_begin + local[k];
    if (sel_votes) sel_votes[k] = sets.member[pos];
    if (sel_workers) sel_workers[k] = winner_in_set_order[pos];
}

int round_up_warp(int m) { return (m + 31) / 32 * 32; }

}  // namespace

size_t select_ws_bytes(int m) {
    return align_up((size_t)m * m * sizeof(double)) + 2 * align_up((size_t)m * m * sizeof(int32_t)) +
           align_up((size_t)m * sizeof(double));
}

detox_status launch_multikrum_select(const double* D, int m, int f, int m_sel, int32_t* sel_dev, double* scores_dev,
                                     void* ws, cudaStream_t s) {
    SelectWs w = carve(ws, m);
    rank_rows_kernel<<<m, 256, (size_t)m * sizeof(double), s>>>(D, m, w.sorted_d, w.sorted_j, w.pos_t);
    detox_status st = launch_status();
    if (st != DETOX_OK) return st;
    multikrum_select_kernel<<<1, round_up_warp(m), 0, s>>>(w.sorted_d, m, f, m_sel, sel_dev, scores_dev);
    return launch_status();
}

detox_status launch_bulyan_select(const double* D, int m, int f, int32_t* sel_dev, void* ws, cudaStream_t s) {
    SelectWs w = carve(ws, m);
    rank_rows_kernel<<<m, 256, (size_t)m * sizeof(double), s>>>(D, m, w.sorted_d, w.sorted_j, w.pos_t);
    detox_status st = launch_status();
    if (st != DETOX_OK) return st;
    if (m <= kCachedSelectRows) {
        const size_t smem = (size_t)2 * m * m + (m <= kCachedDistRows ? (size_t)m * m * sizeof(double) : 0);
        if (cudaFuncSetAttribute(bulyan_select_cached_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
            cudaSuccess)
            return DETOX_ERR_CUDA;
        bulyan_select_cached_kernel<<<1, round_up_warp(m), smem, s>>>(w.sorted_d, w.sorted_j, w.pos_t, m, f, sel_dev);
    } else {
        bulyan_select_kernel<<<1, round_up_warp(m), 0, s>>>(w.sorted_d, w.sorted_j, w.pos_t, m, f, sel_dev);
    }
    return launch_status();
}

detox_status launch_krum_small(bool bulyan, const double* partial, int nblocks, int m, int f, int m_sel,
                               const int32_t* rows_dev, int32_t* sel_dev, int32_t* mapped_dev, double* scores_dev,
                               int* status_dev, cudaStream_t s) {
    if (m < 2 || m > kSmallRows) return DETOX_ERR_UNSUPPORTED;
    if (bulyan)
        krum_small_kernel<true><<<1, kSmallThreads, 0, s>>>(partial, nblocks, m, f, m_sel, rows_dev, sel_dev, mapped_dev,
                                                           scores_dev, status_dev);
    else
        krum_small_kernel<false><<<1, kSmallThreads, 0, s>>>(partial, nblocks, m, f, m_sel, rows_dev, sel_dev, mapped_dev,
                                                            scores_dev, status_dev);
    return launch_status();
}

detox_status launch_map_indices(const int32_t* idx, const int32_t* map, int cnt, int32_t* out, cudaStream_t s) {
    if (cnt <= 0) return DETOX_OK;
    map_indices_kernel<<<(cnt + 127) / 128, 128, 0, s>>>(idx, map, cnt, out);
    return launch_status();
}

detox_status launch_scatter_by_set_order(const int32_t* src, const SetTable& sets, int G, int32_t* dst,
                                         cudaStream_t s) {
    scatter_by_set_order_kernel<<<(G + 127) / 128, 128, 0, s>>>(src, sets, G, dst);
    return launch_status();
}

detox_status launch_map_set_selection(const int32_t* local, int cnt, const SetTable& sets, int set_begin,
                                      const int32_t* winner_in_set_order, int32_t* sel_votes, int32_t* sel_workers,
                                      cudaStream_t s) {
    if (cnt <= 0 || (!sel_votes && !sel_workers)) return DETOX_OK;
    map_set_selection_kernel<<<(cnt + 127) / 128, 128, 0, s>>>(local, cnt, sets, set_begin, winner_in_set_order,
                                                               sel_votes, sel_workers);
    return launch_status();
}

}  // namespace detox
