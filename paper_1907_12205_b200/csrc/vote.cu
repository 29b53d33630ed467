// Filtering step of DETOX (Section 3; Algorithm 1, "Filtering step"): majority vote inside each node
// group, on bitwise equality of whole d-vectors.
//
// One streaming pass.  A strict majority of the whole vectors, when it exists, is also a strict
// majority on every 16-byte piece, and it is then the only one there.  So each thread compares the
// r members on its own piece, writes that piece's local majority value (or zeros) to Z at once, and
// ORs "member a differs from member b" bits into a per-group word.  After the pass the bits tell
// whether a global majority exists; only groups without one have their Z row cleared again.
// Traffic: n*d*4 bytes read, G*d*4 bytes written, once.
#include "common.cuh"
#include "sortnet.cuh"

namespace detox {

namespace {

constexpr int kVoteThreads = 256;

template <int R>
struct VoteShape {
    static constexpr int kPairs = R * (R - 1) / 2;
    static constexpr int kWords = kPairs == 0 ? 1 : (kPairs + 31) / 32;
    // pieces per thread and item: enough independent 16-byte loads in flight per thread
    static constexpr int kUnroll = R <= 3 ? 4 : (R <= 7 ? 2 : 1);
};

__host__ __device__ constexpr int pair_index(int r, int a, int b) {  // a < b
    return a * (2 * r - a - 1) / 2 + (b - a - 1);
}

template <int VEC>
struct Piece;
template <>
struct Piece<4> {
    uint4 v;
    __device__ __forceinline__ bool differs(const Piece& o) const {
        return ((v.x ^ o.v.x) | (v.y ^ o.v.y) | (v.z ^ o.v.z) | (v.w ^ o.v.w)) != 0u;
    }
    __device__ __forceinline__ void clear() { v = make_uint4(0u, 0u, 0u, 0u); }
    __device__ __forceinline__ void load(const float* p, int valid) {
        if (valid >= 4) {
            v = ld_stream_u4(p);
        } else {
            v.x = valid > 0 ? ld_stream_u1(p) : 0u;
            v.y = valid > 1 ? ld_stream_u1(p + 1) : 0u;
            v.z = valid > 2 ? ld_stream_u1(p + 2) : 0u;
            v.w = 0u;
        }
    }
    __device__ __forceinline__ void store(float* p, int valid) const {
        if (valid >= 4) {
            st_stream_u4(p, v);
        } else {
            uint32_t* q = reinterpret_cast<uint32_t*>(p);
            if (valid > 0) q[0] = v.x;
            if (valid > 1) q[1] = v.y;
            if (valid > 2) q[2] = v.z;
        }
    }
};
template <>
struct Piece<1> {
    uint32_t v;
    __device__ __forceinline__ bool differs(const Piece& o) const { return v != o.v; }
    __device__ __forceinline__ void clear() { v = 0u; }
    __device__ __forceinline__ void load(const float* p, int valid) { v = valid > 0 ? ld_stream_u1(p) : 0u; }
    __device__ __forceinline__ void store(float* p, int valid) const {
        if (valid > 0) *reinterpret_cast<uint32_t*>(p) = v;
    }
};

template <int R, int VEC, bool WRITE_Z>
__global__ void __launch_bounds__(kVoteThreads)
vote_kernel(const float* __restrict__ X, int64_t ld, int64_t d, int64_t tiles_per_group,
            const __grid_constant__ IdTable members, float* __restrict__ Z, int64_t ldz,
            uint32_t* __restrict__ pairdiff) {
    using Shape = VoteShape<R>;
    constexpr int U = Shape::kUnroll;
    constexpr int64_t kTile = (int64_t)kVoteThreads * VEC * U;

    const int64_t item = blockIdx.x;
    const int g = (int)(item / tiles_per_group);
    const int64_t tile = item - (int64_t)g * tiles_per_group;

    const float* row[R];
#pragma unroll
    for (int a = 0; a < R; ++a) row[a] = X + (int64_t)members.id[g * R + a] * ld;

    Piece<VEC> v[U][R];
    int valid[U];
    int64_t col[U];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        col[u] = tile * kTile + ((int64_t)u * kVoteThreads + threadIdx.x) * VEC;
        int64_t left = d - col[u];
        valid[u] = left >= VEC ? VEC : (left > 0 ? (int)left : 0);
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
#pragma unroll
        for (int a = 0; a < R; ++a) {
            if (valid[u] > 0) v[u][a].load(row[a] + col[u], valid[u]);
            else v[u][a].clear();
        }
    }

    uint32_t diff[Shape::kWords];
#pragma unroll
    for (int w = 0; w < Shape::kWords; ++w) diff[w] = 0u;

#pragma unroll
    for (int u = 0; u < U; ++u) {
        uint32_t loc[Shape::kWords];
#pragma unroll
        for (int w = 0; w < Shape::kWords; ++w) loc[w] = 0u;
#pragma unroll
        for (int a = 0; a < R; ++a) {
#pragma unroll
            for (int b = a + 1; b < R; ++b) {
                const int p = pair_index(R, a, b);
                if (v[u][a].differs(v[u][b])) loc[p >> 5] |= 1u << (p & 31);
            }
        }
#pragma unroll
        for (int w = 0; w < Shape::kWords; ++w) diff[w] |= loc[w];

        if (WRITE_Z) {
            // local majority: the first member that agrees with more than r/2 members (itself included)
            Piece<VEC> pick;
            pick.clear();
#pragma unroll
            for (int a = R - 1; a >= 0; --a) {
                int agree = 1;
#pragma unroll
                for (int b = 0; b < R; ++b) {
                    if (b == a) continue;
                    const int p = a < b ? pair_index(R, a, b) : pair_index(R, b, a);
                    agree += ((loc[p >> 5] >> (p & 31)) & 1u) ? 0 : 1;
                }
                if (2 * agree > R) pick = v[u][a];
            }
            if (valid[u] > 0) pick.store(Z + (int64_t)g * ldz + col[u], valid[u]);
        }
    }

    // one OR per warp and word, and only when it would set a new bit
#pragma unroll
    for (int w = 0; w < Shape::kWords; ++w) {
        uint32_t bits = __reduce_or_sync(0xffffffffu, diff[w]);
        if ((threadIdx.x & 31) == 0 && bits != 0u) {
            uint32_t* word = pairdiff + (int64_t)g * kPairWords + w;
            uint32_t seen = *reinterpret_cast<volatile uint32_t*>(word);
            if (bits & ~seen) atomicOr(word, bits);
        }
    }
}

// One thread per group: read the "differs" bits, find the class with more than r/2 members.
// none_flag (optional): set to 1 when some group has no majority.
__global__ void vote_finalize_kernel(int G, int r, const __grid_constant__ IdTable members,
                                     const uint32_t* __restrict__ pairdiff, int32_t* __restrict__ winner,
                                     int* __restrict__ none_flag = nullptr) {
    int g = blockIdx.x * blockDim.x + threadIdx.x;
    if (g >= G) return;
    const uint32_t* bits = pairdiff + (int64_t)g * kPairWords;
    int win = -1;
    for (int a = 0; a < r && win < 0; ++a) {
        int agree = 1;
        int lowest = members.id[g * r + a];
        for (int b = 0; b < r; ++b) {
            if (b == a) continue;
            int p = a < b ? pair_index(r, a, b) : pair_index(r, b, a);
            if (((bits[p >> 5] >> (p & 31)) & 1u) == 0u) {
                ++agree;
                int idb = members.id[g * r + b];
                lowest = idb < lowest ? idb : lowest;
            }
        }
        if (2 * agree > r) win = lowest;
    }
    winner[g] = win;
    if (none_flag != nullptr && win < 0) *none_flag = 1;
}

// The votes of groups of three as rows of Z, written only when *gate is not zero (the distance pass that votes while
// it reads keeps no votes; when its result cannot be used the pass is repeated on stored ones).  Groups without a
// majority get their piece-local values here and are cleared by vote_clear_kernel afterwards.
__global__ void __launch_bounds__(kVoteThreads)
vote_store_gated_kernel(const float* __restrict__ X, int64_t ld, int64_t d, const __grid_constant__ IdTable members,
                        float* __restrict__ Z, int64_t ldz, const int* __restrict__ gate) {
    if (*gate == 0) return;
    const int g = blockIdx.y;
    const float* row[3];
#pragma unroll
    for (int a = 0; a < 3; ++a) row[a] = X + (int64_t)members.id[g * 3 + a] * ld;
    for (int64_t col = ((int64_t)blockIdx.x * kVoteThreads + threadIdx.x) * 4; col < d;
         col += (int64_t)gridDim.x * kVoteThreads * 4) {
        const int64_t left = d - col;
        const int valid = left >= 4 ? 4 : (int)left;
        Piece<4> v[3];
#pragma unroll
        for (int a = 0; a < 3; ++a) v[a].load(row[a] + col, valid);
        Piece<4> pick;
        pick.clear();
        if (!v[1].differs(v[2])) pick = v[1];
        if (!v[0].differs(v[1]) || !v[0].differs(v[2])) pick = v[0];
        pick.store(Z + (int64_t)g * ldz + col, valid);
    }
}

// Clears the vote of every group that turned out to have no majority (rare).
__global__ void vote_clear_kernel(const int32_t* __restrict__ winner, float* __restrict__ Z, int64_t ldz,
                                  int64_t d) {
    int g = blockIdx.y;
    if (winner[g] >= 0) return;
    float* z = Z + (int64_t)g * ldz;
    for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < d; c += (int64_t)gridDim.x * blockDim.x)
        z[c] = 0.0f;
}

// ---------------------------------------------------------------------------------------------
// Vote fused with A_0 = mean (Algorithm 1's filtering step + Algorithm 2, step 3, in one pass): the
// piece-local majority of every group of a vote set is added up in the set's member order and only
// the set mean is written, so the votes themselves never travel to memory (n*d*4 bytes read,
// S*d*4 written).  The "differs" bits are collected as in vote_kernel.  Sets that contain a group
// without a majority are recomputed afterwards from the winners' rows (vote_mean_fix_kernel).
// ---------------------------------------------------------------------------------------------
template <int VEC>
struct PieceSum;
template <>
struct PieceSum<4> {
    float4 a;
    __device__ __forceinline__ void zero() { a = make_float4(0.f, 0.f, 0.f, 0.f); }
    __device__ __forceinline__ void add(const Piece<4>& p) {
        a.x += __uint_as_float(p.v.x); a.y += __uint_as_float(p.v.y);
        a.z += __uint_as_float(p.v.z); a.w += __uint_as_float(p.v.w);
    }
    __device__ __forceinline__ void store_mean(float* dst, float k, int valid) const {
        const float4 m = make_float4(a.x / k, a.y / k, a.z / k, a.w / k);
        if (valid >= 4) { st_stream_f4(dst, m); return; }
        if (valid > 0) dst[0] = m.x;
        if (valid > 1) dst[1] = m.y;
        if (valid > 2) dst[2] = m.z;
    }
};
template <>
struct PieceSum<1> {
    float a;
    __device__ __forceinline__ void zero() { a = 0.f; }
    __device__ __forceinline__ void add(const Piece<1>& p) { a += __uint_as_float(p.v); }
    __device__ __forceinline__ void store_mean(float* dst, float k, int valid) const {
        if (valid > 0) dst[0] = a / k;
    }
};

template <int R, int VEC>
__global__ void __launch_bounds__(kVoteThreads)
vote_mean_kernel(const float* __restrict__ X, int64_t ld, int64_t d, const __grid_constant__ IdTable members,
                 const __grid_constant__ SetTable sets, float* __restrict__ M, int64_t ldm,
                 uint32_t* __restrict__ pairdiff) {
    using Shape = VoteShape<R>;
    const int s = blockIdx.y;
    const int64_t col = ((int64_t)blockIdx.x * kVoteThreads + threadIdx.x) * VEC;
    const int64_t left = d - col;
    const int valid = left >= VEC ? VEC : (left > 0 ? (int)left : 0);
    const int b = sets.offset[s], e = sets.offset[s + 1];

    PieceSum<VEC> sum;
    sum.zero();
#pragma unroll 2
    for (int t = b; t < e; ++t) {
        const int g = sets.member[t];
        Piece<VEC> v[R];
#pragma unroll
        for (int a = 0; a < R; ++a) {
            if (valid > 0) v[a].load(X + (int64_t)members.id[g * R + a] * ld + col, valid);
            else v[a].clear();
        }
        uint32_t loc[Shape::kWords];
#pragma unroll
        for (int w = 0; w < Shape::kWords; ++w) loc[w] = 0u;
#pragma unroll
        for (int a = 0; a < R; ++a) {
#pragma unroll
            for (int c = a + 1; c < R; ++c) {
                const int p = pair_index(R, a, c);
                if (v[a].differs(v[c])) loc[p >> 5] |= 1u << (p & 31);
            }
        }
        Piece<VEC> pick;
        pick.clear();
#pragma unroll
        for (int a = R - 1; a >= 0; --a) {
            int agree = 1;
#pragma unroll
            for (int c = 0; c < R; ++c) {
                if (c == a) continue;
                const int p = a < c ? pair_index(R, a, c) : pair_index(R, c, a);
                agree += ((loc[p >> 5] >> (p & 31)) & 1u) ? 0 : 1;
            }
            if (2 * agree > R) pick = v[a];
        }
        sum.add(pick);
#pragma unroll
        for (int w = 0; w < Shape::kWords; ++w) {
            const uint32_t bits = __reduce_or_sync(0xffffffffu, loc[w]);
            if ((threadIdx.x & 31) == 0 && bits != 0u) {
                uint32_t* word = pairdiff + (int64_t)g * kPairWords + w;
                const uint32_t seen = *reinterpret_cast<volatile uint32_t*>(word);
                if (bits & ~seen) atomicOr(word, bits);
            }
        }
    }
    if (valid > 0) sum.store_mean(M + (int64_t)s * ldm + col, (float)(e - b), valid);
}

// Recomputes the mean of every set that holds a group without a majority: such a group counts as a zero
// row, the others contribute their winner's row (bitwise the vote).  Same order of additions.
__global__ void vote_mean_fix_kernel(const float* __restrict__ X, int64_t ld, int64_t d,
                                     const __grid_constant__ SetTable sets, const int32_t* __restrict__ winner,
                                     float* __restrict__ M, int64_t ldm) {
    const int s = blockIdx.y;
    const int b = sets.offset[s], e = sets.offset[s + 1];
    bool broken = false;
    for (int t = b; t < e; ++t) broken |= winner[sets.member[t]] < 0;
    if (!broken) return;
    for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < d; c += (int64_t)gridDim.x * blockDim.x) {
        float acc = 0.f;
        for (int t = b; t < e; ++t) {
            const int w = winner[sets.member[t]];
            acc += w >= 0 ? X[(int64_t)w * ld + c] : 0.f;
        }
        M[(int64_t)s * ldm + c] = acc / (float)(e - b);
    }
}

// ---------------------------------------------------------------------------------------------
// Vote, A_0 = mean and a coordinate-wise A_1 over the set means in one pass (Algorithm 1's filtering step + the
// whole of Algorithm 2 when A_1 works coordinate by coordinate): a CTA covers ALL vote sets for its 128 columns, the
// S set means meet in shared memory and A_1 is applied to them at once, so that neither the votes nor the set means
// travel to memory (n*d*4 bytes read, d*4 written).  The set means are formed exactly as in vote_mean_kernel and
// A_1 exactly as in the order-statistic kernels, so the result is bitwise the one of the separate kernels.
//   mode == 0: median;  mode < 0: mean of the middle -mode values (S + mode even);  mode == kSelectMean: mean.
// SM = size of the sorting network: S rounded up (same parity) with (SM - S) / 2 lowest and as many highest keys.
// If a group turns out to have no majority, the output is recomputed from the winners' rows afterwards
// (vote_mean_select_fix_kernel).
// ---------------------------------------------------------------------------------------------
constexpr int kSelectMean = 0x40000000;
constexpr int kMaxFusedSets = 16;

// A_1 over v[0..S-1] (SM >= S, SM - S even).
template <int SM>
__device__ __forceinline__ float select_over_sets(const float (&v)[SM], int S, int mode) {
    if (mode == kSelectMean) {
        float acc = 0.f;
#pragma unroll
        for (int i = 0; i < SM; ++i)
            if (i < S) acc += v[i];
        return acc / (float)S;
    }
    const int pad = (SM - S) >> 1;
    int32_t key[SM];
#pragma unroll
    for (int i = 0; i < SM; ++i)
        key[i] = i < S ? key_of_bits(__float_as_uint(v[i])) : (i - S < pad ? (int32_t)0x80000000 : 0x7fffffff);
    sort_registers<SM>(key);
    if (mode == 0) {
        if (SM & 1) return float_of_key(key[SM / 2]);
        return (float_of_key(key[SM / 2 > 0 ? SM / 2 - 1 : 0]) + float_of_key(key[SM / 2])) * 0.5f;
    }
    const int cnt = -mode, L = pad + ((S - cnt) >> 1);
    float acc = 0.f;
#pragma unroll
    for (int i = 0; i < SM; ++i)
        if (i >= L && i < L + cnt) acc += float_of_key(key[i]);
    return acc / (float)cnt;
}

// CTA = 64 column pieces (256 columns) x S sets: the two warps of row y form set y's mean of the CTA's 256 columns exactly as
// vote_mean_kernel does (few registers, all loads of a group in flight, full occupancy), leaves it in shared memory,
// and after one barrier the first 256 threads apply A_1 to the S means of one column each.
constexpr int kFusedPieces = 64;   // (32 pieces: 1.83 ms on the 105 x 28 M configuration, 64: 1.75 ms)
template <int R, int SM>
__global__ void __launch_bounds__(kFusedPieces * kMaxFusedSets)
vote_mean_select_kernel(const float* __restrict__ X, int64_t ld, int64_t d, const __grid_constant__ IdTable members,
                        const __grid_constant__ SetTable sets, int S, int mode, float* __restrict__ out,
                        uint32_t* __restrict__ pairdiff) {
    using Shape = VoteShape<R>;
    __shared__ __align__(16) float means[kMaxFusedSets][kFusedPieces * 4];
    const int s = threadIdx.y;
    const int64_t col0 = (int64_t)blockIdx.x * (kFusedPieces * 4);
    const int64_t col = col0 + threadIdx.x * 4;
    const int64_t left = d - col;
    const int valid = left >= 4 ? 4 : (left > 0 ? (int)left : 0);
    // (with fewer than four sets the CTA still has four rows of threads: the spare ones only help with A_1)
    const int b = s < S ? sets.offset[s] : 0, e = s < S ? sets.offset[s + 1] : 0;

    PieceSum<4> sum;
    sum.zero();
#pragma unroll 2
    for (int t = b; t < e; ++t) {
        const int g = sets.member[t];
        Piece<4> v[R];
#pragma unroll
        for (int a = 0; a < R; ++a) {
            if (valid > 0) v[a].load(X + (int64_t)members.id[g * R + a] * ld + col, valid);
            else v[a].clear();
        }
        uint32_t loc[Shape::kWords];
#pragma unroll
        for (int w = 0; w < Shape::kWords; ++w) loc[w] = 0u;
#pragma unroll
        for (int a = 0; a < R; ++a) {
#pragma unroll
            for (int c = a + 1; c < R; ++c) {
                const int p = pair_index(R, a, c);
                if (v[a].differs(v[c])) loc[p >> 5] |= 1u << (p & 31);
            }
        }
        Piece<4> pick;
        pick.clear();
#pragma unroll
        for (int a = R - 1; a >= 0; --a) {
            int agree = 1;
#pragma unroll
            for (int c = 0; c < R; ++c) {
                if (c == a) continue;
                const int p = a < c ? pair_index(R, a, c) : pair_index(R, c, a);
                agree += ((loc[p >> 5] >> (p & 31)) & 1u) ? 0 : 1;
            }
            if (2 * agree > R) pick = v[a];
        }
        sum.add(pick);
#pragma unroll
        for (int w = 0; w < Shape::kWords; ++w) {
            const uint32_t bits = __reduce_or_sync(0xffffffffu, loc[w]);
            if ((threadIdx.x & 31) == 0 && bits != 0u) {
                uint32_t* word = pairdiff + (int64_t)g * kPairWords + w;
                const uint32_t seen = *reinterpret_cast<volatile uint32_t*>(word);
                if (bits & ~seen) atomicOr(word, bits);
            }
        }
    }
    const float k = (float)(e - b);
    if (s < S)
        *reinterpret_cast<float4*>(&means[s][threadIdx.x * 4]) = make_float4(sum.a.x / k, sum.a.y / k, sum.a.z / k, sum.a.w / k);
    __syncthreads();
    const int tid = threadIdx.y * kFusedPieces + threadIdx.x;
    if (tid >= kFusedPieces * 4 || col0 + tid >= d) return;
    float v[SM];
#pragma unroll
    for (int i = 0; i < SM; ++i) v[i] = i < S ? means[i][tid] : 0.f;
    out[col0 + tid] = select_over_sets<SM>(v, S, mode);
}

// After the winners are known: nothing to do unless some group has no majority (rare).  Then every coordinate is
// recomputed from the winners' rows: such a group counts as a zero row, the others contribute their winner's row
// (bitwise the vote), with the same order of additions and the same A_1.
template <int SM>
__global__ void vote_mean_select_fix_kernel(const float* __restrict__ X, int64_t ld, int64_t d,
                                            const __grid_constant__ SetTable sets, int S, int G,
                                            const int32_t* __restrict__ winner, int mode, float* __restrict__ out) {
    int broken = 0;
    for (int g = threadIdx.x; g < G; g += blockDim.x) broken |= winner[g] < 0;
    if (!__syncthreads_or(broken)) return;
    for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < d; c += (int64_t)gridDim.x * blockDim.x) {
        float mean[SM];
#pragma unroll
        for (int s = 0; s < SM; ++s) {
            mean[s] = 0.f;
            if (s < S) {
                const int b = sets.offset[s], e = sets.offset[s + 1];
                float acc = 0.f;
                for (int t = b; t < e; ++t) {
                    const int w = winner[sets.member[t]];
                    acc += w >= 0 ? X[(int64_t)w * ld + c] : 0.f;
                }
                mean[s] = acc / (float)(e - b);
            }
        }
        out[c] = select_over_sets<SM>(mean, S, mode);
    }
}

template <int R, int SM>
detox_status launch_vote_mean_select_rs(const float* X, int64_t ld, int G, int64_t d, const IdTable& members,
                                        const SetTable& sets, int S, int mode, float* out, int32_t* winner,
                                        uint32_t* pairdiff, cudaStream_t s) {
    const int64_t bx = ceil_div(d, (int64_t)kFusedPieces * 4);
    if (bx > 0x7fffffffLL) return DETOX_ERR_UNSUPPORTED;
    // at least four rows of threads, so that the 256 columns of a CTA all get their A_1
    const int by = S < 4 ? 4 : S;
    vote_mean_select_kernel<R, SM><<<(unsigned)bx, dim3(kFusedPieces, (unsigned)by), 0, s>>>(X, ld, d, members, sets, S, mode,
                                                                                         out, pairdiff);
    detox_status st = launch_status();
    if (st != DETOX_OK) return st;
    vote_finalize_kernel<<<(G + 127) / 128, 128, 0, s>>>(G, R, members, pairdiff, winner);
    if ((st = launch_status()) != DETOX_OK) return st;
    const unsigned fx = (unsigned)(ceil_div(d, 256) < 4 * kSMs ? ceil_div(d, 256) : 4 * kSMs);
    vote_mean_select_fix_kernel<SM><<<fx, 256, 0, s>>>(X, ld, d, sets, S, G, winner, mode, out);
    return launch_status();
}

template <int R>
detox_status launch_vote_mean_select_r(const float* X, int64_t ld, int G, int64_t d, const IdTable& members,
                                       const SetTable& sets, int S, int mode, float* out, int32_t* winner,
                                       uint32_t* pairdiff, cudaStream_t s) {
    // network sizes 7, 8, 15, 16: S rounded up with its parity kept
    if (S <= 8) {
        if (S & 1) return launch_vote_mean_select_rs<R, 7>(X, ld, G, d, members, sets, S, mode, out, winner, pairdiff, s);
        return launch_vote_mean_select_rs<R, 8>(X, ld, G, d, members, sets, S, mode, out, winner, pairdiff, s);
    }
    if (S & 1) return launch_vote_mean_select_rs<R, 15>(X, ld, G, d, members, sets, S, mode, out, winner, pairdiff, s);
    return launch_vote_mean_select_rs<R, 16>(X, ld, G, d, members, sets, S, mode, out, winner, pairdiff, s);
}

template <int VEC>
detox_status launch_vote_mean_vec(const float* X, int64_t ld, int r, int64_t d, const IdTable& members,
                                  const SetTable& sets, int S, float* M, int64_t ldm, uint32_t* pairdiff,
                                  cudaStream_t s) {
    int64_t bx = ceil_div(d, (int64_t)kVoteThreads * VEC);
    if (bx > 0x7fffffffLL || S > 65535) return DETOX_ERR_UNSUPPORTED;
    dim3 grid((unsigned)bx, (unsigned)S);
    switch (r) {
#define DETOX_CASE(R) \
    case R: vote_mean_kernel<R, VEC><<<grid, kVoteThreads, 0, s>>>(X, ld, d, members, sets, M, ldm, pairdiff); break;
        DETOX_CASE(1) DETOX_CASE(3) DETOX_CASE(5) DETOX_CASE(7) DETOX_CASE(9) DETOX_CASE(11) DETOX_CASE(13)
        DETOX_CASE(15)
#undef DETOX_CASE
        default: return DETOX_ERR_UNSUPPORTED;
    }
    return launch_status();
}

template <int R, int VEC>
detox_status launch_vote_r(const float* X, int64_t ld, int G, int64_t d, const IdTable& members, float* Z,
                           int64_t ldz, uint32_t* pairdiff, cudaStream_t s) {
    constexpr int64_t kTile = (int64_t)kVoteThreads * VEC * VoteShape<R>::kUnroll;
    int64_t tiles = ceil_div(d, kTile);
    int64_t items = tiles * G;
    if (items > 0x7fffffffLL) return DETOX_ERR_UNSUPPORTED;
    if (Z)
        vote_kernel<R, VEC, true><<<(unsigned)items, kVoteThreads, 0, s>>>(X, ld, d, tiles, members, Z, ldz, pairdiff);
    else
        vote_kernel<R, VEC, false><<<(unsigned)items, kVoteThreads, 0, s>>>(X, ld, d, tiles, members, Z, ldz, pairdiff);
    return launch_status();
}

template <int VEC>
detox_status launch_vote_vec(const float* X, int64_t ld, int G, int r, int64_t d, const IdTable& members,
                             float* Z, int64_t ldz, uint32_t* pairdiff, cudaStream_t s) {
    switch (r) {
        case 1: return launch_vote_r<1, VEC>(X, ld, G, d, members, Z, ldz, pairdiff, s);
        case 3: return launch_vote_r<3, VEC>(X, ld, G, d, members, Z, ldz, pairdiff, s);
        case 5: return launch_vote_r<5, VEC>(X, ld, G, d, members, Z, ldz, pairdiff, s);
        case 7: return launch_vote_r<7, VEC>(X, ld, G, d, members, Z, ldz, pairdiff, s);
        case 9: return launch_vote_r<9, VEC>(X, ld, G, d, members, Z, ldz, pairdiff, s);
        case 11: return launch_vote_r<11, VEC>(X, ld, G, d, members, Z, ldz, pairdiff, s);
        case 13: return launch_vote_r<13, VEC>(X, ld, G, d, members, Z, ldz, pairdiff, s);
        case 15: return launch_vote_r<15, VEC>(X, ld, G, d, members, Z, ldz, pairdiff, s);
        default: return DETOX_ERR_UNSUPPORTED;
    }
}

}  // namespace

size_t vote_ws_bytes(int n, int r) {
    int G = r > 0 ? n / r : 0;
    return align_up((size_t)G * kPairWords * sizeof(uint32_t));
}

detox_status launch_vote(const float* X, int64_t ld, int n, int r, int64_t d, const IdTable& members,
                         float* Z, int64_t ldz, int32_t* winner, void* ws, cudaStream_t s, size_t clear_before) {
    const int G = n / r;
    uint32_t* pairdiff = static_cast<uint32_t*>(ws);
    if (cudaMemsetAsync(static_cast<char*>(ws) - clear_before, 0,
                        clear_before + (size_t)G * kPairWords * sizeof(uint32_t), s) != cudaSuccess)
        return DETOX_ERR_CUDA;
    const bool vec = aligned16(X) && ld % 4 == 0 && (!Z || (aligned16(Z) && ldz % 4 == 0));
    detox_status st = vec ? launch_vote_vec<4>(X, ld, G, r, d, members, Z, ldz, pairdiff, s)
                          : launch_vote_vec<1>(X, ld, G, r, d, members, Z, ldz, pairdiff, s);
    if (st != DETOX_OK) return st;
    vote_finalize_kernel<<<(G + 127) / 128, 128, 0, s>>>(G, r, members, pairdiff, winner);
    if ((st = launch_status()) != DETOX_OK) return st;
    if (Z) {
        unsigned bx = (unsigned)(ceil_div(d, 256 * 8) < 64 ? ceil_div(d, 256 * 8) : 64);
        vote_clear_kernel<<<dim3(bx, (unsigned)G), 256, 0, s>>>(winner, Z, ldz, d);
        st = launch_status();
    }
    return st;
}

detox_status launch_vote_finalize(int n, int r, const IdTable& members, const void* ws, int32_t* winner, int* none_flag,
                                  cudaStream_t s) {
    const int G = n / r;
    vote_finalize_kernel<<<(G + 127) / 128, 128, 0, s>>>(G, r, members, static_cast<const uint32_t*>(ws), winner, none_flag);
    return launch_status();
}

detox_status launch_vote_store_gated(const float* X, int64_t ld, int n, int64_t d, const IdTable& members, float* Z,
                                     int64_t ldz, const int32_t* winner, const int* gate, cudaStream_t s) {
    if (!(aligned16(X) && ld % 4 == 0 && aligned16(Z) && ldz % 4 == 0)) return DETOX_ERR_UNSUPPORTED;
    const int G = n / 3;
    // a few waves of CTAs that stride over the columns: the launch that finds its gate closed should cost next to nothing
    const int64_t want = ceil_div(d, (int64_t)kVoteThreads * 4);
    const int64_t fill = ceil_div((int64_t)kSMs * 16, G);
    const unsigned bx = (unsigned)(want < fill ? want : fill);
    vote_store_gated_kernel<<<dim3(bx, (unsigned)G), kVoteThreads, 0, s>>>(X, ld, d, members, Z, ldz, gate);
    detox_status st = launch_status();
    if (st != DETOX_OK) return st;
    // (winner[g] < 0 only ever goes with *gate != 0, so the clearing needs no gate of its own)
    unsigned cx = (unsigned)(ceil_div(d, 256 * 8) < 64 ? ceil_div(d, 256 * 8) : 64);
    vote_clear_kernel<<<dim3(cx, (unsigned)G), 256, 0, s>>>(winner, Z, ldz, d);
    return launch_status();
}

detox_status launch_vote_mean(const float* X, int64_t ld, int n, int r, int64_t d, const IdTable& members,
                              const SetTable& sets, int S, float* M, int64_t ldm, int32_t* winner, void* ws,
                              cudaStream_t s, size_t clear_before) {
    const int G = n / r;
    uint32_t* pairdiff = static_cast<uint32_t*>(ws);
    if (cudaMemsetAsync(static_cast<char*>(ws) - clear_before, 0,
                        clear_before + (size_t)G * kPairWords * sizeof(uint32_t), s) != cudaSuccess)
        return DETOX_ERR_CUDA;
    const bool vec = aligned16(X) && ld % 4 == 0 && aligned16(M) && ldm % 4 == 0;
    detox_status st = vec ? launch_vote_mean_vec<4>(X, ld, r, d, members, sets, S, M, ldm, pairdiff, s)
                          : launch_vote_mean_vec<1>(X, ld, r, d, members, sets, S, M, ldm, pairdiff, s);
    if (st != DETOX_OK) return st;
    vote_finalize_kernel<<<(G + 127) / 128, 128, 0, s>>>(G, r, members, pairdiff, winner);
    if ((st = launch_status()) != DETOX_OK) return st;
    unsigned bx = (unsigned)(ceil_div(d, 256 * 8) < 64 ? ceil_div(d, 256 * 8) : 64);
    vote_mean_fix_kernel<<<dim3(bx, (unsigned)S), 256, 0, s>>>(X, ld, d, sets, winner, M, ldm);
    return launch_status();
}

bool vote_mean_select_supported(const float* X, int64_t ld, int r, int S, const float* out) {
    return (r == 1 || r == 3 || r == 5) && S >= 1 && S <= kMaxFusedSets && aligned16(X) && ld % 4 == 0 && aligned16(out);
}

detox_status launch_vote_mean_select(const float* X, int64_t ld, int n, int r, int64_t d, const IdTable& members,
                                     const SetTable& sets, int S, int beta, bool mean, float* out, int32_t* winner,
                                     void* ws, cudaStream_t s, size_t clear_before) {
    if (!vote_mean_select_supported(X, ld, r, S, out)) return DETOX_ERR_UNSUPPORTED;
    if (!mean && beta > 0) return DETOX_ERR_UNSUPPORTED;
    if (!mean && beta < 0 && (-beta > S || ((S + beta) & 1))) return DETOX_ERR_BAD_ARG;
    const int G = n / r;
    const int mode = mean ? kSelectMean : beta;
    uint32_t* pairdiff = static_cast<uint32_t*>(ws);
    if (cudaMemsetAsync(static_cast<char*>(ws) - clear_before, 0,
                        clear_before + (size_t)G * kPairWords * sizeof(uint32_t), s) != cudaSuccess)
        return DETOX_ERR_CUDA;
    switch (r) {
        case 1: return launch_vote_mean_select_r<1>(X, ld, G, d, members, sets, S, mode, out, winner, pairdiff, s);
        case 3: return launch_vote_mean_select_r<3>(X, ld, G, d, members, sets, S, mode, out, winner, pairdiff, s);
        case 5: return launch_vote_mean_select_r<5>(X, ld, G, d, members, sets, S, mode, out, winner, pairdiff, s);
        default: return DETOX_ERR_UNSUPPORTED;
    }
}

}  // namespace detox
