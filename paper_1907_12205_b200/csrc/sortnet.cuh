// Compile-time sorting networks for fixed sizes (Batcher's merge exchange, valid for any length),
// applied to register arrays.  Comparators are emitted one by one with constant indices, so the array
// never leaves registers and the compiler drops every comparator that cannot reach an output that
// is actually used (a median needs far fewer than a full sort).
#pragma once

#include <stdint.h>

#include <utility>

namespace detox {

// Number of comparators of the merge-exchange network on M inputs.
template <int M>
__host__ __device__ constexpr int merge_exchange_count() {
    int c = 0;
    for (int p = 1; p < M; p <<= 1)
        for (int k = p; k >= 1; k >>= 1)
            for (int j = k % p; j <= M - 1 - k; j += 2 * k) {
                const int imax = k - 1 < M - j - k - 1 ? k - 1 : M - j - k - 1;
                for (int i = 0; i <= imax; ++i)
                    if ((i + j) / (2 * p) == (i + j + k) / (2 * p)) ++c;
            }
    return c;
}

// The comparators (a < b, minimum goes to a) in network order, built once per M at compile time.
template <int M>
struct MergeExchangeNet {
    static constexpr int kCount = merge_exchange_count<M>();
    int16_t a[kCount > 0 ? kCount : 1];
    int16_t b[kCount > 0 ? kCount : 1];
    __host__ __device__ constexpr MergeExchangeNet() : a{}, b{} {
        int c = 0;
        for (int p = 1; p < M; p <<= 1)
            for (int k = p; k >= 1; k >>= 1)
                for (int j = k % p; j <= M - 1 - k; j += 2 * k) {
                    const int imax = k - 1 < M - j - k - 1 ? k - 1 : M - j - k - 1;
                    for (int i = 0; i <= imax; ++i)
                        if ((i + j) / (2 * p) == (i + j + k) / (2 * p)) {
                            a[c] = (int16_t)(i + j);
                            b[c] = (int16_t)(i + j + k);
                            ++c;
                        }
                }
    }
};

template <int M, int I>
__device__ __forceinline__ void compare_exchange(int32_t (&k)[M]) {
    constexpr MergeExchangeNet<M> net{};
    constexpr int a = net.a[I], b = net.b[I];
    const int32_t lo = min(k[a], k[b]);
    const int32_t hi = max(k[a], k[b]);
    k[a] = lo;
    k[b] = hi;
}

template <int M, int... Is>
__device__ __forceinline__ void run_network(int32_t (&k)[M], std::integer_sequence<int, Is...>) {
    (compare_exchange<M, Is>(k), ...);
}

// Ascending sort of k[0..M-1] (signed compare).
template <int M>
__device__ __forceinline__ void sort_registers(int32_t (&k)[M]) {
    if constexpr (M > 1) run_network<M>(k, std::make_integer_sequence<int, MergeExchangeNet<M>::kCount>{});
}

}  // namespace detox

namespace detox {

// Bitonic merge for any length H: sorts, ascending, H keys that rise and then fall (or any cyclic shift of that).
// It is the merge network on P wires, P the next power of two, with P - H lowest keys imagined behind the last
// real one (the sequence stays bitonic in the cyclic sense).  A comparator that meets an imagined key needs no
// instruction -- the real key just changes wires -- so the wires are followed at compile time and only the
// comparators between two real keys are emitted: 304 instead of 448 for H = 96.  Registers keep their index;
// pos[r] tells at which sorted position the key of register r ends up.
template <int H>
struct BitonicMergeNet {
    static constexpr int pow2ceil(int n) { int p = 1; while (p < n) p <<= 1; return p; }
    static constexpr int P = pow2ceil(H);
    static constexpr int log2p() { int l = 0; while ((1 << l) < P) ++l; return l; }
    static constexpr int kMax = (P / 2) * (log2p() > 0 ? log2p() : 1);
    int count;
    int16_t a[kMax], b[kMax];
    int16_t pos[H];
    __host__ __device__ constexpr BitonicMergeNet() : count(0), a{}, b{}, pos{} {
        int slot[P] = {};                       // register on each wire, -1 for an imagined lowest key
        for (int w = 0; w < P; ++w) slot[w] = w < H ? w : -1;
        for (int s = P / 2; s >= 1; s >>= 1)
            for (int i = 0; i < P; ++i) {
                if (i & s) continue;
                const int j = i + s;
                if (slot[i] >= 0 && slot[j] >= 0) {
                    a[count] = (int16_t)slot[i];
                    b[count] = (int16_t)slot[j];
                    ++count;
                } else if (slot[i] >= 0) {      // the imagined key is the minimum: the real one moves up
                    slot[j] = slot[i];
                    slot[i] = -1;
                }
            }
        for (int w = P - H; w < P; ++w) pos[slot[w]] = (int16_t)(w - (P - H));
    }
};

template <int H, int I>
__device__ __forceinline__ void bitonic_merge_step(int32_t (&k)[H]) {
    constexpr BitonicMergeNet<H> net{};
    if constexpr (I < net.count) {
        constexpr int a = net.a[I], b = net.b[I];
        const int32_t lo = min(k[a], k[b]);
        const int32_t hi = max(k[a], k[b]);
        k[a] = lo;
        k[b] = hi;
    }
}

template <int H, int... Is>
__device__ __forceinline__ void bitonic_merge_run(int32_t (&k)[H], std::integer_sequence<int, Is...>) {
    (bitonic_merge_step<H, Is>(k), ...);
}

// After this, the key of register r is the BitonicMergeNet<H>::pos[r]-th smallest.
template <int H>
__device__ __forceinline__ void bitonic_merge_registers(int32_t (&k)[H]) {
    bitonic_merge_run<H>(k, std::make_integer_sequence<int, BitonicMergeNet<H>::kMax>{});
}

}  // namespace detox
