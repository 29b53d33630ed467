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
