// Compile-time sorting networks for small fixed sizes (Batcher's merge exchange, valid for any length),
// applied to register arrays.  Comparators are emitted one by one with constant indices, so the array
// never leaves registers and the compiler drops every comparator that cannot reach an output that
// is actually used (a median needs far fewer than a full sort).
#pragma once

#include <stdint.h>

#include <utility>

namespace detox {

struct Comparator {
    int a, b;
};

template <int M>
struct MergeExchange {
    // Visit the comparators in network order; stop and return the idx-th one (or count them all).
    __host__ __device__ static constexpr Comparator nth(int idx, int* total) {
        int c = 0;
        for (int p = 1; p < M; p <<= 1) {
            for (int k = p; k >= 1; k >>= 1) {
                for (int j = k % p; j <= M - 1 - k; j += 2 * k) {
                    int imax = k - 1 < M - j - k - 1 ? k - 1 : M - j - k - 1;
                    for (int i = 0; i <= imax; ++i) {
                        if ((i + j) / (2 * p) == (i + j + k) / (2 * p)) {
                            if (c == idx) return Comparator{i + j, i + j + k};
                            ++c;
                        }
                    }
                }
            }
        }
        if (total) *total = c;
        return Comparator{0, 0};
    }
    __host__ __device__ static constexpr int count() {
        int t = 0;
        nth(-1, &t);
        return t;
    }
};

template <int M, int I>
__device__ __forceinline__ void compare_exchange(int32_t (&k)[M]) {
    constexpr Comparator c = MergeExchange<M>::nth(I, nullptr);
    const int32_t lo = min(k[c.a], k[c.b]);
    const int32_t hi = max(k[c.a], k[c.b]);
    k[c.a] = lo;
    k[c.b] = hi;
}

template <int M, int... Is>
__device__ __forceinline__ void run_network(int32_t (&k)[M], std::integer_sequence<int, Is...>) {
    (compare_exchange<M, Is>(k), ...);
}

// Ascending sort of k[0..M-1] (signed compare).
template <int M>
__device__ __forceinline__ void sort_registers(int32_t (&k)[M]) {
    if constexpr (M > 1) run_network<M>(k, std::make_integer_sequence<int, MergeExchange<M>::count()>{});
}

}  // namespace detox
