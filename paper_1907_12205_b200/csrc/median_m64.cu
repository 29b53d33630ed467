// Register order-statistic kernels for the network sizes 39..64 (one translation unit per
// size range keeps the build parallel).
#include "median_impl.cuh"

namespace detox {

detox_status launch_reg_upto64(int M, const float* X, int64_t ld, int m, int64_t d, const int32_t* rows, int beta,
                               float* out, bool vec, cudaStream_t s) {
    switch (M) {
#define DETOX_CASE(MM) \
    case MM: return regselect::launch_reg_m<MM>(X, ld, m, d, rows, beta, out, vec, s);
        DETOX_CASE(39) DETOX_CASE(40) DETOX_CASE(47) DETOX_CASE(48) DETOX_CASE(55) DETOX_CASE(56) DETOX_CASE(63) DETOX_CASE(64)
#undef DETOX_CASE
        default: return DETOX_ERR_UNSUPPORTED;
    }
}

}  // namespace detox
