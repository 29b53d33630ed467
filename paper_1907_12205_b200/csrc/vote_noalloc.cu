// detox_vote_noalloc: the majority vote for callers that cannot allocate device memory.
//
// The vote needs a few words of scratch per node group (the "member a differs from member b" bits).
// Here that scratch is a fixed array inside the library image instead of a caller-provided
// workspace, so the call needs no cudaMalloc and no allocating library routine at all.
#include <mutex>

#include "common.cuh"

namespace {

constexpr int kMaxGroups = DETOX_NOALLOC_MAX_GROUPS;
constexpr int kWordsPerGroup = 4;
constexpr int kMaxDevices = 64;

// Lives in the global memory of every GPU that loads the library, until the process exits (4 KiB).
static __device__ __align__(256) uint32_t g_vote_scratch[kMaxGroups * kWordsPerGroup];

std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices];  // device address of g_vote_scratch on each device; null until set up

// In host code `g_vote_scratch` is only a handle; the address a kernel can use has to be asked for,
// once per device, with that device current.
detox_status scratch_for_current_device(void** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return DETOX_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_vote_scratch) != cudaSuccess || !p) return DETOX_ERR_CUDA;
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return DETOX_OK;
}

}  // namespace

extern "C" detox_status detox_vote_noalloc(const float* X, int64_t ld, int n, int r, int64_t d,
                                           const int32_t* members, float* Z, int64_t ldz, int32_t* winner,
                                           void* stream) {
    using namespace detox;
    if (n < 1 || r < 1 || (r & 1) == 0 || n % r != 0 || !members || !X || !winner || d < 1 || ld < d)
        return DETOX_ERR_BAD_ARG;
    if (n > kMaxRows || r > kMaxR) return DETOX_ERR_UNSUPPORTED;
    if (n / r > kMaxGroups) return DETOX_ERR_UNSUPPORTED;  // more groups than the built-in scratch holds
    if ((reinterpret_cast<uintptr_t>(X) & 3u) || (Z && ((reinterpret_cast<uintptr_t>(Z) & 3u) || ldz < d)))
        return DETOX_ERR_BAD_ARG;
    IdTable tab;
    bool seen[kMaxRows] = {false};
    for (int k = 0; k < n; ++k) {
        const int32_t id = members[k];
        if (id < 0 || id >= n || seen[id]) return DETOX_ERR_BAD_ARG;
        seen[id] = true;
        tab.id[k] = (uint16_t)id;
    }
    void* scratch = nullptr;
    detox_status st = scratch_for_current_device(&scratch);
    if (st != DETOX_OK) return st;
    // launch_vote clears the words it uses (stream-ordered) before the vote kernel sets them.
    return launch_vote(X, ld, n, r, d, tab, Z, ldz, winner, scratch, static_cast<cudaStream_t>(stream));
}
