// What the tensor-core distance kernels (gram_tc.cu: split TF32; gram_f16.cu: split fp16) share: the way columns are
// dealt to CTAs and slabs to output slots, and the buffers a launch is given.
#pragma once

#include "common.cuh"

namespace detox {

constexpr int kProdWarps = 16;                 // transform warps of every kernel
constexpr int kProdThreads = kProdWarps * 32;
constexpr int kMaxCentreRows = 16;             // the subtracted vector is the mean of at most this many rows
constexpr size_t kSmemBudget = 227 * 1024;     // dynamic shared memory one CTA may have
constexpr int64_t kSlabCols = 4096;            // columns accumulated in tensor memory before a drain
constexpr int kItemSlabs = 4;                  // consecutive slabs of a CTA that are added into one output slot
constexpr int kTargetRmsLog2 = 6;              // split fp16: every row is scaled so that its typical entry is near 2^6

// What a launch is given besides its plan.  redo: null for the first launch of a call; for the second the flag the
// check of the first one has set (the kernel returns at once when it reads 0).
struct TcBuffers {
    float* partial;     // [slot][m][ncol] fp32 sums of products
    float* norms;       // [slot][group][m] exact squared norms of the rows as the tensor cores saw them
    const int* centre;  // [0] rows averaged into the subtracted vector (0: none), [1] redo flag, [2..] the rows
    const int* redo;
    int* status;
};

// gram_f16.cu: the split-fp16 pass (16 < m <= 256).  expo[i]: row i is multiplied by 2^expo[i] before it is split.
int f16_nitems(int m, int64_t d);
int f16_groups(int m);
detox_status launch_gram_f16(const float* X, int64_t ld, int m, int64_t d, const TcBuffers& b, const int* expo,
                             cudaStream_t s);
// The same pass over the votes of n / 3 groups of three rows of X, formed inside the pass (Section 3: the filtering
// step); ORs the "members differed" bits of every group into pairdiff (vote kernels' format), which the caller has cleared.
bool f16_vote_supported(int n, int r);
detox_status launch_gram_f16_vote(const float* X, int64_t ld, int n, int64_t d, const IdTable& groups,
                                  uint32_t* pairdiff, const TcBuffers& b, const int* expo, cudaStream_t s);

// The driver's tensor-map encoder for X as a 2-D fp32 tensor (d columns innermost, m rows, row pitch ld), zero fill
// outside; swizzle128 = false: rows of a box land one after another.
detox_status make_xmap(void* map, const float* X, int64_t ld, int m, int64_t d, int box_cols, int box_rows, bool swizzle128);

}  // namespace detox
