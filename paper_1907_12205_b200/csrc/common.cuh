// Shared device helpers and the launcher declarations of libdetox (internal).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "detox.h"

namespace detox {

constexpr int kSMs = 148;            // B200: 2 dies x 74 SMs; grids are sized in multiples of this
constexpr int kMaxRows = DETOX_MAX_ROWS;
constexpr int kMaxR = DETOX_MAX_R;

constexpr int kPairWords = 4;        // "members a and b differed" bits per node group: r <= 15 -> at most 105 pairs

// Small host-side index tables travel as kernel parameters (no copy, no allocation).
struct IdTable {
    uint16_t id[kMaxRows];
};
struct SetTable {
    uint16_t offset[kMaxRows + 1];
    uint16_t member[kMaxRows];
};
// The member rows of at most 85 groups of three (the distance pass that votes while it reads).
struct VoteMembers {
    uint8_t id[256];
};

// ---- order-preserving integer key for fp32 bit patterns -------------------------------------
// Signed compare on the key gives -NaN < -Inf < ... < -0 < +0 < ... < +Inf < +NaN.
// The map is its own inverse.
__device__ __forceinline__ int32_t key_of_bits(uint32_t b) {
    int32_t s = (int32_t)b;
    return s ^ ((s >> 31) & 0x7fffffff);
}
__device__ __forceinline__ float float_of_key(int32_t k) {
    return __int_as_float(k ^ ((k >> 31) & 0x7fffffff));
}

// ---- streaming loads / stores (data is touched once; keep it out of the way in L1) ----------
__device__ __forceinline__ uint4 ld_stream_u4(const void* p) {
    return __ldcs(reinterpret_cast<const uint4*>(p));
}
__device__ __forceinline__ float4 ld_stream_f4(const void* p) {
    return __ldcs(reinterpret_cast<const float4*>(p));
}
__device__ __forceinline__ uint32_t ld_stream_u1(const void* p) {
    return __ldcs(reinterpret_cast<const unsigned int*>(p));
}
__device__ __forceinline__ void st_stream_u4(void* p, uint4 v) {
    __stcs(reinterpret_cast<uint4*>(p), v);
}
__device__ __forceinline__ void st_stream_f4(void* p, float4 v) {
    __stcs(reinterpret_cast<float4*>(p), v);
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline size_t align_up(size_t x, size_t a = 256) { return (x + a - 1) / a * a; }

// Called once after every kernel launch: the launch's error status; also counts the launch (api.cu).
detox_status launch_status();

// ---- launchers (each enqueues on `s`; none synchronises) ------------------------------------

// vote.cu
size_t vote_ws_bytes(int n, int r);
// clear_before: bytes directly in front of `ws` that the launcher's clearing memset zeroes along with the words it
// uses itself (the pipeline keeps its device status word there)
detox_status launch_vote(const float* X, int64_t ld, int n, int r, int64_t d, const IdTable& members,
                         float* Z, int64_t ldz, int32_t* winner, void* ws, cudaStream_t s, size_t clear_before = 0);

// the last step of a vote on its own: winners from the "members differed" bits in ws; *none_flag (optional, device) is
// set to 1 when a group has no majority
detox_status launch_vote_finalize(int n, int r, const IdTable& members, const void* ws, int32_t* winner, int* none_flag,
                                  cudaStream_t s);
// r = 3: the votes as rows of Z (zero rows where winner[g] < 0), written only when *gate (device) is not zero
detox_status launch_vote_store_gated(const float* X, int64_t ld, int n, int64_t d, const IdTable& members, float* Z,
                                     int64_t ldz, const int32_t* winner, const int* gate, cudaStream_t s);

// vote + A_0 = mean in one pass: M[s] = mean of the votes of set s; the votes themselves are not stored
detox_status launch_vote_mean(const float* X, int64_t ld, int n, int r, int64_t d, const IdTable& members,
                              const SetTable& sets, int S, float* M, int64_t ldm, int32_t* winner, void* ws,
                              cudaStream_t s, size_t clear_before = 0);

// vote + A_0 = mean + a coordinate-wise A_1 over the S <= 16 set means in one pass: out = A_1(set means); neither votes
// nor set means are stored.  beta as in launch_coord_select (0: median; <= -1: mean of the middle -beta values);
// mean = true: the mean of the set means.  Needs 16-byte aligned rows and r in {1, 3, 5}.
bool vote_mean_select_supported(const float* X, int64_t ld, int r, int S, const float* out);
detox_status launch_vote_mean_select(const float* X, int64_t ld, int n, int r, int64_t d, const IdTable& members,
                                     const SetTable& sets, int S, int beta, bool mean, float* out, int32_t* winner,
                                     void* ws, cudaStream_t s, size_t clear_before = 0);

// mean.cu
// (sign = true: coordinate-wise sign majority sign(sum sign(x)) instead of the mean, in both launchers)
detox_status launch_hier_mean(const float* Z, int64_t ldz, int64_t d, const SetTable& sets, int S,
                              float* M, int64_t ldm, cudaStream_t s, bool sign = false);
// mean of k rows of X listed in rows_dev (device int32; NULL = rows 0..k-1; a negative entry = a zero row)
detox_status launch_mean_rows(const float* X, int64_t ld, int64_t d, const int32_t* rows_dev, int k,
                              float* out, cudaStream_t s, bool sign = false);

// median.cu: per-coordinate order statistics over m rows (rows_dev: device int32 list or NULL; a negative
// entry = a zero row)
//   beta == 0 : coordinate median;  beta >= 1 : mean of the beta values closest to the median;
//   beta <= -1 : mean of the middle -beta values of the sorted column (m + beta even): the trimmed mean
detox_status launch_coord_select(const float* X, int64_t ld, int m, int64_t d, const int32_t* rows_dev,
                                 int beta, float* out, cudaStream_t s);

// dist.cu: squared distances D (m x m, fp64, symmetric, zero diagonal)
//   status: device int32, must be 0 on entry; set to DETOX_ERR_TIMEOUT (and D to NaN) if a bounded
//   device-side wait of the tensor-core path runs out
size_t dist_ws_bytes(int m, int64_t d);
//   rows: optional device list of the m rows of X to use (m <= 16 only); a negative entry stands for a zero row
detox_status launch_sqdist(const float* X, int64_t ld, int m, int64_t d, const int32_t* rows, double* D, void* ws,
                           int* status, cudaStream_t s);

// gram_tc.cu: the tcgen05 path for 16 < m <= 256 (needs 16-byte aligned rows)
bool tc_supported(const float* X, int64_t ld, int m, int64_t d);
size_t tc_ws_bytes(int m, int64_t d);
// which operand split the pass tries first (DETOX_SPLIT_*); returns the previous mode
int tc_split_mode(int mode);
// how many calls on the current device had their tensor-core pass repeated so far (synchronises the device)
unsigned long long tc_repeated_passes();
// 2 <= m <= 16: the direct kernels' per-CTA pair partials only (consumed by launch_krum_small).  When
// sqdist_partials_use_status() holds the kernel clears the device status word itself and may set it to
// DETOX_ERR_TIMEOUT, so the consumer must leave it alone.
bool sqdist_partials_use_status(int m, const float* X, int64_t ld, int64_t d);
// clear_status: whether that kernel clears the word first (false: the word is shared with other stages and only ever set)
detox_status launch_sqdist_partials(const float* X, int64_t ld, int m, int64_t d, const int32_t* rows, void* ws,
                                    int* status, bool clear_status, int* nblocks, cudaStream_t s);
detox_status launch_sqdist_tc(const float* X, int64_t ld, int m, int64_t d, double* D, void* ws, int* status,
                              cudaStream_t s);
// The filtering step and the distance pass in one (r = 3, 16 < n / 3 <= 85 groups): the distances between the votes of
// the groups, formed while the members' rows stream through the tensor-core pass, and winner[]; no vote is stored
// unless the pass has to be repeated (a group without a majority, an entry outside the fp16 range), in which case
// the votes go to Z (n / 3 rows of pitch ldz) and the split-TF32 kernels run on them.  vote_ws: the vote's cleared
// workspace words.  ws as for launch_sqdist_tc with m = n / 3.
bool sqdist_vote_tc_supported(const float* X, int64_t ld, int n, int r, int64_t d);
detox_status launch_sqdist_vote_tc(const float* X, int64_t ld, int n, int64_t d, const IdTable& members, int32_t* winner,
                                   void* vote_ws, float* Z, int64_t ldz, double* D, void* ws, int* status, cudaStream_t s);

// centre.cu: the centring rows for the tensor-core distance pass (m <= 256), chosen on a sample of the columns
//   centre[0] = how many rows are averaged into the vector that is subtracted from every row (0 when the rows hover
//   around zero anyway), centre[1] = redo flag (below), centre[2..17] = the rows; expo[m] = every row's power-of-two
//   scale for the split-fp16 pass
size_t centre_ws_bytes(int m, int64_t d);
//   members != null: the m rows are the votes of the groups of three rows of X listed there, formed on the fly;
//   centre[18..33] = for every listed vote the row of X of a member that gave it
detox_status launch_pick_centre(const float* X, int64_t ld, int m, int64_t d, void* ws, int* centre, int* expo,
                                cudaStream_t s, const VoteMembers* members = nullptr);
//   after the pass: norms = the rows' exact squared norms after the subtraction (nitems x groups x m), partial = the
//   slots' sums of products (nitems x m x ncol).  Withdraws the centring (centre[0] = 0) when the typical row came out
//   far larger than the sample predicted for the rows as they were; expo != null: the split-fp16 pass ran with these
//   row scales, and its tensor-core norms are checked against the exact ones.  *redo = 1 when the pass has to be
//   repeated (by the split-TF32 kernels), 0 otherwise.
detox_status launch_check_centre(const float* norms, const float* partial, int nitems, int groups, int m, int ncol,
                                 void* ws, int64_t d, int* centre, int* redo, const int* expo, cudaStream_t s);

// geomed.cu: Weiszfeld iterations for the geometric median of m <= 32 rows
size_t geomed_ws_bytes(int64_t d);
detox_status launch_geometric_median(const float* X, int64_t ld, int m, int64_t d, int iters, float eps, float* out,
                                     void* ws, cudaStream_t s);

// select.cu
size_t select_ws_bytes(int m);
// Multi-Krum scoring + selection of the m_sel best rows (ascending indices in sel_dev)
detox_status launch_multikrum_select(const double* D, int m, int f, int m_sel, int32_t* sel_dev,
                                     double* scores_dev, void* ws, cudaStream_t s);
// Bulyan stage 1: theta = m - 2f rounds; sel_dev in selection order
// 2 <= m <= 16: pair partials -> distances -> ranked lists -> selection (-> rows of X through the row list), one CTA
detox_status launch_krum_small(bool bulyan, const double* partial, int nblocks, int m, int f, int m_sel,
                               const int32_t* rows_dev, int32_t* sel_dev, int32_t* mapped_dev, double* scores_dev,
                               int* status_dev, cudaStream_t s);
detox_status launch_bulyan_select(const double* D, int m, int f, int32_t* sel_dev, void* ws,
                                  cudaStream_t s);
// out[k] = map[idx[k]] (k < cnt), all device int32
detox_status launch_map_indices(const int32_t* idx, const int32_t* map, int cnt, int32_t* out,
                                cudaStream_t s);

// votes computed in set order: winner back to group order; selections inside a set to vote / worker ids
detox_status launch_scatter_by_set_order(const int32_t* src, const SetTable& sets, int G, int32_t* dst,
                                         cudaStream_t s);
detox_status launch_map_set_selection(const int32_t* local, int cnt, const SetTable& sets, int set_begin,
                                      const int32_t* winner_in_set_order, int32_t* sel_votes, int32_t* sel_workers,
                                      cudaStream_t s);

}  // namespace detox
