/*
 * libdetox — DETOX parameter-server gradient aggregation for NVIDIA B200 (sm_100a).
 *
 * C ABI.  Every entry point enqueues its kernels on the caller's CUDA stream and returns without
 * synchronising the host.  The library allocates nothing and keeps no state between calls: every
 * buffer, including scratch ("workspace"), belongs to the caller (the one exception, a fixed
 * scratch array inside the library, is detox_vote_noalloc below).
 *
 * Notation follows arXiv 1907.12205: n compute nodes (the paper's p) each send a gradient of
 * dimension d; node groups have size r (odd, r divides n), so there are G = n / r votes; f is the
 * Byzantine tolerance handed to Multi-Krum / Bulyan.
 *
 * Common conventions
 *   - "dev" pointers are device pointers valid on the current device; "host" pointers are ordinary
 *     host memory, read before the call returns.
 *   - Matrices are row-major fp32 with a row stride `ld` in ELEMENTS (ld >= d).  The vectorised paths
 *     need a 16-byte aligned base and ld % 4 == 0; any other layout takes a slower scalar path with the
 *     same results.
 *   - Index outputs are int32.  Limits: n, m <= DETOX_MAX_ROWS; r <= DETOX_MAX_R.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Workspace pointers must be 256-byte aligned; sizes come from the *_workspace_bytes helpers.
 *   - Errors: argument problems are reported before anything is launched; a failed launch returns
 *     DETOX_ERR_CUDA.  Nothing aborts or throws.  Multi-Krum and Bulyan run kernels that wait on
 *     asynchronous copies (9 to 16 long rows) or on the tensor cores (17 to 256 rows); every such
 *     device-side wait is bounded.  Device status word: the first int32 of the workspace passed to
 *     agg_multikrum, agg_bulyan or detox_aggregate.  The call clears it; should a wait run out in any
 *     stage of the call it reads DETOX_ERR_TIMEOUT once the stream has been synchronised (0 otherwise),
 *     the outputs are then not valid (the index outputs still hold in-range indices), and nothing
 *     hangs or faults.
 *   - Non-finite values: the vote and the order statistics are fully defined on them (bit patterns).
 *     In Multi-Krum / Bulyan a row with an Inf or NaN entry is infinitely far from every other row
 *     (a NaN distance counts as +Inf), so it is never preferred to a finite row.
 *   - Ranking of values (medians, "closest to the median") uses the total order
 *     -NaN < -Inf < ... < -0 < +0 < ... < +Inf < +NaN on fp32 bit patterns.
 */
#ifndef DETOX_H_
#define DETOX_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DETOX_MAX_ROWS 1024
#define DETOX_MAX_R 15

typedef enum {
    DETOX_OK = 0,
    DETOX_ERR_BAD_ARG = 1,      /* null pointer, size out of range, r even or not dividing n, bad partition */
    DETOX_ERR_UNSUPPORTED = 2,  /* valid request outside the built limits */
    DETOX_ERR_WORKSPACE = 3,    /* workspace missing, misaligned or too small */
    DETOX_ERR_CUDA = 4,         /* a CUDA call or launch failed */
    DETOX_ERR_TIMEOUT = 5       /* a bounded device-side wait ran out (reported through the status word) */
} detox_status;

typedef enum {
    DETOX_AGG_NONE = 0,         /* A_0 only: pass the votes through */
    DETOX_AGG_MEAN = 1,
    DETOX_AGG_COORD_MEDIAN = 2,
    DETOX_AGG_MULTIKRUM = 3,
    DETOX_AGG_BULYAN = 4,
    DETOX_AGG_TRIMMED_MEAN = 5, /* A_1 only: drops the f smallest and f largest values per coordinate */
    DETOX_AGG_GEOMETRIC_MEDIAN = 6, /* A_1 only: gm_iters Weiszfeld iterations over at most 32 rows */
    DETOX_AGG_SIGN_MAJORITY = 7 /* A_0 and A_1: coordinate-wise sign(sum of signs), the signSGD pairing */
} detox_agg;

const char* detox_status_string(detox_status s);

/* ---------------------------------------------------------------------------------------------
 * Filtering step (Section 3; Algorithm 1, "Filtering step"): for every node group A_j the majority
 * vote z_j = maj{ g_i : i in A_j }, and z_j = 0 when no value is sent by more than r/2 members.
 * Two members agree when their d-vectors are bitwise identical.
 *
 *   X        dev, n x ld      the n received gradients (read only)
 *   members  host, G*r        worker ids; group j owns members[j*r .. j*r+r-1]; a partition of 0..n-1
 *   Z        dev, G x ldz     out: the votes; may be NULL when only `winner` is wanted
 *   winner   dev, G           out: lowest worker id of the winning class, or -1 (then Z[j] = 0)
 *   ws       dev              detox_vote_workspace_bytes(n, r) bytes
 * ------------------------------------------------------------------------------------------- */
size_t detox_vote_workspace_bytes(int n, int r);
detox_status detox_vote(const float* X, int64_t ld, int n, int r, int64_t d, const int32_t* members,
                        float* Z, int64_t ldz, int32_t* winner, void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * detox_vote without a workspace, for callers that must not allocate device memory.  (The paper has
 * no counterpart; this is a packaging variant of detox_vote and computes exactly the same votes.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a framework's allocator
 * callback, in a latency-critical serving loop with a frozen memory plan, or in a process whose
 * memory budget is fixed at start-up - and that has nowhere to keep a workspace buffer.
 *
 * The scratch words of the vote live in a fixed array inside the library (4 KiB of global memory on
 * every GPU that loads the library, held until the process exits), so at most
 * DETOX_NOALLOC_MAX_GROUPS node groups (n / r) are accepted; more returns DETOX_ERR_UNSUPPORTED.
 * The call itself performs no cudaMalloc / cudaFree and calls no allocating routine.
 *
 *   - Arguments as in detox_vote, minus ws / ws_bytes.  Inputs and outputs are still the caller's.
 *   - The first call on each device looks up the device address of the built-in array (a one-time
 *     set-up step, done with that device current).  Make that first call before any stream capture.
 *   - All calls on a device share the one array.  Each call clears the words it uses before using
 *     them, so results never depend on an earlier call; but two calls whose kernels overlap on the
 *     GPU (different streams, no dependency between them) race on it.  Serialise them.
 * ------------------------------------------------------------------------------------------- */
#define DETOX_NOALLOC_MAX_GROUPS 256
detox_status detox_vote_noalloc(const float* X, int64_t ld, int n, int r, int64_t d, const int32_t* members,
                                float* Z, int64_t ldz, int32_t* winner, void* stream);

/* ---------------------------------------------------------------------------------------------
 * A_0 = mean over each vote group (Algorithm 2, step 3, with A_0 the mean as analysed in Section 4):
 * M[s] = (1/|Z_s|) sum_{j in Z_s} z_j.  A zero vote (no majority) counts as an ordinary member.
 *
 *   Z            dev, G x ldz   the votes
 *   set_offsets  host, S+1      set s owns set_members[set_offsets[s] .. set_offsets[s+1]-1]; sets may be
 *                               uneven (e.g. 7 and 8 out of 15, Appendix B.1) but not empty
 *   set_members  host, G        vote indices, a partition of 0..G-1
 *   M            dev, S x ldm   out
 * ------------------------------------------------------------------------------------------- */
detox_status detox_hier_mean(const float* Z, int64_t ldz, int G, int64_t d, const int32_t* set_offsets,
                             const int32_t* set_members, int S, float* M, int64_t ldm, void* stream);

/* ---------------------------------------------------------------------------------------------
 * detox_vote followed by detox_hier_mean, in one pass over X (Algorithm 1's filtering step and
 * Algorithm 2, step 3 with A_0 the mean): M[s] is the mean of the votes of set s, bit for bit what
 * the two calls give, but the votes are never written to memory (n*d*4 bytes read, S*d*4 written).
 * detox_aggregate uses this path whenever a0 = DETOX_AGG_MEAN.
 *
 *   arguments as in detox_vote (without Z) and detox_hier_mean (without Z, G);
 *   ws: detox_vote_workspace_bytes(n, r) bytes.
 * ------------------------------------------------------------------------------------------- */
detox_status detox_vote_hier_mean(const float* X, int64_t ld, int n, int r, int64_t d, const int32_t* members,
                                  const int32_t* set_offsets, const int32_t* set_members, int S, float* M,
                                  int64_t ldm, int32_t* winner, void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * The same two steps for very many nodes with short vectors - the regime of the paper's synthetic
 * experiment (Section 5.3, "Mean estimation on synthetic data": p = 220,000 nodes, r = 11, d <= 100), where
 * the tables above (at most DETOX_MAX_ROWS nodes) do not reach.  One warp votes per node group; the
 * group table lives in device memory; a vote set is a run of consecutive groups (the group table is a
 * random partition already, so consecutive groups are a random set).  The S set means then go to
 * agg_geometric_median / agg_coord_median as ordinary rows.
 *
 *   X            dev, n x ld     n <= 2^30 nodes, d <= DETOX_MANY_MAX_D
 *   members      dev, n          worker ids, group j owns members[j*r .. j*r+r-1]; must be a partition of
 *                                0..n-1 (not checked; a group holding an id outside 0..n-1 gets no vote)
 *   set_offsets  host, S+1       set s owns the groups set_offsets[s] .. set_offsets[s+1]-1; S <= DETOX_MAX_ROWS
 *   M            dev, S x ldm    out: mean of the votes of each set (a group without a majority counts as a
 *                                zero vote); may be NULL, then only `winner` is produced and sets are ignored
 *   winner       dev, n / r      out, as in detox_vote
 * No workspace.
 * ------------------------------------------------------------------------------------------- */
#define DETOX_MANY_MAX_D 1024
detox_status detox_vote_hier_mean_many(const float* X, int64_t ld, int64_t n, int r, int d, const int32_t* members,
                                       const int32_t* set_offsets, int S, float* M, int64_t ldm, int32_t* winner,
                                       void* stream);

/* ---------------------------------------------------------------------------------------------
 * Coordinate-wise median (Section 4; Appendix B.1): out[c] = median_i X[i][c] over the m rows.
 * Odd m: the middle value, bit for bit one of the inputs.  Even m: fp32 (lo + hi) * 0.5f.
 *   out  dev, d.   ws: agg_coord_median_workspace_bytes(m, d) bytes.  Every size built so far works in
 *   registers or shared memory, so that is 0 and ws is not touched (pass NULL); the arguments keep the
 *   signature of the other aggregators.
 * ------------------------------------------------------------------------------------------- */
size_t agg_coord_median_workspace_bytes(int m, int64_t d);
detox_status agg_coord_median(const float* X, int64_t ld, int m, int64_t d, float* out, void* ws,
                              size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Coordinate-wise alpha-trimmed mean (one of the A_1 choices analysed in Section 4, Theorem 4 with
 * alpha = 1/4): per coordinate, drop the `trim` smallest and the `trim` largest of the m values and
 * average the other m - 2*trim.  0 <= trim, m - 2*trim >= 1.  trim = 0 is the plain mean.
 *   out  dev, d.   No workspace.
 * ------------------------------------------------------------------------------------------- */
detox_status agg_trimmed_mean(const float* X, int64_t ld, int m, int64_t d, int trim, float* out, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Coordinate-wise sign majority, the aggregator of signSGD with majority vote (Section 5.2, setup 4:
 * A_0 = A_1 = coordinate-wise majority): out[c] = sign(sum_i sign(X[i][c])), one of -1, 0, +1
 * (sign(0) = sign(NaN) = 0; a tie gives 0).
 *   out  dev, d.   No workspace.
 * ------------------------------------------------------------------------------------------- */
detox_status agg_sign_majority(const float* X, int64_t ld, int m, int64_t d, float* out, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Geometric median (one of the A_1 choices analysed in Section 4, Theorem 4; the paper does not fix
 * an algorithm).  Computed by Weiszfeld's iteration started at the mean:
 *     y <- sum_j w_j x_j / sum_j w_j,   w_j = 1 / max(||x_j - y||_2, eps),   `iters` times.
 * m <= 32 rows (it aggregates the few set results of the hierarchical step); more returns
 * DETOX_ERR_UNSUPPORTED.  iters >= 0 (0 gives the mean), eps > 0.
 *   out  dev, d.   ws: agg_geometric_median_workspace_bytes(m, d) bytes.
 * ------------------------------------------------------------------------------------------- */
size_t agg_geometric_median_workspace_bytes(int m, int64_t d);
detox_status agg_geometric_median(const float* X, int64_t ld, int m, int64_t d, int iters, float eps, float* out,
                                  void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Pairwise squared Euclidean distances between the m rows, the O(p^2 d) step that Section 4 ("Improved
 * speed") names as the cost of Krum, Multi-Krum and Bulyan: D[i][j] = sum_c (X[i][c] - X[j][c])^2.
 * This is the first stage of agg_multikrum / agg_bulyan on its own (same kernels, same results).
 *   D   dev, m x m fp64, row-major, symmetric, zero diagonal (8-byte aligned)
 *   ws  agg_pairwise_sqdist_workspace_bytes(m, d) bytes; its first int32 is the device status word
 * ------------------------------------------------------------------------------------------- */
size_t agg_pairwise_sqdist_workspace_bytes(int m, int64_t d);
detox_status agg_pairwise_sqdist(const float* X, int64_t ld, int m, int64_t d, double* D, void* ws, size_t ws_bytes,
                                 void* stream);

/* ---------------------------------------------------------------------------------------------
 * Multi-Krum (cited in Section 4 "Improved speed" as the O(p^2 d) aggregator; requirement
 * m >= 2f+3 in Appendix B.1).  score_i = sum of the nb smallest squared distances from row i to the
 * other rows, nb = m - f - 2 clamped to [1, m-1]; the m_sel rows of smallest score (equal scores:
 * lower index first) are averaged.  m < 2f+3 is accepted (the clamp applies) down to m >= 1.
 *
 *   out     dev, d         the average of the selected rows
 *   sel     dev, m_sel     out, ascending row indices; may be NULL
 *   scores  dev, m (fp64)  out; may be NULL
 *   ws      agg_multikrum_workspace_bytes(m, d) bytes
 * ------------------------------------------------------------------------------------------- */
size_t agg_multikrum_workspace_bytes(int m, int64_t d);
detox_status agg_multikrum(const float* X, int64_t ld, int m, int64_t d, int f, int m_sel, float* out,
                           int32_t* sel, double* scores, void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Bulyan (cited in Section 4; requirement m >= 4f+3 in Appendix B.1, enforced here).  Stage 1:
 * theta = m - 2f rounds of Krum on the shrinking candidate set (scores recomputed from the cached
 * distances with nb = |remaining| - f - 2, clamped as above).  Stage 2, per coordinate: the median of
 * the theta selected values, then the mean of the beta = theta - 2f values closest to it (closeness
 * |v - median| in fp32; equally close: the smaller value first).
 *
 *   out  dev, d
 *   sel  dev, theta   out, row indices in the order they were selected; may be NULL
 *   ws   agg_bulyan_workspace_bytes(m, d) bytes
 * ------------------------------------------------------------------------------------------- */
size_t agg_bulyan_workspace_bytes(int m, int64_t d);
detox_status agg_bulyan(const float* X, int64_t ld, int m, int64_t d, int f, float* out, int32_t* sel,
                        void* ws, size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * The whole parameter-server step (Algorithm 1, filtering + hierarchical aggregation; Algorithm 2):
 * vote over the node groups, A_0 over each vote group, A_1 over the results.
 *
 *   a0 = DETOX_AGG_NONE : the G votes go to A_1 directly (sets are ignored).  The votes are rows of X, so they are
 *        read through winner[] and not stored; with a1 = MULTIKRUM or BULYAN over 17 to 85 votes of groups of r = 3
 *        (16-byte aligned rows) the vote itself runs inside the distance pass, one pass over X for both (the votes are
 *        stored, and the pass repeated on them, only when a group has no majority or an entry leaves the range of the
 *        pass's fp16 operands; the results are the same either way)
 *   a0 = DETOX_AGG_MEAN : the S set means go to A_1 (with a1 = MEAN, COORD_MEDIAN or TRIMMED_MEAN over at most 16 sets,
 *        r in {1, 3, 5} and 16-byte aligned rows of X and out, the whole step is one pass over X and the set means
 *        are never stored; the result is bitwise the same either way)
 *   a0 = DETOX_AGG_SIGN_MAJORITY : the S coordinate-wise sign majorities of the sets go to A_1
 *   a0 = DETOX_AGG_MULTIKRUM | DETOX_AGG_BULYAN : the aggregator runs inside every vote set (the pairings the
 *        paper found most resilient, Section 5.2, setups 2 and 3; set shapes as in Appendix B.1, e.g. 7 + 8 or
 *        one set of 15) and its S results go to A_1, which must then be MEAN or COORD_MEDIAN.  f and m_sel
 *        belong to A_0: every set of k votes averages its m_sel best (m_sel = 0: its k - f best), or, for
 *        Bulyan, needs k >= 4f+3.
 *   a1 = MEAN | SIGN_MAJORITY | COORD_MEDIAN | TRIMMED_MEAN (f per side) | GEOMETRIC_MEDIAN (gm_iters, gm_eps; at most 32 rows
 *        enter it) | MULTIKRUM (f, m_sel) | BULYAN (f)
 *
 *   out          dev, d
 *   winner       dev, G        out, as in detox_vote; may be NULL
 *   sel          dev           out, rows chosen by Multi-Krum (m_sel, ascending) or Bulyan (theta, in
 *                              selection order): indices among the rows that entered A_1 when A_1 is the
 *                              Krum-type stage; vote (group) indices, set after set, when A_0 is; may be NULL
 *   sel_workers  dev           out, the same rows as worker ids (winner[vote]), meaningful whenever sel
 *                              indexes votes (a0 = NONE, MULTIKRUM or BULYAN); may be NULL
 *   ws           detox_aggregate_workspace_bytes(desc) bytes (holds the votes and set means too); its first
 *                int32 is the device status word of the whole step (see "Errors" above)
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    int32_t n;                   /* compute nodes */
    int32_t r;                   /* redundancy ratio (odd, divides n) */
    int64_t d;                   /* gradient dimension */
    const int32_t* members;      /* host, G*r */
    int32_t a0;                  /* detox_agg: NONE, MEAN, SIGN_MAJORITY, MULTIKRUM or BULYAN */
    int32_t n_sets;              /* S, used unless a0 = NONE */
    const int32_t* set_offsets;  /* host, S+1 */
    const int32_t* set_members;  /* host, G */
    int32_t a1;                  /* detox_agg: MEAN, COORD_MEDIAN, TRIMMED_MEAN, GEOMETRIC_MEDIAN, MULTIKRUM or BULYAN */
    int32_t f;                   /* tolerance given to Multi-Krum / Bulyan */
    int32_t m_sel;               /* rows averaged by Multi-Krum */
    int32_t gm_iters;            /* Weiszfeld iterations when a1 = GEOMETRIC_MEDIAN */
    float gm_eps;                /* floor on the distances in its weights (> 0) */
} detox_pipeline_desc;

size_t detox_aggregate_workspace_bytes(const detox_pipeline_desc* desc);
detox_status detox_aggregate(const detox_pipeline_desc* desc, const float* X, int64_t ld, float* out,
                             int32_t* winner, int32_t* sel, int32_t* sel_workers, void* ws,
                             size_t ws_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Self-test of the bounded device-side waits (no counterpart in the paper; a diagnostic).  Launches one
 * warp that waits, with the same wait routine the distance kernels use, on a barrier that nothing will
 * ever complete, for at most `limit_cycles` SM clocks (1 .. 2e9).  The wait must give up by itself: after
 * the stream has been synchronised *status reads DETOX_ERR_TIMEOUT (any other value is a failure of the
 * wait routine), the kernel has exited normally and the context is intact.
 *   status  dev, one int32 (cleared by the call)
 * ------------------------------------------------------------------------------------------- */
detox_status detox_selftest_bounded_wait(int32_t* status, int64_t limit_cycles, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Which operand split the tensor-core distance pass (17 .. 256 aligned rows; Section 4, "Improved speed": the
 * O(p^2 d) part of Multi-Krum and Bulyan) tries first.  Process-wide; returns the previous mode; any other value of
 * `mode` only queries.
 *   DETOX_SPLIT_AUTO  (default) every entry as two fp16 numbers after a per-row power-of-two scale; a check after the
 *                     pass repeats it with the split-TF32 kernels when an entry left the fp16 range (distances are
 *                     the same to within the accuracy both give; only the time differs)
 *   DETOX_SPLIT_TF32  the split-TF32 kernels (three-product TF32 with the cross terms folded) from the start
 * A switch for measurements and tests; not meant to be flipped while calls are in flight on other threads.
 * ------------------------------------------------------------------------------------------- */
enum { DETOX_SPLIT_AUTO = 0, DETOX_SPLIT_TF32 = 1 };
int detox_tc_split_mode(int mode);

/* How many calls on the current device have had their tensor-core distance pass repeated so far in this process:
 * by the split-TF32 kernels after an entry left the fp16 range, or without the common vector after the check
 * withdrew it (a diagnostic counter, no counterpart in the paper).  Waits for the device's pending work;
 * ~0 on a CUDA error. */
unsigned long long detox_tc_repeated_passes(void);

/* Number of kernels this library has launched in this process so far (a diagnostic counter, no counterpart in
 * the paper; the one piece of state the library keeps, besides the scratch of detox_vote_noalloc). */
unsigned long long detox_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* DETOX_H_ */
