// C ABI of libdetox: argument validation, workspace carving and kernel sequencing.
// Nothing here touches gradient data on the host, allocates, or synchronises.
#include <string.h>

#include <atomic>

#include "common.cuh"

using namespace detox;

namespace detox {
namespace {
std::atomic<unsigned long long> g_kernel_launches{0};
}
detox_status launch_status() {
    g_kernel_launches.fetch_add(1, std::memory_order_relaxed);
    return cudaGetLastError() == cudaSuccess ? DETOX_OK : DETOX_ERR_CUDA;
}
}  // namespace detox

namespace {

constexpr size_t kStatusBytes = 256;   // the device status word has an aligned slot of its own

bool ws_ok(const void* ws, size_t have, size_t need) {
    if (need == 0) return true;
    return ws != nullptr && (reinterpret_cast<uintptr_t>(ws) & 255u) == 0 && have >= need;
}

// members must be a partition of 0..n-1 into n/r groups
detox_status check_groups(int n, int r, const int32_t* members, IdTable* tab) {
    if (n < 1 || n > kMaxRows || r < 1 || r > kMaxR || (r & 1) == 0 || n % r != 0 || !members)
        return (n > kMaxRows || r > kMaxR) ? DETOX_ERR_UNSUPPORTED : DETOX_ERR_BAD_ARG;
    bool seen[kMaxRows];
    memset(seen, 0, sizeof(seen));
    for (int k = 0; k < n; ++k) {
        int32_t id = members[k];
        if (id < 0 || id >= n || seen[id]) return DETOX_ERR_BAD_ARG;
        seen[id] = true;
        tab->id[k] = (uint16_t)id;
    }
    return DETOX_OK;
}

detox_status check_sets(int G, int S, const int32_t* offsets, const int32_t* set_members, SetTable* tab) {
    if (G < 1 || G > kMaxRows || S < 1 || S > G || !offsets || !set_members) return DETOX_ERR_BAD_ARG;
    if (offsets[0] != 0 || offsets[S] != G) return DETOX_ERR_BAD_ARG;
    for (int s = 0; s < S; ++s)
        if (offsets[s + 1] <= offsets[s]) return DETOX_ERR_BAD_ARG;  // empty or unordered set
    bool seen[kMaxRows];
    memset(seen, 0, sizeof(seen));
    for (int k = 0; k < G; ++k) {
        int32_t v = set_members[k];
        if (v < 0 || v >= G || seen[v]) return DETOX_ERR_BAD_ARG;
        seen[v] = true;
        tab->member[k] = (uint16_t)v;
    }
    for (int s = 0; s <= S; ++s) tab->offset[s] = (uint16_t)offsets[s];
    return DETOX_OK;
}

detox_status check_matrix(const float* X, int64_t ld, int m, int64_t d) {
    if (!X || m < 1 || d < 1 || ld < d) return DETOX_ERR_BAD_ARG;
    if ((reinterpret_cast<uintptr_t>(X) & 3u) != 0) return DETOX_ERR_BAD_ARG;
    if (m > kMaxRows) return DETOX_ERR_UNSUPPORTED;
    return DETOX_OK;
}

// workspace of the Krum-type aggregators: D | distance scratch | selection scratch | index list
struct KrumWs {
    int* status;
    double* D;
    void* dist;
    void* select;
    int32_t* sel;
    int32_t* mapped;   // the selection as rows of X when the m rows are given by a row list
    size_t total;
};

KrumWs krum_ws(void* ws, int m, int64_t d) {
    KrumWs k;
    char* p = static_cast<char*>(ws);
    size_t off = 0;
    k.status = reinterpret_cast<int*>(p + off);   // first word of the workspace: device-side status
    off += kStatusBytes;
    k.D = reinterpret_cast<double*>(p + off);
    off += align_up((size_t)m * m * sizeof(double));
    k.dist = p + off;
    off += dist_ws_bytes(m, d);
    k.select = p + off;
    off += select_ws_bytes(m);
    k.sel = reinterpret_cast<int32_t*>(p + off);
    off += align_up((size_t)m * sizeof(int32_t));
    k.mapped = reinterpret_cast<int32_t*>(p + off);
    off += align_up((size_t)m * sizeof(int32_t));
    k.total = off;
    return k;
}

// The filtering step folded into the distance pass (more than 16 votes of groups of three): the m rows are the votes,
// `rows` is winner[], which the pass fills in before anything reads it.
struct VoteFuse {
    const IdTable* members;
    int n;
    void* vote_ws;     // the vote's workspace words (cleared by the caller)
    float* Z;          // where the votes go if the pass has to be repeated on stored rows
    int64_t ldz;
    int32_t* winner;
};

// `rows` (optional, device, m <= 16): the m rows are X[rows[i]], a negative entry standing for a zero row
// (this is how the votes are consumed straight from the workers' rows through winner[], without a copy).
//
// `status` (device): the word that a bounded device-side wait sets to DETOX_ERR_TIMEOUT when it runs out.  NULL: the
// first word of `ws`, cleared here (the stand-alone aggregators).  Otherwise the caller's word, which the caller has
// cleared and which is only ever set, never cleared, from here on (the pipeline: one word for all its stages).
detox_status run_multikrum(const float* X, int64_t ld, int m, int64_t d, const int32_t* rows, int f, int m_sel,
                           float* out, int32_t* sel, double* scores, void* ws, int* status, cudaStream_t s,
                           const VoteFuse* vf = nullptr) {
    KrumWs k = krum_ws(ws, m, d);
    const bool own_status = status == nullptr;
    if (own_status) status = k.status;
    int32_t* sel_buf = sel ? sel : k.sel;
    detox_status st;
    if (m >= 2 && m <= 16) {   // distance pass, then one small kernel for everything up to the chosen rows
        int nblocks = 0;
        if ((st = launch_sqdist_partials(X, ld, m, d, rows, k.dist, status, own_status, &nblocks, s)) != DETOX_OK) return st;
        st = launch_krum_small(false, static_cast<const double*>(k.dist), nblocks, m, f, m_sel, rows, sel_buf, k.mapped,
                               scores, own_status && !sqdist_partials_use_status(m, X, ld, d) ? status : nullptr, s);
        if (st != DETOX_OK) return st;
        return launch_mean_rows(X, ld, d, rows ? k.mapped : sel_buf, m_sel, out, s);
    }
    if (own_status && cudaMemsetAsync(status, 0, sizeof(int), s) != cudaSuccess) return DETOX_ERR_CUDA;
    st = vf ? launch_sqdist_vote_tc(X, ld, vf->n, d, *vf->members, vf->winner, vf->vote_ws, vf->Z, vf->ldz, k.D, k.dist,
                                    status, s)
            : launch_sqdist(X, ld, m, d, rows, k.D, k.dist, status, s);
    if (st != DETOX_OK) return st;
    st = launch_multikrum_select(k.D, m, f, m_sel, sel_buf, scores, k.select, s);
    if (st != DETOX_OK) return st;
    const int32_t* take = sel_buf;
    if (rows) {
        if ((st = launch_map_indices(sel_buf, rows, m_sel, k.mapped, s)) != DETOX_OK) return st;
        take = k.mapped;
    }
    return launch_mean_rows(X, ld, d, take, m_sel, out, s);
}

detox_status run_bulyan(const float* X, int64_t ld, int m, int64_t d, const int32_t* rows, int f, float* out,
                        int32_t* sel, void* ws, int* status, cudaStream_t s, const VoteFuse* vf = nullptr) {
    KrumWs k = krum_ws(ws, m, d);
    const bool own_status = status == nullptr;
    if (own_status) status = k.status;
    int32_t* sel_buf = sel ? sel : k.sel;
    const int theta = m - 2 * f, beta = theta - 2 * f;
    detox_status st;
    if (m >= 2 && m <= 16) {   // distance pass, then one small kernel for everything up to the chosen rows
        int nblocks = 0;
        if ((st = launch_sqdist_partials(X, ld, m, d, rows, k.dist, status, own_status, &nblocks, s)) != DETOX_OK) return st;
        st = launch_krum_small(true, static_cast<const double*>(k.dist), nblocks, m, f, 0, rows, sel_buf, k.mapped, nullptr,
                               own_status && !sqdist_partials_use_status(m, X, ld, d) ? status : nullptr, s);
        if (st != DETOX_OK) return st;
        return launch_coord_select(X, ld, theta, d, rows ? k.mapped : sel_buf, beta, out, s);
    }
    if (own_status && cudaMemsetAsync(status, 0, sizeof(int), s) != cudaSuccess) return DETOX_ERR_CUDA;
    st = vf ? launch_sqdist_vote_tc(X, ld, vf->n, d, *vf->members, vf->winner, vf->vote_ws, vf->Z, vf->ldz, k.D, k.dist,
                                    status, s)
            : launch_sqdist(X, ld, m, d, rows, k.D, k.dist, status, s);
    if (st != DETOX_OK) return st;
    st = launch_bulyan_select(k.D, m, f, sel_buf, k.select, s);
    if (st != DETOX_OK) return st;
    const int32_t* take = sel_buf;
    if (rows) {
        if ((st = launch_map_indices(sel_buf, rows, theta, k.mapped, s)) != DETOX_OK) return st;
        take = k.mapped;
    }
    return launch_coord_select(X, ld, theta, d, take, beta, out, s);
}

detox_status check_multikrum(int m, int f, int m_sel) {
    if (f < 0 || m_sel < 1 || m_sel > m) return DETOX_ERR_BAD_ARG;
    return DETOX_OK;
}
detox_status check_bulyan(int m, int f) {
    if (f < 0) return DETOX_ERR_BAD_ARG;
    if (f == 0) return DETOX_OK;  // theta = beta = m: the plain mean
    return m >= 4 * f + 3 ? DETOX_OK : DETOX_ERR_BAD_ARG;
}

int64_t pad_ld(int64_t d) { return (d + 31) / 32 * 32; }

bool krum_type(int a) { return a == DETOX_AGG_MULTIKRUM || a == DETOX_AGG_BULYAN; }

// rows a Krum-type A_0 keeps from a vote set of k rows
int a0_selected(const detox_pipeline_desc* p, int k) {
    if (p->a0 == DETOX_AGG_BULYAN) return k - 2 * p->f;
    return p->m_sel > 0 ? p->m_sel : (k - p->f > 1 ? k - p->f : 1);
}

// With A_0 = none the votes are rows of X, so A_1 can read them through winner[] and the votes need not be
// written: always for the per-coordinate aggregators, and for the Krum type up to 16 votes (the
// direct-difference distance kernel takes a row list; the tensor-core Gram wants consecutive rows).
bool votes_by_index(const detox_pipeline_desc* p) {
    if (krum_type(p->a0)) {
        // Multi-Krum / Bulyan inside the vote sets: every set of at most 16 votes is read through its winners
        for (int s = 0; s < p->n_sets; ++s)
            if (p->set_offsets[s + 1] - p->set_offsets[s] > 16) return false;
        return true;
    }
    if (p->a0 != DETOX_AGG_NONE || p->a1 == DETOX_AGG_GEOMETRIC_MEDIAN) return false;
    return !krum_type(p->a1) || p->n / p->r <= 16;
}

struct PipeWs {
    int* status;                 // first word of the workspace: DETOX_ERR_TIMEOUT if a bounded device-side wait ran out
    int32_t* winner_set_order;   // Krum-type A_0: winners in set order
    int32_t* sel_local;          // Krum-type A_0: rows chosen inside the current set
    void* vote;
    float* Z;
    float* M;
    int32_t* winner;
    void* agg;
    size_t total;
    int64_t ldz;
};

PipeWs pipe_ws(void* ws, const detox_pipeline_desc* p) {
    PipeWs w;
    char* base = static_cast<char*>(ws);
    const int G = p->n / p->r;
    const int rows1 = p->a0 != DETOX_AGG_NONE ? p->n_sets : G;
    size_t off = 0;
    w.ldz = pad_ld(p->d);
    w.status = reinterpret_cast<int*>(base);
    off += kStatusBytes;
    w.vote = base + off;         // directly behind the status word: the vote's clearing memset takes both
    off += vote_ws_bytes(p->n, p->r);
    w.winner = reinterpret_cast<int32_t*>(base + off);
    off += align_up((size_t)G * sizeof(int32_t));
    w.Z = reinterpret_cast<float*>(base + off);
    if (p->a0 != DETOX_AGG_MEAN && !votes_by_index(p))
        off += align_up((size_t)G * w.ldz * sizeof(float));   // the votes are stored only when a stage needs them as a matrix
    w.M = reinterpret_cast<float*>(base + off);
    if (p->a0 != DETOX_AGG_NONE) off += align_up((size_t)p->n_sets * w.ldz * sizeof(float));
    w.winner_set_order = reinterpret_cast<int32_t*>(base + off);
    off += align_up((size_t)G * sizeof(int32_t));
    w.sel_local = reinterpret_cast<int32_t*>(base + off);
    off += align_up((size_t)G * sizeof(int32_t));
    w.agg = base + off;
    if (krum_type(p->a1)) off += krum_ws(nullptr, rows1, p->d).total;
    if (p->a1 == DETOX_AGG_GEOMETRIC_MEDIAN) off += geomed_ws_bytes(p->d);
    if (krum_type(p->a0)) {
        // the sets run one after another in the same region; its size is the largest any set needs (the need is not
        // monotone in the set size: the distance kernels change plan with the row count)
        size_t need = 0;
        for (int s = 0; s < p->n_sets; ++s) {
            const int k = p->set_offsets[s + 1] - p->set_offsets[s];
            const size_t t = krum_ws(nullptr, k, p->d).total;
            need = t > need ? t : need;
        }
        off += need;
    }
    w.total = off;
    return w;
}

detox_status check_desc(const detox_pipeline_desc* p) {
    if (!p || p->d < 1) return DETOX_ERR_BAD_ARG;
    if (p->n < 1 || p->r < 1 || (p->r & 1) == 0 || p->n % p->r != 0) return DETOX_ERR_BAD_ARG;
    if (p->n > kMaxRows || p->r > kMaxR) return DETOX_ERR_UNSUPPORTED;
    if (p->a0 != DETOX_AGG_NONE && p->a0 != DETOX_AGG_MEAN && p->a0 != DETOX_AGG_SIGN_MAJORITY && !krum_type(p->a0))
        return DETOX_ERR_BAD_ARG;
    const int G = p->n / p->r;
    if (p->a0 != DETOX_AGG_NONE && (p->n_sets < 1 || p->n_sets > G)) return DETOX_ERR_BAD_ARG;
    if (krum_type(p->a0)) {
        // Multi-Krum / Bulyan inside every vote set (f, m_sel belong to A_0), then a plain A_1 over the set results
        if (p->a1 != DETOX_AGG_MEAN && p->a1 != DETOX_AGG_COORD_MEDIAN && p->a1 != DETOX_AGG_GEOMETRIC_MEDIAN)
            return DETOX_ERR_UNSUPPORTED;  // f and m_sel are A_0's
        if (p->a1 == DETOX_AGG_GEOMETRIC_MEDIAN && (p->gm_iters < 0 || !(p->gm_eps > 0.f) || p->n_sets > 32))
            return p->n_sets > 32 ? DETOX_ERR_UNSUPPORTED : DETOX_ERR_BAD_ARG;
        if (!p->set_offsets || p->f < 0 || p->m_sel < 0) return DETOX_ERR_BAD_ARG;
        if (p->set_offsets[0] != 0 || p->set_offsets[p->n_sets] != G) return DETOX_ERR_BAD_ARG;
        for (int s = 0; s < p->n_sets; ++s) {
            const int k = p->set_offsets[s + 1] - p->set_offsets[s];
            if (k < 1) return DETOX_ERR_BAD_ARG;
            if (p->a0 == DETOX_AGG_BULYAN && check_bulyan(k, p->f) != DETOX_OK) return DETOX_ERR_BAD_ARG;
            if (p->a0 == DETOX_AGG_MULTIKRUM && p->m_sel > k) return DETOX_ERR_BAD_ARG;
        }
        return DETOX_OK;
    }
    const int rows1 = p->a0 != DETOX_AGG_NONE ? p->n_sets : G;
    switch (p->a1) {
        case DETOX_AGG_MEAN:
        case DETOX_AGG_SIGN_MAJORITY:
        case DETOX_AGG_COORD_MEDIAN: return DETOX_OK;
        case DETOX_AGG_TRIMMED_MEAN: return (p->f >= 0 && rows1 - 2 * p->f >= 1) ? DETOX_OK : DETOX_ERR_BAD_ARG;
        case DETOX_AGG_GEOMETRIC_MEDIAN:
            if (p->gm_iters < 0 || !(p->gm_eps > 0.f)) return DETOX_ERR_BAD_ARG;
            return rows1 <= 32 ? DETOX_OK : DETOX_ERR_UNSUPPORTED;
        case DETOX_AGG_MULTIKRUM: return check_multikrum(rows1, p->f, p->m_sel);
        case DETOX_AGG_BULYAN: return check_bulyan(rows1, p->f);
        default: return DETOX_ERR_BAD_ARG;
    }
}

}  // namespace

extern "C" {

const char* detox_status_string(detox_status s) {
    switch (s) {
        case DETOX_OK: return "ok";
        case DETOX_ERR_BAD_ARG: return "bad argument";
        case DETOX_ERR_UNSUPPORTED: return "unsupported size or option";
        case DETOX_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case DETOX_ERR_CUDA: return "CUDA error";
        case DETOX_ERR_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}

size_t detox_vote_workspace_bytes(int n, int r) {
    if (n < 1 || r < 1 || n % r != 0) return 0;
    return vote_ws_bytes(n, r);
}

detox_status detox_vote(const float* X, int64_t ld, int n, int r, int64_t d, const int32_t* members, float* Z,
                        int64_t ldz, int32_t* winner, void* ws, size_t ws_bytes, void* stream) {
    IdTable tab;
    detox_status st = check_groups(n, r, members, &tab);
    if (st != DETOX_OK) return st;
    if ((st = check_matrix(X, ld, n, d)) != DETOX_OK) return st;
    if (!winner) return DETOX_ERR_BAD_ARG;
    if (Z && (ldz < d || (reinterpret_cast<uintptr_t>(Z) & 3u))) return DETOX_ERR_BAD_ARG;
    if (!ws_ok(ws, ws_bytes, vote_ws_bytes(n, r))) return DETOX_ERR_WORKSPACE;
    return launch_vote(X, ld, n, r, d, tab, Z, ldz, winner, ws, static_cast<cudaStream_t>(stream));
}

detox_status detox_hier_mean(const float* Z, int64_t ldz, int G, int64_t d, const int32_t* set_offsets,
                             const int32_t* set_members, int S, float* M, int64_t ldm, void* stream) {
    SetTable tab;
    detox_status st = check_sets(G, S, set_offsets, set_members, &tab);
    if (st != DETOX_OK) return st;
    if ((st = check_matrix(Z, ldz, G, d)) != DETOX_OK) return st;
    if (!M || ldm < d || (reinterpret_cast<uintptr_t>(M) & 3u)) return DETOX_ERR_BAD_ARG;
    return launch_hier_mean(Z, ldz, d, tab, S, M, ldm, static_cast<cudaStream_t>(stream));
}

detox_status detox_vote_hier_mean(const float* X, int64_t ld, int n, int r, int64_t d, const int32_t* members,
                                  const int32_t* set_offsets, const int32_t* set_members, int S, float* M,
                                  int64_t ldm, int32_t* winner, void* ws, size_t ws_bytes, void* stream) {
    IdTable groups;
    detox_status st = check_groups(n, r, members, &groups);
    if (st != DETOX_OK) return st;
    SetTable sets;
    if ((st = check_sets(n / r, S, set_offsets, set_members, &sets)) != DETOX_OK) return st;
    if ((st = check_matrix(X, ld, n, d)) != DETOX_OK) return st;
    if (!winner || !M || ldm < d || (reinterpret_cast<uintptr_t>(M) & 3u)) return DETOX_ERR_BAD_ARG;
    if (!ws_ok(ws, ws_bytes, vote_ws_bytes(n, r))) return DETOX_ERR_WORKSPACE;
    return launch_vote_mean(X, ld, n, r, d, groups, sets, S, M, ldm, winner, ws, static_cast<cudaStream_t>(stream));
}

size_t agg_coord_median_workspace_bytes(int m, int64_t d) {
    (void)m;
    (void)d;
    return 0;
}

detox_status agg_coord_median(const float* X, int64_t ld, int m, int64_t d, float* out, void* ws, size_t ws_bytes,
                              void* stream) {
    (void)ws;
    (void)ws_bytes;
    detox_status st = check_matrix(X, ld, m, d);
    if (st != DETOX_OK) return st;
    if (!out || (reinterpret_cast<uintptr_t>(out) & 3u)) return DETOX_ERR_BAD_ARG;
    return launch_coord_select(X, ld, m, d, nullptr, 0, out, static_cast<cudaStream_t>(stream));
}

detox_status agg_trimmed_mean(const float* X, int64_t ld, int m, int64_t d, int trim, float* out, void* stream) {
    detox_status st = check_matrix(X, ld, m, d);
    if (st != DETOX_OK) return st;
    if (!out || (reinterpret_cast<uintptr_t>(out) & 3u) || trim < 0 || m - 2 * trim < 1) return DETOX_ERR_BAD_ARG;
    return launch_coord_select(X, ld, m, d, nullptr, -(m - 2 * trim), out, static_cast<cudaStream_t>(stream));
}

detox_status agg_sign_majority(const float* X, int64_t ld, int m, int64_t d, float* out, void* stream) {
    detox_status st = check_matrix(X, ld, m, d);
    if (st != DETOX_OK) return st;
    if (!out || (reinterpret_cast<uintptr_t>(out) & 3u)) return DETOX_ERR_BAD_ARG;
    return launch_mean_rows(X, ld, d, nullptr, m, out, static_cast<cudaStream_t>(stream), true);
}

size_t agg_geometric_median_workspace_bytes(int m, int64_t d) {
    if (m < 1 || m > 32 || d < 1) return 0;
    return geomed_ws_bytes(d);
}

detox_status agg_geometric_median(const float* X, int64_t ld, int m, int64_t d, int iters, float eps, float* out,
                                  void* ws, size_t ws_bytes, void* stream) {
    detox_status st = check_matrix(X, ld, m, d);
    if (st != DETOX_OK) return st;
    if (!out || (reinterpret_cast<uintptr_t>(out) & 3u) || iters < 0 || !(eps > 0.f)) return DETOX_ERR_BAD_ARG;
    if (m > 32) return DETOX_ERR_UNSUPPORTED;
    if (!ws_ok(ws, ws_bytes, geomed_ws_bytes(d))) return DETOX_ERR_WORKSPACE;
    return launch_geometric_median(X, ld, m, d, iters, eps, out, ws, static_cast<cudaStream_t>(stream));
}

size_t agg_multikrum_workspace_bytes(int m, int64_t d) {
    if (m < 1 || m > kMaxRows || d < 1) return 0;
    return krum_ws(nullptr, m, d).total;
}

detox_status agg_multikrum(const float* X, int64_t ld, int m, int64_t d, int f, int m_sel, float* out, int32_t* sel,
                           double* scores, void* ws, size_t ws_bytes, void* stream) {
    detox_status st = check_matrix(X, ld, m, d);
    if (st != DETOX_OK) return st;
    if ((st = check_multikrum(m, f, m_sel)) != DETOX_OK) return st;
    if (!out || (reinterpret_cast<uintptr_t>(out) & 3u)) return DETOX_ERR_BAD_ARG;
    if (!ws_ok(ws, ws_bytes, krum_ws(nullptr, m, d).total)) return DETOX_ERR_WORKSPACE;
    return run_multikrum(X, ld, m, d, nullptr, f, m_sel, out, sel, scores, ws, nullptr, static_cast<cudaStream_t>(stream));
}

size_t agg_bulyan_workspace_bytes(int m, int64_t d) {
    if (m < 1 || m > kMaxRows || d < 1) return 0;
    return krum_ws(nullptr, m, d).total;
}

detox_status agg_bulyan(const float* X, int64_t ld, int m, int64_t d, int f, float* out, int32_t* sel, void* ws,
                        size_t ws_bytes, void* stream) {
    detox_status st = check_matrix(X, ld, m, d);
    if (st != DETOX_OK) return st;
    if ((st = check_bulyan(m, f)) != DETOX_OK) return st;
    if (!out || (reinterpret_cast<uintptr_t>(out) & 3u)) return DETOX_ERR_BAD_ARG;
    if (!ws_ok(ws, ws_bytes, krum_ws(nullptr, m, d).total)) return DETOX_ERR_WORKSPACE;
    return run_bulyan(X, ld, m, d, nullptr, f, out, sel, ws, nullptr, static_cast<cudaStream_t>(stream));
}

size_t agg_pairwise_sqdist_workspace_bytes(int m, int64_t d) {
    if (m < 1 || m > kMaxRows || d < 1) return 0;
    return kStatusBytes + dist_ws_bytes(m, d);
}

detox_status agg_pairwise_sqdist(const float* X, int64_t ld, int m, int64_t d, double* D, void* ws, size_t ws_bytes,
                                 void* stream) {
    detox_status st = check_matrix(X, ld, m, d);
    if (st != DETOX_OK) return st;
    if (!D || (reinterpret_cast<uintptr_t>(D) & 7u)) return DETOX_ERR_BAD_ARG;
    if (!ws_ok(ws, ws_bytes, kStatusBytes + dist_ws_bytes(m, d))) return DETOX_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int* status = static_cast<int*>(ws);
    if (cudaMemsetAsync(status, 0, sizeof(int), s) != cudaSuccess) return DETOX_ERR_CUDA;
    return launch_sqdist(X, ld, m, d, nullptr, D, static_cast<char*>(ws) + kStatusBytes, status, s);
}

int detox_tc_split_mode(int mode) { return tc_split_mode(mode); }

unsigned long long detox_tc_repeated_passes(void) { return tc_repeated_passes(); }

unsigned long long detox_kernel_launch_count(void) { return g_kernel_launches.load(std::memory_order_relaxed); }

size_t detox_aggregate_workspace_bytes(const detox_pipeline_desc* desc) {
    if (check_desc(desc) != DETOX_OK) return 0;
    return pipe_ws(nullptr, desc).total;
}

detox_status detox_aggregate(const detox_pipeline_desc* p, const float* X, int64_t ld, float* out, int32_t* winner,
                             int32_t* sel, int32_t* sel_workers, void* ws, size_t ws_bytes, void* stream) {
    detox_status st = check_desc(p);
    if (st != DETOX_OK) return st;
    IdTable groups;
    if ((st = check_groups(p->n, p->r, p->members, &groups)) != DETOX_OK) return st;
    if ((st = check_matrix(X, ld, p->n, p->d)) != DETOX_OK) return st;
    if (!out || (reinterpret_cast<uintptr_t>(out) & 3u)) return DETOX_ERR_BAD_ARG;
    const int G = p->n / p->r;
    SetTable sets;
    if (p->a0 != DETOX_AGG_NONE &&
        (st = check_sets(G, p->n_sets, p->set_offsets, p->set_members, &sets)) != DETOX_OK)
        return st;
    PipeWs w = pipe_ws(ws, p);
    if (!ws_ok(ws, ws_bytes, w.total)) return DETOX_ERR_WORKSPACE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    int32_t* win = winner ? winner : w.winner;

    // filtering step, then A_0, then A_1 (the mean as A_0 is folded into the vote's pass)
    const float* rows = w.Z;
    int64_t row_ld = w.ldz;
    const int32_t* row_list = nullptr;
    VoteFuse fuse;
    const VoteFuse* vf = nullptr;
    int m = G;
    if (p->a0 == DETOX_AGG_MEAN) {
        // A_1 that works coordinate by coordinate over at most 16 set means: everything in one pass over X
        const bool coordwise = p->a1 == DETOX_AGG_COORD_MEDIAN || p->a1 == DETOX_AGG_TRIMMED_MEAN || p->a1 == DETOX_AGG_MEAN;
        if (coordwise && vote_mean_select_supported(X, ld, p->r, p->n_sets, out)) {
            const int beta = p->a1 == DETOX_AGG_TRIMMED_MEAN ? -(p->n_sets - 2 * p->f) : 0;
            return launch_vote_mean_select(X, ld, p->n, p->r, p->d, groups, sets, p->n_sets, beta, p->a1 == DETOX_AGG_MEAN, out,
                                           win, w.vote, s, kStatusBytes);
        }
        if ((st = launch_vote_mean(X, ld, p->n, p->r, p->d, groups, sets, p->n_sets, w.M, w.ldz, win, w.vote, s, kStatusBytes)) !=
            DETOX_OK)
            return st;
        rows = w.M;
        m = p->n_sets;
    } else if (p->a0 == DETOX_AGG_SIGN_MAJORITY) {
        // signSGD pairing (Section 5.2, setup 4): coordinate-wise sign majority inside every vote set
        if ((st = launch_vote(X, ld, p->n, p->r, p->d, groups, w.Z, w.ldz, win, w.vote, s, kStatusBytes)) != DETOX_OK) return st;
        if ((st = launch_hier_mean(w.Z, w.ldz, p->d, sets, p->n_sets, w.M, w.ldz, s, true)) != DETOX_OK) return st;
        rows = w.M;
        m = p->n_sets;
    } else if (krum_type(p->a0)) {
        // The paper's preferred pairings (Section 5.2, setups 2 and 3): Multi-Krum or Bulyan inside every
        // vote set, then A_1.  The vote runs over the groups in set order, so each set's votes are
        // consecutive rows of Z and the aggregators take them as ordinary matrices.
        IdTable in_set_order;
        for (int k = 0; k < G; ++k)
            for (int a = 0; a < p->r; ++a) in_set_order.id[k * p->r + a] = groups.id[sets.member[k] * p->r + a];
        // Sets of at most 16 votes take the distance kernels that read rows through a list: the votes are then the
        // winners' rows of X (a negative entry: the zero row) and no vote matrix is written.
        const bool by_index = votes_by_index(p);
        if ((st = launch_vote(X, ld, p->n, p->r, p->d, in_set_order, by_index ? nullptr : w.Z, w.ldz, w.winner_set_order,
                              w.vote, s, kStatusBytes)) != DETOX_OK)
            return st;
        if ((st = launch_scatter_by_set_order(w.winner_set_order, sets, G, win, s)) != DETOX_OK) return st;
        int emitted = 0;
        for (int t = 0; t < p->n_sets; ++t) {
            const int b = sets.offset[t], k = sets.offset[t + 1] - b;
            const int keep = a0_selected(p, k);
            const float* rows_t = by_index ? X : w.Z + (int64_t)b * w.ldz;
            const int64_t ld_t = by_index ? ld : w.ldz;
            const int32_t* list_t = by_index ? w.winner_set_order + b : nullptr;
            float* out_t = w.M + (int64_t)t * w.ldz;
            st = p->a0 == DETOX_AGG_MULTIKRUM
                     ? run_multikrum(rows_t, ld_t, k, p->d, list_t, p->f, keep, out_t, w.sel_local, nullptr, w.agg, w.status, s)
                     : run_bulyan(rows_t, ld_t, k, p->d, list_t, p->f, out_t, w.sel_local, w.agg, w.status, s);
            if (st != DETOX_OK) return st;
            st = launch_map_set_selection(w.sel_local, keep, sets, b, w.winner_set_order, sel ? sel + emitted : nullptr,
                                          sel_workers ? sel_workers + emitted : nullptr, s);
            if (st != DETOX_OK) return st;
            emitted += keep;
        }
        rows = w.M;
        m = p->n_sets;
    } else if (votes_by_index(p)) {
        // The votes are rows of X: only winner[] is produced and A_1 reads the winners' rows through it
        // (a group without a majority has winner -1, which the consumers take as a zero row).
        if ((st = launch_vote(X, ld, p->n, p->r, p->d, groups, nullptr, 0, win, w.vote, s, kStatusBytes)) != DETOX_OK) return st;
        rows = X;
        row_ld = ld;
        row_list = win;
    } else if (krum_type(p->a1) && sqdist_vote_tc_supported(X, ld, p->n, p->r, p->d)) {
        // More than 16 votes of groups of three under a Krum-type A_1: the vote runs inside the tensor-core distance
        // pass, winner[] comes out of it, and everything after the distances reads the winners' rows of X.
        if (cudaMemsetAsync(w.status, 0, kStatusBytes + vote_ws_bytes(p->n, p->r), s) != cudaSuccess) return DETOX_ERR_CUDA;
        fuse = VoteFuse{&groups, p->n, w.vote, w.Z, w.ldz, win};
        vf = &fuse;
        rows = X;
        row_ld = ld;
        row_list = win;
    } else if ((st = launch_vote(X, ld, p->n, p->r, p->d, groups, w.Z, w.ldz, win, w.vote, s, kStatusBytes)) != DETOX_OK) {
        return st;
    }
    int cnt = 0;
    int32_t* sel_buf = nullptr;
    switch (p->a1) {
        case DETOX_AGG_MEAN: st = launch_mean_rows(rows, row_ld, p->d, row_list, m, out, s); break;
        case DETOX_AGG_SIGN_MAJORITY: st = launch_mean_rows(rows, row_ld, p->d, row_list, m, out, s, true); break;
        case DETOX_AGG_COORD_MEDIAN: st = launch_coord_select(rows, row_ld, m, p->d, row_list, 0, out, s); break;
        case DETOX_AGG_TRIMMED_MEAN:
            st = launch_coord_select(rows, row_ld, m, p->d, row_list, -(m - 2 * p->f), out, s);
            break;
        case DETOX_AGG_GEOMETRIC_MEDIAN:
            st = launch_geometric_median(rows, row_ld, m, p->d, p->gm_iters, p->gm_eps, out, w.agg, s);
            break;
        case DETOX_AGG_MULTIKRUM:
            cnt = p->m_sel;
            sel_buf = sel ? sel : krum_ws(w.agg, m, p->d).sel;
            st = run_multikrum(rows, row_ld, m, p->d, row_list, p->f, p->m_sel, out, sel_buf, nullptr, w.agg, w.status, s, vf);
            break;
        case DETOX_AGG_BULYAN:
            cnt = m - 2 * p->f;
            sel_buf = sel ? sel : krum_ws(w.agg, m, p->d).sel;
            st = run_bulyan(rows, row_ld, m, p->d, row_list, p->f, out, sel_buf, w.agg, w.status, s, vf);
            break;
        default: st = DETOX_ERR_BAD_ARG;
    }
    if (st != DETOX_OK) return st;
    if (sel_workers && sel_buf && p->a0 == DETOX_AGG_NONE) st = launch_map_indices(sel_buf, win, cnt, sel_workers, s);
    return st;
}

}  // extern "C"
