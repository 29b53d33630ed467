// Pairwise squared distances for 16 < m <= 256 on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// G = X X^T is computed with error-compensated TF32: every fp32 x is split into hi = tf32(x) and
// lo = x - hi (exact), and  x_i . x_j  ~=  hi_i.hi_j + hi_i.lo_j + lo_i.hi_j.  The last two terms are
// folded by symmetry: with T = hi (hi + 2 lo)^T, accumulated as two MMAs per K-step into ONE fp32
// accumulator in tensor memory, G_ij = (T_ij + T_ji) / 2.  Both MMA operands come from the same
// shared-memory tiles (rows of X), so every row of X is read from HBM exactly once.
//
// One persistent CTA per SM: copy-issuing threads stream column blocks of all m rows into shared memory with
// TMA (rows and columns outside the matrix arrive as zeros), warps 0-15 form 2 lo = 2 (x - (x with its low 13
// bits cleared)) -- the raw fp32 values themselves serve as `hi`, because a TF32 MMA reads only the upper 19
// bits of each word -- and lane 0 of the warps after them (two, or four up to 64 rows) issues the MMAs;
// mbarriers form rings of stages between the roles.  Two kernels share this scheme: up to 128 rows the copies are 64 columns wide, land in a staging ring
// and the transform warps write both MMA operands (see the staged kernel); above, the copies land directly in
// the swizzled hi tile (see the wide kernel).
// Column blocks are dealt round-robin to the CTAs and every 4096 columns of a CTA form a slab; at the end
// of a slab the accumulator is drained into an fp32 partial in global memory (four consecutive slabs of a CTA
// share one: the drain adds to what the slab before left there) and the partials are added in fp64 in a fixed
// order afterwards, so the long sum never lives in one fp32 accumulator and
// the result is deterministic.
//
// The tensor cores add into their fp32 accumulator by truncation, so a long same-sign sum (a row with
// itself, or with a copy of itself) comes out low by about 1e-5 relative per 4096 columns.  The producers
// therefore also accumulate each row's exact squared norm per slab on the CUDA cores; the final
// reduction rescales every slab's T_ij by the mean of (exact norm / tensor-core norm) of rows i and
// j.  The diagonal becomes exact, a pair of identical rows keeps distance zero, and entries
// between unrelated rows (which hover around zero and lose nothing to truncation) are unchanged.
//
// Every wait on an mbarrier is bounded; if one runs out the kernel records DETOX_ERR_TIMEOUT in the
// status word, stops waiting everywhere, frees its tensor memory and returns.
#include <cuda.h>

#include <atomic>

#include "common.cuh"
#include "mbarrier.cuh"
#include "gram_tc.cuh"
#include "tcgen05.cuh"

namespace detox {

namespace {

constexpr int kKB = 32;                      // fp32 columns per K-block: one 128-byte swizzle row
constexpr int kMmaWarps = 2;                   // issuing threads of the wide kernel (the staged kernel has two or four):
                                               // one's bookkeeping overlaps the other's MMAs
constexpr int kTmaWarps = 2;                   // copy-issuing warps of the wide kernel (it uses the first only; the second
                                               // one does the centring)
// copy-issuing threads of the staged kernel: one per group of transform warps (above 64 rows a stage takes HBM longer
// than one thread's wait / expect / copy loop, so one thread keeps up)
__host__ __device__ constexpr int staged_tma_warps(int lx) { return lx; }
constexpr int kCentreWarps = 1;                // forms the vector that is subtracted from every row (when one is)
constexpr int kTcThreads = kProdThreads + 32 * (kMmaWarps + kTmaWarps);   // wide kernel: its second copy warp does the centring
constexpr int kMinReduceChunks = 32, kMaxReduceChunks = 256;

// Slab slots are added up in `chunks` independent groups (one CTA per group and pair of 32-row blocks), enough
// of them to fill the GPU when m is small.
int reduce_chunks(int m, int nitems) {
    const int nt = (m + 31) / 32, pairs = nt * (nt + 1) / 2;
    int c = (8 * kSMs + pairs - 1) / pairs;
    if (c < kMinReduceChunks) c = kMinReduceChunks;
    if (c > kMaxReduceChunks) c = kMaxReduceChunks;
    if (c > nitems) c = nitems;
    return c;
}

// ------------------------------------------------------------------------------------ 128 < m <= 256: wide kernel
//
// The accumulator has two halves of 128 rows, one per MMA-issuing thread; per K-step each thread issues
// A = hi rows of its half with B = hi and with B = 2lo.  Sixteen MMAs of N = ncol per K-block keep the tensor pipe
// busier than the copies, so the copies stay 32 columns wide and land directly in the swizzled hi tile.
constexpr int kMaxWideStages = 4;

struct WidePlan {
    int box_rows;     // rows the TMA box brings in: m rounded up to 8
    int ncol;         // m rounded up to 16
    int tmem_cols;    // power of two >= 2 ncol
    int stages;
    uint32_t lo_off;       // where the 2lo tile starts inside a stage: after 256 hi rows (the second half's A operand
                           // reads rows 128..255)
    uint32_t stage_bytes;
    int nkb_total;    // K-blocks in all: d / 32 rounded up
    int nitems;       // slab slots: grid x the largest number of slabs a CTA has
    int grid;
    size_t smem_bytes;
};

WidePlan wide_plan(int m, int64_t d) {
    WidePlan p;
    p.box_rows = (m + 7) / 8 * 8;
    p.ncol = (m + 15) / 16 * 16;
    p.tmem_cols = 512;
    p.lo_off = 256u * 128u;
    p.stage_bytes = p.lo_off + (uint32_t)p.ncol * 128u;
    p.stages = (int)((kSmemBudget - 2048) / p.stage_bytes);
    if (p.stages > kMaxWideStages) p.stages = kMaxWideStages;
    // K-blocks are dealt round-robin to the CTAs, so that every CTA has the same number of them (to within one)
    // whatever d is, and neighbouring CTAs read neighbouring 128-byte pieces of a row
    p.nkb_total = (int)ceil_div(d, (int64_t)kKB);
    p.grid = p.nkb_total < kSMs ? p.nkb_total : kSMs;
    const int per_cta = (p.nkb_total + p.grid - 1) / p.grid;
    p.nitems = p.grid * (int)ceil_div(ceil_div((int64_t)per_cta, kSlabCols / kKB), (int64_t)kItemSlabs);
    p.smem_bytes = (size_t)p.stage_bytes * p.stages + 1024 /*barriers*/ + 1024 /*alignment slack*/;
    return p;
}

struct WideSmem {
    uint64_t landed[kMaxWideStages];   // TMA bytes of the raw tile have arrived
    uint64_t full[kMaxWideStages];     // the 2lo tile is written: both tiles ready for the MMA
    uint64_t empty[kMaxWideStages];
    uint64_t accum_full;
    uint64_t accum_empty;
    uint64_t c_full[kMaxWideStages];   // the subtracted vector's piece for this stage is written
    uint32_t tmem_base;
    int abort_flag;
    int crow[kMaxCentreRows];
    __align__(16) float cring[kMaxWideStages][kKB];
};

// J = 16-byte pieces per transform thread and K-block (m * 8 / 512, rounded up)
template <int J>
__global__ void __launch_bounds__(kTcThreads, 1)
gram_wide_kernel(const __grid_constant__ CUtensorMap xmap, int m, uint32_t lo_off, uint32_t stage_bytes, int box_rows,
                 int ncol, int tmem_cols, int stages, int nkb_total, int nitems, float* __restrict__ partial,
                 float* __restrict__ norms, const int* __restrict__ centre_ptr,
                 const int* __restrict__ redo_ptr, int* __restrict__ status) {
    // second launch of a call: only runs when the first one's centring was withdrawn
    if (redo_ptr != nullptr && *redo_ptr == 0) return;
    // Centring: centre_ptr[0] rows, listed from centre_ptr[2] on, are averaged column by column and the average is
    // subtracted from every row before the products (distances do not change; 0 rows: nothing is subtracted).
    const int ncentre = *centre_ptr;
    extern __shared__ uint8_t smem_raw[];
    // tiles need 1024-byte alignment for the 128-byte swizzle pattern
    const uint32_t raw = smem_u32(smem_raw);
    uint8_t* base = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
    WideSmem* sm = reinterpret_cast<WideSmem*>(base + (size_t)stage_bytes * stages);
    volatile int* abort_flag = &sm->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&sm->landed[s], 1);
            mbar_init(&sm->full[s], kProdWarps);
            mbar_init(&sm->empty[s], kMmaWarps);
            mbar_init(&sm->c_full[s], 1);
        }
        mbar_init(&sm->accum_full, kMmaWarps);
        mbar_init(&sm->accum_empty, kProdWarps);
        sm->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < ncentre) sm->crow[tid] = centre_ptr[2 + tid];
    // rows beyond the TMA box are never written: clear all tiles once so the padded rows are zeros
    for (uint32_t off = (uint32_t)tid * 16u; off < stage_bytes * (uint32_t)stages; off += kTcThreads * 16u)
        *reinterpret_cast<uint4*>(base + off) = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async_smem();
    if (warp == 0) tmem_alloc(&sm->tmem_base, (uint32_t)tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sm->tmem_base;

    // This CTA owns the K-blocks b, b + G, b + 2G, ... (b = blockIdx.x, G = gridDim.x), t = 0 .. total-1 in its own
    // count; K-block t goes through stage t % stages; a slab is kBlocksPerSlab consecutive ones of them (the last
    // slab may be shorter) and goes to slot b + G * (slab number).
    constexpr int kBlocksPerSlab = (int)(kSlabCols / kKB);
    const int total = (nkb_total - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    const int my_items = (total + kBlocksPerSlab - 1) / kBlocksPerSlab;
    const int last_nkb = total - (my_items - 1) * kBlocksPerSlab;

    if (warp < kProdWarps) {
        // ------------------------------------------------ transform warps, then epilogue of each slab
        const int npieces = m * 8;
        // this thread's pieces are (row, c) = ((tid >> 3) + 64 j, tid & 7) in every K-block; 64 is a multiple of 8,
        // so the swizzle term is the same for all j
        const int row0 = tid >> 3, c = tid & 7;
        const uint32_t off0 = (uint32_t)(row0 >> 3) * 1024u + (uint32_t)(row0 & 7) * 128u + (uint32_t)((c ^ (row0 & 7)) << 4);
        constexpr uint32_t kOffStep = (uint32_t)(kProdThreads / 64) * 1024u;
        uint64_t sq[J];   // packed pair of partial sums of squares per piece (of the centred values)
#pragma unroll
        for (int j = 0; j < J; ++j) sq[j] = 0ull;

        int s = 0, t = 0;
        uint32_t ph = 0;
        for (int li = 0; li < my_items; ++li) {
            const int nkb = li == my_items - 1 ? last_nkb : kBlocksPerSlab;
            const int t_end = li * kBlocksPerSlab + nkb;
            for (; t < t_end; ++t) {
                mbar_wait(&sm->landed[s], ph, abort_flag, status);
                uint8_t* hi_tile = base + (size_t)s * stage_bytes + off0;
                uint8_t* lo_tile = base + (size_t)s * stage_bytes + lo_off + off0;
                if (ncentre == 0) {
#pragma unroll
                    for (int j = 0; j < J; ++j) {
                        if (tid + j * kProdThreads < npieces) {
                            const ulonglong2 x = *reinterpret_cast<const ulonglong2*>(hi_tile + j * kOffStep);
                            sq[j] = fma2(x.x, x.x, fma2(x.y, x.y, sq[j]));
                            *reinterpret_cast<ulonglong2*>(lo_tile + j * kOffStep) = make_ulonglong2(lo2_of(x.x), lo2_of(x.y));
                        }
                    }
                } else {
                    // the hi tile is rewritten in place with the centred values; the warp that forms the subtracted
                    // vector has read its rows by the time c_full completes
                    mbar_wait(&sm->c_full[s], ph, abort_flag, status);
                    const ulonglong2 ck = *reinterpret_cast<const ulonglong2*>(&sm->cring[s][c * 4]);
#pragma unroll
                    for (int j = 0; j < J; ++j) {
                        if (tid + j * kProdThreads < npieces) {
                            const ulonglong2 x = *reinterpret_cast<const ulonglong2*>(hi_tile + j * kOffStep);
                            const ulonglong2 a = make_ulonglong2(sub2(x.x, ck.x), sub2(x.y, ck.y));
                            sq[j] = fma2(a.x, a.x, fma2(a.y, a.y, sq[j]));
                            *reinterpret_cast<ulonglong2*>(hi_tile + j * kOffStep) = a;
                            *reinterpret_cast<ulonglong2*>(lo_tile + j * kOffStep) = make_ulonglong2(lo2_of(a.x), lo2_of(a.y));
                        }
                    }
                }
                fence_proxy_async_smem();   // make the generic-proxy stores visible to the MMA's reads
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm->full[s]);   // one arrival per transform warp
                if (++s == stages) { s = 0; ph ^= 1u; }
            }
            // output slot of this slab, and whether the slab opens / closes it
            const int item = (int)blockIdx.x + (li / kItemSlabs) * (int)gridDim.x;
            const bool opens = li % kItemSlabs == 0, closes = li % kItemSlabs == kItemSlabs - 1 || li == my_items - 1;

            // ---- end of a slab: exact squared norms (the 8 lanes that share a row add up) ...
#pragma unroll
            for (int j = 0; j < J; ++j) {
                float v = __uint_as_float((uint32_t)sq[j]) + __uint_as_float((uint32_t)(sq[j] >> 32));
                v += __shfl_xor_sync(0xffffffffu, v, 1);
                v += __shfl_xor_sync(0xffffffffu, v, 2);
                v += __shfl_xor_sync(0xffffffffu, v, 4);
                const int row = row0 + (kProdThreads / 8) * j;
                if (closes) {
                    if (c == 0 && row < m) norms[(int64_t)item * m + row] = v;
                    sq[j] = 0ull;
                }
            }
            // ... and the accumulator drain: warp w reads TMEM lanes 32*(w%4)..+31 (accumulator row i of a half sits
            // in lane i); the warps that share a lane quarter take 16-column chunks round-robin
            mbar_wait(&sm->accum_full, (uint32_t)(li & 1), abort_flag, status);
            tc_fence_after();
            const int quarter = warp & 3;
            float* out_item = partial + (int64_t)item * m * ncol;
            for (int h = 0; h < 2; ++h) {
                const int row = h * 128 + quarter * 32 + lane;
                for (int cc = warp >> 2; cc * 16 < ncol; cc += kProdWarps / 4) {   // ncol is a multiple of 16
                    uint32_t v[16];
                    tmem_load16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(h * ncol + cc * 16), v);
                    if (row < m) {
                        float* dstp = out_item + (int64_t)row * ncol + cc * 16;
#pragma unroll
                        for (int j = 0; j < 16; j += 4) {
                            const float4 o = make_float4(__uint_as_float(v[j]), __uint_as_float(v[j + 1]), __uint_as_float(v[j + 2]),
                                                         __uint_as_float(v[j + 3]));
                            if (opens) *reinterpret_cast<float4*>(dstp + j) = o;
                            else red_add_f4(dstp + j, o);   // this thread wrote the slot's earlier slabs itself
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm->accum_empty);
        }
        // slots of slabs this CTA does not have (it owns one K-block fewer than others) read as zero
        for (int l2 = (my_items + kItemSlabs - 1) / kItemSlabs; l2 * (int)gridDim.x < nitems; ++l2) {
            const int64_t item = (int64_t)blockIdx.x + (int64_t)l2 * gridDim.x;
            for (int e = tid; e < m * ncol; e += kProdThreads) partial[item * m * ncol + e] = 0.f;
            for (int e = tid; e < m; e += kProdThreads) norms[item * m + e] = 0.f;
        }
    } else if (warp == kProdWarps + kMmaWarps) {
        // ------------------------------------------------ the TMA thread
        if (lane == 0) {
            const uint32_t tx_bytes = (uint32_t)box_rows * 128u;
            int issued = 0;
            int s = 0;
            uint32_t ph = 0;
            int64_t c0 = (int64_t)blockIdx.x * kKB;                  // first column of the current K-block
            for (int t = 0; t < total; ++t) {
                // the MMAs that read this stage are done
                if (!mbar_wait(&sm->empty[s], ph ^ 1u, abort_flag, status)) break;
                mbar_expect_tx(&sm->landed[s], tx_bytes);
                tma_load_2d(base + (size_t)s * stage_bytes, &xmap, (int)c0, 0, &sm->landed[s]);
                issued = t + 1;
                if (++s == stages) { s = 0; ph ^= 1u; }
                c0 += (int64_t)gridDim.x * kKB;
            }
            if (*abort_flag) {
                // give the copies still in flight a bounded time to land before the CTA goes away
                for (int tt = issued > stages ? issued - stages : 0; tt < issued; ++tt) {
                    const int s2 = (int)((uint32_t)tt % (uint32_t)stages);
                    const uint32_t ph2 = ((uint32_t)tt / (uint32_t)stages) & 1u;
                    for (uint32_t spin = 0; spin < (1u << 16) && !mbar_test(&sm->landed[s2], ph2); ++spin) __nanosleep(64);
                }
            }
        }
    } else if (warp == kProdWarps + kMmaWarps + 1) {
        // ------------------------------------------------ the centring warp: lane l averages column l of the listed
        // rows of every K-block as it lands (non-finite entries count as zero) and hands the 32 averages on
        if (ncentre > 0) {
            const float inv = 1.f / (float)ncentre;
            // byte offset of this lane's column in every listed row (swizzled layout); all loads of a K-block are
            // issued together
            uint32_t off[kMaxCentreRows];
#pragma unroll
            for (int k = 0; k < kMaxCentreRows; ++k) {
                const int r = sm->crow[k < ncentre ? k : 0];
                off[k] = (uint32_t)(r >> 3) * 1024u + (uint32_t)(r & 7) * 128u + (uint32_t)(((lane >> 2) ^ (r & 7)) << 4) +
                         (uint32_t)(lane & 3) * 4u;
            }
            int s = 0;
            uint32_t ph = 0;
            for (int t = 0; t < total; ++t) {
                if (!mbar_wait(&sm->landed[s], ph, abort_flag, status)) break;
                const uint8_t* tile = base + (size_t)s * stage_bytes;
                float v[kMaxCentreRows];
#pragma unroll
                for (int k = 0; k < kMaxCentreRows; ++k) v[k] = *reinterpret_cast<const float*>(tile + off[k]);
                float acc = 0.f;
#pragma unroll
                for (int k = 0; k < kMaxCentreRows; ++k)
                    if (k < ncentre) acc += v[k];
                sm->cring[s][lane] = finite_or_zero(acc) * inv;   // a column whose sum is not finite is left uncentred
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm->c_full[s]);
                if (++s == stages) { s = 0; ph ^= 1u; }
            }
        }
    } else if (warp < kProdWarps + kMmaWarps && lane == 0) {
        // ------------------------------------------------ the MMA threads (lane 0 of the two warps after the
        // transform warps): thread g owns the accumulator half of rows 128 g .. 128 g + 127
        const int g = warp - kProdWarps;
        const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(ncol >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
        const uint32_t dcol = tmem_base + (uint32_t)(g * ncol);
        int s = 0;
        uint32_t ph = 0;
        for (int li = 0; li < my_items; ++li) {
            const int nkb = li == my_items - 1 ? last_nkb : kBlocksPerSlab;
            if (li > 0) mbar_wait(&sm->accum_empty, (uint32_t)((li - 1) & 1), abort_flag, status);
            tc_fence_after();
            bool first = true;   // this thread's first MMA of the slab overwrites its accumulator
            for (int kb = 0; kb < nkb; ++kb) {
                mbar_wait(&sm->full[s], ph, abort_flag, status);
                tc_fence_after();
                const uint32_t hi_addr = smem_u32(base + (size_t)s * stage_bytes);
                const uint64_t hi_desc = smem_desc(hi_addr);
                const uint64_t lo_desc = smem_desc(hi_addr + lo_off);
#pragma unroll
                for (int kk = 0; kk < kKB / 8; ++kk) {       // one MMA covers 8 columns = 32 bytes
                    const uint64_t a = hi_desc + (uint64_t)(kk * 2 + g * (128 * 128 / 16));
                    mma_tf32(dcol, a, hi_desc + (uint64_t)(kk * 2), idesc, first ? 0u : 1u);
                    mma_tf32(dcol, a, lo_desc + (uint64_t)(kk * 2), idesc, 1u);
                    first = false;
                }
                mma_commit(&sm->empty[s]);   // the stage may be refilled once both threads' MMAs have read it
                if (++s == stages) { s = 0; ph ^= 1u; }
            }
            mma_commit(&sm->accum_full);
        }
    }

    __syncwarp();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 0) tmem_dealloc(tmem_base, (uint32_t)tmem_cols);
}

// ------------------------------------------------------------------------------------ m <= 128: staged kernel
//
// A TMA box with the 128-byte swizzle is at most 32 fp32 columns wide, and the copy engine takes about 8 cycles
// per row of a box whatever the row's width: boxes of 128-byte rows top out near 4.5 TB/s over all SMs, boxes of
// 256-byte rows reach the HBM rate.  So for m <= 128 the copies are 64 columns wide and land, unswizzled, in a
// staging ring; the transform warps read a staging stage (two K-blocks), and write both MMA operands of each
// K-block, the raw values (= hi for the MMA) and 2 lo, into a ring of MMA stages in the swizzled K-major layout.
constexpr int kStageCols = 64;                       // columns per staging stage: two K-blocks
constexpr int kKbPerStage = kStageCols / kKB;
constexpr int kMaxStg = 8, kMaxMst = 4;

// Stages per slab: 4096 columns, a multiple of the transform groups and of the MMA-issuing threads.
__host__ __device__ constexpr int staged_slab_stages(int) { return (int)(kSlabCols / kStageCols); }

struct StagedPlan {
    int mrows, box_rows, ncol, tmem_cols;
    int nmma;                    // MMA-issuing threads: four up to 64 rows, else two
    int groups;                  // groups of transform warps, each on a stage of its own
    int nstg, nmst;              // staging stages, MMA stages
    uint32_t stg_bytes;          // box_rows x 256 bytes
    uint32_t tile_bytes;         // one K-block's [hi ; 2lo] tile: 2 ncol rows of 128 bytes
    int nst_total;               // 64-column stages in all
    int nitems, grid;
    size_t smem_bytes;
};

StagedPlan staged_plan(int m, int64_t d) {
    StagedPlan p;
    p.mrows = m <= 64 ? 64 : 128;
    p.box_rows = (m + 7) / 8 * 8;
    p.ncol = (m + 15) / 16 * 16;
    p.nmma = m <= 64 ? 4 : 2;
    p.tmem_cols = 32;
    while (p.tmem_cols < p.nmma * 2 * p.ncol) p.tmem_cols <<= 1;
    p.stg_bytes = (uint32_t)p.box_rows * (uint32_t)kStageCols * 4u;
    p.tile_bytes = 2u * (uint32_t)p.ncol * 128u;
    const size_t mst_bytes = (size_t)kKbPerStage * p.tile_bytes;
    // up to 64 rows there is room for four MMA stages: two groups of transform warps write two of them while the
    // tensor cores read the others; above, two MMA stages and one group
    p.nmst = m <= 64 ? 4 : 2;
    p.groups = m <= 64 ? 2 : 1;
    const size_t left = kSmemBudget - 4096 - p.nmst * mst_bytes;
    p.nstg = (int)(left / p.stg_bytes);
    if (p.nstg > kMaxStg) p.nstg = kMaxStg;
    while (p.nstg > 2 && (size_t)p.nstg * p.stg_bytes > 112 * 1024) --p.nstg;   // ~100 KB in flight saturates HBM
    // With two transform groups a staging slot must always hold stages of the same group (an even slot count), so that
    // each copy-issuing thread follows one group only: a parity wait cannot tell phases two apart.
    if (p.groups == 2) p.nstg &= ~1;
    p.nst_total = (int)ceil_div(d, (int64_t)kStageCols);
    p.grid = p.nst_total < kSMs ? p.nst_total : kSMs;
    const int per_cta = (p.nst_total + p.grid - 1) / p.grid;
    p.nitems = p.grid * (int)ceil_div(ceil_div((int64_t)per_cta, (int64_t)staged_slab_stages(p.nmma)), (int64_t)kItemSlabs);
    p.smem_bytes = (size_t)p.nstg * p.stg_bytes + p.nmst * mst_bytes + 3072 /*barriers, centring ring*/ + 1024 /*alignment slack*/;
    return p;
}

struct StagedSmem {
    uint64_t stg_full[kMaxStg];    // TMA bytes of a staging stage have arrived
    uint64_t stg_empty[kMaxStg];   // the transform warps have read it
    uint64_t mst_full[kMaxMst];    // both operands of both K-blocks are written
    uint64_t mst_empty[kMaxMst];   // the MMAs that read them are done
    uint64_t accum_full;
    uint64_t accum_empty;
    uint64_t c_full[kMaxStg];      // the subtracted vector's piece for this staging stage is written
    uint32_t tmem_base;
    int abort_flag;
    int crow[kMaxCentreRows];
    __align__(16) float cring[kMaxStg][kStageCols];
};
static_assert(sizeof(StagedSmem) <= 3072, "fits the shared memory reserved behind the tiles");

// LX = groups of transform warps; J = 16-byte pieces per transform thread and stage (m * 16 / (512 / LX), rounded up);
// NMMA = MMA-issuing threads, each with an accumulator of its own.  Up to 64 rows an MMA sits on its 59-cycle floor and
// a stage's eight MMAs take less time than one thread's wait / fence / commit around them: four threads keep the
// tensor pipe fed where two left it idle a quarter of the time.  NMMA must be a multiple of LX and divide the number
// of MMA slots, so that a thread always serves the same slots and the same transform group: a parity wait tells two
// consecutive phases of a barrier apart, no more, and a thread that followed one group's stages could otherwise get
// more than a phase ahead of the other group's.
template <int J, int LX, int NMMA>
__global__ void __launch_bounds__(kProdThreads + 32 * (NMMA + staged_tma_warps(LX) + kCentreWarps), 1)
gram_staged_kernel(const __grid_constant__ CUtensorMap xmap, int m, uint32_t stg_bytes, uint32_t tile_bytes, int mrows,
                   int ncol, int tmem_cols, int nstg, int nmst, int nst_total, int nitems, float* __restrict__ partial,
                   float* __restrict__ norms, const int* __restrict__ centre_ptr,
                   const int* __restrict__ redo_ptr, int* __restrict__ status) {
    // second launch of a call: only runs when the first one's centring was withdrawn
    if (redo_ptr != nullptr && *redo_ptr == 0) return;
    // Centring: centre_ptr[0] rows, listed from centre_ptr[2] on, are averaged column by column and the average is
    // subtracted from every row before the products (distances do not change; 0 rows: nothing is subtracted).
    const int ncentre = *centre_ptr;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    uint8_t* stg_base = smem_raw + ((1024u - (raw & 1023u)) & 1023u);       // MMA tiles need 1024-byte alignment
    const uint32_t mst_bytes = (uint32_t)kKbPerStage * tile_bytes;
    uint8_t* mst_base = stg_base + (size_t)nstg * stg_bytes;                // stg_bytes is a multiple of 2048
    StagedSmem* sm = reinterpret_cast<StagedSmem*>(mst_base + (size_t)nmst * mst_bytes);
    volatile int* abort_flag = &sm->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr int kTma = staged_tma_warps(LX);
    constexpr int kThreads = kProdThreads + 32 * (NMMA + kTma + kCentreWarps);
    constexpr int kGroupThreads = kProdThreads / LX, kGroupWarps = kProdWarps / LX;

    if (tid == 0) {
        for (int s = 0; s < nstg; ++s) {
            mbar_init(&sm->stg_full[s], 1);
            mbar_init(&sm->stg_empty[s], kGroupWarps);
            mbar_init(&sm->c_full[s], 1);
        }
        for (int s = 0; s < nmst; ++s) {
            mbar_init(&sm->mst_full[s], kGroupWarps);
            mbar_init(&sm->mst_empty[s], 1);
        }
        mbar_init(&sm->accum_full, NMMA);
        mbar_init(&sm->accum_empty, kProdWarps);
        sm->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < ncentre) sm->crow[tid] = centre_ptr[2 + tid];
    // rows m .. 2 ncol of the MMA tiles are never written: clear the MMA stages once so that they read as zeros
    for (uint32_t off = (uint32_t)tid * 16u; off < mst_bytes * (uint32_t)nmst; off += kThreads * 16u)
        *reinterpret_cast<uint4*>(mst_base + off) = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async_smem();
    if (warp == 0) tmem_alloc(&sm->tmem_base, (uint32_t)tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sm->tmem_base;

    // This CTA owns the 64-column stages b, b + G, b + 2G, ... (b = blockIdx.x, G = gridDim.x), t = 0 .. total-1 in
    // its own count; stage t lands in staging slot t % nstg and is transformed into MMA slot t % nmst; a slab is
    // kStagesPerSlab consecutive ones (the last slab may be shorter) and goes to slot b + G * (slab number).
    constexpr int kStagesPerSlab = staged_slab_stages(NMMA);
    static_assert(kStagesPerSlab % LX == 0 && kStagesPerSlab % NMMA == 0, "slabs start at every role's own offset");
    static_assert(NMMA % LX == 0 && kMaxMst % NMMA == 0, "an MMA-issuing thread serves the same slots and group throughout");
    const int total = (nst_total - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    const int my_items = (total + kStagesPerSlab - 1) / kStagesPerSlab;
    const int last_nst = total - (my_items - 1) * kStagesPerSlab;

    if (warp < kProdWarps) {
        // ------------------------------------------------ transform warps, then epilogue of each slab
        const int group = warp / kGroupWarps, gtid = tid - group * kGroupThreads;
        const int npieces = m * (kStageCols / 4);
        // this thread's pieces are (row, q) = ((gtid >> 4) + (kGroupThreads / 16) j, gtid & 15): 16 bytes at column
        // 4 q of the stage, i.e. piece q & 7 of K-block q >> 3.  kGroupThreads / 16 is a multiple of 8, so the
        // swizzle term of the destination is the same for all j.
        const int row0 = gtid >> 4, q = gtid & 15, cq = q & 7;
        const uint32_t src0 = (uint32_t)row0 * (uint32_t)(kStageCols * 4) + (uint32_t)q * 16u;
        constexpr uint32_t kSrcStep = (uint32_t)(kGroupThreads / 16) * (uint32_t)(kStageCols * 4);
        const uint32_t dst0 = (uint32_t)(q >> 3) * tile_bytes + (uint32_t)(row0 >> 3) * 1024u + (uint32_t)(row0 & 7) * 128u +
                              (uint32_t)((cq ^ (row0 & 7)) << 4);
        constexpr uint32_t kDstStep = (uint32_t)(kGroupThreads / 128) * 1024u;
        const uint32_t lo_off = (uint32_t)ncol * 128u;      // the 2lo rows follow the hi rows inside a tile
        uint64_t sq[J];   // packed pair of partial sums of squares per piece (of the centred values)
#pragma unroll
        for (int j = 0; j < J; ++j) sq[j] = 0ull;

        // slots / phases are carried along instead of divided out every stage (LX <= nstg, nmst)
        int ss = group, ms = group, t = group;
        uint32_t sph = 0, mph = 0;
        for (int li = 0; li < my_items; ++li) {
            const int nst = li == my_items - 1 ? last_nst : kStagesPerSlab;
            const int t_end = li * kStagesPerSlab + nst;
            for (; t < t_end; t += LX) {
                // (the centring warp works ahead of the transform warps, so its barrier has usually completed; waiting
                // for it first lets the load of the subtracted vector travel with the loads of the rows)
                if (ncentre > 0) {
                    const bool c_ok = mbar_try(&sm->c_full[ss], sph), x_ok = mbar_try(&sm->stg_full[ss], sph);
                    if (!(c_ok && x_ok)) {
                        mbar_wait(&sm->c_full[ss], sph, abort_flag, status);
                        mbar_wait(&sm->stg_full[ss], sph, abort_flag, status);
                    }
                } else {
                    mbar_wait(&sm->stg_full[ss], sph, abort_flag, status);
                }
                const uint8_t* src = stg_base + (size_t)ss * stg_bytes + src0;
                ulonglong2 x[J];
#pragma unroll
                for (int j = 0; j < J; ++j)
                    if (gtid + j * kGroupThreads < npieces) x[j] = *reinterpret_cast<const ulonglong2*>(src + j * kSrcStep);
                if (ncentre > 0) {
                    const ulonglong2 ck = *reinterpret_cast<const ulonglong2*>(&sm->cring[ss][q * 4]);
#pragma unroll
                    for (int j = 0; j < J; ++j)
                        if (gtid + j * kGroupThreads < npieces) x[j] = make_ulonglong2(sub2(x[j].x, ck.x), sub2(x[j].y, ck.y));
                }
                mbar_wait(&sm->mst_empty[ms], mph ^ 1u, abort_flag, status);   // the MMAs that read this slot are done
                uint8_t* dst = mst_base + (size_t)ms * mst_bytes + dst0;
#pragma unroll
                for (int j = 0; j < J; ++j) {
                    if (gtid + j * kGroupThreads < npieces) {
                        sq[j] = fma2(x[j].x, x[j].x, fma2(x[j].y, x[j].y, sq[j]));
                        *reinterpret_cast<ulonglong2*>(dst + j * kDstStep) = x[j];
                        *reinterpret_cast<ulonglong2*>(dst + lo_off + j * kDstStep) = make_ulonglong2(lo2_of(x[j].x), lo2_of(x[j].y));
                    }
                }
                fence_proxy_async_smem();   // make the generic-proxy stores visible to the MMA's reads
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(&sm->stg_empty[ss]);   // the staging slot has been read: it may be refilled
                    mbar_arrive(&sm->mst_full[ms]);    // one arrival per transform warp of the group
                }
                ss += LX;
                if (ss >= nstg) { ss -= nstg; sph ^= 1u; }
                ms += LX;
                if (ms >= nmst) { ms -= nmst; mph ^= 1u; }
            }
            // output slot of this slab, and whether the slab opens / closes it
            const int item = (int)blockIdx.x + (li / kItemSlabs) * (int)gridDim.x;
            const bool opens = li % kItemSlabs == 0, closes = li % kItemSlabs == kItemSlabs - 1 || li == my_items - 1;

            // ---- end of a slab: this group's share of the exact squared norms (the 16 lanes that share a row
            // add up; the reduction kernel adds the groups) ...
#pragma unroll
            for (int j = 0; j < J; ++j) {
                float v = __uint_as_float((uint32_t)sq[j]) + __uint_as_float((uint32_t)(sq[j] >> 32));
                v += __shfl_xor_sync(0xffffffffu, v, 1);
                v += __shfl_xor_sync(0xffffffffu, v, 2);
                v += __shfl_xor_sync(0xffffffffu, v, 4);
                v += __shfl_xor_sync(0xffffffffu, v, 8);
                const int row = row0 + (kGroupThreads / 16) * j;
                if (closes) {
                    if (q == 0 && row < m) norms[((int64_t)item * LX + group) * m + row] = v;
                    sq[j] = 0ull;
                }
            }
            // ... and the accumulator drain: warp w reads TMEM lanes 32*(w%4)..+31; the warps that share a
            // lane quarter take 16-column chunks round-robin
            mbar_wait(&sm->accum_full, (uint32_t)(li & 1), abort_flag, status);
            tc_fence_after();
            const int quarter = warp & 3;
            float* out_item = partial + (int64_t)item * m * ncol;
            // M = 128: accumulator row i sits in TMEM lane i; M = 64: in lane 32 (i / 16) + i % 16
            const int row = mrows == 64 ? (lane < 16 ? quarter * 16 + lane : m) : quarter * 32 + lane;
            // the hi.hi and hi.2lo parts of every issuing thread's accumulator (a slab of a single stage leaves the
            // second thread's accumulator untouched: skip it)
            const int nparts = 2 * (nst < NMMA ? nst : NMMA);
            for (int cc = warp >> 2; cc * 16 < ncol; cc += kProdWarps / 4) {   // ncol is a multiple of 16
                float acc[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) acc[j] = 0.f;
                for (int part = 0; part < nparts; ++part) {
                    uint32_t v[16];
                    tmem_load16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(part * ncol + cc * 16), v);
#pragma unroll
                    for (int j = 0; j < 16; ++j) acc[j] += __uint_as_float(v[j]);
                }
                if (row < m) {
                    float* dstp = out_item + (int64_t)row * ncol + cc * 16;
#pragma unroll
                    for (int j = 0; j < 16; j += 4) {
                        const float4 o = make_float4(acc[j], acc[j + 1], acc[j + 2], acc[j + 3]);
                        if (opens) *reinterpret_cast<float4*>(dstp + j) = o;
                        else red_add_f4(dstp + j, o);   // this thread wrote the slot's earlier slabs itself
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm->accum_empty);
        }
        // slots of slabs this CTA does not have (it owns one stage fewer than others) read as zero
        for (int l2 = (my_items + kItemSlabs - 1) / kItemSlabs; l2 * (int)gridDim.x < nitems; ++l2) {
            const int64_t item = (int64_t)blockIdx.x + (int64_t)l2 * gridDim.x;
            for (int e = tid; e < m * ncol; e += kProdThreads) partial[item * m * ncol + e] = 0.f;
            for (int e = tid; e < m * LX; e += kProdThreads) norms[item * LX * m + e] = 0.f;
        }
    } else if (warp == kProdWarps + NMMA + kTma) {
        // ------------------------------------------------ the centring warp: averages the listed rows of every stage as
        // it lands and hands the 64 averages on.  Lanes 0-15 add the first eight listed rows, lanes 16-31 the others,
        // four columns (16 bytes) a lane; the halves meet through shuffles.  A column whose sum is not finite is left
        // uncentred (zero is subtracted there).  The warp shares its scheduler with transform warps that are always
        // ready, so it is kept to a few dozen instructions a stage.
        if (ncentre > 0) {
            const float inv = 1.f / (float)ncentre;
            const int half = lane >> 4;
            constexpr int kPerHalf = kMaxCentreRows / 2;
            uint32_t off[kPerHalf];
#pragma unroll
            for (int k = 0; k < kPerHalf; ++k) {
                const int kk = half * kPerHalf + k;
                off[k] = (uint32_t)sm->crow[kk < ncentre ? kk : 0] * (uint32_t)(kStageCols * 4) + (uint32_t)(lane & 15) * 16u;
            }
            const int mine = ncentre - half * kPerHalf;   // listed rows in this half (may be <= 0)
            int s = 0;
            uint32_t ph = 0;
            for (int t = 0; t < total; ++t) {
                if (!mbar_wait(&sm->stg_full[s], ph, abort_flag, status)) break;
                const uint8_t* stg = stg_base + (size_t)s * stg_bytes;
                float4 v[kPerHalf];
#pragma unroll
                for (int k = 0; k < kPerHalf; ++k) v[k] = *reinterpret_cast<const float4*>(stg + off[k]);
                float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int k = 0; k < kPerHalf; ++k) {
                    if (k < mine) { acc.x += v[k].x; acc.y += v[k].y; acc.z += v[k].z; acc.w += v[k].w; }
                }
                acc.x += __shfl_xor_sync(0xffffffffu, acc.x, 16);
                acc.y += __shfl_xor_sync(0xffffffffu, acc.y, 16);
                acc.z += __shfl_xor_sync(0xffffffffu, acc.z, 16);
                acc.w += __shfl_xor_sync(0xffffffffu, acc.w, 16);
                if (lane < 16)
                    *reinterpret_cast<float4*>(&sm->cring[s][4 * lane]) =
                        make_float4(finite_or_zero(acc.x) * inv, finite_or_zero(acc.y) * inv, finite_or_zero(acc.z) * inv,
                                    finite_or_zero(acc.w) * inv);
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm->c_full[s]);
                if (++s == nstg) { s = 0; ph ^= 1u; }
            }
        }
    } else if (warp >= kProdWarps + NMMA) {
        // ------------------------------------------------ the TMA threads: thread l issues the stages l, l + kTma, ...
        if (lane == 0) {
            const int l = warp - (kProdWarps + NMMA);
            int last = -1;
            int s = l % nstg;
            uint32_t ph = (uint32_t)(l / nstg) & 1u;
            int64_t c0 = ((int64_t)blockIdx.x + (int64_t)l * gridDim.x) * kStageCols;   // first column of the stage
            for (int t = l; t < total; t += kTma) {
                if (!mbar_wait(&sm->stg_empty[s], ph ^ 1u, abort_flag, status)) break;   // the slot has been read
                mbar_expect_tx(&sm->stg_full[s], stg_bytes);
                tma_load_2d(stg_base + (size_t)s * stg_bytes, &xmap, (int)c0, 0, &sm->stg_full[s]);
                last = t;
                s += kTma;
                while (s >= nstg) { s -= nstg; ph ^= 1u; }
                c0 += (int64_t)kTma * gridDim.x * kStageCols;
            }
            if (*abort_flag) {
                // give this thread's copies still in flight a bounded time to land before the CTA goes away
                for (int tt = last; tt >= 0 && tt > last - nstg; tt -= kTma) {
                    const int s2 = (int)((uint32_t)tt % (uint32_t)nstg);
                    const uint32_t ph2 = ((uint32_t)tt / (uint32_t)nstg) & 1u;
                    for (uint32_t spin = 0; spin < (1u << 16) && !mbar_test(&sm->stg_full[s2], ph2); ++spin) __nanosleep(64);
                }
            }
        }
    } else if (lane == 0) {
        // ------------------------------------------------ the MMA threads (lane 0 of the NMMA warps after the
        // transform warps): they take the stages in turn and own one accumulator of 2 ncol columns each
        const int g = warp - kProdWarps;
        const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)((2 * ncol) >> 3) << 17) | ((uint32_t)(mrows >> 4) << 24);
        const uint32_t dcol = tmem_base + (uint32_t)(g * 2 * ncol);
        int s = 0, turn = 0;
        uint32_t ph = 0;
        for (int li = 0; li < my_items; ++li) {
            const int nst = li == my_items - 1 ? last_nst : kStagesPerSlab;
            if (li > 0) mbar_wait(&sm->accum_empty, (uint32_t)((li - 1) & 1), abort_flag, status);
            tc_fence_after();
            bool first = true;   // this thread's first MMA of the slab overwrites its accumulator
            for (int k = 0; k < nst; ++k) {
                const int my_s = s;
                const uint32_t my_ph = ph;
                const bool skip = turn != g;
                if (++s == nmst) { s = 0; ph ^= 1u; }
                if (++turn == NMMA) turn = 0;
                if (skip) continue;
                mbar_wait(&sm->mst_full[my_s], my_ph, abort_flag, status);
                tc_fence_after();
                const uint32_t addr = smem_u32(mst_base + (size_t)my_s * mst_bytes);
#pragma unroll
                for (int kb = 0; kb < kKbPerStage; ++kb) {
                    const uint64_t desc = smem_desc(addr + (uint32_t)kb * tile_bytes);
#pragma unroll
                    for (int kk = 0; kk < kKB / 8; ++kk) {       // one MMA covers 8 columns = 32 bytes
                        const uint64_t ab = desc + (uint64_t)(kk * 2);
                        mma_tf32(dcol, ab, ab, idesc, first ? 0u : 1u);   // A = hi rows, B = [hi ; 2lo]
                        first = false;
                    }
                }
                mma_commit(&sm->mst_empty[my_s]);   // the slot may be rewritten once these MMAs have read it
            }
            mma_commit(&sm->accum_full);
        }
    }

    __syncwarp();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (warp == 0) tmem_dealloc(tmem_base, (uint32_t)tmem_cols);
}

// For one chunk of slab slots: dpart[chunk][i*m+j] (i < j) = sum over the slots s of the squared distance that slot
// contributes,
//     r_i T_ii + r_j T_jj - (r_i + r_j) sym(T)_ij,     sym(T)_ij = (T_ij + T_ji) / 2,
// with r_i(s) = exact norm / tensor-core norm of row i in slot s (the exact norm comes in `ngroups` shares, added
// here in a fixed order): the slot's exact norms n_i = r_i T_ii and n_j, minus twice the rescaled inner product.
// Every product and sum is rounded on its own (no fused multiply-add), so that two bitwise-equal rows, for which
// T_ii = T_jj = T_ij = T_ji and r_i = r_j, get exactly zero from every slot.
// One CTA per pair of 32-row blocks (bi <= bj) and chunk: per slot it reads the tile T[bi][bj] and the
// mirrored tile T[bj][bi] row by row (coalesced) and transposes the second through shared memory.
constexpr int kRT = 32;
__global__ void __launch_bounds__(kRT * 8)
tc_reduce_kernel(const float* __restrict__ partial, const float* __restrict__ norms, int ngroups, int nitems,
                 int ngroups_redo, int nitems_redo, const int* __restrict__ expo, const int* __restrict__ redo, int m,
                 int ncol, double* __restrict__ dpart) {
    __shared__ float mirror[kRT][kRT + 1];
    __shared__ double ratio_i[kRT], ratio_j[kRT], diag_i[kRT], diag_j[kRT];
    __shared__ int expo_i[kRT], expo_j[kRT];
    // The slots hold the split-fp16 pass's sums (rows scaled by 2^expo) unless that pass was repeated by the
    // split-TF32 kernels (*redo != 0), whose rows are unscaled and whose slot count may differ.
    const bool scaled = expo != nullptr && *redo == 0;
    if (expo != nullptr && !scaled) { ngroups = ngroups_redo; nitems = nitems_redo; }
    const int nt = (m + kRT - 1) / kRT;
    int bi = 0, rem = blockIdx.x;
    while (rem >= nt - bi) { rem -= nt - bi; ++bi; }
    const int bj = bi + rem;
    const int chunk = blockIdx.y;
    const int per = (nitems + (int)gridDim.y - 1) / (int)gridDim.y;
    const int s0 = chunk * per, s1 = (s0 + per) < nitems ? (s0 + per) : nitems;
    const int64_t elems = (int64_t)m * ncol;
    const int tx = threadIdx.x & (kRT - 1), ty = threadIdx.x / kRT;   // ty = 0..7

    double acc[kRT / 8];
#pragma unroll
    for (int k = 0; k < kRT / 8; ++k) acc[k] = 0.0;
    const int j = bj * kRT + tx;             // this thread's column of the tile
    if (ty < 2) {
        const int r = (ty == 0 ? bi : bj) * kRT + tx;
        (ty == 0 ? expo_i : expo_j)[tx] = (scaled && r < m) ? expo[r] : 0;
    }

    for (int s = s0; s < s1; ++s) {
        const float* T = partial + (int64_t)s * elems;
        const float* nrm = norms + (int64_t)s * ngroups * m;   // one share per group of transform warps
        if (ty < 2) {
            const int r = (ty == 0 ? bi : bj) * kRT + tx;
            double ratio = 1.0, t = 0.0;
            if (r < m) {
                t = (double)T[(int64_t)r * ncol + r];
                double nv = 0.0;
                for (int g = 0; g < ngroups; ++g) nv += (double)nrm[g * m + r];
                if (t > 0.0) ratio = nv / t;
                else t = nv;   // an all-zero row (or a non-finite one): its norm as it is
            }
            (ty == 0 ? ratio_i : ratio_j)[tx] = ratio;
            (ty == 0 ? diag_i : diag_j)[tx] = t;
        }
        float a[kRT / 8];
#pragma unroll
        for (int k = 0; k < kRT / 8; ++k) {
            const int rl = ty + 8 * k;
            const int ri = bi * kRT + rl, rj = bj * kRT + rl;
            a[k] = (ri < m && j < m) ? T[(int64_t)ri * ncol + j] : 0.f;                                  // T[bi][bj]
            mirror[rl][tx] = (rj < m && bi * kRT + tx < m) ? T[(int64_t)rj * ncol + bi * kRT + tx] : 0.f;   // T[bj][bi]
        }
        __syncthreads();
#pragma unroll
        for (int k = 0; k < kRT / 8; ++k) {
            const int il = ty + 8 * k;
            const double tij = 0.5 * ((double)a[k] + (double)mirror[tx][il]);
            const double ri = ratio_i[il], rj = ratio_j[tx];
            // (the rows' power-of-two scales come off exactly; for equal rows they are equal)
            const int ei = expo_i[il], ej = expo_j[tx];
            const double norms_ij = __dadd_rn(scalbn(__dmul_rn(ri, diag_i[il]), -2 * ei), scalbn(__dmul_rn(rj, diag_j[tx]), -2 * ej));
            acc[k] += __dadd_rn(norms_ij, -scalbn(__dmul_rn(__dadd_rn(ri, rj), tij), -ei - ej));
        }
        __syncthreads();
    }
    const int64_t total = (int64_t)m * m;
#pragma unroll
    for (int k = 0; k < kRT / 8; ++k) {
        const int i = bi * kRT + ty + 8 * k;
        if (i < m && j < m && i < j) dpart[(int64_t)chunk * total + (int64_t)i * m + j] = acc[k];
    }
}

// D_ij = sum of the chunks' contributions (never negative, zero diagonal); a NaN (rows with non-finite entries)
// reads as +Inf, "as far as it gets", never as zero; status != 0 -> NaN.
// One warp per pair i < j: the lanes add the chunks round-robin, then a fixed butterfly.
__global__ void tc_dist_kernel(const double* __restrict__ dpart, int nchunks, int m, const int* __restrict__ status,
                               double* __restrict__ D) {
    const bool bad = *status != 0;
    const int64_t total = (int64_t)m * m;
    const int lane = threadIdx.x & 31;
    const int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    if (warp >= total) return;
    const int i = (int)(warp / m), j = (int)(warp - (int64_t)i * m);
    if (i > j) return;
    if (i == j) {
        if (lane == 0) D[warp] = bad ? __longlong_as_double(0x7ff8000000000000LL) : 0.0;
        return;
    }
    double v = 0.0;
    for (int c = lane; c < nchunks; c += 32) v += dpart[(int64_t)c * total + (int64_t)i * m + j];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    if (lane == 0) {
        v = v > 0.0 ? v : (v != v ? __longlong_as_double(0x7ff0000000000000LL) : 0.0);
        if (bad) v = __longlong_as_double(0x7ff8000000000000LL);
        D[(int64_t)i * m + j] = v;
        D[(int64_t)j * m + i] = v;
    }
}

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The driver's tensor-map encoder, looked up through the runtime (no link against libcuda).
EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

}  // namespace

// X as a 2-D fp32 tensor (d columns innermost, m rows, row pitch ld), zero fill outside the matrix.
detox_status make_xmap(void* map, const float* X, int64_t ld, int m, int64_t d, int box_cols, int box_rows, bool swizzle128) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return DETOX_ERR_CUDA;
    const cuuint64_t gdim[2] = {(cuuint64_t)d, (cuuint64_t)m};
    const cuuint64_t gstride[1] = {(cuuint64_t)ld * sizeof(float)};
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    const cuuint32_t estride[2] = {1, 1};
    CUresult r = enc(static_cast<CUtensorMap*>(map), CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(X), gdim, gstride,
                     box, estride, CU_TENSOR_MAP_INTERLEAVE_NONE,
                     swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? DETOX_OK : DETOX_ERR_CUDA;
}

namespace {

template <int J>
detox_status launch_wide(const WidePlan& p, const CUtensorMap& xmap, int m, const TcBuffers& b, cudaStream_t s) {
    if (cudaFuncSetAttribute(gram_wide_kernel<J>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem_bytes) !=
        cudaSuccess)
        return DETOX_ERR_CUDA;
    gram_wide_kernel<J><<<p.grid, kTcThreads, p.smem_bytes, s>>>(xmap, m, p.lo_off, p.stage_bytes, p.box_rows, p.ncol,
                                                                 p.tmem_cols, p.stages, p.nkb_total, p.nitems, b.partial,
                                                                 b.norms, b.centre, b.redo, b.status);
    return launch_status();
}

template <int J, int LX, int NMMA>
detox_status launch_staged(const StagedPlan& p, const CUtensorMap& xmap, int m, const TcBuffers& b, cudaStream_t s) {
    if (cudaFuncSetAttribute(gram_staged_kernel<J, LX, NMMA>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)p.smem_bytes) != cudaSuccess)
        return DETOX_ERR_CUDA;
    constexpr int kThreads = kProdThreads + 32 * (NMMA + staged_tma_warps(LX) + kCentreWarps);
    gram_staged_kernel<J, LX, NMMA><<<p.grid, kThreads, p.smem_bytes, s>>>(xmap, m, p.stg_bytes, p.tile_bytes, p.mrows, p.ncol,
                                                                          p.tmem_cols, p.nstg, p.nmst, p.nst_total,
                                                                          p.nitems, b.partial, b.norms, b.centre, b.redo,
                                                                          b.status);
    return launch_status();
}

// What the kernels' outputs look like to the reduction: slab slots, shares of the norms per slot, row pitch -- of
// the split-TF32 kernel that fits m, and of the split-fp16 kernel.
struct TcShape {
    bool staged;
    int nitems, groups, ncol;
    int nitems_f16, groups_f16;
    int max_items() const { return nitems > nitems_f16 ? nitems : nitems_f16; }
    int max_shares() const {
        const int a = nitems * groups, b = nitems_f16 * groups_f16;
        return a > b ? a : b;
    }
};
TcShape tc_shape(int m, int64_t d) {
    TcShape o;
    o.staged = m <= 128;
    if (o.staged) {
        const StagedPlan p = staged_plan(m, d);
        o.nitems = p.nitems, o.groups = p.groups, o.ncol = p.ncol;
    } else {
        const WidePlan p = wide_plan(m, d);
        o.nitems = p.nitems, o.groups = 1, o.ncol = p.ncol;
    }
    o.nitems_f16 = f16_nitems(m, d);
    o.groups_f16 = f16_groups(m);
    return o;
}

std::atomic<int> g_split_mode{DETOX_SPLIT_AUTO};

}  // namespace

bool tc_supported(const float* X, int64_t ld, int m, int64_t d) {
    // TMA needs a 16-byte aligned base and row pitch; coordinates are 32-bit
    return m > 16 && m <= 256 && aligned16(X) && ld % 4 == 0 && d < (int64_t)1 << 31 && encode_tiled_fn() != nullptr;
}

int tc_split_mode(int mode) {
    if (mode != DETOX_SPLIT_AUTO && mode != DETOX_SPLIT_TF32) return g_split_mode.load();
    return g_split_mode.exchange(mode);
}

// workspace: slab partials | norms | per-chunk distance sums | centring rows, redo flag | row scales |
// scratch of the centre choice
struct TcWs {
    float* partial;
    float* norms;
    double* dpart;
    int* centre;     // [0] how many rows are averaged into the subtracted vector (0: none), [1] the redo flag, [2..] the rows
    int* expo;       // [m] power-of-two scale of every row for the split-fp16 pass
    void* pick;
    size_t total;
};
TcWs tc_carve(void* ws, int m, int64_t d, const TcShape& o) {
    TcWs w;
    char* p = static_cast<char*>(ws);
    size_t off = 0;
    const size_t elems = (size_t)m * o.ncol;
    w.partial = reinterpret_cast<float*>(p + off);
    off += align_up((size_t)o.max_items() * elems * sizeof(float));
    w.norms = reinterpret_cast<float*>(p + off);
    off += align_up((size_t)o.max_shares() * m * sizeof(float));
    w.dpart = reinterpret_cast<double*>(p + off);
    off += align_up((size_t)reduce_chunks(m, o.max_items()) * m * m * sizeof(double));
    w.centre = reinterpret_cast<int*>(p + off);
    off += 256;
    w.expo = reinterpret_cast<int*>(p + off);
    off += align_up((size_t)m * sizeof(int));
    w.pick = p + off;
    off += centre_ws_bytes(m, d);
    w.total = off;
    return w;
}

size_t tc_ws_bytes(int m, int64_t d) { return tc_carve(nullptr, m, d, tc_shape(m, d)).total; }

namespace {

// One launch of the streaming kernel that fits m.
detox_status launch_tc_gram(const float* X, int64_t ld, int m, int64_t d, const TcShape& o, const TcBuffers& b,
                            cudaStream_t s) {
    CUtensorMap xmap;
    detox_status st;
    if (o.staged) {
        const StagedPlan p = staged_plan(m, d);
        if ((st = make_xmap(&xmap, X, ld, m, d, kStageCols, p.box_rows, false)) != DETOX_OK) return st;
        // 16-byte pieces per transform thread and stage: m * 16 / (threads of a group), rounded up
        const int gt = kProdThreads / p.groups;
        const int per_thread = (m * (kStageCols / 4) + gt - 1) / gt;
        if (p.groups == 2) {   // up to 64 rows: two transform groups, four MMA-issuing threads
            if (per_thread <= 2) return launch_staged<2, 2, 4>(p, xmap, m, b, s);
            if (per_thread <= 3) return launch_staged<3, 2, 4>(p, xmap, m, b, s);
            return launch_staged<4, 2, 4>(p, xmap, m, b, s);
        }
        if (per_thread <= 2) return launch_staged<2, 1, 2>(p, xmap, m, b, s);
        if (per_thread <= 3) return launch_staged<3, 1, 2>(p, xmap, m, b, s);
        return launch_staged<4, 1, 2>(p, xmap, m, b, s);
    }
    const WidePlan p = wide_plan(m, d);
    if ((st = make_xmap(&xmap, X, ld, m, d, kKB, p.box_rows, true)) != DETOX_OK) return st;
    // 16-byte pieces per transform thread and K-block: m * 8 / 512, rounded up
    if (m * 8 <= 3 * kProdThreads) return launch_wide<3>(p, xmap, m, b, s);
    return launch_wide<4>(p, xmap, m, b, s);
}

}  // namespace

// Sequence: choose the centring rows and the rows' scales on a column sample -> the split-fp16 pass -> check that the
// centred rows really got smaller and that no entry left the fp16 range -> the split-TF32 pass, which returns at once
// unless the check asked for it -> reduction of the slab partials to distances.  (DETOX_SPLIT_TF32: the split-TF32
// pass runs first and the check only looks at the centring, as it did before there was an fp16 pass.)
detox_status launch_sqdist_tc(const float* X, int64_t ld, int m, int64_t d, double* D, void* ws, int* status,
                              cudaStream_t s) {
    const TcShape o = tc_shape(m, d);
    const TcWs w = tc_carve(ws, m, d, o);
    const bool fast = g_split_mode.load() == DETOX_SPLIT_AUTO;
    detox_status st;
    if ((st = launch_pick_centre(X, ld, m, d, w.pick, w.centre, w.expo, s)) != DETOX_OK) return st;
    TcBuffers b{w.partial, w.norms, w.centre, nullptr, status};
    if (fast) {
        if ((st = launch_gram_f16(X, ld, m, d, b, w.expo, s)) != DETOX_OK) return st;
        st = launch_check_centre(w.norms, w.partial, o.nitems_f16, o.groups_f16, m, o.ncol, w.pick, d, w.centre, w.centre + 1,
                                 w.expo, s);
    } else {
        if ((st = launch_tc_gram(X, ld, m, d, o, b, s)) != DETOX_OK) return st;
        st = launch_check_centre(w.norms, w.partial, o.nitems, o.groups, m, o.ncol, w.pick, d, w.centre, w.centre + 1, nullptr, s);
    }
    if (st != DETOX_OK) return st;
    b.redo = w.centre + 1;
    if ((st = launch_tc_gram(X, ld, m, d, o, b, s)) != DETOX_OK) return st;
    const int nt = (m + kRT - 1) / kRT;
    const int nchunks = reduce_chunks(m, o.max_items());
    tc_reduce_kernel<<<dim3((unsigned)(nt * (nt + 1) / 2), (unsigned)nchunks), kRT * 8, 0, s>>>(
        w.partial, w.norms, fast ? o.groups_f16 : o.groups, fast ? o.nitems_f16 : o.nitems, o.groups, o.nitems,
        fast ? w.expo : nullptr, w.centre + 1, m, o.ncol, w.dpart);
    if ((st = launch_status()) != DETOX_OK) return st;
    tc_dist_kernel<<<(unsigned)ceil_div((int64_t)m * m * 32, 256), 256, 0, s>>>(w.dpart, nchunks, m, status, D);
    return launch_status();
}

bool sqdist_vote_tc_supported(const float* X, int64_t ld, int n, int r, int64_t d) {
    return f16_vote_supported(n, r) && tc_supported(X, ld, n / 3, d) && g_split_mode.load() == DETOX_SPLIT_AUTO;
}

// Sequence: sample (votes formed on the fly) and pick -> the split-fp16 pass that votes while it reads -> check ->
// winners from the vote's bits (a group without a majority also raises the redo flag) -> only if the flag is up: the
// votes are stored and the split-TF32 pass runs on them -> reduction to distances.
detox_status launch_sqdist_vote_tc(const float* X, int64_t ld, int n, int64_t d, const IdTable& members, int32_t* winner,
                                   void* vote_ws, float* Z, int64_t ldz, double* D, void* ws, int* status, cudaStream_t s) {
    const int m = n / 3;
    const TcShape o = tc_shape(m, d);
    const TcWs w = tc_carve(ws, m, d, o);
    VoteMembers vm;
    for (int i = 0; i < 256; ++i) vm.id[i] = i < n ? (uint8_t)members.id[i] : 0;
    detox_status st;
    if ((st = launch_pick_centre(X, ld, m, d, w.pick, w.centre, w.expo, s, &vm)) != DETOX_OK) return st;
    TcBuffers b{w.partial, w.norms, w.centre, nullptr, status};
    if ((st = launch_gram_f16_vote(X, ld, n, d, members, static_cast<uint32_t*>(vote_ws), b, w.expo, s)) != DETOX_OK) return st;
    st = launch_check_centre(w.norms, w.partial, o.nitems_f16, o.groups_f16, m, o.ncol, w.pick, d, w.centre, w.centre + 1,
                             w.expo, s);
    if (st != DETOX_OK) return st;
    if ((st = launch_vote_finalize(n, 3, members, vote_ws, winner, w.centre + 1, s)) != DETOX_OK) return st;
    if ((st = launch_vote_store_gated(X, ld, n, d, members, Z, ldz, winner, w.centre + 1, s)) != DETOX_OK) return st;
    b.redo = w.centre + 1;
    if ((st = launch_tc_gram(Z, ldz, m, d, o, b, s)) != DETOX_OK) return st;
    const int nt = (m + kRT - 1) / kRT;
    const int nchunks = reduce_chunks(m, o.max_items());
    tc_reduce_kernel<<<dim3((unsigned)(nt * (nt + 1) / 2), (unsigned)nchunks), kRT * 8, 0, s>>>(
        w.partial, w.norms, o.groups_f16, o.nitems_f16, o.groups, o.nitems, w.expo, w.centre + 1, m, o.ncol, w.dpart);
    if ((st = launch_status()) != DETOX_OK) return st;
    tc_dist_kernel<<<(unsigned)ceil_div((int64_t)m * m * 32, 256), 256, 0, s>>>(w.dpart, nchunks, m, status, D);
    return launch_status();
}

}  // namespace detox
