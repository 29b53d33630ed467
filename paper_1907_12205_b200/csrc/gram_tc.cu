// Pairwise squared distances for 16 < m <= 256 on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// G = X X^T is computed with error-compensated TF32: every fp32 x is split into hi = tf32(x) and
// lo = x - hi (exact), and  x_i . x_j  ~=  hi_i.hi_j + hi_i.lo_j + lo_i.hi_j.  The last two terms are
// folded by symmetry: with T = hi (hi + 2 lo)^T, accumulated as two MMAs per K-step into ONE fp32
// accumulator in tensor memory, G_ij = (T_ij + T_ji) / 2.  Both MMA operands come from the same
// shared-memory tiles (rows of X), so every row of X is read from HBM exactly once.
//
// One persistent CTA per SM.  One thread streams K-blocks of 32 columns (all m rows) into shared
// memory with TMA (128-byte swizzle, which is the K-major layout the MMA expects; rows and columns
// outside the matrix arrive as zeros).  The raw fp32 tile itself serves as the `hi` operand: a TF32
// MMA reads only the upper 19 bits of each word.  Warps 0-15 read the tile back, form
// 2 lo = 2 (x - (x with its low 13 bits cleared)) and write the second tile; lane 0 of warps 16, 17
// issue the MMAs; mbarriers form a ring of stages between the three roles.
// K-blocks are dealt round-robin to the CTAs and every 128 of a CTA's K-blocks form a slab; at the end
// of a slab the accumulator is drained to a per-slab fp32 partial in global memory and the slabs are
// added in fp64 in a fixed order afterwards, so the long sum never lives in one fp32 accumulator and
// the result is deterministic.
//
// The tensor cores add into their fp32 accumulator by truncation, so a long same-sign sum (a row with
// itself, or with a copy of itself) comes out low by a few 1e-5 relative per slab.  The producers
// therefore also accumulate each row's exact squared norm per slab on the CUDA cores; the final
// reduction rescales every slab's T_ij by the mean of (exact norm / tensor-core norm) of rows i and
// j.  The diagonal becomes exact, a pair of identical rows keeps distance zero, and entries
// between unrelated rows (which hover around zero and lose nothing to truncation) are unchanged.
//
// Every wait on an mbarrier is bounded; if one runs out the kernel records DETOX_ERR_TIMEOUT in the
// status word, stops waiting everywhere, frees its tensor memory and returns.
#include <cuda.h>

#include "common.cuh"

namespace detox {

namespace {

constexpr int kKB = 32;                      // fp32 columns per K-block: one 128-byte swizzle row
constexpr int kProdWarps = 16;
constexpr int kProdThreads = kProdWarps * 32;
constexpr int kMmaWarps = 2;                   // two issuing threads, so one's bookkeeping overlaps the other's MMAs
constexpr int kTcThreads = kProdThreads + 32 * (kMmaWarps + 1);  // + the MMA warps + the TMA warp
constexpr int kMaxStages = 12;
constexpr long long kWaitLimitCycles = 2000000000LL;  // ~1 s at the SM clock
constexpr int64_t kSlabCols = 4096;          // columns (128 K-blocks) accumulated in tensor memory before a drain
constexpr int kMinReduceChunks = 32, kMaxReduceChunks = 256;

struct TcPlan {
    int rows_pad;    // rows of each shared-memory tile (64, 128 or 256); a stage holds two tiles
    int mrows;       // M of the MMA: 64 for m <= 64, else 128
    int box_rows;    // rows the TMA box brings in: m rounded up to 8
    int nhalf;       // accumulator halves of 128 rows
    int ncol;        // N of the MMA: m rounded up to 16
    int chains;      // m <= 128: accumulators, one per MMA-issuing thread
    int tmem_cols;   // power of two >= the accumulator columns, >= 32
    int stages;
    int nkb_total;   // K-blocks in all: d / 32 rounded up
    int nitems;      // slab slots: grid x the largest number of slabs a CTA has
    int grid;
    size_t smem_bytes;
};

TcPlan tc_plan(int m, int64_t d) {
    TcPlan p;
    p.nhalf = m > 128 ? 2 : 1;
    p.mrows = m <= 64 ? 64 : 128;
    p.rows_pad = m <= 64 ? 64 : 128 * p.nhalf;
    p.box_rows = (m + 7) / 8 * 8;
    p.ncol = (m + 15) / 16 * 16;
    // m <= 128: one MMA per K-step with B = [hi ; 2lo] stacked (N = 2 ncol); the two issuing threads take
    //           alternate K-blocks and own one accumulator each;
    // m  > 128: two 128-row halves, one per issuing thread, B = hi and B = 2lo as separate MMAs
    p.chains = p.nhalf == 1 ? kMmaWarps : 1;
    int need = p.nhalf == 1 ? p.chains * 2 * p.ncol : 2 * p.ncol;
    p.tmem_cols = 32;
    while (p.tmem_cols < need) p.tmem_cols <<= 1;
    size_t stage = (size_t)2 * p.rows_pad * 128;
    p.stages = (int)((192 * 1024) / stage);
    if (p.stages > kMaxStages) p.stages = kMaxStages;
    // K-blocks are dealt round-robin to the CTAs, so that every CTA has the same number of them (to within one)
    // whatever d is, and neighbouring CTAs read neighbouring 128-byte pieces of a row
    p.nkb_total = (int)ceil_div(d, (int64_t)kKB);
    p.grid = p.nkb_total < kSMs ? p.nkb_total : kSMs;
    const int per_cta = (p.nkb_total + p.grid - 1) / p.grid;
    p.nitems = p.grid * (int)ceil_div((int64_t)per_cta, kSlabCols / kKB);
    p.smem_bytes = stage * p.stages + 1024 /*barriers*/ + 1024 /*alignment slack*/;
    return p;
}

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

// ------------------------------------------------------------------------------------ PTX wrappers

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Hardware-assisted wait: the thread is suspended until the phase completes or a short
// implementation-defined time passes, whichever is first.
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait (about a second of SM clocks).  Returns false, and raises the CTA-wide abort flag,
// when the limit is hit; returns false at once when another thread has already given up.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort_flag, int* status) {
    if (mbar_try(bar, parity)) return true;
    const long long start = clock64();
    for (;;) {
        if (mbar_try(bar, parity)) return true;
        if (*abort_flag) return false;
        if (clock64() - start > kWaitLimitCycles) break;
    }
    *abort_flag = 1;
    atomicExch(status, (int)DETOX_ERR_TIMEOUT);
    return false;
}

__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_alloc(uint32_t* slot, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}

// Shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows packed 128 bytes apart,
// 8-row groups 1024 bytes apart.  `addr` must lie in a 1024-byte aligned tile.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
    uint64_t desc = (uint64_t)((addr & 0x3FFFFu) >> 4);   // start address, 16-byte units
    desc |= (uint64_t)1 << 16;                              // leading byte offset (unused for swizzled K-major)
    desc |= (uint64_t)(1024 >> 4) << 32;                    // stride byte offset: next 8-row group
    desc |= (uint64_t)1 << 46;                              // descriptor version of this architecture
    desc |= (uint64_t)2 << 61;                              // 128-byte swizzle
    return desc;
}

// D[tmem] (+)= A[smem] * B[smem]^T, TF32 inputs, fp32 accumulate; M and N come with the instruction descriptor.
__device__ __forceinline__ void mma_tf32(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// Arrive on `bar` once every MMA issued so far by this thread has finished.
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}

__device__ __forceinline__ void tmem_load32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
          "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
          "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
          "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// 2-D tiled TMA load (no multicast): box at (x = column, y = row) -> shared memory, completion on `bar`.
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(smem_u32(dst)), "l"(reinterpret_cast<uint64_t>(map)), "r"(x), "r"(y), "r"(smem_u32(bar))
        : "memory");
}

// Packed pairs of fp32 (one instruction for two lanes).
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
// What a TF32 MMA sees of x is hi = x with the low 13 mantissa bits cleared; x - hi is exact in fp32
// and so is its double.  (The MMA again reads only the upper 19 bits of 2 lo.)
__device__ __forceinline__ uint64_t lo2_of(uint64_t x2) {
    const uint64_t t = sub2(x2, x2 & 0xFFFFE000FFFFE000ull);
    return add2(t, t);
}

struct TcSmem {
    uint64_t landed[kMaxStages];   // TMA bytes of the raw tile have arrived
    uint64_t full[kMaxStages];     // the 2lo tile is written: both tiles ready for the MMA
    uint64_t empty[kMaxStages];
    uint64_t accum_full;
    uint64_t accum_empty;
    uint32_t tmem_base;
    int abort_flag;
};

// J = 16-byte chunks per transform thread and K-block (m * 8 / 512 rounded up to a power of two)
template <int J>
__global__ void __launch_bounds__(kTcThreads, 1)
gram_tc_kernel(const __grid_constant__ CUtensorMap xmap, int m, int64_t d, int rows_pad, int mrows, int box_rows, int nhalf,
               int ncol, int chains, int tmem_cols, int stages, int nkb_total, int nitems, float* __restrict__ partial,
               float* __restrict__ norms, int* __restrict__ status) {
    extern __shared__ uint8_t smem_raw[];
    // tiles need 1024-byte alignment for the 128-byte swizzle pattern
    const uint32_t raw = smem_u32(smem_raw);
    uint8_t* base = smem_raw + ((1024u - (raw & 1023u)) & 1023u);
    const uint32_t tile_bytes = (uint32_t)rows_pad * 128u;
    const uint32_t stage_bytes = 2u * tile_bytes;
    TcSmem* sm = reinterpret_cast<TcSmem*>(base + (size_t)stage_bytes * stages);
    volatile int* abort_flag = &sm->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

    if (tid == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(&sm->landed[s], 1);
            mbar_init(&sm->full[s], kProdWarps);
            mbar_init(&sm->empty[s], nhalf == 1 ? 1 : kMmaWarps);
        }
        mbar_init(&sm->accum_full, kMmaWarps);
        mbar_init(&sm->accum_empty, kProdWarps);
        sm->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
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
    // count; a slab is kBlocksPerSlab consecutive ones of them (the last slab may be shorter) and goes to slot
    // b + G * (slab number).
    constexpr int kBlocksPerSlab = (int)(kSlabCols / kKB);
    const int total = (nkb_total - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    const int my_items = (total + kBlocksPerSlab - 1) / kBlocksPerSlab;
    const int last_nkb = total - (my_items - 1) * kBlocksPerSlab;

    if (warp < kProdWarps) {
        // ------------------------------------------------ transform warps, then epilogue of each slab
        const int nchunks = m * 8;
        // this thread's chunks are (row, c) = ((tid >> 3) + 64 j, tid & 7) in every K-block
        uint32_t off[J];
#pragma unroll
        for (int j = 0; j < J; ++j) {
            const int row = (tid >> 3) + (kProdThreads / 8) * j, c = tid & 7;
            off[j] = (uint32_t)(row >> 3) * 1024u + (uint32_t)(row & 7) * 128u + (uint32_t)((c ^ (row & 7)) << 4);
        }
        uint64_t sq[J];   // packed pair of partial sums of squares per chunk
#pragma unroll
        for (int j = 0; j < J; ++j) sq[j] = 0ull;

        // m <= 128: the 2lo rows follow the hi rows at row `ncol` of the same tile (ncol % 8 == 0);
        // m  > 128: they form a tile of their own
        const uint32_t lo_off = nhalf == 1 ? (uint32_t)ncol * 128u : tile_bytes;
        // stage / phase / slab position are carried along instead of divided out every K-block
        int s = 0, li = 0, kb = 0;
        uint32_t ph = 0;
        for (int t = 0; t < total; ++t) {
            mbar_wait(&sm->landed[s], ph, abort_flag, status);
            const uint8_t* hi_tile = base + (size_t)s * stage_bytes;
            uint8_t* lo_tile = base + (size_t)s * stage_bytes + lo_off;
#pragma unroll
            for (int j = 0; j < J; ++j) {
                if (tid + j * kProdThreads < nchunks) {
                    const ulonglong2 x = *reinterpret_cast<const ulonglong2*>(hi_tile + off[j]);
                    sq[j] = fma2(x.x, x.x, fma2(x.y, x.y, sq[j]));
                    *reinterpret_cast<ulonglong2*>(lo_tile + off[j]) = make_ulonglong2(lo2_of(x.x), lo2_of(x.y));
                }
            }
            fence_proxy_async_smem();   // make the generic-proxy stores visible to the MMA's reads
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm->full[s]);   // one arrival per transform warp
            if (++s == stages) { s = 0; ph ^= 1u; }

            const int nkb = li == my_items - 1 ? last_nkb : kBlocksPerSlab;
            if (++kb != nkb) continue;
            const int item = (int)blockIdx.x + li * (int)gridDim.x;

            // ---- end of a slab: exact squared norms (the 8 lanes that share a row add up) ...
#pragma unroll
            for (int j = 0; j < J; ++j) {
                float v = __uint_as_float((uint32_t)sq[j]) + __uint_as_float((uint32_t)(sq[j] >> 32));
                v += __shfl_xor_sync(0xffffffffu, v, 1);
                v += __shfl_xor_sync(0xffffffffu, v, 2);
                v += __shfl_xor_sync(0xffffffffu, v, 4);
                const int row = (tid >> 3) + (kProdThreads / 8) * j;
                if ((tid & 7) == 0 && row < m) norms[(int64_t)item * m + row] = v;
                sq[j] = 0ull;
            }
            // ... and the accumulator drain: warp w reads TMEM lanes 32*(w%4)..+31; the warps that share a
            // lane quarter take 32-column chunks round-robin
            mbar_wait(&sm->accum_full, (uint32_t)(li & 1), abort_flag, status);
            tc_fence_after();
            const int quarter = warp & 3;
            float* out_item = partial + (int64_t)item * m * ncol;
            for (int h = 0; h < nhalf; ++h) {
                // M = 128: accumulator row i sits in TMEM lane i; M = 64: in lane 32 (i / 16) + i % 16
                const int row = mrows == 64 ? (lane < 16 ? quarter * 16 + lane : m) : h * 128 + quarter * 32 + lane;
                for (int cc = warp >> 2; cc * 32 < ncol; cc += kProdWarps / 4) {
                    float acc[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) acc[j] = 0.f;
                    // m <= 128: add the hi.hi and hi.2lo parts of every chain; m > 128: one accumulator per half
                    // (a slab of a single K-block leaves the second issuing thread's accumulator untouched: skip it)
                    const int nparts = nhalf == 1 ? 2 * (nkb < chains ? nkb : chains) : 1;
                    for (int part = 0; part < nparts; ++part) {
                        uint32_t v[32];
                        const int col = (nhalf == 1 ? part * ncol : h * ncol) + cc * 32;
                        tmem_load32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)col, v);
#pragma unroll
                        for (int j = 0; j < 32; ++j) acc[j] += __uint_as_float(v[j]);
                    }
                    if (row < m) {
                        float* dst = out_item + (int64_t)row * ncol + cc * 32;
                        const int nvalid = ncol - cc * 32 < 32 ? ncol - cc * 32 : 32;
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            if (j < nvalid)
                                *reinterpret_cast<float4*>(dst + j) = make_float4(acc[j], acc[j + 1], acc[j + 2], acc[j + 3]);
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm->accum_empty);
            kb = 0;
            ++li;
        }
        // slots of slabs this CTA does not have (it owns one K-block fewer than others) read as zero
        for (int l2 = my_items; l2 * (int)gridDim.x < nitems; ++l2) {
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
                mbar_wait(&sm->empty[s], ph ^ 1u, abort_flag, status);   // MMAs that read this stage are done
                if (*abort_flag) break;
                mbar_expect_tx(&sm->landed[s], tx_bytes);
                tma_load_2d(base + (size_t)s * stage_bytes, &xmap, (int)c0, 0, &sm->landed[s]);
                issued = t + 1;
                if (++s == stages) { s = 0; ph ^= 1u; }
                c0 += (int64_t)gridDim.x * kKB;
            }
            if (*abort_flag) {
                // give the copies still in flight a bounded time to land before the CTA goes away
                for (int t = issued > stages ? issued - stages : 0; t < issued; ++t) {
                    const int s = (int)((uint32_t)t % (uint32_t)stages);
                    const uint32_t ph = ((uint32_t)t / (uint32_t)stages) & 1u;
                    for (uint32_t spin = 0; spin < (1u << 16) && !mbar_test(&sm->landed[s], ph); ++spin) __nanosleep(64);
                }
            }
        }
    } else if (lane == 0) {
        // ------------------------------------------------ the MMA threads
        // ------------------------------------------------ (lane 0 of the two warps after the transform warps)
        const int g = warp - kProdWarps;
        const int n_mma = nhalf == 1 ? 2 * ncol : ncol;
        const uint32_t idesc = (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)(n_mma >> 3) << 17) | ((uint32_t)(mrows >> 4) << 24);
        int s = 0, turn = 0;
        uint32_t ph = 0;
        for (int local_item = 0; local_item < my_items; ++local_item) {
            const int nkb = local_item == my_items - 1 ? last_nkb : kBlocksPerSlab;
            if (local_item > 0) mbar_wait(&sm->accum_empty, (uint32_t)((local_item - 1) & 1), abort_flag, status);
            tc_fence_after();
            bool first = true;   // this thread's first MMA of the slab overwrites its accumulator
            for (int kb = 0; kb < nkb; ++kb) {
                const int my_s = s;
                const uint32_t my_ph = ph;
                const bool skip = nhalf == 1 && turn != g;   // m <= 128: the two threads alternate K-blocks
                if (++s == stages) { s = 0; ph ^= 1u; }
                turn ^= 1;
                if (skip) continue;
                mbar_wait(&sm->full[my_s], my_ph, abort_flag, status);
                tc_fence_after();
                const uint32_t hi_addr = smem_u32(base + (size_t)my_s * stage_bytes);
                const uint64_t hi_desc = smem_desc(hi_addr);
                if (nhalf == 1) {
                    const uint32_t dcol = tmem_base + (uint32_t)(g * 2 * ncol);
#pragma unroll
                    for (int kk = 0; kk < kKB / 8; ++kk) {       // one MMA covers 8 columns = 32 bytes
                        const uint64_t ab = hi_desc + (uint64_t)(kk * 2);
                        mma_tf32(dcol, ab, ab, idesc, first ? 0u : 1u);
                        first = false;
                    }
                } else {
                    const uint64_t lo_desc = smem_desc(hi_addr + tile_bytes);
                    const uint32_t dcol = tmem_base + (uint32_t)(g * ncol);
#pragma unroll
                    for (int kk = 0; kk < kKB / 8; ++kk) {
                        const uint64_t a = hi_desc + (uint64_t)(kk * 2 + g * (128 * 128 / 16));
                        mma_tf32(dcol, a, hi_desc + (uint64_t)(kk * 2), idesc, first ? 0u : 1u);
                        mma_tf32(dcol, a, lo_desc + (uint64_t)(kk * 2), idesc, 1u);
                        first = false;
                    }
                }
                mma_commit(&sm->empty[my_s]);   // the stage may be refilled once these MMAs have read it
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

// For one chunk of slabs: gpart[chunk][i*m+j] (i < j) = sum_s sym(T(s))_ij * (r_i(s) + r_j(s)) / 2 with
// r_i(s) = exact norm / tensor-core norm of row i in slab s; gpart[chunk][i*m+i] = sum_s exact norm.
// One CTA per pair of 32-row blocks (bi <= bj) and chunk: per slab it reads the tile T[bi][bj] and the
// mirrored tile T[bj][bi] row by row (coalesced) and transposes the second through shared memory.
constexpr int kRT = 32;
__global__ void __launch_bounds__(kRT * 8)
tc_reduce_kernel(const float* __restrict__ partial, const float* __restrict__ norms, int nitems, int m, int ncol,
                 double* __restrict__ gpart) {
    __shared__ float mirror[kRT][kRT + 1];
    __shared__ double ratio_i[kRT], ratio_j[kRT];
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
    double nsum = 0.0;                       // ty == 0 on a diagonal tile: exact norm of row bi*32 + tx
    const int j = bj * kRT + tx;             // this thread's column of the tile

    for (int s = s0; s < s1; ++s) {
        const float* T = partial + (int64_t)s * elems;
        const float* nrm = norms + (int64_t)s * m;
        if (ty < 2) {
            const int r = (ty == 0 ? bi : bj) * kRT + tx;
            double ratio = 1.0;
            if (r < m) {
                const double t = (double)T[(int64_t)r * ncol + r], nv = (double)nrm[r];
                if (t > 0.0) ratio = nv / t;
                if (ty == 0 && bi == bj) nsum += nv;
            }
            (ty == 0 ? ratio_i : ratio_j)[tx] = ratio;
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
            acc[k] += tij * (0.5 * (ratio_i[il] + ratio_j[tx]));
        }
        __syncthreads();
    }
    const int64_t total = (int64_t)m * m;
#pragma unroll
    for (int k = 0; k < kRT / 8; ++k) {
        const int i = bi * kRT + ty + 8 * k;
        if (i < m && j < m && i < j) gpart[(int64_t)chunk * total + (int64_t)i * m + j] = acc[k];
    }
    if (ty == 0 && bi == bj && j < m) gpart[(int64_t)chunk * total + (int64_t)j * m + j] = nsum;
}

// D_ij = n_i + n_j - 2 G_ij (never negative, zero diagonal); status != 0 -> NaN.
// One warp per pair i < j: the lanes add the chunks round-robin, then a fixed butterfly.
__global__ void tc_dist_kernel(const double* __restrict__ gpart, int nchunks, int m, const int* __restrict__ status,
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
    double gii = 0.0, gjj = 0.0, gij = 0.0;
    for (int c = lane; c < nchunks; c += 32) {
        const double* g = gpart + (int64_t)c * total;
        gii += g[(int64_t)i * m + i];
        gjj += g[(int64_t)j * m + j];
        gij += g[(int64_t)i * m + j];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        gii += __shfl_xor_sync(0xffffffffu, gii, o);
        gjj += __shfl_xor_sync(0xffffffffu, gjj, o);
        gij += __shfl_xor_sync(0xffffffffu, gij, o);
    }
    if (lane == 0) {
        double v = gii + gjj - 2.0 * gij;
        v = v > 0.0 ? v : 0.0;
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

// X as a 2-D fp32 tensor (d columns innermost, m rows, row pitch ld); box = 32 columns x box_rows rows,
// 128-byte swizzle, zero fill outside.
detox_status make_xmap(CUtensorMap* map, const float* X, int64_t ld, int m, int64_t d, int box_rows) {
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return DETOX_ERR_CUDA;
    const cuuint64_t gdim[2] = {(cuuint64_t)d, (cuuint64_t)m};
    const cuuint64_t gstride[1] = {(cuuint64_t)ld * sizeof(float)};
    const cuuint32_t box[2] = {(cuuint32_t)kKB, (cuuint32_t)box_rows};
    const cuuint32_t estride[2] = {1, 1};
    CUresult r = enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(X), gdim, gstride, box, estride,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? DETOX_OK : DETOX_ERR_CUDA;
}

template <int J>
detox_status launch_tc(const TcPlan& p, const CUtensorMap& xmap, int m, int64_t d, float* partial, float* norms,
                       int* status, cudaStream_t s) {
    if (cudaFuncSetAttribute(gram_tc_kernel<J>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)p.smem_bytes) !=
        cudaSuccess)
        return DETOX_ERR_CUDA;
    gram_tc_kernel<J><<<p.grid, kTcThreads, p.smem_bytes, s>>>(xmap, m, d, p.rows_pad, p.mrows, p.box_rows, p.nhalf, p.ncol,
                                                               p.chains, p.tmem_cols, p.stages, p.nkb_total, p.nitems, partial, norms, status);
    return launch_status();
}

}  // namespace

bool tc_supported(const float* X, int64_t ld, int m, int64_t d) {
    // TMA needs a 16-byte aligned base and row pitch; coordinates are 32-bit
    return m > 16 && m <= 256 && aligned16(X) && ld % 4 == 0 && d < (int64_t)1 << 31 && encode_tiled_fn() != nullptr;
}

size_t tc_ws_bytes(int m, int64_t d) {
    TcPlan p = tc_plan(m, d);
    const size_t elems = (size_t)m * p.ncol;
    return align_up((size_t)p.nitems * elems * sizeof(float)) + align_up((size_t)p.nitems * m * sizeof(float)) +
           align_up((size_t)reduce_chunks(m, p.nitems) * m * m * sizeof(double));
}

detox_status launch_sqdist_tc(const float* X, int64_t ld, int m, int64_t d, double* D, void* ws, int* status,
                              cudaStream_t s) {
    TcPlan p = tc_plan(m, d);
    const int64_t elems = (int64_t)m * p.ncol;
    char* base = static_cast<char*>(ws);
    float* partial = reinterpret_cast<float*>(base);
    float* norms = reinterpret_cast<float*>(base + align_up((size_t)p.nitems * elems * sizeof(float)));
    double* gpart = reinterpret_cast<double*>(base + align_up((size_t)p.nitems * elems * sizeof(float)) +
                                              align_up((size_t)p.nitems * m * sizeof(float)));
    CUtensorMap xmap;
    detox_status st = make_xmap(&xmap, X, ld, m, d, p.box_rows);
    if (st != DETOX_OK) return st;
    // chunks per transform thread: m * 8 / kProdThreads, rounded up to a power of two
    const int per_thread = (m * 8 + kProdThreads - 1) / kProdThreads;
    if (per_thread <= 1) st = launch_tc<1>(p, xmap, m, d, partial, norms, status, s);
    else if (per_thread <= 2) st = launch_tc<2>(p, xmap, m, d, partial, norms, status, s);
    else st = launch_tc<4>(p, xmap, m, d, partial, norms, status, s);
    if (st != DETOX_OK) return st;
    const int nt = (m + kRT - 1) / kRT;
    const int nchunks = reduce_chunks(m, p.nitems);
    tc_reduce_kernel<<<dim3((unsigned)(nt * (nt + 1) / 2), (unsigned)nchunks), kRT * 8, 0, s>>>(partial, norms, p.nitems, m,
                                                                                           p.ncol, gpart);
    if ((st = launch_status()) != DETOX_OK) return st;
    tc_dist_kernel<<<(unsigned)ceil_div((int64_t)m * m * 32, 256), 256, 0, s>>>(gpart, nchunks, m, status, D);
    return launch_status();
}

}  // namespace detox
