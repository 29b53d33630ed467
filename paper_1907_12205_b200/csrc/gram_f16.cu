// Pairwise inner products for 16 < m <= 256 on the tensor cores with every fp32 entry split into two fp16 numbers.
//
// y = 2^e (x - c) is the entry after the row's power-of-two scale (and the common vector c, when one is subtracted);
// hi = fp16(y), lo = fp16(y - hi): together they carry 22 bits of y, as the two TF32 parts of the split-TF32 kernels
// do, but fp16 MMAs run at twice the TF32 rate and their operands take half the shared memory, which is what
// bounds those kernels.  T = hi (hi + 2 lo)^T, accumulated in fp32 in tensor memory; G = (T + T^T) / 2.
//
// fp16 has a narrow exponent, so every row is scaled by a power of two chosen from a sample of its columns so that
// its typical entry sits near 2^6: entries up to about a thousand times the row's typical size stay finite, and
// entries down to 2^-8 of it keep all 22 bits (smaller ones keep an absolute accuracy of 2^-31 of the typical size).
// An entry that overflows becomes Inf, the row's tensor-core norm becomes non-finite, and the check that runs after
// the pass then asks for the split-TF32 pass instead: the scale never costs correctness, only time.
//
// Layout of the work as in the split-TF32 kernels: one persistent CTA per SM, 64-column stages dealt round-robin,
// TMA boxes (64 columns x up to 128 rows, unswizzled) into a staging ring, 16 transform warps that write the two MMA
// operands in the 128-byte-swizzled K-major layout and add up the exact squared norms, MMA-issuing threads, slabs of
// 4096 columns drained from tensor memory into fp32 partials.  Up to 128 rows the B operand is the stacked tile
// [hi ; lo] (one MMA per 16 columns, N = 2 ncol; the drain adds twice the lo part); above, a stage arrives as two boxes (the copy engine handles boxes
// of up to 128 rows best), the accumulator has two halves of 128 rows, one per issuing thread, and each thread issues
// A = its half of hi with B = hi and with B = 2 lo into the same accumulator.
// Every wait is bounded, as in the other kernels.
#include <cuda.h>
#include <cuda_fp16.h>

#include "common.cuh"
#include "gram_tc.cuh"
#include "mbarrier.cuh"
#include "tcgen05.cuh"

namespace detox {

namespace {

constexpr int kStageCols = 64;                                  // fp32 columns per stage = one 128-byte row of fp16
constexpr int kStagesPerSlab = (int)(kSlabCols / kStageCols);
constexpr int kMaxStg = 12, kMaxMst = 8;
constexpr size_t kMaxInFlight = 112 * 1024;   // staging bytes beyond which HBM is no faster (a deeper ring measured no gain)
constexpr size_t kMaxInFlightVote = 136 * 1024;   // the same with the vote inside the pass (slots come in multiples of boxes x groups)
constexpr size_t kSmemTail = 4096;   // barriers and the centring ring behind the tiles
constexpr int kCentreWarps = 1;

}  // namespace

// Groups of transform warps, each on stages of its own.  A group starts its next stage only when it is through with
// the chain  wait - read - convert - write - fence - arrive  of the current one, which takes several hundred cycles
// whatever the row count; with few rows that chain, not HBM, sets the pace, so the fewer the rows, the more groups
// share the warps (a thread handles at most four 16-byte pieces of a stage; with five the registers spill and
// 33 .. 40 rows ran slower in four groups than in two).
int f16_groups(int m) { return m <= 32 ? 4 : (m <= 64 ? 2 : 1); }

namespace {

struct F16Plan {
    bool wide;                   // more than 128 rows: two boxes per stage, two accumulator halves
    int nbox, box_rows;          // TMA boxes per stage; rows per box (a multiple of 8)
    int rows_in;                 // rows of the matrix the boxes are cut from (m, or the n members' rows with the vote)
    int ncol;                    // m rounded up to 16
    int mrows;                   // M of the MMA: 64 up to 64 rows, else 128
    int nmma, groups;            // MMA-issuing threads; groups of transform warps
    int lo_row;                  // first row of the lo tile inside an MMA slot
    uint32_t tile_bytes;         // one MMA slot: (lo_row + ncol) rows of 128 bytes
    uint32_t stg_bytes;          // one staging slot: box_rows x 256 bytes
    int tmem_cols;
    int nstg, nmst;
    int nst_total, nitems, grid;
    size_t smem_bytes;
};

// n_in = 0: the m rows themselves are copied in.  n_in > 0 (the vote inside the pass): the boxes hold the n_in rows of the
// group members, from which the transform warps form the m votes.
F16Plan f16_plan(int m, int64_t d, int n_in = 0) {
    F16Plan p;
    p.wide = m > 128;
    p.rows_in = n_in > 0 ? n_in : m;
    p.nbox = p.rows_in > 128 ? 2 : 1;
    p.box_rows = p.nbox == 2 ? ((p.rows_in + 1) / 2 + 7) / 8 * 8 : (p.rows_in + 7) / 8 * 8;
    p.ncol = (m + 15) / 16 * 16;
    p.mrows = m <= 64 ? 64 : 128;
    p.nmma = m <= 64 ? 4 : 2;
    p.groups = f16_groups(m);
    p.lo_row = p.wide ? 256 : p.ncol;
    p.tile_bytes = (uint32_t)(p.lo_row + p.ncol) * 128u;
    p.stg_bytes = (uint32_t)p.box_rows * (uint32_t)kStageCols * 4u;
    p.tmem_cols = 32;
    while (p.tmem_cols < (p.wide ? 2 * p.ncol : p.nmma * 2 * p.ncol)) p.tmem_cols <<= 1;
    p.nmst = 2 * p.groups;   // two MMA slots per transform group
    const size_t left = kSmemBudget - kSmemTail - 1024 - (size_t)p.nmst * p.tile_bytes;
    p.nstg = (int)(left / p.stg_bytes);
    if (p.nstg > kMaxStg) p.nstg = kMaxStg;
    if (n_in > 0) {
        // a staging slot always holds the same box of the same group's stages: a multiple of boxes x groups, as close
        // to the byte count that keeps HBM busy as that allows
        const int unit = p.nbox * p.groups;
        const size_t ub = (size_t)unit * p.stg_bytes;
        int k = (int)(kMaxInFlightVote / ub);
        if (k < 1) k = 1;
        if ((size_t)k * ub < 96 * 1024 && (size_t)(k + 1) * ub <= 160 * 1024) ++k;
        while (k > 1 && (k * unit > p.nstg)) --k;
        p.nstg = k * unit;
    } else {
        while (p.nstg > 2 && (size_t)p.nstg * p.stg_bytes > kMaxInFlight) --p.nstg;
        // several transform groups: a staging slot always holds stages of the same group (see the split-TF32 staged kernel)
        p.nstg -= p.nstg % p.groups;
    }
    p.nst_total = (int)ceil_div(d, (int64_t)kStageCols);
    p.grid = p.nst_total < kSMs ? p.nst_total : kSMs;
    const int per_cta = (p.nst_total + p.grid - 1) / p.grid;
    p.nitems = p.grid * (int)ceil_div(ceil_div((int64_t)per_cta, (int64_t)kStagesPerSlab), (int64_t)kItemSlabs);
    p.smem_bytes = (size_t)p.nstg * p.stg_bytes + (size_t)p.nmst * p.tile_bytes + kSmemTail + 1024 /*alignment slack*/;
    return p;
}

struct F16Smem {
    uint64_t stg_full[kMaxStg];    // TMA bytes of a staging slot have arrived
    uint64_t stg_empty[kMaxStg];   // the transform warps have read it
    uint64_t mst_full[kMaxMst];    // both operands of the stage are written
    uint64_t mst_empty[kMaxMst];   // the MMAs that read them are done
    uint64_t accum_full;
    uint64_t accum_empty;
    uint64_t c_full[kMaxStg];      // the subtracted vector's piece for a stage is written
    uint32_t tmem_base;
    int abort_flag;
    int crow[kMaxCentreRows];
    __align__(16) float cring[kMaxStg][kStageCols];
};
static_assert(sizeof(F16Smem) <= kSmemTail, "fits the shared memory reserved behind the tiles");

__device__ __forceinline__ float pow2f(int e) { return __uint_as_float((uint32_t)(127 + e) << 23); }

// A packed pair of fp32 rounded to a packed pair of fp16 (first entry in the low half; Inf on overflow), and back.
__device__ __forceinline__ uint32_t half2_of(uint64_t v) {
    uint32_t r;
    asm("{\n\t.reg .b32 lo, hi;\n\tmov.b64 {lo, hi}, %1;\n\tcvt.rn.f16x2.f32 %0, hi, lo;\n\t}" : "=r"(r) : "l"(v));
    return r;
}
__device__ __forceinline__ uint64_t float2_of(uint32_t h2) {
    uint64_t r;
    asm("{\n\t.reg .b16 l, h;\n\t.reg .b32 fl, fh;\n\tmov.b32 {l, h}, %1;\n\tcvt.f32.f16 fl, l;\n\tcvt.f32.f16 fh, h;\n\t"
        "mov.b64 %0, {fl, fh};\n\t}"
        : "=l"(r)
        : "r"(h2));
    return r;
}

// J = 16-byte pieces per transform thread and box; LX = groups of transform warps, each on stages of its own; NMMA =
// MMA-issuing threads.  Not WIDE: the threads take the stages in turn and own an accumulator of 2 ncol columns each
// (NMMA a multiple of LX and a divisor of the MMA slots: a thread always serves the same slots and group).  WIDE: both
// threads work on every stage, each on its half of the rows.
//
// VB > 0: the majority vote of DETOX's filtering step (Section 3) runs inside the pass.  The boxes (VB of them per
// stage) then hold the rows of all n = 3 m group members; for every 16-byte piece of vote row g a transform thread
// reads the pieces of the group's three members, takes the value two of them agree on bitwise (zeros when all three
// differ) and carries on with it as if it had been copied in.  A strict majority of the whole rows is also the strict
// majority of every piece, so whenever the group has a winner the piece is the winner's.  The "members a and b differed
// somewhere" bits are collected per thread and ORed into the group's word of `pairdiff` at the end, in the format the
// vote kernels use; the caller finds the winners from them and, should a group have none, repeats the pass on stored
// votes.  The rows listed for centring are member rows here.
template <int J, int LX, int NMMA, bool WIDE, int VB>
__global__ void __launch_bounds__(kProdThreads + 32 * (NMMA + LX + kCentreWarps), 1)
gram_f16_kernel(const __grid_constant__ CUtensorMap xmap, int m, int box_rows, uint32_t stg_bytes, uint32_t tile_bytes,
                int lo_row, int mrows, int ncol, int tmem_cols, int nstg, int nmst, int nst_total, int nitems,
                float* __restrict__ partial, float* __restrict__ norms, const int* __restrict__ centre_ptr,
                const int* __restrict__ expo, int* __restrict__ status, const __grid_constant__ VoteMembers members,
                uint32_t* __restrict__ pairdiff) {
    constexpr int NBOX = VB > 0 ? VB : (WIDE ? 2 : 1);   // boxes copied in per stage
    constexpr int NOUT = VB > 0 ? 1 : NBOX;              // blocks of rows a transform thread writes per stage
    static_assert(VB == 0 || !WIDE, "votes: at most 85 rows come out of at most 255");
    static_assert(!WIDE || (LX == 1 && NMMA == 2), "the wide form has one transform group and one issuing thread per half");
    static_assert(kStagesPerSlab % LX == 0 && (WIDE || kStagesPerSlab % NMMA == 0), "slabs start at every role's own offset");
    static_assert(WIDE || (NMMA % LX == 0 && kMaxMst % NMMA == 0), "an issuing thread serves the same slots and group throughout");
    // Centring: centre_ptr[0] rows, listed from centre_ptr[2] on, are averaged column by column and the average is
    // subtracted from every row before the split (distances do not change; 0 rows: nothing is subtracted).
    const int ncentre = *centre_ptr;
    extern __shared__ uint8_t smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    uint8_t* stg_base = smem_raw + ((1024u - (raw & 1023u)) & 1023u);       // MMA tiles need 1024-byte alignment
    uint8_t* mst_base = stg_base + (size_t)nstg * stg_bytes;                // stg_bytes is a multiple of 2048
    F16Smem* sm = reinterpret_cast<F16Smem*>(mst_base + (size_t)nmst * tile_bytes);
    volatile int* abort_flag = &sm->abort_flag;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    constexpr int kThreads = kProdThreads + 32 * (NMMA + LX + kCentreWarps);
    constexpr int kGroupThreads = kProdThreads / LX, kGroupWarps = kProdWarps / LX;

    if (tid == 0) {
        for (int s = 0; s < nstg; ++s) {
            mbar_init(&sm->stg_full[s], 1);
            mbar_init(&sm->stg_empty[s], kGroupWarps);
            mbar_init(&sm->c_full[s], 1);
        }
        for (int s = 0; s < nmst; ++s) {
            mbar_init(&sm->mst_full[s], kGroupWarps);
            mbar_init(&sm->mst_empty[s], WIDE ? 2 : 1);
        }
        mbar_init(&sm->accum_full, NMMA);
        mbar_init(&sm->accum_empty, kProdWarps);
        sm->abort_flag = 0;
        mbar_fence_init();
    }
    if (tid < ncentre) sm->crow[tid] = centre_ptr[2 + (VB > 0 ? kMaxCentreRows : 0) + tid];
    // rows of the MMA slots that no piece is written to must read as zeros
    for (uint32_t off = (uint32_t)tid * 16u; off < tile_bytes * (uint32_t)nmst; off += kThreads * 16u)
        *reinterpret_cast<uint4*>(mst_base + off) = make_uint4(0u, 0u, 0u, 0u);
    fence_proxy_async_smem();
    if (warp == 0) tmem_alloc(&sm->tmem_base, (uint32_t)tmem_cols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sm->tmem_base;

    // This CTA owns the stages b, b + G, b + 2G, ... (b = blockIdx.x, G = gridDim.x), t = 0 .. total-1 in its own
    // count.  Box u = NBOX t + h of stage t lands in staging slot u % nstg; the stage is transformed into MMA slot
    // t % nmst; its piece of the subtracted vector sits in ring slot t % nstg.  A slab is kStagesPerSlab consecutive
    // stages (the last slab may be shorter) and goes to output slot b + G * (slab number / kItemSlabs).
    const int total = (nst_total - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    const int my_items = (total + kStagesPerSlab - 1) / kStagesPerSlab;
    const int last_nst = total - (my_items - 1) * kStagesPerSlab;
    const uint32_t lo_off = (uint32_t)lo_row * 128u;

    if (warp < kProdWarps) {
        // ------------------------------------------------ transform warps, then epilogue of each slab
        const int group = warp / kGroupWarps, gtid = tid - group * kGroupThreads;
        // this thread's pieces of a box are (row, q) = ((gtid >> 4) + R j, gtid & 15): 16 bytes at column 4 q of the
        // stage, which become 8 bytes of hi and 8 bytes of lo.  R is a multiple of 8 and so is box_rows, hence the
        // swizzle term of the destination is the same for all j and both boxes.
        constexpr int R = kGroupThreads / 16;
        const int row0 = gtid >> 4, q = gtid & 15;
        const uint32_t src0 = (uint32_t)row0 * (uint32_t)(kStageCols * 4) + (uint32_t)q * 16u;
        constexpr uint32_t kSrcStep = (uint32_t)R * (uint32_t)(kStageCols * 4);
        constexpr uint32_t kDstStep = (uint32_t)(R / 8) * 1024u;
        uint32_t dst0[NOUT];
        float sc[NOUT][J];      // the rows' scales (0: no such row)
        uint64_t sq[NOUT][J];   // packed pair of partial sums of squares per piece (of the scaled, centred values)
        // votes: where the three members' pieces lie inside the stage's boxes (bit 31: in the second box), and the
        // "differed" bits of the member pairs (0,1), (0,2), (1,2) of the thread's j-th group at bits 3j .. 3j + 2
        uint32_t moff[VB > 0 ? J : 1][3];
        uint32_t differed = 0u;
#pragma unroll
        for (int h = 0; h < NOUT; ++h) {
            const int g0 = h * box_rows + row0;
            dst0[h] = (uint32_t)(g0 >> 3) * 1024u + (uint32_t)(g0 & 7) * 128u + (uint32_t)(((q >> 1) ^ (g0 & 7)) << 4) +
                      (uint32_t)(q & 1) * 8u;
#pragma unroll
            for (int j = 0; j < J; ++j) {
                const int local = row0 + R * j, grow = h * box_rows + local;
                sc[h][j] = ((VB > 0 || local < box_rows) && grow < m) ? pow2f(expo[grow]) : 0.f;
                sq[h][j] = 0ull;
            }
        }
        if (VB > 0) {
#pragma unroll
            for (int j = 0; j < J; ++j) {
#pragma unroll
                for (int k = 0; k < 3; ++k) {
                    const int g = row0 + R * j;
                    int xr = g < m ? (int)members.id[g * 3 + k] : 0;
                    uint32_t second = 0u;
                    if (VB == 2 && xr >= box_rows) { xr -= box_rows; second = 0x80000000u; }
                    moff[j][k] = ((uint32_t)xr * (uint32_t)(kStageCols * 4) + (uint32_t)q * 16u) | second;
                }
            }
        }

        // one 16-byte piece (as two packed pairs) -> scaled, centred, added to the row's sum of squares, split into
        // hi and lo and written to the two operand tiles
        auto emit = [&](uint64_t a, uint64_t b, const ulonglong2& ck, float scale, uint64_t& sumsq, uint8_t* to) {
            const uint32_t sb = __float_as_uint(scale);
            const uint64_t s2 = ((uint64_t)sb << 32) | sb;
            if (ncentre > 0) { a = sub2(a, ck.x); b = sub2(b, ck.y); }
            a = mul2(a, s2);
            b = mul2(b, s2);
            sumsq = fma2(a, a, fma2(b, b, sumsq));
            const uint32_t h01 = half2_of(a), h23 = half2_of(b);
            uint64_t la = sub2(a, float2_of(h01)), lb = sub2(b, float2_of(h23));   // exact
            if (WIDE) { la = add2(la, la); lb = add2(lb, lb); }   // (not WIDE: the drain doubles the lo part)
            *reinterpret_cast<uint2*>(to) = make_uint2(h01, h23);
            *reinterpret_cast<uint2*>(to + lo_off) = make_uint2(half2_of(la), half2_of(lb));
        };

        int ss = group * NBOX, ms = group, cs = group, t = group;
        uint32_t sph = 0, mph = 0, cph = 0;
        for (int li = 0; li < my_items; ++li) {
            const int nst = li == my_items - 1 ? last_nst : kStagesPerSlab;
            const int t_end = li * kStagesPerSlab + nst;
            for (; t < t_end; t += LX) {
                ulonglong2 ck = make_ulonglong2(0ull, 0ull);
                if (ncentre > 0) {
                    mbar_wait(&sm->c_full[cs], cph, abort_flag, status);
                    ck = *reinterpret_cast<const ulonglong2*>(&sm->cring[cs][q * 4]);
                }
                if constexpr (VB > 0) {
                    // all boxes of the stage must have landed: a group's members may lie in either
                    const uint8_t* box[2];
                    int slot[2];
#pragma unroll
                    for (int h = 0; h < NBOX; ++h) {
                        mbar_wait(&sm->stg_full[ss], sph, abort_flag, status);
                        box[h] = stg_base + (size_t)ss * stg_bytes;
                        slot[h] = ss;
                        if (++ss >= nstg) { ss -= nstg; sph ^= 1u; }
                    }
                    if (NBOX == 1) { box[1] = box[0]; slot[1] = slot[0]; }
                    ulonglong2 x[J];
#pragma unroll
                    for (int j = 0; j < J; ++j) {
                        if (sc[0][j] != 0.f) {
                            ulonglong2 v[3];
#pragma unroll
                            for (int k = 0; k < 3; ++k)
                                v[k] = *reinterpret_cast<const ulonglong2*>(((moff[j][k] >> 31) ? box[1] : box[0]) +
                                                                            (moff[j][k] & 0x7fffffffu));
                            const bool ne01 = ((v[0].x ^ v[1].x) | (v[0].y ^ v[1].y)) != 0ull;
                            const bool ne02 = ((v[0].x ^ v[2].x) | (v[0].y ^ v[2].y)) != 0ull;
                            const bool ne12 = ((v[1].x ^ v[2].x) | (v[1].y ^ v[2].y)) != 0ull;
                            differed |= ((ne01 ? 1u : 0u) | (ne02 ? 2u : 0u) | (ne12 ? 4u : 0u)) << (3 * j);
                            // the first member when it agrees with another one, else the second when it agrees with
                            // the third, else nothing
                            const bool first = !ne01 || !ne02, other = !ne12;
                            x[j].x = first ? v[0].x : (other ? v[1].x : 0ull);
                            x[j].y = first ? v[0].y : (other ? v[1].y : 0ull);
                        }
                    }
                    // the boxes have been read (the values sit in registers)
                    __syncwarp();
                    if (lane == 0) {
#pragma unroll
                        for (int h = 0; h < NBOX; ++h) mbar_arrive(&sm->stg_empty[slot[h]]);
                    }
                    mbar_wait(&sm->mst_empty[ms], mph ^ 1u, abort_flag, status);   // the MMAs that read this slot are done
                    uint8_t* dst = mst_base + (size_t)ms * tile_bytes + dst0[0];
#pragma unroll
                    for (int j = 0; j < J; ++j)
                        if (sc[0][j] != 0.f) emit(x[j].x, x[j].y, ck, sc[0][j], sq[0][j], dst + j * kDstStep);
                    fence_proxy_async_smem();   // make the generic-proxy stores visible to the MMA's reads
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sm->mst_full[ms]);   // one arrival per transform warp of the group
                } else {
#pragma unroll
                    for (int h = 0; h < NBOX; ++h) {
                        mbar_wait(&sm->stg_full[ss], sph, abort_flag, status);
                        const uint8_t* src = stg_base + (size_t)ss * stg_bytes + src0;
                        ulonglong2 x[J];
#pragma unroll
                        for (int j = 0; j < J; ++j)
                            if (sc[h][j] != 0.f) x[j] = *reinterpret_cast<const ulonglong2*>(src + j * kSrcStep);
                        // the MMAs that read this slot are done
                        if (h == 0) mbar_wait(&sm->mst_empty[ms], mph ^ 1u, abort_flag, status);
                        uint8_t* dst = mst_base + (size_t)ms * tile_bytes + dst0[h];
#pragma unroll
                        for (int j = 0; j < J; ++j)
                            if (sc[h][j] != 0.f) emit(x[j].x, x[j].y, ck, sc[h][j], sq[h][j], dst + j * kDstStep);
                        if (h == NBOX - 1) fence_proxy_async_smem();   // make the generic-proxy stores visible to the MMA's reads
                        __syncwarp();
                        if (lane == 0) {
                            mbar_arrive(&sm->stg_empty[ss]);                       // the staging slot has been read
                            if (h == NBOX - 1) mbar_arrive(&sm->mst_full[ms]);     // one arrival per transform warp of the group
                        }
                        if (++ss >= nstg) { ss -= nstg; sph ^= 1u; }
                    }
                }
                if (LX > 1) {
                    ss += (LX - 1) * NBOX;
                    if (ss >= nstg) { ss -= nstg; sph ^= 1u; }
                }
                ms += LX;
                if (ms >= nmst) { ms -= nmst; mph ^= 1u; }
                cs += LX;
                if (cs >= nstg) { cs -= nstg; cph ^= 1u; }
            }
            // output slot of this slab, and whether the slab opens / closes it
            const int item = (int)blockIdx.x + (li / kItemSlabs) * (int)gridDim.x;
            const bool opens = li % kItemSlabs == 0, closes = li % kItemSlabs == kItemSlabs - 1 || li == my_items - 1;

            // ---- end of a slab: this group's share of the exact squared norms (the 16 lanes that share a row add
            // up; the reduction kernel adds the groups) ...
#pragma unroll
            for (int h = 0; h < NOUT; ++h) {
#pragma unroll
                for (int j = 0; j < J; ++j) {
                    float v = __uint_as_float((uint32_t)sq[h][j]) + __uint_as_float((uint32_t)(sq[h][j] >> 32));
                    v += __shfl_xor_sync(0xffffffffu, v, 1);
                    v += __shfl_xor_sync(0xffffffffu, v, 2);
                    v += __shfl_xor_sync(0xffffffffu, v, 4);
                    v += __shfl_xor_sync(0xffffffffu, v, 8);
                    if (closes) {
                        if (q == 0 && sc[h][j] != 0.f)
                            norms[((int64_t)item * LX + group) * m + (h * box_rows + row0 + R * j)] = v;
                        sq[h][j] = 0ull;
                    }
                }
            }
            // ... and the accumulator drain: warp w reads TMEM lanes 32 (w % 4) .. + 31; the warps that share a lane
            // quarter take 16-column chunks round-robin
            mbar_wait(&sm->accum_full, (uint32_t)(li & 1), abort_flag, status);
            tc_fence_after();
            const int quarter = warp & 3;
            float* out_item = partial + (int64_t)item * m * ncol;
            if (WIDE) {
                // accumulator row i of a half sits in lane i; half h occupies columns h ncol .. h ncol + ncol - 1
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
            } else {
                // M = 128: accumulator row i sits in TMEM lane i; M = 64: in lane 32 (i / 16) + i % 16
                const int row = mrows == 64 ? (lane < 16 ? quarter * 16 + lane : m) : quarter * 32 + lane;
                // the hi.hi and hi.lo parts of every issuing thread's accumulator (a slab shorter than the number of
                // issuing threads leaves the later threads' accumulators untouched: skip them)
                const int nparts = 2 * (nst < NMMA ? nst : NMMA);
                for (int cc = warp >> 2; cc * 16 < ncol; cc += kProdWarps / 4) {
                    float acc[16];
#pragma unroll
                    for (int j = 0; j < 16; ++j) acc[j] = 0.f;
                    for (int part = 0; part < nparts; ++part) {
                        uint32_t v[16];
                        tmem_load16(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(part * ncol + cc * 16), v);
                        const float w = (part & 1) ? 2.f : 1.f;   // odd parts are hi.lo: T = hi (hi + 2 lo)^T
#pragma unroll
                        for (int j = 0; j < 16; ++j) acc[j] = fmaf(__uint_as_float(v[j]), w, acc[j]);
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
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm->accum_empty);
        }
        if constexpr (VB > 0) {
            // the vote's evidence: which member pairs of this thread's groups differed anywhere in this CTA's columns
            // (the 16 lanes that share a row combine theirs first)
#pragma unroll
            for (int j = 0; j < J; ++j) {
                uint32_t bits = (differed >> (3 * j)) & 7u;
                bits |= __shfl_xor_sync(0xffffffffu, bits, 1);
                bits |= __shfl_xor_sync(0xffffffffu, bits, 2);
                bits |= __shfl_xor_sync(0xffffffffu, bits, 4);
                bits |= __shfl_xor_sync(0xffffffffu, bits, 8);
                const int g = row0 + R * j;
                if (q == 0 && g < m && bits != 0u) atomicOr(pairdiff + (int64_t)g * kPairWords, bits);
            }
        }
        // slots of slabs this CTA does not have (it owns one stage fewer than others) read as zero
        for (int l2 = (my_items + kItemSlabs - 1) / kItemSlabs; l2 * (int)gridDim.x < nitems; ++l2) {
            const int64_t item = (int64_t)blockIdx.x + (int64_t)l2 * gridDim.x;
            for (int e = tid; e < m * ncol; e += kProdThreads) partial[item * m * ncol + e] = 0.f;
            for (int e = tid; e < m * LX; e += kProdThreads) norms[item * LX * m + e] = 0.f;
        }
    } else if (warp == kProdWarps + NMMA + LX) {
        // ------------------------------------------------ the centring warp: averages the listed rows of every stage
        // as it lands and hands the 64 averages on.  Lanes 0-15 add the first eight listed rows, lanes 16-31 the
        // others, four columns (16 bytes) a lane; the halves meet through shuffles.  A column whose sum is not finite
        // is left uncentred (zero is subtracted there).
        if (ncentre > 0) {
            const float inv = 1.f / (float)ncentre;
            const int half = lane >> 4;
            constexpr int kPerHalf = kMaxCentreRows / 2;
            uint32_t off[kPerHalf];
            uint32_t second = 0;   // bit k: listed row k of this half arrives in the second box of a stage
#pragma unroll
            for (int k = 0; k < kPerHalf; ++k) {
                const int kk = half * kPerHalf + k;
                int r = sm->crow[kk < ncentre ? kk : 0];
                if (NBOX == 2 && r >= box_rows) { r -= box_rows; second |= 1u << k; }
                off[k] = (uint32_t)r * (uint32_t)(kStageCols * 4) + (uint32_t)(lane & 15) * 16u;
            }
            const int mine = ncentre - half * kPerHalf;   // listed rows in this half (may be <= 0)
            int s = 0, cs = 0;
            uint32_t ph = 0, cph = 0;
            (void)cph;
            for (int t = 0; t < total; ++t) {
                if (!mbar_wait(&sm->stg_full[s], ph, abort_flag, status)) break;
                const uint8_t* box0 = stg_base + (size_t)s * stg_bytes;
                const uint8_t* box1 = box0;
                if (++s == nstg) { s = 0; ph ^= 1u; }
                if (NBOX == 2) {
                    if (!mbar_wait(&sm->stg_full[s], ph, abort_flag, status)) break;
                    box1 = stg_base + (size_t)s * stg_bytes;
                    if (++s == nstg) { s = 0; ph ^= 1u; }
                }
                float4 v[kPerHalf];
#pragma unroll
                for (int k = 0; k < kPerHalf; ++k)
                    v[k] = *reinterpret_cast<const float4*>(((second >> k) & 1u ? box1 : box0) + off[k]);
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
                    *reinterpret_cast<float4*>(&sm->cring[cs][4 * lane]) =
                        make_float4(finite_or_zero(acc.x) * inv, finite_or_zero(acc.y) * inv, finite_or_zero(acc.z) * inv,
                                    finite_or_zero(acc.w) * inv);
                __syncwarp();
                if (lane == 0) mbar_arrive(&sm->c_full[cs]);
                if (++cs == nstg) cs = 0;
            }
        }
    } else if (warp >= kProdWarps + NMMA) {
        // ------------------------------------------------ the TMA threads: thread l issues the stages l, l + LX, ...
        // (all boxes of a stage), i.e. always the stages of transform group l
        if (lane == 0) {
            const int l = warp - (kProdWarps + NMMA);
            int issued = 0;   // boxes this thread has issued
            int s = (l * NBOX) % nstg;
            uint32_t ph = (uint32_t)((l * NBOX) / nstg) & 1u;
            int64_t c0 = ((int64_t)blockIdx.x + (int64_t)l * gridDim.x) * kStageCols;   // first column of the stage
            bool ok = true;
            for (int t = l; t < total && ok; t += LX) {
#pragma unroll
                for (int h = 0; h < NBOX; ++h) {
                    if (!mbar_wait(&sm->stg_empty[s], ph ^ 1u, abort_flag, status)) { ok = false; break; }   // the slot has been read
                    mbar_expect_tx(&sm->stg_full[s], stg_bytes);
                    tma_load_2d(stg_base + (size_t)s * stg_bytes, &xmap, (int)c0, h * box_rows, &sm->stg_full[s]);
                    ++issued;
                    if (++s >= nstg) { s -= nstg; ph ^= 1u; }
                }
                if (LX > 1) {
                    s += (LX - 1) * NBOX;
                    if (s >= nstg) { s -= nstg; ph ^= 1u; }
                }
                c0 += (int64_t)LX * gridDim.x * kStageCols;
            }
            if (*abort_flag) {
                // give this thread's copies still in flight a bounded time to land before the CTA goes away
                for (int i = issued > nstg ? issued - nstg : 0; i < issued; ++i) {
                    const int u = (l + LX * (i / NBOX)) * NBOX + i % NBOX;   // the box's number in the CTA's sequence
                    const int s2 = (int)((uint32_t)u % (uint32_t)nstg);
                    const uint32_t ph2 = ((uint32_t)u / (uint32_t)nstg) & 1u;
                    for (uint32_t spin = 0; spin < (1u << 16) && !mbar_test(&sm->stg_full[s2], ph2); ++spin) __nanosleep(64);
                }
            }
        }
    } else if (lane == 0) {
        // ------------------------------------------------ the MMA threads (lane 0 of the NMMA warps after the
        // transform warps)
        const int g = warp - kProdWarps;
        // instruction descriptor: fp32 accumulator, fp16 A and B, both K-major, N / 8 and M / 16
        const int n_mma = WIDE ? ncol : 2 * ncol;
        const uint32_t idesc = (1u << 4) | ((uint32_t)(n_mma >> 3) << 17) | ((uint32_t)(mrows >> 4) << 24);
        const uint32_t dcol = tmem_base + (uint32_t)(g * n_mma);
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
                const bool skip = !WIDE && turn != g;
                if (++s == nmst) { s = 0; ph ^= 1u; }
                if (++turn == NMMA) turn = 0;
                if (skip) continue;
                mbar_wait(&sm->mst_full[my_s], my_ph, abort_flag, status);
                tc_fence_after();
                const uint32_t addr = smem_u32(mst_base + (size_t)my_s * tile_bytes);
                const uint64_t desc = smem_desc(addr);
                if (WIDE) {
                    const uint64_t lo_desc = smem_desc(addr + lo_off);
#pragma unroll
                    for (int kk = 0; kk < kStageCols / 16; ++kk) {   // one MMA covers 16 columns = 32 bytes
                        const uint64_t a = desc + (uint64_t)(kk * 2 + g * (128 * 128 / 16));
                        mma_f16(dcol, a, desc + (uint64_t)(kk * 2), idesc, first ? 0u : 1u);   // A = this half of hi, B = hi
                        mma_f16(dcol, a, lo_desc + (uint64_t)(kk * 2), idesc, 1u);            // ... and B = 2 lo
                        first = false;
                    }
                } else {
#pragma unroll
                    for (int kk = 0; kk < kStageCols / 16; ++kk) {
                        const uint64_t ab = desc + (uint64_t)(kk * 2);
                        mma_f16(dcol, ab, ab, idesc, first ? 0u : 1u);   // A = hi rows, B = [hi ; lo]
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

template <int J, int LX, int NMMA, bool WIDE, int VB = 0>
detox_status launch_f16(const F16Plan& p, const CUtensorMap& xmap, int m, const TcBuffers& b, const int* expo,
                        cudaStream_t s, const VoteMembers& members = VoteMembers{}, uint32_t* pairdiff = nullptr) {
    if (p.smem_bytes > kSmemBudget || p.nstg > kMaxStg || p.nstg < p.nbox * LX) return DETOX_ERR_UNSUPPORTED;
    if (cudaFuncSetAttribute(gram_f16_kernel<J, LX, NMMA, WIDE, VB>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)p.smem_bytes) != cudaSuccess)
        return DETOX_ERR_CUDA;
    constexpr int kThreads = kProdThreads + 32 * (NMMA + LX + kCentreWarps);
    gram_f16_kernel<J, LX, NMMA, WIDE, VB><<<p.grid, kThreads, p.smem_bytes, s>>>(
        xmap, m, p.box_rows, p.stg_bytes, p.tile_bytes, p.lo_row, p.mrows, p.ncol, p.tmem_cols, p.nstg, p.nmst, p.nst_total,
        p.nitems, b.partial, b.norms, b.centre, expo, b.status, members, pairdiff);
    return launch_status();
}

}  // namespace

int f16_nitems(int m, int64_t d) { return f16_plan(m, d).nitems; }

detox_status launch_gram_f16(const float* X, int64_t ld, int m, int64_t d, const TcBuffers& b, const int* expo,
                             cudaStream_t s) {
    const F16Plan p = f16_plan(m, d);
    CUtensorMap xmap;
    detox_status st = make_xmap(&xmap, X, ld, m, d, kStageCols, p.box_rows, false);
    if (st != DETOX_OK) return st;
    // 16-byte pieces per transform thread and box: box rows x 16 / (threads of a group), rounded up
    const int gt = kProdThreads / p.groups;
    const int per_thread = (p.box_rows * (kStageCols / 4) + gt - 1) / gt;
    if (p.wide) {
        if (per_thread <= 3) return launch_f16<3, 1, 2, true>(p, xmap, m, b, expo, s);
        return launch_f16<4, 1, 2, true>(p, xmap, m, b, expo, s);
    }
    if (p.groups == 4) {   // up to 32 rows: four transform groups, four MMA-issuing threads
        if (per_thread <= 3) return launch_f16<3, 4, 4, false>(p, xmap, m, b, expo, s);
        return launch_f16<4, 4, 4, false>(p, xmap, m, b, expo, s);
    }
    if (p.groups == 2) {   // up to 64 rows: two transform groups, four MMA-issuing threads
        if (per_thread <= 3) return launch_f16<3, 2, 4, false>(p, xmap, m, b, expo, s);
        return launch_f16<4, 2, 4, false>(p, xmap, m, b, expo, s);
    }
    if (per_thread <= 3) return launch_f16<3, 1, 2, false>(p, xmap, m, b, expo, s);
    return launch_f16<4, 1, 2, false>(p, xmap, m, b, expo, s);
}

// The vote inside the pass: every three consecutive entries of `members` (rows of X) give one vote; 16 < G <= 85.
bool f16_vote_supported(int n, int r) { return r == 3 && n % 3 == 0 && n / 3 > 16 && n <= 255; }

detox_status launch_gram_f16_vote(const float* X, int64_t ld, int n, int64_t d, const IdTable& groups,
                                  uint32_t* pairdiff, const TcBuffers& b, const int* expo, cudaStream_t s) {
    if (!f16_vote_supported(n, 3)) return DETOX_ERR_UNSUPPORTED;
    const int m = n / 3;
    VoteMembers members;
    for (int i = 0; i < 256; ++i) members.id[i] = i < n ? (uint8_t)groups.id[i] : 0;
    const F16Plan p = f16_plan(m, d, n);
    CUtensorMap xmap;
    detox_status st = make_xmap(&xmap, X, ld, n, d, kStageCols, p.box_rows, false);
    if (st != DETOX_OK) return st;
    // vote rows per transform thread: one piece of every (threads of a group / 16)-th row
    const int per_thread = (m * (kStageCols / 4) + kProdThreads / p.groups - 1) / (kProdThreads / p.groups);
    if (p.groups == 4) {
        if (per_thread <= 3) return launch_f16<3, 4, 4, false, 1>(p, xmap, m, b, expo, s, members, pairdiff);
        return launch_f16<4, 4, 4, false, 1>(p, xmap, m, b, expo, s, members, pairdiff);
    }
    if (p.groups == 2) {
        if (p.nbox == 1) {
            if (per_thread <= 3) return launch_f16<3, 2, 4, false, 1>(p, xmap, m, b, expo, s, members, pairdiff);
            return launch_f16<4, 2, 4, false, 1>(p, xmap, m, b, expo, s, members, pairdiff);
        }
        if (per_thread <= 3) return launch_f16<3, 2, 4, false, 2>(p, xmap, m, b, expo, s, members, pairdiff);
        return launch_f16<4, 2, 4, false, 2>(p, xmap, m, b, expo, s, members, pairdiff);
    }
    if (p.nbox != 2 || per_thread > 3) return DETOX_ERR_UNSUPPORTED;   // 65 .. 85 votes come from 195 .. 255 rows
    return launch_f16<3, 1, 2, false, 2>(p, xmap, m, b, expo, s, members, pairdiff);
}

}  // namespace detox
