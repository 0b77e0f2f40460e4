// Squared per-example gradient sums on the 5th-generation tensor cores (tcgen05, sm_100a).
//
//   D[m][n] = sum_k A(k,m)^2 * B(k,n)^2          (the contraction behind Eq. 2 / Algorithm 1's
//                                                  "v_i +=" line; N_params*|B| multiply-adds, Sec. 5)
// Operands stay fp32 in global memory.  Per 32-deep k slice a thread block
//   1. TMA-loads the raw fp32 tiles of A (128 rows) and B (kBN rows) into a pipeline stage
//      (128-byte swizzle, out-of-range parts filled with zeros),
//   2. squares every element in fp32 and splits the square into two TF32 numbers hi + lo
//      (hi = x*x rounded to 11 significant bits, lo = x*x - hi, of which the tensor core reads the
//      leading 11 bits); the transform is elementwise
//      and in place (hi overwrites the raw tile, lo goes beside it), so both inherit the swizzled
//      layout the tensor core wants,
//   3. issues three tcgen05.mma per 8-deep step -- hi*hi, hi*lo, lo*hi -- into a TMEM
//      accumulator (the dropped lo*lo term is 2^-22 relative).  In the TMA-fed K-major form the two
//      cross terms use bf16 copies of hi and lo instead (kind::f16, 16 deep per instruction): a
//      cross term is 2^-11 of the product, so 8-bit operands leave an error below 2^-18 of it.
// The tensor core's fp32 accumulation is not trusted over long reductions: every kChunk k slices
// the accumulator is drained by four epilogue warps (tcgen05.ld) and added, round-to-nearest, to
// fp32 registers while the next chunk accumulates into the second TMEM buffer.
// Work distribution: the (layer, tile, k slice) space of a launch is laid out linearly and cut into one
// contiguous range per thread block, with at most one block per SM; a block walks its range segment by
// segment (a segment = consecutive slices of one output tile) with the pipeline running across segment
// borders.  A segment that covers a tile's whole reduction writes the result; otherwise it writes a partial
// tile to scratch and a second kernel adds the partial tiles of a tile in a fixed order.
//
// Operand layouts:
//   dense layer: A = delta[z][out], B = x[z][in]  (m / n innermost: MN-major tiles, both by TMA)
//   conv layer:  the error tile is delta[z][o][p], p = (ho,wo) innermost (K-major); the input tile is
//                the im2col view of x, row (c,kh,kw), column k = (z,ho,wo).  Each example contributes
//                ceil(P/32) slices.  Error tile: TMA when the row pitch P*4 is a multiple of 16 bytes,
//                else gathered.  Input tile: TMA for a 1x1 / stride 1 / unpadded kernel (then it is
//                just x[z][c][p]); otherwise the transform warps gather it straight from global
//                memory, four consecutive k per thread, zero outside the image -- im2col is never
//                materialised.  With few output channels (Cout <= 64) the roles are swapped: the
//                im2col rows become the 128-row A tile and the errors the narrow B tile.
//
// Warp roles (448 threads): 0 TMA producer, 1 MMA issuer + TMEM owner, 2-9 transform, 10-13 epilogue.
// While the epilogue warps write a segment's tile out, the other roles are already working on the next one.
// Every wait on an mbarrier is bounded; on expiry the block raises an abort flag, all roles fall
// through to the common exit, outstanding TMA loads are waited for (bounded) and TMEM is freed.
#include <cuda.h>
#include <cuda_bf16.h>

#include <cstdlib>

#include "vgc_common.cuh"

namespace vgc {

namespace tc {

constexpr int kBM = 128;            // output rows per block (UMMA M)
constexpr int kBN = 128;            // output columns per block (UMMA N)
constexpr int kBK = 32;             // k per pipeline slice (= 128 bytes of fp32)
#ifndef VGC_TC_RAW_SLOTS
#define VGC_TC_RAW_SLOTS 5
#endif
#ifndef VGC_TC_LO_SLOTS
#define VGC_TC_LO_SLOTS 2
#endif
// The pipeline is bound by how many bytes are in flight, so the raw tiles get as many slots as fit:
// a raw slot holds the fp32 tiles of one slice (overwritten in place by their hi parts), a lo slot the
// lo parts, which only exist between the transform and the MMAs that consume them.
constexpr int kRawSlots = VGC_TC_RAW_SLOTS;
constexpr int kLoSlots = VGC_TC_LO_SLOTS;
#ifndef VGC_TC_GROUPS
#define VGC_TC_GROUPS 2
#endif
// Transform warps: groups of four warps; in the forms whose slices are taken by one group each, the groups work on
// consecutive slices side by side (a slice's transform is a chain of shared-memory round trips, waits and fences: its
// latency, not the arithmetic, sets the pace, so slices in flight are what counts).  The element-wise gathers share a
// slice among eight warps (the first two groups).
constexpr int kGroups = VGC_TC_GROUPS;
constexpr int kTransformWarps = 4 * kGroups;
constexpr int kGatherThreads = 256;                                 // threads sharing a slice in the one-group forms
constexpr int kEpilogueWarps = 4;
constexpr int kThreadsTc = 32 * (2 + kTransformWarps + kEpilogueWarps);
constexpr uint32_t kRawBytesA = kBM * kBK * 4;                      // 16 KB
constexpr uint32_t kRawBytesB = kBN * kBK * 4;                      // 16 KB
constexpr uint32_t kRawStageBytes = kRawBytesA + kRawBytesB;        // 32 KB: [A raw/hi][B raw/hi], same for lo
constexpr uint32_t kLoBase = kRawSlots * kRawStageBytes;            // lo slots follow the raw slots
constexpr uint32_t kSmemBytes = (kRawSlots + kLoSlots) * kRawStageBytes + 1024 /*align*/ + 128;
// With the A operand in tensor memory a lo slot holds the B tile only, so twice as many fit; the A
// operand ring in TMEM has the same number of slots and shares their barrier.
constexpr int kLoSlotsAT = 2 * kLoSlots;
// Pure TMA form with A in tensor memory ("split rings"): the raw A tile is dead as soon as the transform has
// read it, long before the MMAs of its slice retire.  It therefore gets a ring of its own that is freed
// early, and the 16-KB units this saves hold more B tiles: more slices in flight from the same shared memory.
constexpr int kSplitA = 4, kSplitB = kGroups > 2 ? 6 : 7, kSplitLo = kGroups > 2 ? 4 : 3;   // 16-KB units: A raw, B raw/hi, B lo (+ A in TMEM)
static_assert((kSplitA + kSplitB + kSplitLo) * kRawBytesA <= (kRawSlots + kLoSlots) * kRawStageBytes, "smem budget");
constexpr uint32_t kTmemColsA = 64;                                 // per slot: 32 columns hi + 32 columns lo
constexpr uint32_t kTmemCols = 512;                                 // two accumulator buffers + the A operand ring
constexpr uint32_t kWaitLimit = 1u << 22;                           // polls before a wait gives up

enum { kMajorK = 0, kMajorMN = 1 };

// how a tile gets its rows; kGatherTaps4 / kGatherTaps2: im2col rows of a Kw = 3, stride 1, pad_w = 1 kernel
// gathered three taps at a time (output width a multiple of 4 / of 2)
// kGatherTaps4S2 / kGatherTaps2S2: the same for stride 2 along w (input width twice the output width)
// kGatherTaps7S2: seven taps at a time for a Kw = 7, stride-2, pad-3 kernel (the first layer of the ImageNet networks)
enum { kTma = 0, kGatherErr = 1, kGatherIm2col = 2, kGatherTaps4 = 3, kGatherTaps2 = 4, kGatherTaps4S2 = 5,
       kGatherTaps2S2 = 6, kGatherTaps7S2 = 7 };

struct Params {
    int M, N;                // rows of the A tile space / of the B tile space
    int k_slices;            // 32-deep slices of one tile's reduction
    int p_slices;            // conv: slices per example (ceil(P/32)); dense: 1
    int chunk;               // slices per accumulator drain
    int unit;                // slices that stay in one block: the reduction is cut between units only
    int units_per_tile;      // k_slices / unit
    int units_total;         // layers * tiles * units_per_tile: the launch's work, cut evenly over the blocks:
    int units_q, units_r;    // block b owns units [b q + min(b, r), ...) with q = total / blocks, r = total % blocks
    int tiles_x, tiles_y;    // 128-column / 128-row tiles of one layer's result
    uint32_t tx_bytes;       // bytes the TMA loads of one slice deliver
    uint32_t tx_bytes_a;     // of which the A tile's
    float scale;
    int accumulate;
    int C, H, W, Cout, Kh, Kw, sh, sw, ph, pw, Wo, P;     // conv geometry (gathered tiles)
    int chw;                 // C*H*W
    unsigned wo_magic;       // floor(2^32 / Wo) + 1: p / Wo == umulhi(p, wo_magic) for p * Wo < 2^32
    long long ld_m, ld_n;    // result: element (m, n) lives at S[m*ld_m + n*ld_n]; one of the two is 1
    float *partial;          // scratch for partial tiles [2 * block + (0: a block's first segment, 1: its last)][column][row]
    uint32_t *status;        // device word; VGC_DEV_TIMEOUT is OR-ed in if a wait expired
};

// Layers of one geometry computed by one launch: their tensor maps and pointers.
constexpr int kMaxBatch = 8;
struct Batch {
    CUtensorMap a[kMaxBatch], b[kMaxBatch];
    const float *x[kMaxBatch], *delta[kMaxBatch];   // raw operands (gathered tiles)
    float *S[kMaxBatch];
};

// ---- PTX wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when it gave up or when another role already raised the abort flag.
// After a few immediate retries the waiter sleeps `sleep_ns` between polls so that it does not take
// issue slots from the warps it is waiting for.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag,
                                          uint32_t sleep_ns = 32)
{
    for (uint32_t i = 0; i < kWaitLimit; ++i) {
        if (mbar_try(bar, parity)) return true;
        if (i >= 4) {
            if (*abort_flag) return false;
            if (sleep_ns) __nanosleep(sleep_ns);
        }
    }
    *abort_flag = 1;
    return false;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint32_t bar, int c0, int c1, int c2)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tc_mma_tf32(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// same with the A operand read from tensor memory (lane = row, one 32-bit column per k)
__device__ __forceinline__ void tc_mma_tf32_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// the same two with "accumulate" fixed to true (no predicate to compute in the issuing thread)
__device__ __forceinline__ void tc_mma_tf32_acc(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.eq.u32 p, 1, 1;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc)
        : "memory");
}
__device__ __forceinline__ void tc_mma_tf32_ts_acc(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.eq.u32 p, 1, 1;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc)
        : "memory");
}
// the same with bf16 operands (two k per 32-bit column of the A block in tensor memory, 16 k per instruction)
__device__ __forceinline__ void tc_mma_bf16_ts_acc(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.eq.u32 p, 1, 1;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc)
        : "memory");
}
// 32 lanes x 8 columns
__device__ __forceinline__ void tc_st_32x8(uint32_t taddr, const uint32_t (&r)[8])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
        : "memory");
}
// two consecutive k as one 32-bit word of bf16 (round to nearest even): k in the low half, k + 1 in the high half
__device__ __forceinline__ uint32_t pack_bf16(float k0, float k1)
{
    const __nv_bfloat162 v = __floats2bfloat162_rn(k0, k1);
    return *reinterpret_cast<const uint32_t *>(&v);
}
// 32 lanes x 16 columns: each thread stores 16 registers into its lane's row
__device__ __forceinline__ void tc_st_32x16(uint32_t taddr, const uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// 32 lanes x 32 columns of 32-bit accumulators -> 32 registers per thread (thread = lane = row)
__device__ __forceinline__ void tc_ld_32x32(uint32_t taddr, uint32_t (&r)[32])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// fp32 -> tf32 (10 explicit mantissa bits), round to nearest with ties away from zero, as the integer
// form of cvt.rna.tf32.f32: add half a tf32 ulp to the bit pattern and clear the 13 low bits.
__device__ __forceinline__ uint32_t to_tf32(float x) { return (__float_as_uint(x) + 0x1000u) & 0xFFFFE000u; }

// Shared-memory matrix descriptor (sm_100 format): start address, leading / stride byte offsets
// (all >> 4), descriptor version 1, swizzle mode (2: 128-byte swizzle of 16-byte units, the K-major
// form; 1: 128-byte swizzle of 32-byte units, the only form tf32 operands may use MN-major).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes, uint32_t layout)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFFu);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
    d |= 1ull << 46;            // version
    d |= (uint64_t)layout << 61;
    return d;
}

// Instruction descriptor: D fp32, A and B tf32, given major-ness, M = 128, N = n (multiple of 16).
__host__ __device__ constexpr uint32_t instr_desc(int major, int n, int m = kBM)
{
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)major << 15) | ((uint32_t)major << 16) |
           ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// The same for bf16 operands (both K-major), used for the two cross terms of the bf16-cross form.
__host__ __device__ constexpr uint32_t instr_desc_bf16(int n, int m = kBM)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

// One 16-byte chunk (4 consecutive k of one row) of a K-major 128-byte-swizzled tile.
__device__ __forceinline__ uint32_t chunk_offset(int row, int kq) { return (uint32_t)row * 128u + (uint32_t)((kq ^ (row & 7)) << 4); }

// kSquare = false: the values themselves are split (per-example form: the products are summed over the positions of
// an example first and squared afterwards), hi + lo = v with either sign
template <bool kSquare = true>
__device__ __forceinline__ void split_store(uint8_t *hi_tile, uint8_t *lo_tile, uint32_t off, float v0, float v1, float v2, float v3)
{
    const float q0 = kSquare ? __fmul_rn(v0, v0) : v0, q1 = kSquare ? __fmul_rn(v1, v1) : v1;
    const float q2 = kSquare ? __fmul_rn(v2, v2) : v2, q3 = kSquare ? __fmul_rn(v3, v3) : v3;
    uint4 h, l;
    h.x = to_tf32(q0); h.y = to_tf32(q1); h.z = to_tf32(q2); h.w = to_tf32(q3);
    // lo = q - hi is exact in fp32; the tensor core reads only its upper 19 bits, an error of at most
    // 2^-10 * |lo| <= 2^-22 * q whose sign follows lo (no systematic bias)
    l.x = __float_as_uint(__fsub_rn(q0, __uint_as_float(h.x)));
    l.y = __float_as_uint(__fsub_rn(q1, __uint_as_float(h.y)));
    l.z = __float_as_uint(__fsub_rn(q2, __uint_as_float(h.z)));
    l.w = __float_as_uint(__fsub_rn(q3, __uint_as_float(h.w)));
    *reinterpret_cast<uint4 *>(hi_tile + off) = h;
    *reinterpret_cast<uint4 *>(lo_tile + off) = l;
}

constexpr int kRowsPerThread = kBM * 8 / kGatherThreads;        // 4 gathered chunks per thread per tile

// The four rows (row0 + 32*i) of a gathered tile that one transform thread owns.
template <int kMode>
struct GatherRows {
    int base[kRowsPerThread], dh[kRowsPerThread], dw[kRowsPerThread];
    bool ok[kRowsPerThread];
    const float *src;       // x (im2col rows) or delta (error rows) of this block's layer

    __device__ __forceinline__ void init(const Params &prm, const float *x, const float *delta, int first_row, int limit)
    {
        if (kMode == kTma) return;
        src = kMode == kGatherIm2col ? x : delta;
        const int khw = prm.Kh * prm.Kw;
#pragma unroll
        for (int i = 0; i < kRowsPerThread; ++i) {
            const int idx = first_row + 32 * i;
            ok[i] = idx < limit;
            const int ii = ok[i] ? idx : 0;
            if (kMode == kGatherIm2col) {
                const int c = ii / khw, rem = ii - c * khw;
                const int kh = rem / prm.Kw, kw = rem - kh * prm.Kw;
                dh[i] = kh - prm.ph;
                dw[i] = kw - prm.pw;
                base[i] = (c * prm.H + dh[i]) * prm.W + dw[i];
            } else {
                base[i] = ii * prm.P;   // offset of the output channel's plane
                dh[i] = dw[i] = 0;
            }
        }
    }
    // loads this thread's 4 rows x 4 consecutive k: example z, output positions pbase .. pbase+3
    __device__ __forceinline__ void load(const Params &prm, int z, int pbase, float (&v)[kRowsPerThread][4]) const
    {
        if (kMode == kGatherIm2col) {
            const float *xz = src + (size_t)z * prm.chw;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int p = pbase + j;
                const int ho = prm.Wo == 1 ? p : (int)__umulhi((unsigned)p, prm.wo_magic), wo = p - ho * prm.Wo;
                const int hs = ho * prm.sh, ws = wo * prm.sw;
                const float *xp = xz + (hs * prm.W + ws);
                const bool pv = p < prm.P;
#pragma unroll
                for (int i = 0; i < kRowsPerThread; ++i) {
                    const bool in = pv && ok[i] && (unsigned)(hs + dh[i]) < (unsigned)prm.H &&
                                    (unsigned)(ws + dw[i]) < (unsigned)prm.W;
                    v[i][j] = in ? __ldg(xp + base[i]) : 0.f;
                }
            }
        } else if (kMode == kGatherErr) {
            const float *dz = src + (size_t)z * prm.Cout * prm.P + pbase;
#pragma unroll
            for (int i = 0; i < kRowsPerThread; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) v[i][j] = (ok[i] && pbase + j < prm.P) ? __ldg(dz + (base[i] + j)) : 0.f;
        }
    }
};

// Kw = 3, stride 1, pad_w = 1: the three rows (c, kh, kw = 0..2) of the im2col view read the same input row
// shifted by one, so a thread takes whole triples: for 4 (or 2 + 2) consecutive output positions it loads
// the input row segment once -- one aligned vector and its two neighbours -- and feeds all three rows from
// it.  A thread owns the triples first_triple + grp + 32*i (i = 0, 1) of the tile's rows; triples that
// straddle the tile's first or last row are handled by the row test at store time.
// kTriples = 2: 256 threads share a slice (triples grp + 32 i); kTriples = 3: 128 threads do (grp + 16 i).
template <int kSpan, int kTriples>      // kSpan: output positions covered by one aligned vector load, 4 or 2
struct GatherTaps {
    static constexpr int kStride = kTriples == 2 ? 32 : 16;
    static constexpr int kKw = 3;
    static constexpr int kSlots = 8;                         // registers per triple
    static constexpr int kLoaded = kSpan == 4 ? 6 : 8;       // of which loaded
    // register that holds the input of tap kw for the j-th of the thread's four output positions
    __device__ __forceinline__ static constexpr int idx(int kw, int j) { return kSpan == 4 ? kw + j : (j >> 1) * 4 + (j & 1) + kw; }
    int base[kTriples], dh[kTriples], row_local[kTriples];
    bool ok[kTriples];
    const float *src;

    __device__ __forceinline__ void init(const Params &prm, const float *x, int tile_origin, int grp, int limit)
    {
        src = x;
        const int first_triple = tile_origin / 3;
#pragma unroll
        for (int i = 0; i < kTriples; ++i) {
            const int T = first_triple + grp + kStride * i;          // triple = (c, kh)
            ok[i] = 3 * T < limit;
            const int tt = ok[i] ? T : 0;
            const int c = tt / prm.Kh, kh = tt - c * prm.Kh;
            dh[i] = kh - prm.ph;
            base[i] = (c * prm.H + dh[i]) * prm.W;
            row_local[i] = 3 * T - tile_origin;                      // tile row of the kw = 0 tap (may be -2, -1)
        }
    }
    // v[i][0..7]: kSpan = 4: {left, m0, m1, m2, m3, right, -, -} for positions pbase..pbase+3;
    //             kSpan = 2: {left, m0, m1, right} for pbase, pbase+1 and the same for pbase+2, pbase+3
    __device__ __forceinline__ void load(const Params &prm, int z, int pbase, float (&v)[kTriples][8]) const
    {
        const float *xz = src + (size_t)z * prm.chw;
#pragma unroll
        for (int s = 0; s < 4 / kSpan; ++s) {
            const int p = pbase + s * kSpan;
            const int ho = (int)__umulhi((unsigned)p, prm.wo_magic), wo = p - ho * prm.Wo;
            const bool pv = p < prm.P;
            const float *xp = xz + (ho * prm.W + wo);
#pragma unroll
            for (int i = 0; i < kTriples; ++i) {
                const bool in = pv && ok[i] && (unsigned)(ho + dh[i]) < (unsigned)prm.H;
                const float *q = xp + base[i];
                float *o = &v[i][s * 4];
                if (kSpan == 4) {
                    const float4 m = in ? __ldg(reinterpret_cast<const float4 *>(q)) : make_float4(0.f, 0.f, 0.f, 0.f);
                    o[0] = (in && wo > 0) ? __ldg(q - 1) : 0.f;
                    o[1] = m.x; o[2] = m.y; o[3] = m.z; o[4] = m.w;
                    o[5] = (in && wo + 4 < prm.W) ? __ldg(q + 4) : 0.f;
                } else {
                    const float2 m = in ? __ldg(reinterpret_cast<const float2 *>(q)) : make_float2(0.f, 0.f);
                    o[0] = (in && wo > 0) ? __ldg(q - 1) : 0.f;
                    o[1] = m.x; o[2] = m.y;
                    o[3] = (in && wo + 2 < prm.W) ? __ldg(q + 2) : 0.f;
                }
            }
        }
    }
    // the four k of tap kw of triple i
    __device__ __forceinline__ static void tap(const float (&v)[kTriples][8], int i, int kw, float (&out)[4])
    {
        if (kSpan == 4) {
            out[0] = v[i][kw]; out[1] = v[i][kw + 1]; out[2] = v[i][kw + 2]; out[3] = v[i][kw + 3];
        } else {
            out[0] = v[i][kw]; out[1] = v[i][kw + 1]; out[2] = v[i][4 + kw]; out[3] = v[i][4 + kw + 1];
        }
    }
};

// Stride 2 along w with Kw = 3, pad_w = 1 and W == 2 Wo: the 4 (or 2) output positions of a span read the input
// columns 2 wo - 1 .. 2 wo + 7 (or + 3): one neighbour on the left and two (one) aligned 4-vectors, never past the
// row's end.  Tap kw of output j is element 2 j + kw of that segment.
template <int kSpan, int kTriples>
struct GatherTapsS2 {
    static constexpr int kStride = kTriples == 2 ? 32 : 16;
    static constexpr int kPerSpan = kSpan == 4 ? 9 : 5;
    static constexpr int kKw = 3;
    static constexpr int kSlots = 10;
    static constexpr int kLoaded = kSpan == 4 ? 9 : 10;
    __device__ __forceinline__ static constexpr int idx(int kw, int j)
    {
        return kSpan == 4 ? 2 * j + kw : (j >> 1) * 5 + 2 * (j & 1) + kw;
    }
    int base[kTriples], dh[kTriples], row_local[kTriples];
    bool ok[kTriples];
    const float *src;

    __device__ __forceinline__ void init(const Params &prm, const float *x, int tile_origin, int grp, int limit)
    {
        src = x;
        const int first_triple = tile_origin / 3;
#pragma unroll
        for (int i = 0; i < kTriples; ++i) {
            const int T = first_triple + grp + kStride * i;          // triple = (c, kh)
            ok[i] = 3 * T < limit;
            const int tt = ok[i] ? T : 0;
            const int c = tt / prm.Kh, kh = tt - c * prm.Kh;
            dh[i] = kh - prm.ph;
            base[i] = (c * prm.H + dh[i]) * prm.W;
            row_local[i] = 3 * T - tile_origin;
        }
    }
    __device__ __forceinline__ void load(const Params &prm, int z, int pbase, float (&v)[kTriples][kSlots]) const
    {
        const float *xz = src + (size_t)z * prm.chw;
#pragma unroll
        for (int s = 0; s < 4 / kSpan; ++s) {
            const int p = pbase + s * kSpan;
            const int ho = (int)__umulhi((unsigned)p, prm.wo_magic), wo = p - ho * prm.Wo;
            const bool pv = p < prm.P;
            const int hs = ho * prm.sh;
            const float *xp = xz + (hs * prm.W + 2 * wo);
#pragma unroll
            for (int i = 0; i < kTriples; ++i) {
                const bool in = pv && ok[i] && (unsigned)(hs + dh[i]) < (unsigned)prm.H;
                const float *q = xp + base[i];
                float *o = &v[i][s * kPerSpan];
                const float4 zero = make_float4(0.f, 0.f, 0.f, 0.f);
                const float4 m0 = in ? __ldg(reinterpret_cast<const float4 *>(q)) : zero;
                o[0] = (in && wo > 0) ? __ldg(q - 1) : 0.f;
                o[1] = m0.x; o[2] = m0.y; o[3] = m0.z; o[4] = m0.w;
                if (kSpan == 4) {
                    const float4 m1 = in ? __ldg(reinterpret_cast<const float4 *>(q) + 1) : zero;
                    o[5] = m1.x; o[6] = m1.y; o[7] = m1.z; o[8] = m1.w;
                }
            }
        }
    }
};

// Kw = 7, stride 2, pad_w = 3, W == 2 Wo, Wo a multiple of 4: the seven rows (c, kh, kw = 0..6) read, for four
// consecutive output positions, the input columns 2 wo - 3 .. 2 wo + 9.  Four aligned 4-vectors from column 2 wo - 4
// on cover them (each wholly inside or wholly outside the row); tap kw of output j is element 1 + 2 j + kw.
// 128 threads share a slice; a thread owns the tuples first_tuple + grp + 16 i, i = 0, 1 (at most 20 touch a tile).
template <int kTuples>
struct GatherTaps7S2 {
    static_assert(kTuples == 2, "used by the two-group form only");
    static constexpr int kStride = 16;
    static constexpr int kKw = 7;
    static constexpr int kSlots = 16;
    static constexpr int kLoaded = 14;
    __device__ __forceinline__ static constexpr int idx(int kw, int j) { return 1 + 2 * j + kw; }
    int base[kTuples], dh[kTuples], row_local[kTuples];
    bool ok[kTuples];
    const float *src;

    __device__ __forceinline__ void init(const Params &prm, const float *x, int tile_origin, int grp, int limit)
    {
        src = x;
        const int first_tuple = tile_origin / 7;
#pragma unroll
        for (int i = 0; i < kTuples; ++i) {
            const int T = first_tuple + grp + kStride * i;           // tuple = (c, kh)
            ok[i] = 7 * T < limit;
            const int tt = ok[i] ? T : 0;
            const int c = tt / prm.Kh, kh = tt - c * prm.Kh;
            dh[i] = kh - prm.ph;
            base[i] = (c * prm.H + dh[i]) * prm.W;
            row_local[i] = 7 * T - tile_origin;
        }
    }
    __device__ __forceinline__ void load(const Params &prm, int z, int pbase, float (&v)[kTuples][kSlots]) const
    {
        const int ho = (int)__umulhi((unsigned)pbase, prm.wo_magic), wo = pbase - ho * prm.Wo;
        const int hs = ho * prm.sh;
        const bool pv = pbase < prm.P;
        const float *xp = src + (size_t)z * prm.chw + (hs * prm.W + 2 * wo - 4);
        const int col0 = 2 * wo - 4;
#pragma unroll
        for (int i = 0; i < kTuples; ++i) {
            const bool in = pv && ok[i] && (unsigned)(hs + dh[i]) < (unsigned)prm.H;
            const float4 *q = reinterpret_cast<const float4 *>(xp + base[i]);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const bool inside = in && (unsigned)(col0 + 4 * u) < (unsigned)prm.W;
                const float4 m = inside ? __ldg(q + u) : make_float4(0.f, 0.f, 0.f, 0.f);
                v[i][4 * u] = m.x; v[i][4 * u + 1] = m.y; v[i][4 * u + 2] = m.z; v[i][4 * u + 3] = m.w;
            }
        }
    }
};

template <int kMode> struct IsTaps {
    static constexpr bool value = kMode == kGatherTaps4 || kMode == kGatherTaps2 || kMode == kGatherTaps4S2 ||
                                  kMode == kGatherTaps2S2 || kMode == kGatherTaps7S2;
};
template <int kMode, int kTriples> struct TapsOf { typedef GatherTaps<kMode == kGatherTaps4 ? 4 : 2, kTriples> type; };
template <int kTriples> struct TapsOf<kGatherTaps4S2, kTriples> { typedef GatherTapsS2<4, kTriples> type; };
template <int kTriples> struct TapsOf<kGatherTaps2S2, kTriples> { typedef GatherTapsS2<2, kTriples> type; };
template <int kTriples> struct TapsOf<kGatherTaps7S2, kTriples> { typedef GatherTaps7S2<2> type; };

// One interface over both gather forms: the registers of one slice, how they are loaded and where their
// squared, split values go in a K-major swizzled tile.  row0 = t >> 3 and kq = t & 7 of transform thread t.
// kHalf: the slice is shared by 128 threads instead of 256 (two transform groups on alternate slices)
template <int kMode, bool kHalf = false, bool kTaps = IsTaps<kMode>::value>
struct Gatherer {
    struct Regs { float v[kRowsPerThread][4]; };
    GatherRows<kMode> g;
    __device__ __forceinline__ void init(const Params &prm, const float *x, const float *delta, int origin, int row0, int limit)
    {
        g.init(prm, x, delta, origin + row0, limit);
    }
    __device__ __forceinline__ void load(const Params &prm, int z, int pbase, Regs &r) const { g.load(prm, z, pbase, r.v); }
    template <bool kSquare>
    __device__ __forceinline__ void store(uint8_t *hi, uint8_t *lo, int row0, int kq, const Regs &r) const
    {
#pragma unroll
        for (int i = 0; i < kRowsPerThread; ++i)
            split_store<kSquare>(hi, lo, chunk_offset(row0 + 32 * i, kq), r.v[i][0], r.v[i][1], r.v[i][2], r.v[i][3]);
    }
};
template <int kMode, bool kHalf>
struct Gatherer<kMode, kHalf, true> {
    static constexpr int kTriples = kMode == kGatherTaps7S2 ? 2 : kHalf ? 3 : 2;      // tuples of rows per thread
    typedef typename TapsOf<kMode, kTriples>::type Impl;
    struct Regs { float v[kTriples][Impl::kSlots]; };
    Impl g;
    __device__ __forceinline__ void init(const Params &prm, const float *x, const float *, int origin, int row0, int limit)
    {
        g.init(prm, x, origin, row0, limit);
    }
    __device__ __forceinline__ void load(const Params &prm, int z, int pbase, Regs &r) const { g.load(prm, z, pbase, r.v); }
    template <bool kSquare>
    __device__ __forceinline__ void store(uint8_t *hi, uint8_t *lo, int, int kq, const Regs &r) const
    {
#pragma unroll
        for (int i = 0; i < kTriples; ++i) {
            if (g.row_local[i] >= kBM || g.row_local[i] <= -Impl::kKw) continue;   // no row of this tuple in the tile
            // square and split every loaded element once; the three taps are views of the same parts
            uint32_t h[Impl::kSlots], l[Impl::kSlots];
#pragma unroll
            for (int e = 0; e < Impl::kLoaded; ++e) {
                const float q = kSquare ? __fmul_rn(r.v[i][e], r.v[i][e]) : r.v[i][e];
                h[e] = to_tf32(q);
                l[e] = __float_as_uint(__fsub_rn(q, __uint_as_float(h[e])));
            }
#pragma unroll
            for (int kw = 0; kw < Impl::kKw; ++kw) {
                const int row = g.row_local[i] + kw;
                if ((unsigned)row < (unsigned)kBM) {                 // kBM == kBN rows in either tile
                    const uint32_t off = chunk_offset(row, kq);
                    *reinterpret_cast<uint4 *>(hi + off) =
                        make_uint4(h[Impl::idx(kw, 0)], h[Impl::idx(kw, 1)], h[Impl::idx(kw, 2)], h[Impl::idx(kw, 3)]);
                    *reinterpret_cast<uint4 *>(lo + off) =
                        make_uint4(l[Impl::idx(kw, 0)], l[Impl::idx(kw, 1)], l[Impl::idx(kw, 2)], l[Impl::idx(kw, 3)]);
                }
            }
        }
    }
};

// ---- work distribution -----------------------------------------------------------------------
// One segment of a block's range: slices [s_begin, s_end) of the reduction of one output tile.
struct Seg {
    int layer, m0, n0;       // layer of the batch, first row / column of the tile
    int n_valid, n_act;      // columns of the tile that exist; the MMAs' N (rounded up to a multiple of 16)
    int s_begin, s_end;
    bool whole;              // the segment is the tile's whole reduction: its block writes the result itself
    int slot;                // otherwise: which partial tile of the scratch it writes
};

// The launch's work is the sequence (layer, tile, unit of the tile's reduction), units_total long; block b owns
// units [b U / G, (b + 1) U / G).  Every role of a block walks the same segments with an iterator of its own.
struct SegIter {
    int pos, end;
    int index;
    __device__ __forceinline__ SegIter(const Params &prm)
    {
        const int b = (int)blockIdx.x;
        pos = b * prm.units_q + min(b, prm.units_r);
        end = pos + prm.units_q + (b < prm.units_r ? 1 : 0);
        index = 0;
    }
    __device__ __forceinline__ bool next(const Params &prm, Seg &sg)
    {
        if (pos >= end) return false;
        const int upt = prm.units_per_tile;
        const int tile = pos / upt;
        const int u0 = pos - tile * upt;
        const int u1 = min(end - tile * upt, upt);
        const int tiles_layer = prm.tiles_x * prm.tiles_y;
        sg.layer = tile / tiles_layer;
        const int rem = tile - sg.layer * tiles_layer;
        const int tile_m = rem / prm.tiles_x, tile_n = rem - tile_m * prm.tiles_x;
        sg.m0 = tile_m * kBM;
        sg.n0 = tile_n * kBN;
        sg.n_valid = min(kBN, prm.N - sg.n0);
        sg.n_act = (sg.n_valid + 15) & ~15;
        sg.s_begin = u0 * prm.unit;
        sg.s_end = u1 * prm.unit;
        sg.whole = u0 == 0 && u1 == upt;
        sg.slot = 2 * (int)blockIdx.x + (index > 0 ? 1 : 0);     // a block's partial segments: its first and / or its last
        pos += u1 - u0;
        ++index;
        return true;
    }
};

// ---- the kernel ------------------------------------------------------------------------------
// kExact: the per-example statistic of a conv layer, S = scale * sum_z (sum_p delta x)^2 -- operands are split without
// squaring, an accumulator is drained at least at every example's end, the epilogue sums the drains of one example
// in registers and adds the square of that sum into a third accumulator kept in tensor memory.
// kBf: the two cross terms hi*lo and lo*hi are taken with bf16 operands (half the shared-memory reads and half the
// tensor-pipe time of a tf32 product each; their rounding, 2^-9 relative on a term that is itself 2^-11 of the
// product, stays below 2^-18 of the result).  A lo slot then holds [B hi as bf16][B lo as bf16], 8 KB each with
// 64-byte rows, and an A slot in tensor memory [hi tf32: 32 columns][hi bf16: 16][lo bf16: 16].
template <int kMajor, int kModeA, int kModeB, bool kATmem, bool kExact = false, bool kBf = false>
__global__ void __launch_bounds__(kThreadsTc, 1)
sqgrad_tc(const __grid_constant__ Batch bt, const Params prm)
{
    static_assert(kMajor == kMajorK || (kModeA == kTma && kModeB == kTma), "gathered tiles are K-major");
    static_assert(!kATmem || (kMajor == kMajorK && kModeA == kTma), "A goes to tensor memory from a K-major TMA tile");
    constexpr bool kGatherA = kModeA != kTma, kGatherB = kModeB != kTma;
    constexpr bool kAnyTma = !kGatherA || !kGatherB;
    constexpr bool kAnyGather = kGatherA || kGatherB;
    constexpr bool kSplit = kATmem && !kAnyGather;                         // A raw tiles in a ring of their own
    static_assert(!kBf || (kSplit && !kExact), "bf16 cross terms: the TMA-fed form with A in tensor memory");
    constexpr int kNA = kSplitA;                                           // slots of the raw A ring (split form)
    // the transform warps work as two groups of four on alternate slices (else all eight on every slice)
    constexpr bool kTwoGroups = !kAnyGather || (IsTaps<kModeB>::value && kModeA == kTma);
    constexpr int kNB = kSplit ? kSplitB : kRawSlots;                      // slots of the raw / hi ring
    // lo slots (and A slots in TMEM); the per-example form needs 128 TMEM columns for its sum of squares
    constexpr int kLoN = (kExact && kATmem) ? 2 : kSplit ? kSplitLo : (kATmem ? kLoSlotsAT : kLoSlots);
    constexpr uint32_t kSqCol = 2 * kBN + (kATmem ? 2 * kTmemColsA : 0);         // where that sum lives
    constexpr uint32_t kLoBytes = kATmem ? kRawBytesB : kRawStageBytes;  // bytes of one lo slot
    // byte offsets of slot s: the [A][B] pair of the raw / hi ring (split form: only its B half exists, the
    // offset points one A tile below it), the lo ring likewise, and the split form's A ring
    auto pair_off = [](int s) -> uint32_t { return kSplit ? (uint32_t)(kSplitA + s - 1) * kRawBytesA : (uint32_t)s * kRawStageBytes; };
    auto lo_off = [](int s) -> uint32_t {
        return kSplit ? (uint32_t)(kSplitA + kSplitB + s - 1) * kRawBytesA
                      : kLoBase + (uint32_t)s * kLoBytes - (kATmem ? kRawBytesA : 0u);
    };
    // bf16-cross form: where the B tile of raw slot s and the [hi bf16][lo bf16] tiles of lo slot s live
    auto b_tile = [&](int s) -> uint32_t { return pair_off(s) + kRawBytesA; };
    auto bf_tile = [&](int s) -> uint32_t { return lo_off(s) + kRawBytesA; };
    constexpr uint32_t kBTile = kRawBytesB;

    extern __shared__ uint8_t smem_raw_[];
    __shared__ __align__(8) uint64_t bars[3 * kSplitB + kLoSlotsAT + 5 + 2 * kSplitA];
    __shared__ uint32_t tmem_base_slot;
    __shared__ volatile uint32_t abort_flag;

    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (smem_u32(smem_raw_) + 1023u) & ~1023u;     // 1024-byte aligned tiles
    uint8_t *smem_gen = smem_raw_ + (smem_base - smem_u32(smem_raw_));

    // per raw slot: raw_full (TMA landed) -> op_full (hi/lo written) -> empty (MMAs that read it retired);
    // a lo slot (and its A slot in tensor memory) is free when the MMAs of the slice that used it last have
    // retired, which is what that slice's `empty` barrier says: no barrier of its own, one commit per slice
    uint64_t *raw_full = bars, *op_full = bars + kNB, *empty = bars + 2 * kNB;
    uint64_t *lo_empty = bars + 3 * kNB;
    uint64_t *acc_full = lo_empty + kLoSlotsAT, *acc_empty = acc_full + 2, *drain = acc_empty + 2;
    uint64_t *a_full = drain + 1, *a_empty = a_full + kNA;                 // split form: the A ring

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int i = 0; i < kNB; ++i) {
            mbar_init(smem_u32(&raw_full[i]), 1);
            mbar_init(smem_u32(&op_full[i]), kTwoGroups ? 4 : kGatherThreads / 32);
            mbar_init(smem_u32(&empty[i]), 1);
        }
        if (kSplit)
            for (int i = 0; i < kNA; ++i) {
                mbar_init(smem_u32(&a_full[i]), 1);
                mbar_init(smem_u32(&a_empty[i]), 4);
            }
        for (int i = 0; i < kLoSlotsAT; ++i) mbar_init(smem_u32(&lo_empty[i]), 1);      // unused, kept initialised
        for (int i = 0; i < 2; ++i) { mbar_init(smem_u32(&acc_full[i]), 1); mbar_init(smem_u32(&acc_empty[i]), kEpilogueWarps); }
        mbar_init(smem_u32(drain), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {      // TMEM: this warp allocates and, at the end, frees
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_slot;

    // `it` below is the running number of a slice within this block (over all of its segments): ring slots and
    // barrier phases follow it, so the pipeline does not drain between segments.
    if (warp == 0) {
        // ================= TMA producer (one thread) =================
        if (lane == 0 && kAnyTma) {
            int it = 0;
            bool ok = true;
            SegIter iter(prm);
            Seg sg;
            while (ok && iter.next(prm, sg)) {
                const CUtensorMap *map_a = &bt.a[sg.layer], *map_b = &bt.b[sg.layer];
                const int m0 = sg.m0, n0 = sg.n0;
                for (int slice = sg.s_begin; slice < sg.s_end; ++slice, ++it) {
                    const int st = it % kNB;
                    const uint32_t ph = (uint32_t)(it / kNB) & 1u;
                    if (!mbar_wait(smem_u32(&empty[st]), ph ^ 1u, &abort_flag, 64)) { ok = false; break; }
                    const uint32_t full = smem_u32(&raw_full[st]);
                    const uint32_t dst_a = smem_base + pair_off(st), dst_b = dst_a + kRawBytesA;
                    if (kSplit) {
                        const int sa = it % kNA;
                        if (!mbar_wait(smem_u32(&a_empty[sa]), ((uint32_t)(it / kNA) & 1u) ^ 1u, &abort_flag, 64)) { ok = false; break; }
                        const uint32_t full_a = smem_u32(&a_full[sa]);
                        const int z = slice / prm.p_slices, p0 = (slice - z * prm.p_slices) * kBK;
                        mbar_expect_tx(full_a, prm.tx_bytes_a);
                        tma_load_3d(smem_base + (uint32_t)sa * kRawBytesA, map_a, full_a, p0, m0, z);
                        mbar_expect_tx(full, prm.tx_bytes - prm.tx_bytes_a);
                        if (kBf) tma_load_3d(smem_base + b_tile(st), map_b, full, p0, n0, z);
                        else tma_load_3d(dst_b, map_b, full, p0, n0, z);
                        continue;
                    }
                    mbar_expect_tx(full, prm.tx_bytes);
                    if (kMajor == kMajorK) {
                        const int z = slice / prm.p_slices, p0 = (slice - z * prm.p_slices) * kBK;
                        if (!kGatherA) tma_load_3d(dst_a, map_a, full, p0, m0, z);
                        if (!kGatherB) tma_load_3d(dst_b, map_b, full, p0, n0, z);
                    } else {
                        const int k0 = slice * kBK;
#pragma unroll
                        for (int j = 0; j < kBM / 32; ++j) tma_load_2d(dst_a + j * 4096, map_a, full, m0 + 32 * j, k0);
#pragma unroll
                        for (int j = 0; j < kBN / 32; ++j) tma_load_2d(dst_b + j * 4096, map_b, full, n0 + 32 * j, k0);
                    }
                }
            }
            // on an abort: loads already issued (slices 0 .. it-1) must land before the block may exit
            if (abort_flag) {
                const int issued = it;
                const int first = issued > kNB ? issued - kNB : 0;
                for (int i = first; i < issued; ++i) {
                    const uint32_t bar = smem_u32(&raw_full[i % kNB]);
                    const uint32_t ph = (uint32_t)(i / kNB) & 1u;
                    for (uint32_t t = 0; t < kWaitLimit && !mbar_try(bar, ph); ++t) {}
                }
                if (kSplit) {
                    const int first_a = issued > kNA ? issued - kNA : 0;
                    for (int i = first_a; i < issued; ++i) {
                        const uint32_t bar = smem_u32(&a_full[i % kNA]);
                        const uint32_t ph = (uint32_t)(i / kNA) & 1u;
                        for (uint32_t t = 0; t < kWaitLimit && !mbar_try(bar, ph); ++t) {}
                    }
                }
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer (one thread) =================
        if (lane == 0) {
            // K-major: rows of 128 B, 8-row groups 1024 B apart (SBO); LBO unused.
            // MN-major: 32-wide column blocks 4096 B apart (LBO); 4-deep k groups 512 B apart (SBO).
            const uint32_t lbo = kMajor == kMajorK ? 16u : 4096u;
            const uint32_t sbo = kMajor == kMajorK ? 1024u : 512u;
            const uint32_t layout = kMajor == kMajorK ? 2u : 1u;
            constexpr uint32_t k_step16 = (kMajor == kMajorK ? 32u : 1024u) >> 4;   // 16-byte units per 8-deep MMA step
            // This one thread feeds the tensor pipe, so its instruction stream is kept short: the descriptor's
            // upper word and the LBO field never change, the start-address field (address >> 4; shared memory
            // is < 256 KB, so it cannot overflow its 14 bits) is one addition per operand and step.
            const uint32_t desc_hi = (uint32_t)(smem_desc(0, lbo, sbo, layout) >> 32);
            const uint32_t desc_lo0 = (uint32_t)smem_desc(0, lbo, sbo, layout);
            auto desc_at = [&](uint32_t lo16) -> uint64_t { return ((uint64_t)desc_hi << 32) | (desc_lo0 + lo16); };
            // bf16 tiles: K-major rows of 64 B with the 64-byte swizzle (mode 4), 8-row groups 512 B apart
            const uint32_t desc_bf_hi = (uint32_t)(smem_desc(0, 16u, 512u, 4u) >> 32);
            const uint32_t desc_bf_lo0 = (uint32_t)smem_desc(0, 16u, 512u, 4u);
            auto desc_bf = [&](uint32_t lo16) -> uint64_t { return ((uint64_t)desc_bf_hi << 32) | (desc_bf_lo0 + lo16); };
            int st = 0, ls = 0;                          // the current slice's raw / hi slot and lo slot
            uint32_t st_phase = 0;
            int c = 0;                                   // running number of the chunk (accumulator buffer c & 1)
            bool ok = true;
            SegIter iter(prm);
            Seg sg;
            while (ok && iter.next(prm, sg)) {
                const uint32_t idesc = instr_desc(kMajor, sg.n_act, kBM);
                const uint32_t idesc_bf = instr_desc_bf16(sg.n_act, kBM);
                // an accumulator is drained every prm.chunk slices, and (kExact) at the end of every example: the
                // segment's slices are runs of seg_len slices (whole examples -- the work is cut that way), each cut
                // into cps chunks
                const int n_slices = sg.s_end - sg.s_begin;
                const int seg_len = kExact ? prm.p_slices : n_slices;
                const int cps = (seg_len + prm.chunk - 1) / prm.chunk;
                const int n_chunks = (n_slices / seg_len) * cps;
                int i = 0;                               // slice within the segment
                for (int cc = 0; cc < n_chunks && ok; ++cc, ++c) {
                    const int b = c & 1;
                    ok = mbar_wait(smem_u32(&acc_empty[b]), ((uint32_t)(c >> 1) & 1u) ^ 1u, &abort_flag, 0);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t d_tmem = tmem_base + (uint32_t)b * kBN;
                    const int run = cc / cps, cq = cc - run * cps;              // run (example) and chunk inside it
                    const int chunk_end = run * seg_len + min(seg_len, (cq + 1) * prm.chunk);
                    for (bool first = true; i < chunk_end; ++i) {
                        ok = mbar_wait(smem_u32(&op_full[st]), st_phase, &abort_flag, 0);
                        if (!ok) break;
                        tc_fence_after();
                        const uint32_t hi_a16 = (smem_base + pair_off(st)) >> 4, hi_b16 = hi_a16 + (kRawBytesA >> 4);
                        const uint32_t lo_a16 = (smem_base + lo_off(ls)) >> 4, lo_b16 = lo_a16 + (kRawBytesA >> 4);   // lo_a unused with A in TMEM
                        const uint32_t ta_hi = tmem_base + 2 * kBN + ls * kTmemColsA, ta_lo = ta_hi + 32;
                        if (kBf) {
                            const uint32_t b16 = (smem_base + b_tile(st)) >> 4;
#pragma unroll
                            for (int kk = 0; kk < kBK / 8; ++kk) {
                                const uint64_t db_hi = desc_at(b16 + kk * k_step16);
                                if (kk == 0) tc_mma_tf32_ts(d_tmem, ta_hi, db_hi, idesc, first ? 0u : 1u);
                                else tc_mma_tf32_ts_acc(d_tmem, ta_hi + kk * 8, db_hi, idesc);
                            }
                            // cross terms, 16 k (32 bytes of a 64-byte row, 8 columns of tensor memory) per instruction
                            const uint32_t bf_hi16 = (smem_base + bf_tile(ls)) >> 4, bf_lo16 = bf_hi16 + (kBTile >> 5);
#pragma unroll
                            for (int kk = 0; kk < kBK / 16; ++kk) {
                                tc_mma_bf16_ts_acc(d_tmem, ta_hi + 32 + kk * 8, desc_bf(bf_lo16 + kk * 2), idesc_bf);
                                tc_mma_bf16_ts_acc(d_tmem, ta_hi + 48 + kk * 8, desc_bf(bf_hi16 + kk * 2), idesc_bf);
                            }
                        } else
#pragma unroll
                        for (int kk = 0; kk < kBK / 8; ++kk) {
                            const uint64_t db_hi = desc_at(hi_b16 + kk * k_step16);
                            const uint64_t db_lo = desc_at(lo_b16 + kk * k_step16);
                            if (kATmem) {
                                if (kk == 0) tc_mma_tf32_ts(d_tmem, ta_hi, db_hi, idesc, first ? 0u : 1u);
                                else tc_mma_tf32_ts_acc(d_tmem, ta_hi + kk * 8, db_hi, idesc);
                                tc_mma_tf32_ts_acc(d_tmem, ta_hi + kk * 8, db_lo, idesc);
                                tc_mma_tf32_ts_acc(d_tmem, ta_lo + kk * 8, db_hi, idesc);
                            } else {
                                const uint64_t da_hi = desc_at(hi_a16 + kk * k_step16);
                                const uint64_t da_lo = desc_at(lo_a16 + kk * k_step16);
                                if (kk == 0) tc_mma_tf32(d_tmem, da_hi, db_hi, idesc, first ? 0u : 1u);
                                else tc_mma_tf32_acc(d_tmem, da_hi, db_hi, idesc);
                                tc_mma_tf32_acc(d_tmem, da_hi, db_lo, idesc);
                                tc_mma_tf32_acc(d_tmem, da_lo, db_hi, idesc);
                            }
                        }
                        first = false;
                        tc_commit(smem_u32(&empty[st]));              // raw, lo and TMEM-A slots are free once these MMAs retire
                        if (++st == kNB) { st = 0; st_phase ^= 1u; }
                        if (++ls == kLoN) ls = 0;
                    }
                    if (ok) tc_commit(smem_u32(&acc_full[b]));
                }
            }
            if (!ok) {      // abort: MMAs already issued must retire before TMEM is freed
                tc_commit(smem_u32(drain));
                for (uint32_t t = 0; t < kWaitLimit && !mbar_try(smem_u32(drain), 0); ++t) {}
            }
        }
    } else if (warp < 2 + kTransformWarps) {
        // ================= transform warps: square and split into TF32 hi / lo =================
        const int t = (int)threadIdx.x - 64;                               // 0 .. 128 * kGroups - 1
        // With nothing to gather the warps work as groups of four that take consecutive slices in turn: the waits,
        // fences and tensor-memory stores of one slice then overlap the arithmetic of the others.  The same split
        // is used when the B tile is gathered several taps at a time next to a TMA-fed A tile.  The element-wise
        // gathers share every slice among the first eight warps; further warps have nothing to do there.
        constexpr int kTT = kTwoGroups ? 128 : kGatherThreads;             // threads sharing a slice
        const int group = kTwoGroups ? (t >> 7) : 0;
        const int tt = kTwoGroups ? (t & 127) : t;
        const int kq = tt & 7, row0 = tt >> 3;                             // gathered chunks: rows row0 + 32*i, k = 4*kq..4*kq+3
        Gatherer<kModeA, kTwoGroups> rows_a;
        Gatherer<kModeB, kTwoGroups> rows_b;
        typedef typename Gatherer<kModeA, kTwoGroups>::Regs RegsA;
        typedef typename Gatherer<kModeB, kTwoGroups>::Regs RegsB;
        // where the current slice sits: example z, 32-wide block pblk of that example's output positions
        int z = 0, pblk = 0;
        auto advance = [&]() {
            if (++pblk == prm.p_slices) { pblk = 0; ++z; }
        };
        auto gather = [&](RegsA &ga, RegsB &gb) {
            const int pbase = pblk * kBK + kq * 4;
            rows_a.load(prm, z, pbase, ga);
            rows_b.load(prm, z, pbase, gb);
        };
        // transform of the block's slice number i; gathered elements come in registers, TMA tiles from the raw stage
        auto process = [&](int i, const RegsA &ga, const RegsB &gb) -> bool {
            const int st = i % kNB, ls = i % kLoN;
            const uint32_t ph = (uint32_t)(i / kNB) & 1u;
            const int sa = kSplit ? i % kNA : 0;
            if (kSplit && !mbar_wait(smem_u32(&a_full[sa]), (uint32_t)(i / kNA) & 1u, &abort_flag)) return false;
            // a raw slot is ours once its TMA tiles landed (the producer waited for it to be empty), or, with
            // nothing coming by TMA, once the MMAs that last read it retired; likewise the lo slot
            if (kAnyTma ? !mbar_wait(smem_u32(&raw_full[st]), ph, &abort_flag)
                        : !mbar_wait(smem_u32(&empty[st]), ph ^ 1u, &abort_flag))
                return false;
            if (i >= kLoN) {      // the lo slot's previous user: slice i - kLoN
                const int j = i - kLoN;
                if (!mbar_wait(smem_u32(&empty[j % kNB]), (uint32_t)(j / kNB) & 1u, &abort_flag)) return false;
            }
            uint8_t *hi = smem_gen + pair_off(st);               // raw tiles live here and become the hi tiles
            // lo tiles: [A lo][B lo], or the B tile alone when A lives in tensor memory (then `lo` points
            // one A tile below the slot so that the same chunk offsets address the B part)
            uint8_t *lo = smem_gen + lo_off(ls);
            if (kATmem) {
                // A: this thread's row (TMEM lane) and 16 of the slice's 32 k at a time -> hi / lo straight into
                // TMEM (a warp of the two-group form takes both halves, otherwise its group number picks one)
                tc_fence_after();
                const uint32_t q = warp & 3;
                const int m_local = (int)(q * 32 + lane);
                const uint8_t *arow = (kSplit ? smem_gen + (uint32_t)sa * kRawBytesA : hi) + m_local * 128;
#pragma unroll
                for (int hh = 0; hh < (kTwoGroups ? 2 : 1); ++hh) {
                    const uint32_t h = kTwoGroups ? (uint32_t)hh : (warp - 2) >> 2;
                    float4 c4[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        c4[u] = *reinterpret_cast<const float4 *>(arow + (((4 * h + u) ^ (m_local & 7)) << 4));
                    uint32_t h16[16], l16[16];
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const float e[4] = {c4[u].x, c4[u].y, c4[u].z, c4[u].w};
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const float sq = kExact ? e[j] : __fmul_rn(e[j], e[j]);
                            h16[4 * u + j] = to_tf32(sq);
                            l16[4 * u + j] = __float_as_uint(__fsub_rn(sq, __uint_as_float(h16[4 * u + j])));
                        }
                    }
                    const uint32_t taddr = tmem_base + ((q * 32u) << 16) + 2 * kBN + ls * kTmemColsA + 16 * h;
                    tc_st_32x16(taddr, h16);
                    if (kBf) {
                        uint32_t hb[8], lb[8];
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            hb[j] = pack_bf16(__uint_as_float(h16[2 * j]), __uint_as_float(h16[2 * j + 1]));
                            lb[j] = pack_bf16(__uint_as_float(l16[2 * j]), __uint_as_float(l16[2 * j + 1]));
                        }
                        const uint32_t tb = taddr - 16 * h + 32 + 8 * h;
                        tc_st_32x8(tb, hb);
                        tc_st_32x8(tb + 16, lb);
                    } else
                    tc_st_32x16(taddr + 32, l16);
                }
                if (kSplit) {                     // the raw A tile has been read: its slot may be refilled
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&a_empty[sa]));
                }
            }
            if (kBf) {
                // B tile: a thread takes pairs of adjacent 16-byte chunks (8 consecutive k of one row: the 128-byte
                // swizzle permutes the two chunks of a pair only among themselves).  hi goes back in place as tf32;
                // hi and lo as bf16 make one 16-byte chunk each, and under the 64-byte swizzle that chunk's place in
                // its tile is the pair's place in the raw tile.  Half of each quarter-warp reads the second chunk of
                // its pair first, which keeps the 16-byte accesses free of bank conflicts.
                uint8_t *braw = smem_gen + b_tile(st), *bf_hi = smem_gen + bf_tile(ls), *bf_lo = bf_hi + kBTile / 2;
                const uint32_t s1 = (lane >> 2) & 1u;
#pragma unroll
                for (int u = 0; u < (int)(kBTile / 32) / kTT; ++u) {
                    const uint32_t p = (uint32_t)tt + (uint32_t)u * kTT;          // pair index = 4 * row + pair of the row
                    const uint32_t offx = 32 * p + 16 * s1, offy = 32 * p + 16 * (s1 ^ 1u);
                    const float4 x4 = *reinterpret_cast<const float4 *>(braw + offx);
                    const float4 y4 = *reinterpret_cast<const float4 *>(braw + offy);
                    const float ex[8] = {x4.x, x4.y, x4.z, x4.w, y4.x, y4.y, y4.z, y4.w};
                    uint32_t h[8];
                    float l[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float sq = __fmul_rn(ex[j], ex[j]);
                        h[j] = to_tf32(sq);
                        l[j] = __fsub_rn(sq, __uint_as_float(h[j]));
                    }
                    *reinterpret_cast<uint4 *>(braw + offx) = make_uint4(h[0], h[1], h[2], h[3]);
                    *reinterpret_cast<uint4 *>(braw + offy) = make_uint4(h[4], h[5], h[6], h[7]);
                    const uint32_t hx0 = pack_bf16(__uint_as_float(h[0]), __uint_as_float(h[1]));
                    const uint32_t hx1 = pack_bf16(__uint_as_float(h[2]), __uint_as_float(h[3]));
                    const uint32_t hy0 = pack_bf16(__uint_as_float(h[4]), __uint_as_float(h[5]));
                    const uint32_t hy1 = pack_bf16(__uint_as_float(h[6]), __uint_as_float(h[7]));
                    const uint32_t lx0 = pack_bf16(l[0], l[1]), lx1 = pack_bf16(l[2], l[3]);
                    const uint32_t ly0 = pack_bf16(l[4], l[5]), ly1 = pack_bf16(l[6], l[7]);
                    // the chunk read first holds the lower k iff its place in the pair equals the row's parity
                    const bool x_first = s1 == ((p >> 2) & 1u);
                    *reinterpret_cast<uint4 *>(bf_hi + 16 * p) =
                        x_first ? make_uint4(hx0, hx1, hy0, hy1) : make_uint4(hy0, hy1, hx0, hx1);
                    *reinterpret_cast<uint4 *>(bf_lo + 16 * p) =
                        x_first ? make_uint4(lx0, lx1, ly0, ly1) : make_uint4(ly0, ly1, lx0, lx1);
                }
            } else
            if (kAnyTma) {      // tiles that came by TMA: elementwise, in place, over their 16-byte chunks
                constexpr uint32_t c_begin = (kGatherA || kATmem) ? kRawBytesA / 16 : 0;
                constexpr uint32_t c_end = kGatherB ? kRawBytesA / 16 : kRawStageBytes / 16;
                constexpr int kPerThread = c_end > c_begin ? (c_end - c_begin) / kTT : 1;
                constexpr int kBatch = kPerThread < 4 ? kPerThread : 4;              // chunks in registers at a time
                if (c_end > c_begin) {
#pragma unroll
                    for (int u0 = 0; u0 < kPerThread; u0 += kBatch) {
                        float4 v[kBatch];
#pragma unroll
                        for (int u = 0; u < kBatch; ++u)
                            v[u] = *reinterpret_cast<const float4 *>(hi + 16 * (c_begin + (uint32_t)tt + (u0 + u) * kTT));
#pragma unroll
                        for (int u = 0; u < kBatch; ++u)
                            split_store<!kExact>(hi, lo, 16 * (c_begin + (uint32_t)tt + (u0 + u) * kTT), v[u].x, v[u].y, v[u].z, v[u].w);
                    }
                }
            }
            if (kGatherA) rows_a.template store<!kExact>(hi, lo, row0, kq, ga);
            if (kGatherB) rows_b.template store<!kExact>(hi + kRawBytesA, lo + kRawBytesA, row0, kq, gb);
            if (kATmem) { tc_wait_st(); tc_fence_before(); }      // TMEM stores complete and ordered before the signal
            fence_async_smem();                                   // generic-proxy writes -> tensor core reads
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&op_full[st]));
            return true;
        };

        RegsA a0, a1;
        RegsB b0, b1;
        int it0 = 0;                                 // block-wide number of the segment's first slice
        bool ok = true;
        SegIter iter(prm);
        Seg sg;
        if (!kTwoGroups && t >= kGatherThreads) ok = false;
        while (ok && iter.next(prm, sg)) {
            const int n_slices = sg.s_end - sg.s_begin;
            if (kAnyGather) {
                rows_a.init(prm, bt.x[sg.layer], bt.delta[sg.layer], sg.m0, row0, prm.M);
                rows_b.init(prm, bt.x[sg.layer], bt.delta[sg.layer], sg.n0, row0, prm.N);
                z = sg.s_begin / prm.p_slices;
                pblk = sg.s_begin - z * prm.p_slices;
            }
            if (kTwoGroups) {
                // this group's slices: those whose block-wide number is the group's modulo kGroups.  With a gathered
                // tile: one register set per thread -- the other groups' work covers this group's load latency
                // (measured faster than two sets in turn)
                const int i_first = (group - it0 % kGroups + kGroups) % kGroups;
                if (kAnyGather)
                    for (int sk = 0; sk < i_first; ++sk) advance();
                for (int i = i_first; i < n_slices; i += kGroups) {
                    if (kAnyGather) gather(a0, b0);
                    if (!process(it0 + i, a0, b0)) { ok = false; break; }
                    if (kAnyGather)
                        for (int sk = 0; sk < kGroups; ++sk) advance();
                }
            } else {
                // two register sets in turn: the loads of slice i+1 are in flight while slice i is transformed
                if (kAnyGather) gather(a0, b0);
                for (int i = 0; i < n_slices; i += 2) {
                    if (kAnyGather && i + 1 < n_slices) { advance(); gather(a1, b1); }
                    if (!process(it0 + i, a0, b0)) { ok = false; break; }
                    if (i + 1 < n_slices) {
                        if (kAnyGather && i + 2 < n_slices) { advance(); gather(a0, b0); }
                        if (!process(it0 + i + 1, a1, b1)) { ok = false; break; }
                    }
                }
            }
            it0 += n_slices;
        }
    } else {
        // ================= epilogue warps: drain chunks, accumulate in fp32 registers =================
        const uint32_t q = warp & 3;                                      // TMEM lane quarter of this warp
        const int r_local = (int)(q * 32u + lane);
        float acc[kBN];
        const uint32_t sq_addr = tmem_base + ((q * 32u) << 16) + kSqCol;  // kExact: this warp's rows of the sum of squares
        int c = 0;                                                        // running number of the chunk
        bool ok = true;
        SegIter iter(prm);
        Seg sg;
        while (ok && iter.next(prm, sg)) {
#pragma unroll
            for (int j = 0; j < kBN; ++j) acc[j] = 0.f;
            if (kExact) {
                uint32_t zero[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) zero[j] = 0u;
#pragma unroll
                for (int j0 = 0; j0 < kBN; j0 += 16) tc_st_32x16(sq_addr + j0, zero);
                tc_wait_st();
            }
            const int n_act = sg.n_act, n_valid = sg.n_valid;
            const int n_slices = sg.s_end - sg.s_begin;
            const int seg_len = kExact ? prm.p_slices : n_slices;
            const int cps = (seg_len + prm.chunk - 1) / prm.chunk;
            const int n_chunks = (n_slices / seg_len) * cps;
            for (int cc = 0; cc < n_chunks && ok; ++cc, ++c) {
                const int b = c & 1;
                ok = mbar_wait(smem_u32(&acc_full[b]), (uint32_t)(c >> 1) & 1u, &abort_flag, 256);
                if (!ok) break;
                tc_fence_after();
                const uint32_t taddr = tmem_base + ((q * 32u) << 16) + (uint32_t)b * kBN;
#pragma unroll
                for (int j0 = 0; j0 < kBN; j0 += 32) {
                    if (j0 < n_act) {
                        uint32_t r[32];
                        tc_ld_32x32(taddr + j0, r);
                        tc_wait_ld();
#pragma unroll
                        for (int j = 0; j < 32; ++j) acc[j0 + j] = __fadd_rn(acc[j0 + j], __uint_as_float(r[j]));
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(smem_u32(&acc_empty[b]));
                if (kExact && (cc + 1) % cps == 0) {
                    // end of an example: acc holds its sum over positions; add the squares to the running sum in TMEM
#pragma unroll
                    for (int j0 = 0; j0 < kBN; j0 += 32) {
                        if (j0 < n_act) {
                            uint32_t r[32];
                            tc_ld_32x32(sq_addr + j0, r);
                            tc_wait_ld();
                            uint32_t w0[16], w1[16];
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                w0[j] = __float_as_uint(__fadd_rn(__uint_as_float(r[j]), __fmul_rn(acc[j0 + j], acc[j0 + j])));
                                w1[j] = __float_as_uint(__fadd_rn(__uint_as_float(r[16 + j]), __fmul_rn(acc[j0 + 16 + j], acc[j0 + 16 + j])));
                            }
                            tc_st_32x16(sq_addr + j0, w0);
                            tc_st_32x16(sq_addr + j0 + 16, w1);
                        }
                    }
                    tc_wait_st();
#pragma unroll
                    for (int j = 0; j < kBN; ++j) acc[j] = 0.f;
                }
            }
            if (!ok) break;
            if (kExact) {        // the result is the sum of squares
#pragma unroll
                for (int j0 = 0; j0 < kBN; j0 += 32) {
                    uint32_t r[32];
                    tc_ld_32x32(sq_addr + j0, r);
                    tc_wait_ld();
#pragma unroll
                    for (int j = 0; j < 32; ++j) acc[j0 + j] = __uint_as_float(r[j]);
                }
            }
            // ---- the segment's 128 x 128 sums leave the registers (the other roles are already on the next segment)
            const int m = sg.m0 + r_local;
            float *const S = bt.S[sg.layer];
            if (!sg.whole) {
                // partial tile, column-major inside the tile: consecutive lanes -> consecutive addresses
                float *dst = prm.partial + (size_t)sg.slot * (kBM * kBN) + r_local;
#pragma unroll
                for (int j = 0; j < kBN; ++j)
                    if (j < n_valid) dst[j * kBM] = acc[j];
            } else if (prm.ld_m == 1) {
                // result is contiguous along m: lanes write neighbouring addresses directly
                if (m < prm.M) {
                    float *col = S + (size_t)m + (size_t)sg.n0 * prm.ld_n;
#pragma unroll
                    for (int j0 = 0; j0 < kBN; j0 += 16) {        // old values sixteen at a time, all loads in flight
                        float old[16];
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            old[j] = (prm.accumulate && j0 + j < n_valid) ? col[(size_t)(j0 + j) * prm.ld_n] : 0.f;
#pragma unroll
                        for (int j = 0; j < 16; ++j)
                            if (j0 + j < n_valid) {
                                const float res = __fmul_rn(prm.scale, acc[j0 + j]);
                                col[(size_t)(j0 + j) * prm.ld_n] = prm.accumulate ? __fadd_rn(old[j], res) : res;
                            }
                    }
                }
            } else if (iter.pos >= iter.end) {
                // result is contiguous along n, and this is the block's last segment: the pipeline stages are idle
                // (the last accumulator was complete before we got here), so this warp's 32 x 128 block is transposed
                // through shared memory and written row by row with consecutive lanes on consecutive addresses
                float *tile = reinterpret_cast<float *>(smem_gen) + q * (32 * (kBN + 1));
#pragma unroll
                for (int j = 0; j < kBN; ++j) tile[lane * (kBN + 1) + j] = __fmul_rn(prm.scale, acc[j]);
                __syncwarp();
                for (int r0 = 0; r0 < 32; r0 += 8) {              // eight rows at a time, all loads in flight
                    float old[8][kBN / 32];
#pragma unroll
                    for (int rr = 0; rr < 8; ++rr) {
                        const int mr = sg.m0 + (int)(q * 32u) + r0 + rr;
                        const float *src = S + (size_t)mr * prm.ld_m + sg.n0;
#pragma unroll
                        for (int cblk = 0; cblk < kBN / 32; ++cblk) {
                            const int j = cblk * 32 + (int)lane;
                            old[rr][cblk] = (prm.accumulate && mr < prm.M && j < n_valid) ? src[j] : 0.f;
                        }
                    }
#pragma unroll
                    for (int rr = 0; rr < 8; ++rr) {
                        const int mr = sg.m0 + (int)(q * 32u) + r0 + rr;
                        float *dst = S + (size_t)mr * prm.ld_m + sg.n0;
#pragma unroll
                        for (int cblk = 0; cblk < kBN / 32; ++cblk) {
                            const int j = cblk * 32 + (int)lane;
                            if (mr < prm.M && j < n_valid) {
                                const float res = tile[(r0 + rr) * (kBN + 1) + j];
                                dst[j] = prm.accumulate ? __fadd_rn(old[rr][cblk], res) : res;
                            }
                        }
                    }
                }
            } else if (m < prm.M) {
                // result is contiguous along n, more segments follow (the pipeline is busy with the next one): every
                // lane owns a row and writes it 16 bytes at a time (the halves of a
                // 32-byte sector arrive in consecutive instructions and are merged in L2); rows whose pitch is not a
                // multiple of 16 bytes go element by element
                float *row = S + (size_t)m * prm.ld_m + sg.n0;
                if ((prm.ld_m & 3) == 0) {
#pragma unroll
                    for (int j0 = 0; j0 < kBN; j0 += 16) {
                        float4 old[4];
#pragma unroll
                        for (int u = 0; u < 4; ++u)
                            old[u] = (prm.accumulate && j0 + 4 * u + 3 < n_valid) ? *reinterpret_cast<const float4 *>(row + j0 + 4 * u)
                                                                                  : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            const int j = j0 + 4 * u;
                            if (j + 3 < n_valid) {
                                float4 res = make_float4(__fmul_rn(prm.scale, acc[j]), __fmul_rn(prm.scale, acc[j + 1]),
                                                         __fmul_rn(prm.scale, acc[j + 2]), __fmul_rn(prm.scale, acc[j + 3]));
                                if (prm.accumulate) {
                                    res.x = __fadd_rn(old[u].x, res.x); res.y = __fadd_rn(old[u].y, res.y);
                                    res.z = __fadd_rn(old[u].z, res.z); res.w = __fadd_rn(old[u].w, res.w);
                                }
                                *reinterpret_cast<float4 *>(row + j) = res;
                            } else {
#pragma unroll
                                for (int e = 0; e < 4; ++e)
                                    if (j + e < n_valid) {
                                        const float res = __fmul_rn(prm.scale, acc[j + e]);
                                        row[j + e] = prm.accumulate ? __fadd_rn(row[j + e], res) : res;
                                    }
                            }
                        }
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < kBN; ++j)
                        if (j < n_valid) {
                            const float res = __fmul_rn(prm.scale, acc[j]);
                            row[j] = prm.accumulate ? __fadd_rn(row[j], res) : res;
                        }
                }
            }
        }
    }

    // ---- common exit ----
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
    if (threadIdx.x == 0 && abort_flag) atomicOr(prm.status, VGC_DEV_TIMEOUT);
}

// Adds the partial tiles of every tile that more than one block worked on, in the order of the blocks (a fixed
// order: the result does not depend on scheduling).  One thread block per 32 x 32 patch of a tile: a warp takes
// four columns, a lane one row -- partials are read along rows (their unit stride), four independent sums per
// thread -- and the result is written along whichever of m / n has unit stride.  Tiles that one block covered
// alone were written by that block; their patches return at once.
struct ResultPtrs { float *S[kMaxBatch]; };

__global__ void __launch_bounds__(256)
sqgrad_tc_combine(const float *__restrict__ partial, int units_q, int units_r, int units_per_tile,
                  int tiles_x, int tiles_y, int M, int N, float scale, int accumulate, const ResultPtrs results,
                  long long ld_m, long long ld_n)
{
    __shared__ float patch[32][33];
    const int tile = blockIdx.x >> 4, sub = blockIdx.x & 15;
    // the blocks that hold the tile's first and last unit: the first units_r blocks own units_q + 1 units each, the
    // others units_q
    const int t_lo = ((int)blockIdx.y * (tiles_x * tiles_y) + tile) * units_per_tile;
    const int big = units_r * (units_q + 1);
    auto block_of = [&](int u) -> int { return u < big ? u / (units_q + 1) : units_r + (u - big) / units_q; };
    const int b_first = block_of(t_lo), b_last = block_of(t_lo + units_per_tile - 1);
    if (b_first == b_last) return;
    float *__restrict__ S = results.S[blockIdx.y];                         // blockIdx.y: layer of the batch
    const int tx = tile % tiles_x, ty = tile / tiles_x;
    const int r0 = (sub & 3) * 32, j0 = (sub >> 2) * 32;                  // patch origin inside the tile
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;              // lane -> row, warp -> four columns
    if (ty * kBM + r0 >= M || tx * kBN + j0 >= N) return;
    // the first block's part of this tile is that block's last segment unless its range starts with the tile;
    // every later block's part is its first segment
    const int lo_first = b_first * units_q + min(b_first, units_r);
    const size_t within = (size_t)(j0 + 4 * w) * kBM + r0 + lane;
    const float *src0 = partial + (size_t)(2 * b_first + (lo_first < t_lo ? 1 : 0)) * (kBM * kBN) + within;
    const float *src = partial + within;
    float sum[4];
#pragma unroll
    for (int c = 0; c < 4; ++c) sum[c] = __ldcs(src0 + c * kBM);
    int b = b_first + 1;
    for (; b + 2 <= b_last + 1; b += 2) {                // eight loads in flight, summed in block order
        float v[2][4];
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int c = 0; c < 4; ++c) v[u][c] = __ldcs(src + (size_t)(2 * (b + u)) * (kBM * kBN) + c * kBM);
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int c = 0; c < 4; ++c) sum[c] = __fadd_rn(sum[c], v[u][c]);
    }
    for (; b <= b_last; ++b)
#pragma unroll
        for (int c = 0; c < 4; ++c) sum[c] = __fadd_rn(sum[c], __ldcs(src + (size_t)(2 * b) * (kBM * kBN) + c * kBM));
    if (ld_m == 1) {
        const int m = ty * kBM + r0 + lane;
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const int n = tx * kBN + j0 + 4 * w + c;
            if (m < M && n < N) {
                float *dst = S + (size_t)m + (size_t)n * ld_n;
                const float res = __fmul_rn(scale, sum[c]);
                *dst = accumulate ? __fadd_rn(*dst, res) : res;
            }
        }
        return;
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) patch[4 * w + c][lane] = __fmul_rn(scale, sum[c]);      // patch[column][row]
    __syncthreads();
    {
        const int c0 = (threadIdx.x & 7) * 4, r = threadIdx.x >> 3;       // four consecutive columns of one row
        const int m = ty * kBM + r0 + r, n = tx * kBN + j0 + c0;
        if (m < M) {
            float *dst = S + (size_t)m * ld_m + n;
            if ((ld_m & 3) == 0 && n + 3 < N) {
                float4 out = make_float4(patch[c0][r], patch[c0 + 1][r], patch[c0 + 2][r], patch[c0 + 3][r]);
                if (accumulate) {
                    const float4 old = *reinterpret_cast<const float4 *>(dst);
                    out.x = __fadd_rn(old.x, out.x); out.y = __fadd_rn(old.y, out.y);
                    out.z = __fadd_rn(old.z, out.z); out.w = __fadd_rn(old.w, out.w);
                }
                *reinterpret_cast<float4 *>(dst) = out;
            } else {
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (n + c < N) dst[c] = accumulate ? __fadd_rn(dst[c], patch[c0 + c][r]) : patch[c0 + c][r];
            }
        }
    }
}

// ---- host side --------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn()
{
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

static bool make_map(CUtensorMap *map, const float *base, int rank, const cuuint64_t *dims, const cuuint64_t *strides_bytes,
                     const cuuint32_t *box, CUtensorMapSwizzle swizzle)
{
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint32_t elem_strides[3] = {1, 1, 1};
    const CUresult rc = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, (cuuint32_t)rank, const_cast<float *>(base), dims,
                           strides_bytes, box, elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (rc != CUDA_SUCCESS && debug_enabled()) fprintf(stderr, "vgc: tensor map encode failed with CUresult %d\n", (int)rc);
    return rc == CUDA_SUCCESS;
}

// Slices per accumulator drain.  The tensor core's fp32 accumulation truncates (a one-sided bias of about 1.3e-8 of the
// sum per instruction), so an accumulator is handed to the round-to-nearest register sums after at most 8 slices
// (96 instructions): results then sit 1 - 3e-6 below the exact sum, against the 1e-5 bound.
constexpr int kChunk = 8;
constexpr int kSmCount = 148;            // SMs of a B200
// how many sqgrad launches the caller keeps in flight side by side (vgc_sqgrad_plan_hint)
static int g_concurrent = 1;

struct Plan {
    int unit, units_per_tile, blocks, tiles_x, tiles_y;
    int units_total;
    bool partials;           // some tile is shared by several blocks: partial tiles go through the scratch
};

// How a launch's work -- n_layers x tiles x k_slices slices -- is cut into one contiguous range per block.
// `unit_min`: slices that must stay in one block (the per-example form cuts the reduction between examples only).
// Two candidates: whole tiles per block (no scratch, no second kernel, but the blocks' loads are as even as the
// tile count allows), or an even cut of the slices over all SMs (tiles at the cuts are shared, their partial
// sums combined by a second kernel).  Costs in slice times: a block's longest range, plus what the combine pass
// adds to the call (its launch and the partial tiles' round trip, about 14 slices' worth).
static Plan make_plan(int M, int N, int k_slices, int n_layers, int unit_min)
{
    Plan p;
    p.tiles_x = (N + kBN - 1) / kBN;
    p.tiles_y = (M + kBM - 1) / kBM;
    const long long tiles = (long long)p.tiles_x * p.tiles_y * n_layers;
    const long long upt = k_slices / unit_min, units = tiles * upt;
    bool even;
    long long blocks;
    if (g_concurrent > 1) {
        // Next to other launches the hardware's block scheduler does the balancing: blocks of all launches in flight
        // queue for the SMs and a partly filled wave costs nothing (the neighbours' blocks take the idle SMs).  Each
        // tile's reduction is cut into as many parts as make about half a wave of blocks per launch: shorter blocks
        // pay their start and tail more often, longer ones balance worse (measured on the ResNet-50 pass with 3 to 8
        // launches in flight: 148 blocks per launch 1.90 ms, 111: 1.86, 74: 1.80 - 1.85, 50: 1.99).
        long long parts = (kSmCount / 2) / tiles;
        parts = parts > upt ? upt : (parts < 1 ? 1 : parts);
        even = parts > 1;
        blocks = tiles * parts;
    } else {
        // Alone, the launch is one block per SM at most.  Two candidates, costs in slice times: whole tiles per block
        // (a block's longest range), or an even cut of all slices (plus what the combine pass adds to the call: its
        // launch and the partial tiles' round trip, about 14 slices' worth).
        const long long waves = (tiles + kSmCount - 1) / kSmCount;
        const long long blocks_a = (tiles + waves - 1) / waves;
        const long long cost_a = ((tiles + blocks_a - 1) / blocks_a) * k_slices;
        const long long blocks_b = units < kSmCount ? units : kSmCount;
        const long long cost_b = ((units + blocks_b - 1) / blocks_b) * unit_min + 14;
        even = cost_b < cost_a;
        blocks = even ? blocks_b : blocks_a;
    }
    if (even && units >= (1LL << 31)) {          // unit positions are 32-bit in the kernel: whole tiles then
        even = false;
        blocks = tiles < kSmCount ? tiles : kSmCount;
    }
    p.unit = even ? unit_min : k_slices;
    p.units_per_tile = even ? (int)upt : 1;
    p.units_total = (int)(even ? units : tiles);
    p.blocks = (int)blocks;
    p.partials = false;
    const int q = p.units_total / p.blocks, r = p.units_total % p.blocks;
    for (int b = 1; b < p.blocks && !p.partials; ++b) p.partials = (b * q + (b < r ? b : r)) % p.units_per_tile != 0;
    return p;
}

}  // namespace tc

using namespace tc;

void tc_plan_hint(int concurrent_launches)
{
    g_concurrent = concurrent_launches > 1 ? concurrent_launches : 1;
}

bool tc_linear_supported(int B, int in, int out)
{
    return B >= 32 && in >= 32 && out >= 32 && in % 4 == 0 && out % 4 == 0;
}
bool tc_conv_supported(int B, int C, int H, int W, int Cout, int Kh, int Kw, int sh, int sw, int ph, int pw)
{
    const long Ho = (H + 2 * ph - Kh) / sh + 1, Wo = (W + 2 * pw - Kw) / sw + 1;
    const long P = Ho * Wo, N = (long)C * Kh * Kw;
    // 32-bit index arithmetic inside the kernel
    return B >= 1 && C >= 1 && Cout >= 1 && (long)C * H * W < (1L << 30) && N < (1L << 24) &&
           (long)B * ((P + kBK - 1) / kBK) < (1L << 30);
}

static size_t tc_workspace_bytes(int M, int N, int k_slices, int n_layers = 1, int unit = 1)
{
    const Plan p = make_plan(M, N, k_slices, n_layers, unit);
    // status word (256 bytes) + two partial tiles per block (the first and the last segment of its range)
    return 256 + (p.partials ? (size_t)2 * p.blocks * kBM * kBN * sizeof(float) : 0);
}

typedef void (*KernelFn)(const Batch, const Params);

static vgc_status tc_launch(KernelFn kernel, const Batch &bt, int n_layers, Params prm, int M, int N,
                            int k_slices, void *ws, size_t ws_bytes, cudaStream_t st, int unit = 1)
{
    const Plan plan = make_plan(M, N, k_slices, n_layers, unit);
    if (ws_bytes < tc_workspace_bytes(M, N, k_slices, n_layers, unit)) return VGC_ERR_WORKSPACE;
    static KernelFn configured[32];
    static int n_configured = 0;
    bool seen = false;
    for (int i = 0; i < n_configured; ++i) seen = seen || configured[i] == kernel;
    if (!seen) {
        VGC_CUDA_OK(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
        if (n_configured < 32) configured[n_configured++] = kernel;
    }
    prm.M = M; prm.N = N; prm.k_slices = k_slices;
    prm.unit = plan.unit; prm.units_per_tile = plan.units_per_tile; prm.units_total = plan.units_total;
    prm.units_q = plan.units_total / plan.blocks; prm.units_r = plan.units_total % plan.blocks;
    prm.tiles_x = plan.tiles_x; prm.tiles_y = plan.tiles_y;
    prm.chunk = kChunk;
    prm.status = static_cast<uint32_t *>(ws);
    prm.partial = reinterpret_cast<float *>(static_cast<char *>(ws) + 256);
    kernel<<<plan.blocks, kThreadsTc, kSmemBytes, st>>>(bt, prm);
    count_launch();
    if (plan.partials) {
        ResultPtrs results = {};
        for (int l = 0; l < n_layers; ++l) results.S[l] = bt.S[l];
        sqgrad_tc_combine<<<dim3((unsigned)(plan.tiles_x * plan.tiles_y * 16), (unsigned)n_layers), 256, 0, st>>>(
            prm.partial, prm.units_q, prm.units_r, plan.units_per_tile, plan.tiles_x, plan.tiles_y, M, N, prm.scale,
            prm.accumulate, results, prm.ld_m, prm.ld_n);
        count_launch();
    }
    VGC_CUDA_OK(cudaGetLastError());
    return VGC_OK;
}

size_t tc_linear_workspace_bytes(int B, int in, int out) { return tc_workspace_bytes(out, in, (B + kBK - 1) / kBK); }

vgc_status tc_sqgrad_linear(const float *x, const float *delta, int B, int in, int out, float scale, int accumulate,
                            float *S, void *ws, size_t ws_bytes, cudaStream_t st)
{
    Batch bt = {};
    const cuuint32_t box[2] = {32, (cuuint32_t)kBK};
    const cuuint64_t dims_a[2] = {(cuuint64_t)out, (cuuint64_t)B}, str_a[1] = {(cuuint64_t)out * 4};
    const cuuint64_t dims_b[2] = {(cuuint64_t)in, (cuuint64_t)B}, str_b[1] = {(cuuint64_t)in * 4};
    if (!make_map(&bt.a[0], delta, 2, dims_a, str_a, box, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B) ||
        !make_map(&bt.b[0], x, 2, dims_b, str_b, box, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B))
        return VGC_ERR_CUDA;
    bt.x[0] = x; bt.delta[0] = delta; bt.S[0] = S;
    Params prm = {};
    prm.p_slices = 1; prm.tx_bytes = kRawStageBytes; prm.tx_bytes_a = kRawBytesA; prm.scale = scale;
    prm.accumulate = accumulate;
    prm.ld_m = in; prm.ld_n = 1;
    return tc_launch(sqgrad_tc<kMajorMN, kTma, kTma, false>, bt, 1, prm, out, in, (B + kBK - 1) / kBK, ws, ws_bytes, st);
}

// Set for the duration of a per-example (exact) call: planning, repacking and kernel choice consult it.
static thread_local bool t_exact = false;
struct ExactScope {
    bool saved;
    explicit ExactScope(bool on) : saved(t_exact) { t_exact = on; }
    ~ExactScope() { t_exact = saved; }
};

// Cout <= 64: the im2col rows take the 128-row A tile and the errors the narrow B tile
static bool conv_swapped(int Cout, int n_im2col) { return Cout <= 64 && n_im2col > Cout; }

// ---- repacking pre-pass for 1x1 convolutions whose tiles TMA cannot address in place ----------
// A strided 1x1 convolution reads every (sh, sw)-th input position, and planes of P positions with P not
// a multiple of 4 (7x7) have a row pitch TMA does not accept.  One small copy kernel per operand puts
// them into a layout the TMA-fed kernel takes:
//   kRepackPlanes   x_s[z][c][p] = x[z][c][(p / Wo) sh][(p % Wo) sw]: the input subsampled, examples kept
//                   apart (the errors are used where they are)
//   kRepackFlat     x_r[c][z P + p], d_r[o][z P + p]: channel-major, the (example, position) pairs of one
//                   channel back to back -- the layer becomes a 1x1 convolution over ONE example with
//                   B P positions, and its reduction has no per-example padding to whole slices
//   kRepackPadW     a Kw = 3, pad_w = 1 kernel with stride 1 (W == Wo) or 2 (W == 2 Wo) whose output planes have
//                   an odd width (7x7): the errors are copied into planes of width Wo4 = Wo rounded up to 4 and x
//                   into planes of width stride * Wo4, new columns zero.  Zero input columns are what the padding
//                   supplies anyway, zero error columns contribute nothing, so the statistic is unchanged -- and
//                   the padded layer has TMA-able error planes and takes the three-tap gather
enum { kRepackNone = 0, kRepackPlanes = 1, kRepackFlat = 2, kRepackPadW = 3 };

static int repack_mode(int B, int C, int Cout, int Kh, int Kw, int sh, int sw, int ph, int pw, int P, int W = 0, int Ho = 0,
                       int Wo = 0)
{
    if ((long)B * C >= (1L << 31) || (long)B * Cout >= (1L << 31)) return kRepackNone;      // 32-bit row index
    if (Kw == 3 && pw == 1 && Wo % 2 == 1 && Wo >= 3 && (long)Ho * ((Wo + 3) / 4 * 4) >= kBK &&
        ((sw == 1 && sh == 1 && W == Wo) || (sw == 2 && W == 2 * Wo)))
        return kRepackPadW;
    if (Kh != 1 || Kw != 1 || ph != 0 || pw != 0) return kRepackNone;
    const bool planes_ok = P >= kBK && P % 4 == 0;
    if (planes_ok) return (sh > 1 || sw > 1) ? kRepackPlanes : kRepackNone;
    const long flat = (long)B * P;
    if (t_exact) return kRepackNone;                 // the flat form merges the examples' positions
    return (flat >= kBK && flat % 4 == 0 && flat < (1L << 30)) ? kRepackFlat : kRepackNone;
}

// One tensor to repack: out[a][b][p] = in[z][c][(p / Wo) sh W + (p % Wo) sw], zero where p % Wo >= wo_valid, with
// (a, b) = (z, c), or (c, z) when channel_major.  All tensors of a layer group go into one launch.
struct RepackJob {
    const float *in;
    float *out;
    int C, HW, W, Wo, P, sh, sw, channel_major, wo_valid;
};
struct RepackJobs {
    RepackJob job[2 * kMaxBatch];
    int B;
};

// out[a][b][p] = in[z][c][(p / Wo) sh W + (p % Wo) sw] with (a, b) = (z, c), or (c, z) when channel_major.
// One warp per group of four rows of P positions (rows of the output are contiguous), lanes along p, eight
// loads in flight per lane.
__global__ void __launch_bounds__(256)
sqgrad_repack(const __grid_constant__ RepackJobs jobs)
{
    constexpr int kRows = 4, kCols = 2;
    // blockIdx.y picks the tensor; its description is read once (a run-time index into kernel parameters
    // is expensive, so nothing below touches `jobs` again)
    const RepackJob job = jobs.job[blockIdx.y];
    const float *__restrict__ in = job.in;
    float *__restrict__ out = job.out;
    const int B = jobs.B, C = job.C, HW = job.HW, W = job.W, Wo = job.Wo, P = job.P, sh = job.sh, sw = job.sw;
    const int channel_major = job.channel_major, wo_valid = job.wo_valid;
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t rows = (uint32_t)B * (uint32_t)C;
    const bool dense = sh == 1 && sw == 1 && W == Wo && wo_valid == Wo;   // the plane is copied as it is
    for (uint32_t row0 = (blockIdx.x * 8 + (threadIdx.x >> 5)) * kRows; row0 < rows; row0 += gridDim.x * 8 * kRows) {
        const float *src[kRows];
#pragma unroll
        for (int r = 0; r < kRows; ++r) {
            const uint32_t row = row0 + r < rows ? row0 + r : rows - 1;
            uint32_t z, c;
            if (channel_major) { c = row / (uint32_t)B; z = row - c * (uint32_t)B; }
            else               { z = row / (uint32_t)C; c = row - z * (uint32_t)C; }
            src[r] = in + ((size_t)z * C + c) * HW;
        }
        for (uint32_t p0 = 0; p0 < (uint32_t)P; p0 += 32 * kCols) {
            float v[kRows][kCols];
            uint32_t off[kCols];
            bool live[kCols];                                           // columns wo >= wo_valid are zero padding
#pragma unroll
            for (int u = 0; u < kCols; ++u) {
                const uint32_t p = p0 + lane + 32u * u;
                live[u] = p < (uint32_t)P;
                if (dense) off[u] = p;
                else {
                    const uint32_t ho = p / (uint32_t)Wo, wo = p - ho * (uint32_t)Wo;
                    off[u] = ho * sh * W + wo * sw;
                    live[u] = live[u] && wo < (uint32_t)wo_valid;
                }
            }
#pragma unroll
            for (int r = 0; r < kRows; ++r)
#pragma unroll
                for (int u = 0; u < kCols; ++u)
                    v[r][u] = live[u] ? __ldg(src[r] + off[u]) : 0.f;
#pragma unroll
            for (int r = 0; r < kRows; ++r)
#pragma unroll
                for (int u = 0; u < kCols; ++u) {
                    const uint32_t p = p0 + lane + 32u * u;
                    if (row0 + r < rows && p < (uint32_t)P) out[(size_t)(row0 + r) * P + p] = v[r][u];
                }
        }
    }
}

static size_t conv_workspace_plain(int n_layers, int B, int C, int Kh, int Kw, int P, int Cout)
{
    const int p_slices = (P + kBK - 1) / kBK, n_im2col = C * Kh * Kw, k_slices = B * p_slices;
    const int unit = t_exact ? p_slices : 1;
    return conv_swapped(Cout, n_im2col) ? tc_workspace_bytes(n_im2col, Cout, k_slices, n_layers, unit)
                                        : tc_workspace_bytes(Cout, n_im2col, k_slices, n_layers, unit);
}

// Workspace of one launch over n_layers layers of this geometry (n_layers <= kMaxBatch).
static size_t conv_workspace_group(int n_layers, int B, int C, int Kh, int Kw, int sh, int sw, int ph, int pw, int P,
                                   int Cout, int H, int W, int Ho, int Wo)
{
    // the larger of the in-place form and the repacked one, so that either can be chosen at call time
    size_t need = conv_workspace_plain(n_layers, B, C, Kh, Kw, P, Cout);
    const int mode = repack_mode(B, C, Cout, Kh, Kw, sh, sw, ph, pw, P, W, Ho, Wo);
    const size_t x_bytes = round_up(sizeof(float) * (size_t)B * C * P, 256);
    const size_t d_bytes = round_up(sizeof(float) * (size_t)B * Cout * P, 256);
    if (mode == kRepackPadW) {
        const int Wo4 = (Wo + 3) / 4 * 4;
        const size_t xp = round_up(sizeof(float) * (size_t)B * C * H * (sw * Wo4), 256);
        const size_t dp = round_up(sizeof(float) * (size_t)B * Cout * Ho * Wo4, 256);
        const size_t r = round_up(conv_workspace_plain(n_layers, B, C, Kh, Kw, Ho * Wo4, Cout), 256) + n_layers * (xp + dp);
        need = need > r ? need : r;
    } else if (mode == kRepackPlanes) {
        const size_t r = round_up(conv_workspace_plain(n_layers, B, C, 1, 1, P, Cout), 256) + n_layers * x_bytes;
        need = need > r ? need : r;
    } else if (mode == kRepackFlat) {
        const size_t r = round_up(conv_workspace_plain(n_layers, 1, C, 1, 1, B * P, Cout), 256) +
                         n_layers * (x_bytes + d_bytes);
        need = need > r ? need : r;
    }
    return need;
}

size_t tc_conv_workspace_bytes(int n_layers, int B, int C, int H, int W, int Kh, int Kw, int sh, int sw, int ph, int pw,
                               int Ho, int Wo, int Cout, bool exact)
{
    const int P = Ho * Wo;
    ExactScope scope(exact);
    // more layers than one launch takes are processed group after group in the same workspace
    const int first = n_layers < kMaxBatch ? n_layers : kMaxBatch;
    size_t need = conv_workspace_group(first, B, C, Kh, Kw, sh, sw, ph, pw, P, Cout, H, W, Ho, Wo);
    const int rest = n_layers > kMaxBatch ? n_layers % kMaxBatch : 0;
    if (rest) {
        const size_t r = conv_workspace_group(rest, B, C, Kh, Kw, sh, sw, ph, pw, P, Cout, H, W, Ho, Wo);
        need = need > r ? need : r;
    }
    return need;
}

static vgc_status conv_group(int n_layers, const float *const *x, const float *const *delta, float *const *S, int B,
                             int C, int H, int W, int Cout, int Kh, int Kw, int sh, int sw, int ph, int pw, int Ho,
                             int Wo, float scale, int accumulate, void *ws, size_t ws_bytes, cudaStream_t st)
{
    const int P = Ho * Wo, n_im2col = C * Kh * Kw;
    const int mode = repack_mode(B, C, Cout, Kh, Kw, sh, sw, ph, pw, P, W, Ho, Wo);
    // one warp per row; a few rows per warp when there are many
    auto blocks_for = [](size_t rows) { const size_t b = (rows + 31) / 32; return (unsigned)(b < 1 ? 1 : (b > 148 * 32 ? 148 * 32 : b)); };
    if (mode == kRepackPadW) {
        const int Wo4 = (Wo + 3) / 4 * 4, Wx = sw * Wo4;              // padded widths of the errors and of x
        const size_t inner = round_up(conv_workspace_plain(n_layers, B, C, Kh, Kw, Ho * Wo4, Cout), 256);
        const size_t xp = round_up(sizeof(float) * (size_t)B * C * H * Wx, 256);
        const size_t dp = round_up(sizeof(float) * (size_t)B * Cout * Ho * Wo4, 256);
        if (ws_bytes < inner + n_layers * (xp + dp)) return VGC_ERR_WORKSPACE;
        const float *xr[kMaxBatch], *dr[kMaxBatch];
        RepackJobs jobs = {};
        jobs.B = B;
        for (int l = 0; l < n_layers; ++l) {
            char *base = static_cast<char *>(ws) + inner + (size_t)l * (xp + dp);
            float *x_p = reinterpret_cast<float *>(base), *d_p = reinterpret_cast<float *>(base + xp);
            jobs.job[2 * l] = RepackJob{x[l], x_p, C, H * W, W, Wx, H * Wx, 1, 1, 0, W};
            jobs.job[2 * l + 1] = RepackJob{delta[l], d_p, Cout, Ho * Wo, Wo, Wo4, Ho * Wo4, 1, 1, 0, Wo};
            xr[l] = x_p; dr[l] = d_p;
        }
        sqgrad_repack<<<dim3(blocks_for((size_t)B * (C > Cout ? C : Cout)), 2 * n_layers), 256, 0, st>>>(jobs);
        count_launch();
        return conv_group(n_layers, xr, dr, S, B, C, H, Wx, Cout, Kh, Kw, sh, sw, ph, 1, Ho, Wo4, scale, accumulate, ws, inner, st);
    }
    if (mode != kRepackNone) {
        const bool flat = mode == kRepackFlat;
        const size_t inner = round_up(flat ? conv_workspace_plain(n_layers, 1, C, 1, 1, B * P, Cout)
                                           : conv_workspace_plain(n_layers, B, C, 1, 1, P, Cout), 256);
        const size_t x_bytes = round_up(sizeof(float) * (size_t)B * C * P, 256);
        const size_t d_bytes = flat ? round_up(sizeof(float) * (size_t)B * Cout * P, 256) : 0;
        if (ws_bytes < inner + n_layers * (x_bytes + d_bytes)) return VGC_ERR_WORKSPACE;
        const float *xr[kMaxBatch], *dr[kMaxBatch];
        RepackJobs jobs = {};
        jobs.B = B;
        int n_jobs = 0;
        for (int l = 0; l < n_layers; ++l) {
            char *base = static_cast<char *>(ws) + inner + (size_t)l * (x_bytes + d_bytes);
            float *x_r = reinterpret_cast<float *>(base), *d_r = reinterpret_cast<float *>(base + x_bytes);
            jobs.job[n_jobs++] = RepackJob{x[l], x_r, C, H * W, W, Wo, P, sh, sw, flat ? 1 : 0, Wo};
            if (flat) jobs.job[n_jobs++] = RepackJob{delta[l], d_r, Cout, P, Wo, Wo, P, 1, 1, 1, Wo};
            xr[l] = x_r;
            dr[l] = flat ? d_r : delta[l];
        }
        sqgrad_repack<<<dim3(blocks_for((size_t)B * (flat && Cout > C ? Cout : C)), n_jobs), 256, 0, st>>>(jobs);
        count_launch();
        if (flat)
            return conv_group(n_layers, xr, dr, S, 1, C, B * P, 1, Cout, 1, 1, 1, 1, 0, 0, B * P, 1, scale, accumulate, ws,
                              inner, st);
        return conv_group(n_layers, xr, dr, S, B, C, Ho, Wo, Cout, 1, 1, 1, 1, 0, 0, Ho, Wo, scale, accumulate, ws, inner, st);
    }
    // which tiles TMA can deliver: rows of P positions with a 16-byte pitch, at least one slice long; the input
    // tile only when the im2col view is the tensor itself (1x1 kernel, stride 1, no padding)
    const bool err_tma = P >= kBK && P % 4 == 0;
    const bool in_tma = err_tma && Kh == 1 && Kw == 1 && sh == 1 && sw == 1 && ph == 0 && pw == 0;
    const int p_slices = (P + kBK - 1) / kBK;
    const int k_slices = B * p_slices;
    // three taps at a time: Kw = 3, stride 1 along w with pad 1 (then Wo == W), output width even, errors by TMA
    const int taps = (!in_tma && err_tma && Kw == 3 && sw == 1 && sh == 1 && pw == 1 && Wo == W && W % 2 == 0)
                         ? (W % 4 == 0 ? 4 : 2) : 0;
    // the same with stride 2 along w: W == 2 Wo, output width even
    const int taps_s2 = (!in_tma && err_tma && Kw == 3 && sw == 2 && pw == 1 && W == 2 * Wo && Wo % 2 == 0)
                            ? (Wo % 4 == 0 ? 4 : 2) : 0;
    // seven taps at a time: Kw = 7, stride 2, pad 3
    const bool taps7 = !in_tma && err_tma && Kw == 7 && sw == 2 && pw == 3 && W == 2 * Wo && Wo % 4 == 0;
    // with few output channels the roles are swapped -- except in the three-tap form, where keeping the errors as
    // the A operand (in tensor memory, half of its rows unused) measures faster than both operands in shared memory
    const bool swapped = conv_swapped(Cout, n_im2col) && !taps && !taps_s2 && !taps7;
    // both tiles by TMA: A in tensor memory, cross terms in bf16 (the per-example form keeps tf32 cross terms)
    const bool tma_bf = err_tma && in_tma && !t_exact;
    const int rows_err = swapped ? kBN : kBM, rows_in = swapped ? kBM : kBN;
    Batch bt = {};
    uint32_t tx_err = 0, tx_in = 0;
    for (int l = 0; l < n_layers; ++l) {
        CUtensorMap *m_err = swapped ? &bt.b[l] : &bt.a[l], *m_in = swapped ? &bt.a[l] : &bt.b[l];
        if (err_tma) {
            const cuuint32_t box[3] = {(cuuint32_t)kBK, (cuuint32_t)(Cout < rows_err ? Cout : rows_err), 1};
            const cuuint64_t dims[3] = {(cuuint64_t)P, (cuuint64_t)Cout, (cuuint64_t)B};
            const cuuint64_t str[2] = {(cuuint64_t)P * 4, (cuuint64_t)Cout * P * 4};
            if (!make_map(m_err, delta[l], 3, dims, str, box, CU_TENSOR_MAP_SWIZZLE_128B)) return VGC_ERR_CUDA;
            tx_err = box[1] * kBK * 4;
        }
        if (in_tma) {
            const cuuint32_t box[3] = {(cuuint32_t)kBK, (cuuint32_t)(C < rows_in ? C : rows_in), 1};
            const cuuint64_t dims[3] = {(cuuint64_t)P, (cuuint64_t)C, (cuuint64_t)B};
            const cuuint64_t str[2] = {(cuuint64_t)P * 4, (cuuint64_t)C * P * 4};
            if (!make_map(m_in, x[l], 3, dims, str, box, CU_TENSOR_MAP_SWIZZLE_128B)) return VGC_ERR_CUDA;
            tx_in = box[1] * kBK * 4;
        }
        bt.x[l] = x[l]; bt.delta[l] = delta[l]; bt.S[l] = S[l];
    }
    Params prm = {};
    prm.p_slices = p_slices; prm.tx_bytes = tx_err + tx_in; prm.scale = scale;
    prm.tx_bytes_a = swapped ? tx_in : tx_err; prm.accumulate = accumulate;
    prm.C = C; prm.H = H; prm.W = W; prm.Cout = Cout; prm.Kh = Kh; prm.Kw = Kw; prm.sh = sh; prm.sw = sw;
    prm.ph = ph; prm.pw = pw; prm.Wo = Wo; prm.P = P;
    prm.chw = C * H * W;
    prm.wo_magic = (unsigned)(0x100000000ull / (unsigned)Wo) + 1u;
    const bool ex = t_exact;
    const int unit = ex ? p_slices : 1;
    KernelFn fn = nullptr;
#define VGC_TC_FN(A, B_, AT) (ex ? (KernelFn)sqgrad_tc<kMajorK, A, B_, AT, true> : (KernelFn)sqgrad_tc<kMajorK, A, B_, AT, false>)
    if (!swapped) {     // S[o][idx]: m = o, n = idx
        prm.ld_m = n_im2col; prm.ld_n = 1;
        if (taps) fn = taps == 4 ? VGC_TC_FN(kTma, kGatherTaps4, true) : VGC_TC_FN(kTma, kGatherTaps2, true);
        else if (taps_s2) fn = taps_s2 == 4 ? VGC_TC_FN(kTma, kGatherTaps4S2, true) : VGC_TC_FN(kTma, kGatherTaps2S2, true);
        else if (taps7) fn = VGC_TC_FN(kTma, kGatherTaps7S2, true);
        else if (tma_bf) fn = sqgrad_tc<kMajorK, kTma, kTma, true, false, true>;
        else if (err_tma && in_tma) fn = sqgrad_tc<kMajorK, kTma, kTma, true, true>;
        else if (err_tma) fn = VGC_TC_FN(kTma, kGatherIm2col, true);
        else fn = VGC_TC_FN(kGatherErr, kGatherIm2col, false);
        return tc_launch(fn, bt, n_layers, prm, Cout, n_im2col, k_slices, ws, ws_bytes, st, unit);
    }
    prm.ld_m = 1; prm.ld_n = n_im2col;   // m = idx, n = o
    if (tma_bf) fn = sqgrad_tc<kMajorK, kTma, kTma, true, false, true>;
    else if (err_tma && in_tma) fn = sqgrad_tc<kMajorK, kTma, kTma, true, true>;
    else if (err_tma) fn = VGC_TC_FN(kGatherIm2col, kTma, false);
    else fn = VGC_TC_FN(kGatherIm2col, kGatherErr, false);
#undef VGC_TC_FN
    return tc_launch(fn, bt, n_layers, prm, n_im2col, Cout, k_slices, ws, ws_bytes, st, unit);
}

// n_layers layers of one geometry; x, delta, S are host arrays of device pointers
vgc_status tc_sqgrad_conv(int n_layers, const float *const *x, const float *const *delta, float *const *S, int B, int C,
                          int H, int W, int Cout, int Kh, int Kw, int sh, int sw, int ph, int pw, int Ho, int Wo,
                          float scale, int accumulate, void *ws, size_t ws_bytes, cudaStream_t st, bool exact)
{
    ExactScope scope(exact);
    for (int l0 = 0; l0 < n_layers; l0 += kMaxBatch) {
        const int nl = n_layers - l0 < kMaxBatch ? n_layers - l0 : kMaxBatch;
        const vgc_status rc = conv_group(nl, x + l0, delta + l0, S + l0, B, C, H, W, Cout, Kh, Kw, sh, sw, ph, pw, Ho, Wo,
                                         scale, accumulate, ws, ws_bytes, st);
        if (rc != VGC_OK) return rc;
    }
    return VGC_OK;
}

}  // namespace vgc
