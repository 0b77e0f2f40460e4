// Squared per-example gradient sums on the 5th-generation tensor cores (tcgen05, sm_100a).
//
//   D[m][n] = sum_k A(k,m)^2 * B(k,n)^2          (the contraction behind Eq. 2 / Algorithm 1's
//                                                  "v_i +=" line; N_params*|B| multiply-adds, Sec. 5)
// Operands stay fp32 in global memory.  Per 32-deep k slice a thread block
//   1. TMA-loads the raw fp32 tiles of A (128 rows) and B (kBN rows) into shared memory
//      (128-byte swizzle, out-of-range parts filled with zeros),
//   2. squares every element in fp32 and splits the square into two TF32 numbers hi + lo
//      (hi = rna(x*x), lo = rna(x*x - hi)); the transform is elementwise, so the hi and lo tiles
//      inherit the swizzled layout the tensor core wants,
//   3. issues three tcgen05.mma per 8-deep step -- hi*hi, hi*lo, lo*hi -- into a TMEM
//      accumulator (the dropped lo*lo term is 2^-22 relative).
// The tensor core's fp32 accumulation is not trusted over long reductions: every kChunk k slices
// the accumulator is drained by four epilogue warps (tcgen05.ld) and added, round-to-nearest, to
// fp32 registers while the next chunk accumulates into the second TMEM buffer.
// Long reductions are split across blockIdx.z; partial tiles are combined in a fixed order.
//
// Operand layouts:
//   dense layer: A = delta[z][out], B = x[z][in]  (m / n innermost: MN-major tiles, both by TMA)
//   conv layer:  A = delta[z][o][p], p = (ho,wo) innermost (K-major); B is the im2col view of x,
//                row n = (c,kh,kw), column k = (z,ho,wo).  Each example contributes ceil(P/32) slices.
//                A tile: TMA when the row pitch P*4 is a multiple of 16 bytes, else gathered.
//                B tile: TMA for a 1x1 / stride 1 / unpadded kernel (then it is just x[z][c][p]);
//                otherwise the transform warps gather it straight from global memory, four
//                consecutive k per thread, zero outside the image -- im2col is never materialised.
//
// Warp roles (448 threads): 0 TMA producer, 1 MMA issuer + TMEM owner, 2-9 transform, 10-13 epilogue.
// Every wait on an mbarrier is bounded; on expiry the block raises an abort flag, all roles fall
// through to the common exit, outstanding TMA loads are waited for (bounded) and TMEM is freed.
#include <cuda.h>

#include <cstdlib>

#include "vgc_common.cuh"

namespace vgc {

namespace tc {

constexpr int kBM = 128;            // output rows per block (UMMA M)
constexpr int kBN = 128;            // output columns per block (UMMA N)
constexpr int kBK = 32;             // k per pipeline slice (= 128 bytes of fp32)
constexpr int kRawStages = 3;
constexpr int kOpStages = 2;
constexpr int kThreadsTc = 448;
constexpr int kTransformWarps = 8;
constexpr int kTransformThreads = 32 * kTransformWarps;
constexpr int kEpilogueWarps = 4;
constexpr uint32_t kRawBytesA = kBM * kBK * 4;                      // 16 KB
constexpr uint32_t kRawBytesB = kBN * kBK * 4;                      // 16 KB
constexpr uint32_t kRawStageBytes = kRawBytesA + kRawBytesB;        // 32 KB
constexpr uint32_t kOpStageBytes = 2 * kRawStageBytes;              // hi block then lo block
constexpr uint32_t kSmemBytes = kRawStages * kRawStageBytes + kOpStages * kOpStageBytes + 1024 /*align*/ + 256;
constexpr uint32_t kTmemCols = 2 * kBN;                             // two accumulator buffers
constexpr uint32_t kWaitLimit = 1u << 22;                           // polls before a wait gives up

enum { kMajorK = 0, kMajorMN = 1 };

struct Params {
    int M, N;
    int k_slices;            // total 32-deep slices of the reduction
    int slices_per_split;
    int p_slices;            // conv: slices per example (ceil(P/32)); dense: unused
    int chunk;               // slices per accumulator drain
    uint32_t tx_bytes;       // bytes the TMA loads of one slice deliver
    float scale;
    int accumulate;
    const float *x, *delta;  // raw operands (gathered tiles)
    int C, H, W, Cout, Kh, Kw, sh, sw, ph, pw, Wo, P;     // conv geometry (gathered tiles)
    float *S;                // final output [M][N] (used when gridDim.z == 1)
    float *partial;          // [gridDim.z][M][N] otherwise
    uint32_t *error_flag;    // device word, set to 1 if a wait expired
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
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t *abort_flag)
{
    for (uint32_t i = 0; i < kWaitLimit; ++i) {
        if (mbar_try(bar, parity)) return true;
        if (*abort_flag) return false;
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

__device__ __forceinline__ uint32_t to_tf32(float x)
{
    uint32_t r;
    asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
    return r;
}

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

// Instruction descriptor: D fp32, A and B tf32, given major-ness, M = 128, N = kBN.
__host__ __device__ constexpr uint32_t instr_desc(int major)
{
    return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)major << 15) | ((uint32_t)major << 16) |
           ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
}

// ---- the kernel ------------------------------------------------------------------------------
// One 16-byte chunk (4 consecutive k of one row) of a K-major 128-byte-swizzled tile.
__device__ __forceinline__ uint32_t chunk_offset(int row, int kq) { return (uint32_t)row * 128u + (uint32_t)((kq ^ (row & 7)) << 4); }

__device__ __forceinline__ void split_store(uint8_t *hi_tile, uint8_t *lo_tile, uint32_t off, float v0, float v1, float v2, float v3)
{
    const float q0 = __fmul_rn(v0, v0), q1 = __fmul_rn(v1, v1), q2 = __fmul_rn(v2, v2), q3 = __fmul_rn(v3, v3);
    uint4 h, l;
    h.x = to_tf32(q0); h.y = to_tf32(q1); h.z = to_tf32(q2); h.w = to_tf32(q3);
    l.x = to_tf32(__fsub_rn(q0, __uint_as_float(h.x)));
    l.y = to_tf32(__fsub_rn(q1, __uint_as_float(h.y)));
    l.z = to_tf32(__fsub_rn(q2, __uint_as_float(h.z)));
    l.w = to_tf32(__fsub_rn(q3, __uint_as_float(h.w)));
    *reinterpret_cast<uint4 *>(hi_tile + off) = h;
    *reinterpret_cast<uint4 *>(lo_tile + off) = l;
}

template <int kMajor, bool kGatherA, bool kGatherB>
__global__ void __launch_bounds__(kThreadsTc, 1)
sqgrad_tc(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b, const Params prm)
{
    static_assert(kMajor == kMajorK || (!kGatherA && !kGatherB), "gathered tiles are K-major");
    constexpr bool kAnyTma = !kGatherA || !kGatherB;
    extern __shared__ uint8_t smem_raw_[];
    __shared__ __align__(8) uint64_t bars[2 * kRawStages + 2 * kOpStages + 5];
    __shared__ uint32_t tmem_base_slot;
    __shared__ volatile uint32_t abort_flag;

    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (smem_u32(smem_raw_) + 1023u) & ~1023u;     // 1024-byte aligned tiles
    uint8_t *smem_gen = smem_raw_ + (smem_base - smem_u32(smem_raw_));
    const uint32_t raw_base = smem_base;
    const uint32_t op_base = smem_base + kRawStages * kRawStageBytes;

    uint64_t *raw_full = bars, *raw_empty = bars + kRawStages;
    uint64_t *op_full = bars + 2 * kRawStages, *op_empty = op_full + kOpStages;
    uint64_t *acc_full = op_empty + kOpStages, *acc_empty = acc_full + 2, *drain = acc_empty + 2;

    const int m0 = blockIdx.y * kBM, n0 = blockIdx.x * kBN;
    const int slice_begin = blockIdx.z * prm.slices_per_split;
    const int slice_end = min(prm.k_slices, slice_begin + prm.slices_per_split);
    const int n_slices = slice_end - slice_begin;                           // >= 1 by construction
    const int n_chunks = (n_slices + prm.chunk - 1) / prm.chunk;

    if (threadIdx.x == 0) {
        abort_flag = 0;
        for (int i = 0; i < kRawStages; ++i) { mbar_init(smem_u32(&raw_full[i]), 1); mbar_init(smem_u32(&raw_empty[i]), kTransformWarps); }
        for (int i = 0; i < kOpStages; ++i) { mbar_init(smem_u32(&op_full[i]), kTransformWarps); mbar_init(smem_u32(&op_empty[i]), 1); }
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

    if (warp == 0) {
        // ================= TMA producer (one thread) =================
        if (lane == 0 && kAnyTma) {
            int issued = 0;
            for (int i = 0; i < n_slices; ++i) {
                const int st = i % kRawStages;
                const uint32_t ph = (uint32_t)(i / kRawStages) & 1u;
                if (!mbar_wait(smem_u32(&raw_empty[st]), ph ^ 1u, &abort_flag)) break;
                const uint32_t full = smem_u32(&raw_full[st]);
                const uint32_t dst_a = raw_base + st * kRawStageBytes, dst_b = dst_a + kRawBytesA;
                mbar_expect_tx(full, prm.tx_bytes);
                const int slice = slice_begin + i;
                if (kMajor == kMajorK) {
                    const int z = slice / prm.p_slices, p0 = (slice - z * prm.p_slices) * kBK;
                    if (!kGatherA) tma_load_3d(dst_a, &map_a, full, p0, m0, z);
                    if (!kGatherB) tma_load_3d(dst_b, &map_b, full, p0, n0, z);
                } else {
                    const int k0 = slice * kBK;
#pragma unroll
                    for (int j = 0; j < kBM / 32; ++j) tma_load_2d(dst_a + j * 4096, &map_a, full, m0 + 32 * j, k0);
#pragma unroll
                    for (int j = 0; j < kBN / 32; ++j) tma_load_2d(dst_b + j * 4096, &map_b, full, n0 + 32 * j, k0);
                }
                issued = i + 1;
            }
            // on an abort: loads already issued must land before the block may exit
            if (abort_flag) {
                const int first = issued > kRawStages ? issued - kRawStages : 0;
                for (int i = first; i < issued; ++i) {
                    const uint32_t bar = smem_u32(&raw_full[i % kRawStages]);
                    const uint32_t ph = (uint32_t)(i / kRawStages) & 1u;
                    for (uint32_t t = 0; t < kWaitLimit && !mbar_try(bar, ph); ++t) {}
                }
            }
        }
    } else if (warp == 1) {
        // ================= MMA issuer (one thread) =================
        if (lane == 0) {
            constexpr uint32_t idesc = instr_desc(kMajor);
            // K-major: rows of 128 B, 8-row groups 1024 B apart (SBO); LBO unused.
            // MN-major: 32-wide column blocks 4096 B apart (LBO); 4-deep k groups 512 B apart (SBO).
            const uint32_t lbo = kMajor == kMajorK ? 16u : 4096u;
            const uint32_t sbo = kMajor == kMajorK ? 1024u : 512u;
            const uint32_t layout = kMajor == kMajorK ? 2u : 1u;
            const uint32_t k_step = kMajor == kMajorK ? 32u : 1024u;        // bytes per 8-deep MMA step
            int i = 0;
            bool ok = true;
            for (int c = 0; c < n_chunks && ok; ++c) {
                const int b = c & 1;
                ok = mbar_wait(smem_u32(&acc_empty[b]), ((uint32_t)(c >> 1) & 1u) ^ 1u, &abort_flag);
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)b * kBN;
                const int chunk_end = min(n_slices, (c + 1) * prm.chunk);
                for (bool first = true; i < chunk_end; ++i) {
                    const int st = i % kOpStages;
                    ok = mbar_wait(smem_u32(&op_full[st]), (uint32_t)(i / kOpStages) & 1u, &abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t hi_a = op_base + st * kOpStageBytes, hi_b = hi_a + kRawBytesA;
                    const uint32_t lo_a = hi_a + kRawStageBytes, lo_b = lo_a + kRawBytesA;
#pragma unroll
                    for (int kk = 0; kk < kBK / 8; ++kk) {
                        const uint64_t da_hi = smem_desc(hi_a + kk * k_step, lbo, sbo, layout);
                        const uint64_t db_hi = smem_desc(hi_b + kk * k_step, lbo, sbo, layout);
                        const uint64_t da_lo = smem_desc(lo_a + kk * k_step, lbo, sbo, layout);
                        const uint64_t db_lo = smem_desc(lo_b + kk * k_step, lbo, sbo, layout);
                        tc_mma_tf32(d_tmem, da_hi, db_hi, idesc, first ? 0u : 1u);
                        tc_mma_tf32(d_tmem, da_hi, db_lo, idesc, 1u);
                        tc_mma_tf32(d_tmem, da_lo, db_hi, idesc, 1u);
                        first = false;
                    }
                    tc_commit(smem_u32(&op_empty[st]));           // operand slot free once these MMAs retire
                }
                if (ok) tc_commit(smem_u32(&acc_full[b]));
            }
            if (!ok) {      // abort: MMAs already issued must retire before TMEM is freed
                tc_commit(smem_u32(drain));
                for (uint32_t t = 0; t < kWaitLimit && !mbar_try(smem_u32(drain), 0); ++t) {}
            }
        }
    } else if (warp < 2 + kTransformWarps) {
        // ================= transform warps: square and split into TF32 hi / lo =================
        const int t = (int)threadIdx.x - 64;                               // 0..255
        const int kq = t & 7, row0 = t >> 3;                               // gathered chunks: rows row0 + 32*i, k = 4*kq..4*kq+3
        constexpr int kRowsPerThread = kBM * 8 / kTransformThreads;        // 4

        // ---- per-thread constants of the gathered tiles
        int b_base[kRowsPerThread], b_dh[kRowsPerThread], b_dw[kRowsPerThread];
        bool b_ok[kRowsPerThread], a_ok[kRowsPerThread];
        int ho[4], wo[4];                    // output position of this thread's four k in the current slice
        int ho_init[4], wo_init[4];
        int q32 = 0, r32 = 0;
        int z = 0, pblk = 0;
        if (kGatherA || kGatherB) {
            const int khw = prm.Kh * prm.Kw;
#pragma unroll
            for (int i = 0; i < kRowsPerThread; ++i) {
                const int n = n0 + row0 + 32 * i;
                b_ok[i] = n < prm.N;
                const int nn = b_ok[i] ? n : 0;
                const int c = nn / khw, rem = nn - c * khw;
                const int kh = rem / prm.Kw, kw = rem - kh * prm.Kw;
                b_dh[i] = kh - prm.ph;
                b_dw[i] = kw - prm.pw;
                b_base[i] = (c * prm.H + b_dh[i]) * prm.W + b_dw[i];
                a_ok[i] = m0 + row0 + 32 * i < prm.M;
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                ho_init[j] = (kq * 4 + j) / prm.Wo;
                wo_init[j] = (kq * 4 + j) - ho_init[j] * prm.Wo;
            }
            q32 = kBK / prm.Wo;
            r32 = kBK - q32 * prm.Wo;
            z = slice_begin / prm.p_slices;
            pblk = slice_begin - z * prm.p_slices;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int p = pblk * kBK + kq * 4 + j;
                ho[j] = p / prm.Wo;
                wo[j] = p - ho[j] * prm.Wo;
            }
        }
        float va[kGatherA ? kRowsPerThread : 1][4], vb[kGatherB ? kRowsPerThread : 1][4];

        // loads of the gathered chunks of the slice the (z, pblk, ho, wo) state points at
        auto gather = [&](float (&ga)[kGatherA ? kRowsPerThread : 1][4], float (&gb)[kGatherB ? kRowsPerThread : 1][4]) {
            const int pbase = pblk * kBK + kq * 4;
            if (kGatherB) {
                const float *xz = prm.x + (size_t)z * prm.C * prm.H * prm.W;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const bool pv = pbase + j < prm.P;
                    const int hs = ho[j] * prm.sh, ws = wo[j] * prm.sw;
                    const int poff = hs * prm.W + ws;
#pragma unroll
                    for (int i = 0; i < kRowsPerThread; ++i) {
                        const bool ok = pv && b_ok[i] && (unsigned)(hs + b_dh[i]) < (unsigned)prm.H &&
                                        (unsigned)(ws + b_dw[i]) < (unsigned)prm.W;
                        gb[i][j] = ok ? __ldg(xz + (b_base[i] + poff)) : 0.f;
                    }
                }
            }
            if (kGatherA) {
#pragma unroll
                for (int i = 0; i < kRowsPerThread; ++i) {
                    const float *dr = prm.delta + ((size_t)z * prm.Cout + (m0 + row0 + 32 * i)) * prm.P + pbase;
#pragma unroll
                    for (int j = 0; j < 4; ++j) ga[i][j] = (a_ok[i] && pbase + j < prm.P) ? __ldg(dr + j) : 0.f;
                }
            }
        };
        auto advance = [&]() {
            if (++pblk == prm.p_slices) {
                pblk = 0;
                ++z;
#pragma unroll
                for (int j = 0; j < 4; ++j) { ho[j] = ho_init[j]; wo[j] = wo_init[j]; }
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    ho[j] += q32;
                    wo[j] += r32;
                    if (wo[j] >= prm.Wo) { wo[j] -= prm.Wo; ++ho[j]; }
                }
            }
        };

        if (kGatherA || kGatherB) gather(va, vb);
        for (int i = 0; i < n_slices; ++i) {
            const int rs = i % kRawStages, os = i % kOpStages;
            float wa[kGatherA ? kRowsPerThread : 1][4], wb[kGatherB ? kRowsPerThread : 1][4];
            if ((kGatherA || kGatherB) && i + 1 < n_slices) {           // next slice's loads fly during this transform
                advance();
                gather(wa, wb);
            }
            if (kAnyTma && !mbar_wait(smem_u32(&raw_full[rs]), (uint32_t)(i / kRawStages) & 1u, &abort_flag)) break;
            if (!mbar_wait(smem_u32(&op_empty[os]), ((uint32_t)(i / kOpStages) & 1u) ^ 1u, &abort_flag)) break;
            uint8_t *raw = smem_gen + rs * kRawStageBytes;
            uint8_t *hi = smem_gen + kRawStages * kRawStageBytes + os * kOpStageBytes;
            uint8_t *lo = hi + kRawStageBytes;
            // tiles that came by TMA: elementwise over their 16-byte chunks (layout is inherited)
            {
                const uint32_t c_begin = kGatherA ? kRawBytesA / 16 : 0;
                const uint32_t c_end = kGatherB ? kRawBytesA / 16 : kRawStageBytes / 16;
#pragma unroll 4
                for (uint32_t c = c_begin + (uint32_t)t; c < c_end; c += kTransformThreads) {
                    const float4 v = *reinterpret_cast<const float4 *>(raw + 16 * c);
                    split_store(hi, lo, 16 * c, v.x, v.y, v.z, v.w);
                }
            }
            if (kGatherA) {
#pragma unroll
                for (int r = 0; r < kRowsPerThread; ++r)
                    split_store(hi, lo, chunk_offset(row0 + 32 * r, kq), va[r][0], va[r][1], va[r][2], va[r][3]);
            }
            if (kGatherB) {
#pragma unroll
                for (int r = 0; r < kRowsPerThread; ++r)
                    split_store(hi + kRawBytesA, lo + kRawBytesA, chunk_offset(row0 + 32 * r, kq), vb[r][0], vb[r][1],
                                vb[r][2], vb[r][3]);
            }
            fence_async_smem();                                   // generic-proxy writes -> tensor core reads
            __syncwarp();
            if (lane == 0) {
                mbar_arrive(smem_u32(&op_full[os]));
                if (kAnyTma) mbar_arrive(smem_u32(&raw_empty[rs]));
            }
            if (kGatherA) {
#pragma unroll
                for (int r = 0; r < kRowsPerThread; ++r)
#pragma unroll
                    for (int j = 0; j < 4; ++j) va[r][j] = wa[r][j];
            }
            if (kGatherB) {
#pragma unroll
                for (int r = 0; r < kRowsPerThread; ++r)
#pragma unroll
                    for (int j = 0; j < 4; ++j) vb[r][j] = wb[r][j];
            }
        }
    } else {
        // ================= epilogue warps: drain chunks, accumulate in fp32 registers =================
        const uint32_t q = warp & 3;                                      // TMEM lane quarter of this warp
        float acc[kBN];
#pragma unroll
        for (int j = 0; j < kBN; ++j) acc[j] = 0.f;
        bool ok = true;
        for (int c = 0; c < n_chunks && ok; ++c) {
            const int b = c & 1;
            ok = mbar_wait(smem_u32(&acc_full[b]), (uint32_t)(c >> 1) & 1u, &abort_flag);
            if (!ok) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((q * 32u) << 16) + (uint32_t)b * kBN;
#pragma unroll
            for (int j0 = 0; j0 < kBN; j0 += 32) {
                uint32_t r[32];
                tc_ld_32x32(taddr + j0, r);
                tc_wait_ld();
#pragma unroll
                for (int j = 0; j < 32; ++j) acc[j0 + j] = __fadd_rn(acc[j0 + j], __uint_as_float(r[j]));
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&acc_empty[b]));
        }
        if (ok) {
            const int m = m0 + (int)(q * 32u + lane);
            if (m < prm.M) {
                const bool direct = gridDim.z == 1;
                float *row = direct ? prm.S + (size_t)m * prm.N : prm.partial + ((size_t)blockIdx.z * prm.M + m) * prm.N;
                const int n_valid = min(kBN, prm.N - n0);
                if (direct) {
#pragma unroll
                    for (int j = 0; j < kBN; ++j)
                        if (j < n_valid) {
                            const float res = __fmul_rn(prm.scale, acc[j]);
                            row[n0 + j] = prm.accumulate ? __fadd_rn(row[n0 + j], res) : res;
                        }
                } else {
#pragma unroll
                    for (int j = 0; j < kBN; ++j)
                        if (j < n_valid) row[n0 + j] = acc[j];
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
    if (threadIdx.x == 0 && abort_flag) atomicExch(prm.error_flag, 1u);
}

// combine split-K partial tiles in a fixed order
__global__ void __launch_bounds__(256)
sqgrad_tc_combine(const float *__restrict__ partial, int splits, size_t mn, float scale, int accumulate,
                  float *__restrict__ S)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= mn) return;
    float sum = 0.f;
    for (int z = 0; z < splits; ++z) sum = __fadd_rn(sum, partial[(size_t)z * mn + i]);
    const float res = __fmul_rn(scale, sum);
    S[i] = accumulate ? __fadd_rn(S[i], res) : res;
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
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, (cuuint32_t)rank, const_cast<float *>(base), dims, strides_bytes, box,
              elem_strides, CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static int default_chunk()
{
    static int chunk = 0;
    if (!chunk) {
        const char *e = getenv("VGC_TC_CHUNK");
        chunk = e ? atoi(e) : 4;
        if (chunk < 1) chunk = 1;
    }
    return chunk;
}

struct Plan {
    int splits, slices_per_split, k_slices;
};

static Plan make_plan(int M, int N, int k_slices)
{
    const long tiles = (long)((M + kBM - 1) / kBM) * ((N + kBN - 1) / kBN);
    long want = (148 + tiles - 1) / tiles;                 // fill the SMs once
    if (want > k_slices) want = k_slices;
    if (want < 1) want = 1;
    Plan p;
    p.k_slices = k_slices;
    p.slices_per_split = (int)((k_slices + want - 1) / want);
    p.splits = (k_slices + p.slices_per_split - 1) / p.slices_per_split;
    return p;
}

}  // namespace tc

using namespace tc;

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

size_t tc_workspace_bytes(int M, int N, int k_slices)
{
    const Plan p = make_plan(M, N, k_slices);
    return 256 + (p.splits > 1 ? (size_t)p.splits * M * N * sizeof(float) : 0);
}

enum Variant { kDense, kConvTmaTma, kConvTmaGather, kConvGatherGather };

static vgc_status tc_launch(Variant variant, const CUtensorMap &ma, const CUtensorMap &mb, Params prm, int M, int N,
                            int k_slices, void *ws, size_t ws_bytes, cudaStream_t st)
{
    const Plan plan = make_plan(M, N, k_slices);
    if (ws_bytes < tc_workspace_bytes(M, N, k_slices)) return VGC_ERR_WORKSPACE;
    static bool attr_set = false;
    if (!attr_set) {
        VGC_CUDA_OK(cudaFuncSetAttribute(sqgrad_tc<kMajorMN, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
        VGC_CUDA_OK(cudaFuncSetAttribute(sqgrad_tc<kMajorK, false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
        VGC_CUDA_OK(cudaFuncSetAttribute(sqgrad_tc<kMajorK, false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
        VGC_CUDA_OK(cudaFuncSetAttribute(sqgrad_tc<kMajorK, true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes));
        attr_set = true;
    }
    prm.M = M; prm.N = N; prm.k_slices = k_slices; prm.slices_per_split = plan.slices_per_split;
    prm.chunk = default_chunk();
    prm.error_flag = static_cast<uint32_t *>(ws);
    prm.partial = reinterpret_cast<float *>(static_cast<char *>(ws) + 256);
    VGC_CUDA_OK(cudaMemsetAsync(ws, 0, 4, st));
    dim3 grid((N + kBN - 1) / kBN, (M + kBM - 1) / kBM, plan.splits);
    switch (variant) {
        case kDense: sqgrad_tc<kMajorMN, false, false><<<grid, kThreadsTc, kSmemBytes, st>>>(ma, mb, prm); break;
        case kConvTmaTma: sqgrad_tc<kMajorK, false, false><<<grid, kThreadsTc, kSmemBytes, st>>>(ma, mb, prm); break;
        case kConvTmaGather: sqgrad_tc<kMajorK, false, true><<<grid, kThreadsTc, kSmemBytes, st>>>(ma, mb, prm); break;
        case kConvGatherGather: sqgrad_tc<kMajorK, true, true><<<grid, kThreadsTc, kSmemBytes, st>>>(ma, mb, prm); break;
    }
    count_launch();
    if (plan.splits > 1) {
        const size_t mn = (size_t)M * N;
        sqgrad_tc_combine<<<(unsigned)((mn + 255) / 256), 256, 0, st>>>(prm.partial, plan.splits, mn, prm.scale,
                                                                         prm.accumulate, prm.S);
        count_launch();
    }
    return cudaGetLastError() == cudaSuccess ? VGC_OK : VGC_ERR_CUDA;
}

size_t tc_linear_workspace_bytes(int B, int in, int out) { return tc_workspace_bytes(out, in, (B + kBK - 1) / kBK); }

vgc_status tc_sqgrad_linear(const float *x, const float *delta, int B, int in, int out, float scale, int accumulate,
                            float *S, void *ws, size_t ws_bytes, cudaStream_t st)
{
    CUtensorMap ma, mb;
    const cuuint32_t box[2] = {32, (cuuint32_t)kBK};
    const cuuint64_t dims_a[2] = {(cuuint64_t)out, (cuuint64_t)B}, str_a[1] = {(cuuint64_t)out * 4};
    const cuuint64_t dims_b[2] = {(cuuint64_t)in, (cuuint64_t)B}, str_b[1] = {(cuuint64_t)in * 4};
    if (!make_map(&ma, delta, 2, dims_a, str_a, box, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B) ||
        !make_map(&mb, x, 2, dims_b, str_b, box, CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B))
        return VGC_ERR_CUDA;
    Params prm = {};
    prm.p_slices = 1; prm.tx_bytes = kRawStageBytes; prm.scale = scale; prm.accumulate = accumulate; prm.S = S;
    return tc_launch(kDense, ma, mb, prm, out, in, (B + kBK - 1) / kBK, ws, ws_bytes, st);
}

size_t tc_conv_workspace_bytes(int B, int C, int Kh, int Kw, int P, int Cout)
{
    return tc_workspace_bytes(Cout, C * Kh * Kw, B * ((P + kBK - 1) / kBK));
}

vgc_status tc_sqgrad_conv(const float *x, const float *delta, int B, int C, int H, int W, int Cout, int Kh, int Kw,
                          int sh, int sw, int ph, int pw, int Ho, int Wo, float scale, int accumulate, float *S,
                          void *ws, size_t ws_bytes, cudaStream_t st)
{
    const int P = Ho * Wo, N = C * Kh * Kw;
    const int p_slices = (P + kBK - 1) / kBK;
    const bool a_tma = P >= kBK && P % 4 == 0;
    const bool b_tma = a_tma && Kh == 1 && Kw == 1 && sh == 1 && sw == 1 && ph == 0 && pw == 0;
    CUtensorMap ma = {}, mb = {};
    uint32_t tx = 0;
    if (a_tma) {
        const cuuint32_t box_a[3] = {(cuuint32_t)kBK, (cuuint32_t)(Cout < kBM ? Cout : kBM), 1};
        const cuuint64_t dims_a[3] = {(cuuint64_t)P, (cuuint64_t)Cout, (cuuint64_t)B};
        const cuuint64_t str_a[2] = {(cuuint64_t)P * 4, (cuuint64_t)Cout * P * 4};
        if (!make_map(&ma, delta, 3, dims_a, str_a, box_a, CU_TENSOR_MAP_SWIZZLE_128B)) return VGC_ERR_CUDA;
        tx += box_a[1] * kBK * 4;
    }
    if (b_tma) {
        const cuuint32_t box_b[3] = {(cuuint32_t)kBK, (cuuint32_t)(C < kBN ? C : kBN), 1};
        const cuuint64_t dims_b[3] = {(cuuint64_t)P, (cuuint64_t)C, (cuuint64_t)B};
        const cuuint64_t str_b[2] = {(cuuint64_t)P * 4, (cuuint64_t)C * P * 4};
        if (!make_map(&mb, x, 3, dims_b, str_b, box_b, CU_TENSOR_MAP_SWIZZLE_128B)) return VGC_ERR_CUDA;
        tx += box_b[1] * kBK * 4;
    }
    Params prm = {};
    prm.p_slices = p_slices; prm.tx_bytes = tx; prm.scale = scale; prm.accumulate = accumulate; prm.S = S;
    prm.x = x; prm.delta = delta;
    prm.C = C; prm.H = H; prm.W = W; prm.Cout = Cout; prm.Kh = Kh; prm.Kw = Kw; prm.sh = sh; prm.sw = sw;
    prm.ph = ph; prm.pw = pw; prm.Wo = Wo; prm.P = P;
    const Variant v = b_tma ? kConvTmaTma : (a_tma ? kConvTmaGather : kConvGatherGather);
    return tc_launch(v, ma, mb, prm, Cout, N, B * p_slices, ws, ws_bytes, st);
}

}  // namespace vgc
