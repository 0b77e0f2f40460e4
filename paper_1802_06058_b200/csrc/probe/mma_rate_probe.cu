// Tensor-pipe rate probe (diagnostic, no counterpart in the paper): how long one tcgen05.mma instruction of a given
// shape occupies the tensor pipe of an SM.  The squared-gradient contraction is bounded by this figure, not by the
// nominal flop rate: an instruction with M = 128 takes the same time for N = 64 and N = 128, so the ceiling of a
// kernel depends on the instruction shape it can use.  `bench.py --mma-rates` prints the table.
// Not part of libvgc.so: built on request into libvgc_probe.so (paper_1802_06058_b200._build.build_probe) and loaded by
// the benchmark only.
//
// One CTA per block issues `reps` back-to-back MMAs (operands: zeros in shared / tensor memory, one accumulator),
// then commits and waits -- bounded -- for them to retire; the cycle count of block 0 and the event time of the
// launch are returned.
#include <cuda.h>

#include "vgc_common.cuh"

namespace vgc {

namespace probe {

constexpr uint32_t kWaitLimit = 1u << 24;
constexpr uint32_t kSmem = 16384 + 32768 + 1024;        // A tile (128 rows), B tile (256 rows), alignment

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }

// K-major tile with 128-byte rows and the 128-byte swizzle: 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr)
{
    uint64_t d = 0;
    d |= (uint64_t)((addr >> 4) & 0x3FFFu);
    d |= (uint64_t)(16u >> 4) << 16;
    d |= (uint64_t)(1024u >> 4) << 32;
    d |= 1ull << 46;
    d |= 2ull << 61;
    return d;
}

// kind: 0 = tf32 (8 k per instruction), 1 = bf16 (16 k); a_tmem: A operand from tensor memory instead of shared memory
__global__ void __launch_bounds__(128, 1) mma_rate(int kind, int a_tmem, int m, int n, int reps, long long *cycles, uint32_t *status)
{
    extern __shared__ uint8_t raw[];
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t tmem_slot;
    const uint32_t base = (smem_u32(raw) + 1023u) & ~1023u;
    uint32_t *tiles = reinterpret_cast<uint32_t *>(raw + (base - smem_u32(raw)));
    for (uint32_t i = threadIdx.x; i < (16384 + 32768) / 4; i += blockDim.x) tiles[i] = 0;
    const uint32_t warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bar)) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = tmem_slot;
    if (threadIdx.x == 0) {
        const uint32_t fmt = kind ? 1u : 2u;
        const uint32_t idesc = (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
        const uint64_t da = smem_desc(base), db = smem_desc(base + 16384);
        const long long t0 = clock64();
        for (int r = 0; r < reps; ++r) {
            const uint64_t dbk = db + (uint64_t)((r & 3) * 2);       // the four 32-byte k steps of a 128-byte row in turn
            if (kind) {
                if (a_tmem)
                    asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.u32 p, 1, 1;\n\t"
                                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                                 ::"r"(tmem), "r"(tmem + 480), "l"(dbk), "r"(idesc) : "memory");
                else
                    asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.u32 p, 1, 1;\n\t"
                                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                                 ::"r"(tmem), "l"(da), "l"(dbk), "r"(idesc) : "memory");
            } else {
                if (a_tmem)
                    asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.u32 p, 1, 1;\n\t"
                                 "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}"
                                 ::"r"(tmem), "r"(tmem + 480), "l"(dbk), "r"(idesc) : "memory");
                else
                    asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.u32 p, 1, 1;\n\t"
                                 "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
                                 ::"r"(tmem), "l"(da), "l"(dbk), "r"(idesc) : "memory");
            }
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&bar)) : "memory");
        bool done = false;
        for (uint32_t t = 0; t < kWaitLimit && !done; ++t) {
            uint32_t ok;
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                         : "=r"(ok) : "r"(smem_u32(&bar)), "r"(0u) : "memory");
            done = ok != 0;
        }
        const long long t1 = clock64();
        if (!done) atomicOr(status, VGC_DEV_TIMEOUT);
        if (blockIdx.x == 0) *cycles = t1 - t0;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
}

}  // namespace probe

}  // namespace vgc

// m: rows of the instruction, 128 (n a multiple of 16) or 64 (n a multiple of 8, A operand from shared memory)
extern "C" int vgc_probe_mma_rate(int kind, int a_tmem, int m, int n, int reps, int blocks, double *cycles_per_mma,
                                         double *tflops)
{
    using namespace vgc;
    if ((kind != 0 && kind != 1) || (m != 64 && m != 128) || (m == 64 && a_tmem) || n < 16 || n > 256 || n % 16 != 0 ||
        reps < 1 || reps > (1 << 20) || blocks < 1 || blocks > 4096 || !cycles_per_mma || !tflops)
        return VGC_ERR_INVALID_ARG;
    static bool configured = false;
    if (!configured) {
        VGC_CUDA_OK(cudaFuncSetAttribute(probe::mma_rate, cudaFuncAttributeMaxDynamicSharedMemorySize, probe::kSmem));
        configured = true;
    }
    long long *d_cycles = nullptr;
    VGC_CUDA_OK(cudaMalloc(&d_cycles, 16));
    uint32_t *d_status = reinterpret_cast<uint32_t *>(d_cycles + 1);
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    int rc = VGC_ERR_CUDA;
    float ms = 0.f;
    long long h[2] = {0, 0};
    if (cudaMemset(d_cycles, 0, 16) == cudaSuccess && cudaEventCreate(&e0) == cudaSuccess && cudaEventCreate(&e1) == cudaSuccess) {
        probe::mma_rate<<<blocks, 128, probe::kSmem>>>(kind, a_tmem, m, n, reps, d_cycles, d_status);   // warm-up
        cudaEventRecord(e0);
        probe::mma_rate<<<blocks, 128, probe::kSmem>>>(kind, a_tmem, m, n, reps, d_cycles, d_status);
        cudaEventRecord(e1);
        if (cudaDeviceSynchronize() == cudaSuccess && cudaEventElapsedTime(&ms, e0, e1) == cudaSuccess &&
            cudaMemcpy(h, d_cycles, 16, cudaMemcpyDeviceToHost) == cudaSuccess)
            rc = (uint32_t)h[1] ? VGC_ERR_CUDA : VGC_OK;
    }
    if (e0) cudaEventDestroy(e0);
    if (e1) cudaEventDestroy(e1);
    cudaFree(d_cycles);
    if (rc != VGC_OK) return rc;
    *cycles_per_mma = (double)h[0] / reps;
    *tflops = 2.0 * m * n * (kind ? 16.0 : 8.0) * reps * blocks / (ms * 1e-3) / 1e12;
    return VGC_OK;
}
