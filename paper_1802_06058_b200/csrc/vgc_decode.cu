// vgc_decode_accumulate: the decode-and-sum half of CommunicateAndUpdate (Sec. 4.3).
//
// Every 32-bit word (index << 4 | sign << 3 | d) of W packed messages is expanded to
// (-1)^sign * 2^(E_k - d), E_k the per-tensor exponent that travels with the message
// (Sec. 4.2), scaled, and added into the dense update buffer.  One launch covers up to
// kMaxViews messages (their pointers travel in the kernel parameters, so nothing is
// allocated); blockIdx.y selects the message, the blocks of a row stride over its words.
// Words of one message are sorted by index, so a thread's four consecutive words almost
// always belong to one weight tensor and the tensor lookup is amortised.
#include "vgc_common.cuh"

namespace vgc {

constexpr int kDecThreads = 256;
constexpr int kMaxViews = 64;
constexpr int kDecOffsSmem = 1024;

struct DecodeViews {
    const uint32_t *words[kMaxViews];
    const uint32_t *nnz[kMaxViews];
    const int32_t *group_exp[kMaxViews];
};

__device__ __forceinline__ void decode_one(uint32_t word, const uint32_t *offs, const int32_t *gexp, int K,
                                           int &k, float scale, float *u, size_t n, bool &bad)
{
    const uint32_t idx = word >> 4;
    if (idx >= n) { bad = true; return; }
    if (idx < offs[k] || idx >= offs[k + 1]) k = group_of(offs, K, idx);
    const int32_t e = gexp[k] - (int32_t)(word & 7u);
    const float value = __uint_as_float(((uint32_t)(e + 127) << 23) | ((word & 8u) << 28));
    atomicAdd(u + idx, __fmul_rn(scale, value));
}

__global__ void __launch_bounds__(kDecThreads)
decode_scatter(const __grid_constant__ DecodeViews views, const uint32_t *__restrict__ group_offsets, int K,
               float scale, float *__restrict__ u, size_t n, uint32_t *dev_status)
{
    __shared__ uint32_t sm_offs[kDecOffsSmem];
    __shared__ int32_t sm_exp[kDecOffsSmem];
    const int w = blockIdx.y;
    const uint32_t *__restrict__ words = views.words[w];
    const uint32_t count = *views.nnz[w];
    const bool in_smem = (K + 1) <= kDecOffsSmem;
    if (in_smem) {
        for (int i = threadIdx.x; i <= K; i += kDecThreads) sm_offs[i] = group_offsets[i];
        for (int i = threadIdx.x; i < K; i += kDecThreads) sm_exp[i] = views.group_exp[w][i];
        __syncthreads();
    }
    const uint32_t *offs = in_smem ? sm_offs : group_offsets;
    const int32_t *gexp = in_smem ? sm_exp : views.group_exp[w];

    bool bad = false;
    int k = 0;
    const bool vec_ok = (reinterpret_cast<uintptr_t>(words) & 15u) == 0;
    const uint32_t n_vec = vec_ok ? count / 4 : 0;
    for (uint32_t q = blockIdx.x * kDecThreads + threadIdx.x; q < n_vec; q += gridDim.x * kDecThreads) {
        const uint4 w4 = *reinterpret_cast<const uint4 *>(words + 4 * (size_t)q);
        decode_one(w4.x, offs, gexp, K, k, scale, u, n, bad);
        decode_one(w4.y, offs, gexp, K, k, scale, u, n, bad);
        decode_one(w4.z, offs, gexp, K, k, scale, u, n, bad);
        decode_one(w4.w, offs, gexp, K, k, scale, u, n, bad);
    }
    for (uint32_t q = 4 * n_vec + blockIdx.x * kDecThreads + threadIdx.x; q < count; q += gridDim.x * kDecThreads)
        decode_one(words[q], offs, gexp, K, k, scale, u, n, bad);
    if (bad) atomicOr(dev_status, VGC_DEV_RANGE);
}

}  // namespace vgc

using namespace vgc;

extern "C" vgc_status vgc_decode_accumulate(const vgc_message_view *msgs, int W,
                                            const uint32_t *group_offsets, int K, float scale,
                                            float *u, size_t n, uint32_t *dev_status, vgc_stream_t stream)
{
    if (W == 0 || n == 0) return VGC_OK;
    if (W < 0 || K < 1 || n > VGC_MAX_PARAMS || !msgs || !group_offsets || !u || !dev_status)
        return VGC_ERR_INVALID_ARG;
    if (!(scale == scale)) return VGC_ERR_INVALID_ARG;
    for (int w = 0; w < W; ++w)
        if (!msgs[w].words || !msgs[w].nnz || !msgs[w].group_exp) return VGC_ERR_INVALID_ARG;

    static int sm_count = 0;
    if (sm_count == 0) {
        int dev = 0, c = 0;
        VGC_CUDA_OK(cudaGetDevice(&dev));
        VGC_CUDA_OK(cudaDeviceGetAttribute(&c, cudaDevAttrMultiProcessorCount, dev));
        sm_count = c > 0 ? c : 148;
    }
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    for (int w0 = 0; w0 < W; w0 += kMaxViews) {
        const int wb = W - w0 < kMaxViews ? W - w0 : kMaxViews;
        DecodeViews views;
        for (int w = 0; w < kMaxViews; ++w) {
            const vgc_message_view &m = msgs[w0 + (w < wb ? w : 0)];
            views.words[w] = m.words;
            views.nnz[w] = m.nnz;
            views.group_exp[w] = m.group_exp;
        }
        int per_msg = (sm_count * 8 + wb - 1) / wb;          // ~8 blocks per SM in total
        if (per_msg < 1) per_msg = 1;
        dim3 grid((unsigned)per_msg, (unsigned)wb);
        decode_scatter<<<grid, kDecThreads, 0, st>>>(views, group_offsets, K, scale, u, n, dev_status);
        count_launch();
    }
    VGC_CUDA_OK(cudaGetLastError());
    return VGC_OK;
}
