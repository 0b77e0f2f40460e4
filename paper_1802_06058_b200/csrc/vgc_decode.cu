// vgc_decode_accumulate: the decode-and-sum half of CommunicateAndUpdate (Sec. 4.3).
//
// Every 32-bit word (index << 4 | sign << 3 | d) of W packed messages is expanded to
// (-1)^sign * 2^(E_k - d), E_k the per-tensor exponent that travels with the message
// (Sec. 4.2), scaled, and added into the dense update buffer.  One launch covers up to
// kMaxViews messages (their pointers travel in the kernel parameters, so nothing is
// allocated); blockIdx.y selects the message, the blocks of a row stride over its words.
// Words of one message are sorted by index, so a thread's four consecutive words almost
// always belong to one weight tensor and the tensor lookup is amortised.
#include <cstdlib>

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


// ------------------------------------------------------------------------------------------
// Segment-merge form (default).  Messages are sorted by index, so the words that fall into a
// contiguous range of u are a contiguous run of every message.  A block owns one range
// (a "chunk" of kChunkElems elements): one warp per message finds the run with a 32-ary search,
// then the block either
//   - scatters the few words of a sparse chunk straight into global memory (atomics), or
//   - walks the chunk in tiles: the tile of u is loaded into shared memory, the messages' words of
//     that tile are added to it one message after the other (plain read-modify-writes: indices
//     inside a message are distinct), and the tile is written back -- u is read and written once,
//     coalesced, however many words hit it, and the sum is formed in message order.
// ------------------------------------------------------------------------------------------
constexpr int kMergeTile = 8192;                 // elements of u per shared-memory tile (32 KB)
constexpr int kMergeWarps = kDecThreads / 32;

// first position in [0, count) whose index is >= bound (count if none); whole warp, 32-ary search
__device__ __forceinline__ uint32_t warp_lower_bound(const uint32_t *__restrict__ words, uint32_t count, uint32_t bound)
{
    const uint32_t lane = threadIdx.x & 31;
    uint32_t lo = 0, hi = count;      // every position < lo is below the bound, every position >= hi is not
    while (hi > lo) {
        const uint32_t step = (hi - lo) / 32 + 1;                 // 32 probes lo, lo+step, ... reach past hi
        const uint32_t pos = lo + step * lane;
        const bool below = pos < hi && (words[pos] >> 4) < bound;
        const uint32_t nb = __popc(__ballot_sync(0xffffffffu, below));   // sorted input: a prefix of the lanes
        if (nb == 0) { hi = lo; break; }
        const uint32_t new_hi = lo + step * nb;                   // first probe that is not below (or past hi)
        lo = lo + step * (nb - 1) + 1;
        hi = new_hi < hi ? new_hi : hi;
    }
    return lo;
}

__global__ void __launch_bounds__(kDecThreads)
decode_merge(const __grid_constant__ DecodeViews views, int W, const uint32_t *__restrict__ group_offsets, int K,
             float scale, float *__restrict__ u, size_t n, uint32_t chunk_elems, uint32_t *dev_status)
{
    __shared__ float tile[kMergeTile];
    __shared__ uint32_t sm_offs[kDecOffsSmem];
    __shared__ uint32_t run_begin[kMaxViews], run_end[kMaxViews];
    __shared__ uint32_t total_words;

    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool in_smem = (K + 1) <= kDecOffsSmem;
    if (in_smem)
        for (int i = threadIdx.x; i <= K; i += kDecThreads) sm_offs[i] = group_offsets[i];
    const uint32_t *offs = in_smem ? sm_offs : group_offsets;
    if (threadIdx.x == 0) total_words = 0;
    __syncthreads();

    const size_t lo = (size_t)blockIdx.x * chunk_elems;
    const size_t hi = lo + chunk_elems < n ? lo + chunk_elems : n;
    const bool last_chunk = hi == n;

    // ---- the run of every message inside [lo, hi)
    for (int w = warp; w < W; w += kMergeWarps) {
        const uint32_t *words = views.words[w];
        const uint32_t count = *views.nnz[w];
        const uint32_t b = warp_lower_bound(words, count, (uint32_t)lo);
        const uint32_t e = b + warp_lower_bound(words + b, count - b, (uint32_t)hi);
        if (lane == 0) {
            run_begin[w] = b;
            run_end[w] = e;
            atomicAdd(&total_words, e - b);
            if (last_chunk && e < count) atomicOr(dev_status, VGC_DEV_RANGE);      // indices >= n: skipped
        }
    }
    __syncthreads();
    const uint32_t total = total_words;
    if (total == 0) return;

    auto value_of = [&](uint32_t word, const int32_t *gexp, int &k) -> float {
        const uint32_t idx = word >> 4;
        if (idx < offs[k] || idx >= offs[k + 1]) k = group_of(offs, K, idx);
        const int32_t e = gexp[k] - (int32_t)(word & 7u);
        return __fmul_rn(scale, __uint_as_float(((uint32_t)(e + 127) << 23) | ((word & 8u) << 28)));
    };

    if ((size_t)total * 8 < hi - lo) {
        // ---- sparse chunk: not worth moving the whole range through shared memory
        for (int w = warp; w < W; w += kMergeWarps) {
            const uint32_t *words = views.words[w];
            const int32_t *gexp = views.group_exp[w];
            int k = 0;
            for (uint32_t i = run_begin[w] + lane; i < run_end[w]; i += 32) {
                const uint32_t word = words[i];
                atomicAdd(u + (word >> 4), value_of(word, gexp, k));
            }
        }
        return;
    }

    // ---- dense chunk: tile by tile through shared memory.  Messages are applied one after the other, in
    // message order, by the whole block: inside one message the indices are distinct, so plain
    // read-modify-writes suffice and every element sees its additions in the order w = 0, 1, ... --
    // the result does not depend on scheduling.
    __shared__ uint32_t cur[kMaxViews], t_end[kMaxViews];
    for (int w = threadIdx.x; w < W; w += kDecThreads) cur[w] = run_begin[w];
    __syncthreads();
    constexpr int kPre = 4;                          // words per thread and message held in registers
    constexpr int kGroup = 8;                        // messages whose words are in flight together
    for (size_t t0 = lo; t0 < hi; t0 += kMergeTile) {
        const uint32_t t_len = (uint32_t)(hi - t0 < kMergeTile ? hi - t0 : kMergeTile);
        const uint32_t t_hi = (uint32_t)(t0 + t_len);
        for (uint32_t i = threadIdx.x; i < t_len; i += kDecThreads) tile[i] = u[t0 + i];
        for (int w = warp; w < W; w += kMergeWarps) {        // where each message's run leaves this tile
            const uint32_t b = cur[w];
            const uint32_t e = b + warp_lower_bound(views.words[w] + b, run_end[w] - b, t_hi);
            if (lane == 0) t_end[w] = e;
        }
        __syncthreads();
        for (int w0 = 0; w0 < W; w0 += kGroup) {             // the words of kGroup messages are fetched together ...
            uint32_t held[kGroup][kPre];
#pragma unroll
            for (int g = 0; g < kGroup; ++g) {
                const int w = w0 + g < W ? w0 + g : W - 1;
                const uint32_t *words = views.words[w];
                const uint32_t b = cur[w], e = t_end[w];
#pragma unroll
                for (int j = 0; j < kPre; ++j) {
                    const uint32_t i = b + threadIdx.x + j * kDecThreads;
                    held[g][j] = i < e ? words[i] : 0u;
                }
            }
#pragma unroll
            for (int g = 0; g < kGroup; ++g) {                // ... and applied one message after the other
                const int w = w0 + g;
                if (w < W) {
                    const uint32_t *words = views.words[w];
                    const int32_t *gexp = views.group_exp[w];
                    const uint32_t b = cur[w], e = t_end[w];
                    int k = 0;
#pragma unroll
                    for (int j = 0; j < kPre; ++j)
                        if (b + threadIdx.x + j * kDecThreads < e)
                            tile[(held[g][j] >> 4) - (uint32_t)t0] += value_of(held[g][j], gexp, k);
                    for (uint32_t i = b + threadIdx.x + kPre * kDecThreads; i < e; i += kDecThreads) {
                        const uint32_t word = words[i];
                        tile[(word >> 4) - (uint32_t)t0] += value_of(word, gexp, k);
                    }
                }
                __syncthreads();
            }
        }
        for (uint32_t i = threadIdx.x; i < t_len; i += kDecThreads) u[t0 + i] = tile[i];
        for (int w = threadIdx.x; w < W; w += kDecThreads) cur[w] = t_end[w];
        __syncthreads();
    }
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
        const char *path = getenv("VGC_DECODE_PATH");
        if (path && path[0] == 's') {                        // per-word scatter (any word order)
            int per_msg = (sm_count * 8 + wb - 1) / wb;          // ~8 blocks per SM in total
            if (per_msg < 1) per_msg = 1;
            dim3 grid((unsigned)per_msg, (unsigned)wb);
            decode_scatter<<<grid, kDecThreads, 0, st>>>(views, group_offsets, K, scale, u, n, dev_status);
        } else {
            // one chunk per block, about four blocks per SM, whole tiles per chunk
            size_t chunk = (n + (size_t)sm_count * 4 - 1) / ((size_t)sm_count * 4);
            chunk = (chunk + kMergeTile - 1) / kMergeTile * kMergeTile;
            const unsigned blocks = (unsigned)((n + chunk - 1) / chunk);
            decode_merge<<<blocks, kDecThreads, 0, st>>>(views, wb, group_offsets, K, scale, u, n, (uint32_t)chunk,
                                                          dev_status);
        }
        count_launch();
    }
    VGC_CUDA_OK(cudaGetLastError());
    return VGC_OK;
}
