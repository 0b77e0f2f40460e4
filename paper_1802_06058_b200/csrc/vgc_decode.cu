// vgc_decode_accumulate / vgc_decode_sum: the decode-and-sum half of CommunicateAndUpdate (Sec. 4.3).
//
// Every 32-bit word (index << 4 | sign << 3 | d) of W packed messages is expanded to
// (-1)^sign * 2^(E_k - d), E_k the per-tensor exponent that travels with the message (Sec. 4.2),
// scaled, and added into the dense update buffer.  One launch covers up to kMaxViews messages (their
// pointers travel in the kernel parameters, so nothing is allocated).
//
// Messages are sorted by index, so the words that fall into a contiguous range of u are a contiguous run of
// every message.  A block owns one range of u; one warp per message finds where the run enters it (32-ary
// search).  Then, per call:
//   sparse (fewer than one word per eight elements): the block's words are added straight into global memory
//     with fp32 atomics -- u is touched only where a word points;
//   dense: every WARP owns a contiguous part of the block's range and walks it in sub-tiles of a few hundred
//     elements held in shared memory.  For a sub-tile it looks at the next words of every message (a window of
//     32 - 128 words per message, all windows of eight messages in flight together), adds those that fall into the
//     sub-tile -- message after message, so an element receives its additions in the order w = 0, 1, ..., the
//     fp32 sequence of a sequential sum, whatever the scheduling -- advances the message cursors past them and
//     writes the sub-tile out.  u is read and written once, coalesced; there is no block-wide barrier and no
//     search inside the loop: a warp's cursors simply move forward with its range.
// kOverwrite: the range starts from zero instead of the old contents of u (u = scale * sum of the messages).
// kHybrid: messages of the hybrid algorithm (Algorithm 2) -- every word stands for +-tau, no exponents.
#include "vgc_common.cuh"

namespace vgc {

constexpr int kMaxViews = 64;
constexpr int kDecOffsSmem = 1024;
constexpr int kTileThreads = 512;
constexpr int kTileWarps = kTileThreads / 32;
constexpr int kSubMax = 1280;                    // largest sub-tile of a warp (elements; 5 KB -- two blocks per SM fit)
constexpr int kSubMin = 256;
constexpr int kGroup = 8;                        // messages whose windows are in flight together
constexpr int kWinMax = 4;                       // 32-word loads per lane and window

struct DecodeViews {
    const uint32_t *words[kMaxViews];
    const uint32_t *nnz[kMaxViews];
    const int32_t *group_exp[kMaxViews];
    uint32_t max_words[kMaxViews];
};

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

template <bool kHybrid, bool kOverwrite>
__global__ void __launch_bounds__(kTileThreads, 2)
decode_tiles(const __grid_constant__ DecodeViews views, int W, const uint32_t *__restrict__ group_offsets, int K,
             float scale, float tau, float *__restrict__ u, size_t n, uint32_t chunk_elems, uint32_t *dev_status)
{
    extern __shared__ __align__(16) float tiles[];               // kTileWarps sub-tiles of kSubMax floats
    __shared__ uint32_t sm_offs[kDecOffsSmem];
    __shared__ uint32_t cur[kMaxViews];                          // where each message's run enters the block's range
    __shared__ uint32_t wcur[kTileWarps][kMaxViews];             // per warp: its cursor into each message
    __shared__ float lut[kTileWarps][kGroup * 16];
    __shared__ uint32_t total_words;
    // the messages' pointers, copied out of the kernel parameters once: parameters cannot be indexed with a
    // run-time value (the compiler turns such an access into a chain of selects over all kMaxViews entries)
    __shared__ const uint32_t *sm_words[kMaxViews];
    __shared__ const int32_t *sm_gexp[kMaxViews];
    __shared__ uint32_t sm_count[kMaxViews];

    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool in_smem = !kHybrid && (K + 1) <= kDecOffsSmem;
    if (in_smem)
        for (int i = tid; i <= K; i += kTileThreads) sm_offs[i] = group_offsets[i];
    const uint32_t *offs = in_smem ? sm_offs : group_offsets;
    if (tid == 0) total_words = 0;
    if (tid < (uint32_t)W) {
        sm_words[tid] = views.words[tid];
        sm_gexp[tid] = views.group_exp[tid];
        // never read past the buffer the caller says it has: a truncated message (VGC_DEV_CAPACITY at the sender)
        // carries the count that was needed, not the count that was written
        const uint32_t said = *views.nnz[tid], have = views.max_words[tid];
        sm_count[tid] = said < have ? said : have;
        if (said > have && blockIdx.x == 0) atomicOr(dev_status, VGC_DEV_CAPACITY);
    }
    __syncthreads();

    const size_t lo = (size_t)blockIdx.x * chunk_elems;
    const size_t hi = lo + chunk_elems < n ? lo + chunk_elems : n;
    const bool last_chunk = hi == n;

    for (int w = warp; w < W; w += kTileWarps) {
        const uint32_t *words = sm_words[w];
        const uint32_t count = sm_count[w];
        const uint32_t b = warp_lower_bound(words, count, (uint32_t)lo);
        if (lane == 0) {
            cur[w] = b;
            atomicAdd(&total_words, count);
            if (last_chunk && count && (words[count - 1] >> 4) >= n) atomicOr(dev_status, VGC_DEV_RANGE);   // skipped
        }
    }
    __syncthreads();
    const uint32_t total = total_words;
    if (total == 0 && !kOverwrite) return;

    bool bad = false;                                           // a word out of place: skipped, reported
    auto value_of = [&](uint32_t word, const int32_t *gexp, int &k) -> float {
        if (kHybrid) return __fmul_rn(scale, (word & 8u) ? -tau : tau);
        const uint32_t idx = word >> 4;
        if (idx < offs[k] || idx >= offs[k + 1]) k = group_of(offs, K, idx);
        const int32_t e = gexp[k] - (int32_t)(word & 7u);
        return __fmul_rn(scale, __uint_as_float(((uint32_t)(e + 127) << 23) | ((word & 8u) << 28)));
    };

    if ((size_t)total * 8 < n) {
        // ---- sparse messages: not worth moving u through shared memory
        if (kOverwrite) {
            for (size_t i = lo + 4 * (size_t)tid; i < hi; i += 4 * kTileThreads) {
                if (i + 3 < hi) *reinterpret_cast<float4 *>(u + i) = make_float4(0.f, 0.f, 0.f, 0.f);
                else for (size_t c = i; c < hi; ++c) u[c] = 0.f;
            }
            __syncthreads();                                        // this block's zeros before this block's additions
        }
        for (int w = warp; w < W; w += kTileWarps) {
            const uint32_t *words = sm_words[w];
            const int32_t *gexp = sm_gexp[w];
            const uint32_t end = sm_count[w];
            int k = 0;
            for (uint32_t i0 = cur[w]; i0 < end; i0 += 32) {           // warp-uniform trip count
                const uint32_t i = i0 + lane;
                const uint32_t word = i < end ? words[i] : 0xFFFFFFFFu;
                const bool in = i < end && (word >> 4) < hi;
                if (in) {
                    if ((word >> 4) >= lo) atomicAdd(u + (word >> 4), value_of(word, gexp, k));
                    else bad = true;                                 // behind the run's start: the message is not sorted
                }
                if (!__all_sync(0xffffffffu, in)) break;             // sorted: the rest belongs to later chunks
            }
        }
        if (bad) atomicOr(dev_status, VGC_DEV_RANGE);
        return;
    }

    // ---- dense: every warp walks its own part of the block's range
    // sub-tile length: about 100 words of an average message per sub-tile, so that one window (at most 128 words)
    // usually holds all of a message's words for it
    const uint32_t per_msg = total / (uint32_t)W + 1;
    const uint64_t sub_want = ((uint64_t)n * 100u) / per_msg;
    uint32_t sub = sub_want > kSubMax ? kSubMax : (sub_want < kSubMin ? kSubMin : (uint32_t)sub_want);
    sub &= ~127u;
    // 32-word loads per window: the expected words per message and sub-tile plus a quarter
    const uint32_t expect = (uint32_t)(((uint64_t)sub * per_msg) / n) + 1;
    const uint32_t nl = expect > 76 ? 4u : expect > 51 ? 3u : expect > 25 ? 2u : 1u;

    uint32_t wchunk = (uint32_t)((hi - lo + kTileWarps - 1) / kTileWarps);
    wchunk = (wchunk + 3u) & ~3u;                                // sub-tiles start on 16-byte boundaries of u
    const size_t wlo = lo + (size_t)warp * wchunk < hi ? lo + (size_t)warp * wchunk : hi;
    const size_t whi = wlo + wchunk < hi ? wlo + wchunk : hi;
    if (wlo >= whi) return;

    // where every message's run enters this warp's part: searched inside the block's run, whose words in this
    // chunk cannot be more than the chunk has elements; eight messages' probes in flight together
    for (int m0 = 0; m0 < W; m0 += kGroup) {
        uint32_t s_lo[kGroup], s_hi[kGroup];
#pragma unroll
        for (int g = 0; g < kGroup; ++g) {
            const int m = m0 + g < W ? m0 + g : W - 1;
            const uint32_t c = cur[m], left = sm_count[m] - c;
            s_lo[g] = c;
            s_hi[g] = c + (left < chunk_elems ? left : chunk_elems);
            if (m0 + g >= W || warp == 0) s_hi[g] = s_lo[g];       // warp 0 starts where the block's run starts
        }
        bool busy = true;
        while (busy) {
            uint32_t probe[kGroup], step[kGroup];
#pragma unroll
            for (int g = 0; g < kGroup; ++g) {
                step[g] = (s_hi[g] - s_lo[g]) / 32 + 1;
                const uint32_t pos = s_lo[g] + step[g] * lane;
                probe[g] = pos < s_hi[g] ? sm_words[m0 + g < W ? m0 + g : W - 1][pos] >> 4 : 0xFFFFFFFFu;
            }
            busy = false;
#pragma unroll
            for (int g = 0; g < kGroup; ++g) {
                if (s_hi[g] > s_lo[g]) {                             // warp-uniform
                    const uint32_t nb = __popc(__ballot_sync(0xffffffffu, probe[g] < (uint32_t)wlo));
                    if (nb == 0) s_hi[g] = s_lo[g];
                    else {
                        const uint32_t new_hi = s_lo[g] + step[g] * nb;
                        s_lo[g] = s_lo[g] + step[g] * (nb - 1) + 1;
                        s_hi[g] = new_hi < s_hi[g] ? new_hi : s_hi[g];
                    }
                    busy = busy || s_hi[g] > s_lo[g];
                }
            }
        }
        if (lane < kGroup && m0 + (int)lane < W) {
            uint32_t mine = 0;
#pragma unroll
            for (int g = 0; g < kGroup; ++g) mine = lane == (uint32_t)g ? s_lo[g] : mine;
            wcur[warp][m0 + lane] = mine;
        }
    }
    __syncwarp();

    float *const tile = tiles + (size_t)warp * kSubMax;
    const uint32_t tile_addr0 = (uint32_t)__cvta_generic_to_shared(tile);
    const uint32_t lut_addr = (uint32_t)__cvta_generic_to_shared(&lut[warp][0]);
    for (size_t t0 = wlo; t0 < whi; t0 += sub) {
        const uint32_t t_lo = (uint32_t)t0;
        const uint32_t t_len = (uint32_t)(whi - t0 < sub ? whi - t0 : sub);
        const uint32_t t_hi = t_lo + t_len;
        const uint32_t n_vec = t_len / 4;
        if (kOverwrite) {
            for (uint32_t q = lane; q < (t_len + 3) / 4; q += 32) reinterpret_cast<float4 *>(tile)[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        } else {
            for (uint32_t q = lane; q < n_vec; q += 32)
                reinterpret_cast<float4 *>(tile)[q] = *reinterpret_cast<const float4 *>(u + t0 + 4 * (size_t)q);
            if (lane < t_len - 4 * n_vec) tile[4 * n_vec + lane] = u[t0 + 4 * n_vec + lane];
        }
        int tile_group = -1;                                        // weight tensor of the sub-tile, -1 if it spans several
        if (!kHybrid) {
            tile_group = group_of(offs, K, t_lo);
            if (t_hi - 1 >= offs[tile_group + 1]) tile_group = -1;
        }
        const bool use_lut = kHybrid || tile_group >= 0;
        // element idx lives at tile_addr + 4 * idx (shared-memory byte address)
        const uint32_t tile_addr = tile_addr0 - 4u * t_lo;

        for (int m0 = 0; m0 < W; m0 += kGroup) {
            // the next words of eight messages: loads of all windows in flight before the first is looked at
            uint32_t win[kGroup][kWinMax];
#pragma unroll
            for (int g = 0; g < kGroup; ++g) {
                const int m = m0 + g < W ? m0 + g : W - 1;
                const uint32_t c = wcur[warp][m], cnt = m0 + g < W ? sm_count[m] : 0u;
                const uint32_t *p = sm_words[m] + c + lane;
#pragma unroll
                for (int j = 0; j < kWinMax; ++j)
                    win[g][j] = ((uint32_t)j < nl && c + lane + 32u * j < cnt) ? p[32 * j] : 0xFFFFFFFFu;
            }
            __syncwarp();                                           // the previous group's look-ups are done with the table
            // the 16 values a word's low four bits (sign, d) can stand for, per message of the group
            if (use_lut)
                for (uint32_t i = lane; i < kGroup * 16; i += 32) {
                    const int m = m0 + (int)(i >> 4) < W ? m0 + (int)(i >> 4) : W - 1;
                    const uint32_t code = i & 15u;
                    float val;
                    if (kHybrid) val = (code & 8u) ? -tau : tau;
                    else {
                        const uint32_t ebits = (uint32_t)(sm_gexp[m][tile_group] + 127) << 23;
                        val = __uint_as_float((ebits - ((code & 7u) << 23)) | ((code & 8u) << 28));
                    }
                    lut[warp][i] = __fmul_rn(scale, val);
                }
            __syncwarp();
#pragma unroll
            for (int g = 0; g < kGroup; ++g) {
                const int m = m0 + g;
                if (m < W) {                                         // warp-uniform
                    const uint32_t c = wcur[warp][m], cnt = sm_count[m];
                    const uint32_t lut_m = lut_addr + 64u * (uint32_t)g;
                    const int32_t *gexp = sm_gexp[m];
                    int k = 0;
                    uint32_t adv = 0;
                    // one batch of 32 words starting at cursor + adv: adds the leading words that fall below the
                    // sub-tile's end; returns whether all 32 did (then the run may continue in the next batch)
                    auto batch = [&](uint32_t word) -> bool {
                        const uint32_t idx = word >> 4;
                        const bool in = c + adv + lane < cnt && idx < t_hi;
                        const uint32_t ballot = __ballot_sync(0xffffffffu, in);
                        const uint32_t lead = ballot == 0xFFFFFFFFu ? 32u : (uint32_t)__ffs(~ballot) - 1u;   // leading words that are in
                        if (lane < lead) {
                            if (idx - t_lo < t_len) {               // also false for an index behind the sub-tile
                                if (use_lut) {
                                    float x, v;
                                    const uint32_t at = tile_addr + 4u * idx;
                                    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(lut_m + ((word & 15u) << 2)));
                                    asm volatile("ld.shared.f32 %0, [%1];" : "=f"(x) : "r"(at) : "memory");
                                    x = __fadd_rn(x, v);
                                    asm volatile("st.shared.f32 [%0], %1;" ::"r"(at), "f"(x) : "memory");
                                } else {
                                    tile[idx - t_lo] = __fadd_rn(tile[idx - t_lo], value_of(word, gexp, k));
                                }
                            } else bad = true;
                        }
                        adv += lead;
                        return lead == 32u;
                    };
                    bool more = true;
#pragma unroll
                    for (int j = 0; j < kWinMax; ++j)
                        if (more && (uint32_t)j < nl) more = batch(win[g][j]);
                    while (more) {                                   // more words than the window held
                        const uint32_t pos = c + adv + lane;
                        more = batch(pos < cnt ? sm_words[m][pos] : 0xFFFFFFFFu);
                    }
                    if (lane == 0) wcur[warp][m] = c + adv;
                    __syncwarp();                                    // the next message may hit the same elements
                }
            }
        }
        for (uint32_t q = lane; q < n_vec; q += 32)
            *reinterpret_cast<float4 *>(u + t0 + 4 * (size_t)q) = reinterpret_cast<const float4 *>(tile)[q];
        if (lane < t_len - 4 * n_vec) u[t0 + 4 * n_vec + lane] = tile[4 * n_vec + lane];
        __syncwarp();
    }
    if (bad) atomicOr(dev_status, VGC_DEV_RANGE);
}

}  // namespace vgc

using namespace vgc;

namespace {
typedef void (*TilesFn)(const DecodeViews, int, const uint32_t *, int, float, float, float *, size_t, uint32_t, uint32_t *);

vgc_status decode_launch(bool hybrid, bool overwrite, const vgc_message_view *msgs, int W, const uint32_t *group_offsets,
                         int K, float scale, float tau, float *u, size_t n, uint32_t *dev_status, cudaStream_t st)
{
    static int sm_count = 0;
    if (sm_count == 0) {
        int dev = 0, c = 0;
        VGC_CUDA_OK(cudaGetDevice(&dev));
        VGC_CUDA_OK(cudaDeviceGetAttribute(&c, cudaDevAttrMultiProcessorCount, dev));
        sm_count = c > 0 ? c : 148;
    }
    if (W == 0) {                                                // vgc_decode_sum of nothing
        VGC_CUDA_OK(cudaMemsetAsync(u, 0, n * sizeof(float), st));
        return VGC_OK;
    }
    for (int w0 = 0; w0 < W; w0 += kMaxViews) {
        const int wb = W - w0 < kMaxViews ? W - w0 : kMaxViews;
        DecodeViews views;
        for (int w = 0; w < kMaxViews; ++w) {
            const vgc_message_view &m = msgs[w0 + (w < wb ? w : 0)];
            views.words[w] = m.words;
            views.nnz[w] = m.nnz;
            views.group_exp[w] = m.group_exp;
            views.max_words[w] = m.max_words;
        }
        // one contiguous range per block, two blocks per SM
        size_t chunk = (n + (size_t)sm_count * 2 - 1) / ((size_t)sm_count * 2);
        chunk = (chunk + 3) / 4 * 4;
        const unsigned blocks = (unsigned)((n + chunk - 1) / chunk);
        const bool ow = overwrite && w0 == 0;                    // later groups of messages add to the first
        TilesFn fn = hybrid ? (ow ? decode_tiles<true, true> : decode_tiles<true, false>)
                            : (ow ? decode_tiles<false, true> : decode_tiles<false, false>);
        constexpr size_t kDynSmem = (size_t)kTileWarps * kSubMax * sizeof(float);
        static TilesFn configured[4];
        static int n_configured = 0;
        bool seen = false;
        for (int i = 0; i < n_configured; ++i) seen = seen || configured[i] == fn;
        if (!seen) {
            VGC_CUDA_OK(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDynSmem));
            if (n_configured < 4) configured[n_configured++] = fn;
        }
        fn<<<blocks, kTileThreads, kDynSmem, st>>>(views, wb, group_offsets, K, scale, tau, u, n, (uint32_t)chunk, dev_status);
        count_launch();
    }
    VGC_CUDA_OK(cudaGetLastError());
    return VGC_OK;
}

bool views_ok(const vgc_message_view *msgs, int W, bool need_exp)
{
    for (int w = 0; w < W; ++w)
        if (!msgs[w].words || !msgs[w].nnz || (need_exp && !msgs[w].group_exp)) return false;
    return true;
}
}  // namespace

extern "C" vgc_status vgc_decode_accumulate(const vgc_message_view *msgs, int W,
                                            const uint32_t *group_offsets, int K, float scale,
                                            float *u, size_t n, uint32_t *dev_status, vgc_stream_t stream)
{
    if (W == 0 || n == 0) return VGC_OK;
    if (W < 0 || K < 1 || n > VGC_MAX_PARAMS || !msgs || !group_offsets || !u || !dev_status || !aligned16(u))
        return VGC_ERR_INVALID_ARG;
    if (!(scale == scale) || !views_ok(msgs, W, true)) return VGC_ERR_INVALID_ARG;
    return decode_launch(false, false, msgs, W, group_offsets, K, scale, 0.f, u, n, dev_status,
                         reinterpret_cast<cudaStream_t>(stream));
}

extern "C" vgc_status vgc_decode_accumulate_hybrid(const vgc_message_view *msgs, int W, float tau, float scale,
                                                   float *u, size_t n, uint32_t *dev_status, vgc_stream_t stream)
{
    if (W == 0 || n == 0) return VGC_OK;
    if (W < 0 || n > VGC_MAX_PARAMS || !msgs || !u || !dev_status || !aligned16(u)) return VGC_ERR_INVALID_ARG;
    if (!(scale == scale) || !(tau == tau) || !views_ok(msgs, W, false)) return VGC_ERR_INVALID_ARG;
    return decode_launch(true, false, msgs, W, nullptr, 0, scale, tau, u, n, dev_status,
                         reinterpret_cast<cudaStream_t>(stream));
}

extern "C" vgc_status vgc_decode_sum(const vgc_message_view *msgs, int W, const uint32_t *group_offsets, int K,
                                     float scale, float *u, size_t n, uint32_t *dev_status, vgc_stream_t stream)
{
    if (n == 0) return VGC_OK;
    if (W < 0 || K < 1 || n > VGC_MAX_PARAMS || (W > 0 && !msgs) || !group_offsets || !u || !dev_status || !aligned16(u))
        return VGC_ERR_INVALID_ARG;
    if (!(scale == scale) || !views_ok(msgs, W, true)) return VGC_ERR_INVALID_ARG;
    return decode_launch(false, true, msgs, W, group_offsets, K, scale, 0.f, u, n, dev_status,
                         reinterpret_cast<cudaStream_t>(stream));
}

extern "C" vgc_status vgc_decode_sum_hybrid(const vgc_message_view *msgs, int W, float tau, float scale, float *u,
                                            size_t n, uint32_t *dev_status, vgc_stream_t stream)
{
    if (n == 0) return VGC_OK;
    if (W < 0 || n > VGC_MAX_PARAMS || (W > 0 && !msgs) || !u || !dev_status || !aligned16(u)) return VGC_ERR_INVALID_ARG;
    if (!(scale == scale) || !(tau == tau) || !views_ok(msgs, W, false)) return VGC_ERR_INVALID_ARG;
    return decode_launch(true, true, msgs, W, nullptr, 0, scale, tau, u, n, dev_status,
                         reinterpret_cast<cudaStream_t>(stream));
}
