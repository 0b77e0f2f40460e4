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

// kHybrid: messages of the hybrid algorithm (Algorithm 2) -- every word stands for +-tau, no exponents.
template <bool kHybrid>
__device__ __forceinline__ void decode_one(uint32_t word, const uint32_t *offs, const int32_t *gexp, int K,
                                           int &k, float scale, float tau, float *u, size_t n, bool &bad)
{
    const uint32_t idx = word >> 4;
    if (idx >= n) { bad = true; return; }
    if (kHybrid) {
        atomicAdd(u + idx, __fmul_rn(scale, (word & 8u) ? -tau : tau));
        return;
    }
    if (idx < offs[k] || idx >= offs[k + 1]) k = group_of(offs, K, idx);
    const int32_t e = gexp[k] - (int32_t)(word & 7u);
    const float value = __uint_as_float(((uint32_t)(e + 127) << 23) | ((word & 8u) << 28));
    atomicAdd(u + idx, __fmul_rn(scale, value));
}

template <bool kHybrid>
__global__ void __launch_bounds__(kDecThreads)
decode_scatter(const __grid_constant__ DecodeViews views, const uint32_t *__restrict__ group_offsets, int K,
               float scale, float tau, float *__restrict__ u, size_t n, uint32_t *dev_status)
{
    __shared__ uint32_t sm_offs[kDecOffsSmem];
    __shared__ int32_t sm_exp[kDecOffsSmem];
    const int w = blockIdx.y;
    const uint32_t *__restrict__ words = views.words[w];
    const uint32_t count = *views.nnz[w];
    const bool in_smem = !kHybrid && (K + 1) <= kDecOffsSmem;
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
        decode_one<kHybrid>(w4.x, offs, gexp, K, k, scale, tau, u, n, bad);
        decode_one<kHybrid>(w4.y, offs, gexp, K, k, scale, tau, u, n, bad);
        decode_one<kHybrid>(w4.z, offs, gexp, K, k, scale, tau, u, n, bad);
        decode_one<kHybrid>(w4.w, offs, gexp, K, k, scale, tau, u, n, bad);
    }
    for (uint32_t q = 4 * n_vec + blockIdx.x * kDecThreads + threadIdx.x; q < count; q += gridDim.x * kDecThreads)
        decode_one<kHybrid>(words[q], offs, gexp, K, k, scale, tau, u, n, bad);
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
constexpr int kMergeTile = 4096;                 // elements of u per shared-memory tile (16 KB)
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

template <bool kHybrid>
__global__ void __launch_bounds__(kDecThreads)
decode_merge(const __grid_constant__ DecodeViews views, int W, const uint32_t *__restrict__ group_offsets, int K,
             float scale, float tau, float *__restrict__ u, size_t n, uint32_t chunk_elems, uint32_t *dev_status)
{
    __shared__ __align__(16) float tile[kMergeTile];
    __shared__ uint32_t sm_offs[kDecOffsSmem];
    __shared__ uint32_t run_begin[kMaxViews], run_end[kMaxViews];
    __shared__ uint32_t total_words;

    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool in_smem = !kHybrid && (K + 1) <= kDecOffsSmem;
    if (in_smem)
        for (int i = threadIdx.x; i <= K; i += kDecThreads) sm_offs[i] = group_offsets[i];
    const uint32_t *offs = in_smem ? sm_offs : group_offsets;
    if (threadIdx.x == 0) total_words = 0;
    __syncthreads();

    const size_t lo = (size_t)blockIdx.x * chunk_elems;
    const size_t hi = lo + chunk_elems < n ? lo + chunk_elems : n;
    const bool last_chunk = hi == n;

    // ---- where every message's run enters [lo, hi); the run ends where its indices reach hi, which the
    // tile loop finds as it goes.  Dense or sparse is decided for the whole call from the messages' sizes.
    for (int w = warp; w < W; w += kMergeWarps) {
        const uint32_t *words = views.words[w];
        const uint32_t count = *views.nnz[w];
        const uint32_t b = warp_lower_bound(words, count, (uint32_t)lo);
        if (lane == 0) {
            run_begin[w] = b;
            run_end[w] = count;
            atomicAdd(&total_words, count);
            if (last_chunk && count && (words[count - 1] >> 4) >= n) atomicOr(dev_status, VGC_DEV_RANGE);   // skipped
        }
    }
    __syncthreads();
    const uint32_t total = total_words;
    if (total == 0) return;

    auto value_of = [&](uint32_t word, const int32_t *gexp, int &k) -> float {
        if (kHybrid) return __fmul_rn(scale, (word & 8u) ? -tau : tau);
        const uint32_t idx = word >> 4;
        if (idx < offs[k] || idx >= offs[k + 1]) k = group_of(offs, K, idx);
        const int32_t e = gexp[k] - (int32_t)(word & 7u);
        return __fmul_rn(scale, __uint_as_float(((uint32_t)(e + 127) << 23) | ((word & 8u) << 28)));
    };

    if ((size_t)total * 8 < n) {
        // ---- sparse messages: not worth moving u through shared memory
        for (int w = warp; w < W; w += kMergeWarps) {
            const uint32_t *words = views.words[w];
            const int32_t *gexp = views.group_exp[w];
            int k = 0;
            for (uint32_t i0 = run_begin[w]; i0 < run_end[w]; i0 += 32) {       // warp-uniform trip count
                const uint32_t i = i0 + lane;
                const uint32_t word = i < run_end[w] ? words[i] : 0xFFFFFFFFu;
                const bool in = i < run_end[w] && (word >> 4) < hi;
                if (in) atomicAdd(u + (word >> 4), value_of(word, gexp, k));
                if (!__all_sync(0xffffffffu, in)) break;             // sorted: the rest belongs to later chunks
            }
        }
        return;
    }

    // ---- dense chunk: tile by tile through shared memory.  Messages are applied one after the other, in
    // message order, by the whole block: inside one message the indices are distinct, so plain
    // read-modify-writes suffice and every element sees its additions in the order w = 0, 1, ... --
    // the result does not depend on scheduling.  A message's words of a tile are the head of what is left of
    // its run: the block loads a window of kPre*256 words, applies those below the tile's end and counts them.
    __shared__ uint32_t cur[kMaxViews], taken[kMaxViews];
    for (int w = threadIdx.x; w < W; w += kDecThreads) { cur[w] = run_begin[w]; taken[w] = 0; }
    constexpr int kPre = 4;                          // words per thread in one window
    constexpr int kGroup = 8;                        // messages whose windows are in flight together
    constexpr int kVec = kMergeTile / 4 / kDecThreads;   // float4 per thread per tile
    const float4 *u4 = reinterpret_cast<const float4 *>(u);          // u is 16-byte aligned, tiles are whole
    float4 ahead[kVec];                              // next tile of u, loaded while the current one is processed
    auto fetch_tile = [&](size_t t0) {
#pragma unroll
        for (int q = 0; q < kVec; ++q) {
            const size_t i = t0 + 4 * (threadIdx.x + q * kDecThreads);
            if (i + 3 < hi) ahead[q] = u4[i / 4];
            else {
                float e[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) e[c] = i + c < hi ? u[i + c] : 0.f;
                ahead[q] = make_float4(e[0], e[1], e[2], e[3]);
            }
        }
    };
    fetch_tile(lo);
    __syncthreads();
    for (size_t t0 = lo; t0 < hi; t0 += kMergeTile) {
        const uint32_t t_len = (uint32_t)(hi - t0 < kMergeTile ? hi - t0 : kMergeTile);
        const uint32_t t_hi = (uint32_t)(t0 + t_len);
        int tile_group = -1;                                  // weight tensor of the tile, -1 if it spans several
        if (!kHybrid) {
            tile_group = group_of(offs, K, (uint32_t)t0);
            if (t_hi - 1 >= offs[tile_group + 1]) tile_group = -1;
        }
#pragma unroll
        for (int q = 0; q < kVec; ++q) reinterpret_cast<float4 *>(tile)[threadIdx.x + q * kDecThreads] = ahead[q];
        if (t0 + kMergeTile < hi) fetch_tile(t0 + kMergeTile);
        __syncthreads();

        // one window of one message: apply the words below t_hi, return how many this thread applied
        auto apply = [&](int w, const uint32_t (&win)[kPre], uint32_t base) -> uint32_t {
            const int32_t *gexp = views.group_exp[w];
            const uint32_t e = run_end[w];
            uint32_t mine = 0;
            if (tile_group >= 0) {
                const uint32_t ebits = (uint32_t)(gexp[tile_group] + 127) << 23;   // one exponent for the tile
#pragma unroll
                for (int j = 0; j < kPre; ++j) {
                    const uint32_t word = win[j];
                    if (base + threadIdx.x + j * kDecThreads < e && (word >> 4) < t_hi) {
                        const float val = __uint_as_float((ebits - ((word & 7u) << 23)) | ((word & 8u) << 28));
                        tile[(word >> 4) - (uint32_t)t0] += __fmul_rn(scale, val);
                        ++mine;
                    }
                }
            } else {
                int k = 0;
#pragma unroll
                for (int j = 0; j < kPre; ++j) {
                    const uint32_t word = win[j];
                    if (base + threadIdx.x + j * kDecThreads < e && (word >> 4) < t_hi) {
                        tile[(word >> 4) - (uint32_t)t0] += value_of(word, gexp, k);
                        ++mine;
                    }
                }
            }
            return mine;
        };
        auto load_window = [&](int w, uint32_t base, uint32_t (&win)[kPre]) {
            const uint32_t *words = views.words[w];
            const uint32_t e = run_end[w];
#pragma unroll
            for (int j = 0; j < kPre; ++j) {
                const uint32_t i = base + threadIdx.x + j * kDecThreads;
                win[j] = i < e ? words[i] : 0xFFFFFFFFu;
            }
        };

        for (int w0 = 0; w0 < W; w0 += kGroup) {
            uint32_t held[kGroup][kPre];
#pragma unroll
            for (int g = 0; g < kGroup; ++g) load_window(w0 + g < W ? w0 + g : W - 1, cur[w0 + g < W ? w0 + g : W - 1], held[g]);
#pragma unroll
            for (int g = 0; g < kGroup; ++g) {
                const int w = w0 + g;
                if (w < W) {                                         // uniform over the block
                    uint32_t base = cur[w];
                    uint32_t mine = apply(w, held[g], base);
                    // block total of `mine`: warp sums, then shared counter
                    uint32_t wsum = mine;
#pragma unroll
                    for (int d = 16; d >= 1; d >>= 1) wsum += __shfl_xor_sync(0xffffffffu, wsum, d);
                    if (lane == 0 && wsum) atomicAdd(&taken[w], wsum);
                    __syncthreads();
                    // a full window means the tile may hold more words of this message
                    while (taken[w] == (base - cur[w]) + kPre * kDecThreads) {
                        base += kPre * kDecThreads;
                        uint32_t win[kPre];
                        load_window(w, base, win);
                        mine = apply(w, win, base);
                        wsum = mine;
#pragma unroll
                        for (int d = 16; d >= 1; d >>= 1) wsum += __shfl_xor_sync(0xffffffffu, wsum, d);
                        __syncthreads();                             // everyone has read taken[w]
                        if (lane == 0 && wsum) atomicAdd(&taken[w], wsum);
                        __syncthreads();
                    }
                }
            }
        }
#pragma unroll
        for (int q = 0; q < kVec; ++q) {
            const size_t i = t0 + 4 * (threadIdx.x + q * kDecThreads);
            const float4 val = reinterpret_cast<const float4 *>(tile)[threadIdx.x + q * kDecThreads];
            if (i + 3 < hi) reinterpret_cast<float4 *>(u)[i / 4] = val;
            else {
                const float e[4] = {val.x, val.y, val.z, val.w};
#pragma unroll
                for (int c = 0; c < 4; ++c)
                    if (i + c < hi) u[i + c] = e[c];
            }
        }
        __syncthreads();
        for (int w = threadIdx.x; w < W; w += kDecThreads) { cur[w] += taken[w]; taken[w] = 0; }
        __syncthreads();
    }
}


// ------------------------------------------------------------------------------------------
// Large-tile form (default).  Same idea as the segment-merge form -- sorted messages, a block owns a
// contiguous range of u and moves it through shared memory once -- with the costs per tile cut down:
//   - tiles of up to 24576 elements (96 KB), two blocks of 512 threads per SM, so a range is 3 or 4 tiles;
//   - the tile comes in by cp.async (no registers, in flight while the warps search);
//   - where a message's run ends inside the tile is found by one warp-wide search per message, confined to
//     the at most tile-length words that can fall into a tile;
//   - messages are applied one after the other, in message order, by the whole block (indices inside one message
//     are distinct, so plain read-modify-writes, a block barrier between messages): 4 x 512 words at a time, the
//     loads of the next batch -- of this message or the next -- in flight meanwhile; an element sees its
//     additions in the order w = 0, 1, ..., the same fp32 sequence as a sequential sum;
//   - a word's value is one look-up in a 16-entry table per message (sign and d are its low four bits) when the
//     tile lies inside one weight tensor.
// kOverwrite: the range starts from zero instead of the old contents of u (u = scale * sum of the messages).
// ------------------------------------------------------------------------------------------
constexpr int kTileThreads = 512;
constexpr int kTileWarps = kTileThreads / 32;
constexpr int kTileMax = 24576;                  // elements per tile
constexpr int kTilePre = 8;                      // words per thread in one batch

__device__ __forceinline__ void cp_async_16(void *smem, const void *gmem)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem)), "l"(gmem)
                 : "memory");
}
__device__ __forceinline__ void cp_async_wait_all()
{
    asm volatile("cp.async.commit_group;\n\tcp.async.wait_group 0;" ::: "memory");
}

template <bool kHybrid, bool kOverwrite>
__global__ void __launch_bounds__(kTileThreads, 2)
decode_tiles(const __grid_constant__ DecodeViews views, int W, const uint32_t *__restrict__ group_offsets, int K,
             float scale, float tau, float *__restrict__ u, size_t n, uint32_t chunk_elems, uint32_t tile_elems,
             uint32_t *dev_status)
{
    extern __shared__ __align__(16) float tile[];                // tile_elems floats
    __shared__ uint32_t sm_offs[kDecOffsSmem];
    __shared__ uint32_t cur[kMaxViews], end[kMaxViews];
    __shared__ float lut[kMaxViews * 16];
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
        sm_count[tid] = *views.nnz[tid];
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
            end[w] = count;
            atomicAdd(&total_words, count);
            if (last_chunk && count && (words[count - 1] >> 4) >= n) atomicOr(dev_status, VGC_DEV_RANGE);   // skipped
        }
    }
    __syncthreads();
    const uint32_t total = total_words;
    if (total == 0 && !kOverwrite) return;

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
            int k = 0;
            for (uint32_t i0 = cur[w]; i0 < end[w]; i0 += 32) {       // warp-uniform trip count
                const uint32_t i = i0 + lane;
                const uint32_t word = i < end[w] ? words[i] : 0xFFFFFFFFu;
                const bool in = i < end[w] && (word >> 4) < hi;
                if (in) atomicAdd(u + (word >> 4), value_of(word, gexp, k));
                if (!__all_sync(0xffffffffu, in)) break;             // sorted: the rest belongs to later chunks
            }
        }
        return;
    }

    // ---- dense: tile by tile
    for (size_t t0 = lo; t0 < hi; t0 += tile_elems) {
        const uint32_t t_len = (uint32_t)(hi - t0 < tile_elems ? hi - t0 : tile_elems);
        const uint32_t t_hi = (uint32_t)(t0 + t_len);
        const uint32_t n_vec = t_len / 4;                           // t0 is a multiple of 4 elements
        if (kOverwrite) {
            for (uint32_t q = tid; q < (t_len + 3) / 4; q += kTileThreads)
                reinterpret_cast<float4 *>(tile)[q] = make_float4(0.f, 0.f, 0.f, 0.f);
        } else {
            for (uint32_t q = tid; q < n_vec; q += kTileThreads) cp_async_16(tile + 4 * q, u + t0 + 4 * (size_t)q);
            if (tid < t_len - 4 * n_vec) tile[4 * n_vec + tid] = u[t0 + 4 * n_vec + tid];
        }
        // where every message's run leaves the tile: at most t_len of its words can lie inside
        for (int w = warp; w < W; w += kTileWarps) {
            const uint32_t *words = sm_words[w];
            const uint32_t count = sm_count[w];
            const uint32_t c = cur[w];
            const uint32_t span = count - c < t_len ? count - c : t_len;
            const uint32_t e = c + warp_lower_bound(words + c, span, t_hi);
            if (lane == 0) end[w] = e;
        }
        int tile_group = -1;                                        // weight tensor of the tile, -1 if it spans several
        if (!kHybrid) {
            tile_group = group_of(offs, K, (uint32_t)t0);
            if (t_hi - 1 >= offs[tile_group + 1]) tile_group = -1;
        }
        // the 16 values a word's low four bits (sign, d) can stand for, per message, when the tile lies in one tensor
        const bool use_lut = kHybrid || tile_group >= 0;
        if (use_lut)
            for (int i = tid; i < W * 16; i += kTileThreads) {
                const int w = i >> 4;
                const uint32_t code = (uint32_t)i & 15u;
                float val;
                if (kHybrid) val = (code & 8u) ? -tau : tau;
                else {
                    const uint32_t ebits = (uint32_t)(sm_gexp[w][tile_group] + 127) << 23;
                    val = __uint_as_float((ebits - ((code & 7u) << 23)) | ((code & 8u) << 28));
                }
                lut[i] = __fmul_rn(scale, val);
            }
        if (!kOverwrite) cp_async_wait_all();
        __syncthreads();

        // messages one after the other, each in batches of kTileBatch words per thread; the loads of the next batch
        // (of this message or of the next one) are in flight while a batch is applied
        constexpr uint32_t kBatchWords = kTilePre * kTileThreads;
        auto batches_of = [&](int w) -> uint32_t { return (end[w] - cur[w] + kBatchWords - 1) / kBatchWords; };
        auto load_batch = [&](int w, uint32_t b, uint32_t (&dst)[kTilePre]) {
            const uint32_t first = cur[w] + b * kBatchWords + tid, e = end[w];
            const uint32_t *p = sm_words[w] + first;
            if (first + (kTilePre - 1) * kTileThreads < e) {         // whole column of this thread inside the run
#pragma unroll
                for (int j = 0; j < kTilePre; ++j) dst[j] = p[j * kTileThreads];
            } else {
#pragma unroll
                for (int j = 0; j < kTilePre; ++j) dst[j] = first + j * kTileThreads < e ? p[j * kTileThreads] : 0u;
            }
        };
        // shared-memory byte addresses: element idx of u lives at tile_addr + 4 * (idx - t0); a word carries
        // idx << 4, so 4 * idx = (word >> 2) & ~3
        const uint32_t tile_addr = (uint32_t)__cvta_generic_to_shared(tile) - 4u * (uint32_t)t0;
        const uint32_t lut_addr = (uint32_t)__cvta_generic_to_shared(lut);
        auto add_at = [&](uint32_t word, uint32_t lut_w) {
            const uint32_t at = tile_addr + ((word >> 2) & 0xFFFFFFFCu);
            float x, v;
            asm volatile("ld.shared.f32 %0, [%1];" : "=f"(v) : "r"(lut_w + ((word & 15u) << 2)));
            asm volatile("ld.shared.f32 %0, [%1];" : "=f"(x) : "r"(at) : "memory");
            x = __fadd_rn(x, v);
            asm volatile("st.shared.f32 [%0], %1;" ::"r"(at), "f"(x) : "memory");
        };
        int w = 0;
        uint32_t b = 0;
        while (w < W && batches_of(w) == 0) ++w;
        uint32_t held[kTilePre], next[kTilePre];
        uint32_t nb = w < W ? batches_of(w) : 0;                     // batches of the current message
        if (w < W) load_batch(w, 0, held);
        int k = 0;
        while (w < W) {
            int w2 = w;
            uint32_t b2 = b + 1, nb2 = nb;
            if (b2 >= nb) {
                w2 = w + 1; b2 = 0;
                while (w2 < W && (nb2 = batches_of(w2)) == 0) ++w2;
            }
            if (w2 < W) load_batch(w2, b2, next);
            const uint32_t first = cur[w] + b * kBatchWords + tid, e = end[w];
            const bool whole = first + (kTilePre - 1) * kTileThreads < e;
            if (use_lut) {
                const uint32_t lut_w = lut_addr + 64u * (uint32_t)w;
                if (whole) {
#pragma unroll
                    for (int j = 0; j < kTilePre; ++j) add_at(held[j], lut_w);
                } else {
#pragma unroll
                    for (int j = 0; j < kTilePre; ++j)
                        if (first + j * kTileThreads < e) add_at(held[j], lut_w);
                }
            } else {
                const int32_t *gexp = sm_gexp[w];
#pragma unroll
                for (int j = 0; j < kTilePre; ++j) {
                    const uint32_t word = held[j];
                    if (first + j * kTileThreads < e) tile[(word >> 4) - (uint32_t)t0] += value_of(word, gexp, k);
                }
            }
            if (w2 != w) __syncthreads();                            // the next message may hit the same elements
#pragma unroll
            for (int j = 0; j < kTilePre; ++j) held[j] = next[j];
            w = w2; b = b2; nb = nb2;
        }
        __syncthreads();
        for (uint32_t q = tid; q < n_vec; q += kTileThreads)
            *reinterpret_cast<float4 *>(u + t0 + 4 * (size_t)q) = reinterpret_cast<const float4 *>(tile)[q];
        if (tid < t_len - 4 * n_vec) u[t0 + 4 * n_vec + tid] = tile[4 * n_vec + tid];
        __syncthreads();
        for (int w = tid; w < W; w += kTileThreads) cur[w] = end[w];
        __syncthreads();
    }
}

}  // namespace vgc

using namespace vgc;

namespace {
typedef void (*TilesFn)(const DecodeViews, int, const uint32_t *, int, float, float, float *, size_t, uint32_t, uint32_t,
                        uint32_t *);

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
    const char *path_env = getenv("VGC_DECODE_PATH");
    if (overwrite && (W == 0 || (path_env && (path_env[0] == 's' || path_env[0] == 'm')))) {
        VGC_CUDA_OK(cudaMemsetAsync(u, 0, n * sizeof(float), st));   // the other forms only accumulate
        overwrite = false;
    }
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
        const bool first_group = w0 == 0;
        if (!(path && (path[0] == 's' || path[0] == 'm'))) {
            // large tiles: one contiguous range per block, two blocks per SM, three or four tiles per range
            size_t chunk = (n + (size_t)sm_count * 2 - 1) / ((size_t)sm_count * 2);
            chunk = (chunk + 3) / 4 * 4;
            const size_t tiles = (chunk + kTileMax - 1) / kTileMax;
            const uint32_t tile_elems = (uint32_t)(((chunk + tiles - 1) / tiles + 3) / 4 * 4);
            const unsigned blocks = (unsigned)((n + chunk - 1) / chunk);
            const bool ow = overwrite && first_group;                // later groups of messages add to the first
            TilesFn fn = hybrid ? (ow ? decode_tiles<true, true> : decode_tiles<true, false>)
                                : (ow ? decode_tiles<false, true> : decode_tiles<false, false>);
            static TilesFn configured[4];
            static int n_configured = 0;
            bool seen = false;
            for (int i = 0; i < n_configured; ++i) seen = seen || configured[i] == fn;
            if (!seen) {
                VGC_CUDA_OK(cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, kTileMax * 4));
                if (n_configured < 4) configured[n_configured++] = fn;
            }
            fn<<<blocks, kTileThreads, (size_t)tile_elems * 4, st>>>(views, wb, group_offsets, K, scale, tau, u, n,
                                                                     (uint32_t)chunk, tile_elems, dev_status);
        } else if (path[0] == 's') {                        // per-word scatter (any word order)
            int per_msg = (sm_count * 8 + wb - 1) / wb;          // ~8 blocks per SM in total
            if (per_msg < 1) per_msg = 1;
            dim3 grid((unsigned)per_msg, (unsigned)wb);
            if (hybrid)
                decode_scatter<true><<<grid, kDecThreads, 0, st>>>(views, group_offsets, K, scale, tau, u, n, dev_status);
            else
                decode_scatter<false><<<grid, kDecThreads, 0, st>>>(views, group_offsets, K, scale, tau, u, n, dev_status);
        } else {
            // one chunk per block, four blocks per SM (all resident at once), whole tiles per chunk
            size_t chunk = (n + (size_t)sm_count * 4 - 1) / ((size_t)sm_count * 4);
            chunk = (chunk + kMergeTile - 1) / kMergeTile * kMergeTile;
            const unsigned blocks = (unsigned)((n + chunk - 1) / chunk);
            if (hybrid)
                decode_merge<true><<<blocks, kDecThreads, 0, st>>>(views, wb, group_offsets, K, scale, tau, u, n,
                                                                    (uint32_t)chunk, dev_status);
            else
                decode_merge<false><<<blocks, kDecThreads, 0, st>>>(views, wb, group_offsets, K, scale, tau, u, n,
                                                                     (uint32_t)chunk, dev_status);
        }
        count_launch();
    }
    VGC_CUDA_OK(cudaGetLastError());
    return VGC_OK;
}
}  // namespace

extern "C" vgc_status vgc_decode_accumulate(const vgc_message_view *msgs, int W,
                                            const uint32_t *group_offsets, int K, float scale,
                                            float *u, size_t n, uint32_t *dev_status, vgc_stream_t stream)
{
    if (W == 0 || n == 0) return VGC_OK;
    if (W < 0 || K < 1 || n > VGC_MAX_PARAMS || !msgs || !group_offsets || !u || !dev_status || !aligned16(u))
        return VGC_ERR_INVALID_ARG;
    if (!(scale == scale)) return VGC_ERR_INVALID_ARG;
    for (int w = 0; w < W; ++w)
        if (!msgs[w].words || !msgs[w].nnz || !msgs[w].group_exp) return VGC_ERR_INVALID_ARG;
    return decode_launch(false, false, msgs, W, group_offsets, K, scale, 0.f, u, n, dev_status,
                         reinterpret_cast<cudaStream_t>(stream));
}

extern "C" vgc_status vgc_decode_accumulate_hybrid(const vgc_message_view *msgs, int W, float tau, float scale,
                                                   float *u, size_t n, uint32_t *dev_status, vgc_stream_t stream)
{
    if (W == 0 || n == 0) return VGC_OK;
    if (W < 0 || n > VGC_MAX_PARAMS || !msgs || !u || !dev_status || !aligned16(u)) return VGC_ERR_INVALID_ARG;
    if (!(scale == scale) || !(tau == tau)) return VGC_ERR_INVALID_ARG;
    for (int w = 0; w < W; ++w)
        if (!msgs[w].words || !msgs[w].nnz) return VGC_ERR_INVALID_ARG;
    return decode_launch(true, false, msgs, W, nullptr, 0, scale, tau, u, n, dev_status,
                         reinterpret_cast<cudaStream_t>(stream));
}

extern "C" vgc_status vgc_decode_sum(const vgc_message_view *msgs, int W, const uint32_t *group_offsets, int K,
                                     float scale, float *u, size_t n, uint32_t *dev_status, vgc_stream_t stream)
{
    if (n == 0) return VGC_OK;
    if (W < 0 || K < 1 || n > VGC_MAX_PARAMS || (W > 0 && !msgs) || !group_offsets || !u || !dev_status || !aligned16(u))
        return VGC_ERR_INVALID_ARG;
    if (!(scale == scale)) return VGC_ERR_INVALID_ARG;
    for (int w = 0; w < W; ++w)
        if (!msgs[w].words || !msgs[w].nnz || !msgs[w].group_exp) return VGC_ERR_INVALID_ARG;
    return decode_launch(false, true, msgs, W, group_offsets, K, scale, 0.f, u, n, dev_status,
                         reinterpret_cast<cudaStream_t>(stream));
}

extern "C" vgc_status vgc_decode_sum_hybrid(const vgc_message_view *msgs, int W, float tau, float scale, float *u,
                                            size_t n, uint32_t *dev_status, vgc_stream_t stream)
{
    if (n == 0) return VGC_OK;
    if (W < 0 || n > VGC_MAX_PARAMS || (W > 0 && !msgs) || !u || !dev_status || !aligned16(u)) return VGC_ERR_INVALID_ARG;
    if (!(scale == scale) || !(tau == tau)) return VGC_ERR_INVALID_ARG;
    for (int w = 0; w < W; ++w)
        if (!msgs[w].words || !msgs[w].nnz) return VGC_ERR_INVALID_ARG;
    return decode_launch(true, true, msgs, W, nullptr, 0, scale, tau, u, n, dev_status,
                         reinterpret_cast<cudaStream_t>(stream));
}
