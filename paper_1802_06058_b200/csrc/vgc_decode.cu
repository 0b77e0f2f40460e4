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
//   dense: the block walks its range in tiles of up to 24576 elements (96 KB of shared memory, two blocks of 512
//     threads per SM).  The tile comes in by cp.async while one warp per message finds where the message's run
//     leaves the tile (a search confined to the at most tile-length words that can lie in it); the messages are
//     then applied one after the other by the whole block, 8 x 512 words at a time with the next batch's loads in
//     flight (indices inside a message are distinct, so plain read-modify-writes, a block barrier between
//     messages): an element receives its additions in the order w = 0, 1, ..., the fp32 sequence of a sequential
//     sum, whatever the scheduling.  A word's value is one look-up in a 16-entry table per message (its low four
//     bits are sign and d) when the tile lies inside one weight tensor.  u is read and written once, coalesced.
// kOverwrite: the range starts from zero instead of the old contents of u (u = scale * sum of the messages).
// kHybrid: messages of the hybrid algorithm (Algorithm 2) -- every word stands for +-tau, no exponents.
#include "vgc_common.cuh"

namespace vgc {

constexpr int kMaxViews = 64;
constexpr int kDecOffsSmem = 1024;

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

// three blocks of eight warps per SM: while one block waits at a barrier or for its first words, the others add
constexpr int kTileThreads = 256;
constexpr int kBlocksPerSm = 3;
constexpr int kTileWarps = kTileThreads / 32;
constexpr int kTileMax = 16384;                  // elements per tile
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
__global__ void __launch_bounds__(kTileThreads, kBlocksPerSm)
decode_tiles(const __grid_constant__ DecodeViews views, int W, const uint32_t *__restrict__ group_offsets, int K,
             float scale, float tau, float *__restrict__ u, size_t n, uint32_t chunk_elems, uint32_t tile_elems,
             uint32_t *dev_status)
{
    extern __shared__ __align__(16) float tile[];                // tile_elems floats
    __shared__ uint32_t sm_offs[kDecOffsSmem];
    __shared__ uint32_t cur[kMaxViews], end[kMaxViews], taken[kMaxViews];
    __shared__ int32_t sm_ex[kMaxViews];                         // the messages' exponents for the current tile's tensor
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
            end[w] = count;
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
            int k = 0;
            for (uint32_t i0 = cur[w]; i0 < end[w]; i0 += 32) {       // warp-uniform trip count
                const uint32_t i = i0 + lane;
                const uint32_t word = i < end[w] ? words[i] : 0xFFFFFFFFu;
                const bool in = i < end[w] && (word >> 4) < hi;
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

    // ---- dense: tile by tile
    int cached_group = -1;
    uint32_t t_len = 0;
    // the exact form (below) reads the messages 16 bytes at a time; with a scale that is a positive, normal power of two
    // its result is the sequential sum's, bit for bit
    const int s_exp = (int)((__float_as_uint(scale) >> 23) & 0xFFu) - 127;
    const bool pow2 = (__float_as_uint(scale) & 0x807FFFFFu) == 0u && s_exp > -127 && s_exp < 128;
    bool exact_possible = s_exp < 128;                          // a finite scale
    if (exact_possible)
        for (int w = 0; w < W; ++w) exact_possible = exact_possible && (reinterpret_cast<uintptr_t>(sm_words[w]) & 15u) == 0u;
    if (kOverwrite || exact_possible) {
        // the whole tile buffer starts as zeros; from then on whoever writes a tile out leaves zeros behind
        for (uint32_t q = tid; q < kTileMax / 4; q += kTileThreads)
            reinterpret_cast<float4 *>(tile)[q] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
    for (size_t t0 = lo; t0 < hi; t0 += t_len) {
        const uint32_t left = (uint32_t)(hi - t0);
        t_len = left < tile_elems ? left : tile_elems;
        int tile_group = -1;                                        // weight tensor of the tile, -1 if it spans several
        if (!kHybrid) {
            // A tile ends where its weight tensor ends (when that keeps the next tile on a 16-byte boundary): a tile
            // inside one tensor has one exponent per message -- the table look-up and the exact form below apply.
            // The buffer holds kTileMax elements, so a tile may grow a little to reach that end; a tensor that needs
            // two more tiles gets two of the same size rather than a sliver at its end.
            const int g = group_of(offs, K, (uint32_t)t0);
            const uint32_t next = offs[g + 1], rem = next - (uint32_t)t0;
            if ((next & 3u) == 0u && rem <= left) {
                // (not for a run of tiny tensors: a tile has a fixed cost of a few microseconds)
                // (a sliver is cut off only where the exact form can make it cheap)
                const bool worth = rem >= 2048u || (exact_possible && g + 2 <= K && offs[g + 2] - next >= 8192u);
                if (rem <= (uint32_t)kTileMax) { if (worth) t_len = rem; }
                else if (rem < t_len + 2048u || rem <= 2u * (uint32_t)kTileMax) {
                    const uint32_t half = (rem / 2u + 3u) & ~3u;
                    if (half <= (uint32_t)kTileMax) t_len = half;
                }
            }
            if ((uint32_t)t0 + t_len - 1u < next) tile_group = g;
        }
        const uint32_t t_hi = (uint32_t)(t0 + t_len);
        const uint32_t n_vec = t_len / 4;                           // t0 is a multiple of 4 elements
        if (tile_group >= 0 && tile_group != cached_group) {       // block-uniform; nobody reads sm_ex between the tiles
            if (tid < (uint32_t)W) sm_ex[tid] = sm_gexp[tid][tile_group];
            __syncthreads();
            cached_group = tile_group;
        }
        // Exact form.  When the exponents of all messages for the tile's tensor lie close enough together, every word
        // is an integer multiple of one power of two, 2^base, and
        // every partial sum of up to W of them stays within 2^22 multiples: all of them are exact fp32 numbers, fp32
        // addition of them is associative, and the sequential sum of the words equals the exact sum (with a power-of-two
        // scale that is the decoder's result bit for bit; otherwise the scale is applied to the exact sum, one rounding
        // instead of one per message, and vgc_decode_accumulate adds the scaled sum to u in one addition).  The
        // tile is then accumulated as int32 multiples of 2^base with shared-memory integer atomics, in any order:
        // no barrier between messages, no search for the runs' ends -- the warps stream every message's words from
        // its cursor until the indices leave the tile -- and one conversion at the end.  Same bits, much less waiting.
        int fast_base = INT32_MIN;                                  // INT32_MIN: not applicable
        if (kHybrid) {
            // every word stands for +tau or -tau: the multiples are +-1 and a sum is at most W of them
            if (exact_possible && t_hi < (1u << 28)) fast_base = 0;
        } else if (exact_possible && tile_group >= 0 && t_hi < (1u << 28)) {
            int e_max = INT32_MIN, e_min = INT32_MAX;
            for (int w = 0; w < W; ++w) {
                const int e = sm_ex[w];
                if (e != VGC_EXP_NONE) { e_max = max(e_max, e); e_min = min(e_min, e); }
            }
            const int base = e_min - 7;                             // the smallest value a word can stand for
            // 2^base and every sum of multiples are normal numbers; with a power-of-two scale so are their products
            if (e_max >= e_min && e_max - base + (32 - __clz((W - 1) | 1)) <= 22 && base >= -126 && base + 22 <= 127 &&
                (!pow2 || (base + s_exp >= -126 && base + 22 + s_exp <= 127)))
                fast_base = base;
        }
        const bool fast = fast_base != INT32_MIN;
        if (!kOverwrite && fast)                                    // the exact form reads u at the tile's end: ask it into L2 now
            for (uint32_t line = tid; line < (t_len + 31u) / 32u; line += kTileThreads)
                asm volatile("prefetch.global.L2 [%0];" ::"l"(u + t0 + 32u * (size_t)line));
        if (!kOverwrite && !fast) {                                 // the ordered form adds to the tile's old content
            for (uint32_t q = tid; q < n_vec; q += kTileThreads) cp_async_16(tile + 4 * q, u + t0 + 4 * (size_t)q);
            if (tid < t_len - 4 * n_vec) tile[4 * n_vec + tid] = u[t0 + 4 * n_vec + tid];
        }
        if (tid < (uint32_t)W) taken[tid] = 0;
        if (!fast) {
            if (kOverwrite) __syncthreads();                        // the cursors of the tile before
        // where every message's run leaves the tile: at most t_len of its words can lie inside
            for (int w = warp; w < W; w += kTileWarps) {
                const uint32_t *words = sm_words[w];
                const uint32_t count = sm_count[w];
                const uint32_t c = cur[w];
                const uint32_t span = count - c < t_len ? count - c : t_len;
                const uint32_t e = c + warp_lower_bound(words + c, span, t_hi);
                if (lane == 0) end[w] = e;
            }
        }
        // the 16 values a word's low four bits (sign, d) can stand for, per message, when the tile lies in one tensor
        const bool use_lut = kHybrid || tile_group >= 0;
        if (use_lut)
            for (int i = tid; i < W * 16; i += kTileThreads) {
                const int w = i >> 4;
                const uint32_t code = (uint32_t)i & 15u;
                float val;
                if (kHybrid && fast) {
                    reinterpret_cast<int *>(lut)[i] = (code & 8u) ? -1 : 1;
                    continue;
                } else if (kHybrid) val = (code & 8u) ? -tau : tau;
                else if (fast) {
                    const int e = sm_ex[w];
                    const int mult = e == VGC_EXP_NONE ? 0 : 1 << (e - (int)(code & 7u) - fast_base);
                    reinterpret_cast<int *>(lut)[i] = (code & 8u) ? -mult : mult;
                    continue;
                } else {
                    const uint32_t ebits = (uint32_t)(sm_ex[w] + 127) << 23;
                    val = __uint_as_float((ebits - ((code & 7u) << 23)) | ((code & 8u) << 28));
                }
                lut[i] = __fmul_rn(scale, val);
            }
        if (!kOverwrite && !fast) cp_async_wait_all();
        __syncthreads();

        if (fast) {
            // ---- exact form: warps stream the messages' words from their cursors.  Message m is shared by the warps
            // m, m + W, ... (W < 8) in turns of 256 words -- or a warp takes the messages warp, warp + 8, ... -- and a
            // warp stops at its first turn that reaches past the tile (or the message's end); the words it found inside
            // are added to the message's count, which moves the cursor once all warps are done.
            const uint32_t tile_addr = (uint32_t)__cvta_generic_to_shared(tile);
            const uint32_t lut_addr = (uint32_t)__cvta_generic_to_shared(lut);
            // a word minus t0 << 4 keeps its low four bits and turns its index into the offset inside the tile; one
            // unsigned comparison then says "inside the tile" (a word behind the tile wraps around to a huge number,
            // and so does the filler 0xFFFFFFFF, because t_hi < 2^28)
            const uint32_t t0s = (uint32_t)t0 << 4, t_len16 = t_len << 4;
            const int sharers = W < kTileWarps ? kTileWarps / W : 1;   // warps per message
            for (int m = (int)warp % W; m < W; m += kTileWarps) {
                if (W < kTileWarps && (int)warp >= sharers * W) break;   // warps left over when W does not divide the warps
                const uint32_t turn0 = W < kTileWarps ? warp / (uint32_t)W : 0u;
                const uint32_t *words = sm_words[m];
                const uint32_t c = cur[m], cnt = sm_count[m];
                const uint32_t a = c & ~3u;                          // 16-byte loads: start at the boundary before the cursor
                const uint32_t lut_m = lut_addr + 64u * (uint32_t)m;
                uint32_t inside = 0, n_in = 0;                       // words up to the tile's end; words added
                // a turn is 256 consecutive words, two 16-byte loads per lane; the next turn's loads are issued before
                // this turn's words are looked at, so the latency of one turn hides under the work of the other
                constexpr int kVecs = 2, kAhead = 4;
                constexpr uint32_t kTurnWords = 128u * kVecs;
                uint4 nxt[kVecs];
                auto fetch = [&](uint32_t turn, uint4 (&dst)[kVecs]) {
                    const uint32_t p0 = a + turn * kTurnWords + 4u * lane;
                    if (a + (turn + 1u) * kTurnWords <= cnt) {          // warp-uniform: the whole turn lies inside the message
#pragma unroll
                        for (int v = 0; v < kVecs; ++v) dst[v] = *reinterpret_cast<const uint4 *>(words + p0 + 128u * v);
                    } else {
#pragma unroll
                        for (int v = 0; v < kVecs; ++v) {
                            const uint32_t p = p0 + 128u * v;
                            dst[v].x = p < cnt ? words[p] : 0xFFFFFFFFu;
                            dst[v].y = p + 1u < cnt ? words[p + 1] : 0xFFFFFFFFu;
                            dst[v].z = p + 2u < cnt ? words[p + 2] : 0xFFFFFFFFu;
                            dst[v].w = p + 3u < cnt ? words[p + 3] : 0xFFFFFFFFu;
                        }
                    }
                    // ... and the turns after it are asked into L2 (no registers held): a turn's loads then find their lines there
                    const uint32_t ahead = a + (turn + (uint32_t)(kAhead * sharers)) * kTurnWords + 32u * lane;
                    if (lane < kTurnWords / 32u && ahead < cnt) asm volatile("prefetch.global.L2 [%0];" ::"l"(words + ahead));
                };
                // one word: inside the tile -> look its multiple up and add it; all of it predicated, no branch
                auto add = [&](uint32_t word) {
                    asm volatile("{\n\t"
                                 ".reg .pred p;\n\t"
                                 ".reg .s32 iv;\n\t"
                                 ".reg .u32 o, at, l;\n\t"
                                 "sub.u32 o, %1, %2;\n\t"
                                 "setp.lt.u32 p, o, %3;\n\t"
                                 "and.b32 l, %1, 15;\n\t"
                                 "shl.b32 l, l, 2;\n\t"
                                 "add.u32 l, l, %4;\n\t"
                                 "shr.u32 at, o, 2;\n\t"
                                 "and.b32 at, at, 0xFFFFFFFC;\n\t"
                                 "add.u32 at, at, %5;\n\t"
                                 "@p ld.shared.s32 iv, [l];\n\t"
                                 "@p red.shared.add.s32 [at], iv;\n\t"
                                 "@p add.u32 %0, %0, 1;\n\t"
                                 "}"
                                 : "+r"(n_in)
                                 : "r"(word), "r"(t0s), "r"(t_len16), "r"(lut_m), "r"(tile_addr)
                                 : "memory");
                };
                fetch(turn0, nxt);
                for (uint32_t turn = turn0;; turn += (uint32_t)sharers) {
                    uint4 wd[kVecs];
#pragma unroll
                    for (int v = 0; v < kVecs; ++v) wd[v] = nxt[v];
                    fetch(turn + (uint32_t)sharers, nxt);
#pragma unroll
                    for (int v = 0; v < kVecs; ++v) { add(wd[v].x); add(wd[v].y); add(wd[v].z); add(wd[v].w); }
                    // sorted words: the turn lies inside the tile when its last word does (and the message goes on)
                    const uint32_t turn_end = a + (turn + 1u) * kTurnWords;
                    const bool last_in = wd[kVecs - 1].w - t0s < t_len16;
                    if (turn_end <= cnt && (__ballot_sync(0xffffffffu, last_in) >> 31)) {
                        inside += kTurnWords - (turn == 0u ? c - a : 0u);
                        continue;
                    }
                    // the last turn of this warp: count the words from the cursor on that lie before the tile's end
                    uint32_t mine = 0;
                    const uint32_t p0 = a + turn * kTurnWords + 4u * lane;
#pragma unroll
                    for (int v = 0; v < kVecs; ++v) {
                        const uint32_t p = p0 + 128u * v;
                        const uint32_t x[4] = {wd[v].x, wd[v].y, wd[v].z, wd[v].w};
#pragma unroll
                        for (uint32_t i = 0; i < 4; ++i) mine += (p + i >= c && p + i < cnt && (x[i] >> 4) < t_hi) ? 1u : 0u;
                    }
                    inside += __reduce_add_sync(0xffffffffu, mine);
                    break;
                }
                // a word before the tile's end that was not added lies behind the tile: the message is not sorted
                if (__reduce_add_sync(0xffffffffu, n_in) != inside) bad = true;
                if (lane == 0 && inside) atomicAdd(&taken[m], inside);
            }
        } else {
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
            // a word of a sorted message lies inside the tile; one that does not (the message is not sorted) is skipped
            if ((word >> 4) - (uint32_t)t0 >= t_len) { bad = true; return; }
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
                    if (first + j * kTileThreads < e) {
                        if ((word >> 4) - (uint32_t)t0 < t_len) tile[(word >> 4) - (uint32_t)t0] += value_of(word, gexp, k);
                        else bad = true;
                    }
                }
            }
            if (w2 != w) __syncthreads();                            // the next message may hit the same elements
#pragma unroll
            for (int j = 0; j < kTilePre; ++j) held[j] = next[j];
            w = w2; b = b2; nb = nb2;
        }
        }
        __syncthreads();
        if (tid < (uint32_t)W) cur[tid] = fast ? cur[tid] + taken[tid] : end[tid];
        if (fast) {
            // multiples of 2^base -> fp32 (a sum is at most 2^22 multiples either way, so 1.5 * 2^23 plus it is a float
            // whose bits are 0x4B400000 plus it), times 2^base (exact), times the scale: one rounding, none when the
            // scale is a power of two.  vgc_decode_accumulate adds the result to u; an element no word points at keeps
            // its bits.
            const float unit = kHybrid ? __fmul_rn(scale, tau) : __uint_as_float((uint32_t)(fast_base + 127) << 23);
            auto value = [&](int mult) {
                const float m = __fmul_rn(__fsub_rn(__int_as_float(0x4B400000 + mult), 12582912.f), unit);
                return kHybrid ? m : __fmul_rn(m, scale);       // hybrid: a word is worth scale * tau, rounded once
            };
            if (kOverwrite) {
                for (uint32_t q = tid; q < n_vec; q += kTileThreads) {
                    const int4 mlt = reinterpret_cast<const int4 *>(tile)[q];
                    reinterpret_cast<int4 *>(tile)[q] = make_int4(0, 0, 0, 0);
                    *reinterpret_cast<float4 *>(u + t0 + 4 * (size_t)q) =
                        make_float4(value(mlt.x), value(mlt.y), value(mlt.z), value(mlt.w));
                }
            } else {
                // four vectors of u per thread in flight (asked into L2 when the tile began)
                for (uint32_t q0 = tid; q0 < n_vec; q0 += 4 * kTileThreads) {
                    float4 o[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t q = q0 + j * kTileThreads;
                        if (q < n_vec) o[j] = *reinterpret_cast<const float4 *>(u + t0 + 4 * (size_t)q);
                    }
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t q = q0 + j * kTileThreads;
                        if (q >= n_vec) break;
                        const int4 mlt = reinterpret_cast<const int4 *>(tile)[q];
                        if ((mlt.x | mlt.y | mlt.z | mlt.w) == 0) continue;
                        reinterpret_cast<int4 *>(tile)[q] = make_int4(0, 0, 0, 0);
                        if (mlt.x) o[j].x = __fadd_rn(o[j].x, value(mlt.x));
                        if (mlt.y) o[j].y = __fadd_rn(o[j].y, value(mlt.y));
                        if (mlt.z) o[j].z = __fadd_rn(o[j].z, value(mlt.z));
                        if (mlt.w) o[j].w = __fadd_rn(o[j].w, value(mlt.w));
                        *reinterpret_cast<float4 *>(u + t0 + 4 * (size_t)q) = o[j];
                    }
                }
            }
            if (tid < t_len - 4 * n_vec) {
                const int mult = reinterpret_cast<const int *>(tile)[4 * n_vec + tid];
                float *dst = u + t0 + 4 * n_vec + tid;
                if (kOverwrite) *dst = value(mult);
                else if (mult) *dst = __fadd_rn(*dst, value(mult));
                tile[4 * n_vec + tid] = 0.f;
            }
        } else {
            const bool zero_after = kOverwrite || exact_possible;
            for (uint32_t q = tid; q < n_vec; q += kTileThreads) {
                *reinterpret_cast<float4 *>(u + t0 + 4 * (size_t)q) = reinterpret_cast<const float4 *>(tile)[q];
                if (zero_after) reinterpret_cast<float4 *>(tile)[q] = make_float4(0.f, 0.f, 0.f, 0.f);
            }
            if (tid < t_len - 4 * n_vec) {
                u[t0 + 4 * n_vec + tid] = tile[4 * n_vec + tid];
                if (zero_after) tile[4 * n_vec + tid] = 0.f;
            }
        }
        // vgc_decode_sum: every thread put zeros back where it read, and the next tile's barrier orders them before
        // the next additions.  vgc_decode_accumulate loads the next tile over this one: wait for the readers.
        if (!kOverwrite) __syncthreads();
    }
    if (bad) atomicOr(dev_status, VGC_DEV_RANGE);
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
        // one contiguous range per block, kBlocksPerSm blocks per SM, three or four tiles per range
        size_t chunk = (n + (size_t)sm_count * kBlocksPerSm - 1) / ((size_t)sm_count * kBlocksPerSm);
        chunk = (chunk + 3) / 4 * 4;
        const size_t tiles = (chunk + kTileMax - 1) / kTileMax;
        const uint32_t tile_elems = (uint32_t)(((chunk + tiles - 1) / tiles + 3) / 4 * 4);
        const unsigned blocks = (unsigned)((n + chunk - 1) / chunk);
        const bool ow = overwrite && w0 == 0;                    // later groups of messages add to the first
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
        fn<<<blocks, kTileThreads, (size_t)kTileMax * 4, st>>>(views, wb, group_offsets, K, scale, tau, u, n, (uint32_t)chunk,
                                                                 tile_elems, dev_status);
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
