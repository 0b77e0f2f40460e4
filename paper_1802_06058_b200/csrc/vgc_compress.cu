// vgc_compress: one step of Algorithm 1 ("Basic") over the flat parameter buffer followed by
// Encode() -- the 4-bit quantiser of Sec. 4.2 in the bit-level form of Sec. 4.4 and the
// 32-bit (value, index) word.
//
// Two kernels on one stream:
//   phase A  streams g, s, r, v once (16 B read + 8 B written per parameter), applies the send
//            test and writes r, v back.  Each tile of 2048 parameters compacts its selected
//            (index, value) pairs, in index order, into its own 2048-slot segment of a staging
//            area and records how many there are; a per-tensor atomicMax on |value| bit
//            patterns yields M_k.  Thread blocks never wait for one another here.
//   phase B  runs over the staged pairs only, one warp per segment, in two kernels: "count"
//            quantises against E_k = floor(log2 M_k) and records how many pairs of each
//            segment survive (d <= 7); "emit" turns those counts into positions (a block sums
//            the totals of the chunks before its own, then scans its 32 segments) and packs
//            the words in ascending index order.
// No thread block ever waits for another one: ordering comes from kernel boundaries only.
// The per-tensor maximum has to be complete before any value can be quantised, which is why
// the work is split; the staged pairs are a small fraction of the buffer and stay in L2
// between the count and emit kernels.
#include "vgc_common.cuh"

namespace vgc {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / kWarp;             // 8
constexpr int kRowsA = 2;                            // float4 vectors per thread per tile
constexpr int kTileA = kThreads * kRowsA * 4;        // 2048 parameters per tile = one staging segment
constexpr int kSegPerChunk = 32;                     // phase B: segments per thread block, one per warp
constexpr int kThreadsB = kSegPerChunk * kWarp;      // 1024
constexpr int kOffsSmem = 1024;                      // group offsets cached in shared memory

struct CompressLayout {
    size_t gmax, tile_count, tile_min, kept_count, chunk_total, stage_idx, stage_val, total;
    size_t zero_bytes;       // the per-tensor maxima are cleared per call
    uint32_t tiles_a, chunks;
};

static CompressLayout compress_layout(size_t n, int K)
{
    CompressLayout L;
    L.tiles_a = (uint32_t)((n + kTileA - 1) / kTileA);
    L.chunks = (L.tiles_a + kSegPerChunk - 1) / kSegPerChunk;
    size_t off = 0;
    L.gmax = off;          off = round_up(off + sizeof(uint32_t) * (size_t)K, 256);
    L.zero_bytes = off;
    L.tile_count = off;    off = round_up(off + sizeof(uint32_t) * L.tiles_a, 256);
    L.tile_min = off;      off = round_up(off + sizeof(int32_t) * L.tiles_a, 256);
    L.kept_count = off;    off = round_up(off + sizeof(uint32_t) * L.tiles_a, 256);
    L.chunk_total = off;   off = round_up(off + sizeof(uint64_t) * L.chunks, 256);
    const size_t slots = (size_t)L.tiles_a * kTileA;
    L.stage_idx = off;     off = round_up(off + sizeof(uint32_t) * slots, 256);
    L.stage_val = off;     off = round_up(off + sizeof(uint32_t) * slots, 256);
    L.total = off;
    return L;
}

// ------------------------------------------------------------------------------------------
// phase A
// ------------------------------------------------------------------------------------------
// kHasS = false: the caller accumulated this step's squared-gradient sums straight into v (the sqgrad entry
// points with accumulate = 1), so the pass reads 12 instead of 16 bytes per parameter.
template <bool kHasS>
__global__ void __launch_bounds__(kThreads, 4)
compress_phase_a(const float *__restrict__ g, const float *__restrict__ s, float *__restrict__ r,
                 float *__restrict__ v, size_t n, const uint32_t *__restrict__ group_offsets, int K,
                 float alpha, float zeta, uint32_t *gmax, uint32_t *__restrict__ tile_count,
                 int32_t *__restrict__ tile_min, uint32_t *__restrict__ stage_idx, uint32_t *__restrict__ stage_val,
                 uint8_t *__restrict__ mask, uint32_t n_tiles)
{
    __shared__ uint32_t sm_offs[kOffsSmem];
    __shared__ uint32_t sm_part[2][32];                 // per-(row, warp) counts, double buffered
    __shared__ uint32_t sm_wmax[2][kWarps];
    __shared__ uint32_t sm_wmin[2][kWarps];             // smallest |value| bit pattern sent by each warp
    __shared__ int sm_grp[2];

    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool offs_in_smem = (K + 1) <= kOffsSmem;
    if (offs_in_smem)
        for (int i = tid; i <= K; i += kThreads) sm_offs[i] = group_offsets[i];
    const uint32_t *offs = offs_in_smem ? sm_offs : group_offsets;
    if (tid < 64) (&sm_part[0][0])[tid] = 0;            // entries past kRowsA*kWarps stay zero
    __syncthreads();

    uint32_t buf = 0;
    for (uint32_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, buf ^= 1) {
        const size_t base = (size_t)tile * kTileA;

        // ---- load: thread t owns elements base + (j*256 + t)*4 + {0..3}
        float4 G[kRowsA], S[kRowsA], R[kRowsA], V[kRowsA];
#pragma unroll
        for (int j = 0; j < kRowsA; ++j) {
            const size_t e = base + (size_t)(j * kThreads + tid) * 4;
            if (e + 3 < n) {
                G[j] = ld_stream_f4(g + e);
                if (kHasS) S[j] = ld_stream_f4(s + e);
                R[j] = *reinterpret_cast<const float4 *>(r + e);
                V[j] = *reinterpret_cast<const float4 *>(v + e);
            } else {
                float tg[4], ts[4], tr[4], tv[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const bool in = e + q < n;
                    tg[q] = in ? g[e + q] : 0.f;  ts[q] = (kHasS && in) ? s[e + q] : 0.f;
                    tr[q] = in ? r[e + q] : 0.f;  tv[q] = in ? v[e + q] : 0.f;
                }
                G[j] = make_float4(tg[0], tg[1], tg[2], tg[3]);  S[j] = make_float4(ts[0], ts[1], ts[2], ts[3]);
                R[j] = make_float4(tr[0], tr[1], tr[2], tr[3]);  V[j] = make_float4(tv[0], tv[1], tv[2], tv[3]);
            }
        }
        if (tid == 0) {                                 // weight tensor of this tile, or -1 if it spans several
            const size_t last = (base + kTileA < n ? base + kTileA : n) - 1;
            const int k = group_of(offs, K, (uint32_t)base);
            sm_grp[buf] = (last < offs[k + 1]) ? k : -1;
        }

        // ---- Algorithm 1 loop body; every operation rounded on its own (no FMA)
        uint32_t send_bits = 0;          // bit j*4+q
        uint32_t packed = 0;             // per-row counts, 8 bits each
        uint32_t my_max = 0, my_min = 0x7FFFFFFFu;
#pragma unroll
        for (int j = 0; j < kRowsA; ++j) {
            const size_t e = base + (size_t)(j * kThreads + tid) * 4;
            float *Gj = reinterpret_cast<float *>(&G[j]);
            const float *Sj = reinterpret_cast<const float *>(&S[j]);
            float *Rj = reinterpret_cast<float *>(&R[j]);
            float *Vj = reinterpret_cast<float *>(&V[j]);
            uint32_t row_bits = 0;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float r1 = __fadd_rn(Rj[q], Gj[q]);
                const float v1 = kHasS ? __fadd_rn(Vj[q], Sj[q]) : Vj[q];
                const float lhs = __fmul_rn(r1, r1);
                const float rhs = __fmul_rn(alpha, v1);
                const bool send = (lhs > rhs) && (e + q < n);
                Gj[q] = r1;                                       // value handed to Encode()
                Rj[q] = send ? 0.f : r1;
                Vj[q] = send ? 0.f : __fmul_rn(v1, zeta);
                if (send) {
                    row_bits |= 1u << q;
                    my_max = max(my_max, __float_as_uint(r1) & 0x7FFFFFFFu);
                    my_min = min(my_min, __float_as_uint(r1) & 0x7FFFFFFFu);
                }
            }
            send_bits |= row_bits << (4 * j);
            packed |= (uint32_t)__popc(row_bits) << (8 * j);
            if (e + 3 < n) {
                *reinterpret_cast<float4 *>(r + e) = R[j];
                *reinterpret_cast<float4 *>(v + e) = V[j];
                if (mask) {
                    const uint32_t m4 = (row_bits & 1u) | ((row_bits & 2u) << 7) | ((row_bits & 4u) << 14) |
                                        ((row_bits & 8u) << 21);
                    *reinterpret_cast<uint32_t *>(mask + e) = m4;
                }
            } else {
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    if (e + q < n) {
                        r[e + q] = Rj[q];
                        v[e + q] = Vj[q];
                        if (mask) mask[e + q] = (row_bits >> q) & 1u;
                    }
            }
        }

        // ---- ordered positions inside the tile: warp scan of the packed per-row counts, then
        //      every warp scans the 16 (row, warp) totals by itself (one barrier per tile)
        uint32_t incl = packed;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t up = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += up;
        }
        const uint32_t warp_max = __reduce_max_sync(0xffffffffu, my_max);
        const uint32_t warp_min = __reduce_min_sync(0xffffffffu, my_min);
        if (lane == 31) {
#pragma unroll
            for (int j = 0; j < kRowsA; ++j) sm_part[buf][j * kWarps + warp] = (incl >> (8 * j)) & 0xFFu;
            sm_wmax[buf][warp] = warp_max;
            sm_wmin[buf][warp] = warp_min;
        }
        __syncthreads();
        const uint32_t part = sm_part[buf][lane];
        uint32_t pincl = part;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t up = __shfl_up_sync(0xffffffffu, pincl, d);
            if (lane >= d) pincl += up;
        }
        const uint32_t total = __shfl_sync(0xffffffffu, pincl, 31);
        const uint32_t pexcl = pincl - part;
        const int grp = sm_grp[buf];
        uint32_t *seg_idx = stage_idx + base;
        uint32_t *seg_val = stage_val + base;
#pragma unroll
        for (int j = 0; j < kRowsA; ++j) {
            const uint32_t row_base = __shfl_sync(0xffffffffu, pexcl, j * kWarps + warp);
            const uint32_t row_bits = (send_bits >> (4 * j)) & 0xFu;
            if (row_bits) {
                const uint32_t e = (uint32_t)(base + (size_t)(j * kThreads + tid) * 4);
                uint32_t at = row_base + ((incl >> (8 * j)) & 0xFFu) - (uint32_t)__popc(row_bits);
                const float *Gj = reinterpret_cast<const float *>(&G[j]);
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    if (row_bits & (1u << q)) {
                        const uint32_t bits = __float_as_uint(Gj[q]);
                        seg_idx[at] = e + q;
                        seg_val[at] = bits;
                        ++at;
                        if (grp < 0) atomicMax(&gmax[group_of(offs, K, e + q)], bits & 0x7FFFFFFFu);
                    }
            }
        }
        if (tid == 0) {
            tile_count[tile] = total;
            // the rounded exponent (Sec. 4.2) of the smallest value sent from this tile: with it the counting
            // pass knows without looking at the values whether any of them will be dropped (d > 7).  Tiles that
            // span several tensors say "unknown".
            uint32_t lo = 0x7FFFFFFFu;
#pragma unroll
            for (int w = 0; w < kWarps; ++w) lo = min(lo, sm_wmin[buf][w]);
            tile_min[tile] = grp >= 0 ? (int32_t)((lo + 0x00400000u) >> 23) - 127 : INT32_MIN;
            if (grp >= 0 && total) {
                uint32_t m = 0;
#pragma unroll
                for (int w = 0; w < kWarps; ++w) m = max(m, sm_wmax[buf][w]);
                if (m > ld_volatile_u32(gmax + grp)) atomicMax(gmax + grp, m);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// phase B
// ------------------------------------------------------------------------------------------
// Quantise one staged pair: returns true if a word is emitted.
__device__ __forceinline__ bool encode_pair(uint32_t idx, uint32_t bits, const uint32_t *offs, int K,
                                            const uint32_t *gmax, int &k, int32_t &Ek, uint32_t &word)
{
    if (idx < offs[k] || idx >= offs[k + 1] || Ek == INT32_MIN) {
        k = group_of(offs, K, idx);
        Ek = (int32_t)((gmax[k] >> 23) & 0xFFu) - 127;                  // floor(log2 M_k)
    }
    const uint32_t a = bits & 0x7FFFFFFFu;
    const int32_t e1 = (int32_t)((a + 0x00400000u) >> 23) - 127;        // nearer power of two, midpoint up
    const int32_t e = e1 < Ek ? e1 : Ek;                                // cut at 2^E_k
    const int32_t d = Ek - e;
    word = (idx << 4) | ((bits >> 31) << 3) | (uint32_t)(d & 7);
    return d <= 7;
}

constexpr uint64_t kPassedShift = 32;       // chunk totals: passed << 32 | kept

// One warp walks one segment in index order, four 32-wide slices per round so that the loads
// of a round are in flight together.  EMIT: write the words from position `pos` on.
// Returns the number of pairs kept.
template <bool EMIT>
__device__ __forceinline__ uint32_t walk_segment(const uint32_t *__restrict__ seg_idx,
                                                 const uint32_t *__restrict__ seg_val, uint32_t count,
                                                 const uint32_t *offs, int K, const uint32_t *gmax,
                                                 uint32_t *__restrict__ words, uint32_t pos, uint32_t capacity)
{
    const uint32_t lane = lane_id();
    int k = 0;
    int32_t Ek = INT32_MIN;
    uint32_t kept = 0;
    for (uint32_t q0 = 0; q0 < count; q0 += 128) {
        uint32_t idx[4], bits[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t q = q0 + u * 32 + lane;
            idx[u] = 0; bits[u] = 0;
            if (q < count) { idx[u] = seg_idx[q]; bits[u] = seg_val[q]; }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t q = q0 + u * 32 + lane;
            bool keep = false;
            uint32_t word = 0;
            if (q < count) keep = encode_pair(idx[u], bits[u], offs, K, gmax, k, Ek, word);
            const uint32_t ballot = __ballot_sync(0xffffffffu, keep);
            if (EMIT) {
                const uint32_t p = pos + kept + __popc(ballot & ((1u << lane) - 1u));
                if (keep && p < capacity) words[p] = word;
            }
            kept += __popc(ballot);
        }
    }
    return kept;
}

__global__ void __launch_bounds__(kThreadsB)
compress_count(const uint32_t *__restrict__ group_offsets, int K, const uint32_t *__restrict__ gmax,
               const uint32_t *__restrict__ tile_count, const int32_t *__restrict__ tile_min, uint32_t n_tiles_a,
               const uint32_t *__restrict__ stage_idx, const uint32_t *__restrict__ stage_val,
               uint32_t *__restrict__ kept_count, uint64_t *__restrict__ chunk_total,
               int32_t *__restrict__ group_exp)
{
    __shared__ uint32_t sm_offs[kOffsSmem];
    __shared__ unsigned long long sm_tot[kSegPerChunk];
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool offs_in_smem = (K + 1) <= kOffsSmem;
    if (offs_in_smem) {
        for (int i = tid; i <= K; i += kThreadsB) sm_offs[i] = group_offsets[i];
        __syncthreads();
    }
    const uint32_t *offs = offs_in_smem ? sm_offs : group_offsets;
    if (blockIdx.x == 0)
        for (int k = tid; k < K; k += kThreadsB) {
            const uint32_t m = gmax[k];
            group_exp[k] = m ? (int32_t)((m >> 23) & 0xFFu) - 127 : VGC_EXP_NONE;
        }
    unsigned long long tot = 0;
    const uint32_t seg = blockIdx.x * kSegPerChunk + warp;              // one warp per segment
    if (seg < n_tiles_a) {
        const uint32_t count = tile_count[seg];
        uint32_t kept = count;
        if (count) {
            // nothing is dropped when even the smallest value sent from the tile is within 7 binades of the
            // tensor's exponent (d = E_k - e <= 7): then the values need not be read at all
            const int32_t lowest = tile_min[seg];
            bool walk = lowest == INT32_MIN;
            if (!walk) {
                const int k = group_of(offs, K, seg * (uint32_t)kTileA);
                const int32_t Ek = (int32_t)((gmax[k] >> 23) & 0xFFu) - 127;
                walk = lowest < Ek - 7;
            }
            if (walk)
                kept = walk_segment<false>(stage_idx + (size_t)seg * kTileA, stage_val + (size_t)seg * kTileA, count, offs,
                                           K, gmax, nullptr, 0, 0);
        }
        if (lane == 0) kept_count[seg] = kept;
        tot = ((unsigned long long)count << kPassedShift) | kept;
    }
    if (lane == 0) sm_tot[warp] = tot;
    __syncthreads();
    if (tid == 0) {
        unsigned long long t = 0;
#pragma unroll
        for (int w = 0; w < kSegPerChunk; ++w) t += sm_tot[w];
        chunk_total[blockIdx.x] = t;
    }
}

__global__ void __launch_bounds__(kThreadsB)
compress_emit(const uint32_t *__restrict__ group_offsets, int K, const uint32_t *__restrict__ gmax,
              const uint32_t *__restrict__ tile_count, uint32_t n_tiles_a,
              const uint32_t *__restrict__ stage_idx, const uint32_t *__restrict__ stage_val,
              const uint32_t *__restrict__ kept_count, const uint64_t *__restrict__ chunk_total,
              uint32_t *__restrict__ words, uint32_t capacity, uint32_t *nnz_out, uint32_t *n_criterion,
              uint32_t *n_dropped, uint32_t *dev_status)
{
    __shared__ uint32_t sm_offs[kOffsSmem];
    __shared__ unsigned long long sm_tot[kSegPerChunk];
    __shared__ uint32_t sm_pos[kSegPerChunk];
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool offs_in_smem = (K + 1) <= kOffsSmem;
    if (offs_in_smem)
        for (int i = tid; i <= K; i += kThreadsB) sm_offs[i] = group_offsets[i];
    const uint32_t *offs = offs_in_smem ? sm_offs : group_offsets;

    // totals of all chunks before this one
    unsigned long long before = 0;
    for (uint32_t c = tid; c < blockIdx.x; c += kThreadsB) before += chunk_total[c];
    before = warp_sum_u64(before);
    if (lane == 0) sm_tot[warp] = before;
    __syncthreads();
    before = 0;
#pragma unroll
    for (int w = 0; w < kSegPerChunk; ++w) before += sm_tot[w];
    const uint32_t kept_before = (uint32_t)(before & 0xFFFFFFFFull);

    if (warp == 0) {                                   // positions of this chunk's 32 segments
        const uint32_t seg = blockIdx.x * kSegPerChunk + lane;
        const uint32_t mine = seg < n_tiles_a ? kept_count[seg] : 0;
        uint32_t incl = mine;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t up = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += up;
        }
        sm_pos[lane] = kept_before + incl - mine;
        if (lane == 31) {
            const uint32_t end = kept_before + incl;
            if (end > capacity) atomicOr(dev_status, VGC_DEV_CAPACITY);
            if (blockIdx.x == gridDim.x - 1) {
                const unsigned long long all = before + chunk_total[blockIdx.x];
                *nnz_out = (uint32_t)(all & 0xFFFFFFFFull);
                *n_criterion = (uint32_t)(all >> kPassedShift);
                *n_dropped = (uint32_t)(all >> kPassedShift) - (uint32_t)(all & 0xFFFFFFFFull);
            }
        }
    }
    __syncthreads();
    const uint32_t seg = blockIdx.x * kSegPerChunk + warp;              // one warp per segment
    if (seg < n_tiles_a)
        walk_segment<true>(stage_idx + (size_t)seg * kTileA, stage_val + (size_t)seg * kTileA, tile_count[seg], offs, K,
                           gmax, words, sm_pos[warp], capacity);
}

}  // namespace vgc

// ------------------------------------------------------------------------------------------
// C ABI
// ------------------------------------------------------------------------------------------
using namespace vgc;

extern "C" size_t vgc_compress_workspace_bytes(size_t n, int K)
{
    if (K < 1) K = 1;
    return compress_layout(n, K).total;
}

extern "C" vgc_status vgc_compress(const float *g, const float *s, float *r, float *v, size_t n,
                                   const uint32_t *group_offsets, int K, float alpha, float zeta,
                                   const vgc_message *out, void *ws, size_t ws_bytes, vgc_stream_t stream)
{
    if (n == 0) return VGC_OK;
    if (n > VGC_MAX_PARAMS || K < 1 || !out) return VGC_ERR_INVALID_ARG;
    if (!(alpha >= 0.f) || !(alpha <= 3.402823466e38f) || !(zeta == zeta) || !(zeta >= -3.402823466e38f) ||
        !(zeta <= 3.402823466e38f))
        return VGC_ERR_INVALID_ARG;
    if (!g || !r || !v || !group_offsets || !ws) return VGC_ERR_INVALID_ARG;
    if (!out->group_exp || !out->nnz || !out->n_criterion || !out->n_dropped || !out->dev_status)
        return VGC_ERR_INVALID_ARG;
    if (out->capacity && !out->words) return VGC_ERR_INVALID_ARG;
    if (!aligned16(g) || (s && !aligned16(s)) || !aligned16(r) || !aligned16(v) || !aligned16(ws) ||
        (out->mask && (reinterpret_cast<uintptr_t>(out->mask) & 3u)))
        return VGC_ERR_INVALID_ARG;
    const CompressLayout L = compress_layout(n, K);
    if (ws_bytes < L.total) return VGC_ERR_WORKSPACE;

    char *base = static_cast<char *>(ws);
    uint32_t *gmax = reinterpret_cast<uint32_t *>(base + L.gmax);
    uint32_t *tile_count = reinterpret_cast<uint32_t *>(base + L.tile_count);
    int32_t *tile_min = reinterpret_cast<int32_t *>(base + L.tile_min);
    uint32_t *kept_count = reinterpret_cast<uint32_t *>(base + L.kept_count);
    uint64_t *chunk_total = reinterpret_cast<uint64_t *>(base + L.chunk_total);
    uint32_t *stage_idx = reinterpret_cast<uint32_t *>(base + L.stage_idx);
    uint32_t *stage_val = reinterpret_cast<uint32_t *>(base + L.stage_val);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);

    static int sm_count = 0;
    if (sm_count == 0) {
        int dev = 0, c = 0;
        VGC_CUDA_OK(cudaGetDevice(&dev));
        VGC_CUDA_OK(cudaDeviceGetAttribute(&c, cudaDevAttrMultiProcessorCount, dev));
        sm_count = c > 0 ? c : 148;
    }

    VGC_CUDA_OK(cudaMemsetAsync(ws, 0, L.zero_bytes, st));
    const uint32_t grid_a = L.tiles_a < (uint32_t)(sm_count * 8) ? L.tiles_a : (uint32_t)(sm_count * 8);
    if (s)
        compress_phase_a<true><<<grid_a, kThreads, 0, st>>>(g, s, r, v, n, group_offsets, K, alpha, zeta, gmax, tile_count,
                                                            tile_min, stage_idx, stage_val, out->mask, L.tiles_a);
    else
        compress_phase_a<false><<<grid_a, kThreads, 0, st>>>(g, nullptr, r, v, n, group_offsets, K, alpha, zeta, gmax,
                                                             tile_count, tile_min, stage_idx, stage_val, out->mask,
                                                             L.tiles_a);
    compress_count<<<L.chunks, kThreadsB, 0, st>>>(group_offsets, K, gmax, tile_count, tile_min, L.tiles_a, stage_idx,
                                                   stage_val, kept_count, chunk_total, out->group_exp);
    compress_emit<<<L.chunks, kThreadsB, 0, st>>>(group_offsets, K, gmax, tile_count, L.tiles_a, stage_idx,
                                                 stage_val, kept_count, chunk_total, out->words, out->capacity,
                                                 out->nnz, out->n_criterion, out->n_dropped, out->dev_status);
    count_launch(3);
    VGC_CUDA_OK(cudaGetLastError());
    return VGC_OK;
}

// ------------------------------------------------------------------------------------------
// Allocation-free variant of vgc_compress: the scratch lives in the library image
// ------------------------------------------------------------------------------------------
// Some callers cannot hand the library a workspace because they cannot allocate device memory at the
// point where they call it: code running under a memory plan fixed ahead of time (every byte of the
// device budget already assigned), plug-ins called from inside another framework's step where
// cudaMalloc would synchronise the device or is simply forbidden, and embedding hosts that expose
// only the tensors they pass in.  For them the scratch of vgc_compress is a fixed array that every
// GPU loading this library reserves until the process exits; its size bounds the buffer length.
namespace vgc {
constexpr size_t kStaticMaxParams = VGC_COMPRESS_STATIC_MAX_PARAMS;
constexpr int kStaticMaxGroups = VGC_COMPRESS_STATIC_MAX_GROUPS;
// worst-case layout: per-tensor maxima, per-tile counts, chunk totals, 8 bytes of staging per parameter
constexpr size_t kStaticScratchBytes = 8 * kStaticMaxParams + (kStaticMaxParams / kTileA) * 12 + kStaticMaxGroups * 4 + 64 * 1024;
static __device__ __align__(256) unsigned char g_compress_scratch[kStaticScratchBytes];
}  // namespace vgc

extern "C" vgc_status vgc_compress_static(const float *g, const float *s, float *r, float *v, size_t n,
                                          const uint32_t *group_offsets, int K, float alpha, float zeta,
                                          const vgc_message *out, vgc_stream_t stream)
{
    if (n > kStaticMaxParams || K > kStaticMaxGroups) return VGC_ERR_UNSUPPORTED;
    if (n == 0) return VGC_OK;
    if (K < 1) return VGC_ERR_INVALID_ARG;
    if (compress_layout(n, K).total > kStaticScratchBytes) return VGC_ERR_UNSUPPORTED;
    // Host code sees g_compress_scratch only as a stand-in for the device array: the address a kernel can
    // use has to be asked for, once per device, with that device current.
    constexpr int kMaxDevices = 64;
    static void *scratch_of_device[kMaxDevices] = {};
    int dev = -1;
    VGC_CUDA_OK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return VGC_ERR_UNSUPPORTED;
    if (!scratch_of_device[dev]) {
        void *p = nullptr;
        VGC_CUDA_OK(cudaGetSymbolAddress(&p, g_compress_scratch));
        if (!p) return VGC_ERR_CUDA;
        scratch_of_device[dev] = p;
    }
    return vgc_compress(g, s, r, v, n, group_offsets, K, alpha, zeta, out, scratch_of_device[dev], kStaticScratchBytes,
                        stream);
}
