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
//   phase B  runs over the staged pairs only: quantises against E_k = floor(log2 M_k), drops
//            d > 7 and packs the words in ascending index order.  One warp owns one segment;
//            positions across thread blocks come from a decoupled look-back over per-tile
//            counts, with tiles numbered by an atomic ticket and every wait bounded.
// The per-tensor maximum has to be complete before any value can be quantised, which is why
// the work is split in two; the staged pairs are a small fraction of the buffer.
#include "vgc_common.cuh"

namespace vgc {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / kWarp;             // 8
constexpr int kRowsA = 2;                            // float4 vectors per thread per tile
constexpr int kTileA = kThreads * kRowsA * 4;        // 2048 parameters per tile = one staging segment
constexpr int kSegPerTileB = kWarps;                 // phase B: one warp per segment
constexpr int kOffsSmem = 1024;                      // group offsets cached in shared memory

struct CompressHeader {      // first bytes of the workspace, zeroed by every call
    uint32_t ticket_b;
    uint32_t pad[3];
};

struct CompressLayout {
    size_t gmax, status_b, tile_count, stage_idx, stage_val, total;
    size_t zero_bytes;       // header + gmax + status array are cleared per call
    uint32_t tiles_a, tiles_b;
};

static CompressLayout compress_layout(size_t n, int K)
{
    CompressLayout L;
    L.tiles_a = (uint32_t)((n + kTileA - 1) / kTileA);
    L.tiles_b = (L.tiles_a + kSegPerTileB - 1) / kSegPerTileB;
    size_t off = sizeof(CompressHeader);
    L.gmax = off;          off = round_up(off + sizeof(uint32_t) * (size_t)K, 16);
    L.status_b = off;      off += sizeof(uint64_t) * L.tiles_b;
    off = round_up(off, 256);
    L.zero_bytes = off;
    L.tile_count = off;    off = round_up(off + sizeof(uint32_t) * L.tiles_a, 256);
    const size_t slots = (size_t)L.tiles_a * kTileA;
    L.stage_idx = off;     off = round_up(off + sizeof(uint32_t) * slots, 256);
    L.stage_val = off;     off = round_up(off + sizeof(uint32_t) * slots, 256);
    L.total = off;
    return L;
}

// ------------------------------------------------------------------------------------------
// phase A
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads, 4)
compress_phase_a(const float *__restrict__ g, const float *__restrict__ s, float *__restrict__ r,
                 float *__restrict__ v, size_t n, const uint32_t *__restrict__ group_offsets, int K,
                 float alpha, float zeta, uint32_t *gmax, uint32_t *__restrict__ tile_count,
                 uint32_t *__restrict__ stage_idx, uint32_t *__restrict__ stage_val,
                 uint8_t *__restrict__ mask, uint32_t n_tiles)
{
    __shared__ uint32_t sm_offs[kOffsSmem];
    __shared__ uint32_t sm_part[2][32];                 // per-(row, warp) counts, double buffered
    __shared__ uint32_t sm_wmax[2][kWarps];
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
                S[j] = ld_stream_f4(s + e);
                R[j] = *reinterpret_cast<const float4 *>(r + e);
                V[j] = *reinterpret_cast<const float4 *>(v + e);
            } else {
                float tg[4], ts[4], tr[4], tv[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const bool in = e + q < n;
                    tg[q] = in ? g[e + q] : 0.f;  ts[q] = in ? s[e + q] : 0.f;
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
        uint32_t my_max = 0;
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
                const float v1 = __fadd_rn(Vj[q], Sj[q]);
                const float lhs = __fmul_rn(r1, r1);
                const float rhs = __fmul_rn(alpha, v1);
                const bool send = (lhs > rhs) && (e + q < n);
                Gj[q] = r1;                                       // value handed to Encode()
                Rj[q] = send ? 0.f : r1;
                Vj[q] = send ? 0.f : __fmul_rn(v1, zeta);
                if (send) {
                    row_bits |= 1u << q;
                    my_max = max(my_max, __float_as_uint(r1) & 0x7FFFFFFFu);
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
        if (lane == 31) {
#pragma unroll
            for (int j = 0; j < kRowsA; ++j) sm_part[buf][j * kWarps + warp] = (incl >> (8 * j)) & 0xFFu;
            sm_wmax[buf][warp] = warp_max;
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

constexpr uint64_t kPassedShift = 31;       // look-back payload: passed << 31 | kept (each < 2^29)

__global__ void __launch_bounds__(kThreads)
compress_phase_b(const uint32_t *__restrict__ group_offsets, int K, CompressHeader *hdr,
                 const uint32_t *__restrict__ gmax, const uint32_t *__restrict__ tile_count, uint32_t n_tiles_a,
                 const uint32_t *__restrict__ stage_idx, const uint32_t *__restrict__ stage_val,
                 uint64_t *status, uint32_t *__restrict__ words, uint32_t capacity,
                 int32_t *__restrict__ group_exp, uint32_t *nnz_out, uint32_t *n_criterion,
                 uint32_t *n_dropped, uint32_t *dev_status)
{
    __shared__ uint32_t sm_offs[kOffsSmem];
    __shared__ uint32_t sm_kept[kWarps], sm_passed[kWarps], sm_excl[kWarps];
    __shared__ uint32_t sm_tile[2];

    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool offs_in_smem = (K + 1) <= kOffsSmem;
    if (offs_in_smem)
        for (int i = tid; i <= K; i += kThreads) sm_offs[i] = group_offsets[i];
    const uint32_t *offs = offs_in_smem ? sm_offs : group_offsets;
    const uint32_t n_tiles = (n_tiles_a + kSegPerTileB - 1) / kSegPerTileB;

    if (blockIdx.x == 0)
        for (int k = tid; k < K; k += kThreads) {
            const uint32_t m = gmax[k];
            group_exp[k] = m ? (int32_t)((m >> 23) & 0xFFu) - 127 : VGC_EXP_NONE;
        }
    if (tid == 0) sm_tile[0] = atomicAdd(&hdr->ticket_b, 1u);
    __syncthreads();

    for (uint32_t it = 0;; ++it) {
        const uint32_t tile = sm_tile[it & 1];
        if (tile >= n_tiles) break;
        if (tid == 0) sm_tile[(it + 1) & 1] = atomicAdd(&hdr->ticket_b, 1u);

        const uint32_t seg = tile * kSegPerTileB + warp;
        const uint32_t count = seg < n_tiles_a ? tile_count[seg] : 0;
        const uint32_t *seg_idx = stage_idx + (size_t)seg * kTileA;
        const uint32_t *seg_val = stage_val + (size_t)seg * kTileA;

        // pass 1: how many of this segment's pairs survive the quantiser
        int k = 0;
        int32_t Ek = INT32_MIN;
        uint32_t kept = 0;
        for (uint32_t q0 = 0; q0 < count; q0 += 32) {
            const uint32_t q = q0 + lane;
            bool keep = false;
            if (q < count) {
                uint32_t word;
                keep = encode_pair(seg_idx[q], seg_val[q], offs, K, gmax, k, Ek, word);
            }
            kept += __popc(__ballot_sync(0xffffffffu, keep));
        }
        if (lane == 0) { sm_kept[warp] = kept; sm_passed[warp] = count; }
        __syncthreads();                                           // (1)
        if (warp == 0) {
            const uint32_t mine = lane < kWarps ? sm_kept[lane] : 0;
            const uint32_t pass = lane < kWarps ? sm_passed[lane] : 0;
            uint32_t ki = mine, pi = pass;
#pragma unroll
            for (int d = 1; d < kWarps; d <<= 1) {
                const uint32_t ku = __shfl_up_sync(0xffffffffu, ki, d);
                const uint32_t pu = __shfl_up_sync(0xffffffffu, pi, d);
                if (lane >= d) { ki += ku; pi += pu; }
            }
            const uint32_t tot_kept = __shfl_sync(0xffffffffu, ki, kWarps - 1);
            const uint32_t tot_pass = __shfl_sync(0xffffffffu, pi, kWarps - 1);
            const uint64_t excl = lookback_exclusive(status, tile, ((uint64_t)tot_pass << kPassedShift) | tot_kept,
                                                     dev_status);
            const uint32_t excl_kept = (uint32_t)(excl & ((1ull << kPassedShift) - 1));
            const uint32_t excl_pass = (uint32_t)(excl >> kPassedShift);
            if (lane < kWarps) sm_excl[lane] = excl_kept + ki - mine;
            if (lane == 0) {
                if (tile == n_tiles - 1) {
                    *nnz_out = excl_kept + tot_kept;
                    *n_criterion = excl_pass + tot_pass;
                    *n_dropped = (excl_pass + tot_pass) - (excl_kept + tot_kept);
                }
                if (excl_kept + tot_kept > capacity) atomicOr(dev_status, VGC_DEV_CAPACITY);
            }
        }
        __syncthreads();                                           // (2)
        // pass 2: same pairs again (cache hits), now with their final positions
        uint32_t pos = sm_excl[warp];
        for (uint32_t q0 = 0; q0 < count; q0 += 32) {
            const uint32_t q = q0 + lane;
            bool keep = false;
            uint32_t word = 0;
            if (q < count) keep = encode_pair(seg_idx[q], seg_val[q], offs, K, gmax, k, Ek, word);
            const uint32_t ballot = __ballot_sync(0xffffffffu, keep);
            const uint32_t p = pos + __popc(ballot & ((1u << lane) - 1u));
            if (keep && p < capacity) words[p] = word;
            pos += __popc(ballot);
        }
    }
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
    if (!g || !s || !r || !v || !group_offsets || !ws) return VGC_ERR_INVALID_ARG;
    if (!out->group_exp || !out->nnz || !out->n_criterion || !out->n_dropped || !out->dev_status)
        return VGC_ERR_INVALID_ARG;
    if (out->capacity && !out->words) return VGC_ERR_INVALID_ARG;
    if (!aligned16(g) || !aligned16(s) || !aligned16(r) || !aligned16(v) || !aligned16(ws) ||
        (out->mask && (reinterpret_cast<uintptr_t>(out->mask) & 3u)))
        return VGC_ERR_INVALID_ARG;
    const CompressLayout L = compress_layout(n, K);
    if (ws_bytes < L.total) return VGC_ERR_WORKSPACE;

    char *base = static_cast<char *>(ws);
    CompressHeader *hdr = reinterpret_cast<CompressHeader *>(base);
    uint32_t *gmax = reinterpret_cast<uint32_t *>(base + L.gmax);
    uint64_t *status_b = reinterpret_cast<uint64_t *>(base + L.status_b);
    uint32_t *tile_count = reinterpret_cast<uint32_t *>(base + L.tile_count);
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
    compress_phase_a<<<grid_a, kThreads, 0, st>>>(g, s, r, v, n, group_offsets, K, alpha, zeta, gmax, tile_count,
                                                  stage_idx, stage_val, out->mask, L.tiles_a);
    const uint32_t grid_b = L.tiles_b < (uint32_t)(sm_count * 8) ? L.tiles_b : (uint32_t)(sm_count * 8);
    compress_phase_b<<<grid_b, kThreads, 0, st>>>(group_offsets, K, hdr, gmax, tile_count, L.tiles_a, stage_idx,
                                                  stage_val, status_b, out->words, out->capacity, out->group_exp,
                                                  out->nnz, out->n_criterion, out->n_dropped, out->dev_status);
    count_launch(2);
    VGC_CUDA_OK(cudaGetLastError());
    return VGC_OK;
}
