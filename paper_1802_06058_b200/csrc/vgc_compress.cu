// vgc_compress: one step of Algorithm 1 ("Basic") over the flat parameter buffer followed by
// Encode() -- the 4-bit quantiser of Sec. 4.2 in the bit-level form of Sec. 4.4 and the
// 32-bit (value, index) word.
//
// Two kernels on one stream:
//   phase A  streams g, s, r, v once (16 B read + 8 B written per parameter), applies the send
//            test, writes r, v back and compacts the selected (index, value) pairs IN INDEX
//            ORDER into a staging area; a per-tensor atomicMax on |value| bit patterns yields
//            M_k.  Ordered compaction across thread blocks uses a decoupled look-back over
//            per-tile counts, with tiles numbered by an atomic ticket.
//   phase B  runs over the staged pairs only: quantises against E_k = floor(log2 M_k), drops
//            d > 7, compacts again in order and packs the words.
// The per-tensor maximum has to be complete before any value can be quantised, which is why
// the work is split in two; the staged pairs are a small fraction of the buffer.
#include "vgc_common.cuh"

namespace vgc {

constexpr int kThreads = 256;
constexpr int kRowsA = 4;                            // float4 vectors per thread per tile
constexpr int kTileA = kThreads * kRowsA * 4;        // 4096 parameters per tile
constexpr int kRowsB = 8;                            // staged pairs per thread per tile
constexpr int kTileB = kThreads * kRowsB;            // 2048 staged pairs per tile
constexpr int kOffsSmem = 1024;                      // group offsets cached in shared memory

struct CompressHeader {      // first bytes of the workspace, zeroed by every call
    uint32_t ticket_a;
    uint32_t ticket_b;
    uint32_t nnz_a;          // elements that passed the send test
    uint32_t pad;
};

struct CompressLayout {
    size_t gmax, status_a, status_b, stage_idx, stage_val, total;
    size_t zero_bytes;       // header + gmax + both status arrays are cleared per call
    uint32_t tiles_a, tiles_b;
};

static CompressLayout compress_layout(size_t n, int K, size_t stage_capacity)
{
    CompressLayout L;
    L.tiles_a = (uint32_t)((n + kTileA - 1) / kTileA);
    L.tiles_b = (uint32_t)((stage_capacity + kTileB - 1) / kTileB);
    size_t off = sizeof(CompressHeader);
    L.gmax = off;          off = round_up(off + sizeof(uint32_t) * (size_t)K, 16);
    L.status_a = off;      off += sizeof(uint64_t) * L.tiles_a;
    L.status_b = off;      off += sizeof(uint64_t) * L.tiles_b;
    off = round_up(off, 256);
    L.zero_bytes = off;
    L.stage_idx = off;     off = round_up(off + sizeof(uint32_t) * stage_capacity, 256);
    L.stage_val = off;     off = round_up(off + sizeof(uint32_t) * stage_capacity, 256);
    L.total = off;
    return L;
}

// ------------------------------------------------------------------------------------------
// phase A
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
compress_phase_a(const float *__restrict__ g, const float *__restrict__ s, float *__restrict__ r,
                 float *__restrict__ v, size_t n, const uint32_t *__restrict__ group_offsets, int K,
                 float alpha, float zeta, CompressHeader *hdr, uint32_t *gmax, uint64_t *status,
                 uint32_t *__restrict__ stage_idx, uint32_t *__restrict__ stage_val, size_t stage_capacity,
                 uint8_t *__restrict__ mask, uint32_t *dev_status, uint32_t n_tiles)
{
    __shared__ uint32_t sm_idx[kTileA];
    __shared__ uint32_t sm_val[kTileA];
    __shared__ uint32_t sm_offs[kOffsSmem];
    __shared__ uint32_t sm_part[kRowsA * (kThreads / kWarp)];   // 32 per-(row, warp) counts
    __shared__ uint32_t sm_tile[2];
    __shared__ uint32_t sm_excl, sm_total, sm_gmax;
    __shared__ int sm_klo, sm_khi;

    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool offs_in_smem = (K + 1) <= kOffsSmem;
    if (offs_in_smem)
        for (int i = tid; i <= K; i += kThreads) sm_offs[i] = group_offsets[i];
    const uint32_t *offs = offs_in_smem ? sm_offs : group_offsets;
    if (tid == 0) sm_tile[0] = atomicAdd(&hdr->ticket_a, 1u);
    __syncthreads();

    for (uint32_t it = 0;; ++it) {
        const uint32_t tile = sm_tile[it & 1];
        if (tile >= n_tiles) break;
        const size_t base = (size_t)tile * kTileA;
        if (tid == 0) {                                // ticket of the next tile, off the critical path
            sm_tile[(it + 1) & 1] = atomicAdd(&hdr->ticket_a, 1u);
            sm_gmax = 0;
        }
        if (tid == 32) {                               // weight tensors this tile touches
            const size_t last = (base + kTileA < n ? base + kTileA : n) - 1;
            sm_klo = group_of(offs, K, (uint32_t)base);
            sm_khi = group_of(offs, K, (uint32_t)last);
        }

        // ---- load: thread t owns elements base + (j*256 + t)*4 + {0..3}, j = 0..3
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

        // ---- ordered positions inside the tile: warp scan of the packed per-row counts
        uint32_t incl = packed;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t up = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += up;
        }
        if (lane == 31) {
#pragma unroll
            for (int j = 0; j < kRowsA; ++j) sm_part[j * (kThreads / kWarp) + warp] = (incl >> (8 * j)) & 0xFFu;
        }
        const uint32_t warp_max = __reduce_max_sync(0xffffffffu, my_max);
        __syncthreads();                                           // (1) parts, sm_gmax = 0, sm_klo/khi
        if (lane == 0 && warp_max) atomicMax(&sm_gmax, warp_max);
        if (warp == 0) {
            const uint32_t t = sm_part[lane];
            uint32_t ti = t;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t up = __shfl_up_sync(0xffffffffu, ti, d);
                if (lane >= d) ti += up;
            }
            const uint32_t total = __shfl_sync(0xffffffffu, ti, 31);
            sm_part[lane] = ti - t;
            const uint32_t excl = lookback_exclusive(status, tile, total, dev_status);
            if (lane == 0) {
                sm_excl = excl;
                sm_total = total;
                if (tile == n_tiles - 1) hdr->nnz_a = excl + total;
                if ((size_t)excl + total > stage_capacity) atomicOr(dev_status, VGC_DEV_CAPACITY);
            }
        }
        __syncthreads();                                           // (2) offsets, prefix, sm_gmax
        const uint32_t excl = sm_excl, total = sm_total;
        const bool one_group = sm_klo == sm_khi;
        if (tid == 0 && one_group && sm_gmax) atomicMax(&gmax[sm_klo], sm_gmax);
#pragma unroll
        for (int j = 0; j < kRowsA; ++j) {
            const uint32_t row_bits = (send_bits >> (4 * j)) & 0xFu;
            if (row_bits) {
                const uint32_t e = (uint32_t)(base + (size_t)(j * kThreads + tid) * 4);
                uint32_t at = sm_part[j * (kThreads / kWarp) + warp] + ((incl >> (8 * j)) & 0xFFu) -
                              (uint32_t)__popc(row_bits);
                const float *Gj = reinterpret_cast<const float *>(&G[j]);
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    if (row_bits & (1u << q)) {
                        const uint32_t bits = __float_as_uint(Gj[q]);
                        sm_idx[at] = e + q;
                        sm_val[at] = bits;
                        ++at;
                        if (!one_group)
                            atomicMax(&gmax[group_of(offs, K, e + q)], bits & 0x7FFFFFFFu);
                    }
            }
        }
        __syncthreads();                                           // (3) compacted tile in shared memory
        for (uint32_t q = tid; q < total; q += kThreads) {
            const size_t p = (size_t)excl + q;
            if (p < stage_capacity) {
                stage_idx[p] = sm_idx[q];
                stage_val[p] = sm_val[q];
            }
        }
        __syncthreads();                                           // (4) before the next tile reuses smem
    }
}

// ------------------------------------------------------------------------------------------
// phase B
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kThreads)
compress_phase_b(const uint32_t *__restrict__ group_offsets, int K, CompressHeader *hdr,
                 const uint32_t *__restrict__ gmax, uint64_t *status,
                 const uint32_t *__restrict__ stage_idx, const uint32_t *__restrict__ stage_val,
                 size_t stage_capacity, uint32_t *__restrict__ words, uint32_t capacity,
                 int32_t *__restrict__ group_exp, uint32_t *nnz_out, uint32_t *n_criterion,
                 uint32_t *n_dropped, uint32_t *dev_status)
{
    __shared__ uint32_t sm_words[kTileB];
    __shared__ uint32_t sm_offs[kOffsSmem];
    __shared__ uint32_t sm_part[kRowsB * (kThreads / kWarp)];   // 64 per-(row, warp) counts
    __shared__ uint32_t sm_tile[2];
    __shared__ uint32_t sm_excl, sm_total;

    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool offs_in_smem = (K + 1) <= kOffsSmem;
    if (offs_in_smem)
        for (int i = tid; i <= K; i += kThreads) sm_offs[i] = group_offsets[i];
    const uint32_t *offs = offs_in_smem ? sm_offs : group_offsets;

    const uint32_t n_passed = hdr->nnz_a;                         // written by phase A
    const uint32_t n_staged = n_passed < stage_capacity ? n_passed : (uint32_t)stage_capacity;
    const uint32_t n_tiles = (n_staged + kTileB - 1) / kTileB;

    if (blockIdx.x == 0) {
        for (int k = tid; k < K; k += kThreads) {
            const uint32_t m = gmax[k];
            group_exp[k] = m ? (int32_t)((m >> 23) & 0xFFu) - 127 : VGC_EXP_NONE;
        }
        if (tid == 0) {
            *n_criterion = n_passed;
            if (n_tiles == 0) { *nnz_out = 0; *n_dropped = n_passed; }
        }
    }
    if (tid == 0) sm_tile[0] = atomicAdd(&hdr->ticket_b, 1u);
    __syncthreads();

    for (uint32_t it = 0;; ++it) {
        const uint32_t tile = sm_tile[it & 1];
        if (tile >= n_tiles) break;
        if (tid == 0) sm_tile[(it + 1) & 1] = atomicAdd(&hdr->ticket_b, 1u);

        uint32_t word[kRowsB];
        uint32_t keep_bits = 0;
        uint32_t my_pos[kRowsB];
#pragma unroll
        for (int j = 0; j < kRowsB; ++j) {
            const uint32_t q = tile * kTileB + j * kThreads + tid;
            bool keep = false;
            word[j] = 0;
            if (q < n_staged) {
                const uint32_t idx = stage_idx[q];
                const uint32_t bits = stage_val[q];
                const uint32_t m = gmax[group_of(offs, K, idx)];
                const int32_t Ek = (int32_t)((m >> 23) & 0xFFu) - 127;       // floor(log2 M_k)
                const uint32_t a = bits & 0x7FFFFFFFu;
                const int32_t e1 = (int32_t)((a + 0x00400000u) >> 23) - 127; // nearer power of two
                const int32_t e = e1 < Ek ? e1 : Ek;                         // cut at 2^E_k
                const int32_t d = Ek - e;
                keep = d <= 7;
                word[j] = (idx << 4) | ((bits >> 31) << 3) | (uint32_t)(d & 7);
            }
            const uint32_t ballot = __ballot_sync(0xffffffffu, keep);
            my_pos[j] = __popc(ballot & ((1u << lane) - 1u));
            if (keep) keep_bits |= 1u << j;
            if (lane == 0) sm_part[j * (kThreads / kWarp) + warp] = __popc(ballot);
        }
        __syncthreads();                                           // (1)
        if (warp == 0) {
            const uint32_t t0 = sm_part[2 * lane], t1 = sm_part[2 * lane + 1];
            const uint32_t t = t0 + t1;
            uint32_t ti = t;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t up = __shfl_up_sync(0xffffffffu, ti, d);
                if (lane >= d) ti += up;
            }
            const uint32_t total = __shfl_sync(0xffffffffu, ti, 31);
            sm_part[2 * lane] = ti - t;
            sm_part[2 * lane + 1] = ti - t + t0;
            const uint32_t excl = lookback_exclusive(status, tile, total, dev_status);
            if (lane == 0) {
                sm_excl = excl;
                sm_total = total;
                if (tile == n_tiles - 1) {
                    *nnz_out = excl + total;
                    *n_dropped = n_passed - (excl + total);
                }
                if (excl + total > capacity) atomicOr(dev_status, VGC_DEV_CAPACITY);
            }
        }
        __syncthreads();                                           // (2)
        const uint32_t excl = sm_excl, total = sm_total;
#pragma unroll
        for (int j = 0; j < kRowsB; ++j)
            if (keep_bits & (1u << j)) sm_words[sm_part[j * (kThreads / kWarp) + warp] + my_pos[j]] = word[j];
        __syncthreads();                                           // (3)
        for (uint32_t q = tid; q < total; q += kThreads)
            if (excl + q < capacity) words[excl + q] = sm_words[q];
        __syncthreads();                                           // (4)
    }
}

}  // namespace vgc

// ------------------------------------------------------------------------------------------
// C ABI
// ------------------------------------------------------------------------------------------
using namespace vgc;

extern "C" size_t vgc_compress_workspace_bytes(size_t n, int K, size_t stage_capacity)
{
    if (K < 1) K = 1;
    if (stage_capacity > n) stage_capacity = n;
    return compress_layout(n, K, stage_capacity).total;
}

extern "C" vgc_status vgc_compress(const float *g, const float *s, float *r, float *v, size_t n,
                                   const uint32_t *group_offsets, int K, float alpha, float zeta,
                                   size_t stage_capacity, const vgc_message *out,
                                   void *ws, size_t ws_bytes, vgc_stream_t stream)
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
    if (stage_capacity > n) stage_capacity = n;
    const CompressLayout L = compress_layout(n, K, stage_capacity);
    if (ws_bytes < L.total) return VGC_ERR_WORKSPACE;

    char *base = static_cast<char *>(ws);
    CompressHeader *hdr = reinterpret_cast<CompressHeader *>(base);
    uint32_t *gmax = reinterpret_cast<uint32_t *>(base + L.gmax);
    uint64_t *status_a = reinterpret_cast<uint64_t *>(base + L.status_a);
    uint64_t *status_b = reinterpret_cast<uint64_t *>(base + L.status_b);
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
    const uint32_t grid_a = L.tiles_a < (uint32_t)(sm_count * 4) ? L.tiles_a : (uint32_t)(sm_count * 4);
    compress_phase_a<<<grid_a, kThreads, 0, st>>>(g, s, r, v, n, group_offsets, K, alpha, zeta, hdr, gmax,
                                                  status_a, stage_idx, stage_val, stage_capacity, out->mask,
                                                  out->dev_status, L.tiles_a);
    uint32_t grid_b = L.tiles_b < (uint32_t)(sm_count * 4) ? L.tiles_b : (uint32_t)(sm_count * 4);
    if (grid_b == 0) grid_b = 1;
    compress_phase_b<<<grid_b, kThreads, 0, st>>>(group_offsets, K, hdr, gmax, status_b, stage_idx, stage_val,
                                                  stage_capacity, out->words, out->capacity, out->group_exp,
                                                  out->nnz, out->n_criterion, out->n_dropped, out->dev_status);
    VGC_CUDA_OK(cudaGetLastError());
    return VGC_OK;
}
