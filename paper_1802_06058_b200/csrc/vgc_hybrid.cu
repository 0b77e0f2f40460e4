// Hybrid algorithm (Algorithm 2): variance criterion on top of the fixed threshold tau of Strom's method,
// with the variance correction of Sec. 4.5.  Two passes like the basic compressor, minus the quantiser:
//
//   hybrid_phase_a   one streaming pass over g, s, r, v (24 bytes per parameter, 20 when s == NULL): the
//                    loop body of Algorithm 2, the r / v write-back, and the sent elements' words
//                    (index << 4 | sign << 3) staged in the 2048-slot segment of their tile, in index order
//   hybrid_totals    sent elements per chunk of 32 tiles
//   hybrid_pack      ordered copy of the staged words into the message, nnz, capacity flag
//
// No block waits on another block anywhere.
#include "vgc_common.cuh"

namespace vgc {
namespace hybrid {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / kWarp;             // 8
constexpr int kRows = 2;                             // float4 vectors per thread per tile
constexpr int kTile = kThreads * kRows * 4;          // 2048 parameters per tile = one staging segment
constexpr int kSegPerChunk = 32;

struct Layout {
    size_t tile_count, chunk_total, stage, total;
    uint32_t tiles, chunks;
};

static Layout layout(size_t n)
{
    Layout L;
    L.tiles = (uint32_t)((n + kTile - 1) / kTile);
    L.chunks = (L.tiles + kSegPerChunk - 1) / kSegPerChunk;
    size_t off = 0;
    L.tile_count = off;   off = round_up(off + sizeof(uint32_t) * L.tiles, 256);
    L.chunk_total = off;  off = round_up(off + sizeof(uint32_t) * L.chunks, 256);
    L.stage = off;        off = round_up(off + sizeof(uint32_t) * (size_t)L.tiles * kTile, 256);
    L.total = off;
    return L;
}

// kHasS = false: this step's squared-gradient sums were accumulated straight into v by the caller.
// kPre: the correction uses |r| from before the subtraction of tau (the (a-b)^2 reading of Sec. 4.5);
// otherwise |r| after it (the order in which the listing of Algorithm 2 states the two updates).
template <bool kHasS, bool kPre>
__global__ void __launch_bounds__(kThreads, 4)
hybrid_phase_a(const float *__restrict__ g, const float *__restrict__ s, float *__restrict__ r,
               float *__restrict__ v, size_t n, float alpha, float zeta, float tau,
               uint32_t *__restrict__ tile_count, uint32_t *__restrict__ stage, uint8_t *__restrict__ mask,
               uint32_t n_tiles)
{
    __shared__ uint32_t sm_part[2][32];                 // per-(row, warp) counts, double buffered
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (tid < 64) (&sm_part[0][0])[tid] = 0;            // entries past kRows*kWarps stay zero
    __syncthreads();
    const float tau_sq = __fmul_rn(tau, tau);

    uint32_t buf = 0;
    for (uint32_t tile = blockIdx.x; tile < n_tiles; tile += gridDim.x, buf ^= 1) {
        const size_t base = (size_t)tile * kTile;
        float4 G[kRows], S[kRows], R[kRows], V[kRows];
#pragma unroll
        for (int j = 0; j < kRows; ++j) {
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

        // ---- Algorithm 2 loop body; every operation rounded on its own (no FMA)
        uint32_t send_bits = 0, sign_bits = 0;   // bit j*4+q
        uint32_t packed = 0;                     // per-row counts, 8 bits each
#pragma unroll
        for (int j = 0; j < kRows; ++j) {
            const size_t e = base + (size_t)(j * kThreads + tid) * 4;
            const float *Gj = reinterpret_cast<const float *>(&G[j]);
            const float *Sj = reinterpret_cast<const float *>(&S[j]);
            float *Rj = reinterpret_cast<float *>(&R[j]);
            float *Vj = reinterpret_cast<float *>(&V[j]);
            uint32_t row_bits = 0, row_sign = 0;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                float r1 = __fadd_rn(Rj[q], Gj[q]);
                float v1 = kHasS ? __fadd_rn(Vj[q], Sj[q]) : Vj[q];
                const float absr = fabsf(r1);
                const bool send = (absr > tau) && (__fmul_rn(r1, r1) > __fmul_rn(alpha, v1)) && (e + q < n);
                if (send) {
                    const bool neg = __float_as_uint(r1) >> 31;
                    const float r2 = neg ? __fadd_rn(r1, tau) : __fsub_rn(r1, tau);     // r -= Sign(r) tau
                    const float a = kPre ? absr : fabsf(r2);
                    const float cross = __fmul_rn(__fmul_rn(2.0f, a), tau);
                    const float corr = __fadd_rn(__fsub_rn(v1, cross), tau_sq);       // v - 2|r|tau + tau^2
                    v1 = corr > 0.f ? corr : 0.f;
                    r1 = r2;
                    row_bits |= 1u << q;
                    row_sign |= (uint32_t)neg << q;
                }
                Rj[q] = r1;
                Vj[q] = __fmul_rn(v1, zeta);                                          // decay at every step
            }
            send_bits |= row_bits << (4 * j);
            sign_bits |= row_sign << (4 * j);
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

        // ---- ordered positions inside the tile: warp scan of the packed per-row counts, then every
        //      warp scans the 16 (row, warp) totals by itself (one barrier per tile)
        uint32_t incl = packed;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t up = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += up;
        }
        if (lane == 31) {
#pragma unroll
            for (int j = 0; j < kRows; ++j) sm_part[buf][j * kWarps + warp] = (incl >> (8 * j)) & 0xFFu;
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
        uint32_t *seg = stage + base;
#pragma unroll
        for (int j = 0; j < kRows; ++j) {
            const uint32_t row_base = __shfl_sync(0xffffffffu, pexcl, j * kWarps + warp);
            const uint32_t row_bits = (send_bits >> (4 * j)) & 0xFu;
            if (row_bits) {
                const uint32_t e = (uint32_t)(base + (size_t)(j * kThreads + tid) * 4);
                uint32_t at = row_base + ((incl >> (8 * j)) & 0xFFu) - (uint32_t)__popc(row_bits);
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    if (row_bits & (1u << q))
                        seg[at++] = ((e + q) << 4) | (((sign_bits >> (4 * j + q)) & 1u) << 3);
            }
        }
        if (tid == 0) tile_count[tile] = total;
    }
}

// one warp per chunk of 32 tiles
__global__ void __launch_bounds__(kThreads)
hybrid_totals(const uint32_t *__restrict__ tile_count, uint32_t n_tiles, uint32_t *__restrict__ chunk_total,
              uint32_t n_chunks)
{
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t chunk = blockIdx.x * kWarps + (threadIdx.x >> 5);
    if (chunk >= n_chunks) return;
    const uint32_t seg = chunk * kSegPerChunk + lane;
    uint32_t c = seg < n_tiles ? tile_count[seg] : 0;
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) c += __shfl_xor_sync(0xffffffffu, c, d);
    if (lane == 0) chunk_total[chunk] = c;
}

constexpr int kThreadsPack = kSegPerChunk * kWarp;   // 1024: one warp per segment of the chunk

__global__ void __launch_bounds__(kThreadsPack)
hybrid_pack(const uint32_t *__restrict__ tile_count, uint32_t n_tiles, const uint32_t *__restrict__ chunk_total,
            const uint32_t *__restrict__ stage, uint32_t *__restrict__ words, uint32_t capacity,
            uint32_t *nnz_out, uint32_t *dev_status)
{
    __shared__ uint32_t sm_tot[kSegPerChunk];
    __shared__ uint32_t sm_pos[kSegPerChunk];
    const uint32_t tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    uint32_t before = 0;                               // words of all chunks before this one
    for (uint32_t c = tid; c < blockIdx.x; c += kThreadsPack) before += chunk_total[c];
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) before += __shfl_xor_sync(0xffffffffu, before, d);
    if (lane == 0) sm_tot[warp] = before;
    __syncthreads();
    before = 0;
#pragma unroll
    for (int w = 0; w < kSegPerChunk; ++w) before += sm_tot[w];

    if (warp == 0) {
        const uint32_t seg = blockIdx.x * kSegPerChunk + lane;
        const uint32_t mine = seg < n_tiles ? tile_count[seg] : 0;
        uint32_t incl = mine;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const uint32_t up = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= d) incl += up;
        }
        sm_pos[lane] = before + incl - mine;
        if (lane == 31) {
            const uint32_t end = before + incl;
            if (end > capacity) atomicOr(dev_status, VGC_DEV_CAPACITY);
            if (blockIdx.x == gridDim.x - 1) *nnz_out = end;
        }
    }
    __syncthreads();
    // one warp per segment, four 32-wide slices per round so that the loads of a round are in flight together
    const uint32_t seg = blockIdx.x * kSegPerChunk + warp;
    if (seg >= n_tiles) return;
    const uint32_t count = tile_count[seg], pos = sm_pos[warp];
    const uint32_t *src = stage + (size_t)seg * kTile;
    for (uint32_t q0 = 0; q0 < count; q0 += 128) {
        uint32_t held[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t q = q0 + 32 * j + lane;
            held[j] = q < count ? src[q] : 0u;
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const uint32_t q = q0 + 32 * j + lane;
            if (q < count && pos + q < capacity) words[pos + q] = held[j];
        }
    }
}

}  // namespace hybrid
}  // namespace vgc

using namespace vgc;

extern "C" size_t vgc_compress_hybrid_workspace_bytes(size_t n) { return hybrid::layout(n).total; }

extern "C" vgc_status vgc_compress_hybrid(const float *g, const float *s, float *r, float *v, size_t n,
                                          float alpha, float zeta, float tau, int correction_from_updated_r,
                                          const vgc_hybrid_message *out, void *ws, size_t ws_bytes,
                                          vgc_stream_t stream)
{
    if (n == 0) return VGC_OK;
    if (n > VGC_MAX_PARAMS || !out) return VGC_ERR_INVALID_ARG;
    const float fmax = 3.402823466e38f;
    if (!(alpha >= 0.f) || !(alpha <= fmax) || !(zeta >= -fmax) || !(zeta <= fmax) || !(tau >= 0.f) || !(tau <= fmax))
        return VGC_ERR_INVALID_ARG;
    if (!g || !r || !v || !ws || !out->nnz || !out->dev_status) return VGC_ERR_INVALID_ARG;
    if (out->capacity && !out->words) return VGC_ERR_INVALID_ARG;
    if (!aligned16(g) || (s && !aligned16(s)) || !aligned16(r) || !aligned16(v) || !aligned16(ws) ||
        (out->mask && (reinterpret_cast<uintptr_t>(out->mask) & 3u)))
        return VGC_ERR_INVALID_ARG;
    const hybrid::Layout L = hybrid::layout(n);
    if (ws_bytes < L.total) return VGC_ERR_WORKSPACE;

    char *base = static_cast<char *>(ws);
    uint32_t *tile_count = reinterpret_cast<uint32_t *>(base + L.tile_count);
    uint32_t *chunk_total = reinterpret_cast<uint32_t *>(base + L.chunk_total);
    uint32_t *stage = reinterpret_cast<uint32_t *>(base + L.stage);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);

    static int sm_count = 0;
    if (sm_count == 0) {
        int dev = 0, c = 0;
        VGC_CUDA_OK(cudaGetDevice(&dev));
        VGC_CUDA_OK(cudaDeviceGetAttribute(&c, cudaDevAttrMultiProcessorCount, dev));
        sm_count = c > 0 ? c : 148;
    }
    const uint32_t grid_a = L.tiles < (uint32_t)(sm_count * 8) ? L.tiles : (uint32_t)(sm_count * 8);
    const bool pre = !correction_from_updated_r;
#define VGC_HYBRID_LAUNCH(HAS_S, PRE)                                                                             \
    hybrid::hybrid_phase_a<HAS_S, PRE><<<grid_a, hybrid::kThreads, 0, st>>>(g, s, r, v, n, alpha, zeta, tau, tile_count, \
                                                                           stage, out->mask, L.tiles)
    if (s) { if (pre) VGC_HYBRID_LAUNCH(true, true); else VGC_HYBRID_LAUNCH(true, false); }
    else   { if (pre) VGC_HYBRID_LAUNCH(false, true); else VGC_HYBRID_LAUNCH(false, false); }
#undef VGC_HYBRID_LAUNCH
    hybrid::hybrid_totals<<<(L.chunks + hybrid::kWarps - 1) / hybrid::kWarps, hybrid::kThreads, 0, st>>>(
        tile_count, L.tiles, chunk_total, L.chunks);
    hybrid::hybrid_pack<<<L.chunks, hybrid::kThreadsPack, 0, st>>>(tile_count, L.tiles, chunk_total, stage, out->words,
                                                               out->capacity, out->nnz, out->dev_status);
    count_launch(3);
    VGC_CUDA_OK(cudaGetLastError());
    return VGC_OK;
}
