// vgc_pack_indices / vgc_unpack_indices: the index field of a packed message stored as differences in a
// variable-length code (Sec. 4.2, last paragraph: "we can further reduce the number of bits by compressing
// parameter indexes" -- the paper names the idea and does not fix a format; the format is this library's).
//
// The words of a message come in ascending index order.  They are taken in runs of 256; word i of a run becomes
//     v = (idx_i - idx_{i-1}) << 4 | (word_i & 15)        (idx_{-1} = 0 at the start of every run)
// -- the difference above the unchanged 4-bit value field -- written in the base-128 code: seven bits per byte, least
// significant group first, the top bit of a byte set when another byte follows (1 to 5 bytes).  The stream is
//     [table: (runs + 1) x uint32, little endian][payload],   table[j] = offset of run j inside the payload,
// table[runs] = payload length, runs = ceil(nnz / 256).  Runs restart so that they can be coded and decoded side by
// side: one warp per run.
//
//   pack:   pack_count   every lane sizes 8 consecutive words of its warp's run; run and block totals are stored
//           pack_emit    a block adds up the totals of the blocks before it (no waiting on other blocks), a warp scans
//                        its lanes' sizes and every lane writes the bytes of its 8 words
//   unpack: one kernel   a warp copies its run's bytes to shared memory, every lane finds the numbers that END in its
//                        32nd of them (a byte with a clear top bit ends one), a warp scan of their counts gives each
//                        its place in the run, and a second scan over the differences gives the indices
#include "vgc_common.cuh"

namespace vgc {

constexpr int kPackRun = VGC_PACK_RUN;                  // words per run
constexpr int kPackWarps = 8;                           // runs per thread block
constexpr int kPackThreads = 32 * kPackWarps;
constexpr int kPerLane = kPackRun / 32;                 // 8 words per lane
constexpr int kRunBytesMax = 5 * kPackRun;              // 1280
constexpr int kBytesPerLane = kRunBytesMax / 32;        // 40

__device__ __forceinline__ uint32_t code_length(uint32_t v)
{
    return v < (1u << 7) ? 1u : v < (1u << 14) ? 2u : v < (1u << 21) ? 3u : v < (1u << 28) ? 4u : 5u;
}

// the numbers of this lane's 8 words of run `run`, and how many of them exist
__device__ __forceinline__ uint32_t lane_numbers(const uint32_t *__restrict__ words, uint32_t n, uint32_t run, uint32_t lane,
                                                 uint32_t (&v)[kPerLane])
{
    const uint32_t first = run * kPackRun + lane * kPerLane;
    uint32_t prev = (lane == 0 || first >= n) ? 0u : words[first - 1] >> 4;
    uint32_t have = 0;
#pragma unroll
    for (int j = 0; j < kPerLane; ++j) {
        v[j] = 0;
        if (first + j < n) {
            const uint32_t w = words[first + j], idx = w >> 4;
            v[j] = ((idx - prev) << 4) | (w & 15u);
            prev = idx;
            ++have;
        }
    }
    return have;
}

__global__ void __launch_bounds__(kPackThreads)
pack_count(const uint32_t *__restrict__ words, const uint32_t *__restrict__ nnz, uint32_t max_words,
           uint32_t *__restrict__ run_bytes, uint32_t *__restrict__ block_bytes)
{
    __shared__ uint32_t sm_tot[kPackWarps];
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t n = min(*nnz, max_words);
    const uint32_t run = blockIdx.x * kPackWarps + warp;
    // the grid covers the buffer's capacity; blocks past the message's last run have nothing anyone reads
    if ((size_t)blockIdx.x * kPackWarps * kPackRun >= n) return;
    uint32_t v[kPerLane];
    const uint32_t have = lane_numbers(words, n, run, lane, v);
    uint32_t bytes = 0;
#pragma unroll
    for (int j = 0; j < kPerLane; ++j) bytes += (uint32_t)j < have ? code_length(v[j]) : 0u;
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) bytes += __shfl_xor_sync(0xffffffffu, bytes, d);
    if (lane == 0) { run_bytes[run] = bytes; sm_tot[warp] = bytes; }
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t t = 0;
#pragma unroll
        for (int w = 0; w < kPackWarps; ++w) t += sm_tot[w];
        block_bytes[blockIdx.x] = t;
    }
}

__global__ void __launch_bounds__(kPackThreads)
pack_emit(const uint32_t *__restrict__ words, const uint32_t *__restrict__ nnz, uint32_t max_words,
          const uint32_t *__restrict__ run_bytes, const uint32_t *__restrict__ block_bytes, uint8_t *__restrict__ packed,
          size_t capacity, uint32_t *__restrict__ packed_bytes, uint32_t *dev_status)
{
    __shared__ unsigned long long sm_part[kPackWarps];
    __shared__ uint32_t sm_run[kPackWarps];
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t n = min(*nnz, max_words);
    const uint32_t runs = (n + kPackRun - 1) / kPackRun;
    const size_t table_bytes = 4 * ((size_t)runs + 1);
    if (blockIdx.x * kPackWarps > runs) return;                         // nothing of the message or its table here
    // payload bytes of all blocks before this one
    unsigned long long before = 0;
    for (uint32_t b = threadIdx.x; b < blockIdx.x; b += kPackThreads) before += block_bytes[b];
    before = warp_sum_u64(before);
    const uint32_t run = blockIdx.x * kPackWarps + warp;
    if (lane == 0) { sm_part[warp] = before; sm_run[warp] = run < runs ? run_bytes[run] : 0u; }
    __syncthreads();
    before = 0;
    uint32_t in_block = 0;
#pragma unroll
    for (int w = 0; w < kPackWarps; ++w) { before += sm_part[w]; in_block += (uint32_t)w < warp ? sm_run[w] : 0u; }
    const unsigned long long run_off = before + in_block;               // this run's first byte inside the payload

    auto put = [&](size_t at, uint8_t byte) {
        if (at < capacity) packed[at] = byte;
    };
    if (run <= runs && lane < 4) put(4 * (size_t)run + lane, (uint8_t)((uint32_t)run_off >> (8 * lane)));   // table[run]
    if (run == runs) {
        // table[runs] is the payload length: written by the warp whose run number is `runs` (its offset is the total)
        if (lane == 0) {
            const unsigned long long total = table_bytes + run_off;
            *packed_bytes = (uint32_t)total;
            if (total > capacity) atomicOr(dev_status, VGC_DEV_CAPACITY);
        }
    }
    if (run >= runs) return;
    uint32_t v[kPerLane];
    const uint32_t have = lane_numbers(words, n, run, lane, v);
    uint32_t mine = 0;
#pragma unroll
    for (int j = 0; j < kPerLane; ++j) mine += (uint32_t)j < have ? code_length(v[j]) : 0u;
    uint32_t incl = mine;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t up = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += up;
    }
    size_t at = table_bytes + run_off + (incl - mine);
#pragma unroll
    for (int j = 0; j < kPerLane; ++j) {
        if ((uint32_t)j < have) {
            uint32_t x = v[j];
            for (;;) {
                const uint32_t low = x & 0x7Fu;
                x >>= 7;
                put(at++, (uint8_t)(low | (x ? 0x80u : 0u)));
                if (!x) break;
            }
        }
    }
}

__global__ void __launch_bounds__(kPackThreads)
unpack_runs(const uint8_t *__restrict__ packed, const uint32_t *__restrict__ nnz, uint32_t max_words,
            uint32_t *__restrict__ words, uint32_t *dev_status)
{
    __shared__ __align__(4) uint8_t sm_bytes[kPackWarps][kRunBytesMax + 8];
    __shared__ uint32_t sm_vals[kPackWarps][kPackRun];
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t n = min(*nnz, max_words);
    const uint32_t runs = (n + kPackRun - 1) / kPackRun;
    const uint32_t run = blockIdx.x * kPackWarps + warp;
    if (run >= runs) return;
    const size_t table_bytes = 4 * ((size_t)runs + 1);
    uint32_t begin = 0, end = 0;
#pragma unroll
    for (int b = 0; b < 4; ++b) {
        begin |= (uint32_t)packed[4 * (size_t)run + b] << (8 * b);
        end |= (uint32_t)packed[4 * (size_t)run + 4 + b] << (8 * b);
    }
    const uint32_t in_run = min((uint32_t)kPackRun, n - run * kPackRun);   // words this run holds
    const uint32_t nb = end - begin;
    // a run of k words takes k .. 5 k bytes; anything else is not a stream this library wrote
    if (end < begin || nb < in_run || nb > 5 * in_run) {
        if (lane == 0) atomicOr(dev_status, VGC_DEV_RANGE);
        for (uint32_t i = lane; i < in_run; i += 32) words[run * kPackRun + i] = 0xFFFFFFFFu;   // an index no buffer has
        return;
    }
    const uint8_t *src = packed + table_bytes + begin;
    // the bytes keep their alignment in shared memory (byte i sits at off + i), so whole 4-byte words can be copied;
    // the word that holds the first byte starts up to 3 bytes earlier (inside the stream: the table is before it), the
    // bytes after the last whole word are copied one by one
    const uint32_t off = (uint32_t)(reinterpret_cast<uintptr_t>(src) & 3u);
    const uint32_t whole = (off + nb) / 4u;
    const uint32_t *src_w = reinterpret_cast<const uint32_t *>(src - off);
    uint32_t *dst_w = reinterpret_cast<uint32_t *>(&sm_bytes[warp][0]);
    for (uint32_t i = lane; i < whole; i += 32) dst_w[i] = src_w[i];
    for (uint32_t i = 4u * whole + lane; i < off + nb; i += 32) sm_bytes[warp][i] = src[i - off];
    __syncwarp();
    const uint8_t *bytes = &sm_bytes[warp][off];
    // numbers that end in this lane's part of the bytes
    const uint32_t span = (nb + 31u) / 32u;                               // at most kBytesPerLane: every lane has a part
    const uint32_t p0 = min(lane * span, nb), p1 = min(p0 + span, nb);
    uint32_t ends = 0;
    for (uint32_t p = p0; p < p1; ++p) ends += (bytes[p] & 0x80u) ? 0u : 1u;
    uint32_t incl = ends;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t up = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += up;
    }
    const uint32_t total = __shfl_sync(0xffffffffu, incl, 31);
    // as many numbers as the run has words, the last byte ending one
    bool bad = total != in_run || (bytes[nb - 1] & 0x80u);
    uint32_t k = incl - ends;                                             // place in the run of the first number ending here
    if (!bad) {
        for (uint32_t p = p0; p < p1; ++p) {
            if (bytes[p] & 0x80u) continue;
            // the number's bytes: this one and the bytes before it whose top bit is set (at most four)
            uint32_t first = p;
            while (first > 0 && p - first < 5 && (bytes[first - 1] & 0x80u)) --first;
            if (p - first > 4) { bad = true; break; }
            uint32_t v = 0;
            for (uint32_t q = first; q <= p; ++q) v |= (uint32_t)(bytes[q] & 0x7Fu) << (7 * (q - first));
            sm_vals[warp][k++] = v;
        }
    }
    bad = __any_sync(0xffffffffu, bad);
    __syncwarp();
    if (bad) {
        if (lane == 0) atomicOr(dev_status, VGC_DEV_RANGE);
        for (uint32_t i = lane; i < in_run; i += 32) words[run * kPackRun + i] = 0xFFFFFFFFu;
        return;
    }
    // indices: running sum of the differences, 8 consecutive words per lane
    uint32_t v[kPerLane], sum = 0;
#pragma unroll
    for (int j = 0; j < kPerLane; ++j) {
        const uint32_t i = lane * kPerLane + j;
        v[j] = i < in_run ? sm_vals[warp][i] : 0u;
        sum += v[j] >> 4;
    }
    uint32_t scan = sum;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t up = __shfl_up_sync(0xffffffffu, scan, d);
        if (lane >= d) scan += up;
    }
    uint32_t idx = scan - sum;
#pragma unroll
    for (int j = 0; j < kPerLane; ++j) {
        const uint32_t i = lane * kPerLane + j;
        idx += v[j] >> 4;
        if (i < in_run) words[run * kPackRun + i] = (idx << 4) | (v[j] & 15u);
    }
}

}  // namespace vgc

using namespace vgc;

namespace {
struct PackLayout { size_t run_bytes, block_bytes, total; uint32_t blocks; };
PackLayout pack_layout(uint32_t max_words)
{
    PackLayout L;
    const uint32_t runs = (max_words + kPackRun - 1) / kPackRun;
    L.blocks = runs / kPackWarps + 1;                      // one more than the runs need: the warp that writes table[runs]
    L.run_bytes = 0;
    L.block_bytes = round_up(sizeof(uint32_t) * (size_t)L.blocks * kPackWarps, 256);
    L.total = L.block_bytes + round_up(sizeof(uint32_t) * (size_t)L.blocks, 256);
    return L;
}
}  // namespace

extern "C" size_t vgc_pack_bound_bytes(uint32_t max_words)
{
    return 4 * ((size_t)(max_words + kPackRun - 1) / kPackRun + 1) + 5 * (size_t)max_words;
}

extern "C" size_t vgc_pack_workspace_bytes(uint32_t max_words) { return pack_layout(max_words).total; }

extern "C" vgc_status vgc_pack_indices(const uint32_t *words, const uint32_t *nnz, uint32_t max_words, uint8_t *packed,
                                       size_t packed_capacity, uint32_t *packed_bytes, uint32_t *dev_status, void *ws,
                                       size_t ws_bytes, vgc_stream_t stream)
{
    if (!nnz || !packed || !packed_bytes || !dev_status || (max_words && !words)) return VGC_ERR_INVALID_ARG;
    if (max_words > VGC_MAX_PARAMS || packed_capacity < 4) return VGC_ERR_INVALID_ARG;
    const PackLayout L = pack_layout(max_words);
    if (!ws || ws_bytes < L.total) return VGC_ERR_WORKSPACE;
    uint32_t *run_bytes = reinterpret_cast<uint32_t *>(static_cast<char *>(ws) + L.run_bytes);
    uint32_t *block_bytes = reinterpret_cast<uint32_t *>(static_cast<char *>(ws) + L.block_bytes);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    pack_count<<<L.blocks, kPackThreads, 0, st>>>(words, nnz, max_words, run_bytes, block_bytes);
    pack_emit<<<L.blocks, kPackThreads, 0, st>>>(words, nnz, max_words, run_bytes, block_bytes, packed, packed_capacity,
                                                 packed_bytes, dev_status);
    count_launch(2);
    VGC_CUDA_OK(cudaGetLastError());
    return VGC_OK;
}

extern "C" vgc_status vgc_unpack_indices(const uint8_t *packed, const uint32_t *nnz, uint32_t max_words, uint32_t *words,
                                         uint32_t *dev_status, vgc_stream_t stream)
{
    if (!packed || !nnz || !dev_status || (max_words && !words)) return VGC_ERR_INVALID_ARG;
    if (max_words > VGC_MAX_PARAMS) return VGC_ERR_INVALID_ARG;
    if (max_words == 0) return VGC_OK;
    const uint32_t runs = (max_words + kPackRun - 1) / kPackRun;
    unpack_runs<<<(runs + kPackWarps - 1) / kPackWarps, kPackThreads, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
        packed, nnz, max_words, words, dev_status);
    count_launch();
    VGC_CUDA_OK(cudaGetLastError());
    return VGC_OK;
}
