// Squared per-example gradient sums on the CUDA cores (fp32 FMA), used for shapes the
// tensor-core kernel does not take and as its cross-check.
//
//   S[m][n] = scale * sum_k A(k,m)^2 * B(k,n)^2
// dense layer:  A = delta [K=B][M=out],  B = x [K=B][N=in]
// conv layer:   k = (example z, output position ho, wo), m = output channel,
//               n = (input channel c, kh, kw);  B(k,n) is the im2col view of x, zero outside.
// This is the right-hand side of Eq. 2 / the "v_i +=" line of Algorithm 1 obtained as one
// contraction of squared operands (N_params * |B| multiply-adds, Sec. 5).
//
// 64x64 output tile per block, 4x4 outputs per thread, 16-deep k slices through shared
// memory.  Partial sums run 256 terms in fp32 and are then promoted to fp64, so the
// accumulated rounding error stays near 1e-6 relative for any K.  Long reductions are split
// across blockIdx.z; the slices are combined in a fixed order by a second kernel.
#include "vgc_common.cuh"

namespace vgc {

constexpr int kBM = 64, kBN = 64, kBK = 16, kSimtThreads = 256;
constexpr int kPromote = 16;        // k slices (of 16) between promotions to fp64

struct LinearOperands {
    const float *x, *delta;
    int in, out;
    static constexpr bool kInnerIsK = false;
    __device__ __forceinline__ float a(int k, int m) const { return delta[(size_t)k * out + m]; }
    __device__ __forceinline__ float b(int k, int n) const { return x[(size_t)k * in + n]; }
    struct NCoord { int n; };
    __device__ __forceinline__ NCoord ncoord(int n) const { return {n}; }
    __device__ __forceinline__ float b(int k, const NCoord &c) const { return x[(size_t)k * in + c.n]; }
};

struct ConvOperands {
    const float *x, *delta;
    int C, H, W, Cout, Kh, Kw, sh, sw, ph, pw, Ho, Wo;
    static constexpr bool kInnerIsK = true;
    __device__ __forceinline__ float a(int k, int m) const
    {
        const int P = Ho * Wo;
        const int z = k / P, p = k - z * P;
        return delta[((size_t)z * Cout + m) * P + p];
    }
    struct NCoord { int c, kh, kw; };
    __device__ __forceinline__ NCoord ncoord(int n) const
    {
        const int kw = n % Kw, t = n / Kw;
        return {t / Kh, t % Kh, kw};
    }
    __device__ __forceinline__ float b(int k, const NCoord &nc) const
    {
        const int P = Ho * Wo;
        const int z = k / P, p = k - z * P;
        const int ho = p / Wo, wo = p - ho * Wo;
        const int hi = ho * sh + nc.kh - ph, wi = wo * sw + nc.kw - pw;
        if (hi < 0 || hi >= H || wi < 0 || wi >= W) return 0.f;
        return x[(((size_t)z * C + nc.c) * H + hi) * W + wi];
    }
};

// out_partial: [gridDim.z][M][N] fp32 when gridDim.z > 1, else the final S.
template <class Ops>
__global__ void __launch_bounds__(kSimtThreads)
sqgrad_simt(const Ops ops, int M, int N, int K, int k_per_split, float scale, int accumulate,
            float *__restrict__ S, float *__restrict__ partial)
{
    __shared__ float As[kBK][kBM + 4];
    __shared__ float Bs[kBK][kBN + 4];
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const int m0 = blockIdx.y * kBM, n0 = blockIdx.x * kBN;
    const int k_begin = blockIdx.z * k_per_split;
    const int k_end = min(K, k_begin + k_per_split);

    // which 4 elements of each operand tile this thread fetches
    int lk[4], lmn[4];
    typename Ops::NCoord nco[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int e = tid + kSimtThreads * i;
        if (Ops::kInnerIsK) { lk[i] = e % kBK; lmn[i] = e / kBK; }
        else                { lk[i] = e / kBM; lmn[i] = e % kBM; }
        nco[i] = ops.ncoord(min(n0 + lmn[i], N - 1));
    }

    float acc[4][4];
    double acc2[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) { acc[i][j] = 0.f; acc2[i][j] = 0.0; }

    int slice = 0;
    for (int k0 = k_begin; k0 < k_end; k0 += kBK) {
        float av[4], bv[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int k = k0 + lk[i];
            const bool kin = k < k_end;
            av[i] = (kin && m0 + lmn[i] < M) ? ops.a(k, m0 + lmn[i]) : 0.f;
            bv[i] = (kin && n0 + lmn[i] < N) ? ops.b(k, nco[i]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            As[lk[i]][lmn[i]] = __fmul_rn(av[i], av[i]);
            Bs[lk[i]][lmn[i]] = __fmul_rn(bv[i], bv[i]);
        }
        __syncthreads();
#pragma unroll
        for (int kk = 0; kk < kBK; ++kk) {
            const float4 a4 = *reinterpret_cast<const float4 *>(&As[kk][ty * 4]);
            const float4 b4 = *reinterpret_cast<const float4 *>(&Bs[kk][tx * 4]);
            const float a[4] = {a4.x, a4.y, a4.z, a4.w}, b[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], b[j], acc[i][j]);
        }
        if (++slice == kPromote) {
            slice = 0;
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) { acc2[i][j] += (double)acc[i][j]; acc[i][j] = 0.f; }
        }
    }
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int m = m0 + ty * 4 + i, n = n0 + tx * 4 + j;
            if (m >= M || n >= N) continue;
            const double sum = acc2[i][j] + (double)acc[i][j];
            if (gridDim.z > 1) {
                partial[((size_t)blockIdx.z * M + m) * N + n] = (float)sum;
            } else {
                const size_t at = (size_t)m * N + n;
                const double res = (double)scale * sum;
                S[at] = accumulate ? (float)((double)S[at] + res) : (float)res;
            }
        }
}

__global__ void __launch_bounds__(256)
sqgrad_combine_splits(const float *__restrict__ partial, int splits, size_t mn, float scale, int accumulate,
                      float *__restrict__ S)
{
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= mn) return;
    double sum = 0.0;
    for (int z = 0; z < splits; ++z) sum += (double)partial[(size_t)z * mn + i];
    const double res = (double)scale * sum;
    S[i] = accumulate ? (float)((double)S[i] + res) : (float)res;
}

int simt_splits(int M, int N, int K)
{
    const long tiles = (long)((M + kBM - 1) / kBM) * ((N + kBN - 1) / kBN);
    long want = (4L * 148 + tiles - 1) / tiles;
    const long max_by_k = (K + kBK * kPromote - 1) / (kBK * kPromote);
    if (want > max_by_k) want = max_by_k;
    if (want > 1024) want = 1024;
    if (want < 1) want = 1;
    return (int)want;
}

size_t simt_workspace_bytes(int M, int N, int K)
{
    const int splits = simt_splits(M, N, K);
    return splits > 1 ? (size_t)splits * M * N * sizeof(float) : 0;
}

template <class Ops>
vgc_status simt_launch(const Ops &ops, int M, int N, int K, float scale, int accumulate, float *S,
                       void *ws, size_t ws_bytes, cudaStream_t st)
{
    if (M <= 0 || N <= 0 || K <= 0) return VGC_ERR_INVALID_ARG;     // empty sums are the caller's business
    int splits = simt_splits(M, N, K);
    if (splits > 1 && ws_bytes < (size_t)splits * M * N * sizeof(float)) return VGC_ERR_WORKSPACE;
    int k_per_split = (K + splits - 1) / splits;
    k_per_split = (k_per_split + kBK - 1) / kBK * kBK;
    splits = (K + k_per_split - 1) / k_per_split;
    dim3 grid((N + kBN - 1) / kBN, (M + kBM - 1) / kBM, splits);
    if (grid.y > 65535u) return VGC_ERR_UNSUPPORTED;
    sqgrad_simt<Ops><<<grid, kSimtThreads, 0, st>>>(ops, M, N, K, k_per_split, scale, accumulate, S,
                                                    static_cast<float *>(ws));
    count_launch();
    if (splits > 1) {
        count_launch();
        const size_t mn = (size_t)M * N;
        sqgrad_combine_splits<<<(unsigned)((mn + 255) / 256), 256, 0, st>>>(static_cast<const float *>(ws), splits,
                                                                            mn, scale, accumulate, S);
    }
    return cudaGetLastError() == cudaSuccess ? VGC_OK : VGC_ERR_CUDA;
}

vgc_status simt_sqgrad_linear(const float *x, const float *delta, int B, int in, int out, float scale,
                              int accumulate, float *S, void *ws, size_t ws_bytes, cudaStream_t st)
{
    LinearOperands ops{x, delta, in, out};
    return simt_launch(ops, out, in, B, scale, accumulate, S, ws, ws_bytes, st);
}

vgc_status simt_sqgrad_conv(const float *x, const float *delta, int B, int C, int H, int W, int Cout,
                            int Kh, int Kw, int sh, int sw, int ph, int pw, int Ho, int Wo, float scale,
                            int accumulate, float *S, void *ws, size_t ws_bytes, cudaStream_t st)
{
    ConvOperands ops{x, delta, C, H, W, Cout, Kh, Kw, sh, sw, ph, pw, Ho, Wo};
    return simt_launch(ops, Cout, C * Kh * Kw, B * Ho * Wo, scale, accumulate, S, ws, ws_bytes, st);
}

}  // namespace vgc
