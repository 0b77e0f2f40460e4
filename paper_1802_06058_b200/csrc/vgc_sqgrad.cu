// C ABI of the squared per-example gradient sums (argument checks and kernel choice).
#include <cstdlib>

#include "vgc_common.cuh"

namespace vgc {
size_t simt_workspace_bytes(int M, int N, int K);
vgc_status simt_sqgrad_linear(const float *x, const float *delta, int B, int in, int out, float scale,
                              int accumulate, float *S, void *ws, size_t ws_bytes, cudaStream_t st);
vgc_status simt_sqgrad_conv(const float *x, const float *delta, int B, int C, int H, int W, int Cout,
                            int Kh, int Kw, int sh, int sw, int ph, int pw, int Ho, int Wo, float scale,
                            int accumulate, float *S, void *ws, size_t ws_bytes, cudaStream_t st);
void tc_plan_hint(int concurrent_launches);
bool tc_linear_supported(int B, int in, int out);
bool tc_conv_supported(int B, int C, int H, int W, int Cout, int Kh, int Kw, int sh, int sw, int ph, int pw);
size_t tc_linear_workspace_bytes(int B, int in, int out);
size_t tc_conv_workspace_bytes(int n_layers, int B, int C, int H, int W, int Kh, int Kw, int sh, int sw, int ph, int pw,
                               int Ho, int Wo, int Cout, bool exact = false);
vgc_status tc_sqgrad_linear(const float *x, const float *delta, int B, int in, int out, float scale, int accumulate,
                            float *S, void *ws, size_t ws_bytes, cudaStream_t st);
vgc_status tc_sqgrad_conv(int n_layers, const float *const *x, const float *const *delta, float *const *S, int B, int C,
                          int H, int W, int Cout, int Kh, int Kw, int sh, int sw, int ph, int pw, int Ho, int Wo,
                          float scale, int accumulate, void *ws, size_t ws_bytes, cudaStream_t st, bool exact = false);
}  // namespace vgc

using namespace vgc;

namespace {
// B == 0: the sum over the mini-batch is empty -- S is cleared (accumulate == 0) or left alone
vgc_status empty_batch(float *const *S, int n_layers, size_t n_weights, int accumulate, cudaStream_t st)
{
    if (!accumulate)
        for (int l = 0; l < n_layers; ++l) VGC_CUDA_OK(cudaMemsetAsync(S[l], 0, n_weights * sizeof(float), st));
    return VGC_OK;
}

bool conv_shape_ok(int B, int C, int H, int W, int Cout, int Kh, int Kw, int sh, int sw, int ph, int pw,
                   int *Ho, int *Wo)
{
    if (B < 0 || C < 0 || H < 1 || W < 1 || Cout < 0 || Kh < 1 || Kw < 1 || sh < 1 || sw < 1 || ph < 0 || pw < 0)
        return false;
    if (H + 2 * ph < Kh || W + 2 * pw < Kw) return false;
    *Ho = (H + 2 * ph - Kh) / sh + 1;
    *Wo = (W + 2 * pw - Kw) / sw + 1;
    const long long k = (long long)B * *Ho * *Wo, n = (long long)C * Kh * Kw;
    return k < (1LL << 31) && n < (1LL << 31) && (long long)Cout * n < (1LL << 40);
}
}  // namespace

extern "C" size_t vgc_sqgrad_linear_workspace_bytes(int B, int in, int out)
{
    if (B <= 0 || in <= 0 || out <= 0) return 0;
    size_t need = simt_workspace_bytes(out, in, B) + 256;
    if (tc_linear_supported(B, in, out)) need = need > tc_linear_workspace_bytes(B, in, out) ? need : tc_linear_workspace_bytes(B, in, out);
    return round_up(need > 256 ? need : 256, 256);
}

extern "C" vgc_status vgc_sqgrad_linear(const float *x, const float *delta, int B, int in, int out,
                                        float scale, int accumulate, float *S,
                                        void *ws, size_t ws_bytes, vgc_stream_t stream)
{
    if (B < 0 || in < 0 || out < 0) return VGC_ERR_INVALID_ARG;
    if (in == 0 || out == 0) return VGC_OK;
    if (!S || !aligned16(S)) return VGC_ERR_INVALID_ARG;
    if (B > 0 && (!x || !delta || !aligned16(x) || !aligned16(delta))) return VGC_ERR_INVALID_ARG;
    if (!(scale == scale)) return VGC_ERR_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (B == 0) return empty_batch(&S, 1, (size_t)in * out, accumulate, st);
    if (ws_bytes < vgc_sqgrad_linear_workspace_bytes(B, in, out) || !ws) return VGC_ERR_WORKSPACE;
    if (tc_linear_supported(B, in, out))
        return tc_sqgrad_linear(x, delta, B, in, out, scale, accumulate, S, ws, ws_bytes, st);
    return simt_sqgrad_linear(x, delta, B, in, out, scale, accumulate, S, static_cast<char *>(ws) + 256,
                              ws_bytes - 256, st);
}

extern "C" size_t vgc_sqgrad_conv_batch_workspace_bytes(int n_layers, int B, int C, int H, int W, int Cout, int Kh,
                                                        int Kw, int stride_h, int stride_w, int pad_h, int pad_w)
{
    int Ho, Wo;
    if (n_layers < 1 || !conv_shape_ok(B, C, H, W, Cout, Kh, Kw, stride_h, stride_w, pad_h, pad_w, &Ho, &Wo)) return 0;
    if (B == 0 || C == 0 || Cout == 0) return 0;
    size_t need = simt_workspace_bytes(Cout, C * Kh * Kw, B * Ho * Wo);
    if (tc_conv_supported(B, C, H, W, Cout, Kh, Kw, stride_h, stride_w, pad_h, pad_w)) {
        const size_t t = tc_conv_workspace_bytes(n_layers, B, C, H, W, Kh, Kw, stride_h, stride_w, pad_h, pad_w, Ho, Wo, Cout);
        need = need > t ? need : t;
    }
    return round_up(need + 256, 256);
}

extern "C" size_t vgc_sqgrad_conv_workspace_bytes(int B, int C, int H, int W, int Cout, int Kh, int Kw,
                                                  int stride_h, int stride_w, int pad_h, int pad_w)
{
    return vgc_sqgrad_conv_batch_workspace_bytes(1, B, C, H, W, Cout, Kh, Kw, stride_h, stride_w, pad_h, pad_w);
}

extern "C" vgc_status vgc_sqgrad_conv_batch(int n_layers, const float *const *x, const float *const *delta,
                                            float *const *S, int B, int C, int H, int W, int Cout, int Kh, int Kw,
                                            int stride_h, int stride_w, int pad_h, int pad_w, float scale,
                                            int accumulate, void *ws, size_t ws_bytes, vgc_stream_t stream)
{
    int Ho, Wo;
    if (n_layers < 0 || !conv_shape_ok(B, C, H, W, Cout, Kh, Kw, stride_h, stride_w, pad_h, pad_w, &Ho, &Wo))
        return VGC_ERR_INVALID_ARG;
    if (n_layers == 0 || C == 0 || Cout == 0) return VGC_OK;
    if (!x || !delta || !S || !(scale == scale)) return VGC_ERR_INVALID_ARG;
    for (int l = 0; l < n_layers; ++l) {
        if (!S[l] || !aligned16(S[l])) return VGC_ERR_INVALID_ARG;
        if (B > 0 && (!x[l] || !delta[l] || !aligned16(x[l]) || !aligned16(delta[l]))) return VGC_ERR_INVALID_ARG;
    }
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (B == 0) return empty_batch(S, n_layers, (size_t)Cout * C * Kh * Kw, accumulate, st);
    if (ws_bytes < vgc_sqgrad_conv_batch_workspace_bytes(n_layers, B, C, H, W, Cout, Kh, Kw, stride_h, stride_w, pad_h,
                                                         pad_w) ||
        !ws)
        return VGC_ERR_WORKSPACE;
    if (tc_conv_supported(B, C, H, W, Cout, Kh, Kw, stride_h, stride_w, pad_h, pad_w))
        return tc_sqgrad_conv(n_layers, x, delta, S, B, C, H, W, Cout, Kh, Kw, stride_h, stride_w, pad_h, pad_w, Ho, Wo,
                              scale, accumulate, ws, ws_bytes, st);
    for (int l = 0; l < n_layers; ++l) {        // CUDA-core kernel: layer after layer
        const vgc_status rc = simt_sqgrad_conv(x[l], delta[l], B, C, H, W, Cout, Kh, Kw, stride_h, stride_w, pad_h, pad_w,
                                               Ho, Wo, scale, accumulate, S[l], static_cast<char *>(ws) + 256,
                                               ws_bytes - 256, st);
        if (rc != VGC_OK) return rc;
    }
    return VGC_OK;
}

extern "C" vgc_status vgc_sqgrad_conv(const float *x, const float *delta, int B, int C, int H, int W, int Cout,
                                      int Kh, int Kw, int stride_h, int stride_w, int pad_h, int pad_w,
                                      float scale, int accumulate, float *S,
                                      void *ws, size_t ws_bytes, vgc_stream_t stream)
{
    return vgc_sqgrad_conv_batch(1, &x, &delta, &S, B, C, H, W, Cout, Kh, Kw, stride_h, stride_w, pad_h, pad_w, scale,
                                 accumulate, ws, ws_bytes, stream);
}

extern "C" size_t vgc_sqgrad_conv_exact_batch_workspace_bytes(int n_layers, int B, int C, int H, int W, int Cout, int Kh,
                                                              int Kw, int stride_h, int stride_w, int pad_h, int pad_w)
{
    int Ho, Wo;
    if (n_layers < 1 || !conv_shape_ok(B, C, H, W, Cout, Kh, Kw, stride_h, stride_w, pad_h, pad_w, &Ho, &Wo)) return 0;
    if (B == 0 || C == 0 || Cout == 0) return 0;
    if (!tc_conv_supported(B, C, H, W, Cout, Kh, Kw, stride_h, stride_w, pad_h, pad_w)) return 0;
    return round_up(tc_conv_workspace_bytes(n_layers, B, C, H, W, Kh, Kw, stride_h, stride_w, pad_h, pad_w, Ho, Wo, Cout, true) +
                        256,
                    256);
}

extern "C" size_t vgc_sqgrad_conv_exact_workspace_bytes(int B, int C, int H, int W, int Cout, int Kh, int Kw,
                                                        int stride_h, int stride_w, int pad_h, int pad_w)
{
    return vgc_sqgrad_conv_exact_batch_workspace_bytes(1, B, C, H, W, Cout, Kh, Kw, stride_h, stride_w, pad_h, pad_w);
}

extern "C" vgc_status vgc_sqgrad_conv_exact_batch(int n_layers, const float *const *x, const float *const *delta,
                                                  float *const *S, int B, int C, int H, int W, int Cout, int Kh, int Kw,
                                                  int stride_h, int stride_w, int pad_h, int pad_w, float scale,
                                                  int accumulate, void *ws, size_t ws_bytes, vgc_stream_t stream)
{
    int Ho, Wo;
    if (n_layers < 0 || !conv_shape_ok(B, C, H, W, Cout, Kh, Kw, stride_h, stride_w, pad_h, pad_w, &Ho, &Wo))
        return VGC_ERR_INVALID_ARG;
    if (n_layers == 0 || C == 0 || Cout == 0) return VGC_OK;
    if (B < 1 || !x || !delta || !S || !(scale == scale)) return VGC_ERR_INVALID_ARG;
    for (int l = 0; l < n_layers; ++l)
        if (!S[l] || !aligned16(S[l]) || !x[l] || !delta[l] || !aligned16(x[l]) || !aligned16(delta[l]))
            return VGC_ERR_INVALID_ARG;
    if (!tc_conv_supported(B, C, H, W, Cout, Kh, Kw, stride_h, stride_w, pad_h, pad_w)) return VGC_ERR_UNSUPPORTED;
    if (ws_bytes < vgc_sqgrad_conv_exact_batch_workspace_bytes(n_layers, B, C, H, W, Cout, Kh, Kw, stride_h, stride_w, pad_h,
                                                               pad_w) ||
        !ws)
        return VGC_ERR_WORKSPACE;
    return tc_sqgrad_conv(n_layers, x, delta, S, B, C, H, W, Cout, Kh, Kw, stride_h, stride_w, pad_h, pad_w, Ho, Wo, scale,
                          accumulate, ws, ws_bytes, reinterpret_cast<cudaStream_t>(stream), true);
}

extern "C" vgc_status vgc_sqgrad_conv_exact(const float *x, const float *delta, int B, int C, int H, int W, int Cout,
                                            int Kh, int Kw, int stride_h, int stride_w, int pad_h, int pad_w,
                                            float scale, int accumulate, float *S, void *ws, size_t ws_bytes,
                                            vgc_stream_t stream)
{
    return vgc_sqgrad_conv_exact_batch(1, &x, &delta, &S, B, C, H, W, Cout, Kh, Kw, stride_h, stride_w, pad_h, pad_w, scale,
                                       accumulate, ws, ws_bytes, stream);
}

extern "C" void vgc_sqgrad_plan_hint(int concurrent_launches) { tc_plan_hint(concurrent_launches); }

extern "C" const char *vgc_status_string(int status)
{
    switch (status) {
        case VGC_OK: return "ok";
        case VGC_ERR_INVALID_ARG: return "invalid argument";
        case VGC_ERR_UNSUPPORTED: return "unsupported shape";
        case VGC_ERR_WORKSPACE: return "workspace too small";
        case VGC_ERR_CUDA: return "CUDA error";
        default: return "unknown status";
    }
}

extern "C" int vgc_version(void) { return 2000; }

namespace vgc { unsigned long long g_launches = 0; }
extern "C" uint64_t vgc_kernel_launch_count(void) { return vgc::g_launches; }
