// vgc_step_host: one worker step driven from HOST buffers -- the end-to-end form of the path.
// Copies each layer's x and delta (and the step's mean gradient g) from host memory into caller-provided
// device buffers, runs the squared-gradient sums of every layer and one compressor step on the device,
// and copies the message back to host memory.  Copies are one cudaMemcpyAsync per tensor on the
// caller's stream; the call waits for the stream twice (the word count must be known on the host
// before the words can be copied).
#include "vgc_common.cuh"

extern "C" vgc_status vgc_step_host(const vgc_layer_host *layers, int n_layers, const float *g_host, float *g_dev,
                                    float *s_dev, float *r, float *v, size_t n, const uint32_t *group_offsets,
                                    int K, float alpha, float zeta, float scale, const vgc_message *out,
                                    uint32_t *words_host, uint32_t *counters_host, void *ws_sqgrad,
                                    size_t ws_sqgrad_bytes, void *ws_compress, size_t ws_compress_bytes,
                                    vgc_stream_t stream)
{
    if (n_layers < 0 || (n_layers && !layers) || !g_host || !g_dev || !s_dev || !out || !words_host || !counters_host)
        return VGC_ERR_INVALID_ARG;
    if (K != n_layers) return VGC_ERR_INVALID_ARG;        // one weight tensor (group) per layer, in order
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    size_t offset = 0;
    for (int l = 0; l < n_layers; ++l) {
        const vgc_layer_host &L = layers[l];
        if (!L.x_host || !L.delta_host || !L.x_dev || !L.delta_dev) return VGC_ERR_INVALID_ARG;
        size_t n_x, n_d, n_w;
        if (L.is_conv) {
            if (L.H + 2 * L.pad_h < L.Kh || L.W + 2 * L.pad_w < L.Kw || L.stride_h < 1 || L.stride_w < 1)
                return VGC_ERR_INVALID_ARG;
            const size_t Ho = (L.H + 2 * L.pad_h - L.Kh) / L.stride_h + 1, Wo = (L.W + 2 * L.pad_w - L.Kw) / L.stride_w + 1;
            n_x = (size_t)L.B * L.C * L.H * L.W;
            n_d = (size_t)L.B * L.Cout * Ho * Wo;
            n_w = (size_t)L.Cout * L.C * L.Kh * L.Kw;
        } else {
            n_x = (size_t)L.B * L.C;
            n_d = (size_t)L.B * L.Cout;
            n_w = (size_t)L.Cout * L.C;
        }
        if (offset + n_w > n) return VGC_ERR_INVALID_ARG;
        VGC_CUDA_OK(cudaMemcpyAsync(L.x_dev, L.x_host, n_x * sizeof(float), cudaMemcpyHostToDevice, st));
        VGC_CUDA_OK(cudaMemcpyAsync(L.delta_dev, L.delta_host, n_d * sizeof(float), cudaMemcpyHostToDevice, st));
        vgc_status rc = L.is_conv
                            ? vgc_sqgrad_conv(L.x_dev, L.delta_dev, L.B, L.C, L.H, L.W, L.Cout, L.Kh, L.Kw, L.stride_h,
                                              L.stride_w, L.pad_h, L.pad_w, scale, 0, s_dev + offset, ws_sqgrad,
                                              ws_sqgrad_bytes, stream)
                            : vgc_sqgrad_linear(L.x_dev, L.delta_dev, L.B, L.C, L.Cout, scale, 0, s_dev + offset,
                                                ws_sqgrad, ws_sqgrad_bytes, stream);
        if (rc != VGC_OK) return rc;
        offset += n_w;
    }
    if (offset != n) return VGC_ERR_INVALID_ARG;
    VGC_CUDA_OK(cudaMemcpyAsync(g_dev, g_host, n * sizeof(float), cudaMemcpyHostToDevice, st));
    vgc_status rc = vgc_compress(g_dev, s_dev, r, v, n, group_offsets, K, alpha, zeta, out, ws_compress, ws_compress_bytes,
                                 stream);
    if (rc != VGC_OK) return rc;
    // counters: nnz, n_criterion, n_dropped, dev_status
    VGC_CUDA_OK(cudaMemcpyAsync(counters_host + 0, out->nnz, 4, cudaMemcpyDeviceToHost, st));
    VGC_CUDA_OK(cudaMemcpyAsync(counters_host + 1, out->n_criterion, 4, cudaMemcpyDeviceToHost, st));
    VGC_CUDA_OK(cudaMemcpyAsync(counters_host + 2, out->n_dropped, 4, cudaMemcpyDeviceToHost, st));
    VGC_CUDA_OK(cudaMemcpyAsync(counters_host + 3, out->dev_status, 4, cudaMemcpyDeviceToHost, st));
    VGC_CUDA_OK(cudaStreamSynchronize(st));
    const uint32_t kept = counters_host[0] < out->capacity ? counters_host[0] : out->capacity;
    if (kept) {
        VGC_CUDA_OK(cudaMemcpyAsync(words_host, out->words, (size_t)kept * 4, cudaMemcpyDeviceToHost, st));
        VGC_CUDA_OK(cudaStreamSynchronize(st));
    }
    return VGC_OK;
}
