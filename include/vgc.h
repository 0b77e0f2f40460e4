/*
 * vgc.h -- C ABI of the variance-based gradient compression hot path for NVIDIA B200 (sm_100a).
 *
 * Method: Tsuzuku, Imachi, Akiba, "Variance-based Gradient Compression for Efficient Distributed
 * Deep Learning".  Per training step and per worker the library computes
 *   (1) the mini-batch sum of squared per-example gradients of a dense or conv layer
 *       (the right-hand side of Eq. 2 / the "v_i +=" line of Algorithm 1),
 *   (2) one pass of Algorithm 1 over the flat parameter buffer: accumulate the residual r and
 *       the variance estimate v, apply the send test r^2 > alpha*v, reset or decay, compact the
 *       selected elements and encode them with the 4-bit quantiser of Sec. 4.2 / 4.4 into
 *       32-bit (value, index) words,
 *   (3) the decode-and-sum half of CommunicateAndUpdate (Sec. 4.3) over W such messages.
 *
 * General rules
 *   - Every pointer is a DEVICE pointer owned by the caller unless a parameter says "host".
 *     The library allocates nothing, keeps no state between calls and never synchronises:
 *     each call only enqueues work on `stream` and returns.
 *   - Pointers to fp32 / u32 arrays must be 16-byte aligned (whole allocations are).
 *   - Return value: a vgc_status detected on the host before anything is enqueued, or
 *     VGC_ERR_CUDA when a launch failed.  Conditions found on the device are OR-ed into the
 *     caller's *dev_status word (VGC_DEV_*), which the caller zeroes and reads.
 *   - Workspaces hold no information between calls; the same workspace may serve successive
 *     calls on one stream.  Calls that overlap on the GPU need separate workspaces.
 */
#ifndef VGC_H_
#define VGC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* cudaStream_t without pulling in the CUDA headers */
typedef struct CUstream_st *vgc_stream_t;

typedef enum {
    VGC_OK = 0,
    VGC_ERR_INVALID_ARG = 1, /* null / misaligned pointer, negative size, n > 2^28, bad alpha or zeta */
    VGC_ERR_UNSUPPORTED = 2, /* shape outside what the kernels cover                               */
    VGC_ERR_WORKSPACE = 3,   /* workspace smaller than the matching *_workspace_bytes()             */
    VGC_ERR_CUDA = 4         /* a CUDA call failed; cudaGetLastError() has the detail               */
} vgc_status;

/* bits OR-ed into *dev_status by kernels */
#define VGC_DEV_CAPACITY 1u /* word buffer too small: message truncated, state still correct             */
#define VGC_DEV_TIMEOUT 2u  /* a bounded wait inside a kernel gave up: outputs of this call are invalid    */
#define VGC_DEV_RANGE 4u    /* decode met an index >= n: that word was skipped                           */

/* group_exp value of a weight tensor from which nothing was sent */
#define VGC_EXP_NONE INT32_MIN

/* largest flat buffer: the word keeps 28 bits for the index (Sec. 4.2, "the rest 28-bits") */
#define VGC_MAX_PARAMS (1u << 28)

const char *vgc_status_string(int status);
/* 1000*major + minor of this library */
int vgc_version(void);
/* Kernels enqueued by this library since it was loaded (host-side bookkeeping for benchmarks;
 * not thread-safe, no paper counterpart). */
uint64_t vgc_kernel_launch_count(void);

/* ---------------------------------------------------------------------------------------------
 * (1) Squared per-example gradient sums.
 *
 * Dense layer y_z = W x_z, delta_z = df_z/dy_z: the gradient of example z for W[j][i] is
 * delta[z][j]*x[z][i], so  S[j][i] = scale * sum_z delta[z][j]^2 * x[z][i]^2  -- the sum of squared
 * per-example gradients that Eq. 2 and Algorithm 1 ("v_i += sum (grad_i f_z / B)^2") need, obtained
 * as one contraction of squared operands without forming any per-example gradient.  Cost
 * N_params*|B| multiply-adds, the leading term of Sec. 5.  Algorithm 1 divides each example's
 * gradient by B: pass scale = 1/B^2 when delta carries no 1/B.
 *
 *   x      [B][in]   fp32 row-major        delta  [B][out]  fp32 row-major
 *   S      [out][in] fp32 row-major (the layer's slice of the flat buffer)
 *   accumulate  0: S = result   1: S += result
 *   ws / ws_bytes  scratch of at least vgc_sqgrad_linear_workspace_bytes(B, in, out) (never less than
 *                  256 bytes).  The first 32-bit word of ws is a status word the caller zeroes once
 *                  (e.g. when allocating ws): kernels only ever OR bits into it -- VGC_DEV_TIMEOUT
 *                  if a bounded wait inside a kernel gave up, in which case S is invalid.
 *
 * Result within 1e-5 relative of the exact sum.  in == 0 or out == 0: no-op, OK.  B == 0: the sum is empty --
 * S is cleared when accumulate == 0 and left alone otherwise; the workspace is not used.
 * ------------------------------------------------------------------------------------------- */
size_t vgc_sqgrad_linear_workspace_bytes(int B, int in, int out);
vgc_status vgc_sqgrad_linear(const float *x, const float *delta, int B, int in, int out,
                             float scale, int accumulate, float *S,
                             void *ws, size_t ws_bytes, vgc_stream_t stream);

/* Conv layer (cross-correlation, zero padding, dilation 1, groups 1).  The paper does not treat
 * conv layers; this entry point takes every (example, output position) pair as one sample:
 *   S[o][c][kh][kw] = scale * sum_z sum_{ho,wo} delta[z][o][ho][wo]^2 * x[z][c][ho*sh+kh-ph][wo*sw+kw-pw]^2
 * which is the contraction of squared im2col inputs with squared errors, and equals the
 * per-example sum of squares whenever there is a single output position.
 *
 *   x      [B][C][H][W]        fp32 NCHW        delta  [B][Cout][Ho][Wo]  fp32
 *   S      [Cout][C][Kh][Kw]   fp32 (OIHW, the layer's slice of the flat buffer)
 *   Ho = (H + 2*pad_h - Kh)/stride_h + 1, Wo likewise; both must be >= 1.  B == 0 as for the dense layer.
 * ------------------------------------------------------------------------------------------- */
size_t vgc_sqgrad_conv_workspace_bytes(int B, int C, int H, int W, int Cout, int Kh, int Kw,
                                       int stride_h, int stride_w, int pad_h, int pad_w);
vgc_status vgc_sqgrad_conv(const float *x, const float *delta, int B, int C, int H, int W, int Cout,
                           int Kh, int Kw, int stride_h, int stride_w, int pad_h, int pad_w,
                           float scale, int accumulate, float *S,
                           void *ws, size_t ws_bytes, vgc_stream_t stream);

/* The per-example statistic of a conv layer, exactly as Eq. 2 / Algorithm 1 define it for any layer:
 *   S[o][c][kh][kw] = scale * sum_z ( sum_{ho,wo} delta[z][o][ho][wo] * x[z][c][ho*sh+kh-ph][wo*sw+kw-pw] )^2
 * i.e. the square of each example's whole weight gradient, cross terms between output positions included
 * (vgc_sqgrad_conv drops them by treating every position as a sample; the two agree when Ho*Wo == 1).  Same
 * tensor-core kernels and the same number of products: the operands are split into TF32 parts without being
 * squared, an example's positions are reduced first, and the epilogue squares that sum and adds it to a running
 * sum kept in tensor memory.  Arguments and layouts as for vgc_sqgrad_conv; workspace from
 * vgc_sqgrad_conv_exact_workspace_bytes.  Accuracy: each example's gradient carries the 3xTF32 product error
 * (about 2^-22 of the sum of |products|), so the result is within 1e-5 of the same statistic of |x| and |delta|
 * (relative to the result itself only where an example's positions do not cancel).  Shapes the tensor-core
 * path cannot take return VGC_ERR_UNSUPPORTED (there is no CUDA-core form of this entry point). */
size_t vgc_sqgrad_conv_exact_workspace_bytes(int B, int C, int H, int W, int Cout, int Kh, int Kw,
                                             int stride_h, int stride_w, int pad_h, int pad_w);
vgc_status vgc_sqgrad_conv_exact(const float *x, const float *delta, int B, int C, int H, int W, int Cout,
                                 int Kh, int Kw, int stride_h, int stride_w, int pad_h, int pad_w,
                                 float scale, int accumulate, float *S,
                                 void *ws, size_t ws_bytes, vgc_stream_t stream);
/* ... for several layers of one geometry in one call, as vgc_sqgrad_conv_batch. */
size_t vgc_sqgrad_conv_exact_batch_workspace_bytes(int n_layers, int B, int C, int H, int W, int Cout, int Kh, int Kw,
                                                   int stride_h, int stride_w, int pad_h, int pad_w);
vgc_status vgc_sqgrad_conv_exact_batch(int n_layers, const float *const *x, const float *const *delta, float *const *S,
                                       int B, int C, int H, int W, int Cout, int Kh, int Kw, int stride_h, int stride_w,
                                       int pad_h, int pad_w, float scale, int accumulate, void *ws, size_t ws_bytes,
                                       vgc_stream_t stream);

/* Planning hint (no counterpart in the paper): how many sqgrad calls the caller keeps in flight side by side on
 * different streams, each with its own workspace (default 1).  A call's kernel runs one thread block per SM at a
 * time.  Alone (1), a call's work is cut evenly over all SMs, one long block each.  With several calls in flight
 * (> 1), each call is cut into about half a wave of shorter blocks, and the hardware's block scheduler balances the
 * SMs across the calls.  Process-wide; set it BEFORE asking for workspace sizes, which depend on it. */
void vgc_sqgrad_plan_hint(int concurrent_launches);

/* Several conv layers of ONE geometry in one call (the residual stages of a deep network repeat the same
 * layer shapes): layer l computes what vgc_sqgrad_conv computes from x[l], delta[l] into S[l].  The tensor-
 * core path runs up to 8 layers per kernel launch and cuts their combined work evenly over the SMs, which a
 * single small layer cannot fill; results are identical to n_layers single calls only up to the order of the
 * fp32 partial sums (same 1e-5 bound).
 *   x, delta, S   HOST arrays of n_layers DEVICE pointers (read during the call only)
 *   ws            at least vgc_sqgrad_conv_batch_workspace_bytes(n_layers, ...) bytes; status word as above
 * The layers' S ranges must not overlap.  n_layers == 0: no-op, OK. */
size_t vgc_sqgrad_conv_batch_workspace_bytes(int n_layers, int B, int C, int H, int W, int Cout, int Kh, int Kw,
                                             int stride_h, int stride_w, int pad_h, int pad_w);
vgc_status vgc_sqgrad_conv_batch(int n_layers, const float *const *x, const float *const *delta, float *const *S,
                                 int B, int C, int H, int W, int Cout, int Kh, int Kw, int stride_h, int stride_w,
                                 int pad_h, int pad_w, float scale, int accumulate, void *ws, size_t ws_bytes,
                                 vgc_stream_t stream);

/* ---------------------------------------------------------------------------------------------
 * (2) Compressor: one step of Algorithm 1 ("Basic") over the flat buffer, then Encode().
 *
 * For every parameter i, in IEEE binary32, round-to-nearest-even, one operation at a time, no FMA:
 *     r1 = r[i] + g[i];  v1 = v[i] + s[i];
 *     send = (r1*r1 > alpha*v1)                       -- strict, Eq. 2
 *     send:  value_i = r1; r[i] = 0; v[i] = 0        else:  r[i] = r1; v[i] = v1*zeta
 * Encode (Sec. 4.2, bit-level recipe of Sec. 4.4), per weight tensor k = [offsets[k], offsets[k+1]):
 *     M_k = max |value_i| over the elements of k being sent;  E_k = floor(log2 M_k) (exponent field)
 *     e   = min(E_k, exponent of |value_i| after adding 1 at the top mantissa bit)   -- nearer power
 *           of two, midpoint up, cut at 2^E_k;   d = E_k - e;   d > 7: nothing is emitted for i
 *     word = i << 4 | sign << 3 | d               -- 28-bit index, 1 sign bit, 3 exponent bits
 * Words come out in ascending index order; the output is a deterministic function of the inputs.
 *
 *   g, s          [n] fp32: this step's sum of per-example gradients / B and sum of their squares
 *                 s may be NULL: then v must already hold v + s (the sqgrad calls with accumulate = 1
 *                 and S pointing into v do exactly that one fp32 addition), and the pass reads 4 bytes
 *                 per parameter less; results are identical bit for bit
 *   r, v          [n] fp32 state, updated in place (all zeros before the first step)
 *   group_offsets [K+1] u32 on the device, offsets[0] = 0, offsets[K] = n, non-decreasing
 *   out           HOST struct of device pointers, see below
 *   ws            at least vgc_compress_workspace_bytes(n, K) (about 8 bytes per parameter: every
 *                 tile of the buffer owns a staging segment that could hold all of its elements)
 *
 * n == 0: no-op, OK (counters are not written).  n > VGC_MAX_PARAMS, alpha < 0, non-finite alpha or
 * zeta, K < 1, null or misaligned pointers: VGC_ERR_INVALID_ARG.  When the word buffer is too small
 * the message is truncated, VGC_DEV_CAPACITY is set, *nnz still holds the count that was needed, and
 * r, v are updated exactly as if it had fit.
 * Inputs containing NaN or Inf are outside the contract; s >= 0 and v >= 0 are assumed.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    uint32_t *words;       /* out [capacity]: packed words, ascending index                          */
    uint32_t capacity;     /*                 how many words fit                                     */
    int32_t *group_exp;    /* out [K]: floor(log2 M_k), or VGC_EXP_NONE                              */
    uint32_t *nnz;         /* out [1]: words emitted                                                 */
    uint32_t *n_criterion; /* out [1]: elements that passed the send test                            */
    uint32_t *n_dropped;   /* out [1]: of those, how many the quantiser rounded to zero (d > 7)      */
    uint8_t *mask;         /* optional out [n] (may be NULL): 1 where the send test passed           */
    uint32_t *dev_status;  /* in/out [1]: VGC_DEV_* bits are OR-ed in                                */
} vgc_message;

size_t vgc_compress_workspace_bytes(size_t n, int K);
vgc_status vgc_compress(const float *g, const float *s, float *r, float *v, size_t n,
                        const uint32_t *group_offsets, int K, float alpha, float zeta,
                        const vgc_message *out, void *ws, size_t ws_bytes, vgc_stream_t stream);

/* vgc_compress without a workspace argument.  (No counterpart in the paper: this is a packaging
 * variant of the call above for hosts that cannot allocate.)
 *
 * Who needs it: callers that are not in a position to allocate device memory where they call the
 * library -- programs whose device memory was planned and handed out in full beforehand, plug-ins
 * invoked in the middle of another framework's step where an allocation would stall the device or is
 * not permitted, and hosts that only ever lend the library the tensors of the call.  Here the scratch
 * is a fixed array inside the library image: every GPU that loads the library sets aside
 * 8 * VGC_COMPRESS_STATIC_MAX_PARAMS bytes (plus a few tens of KB) until the process exits.
 *
 *   - Same arguments, results and error rules as vgc_compress, minus ws / ws_bytes.
 *   - n > VGC_COMPRESS_STATIC_MAX_PARAMS or K > VGC_COMPRESS_STATIC_MAX_GROUPS: VGC_ERR_UNSUPPORTED
 *     (nothing is enqueued).
 *   - The call itself performs no allocation of any kind.  The first call on each device looks up
 *     the device address of the array (one cudaGetSymbolAddress, with that device current); make that
 *     first call before any stream capture starts.
 *   - All calls on a device share the one array and it keeps whatever the previous call left in it
 *     (the call clears the part that must start at zero).  Two calls that overlap on the GPU -- other
 *     streams, other host threads -- race on it: serialise them, or use vgc_compress with separate
 *     workspaces.
 */
#define VGC_COMPRESS_STATIC_MAX_PARAMS (1u << 21)
#define VGC_COMPRESS_STATIC_MAX_GROUPS 1024
vgc_status vgc_compress_static(const float *g, const float *s, float *r, float *v, size_t n,
                               const uint32_t *group_offsets, int K, float alpha, float zeta,
                               const vgc_message *out, vgc_stream_t stream);

/* ---------------------------------------------------------------------------------------------
 * (3) Decoder: the decode-and-sum half of CommunicateAndUpdate (Sec. 4.3; Fig. 1 caption).
 *
 * For every word of every message w:  u[idx] += scale * (-1)^sign * 2^(group_exp_w[k] - d), k the
 * tensor that holds idx.  The W messages are summed ("allreduce" semantics of Sec. 4.3 realised
 * after an allgatherv); scale = 1/W gives the mean.
 *
 *   msgs   HOST array of W views; each view holds DEVICE pointers; the word count is read on the device.
 *          Words must be in ascending index order, as vgc_compress emits them.
 *   u      [n] fp32, accumulated in place (the caller zeroes it when a fresh sum is wanted)
 *
 * Arithmetic.  Every result is a deterministic function of the inputs' bits when the messages together hold at
 * least one word per eight elements (u then moves through shared memory, tensor by tensor), so every worker that
 * decodes the same messages gets the same bits.  Two forms, chosen per weight tensor:
 *   exact    taken when all messages start on 16-byte boundaries and, for the tensor, the messages' exponents lie
 *            close together (E_max - E_min + 7 + ceil(log2 W) <= 22).  The words of an element are then integer
 *            multiples of one power of two and are summed exactly; the element becomes scale * sum (vgc_decode_sum)
 *            or u + scale * sum (vgc_decode_accumulate), each operation rounded once.  With a scale that is a
 *            power of two nothing is rounded before the final addition, and vgc_decode_sum returns the bits of the
 *            sum taken message by message in fp32.  Elements no word points at keep their bits (accumulate).
 *   ordered  otherwise: u[idx] += scale * value, rounded per word, in message order (w = 0, 1, ...) -- the fp32
 *            sequence of a sequential loop.
 *   The two differ by at most the roundings of the sequential loop: (W + 2) half-ulps of |u| + sum |scale * value|.
 * Sparser calls add scale * value with fp32 atomics, in any order: an element hit by three or more messages may
 * then differ from the sequential sum in the last bit.
 *
 * Words whose index is >= n are skipped and VGC_DEV_RANGE is set; a word that breaks the ascending order may
 * be skipped as well (never applied to a wrong element), again with VGC_DEV_RANGE.  A view's word count above
 * its max_words is clamped (VGC_DEV_CAPACITY).  W == 0 or n == 0: no-op, OK.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    const uint32_t *words;    /* [max_words] packed words, of which the first min(*nnz, max_words) are read  */
    const uint32_t *nnz;      /* [1] number of words (a truncated message carries the count that was needed) */
    const int32_t *group_exp; /* [K]                                                                          */
    uint32_t max_words;       /* words the buffer holds: the decoder never reads past it                      */
} vgc_message_view;

vgc_status vgc_decode_accumulate(const vgc_message_view *msgs, int W,
                                 const uint32_t *group_offsets, int K, float scale,
                                 float *u, size_t n, uint32_t *dev_status, vgc_stream_t stream);

/* Same sum, written instead of added:  u = scale * (sum over all words of all messages)  -- every element of
 * u is written (zero where no word points), so the caller need not clear u first and u is not read.  This is
 * the dense update of Sec. 4.3 when nothing else has been accumulated into the buffer. */
vgc_status vgc_decode_sum(const vgc_message_view *msgs, int W, const uint32_t *group_offsets, int K,
                          float scale, float *u, size_t n, uint32_t *dev_status, vgc_stream_t stream);

/* ---------------------------------------------------------------------------------------------
 * One worker step from HOST buffers (end-to-end form of (1) + (2); Algorithm 1 from CalcGrad()'s
 * outputs to the encoded message).  For each layer, in order: copy x and delta from host memory into
 * the given device buffers, compute the layer's squared-gradient sums into its slice of s_dev (layer
 * l is weight tensor l of the flat buffer, K == n_layers); then copy g from the host, run vgc_compress
 * and copy the message back: counters_host[4] = {nnz, n_criterion, n_dropped, dev_status} and the
 * first min(nnz, capacity) words into words_host.  Host buffers should be pinned.  Unlike the other
 * entry points this one WAITS for the stream (twice: the word count has to reach the host before the
 * words can be copied).  `out` holds device pointers as for vgc_compress; r, v are device state.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    int is_conv;                 /* 0: dense layer (C = in, Cout = out; H, W, K*, stride, pad ignored) */
    int B, C, H, W, Cout, Kh, Kw, stride_h, stride_w, pad_h, pad_w;
    const float *x_host, *delta_host; /* host: x [B][C][H][W] or [B][in]; delta [B][Cout][Ho][Wo] or [B][out] */
    float *x_dev, *delta_dev;         /* device staging of the same sizes */
} vgc_layer_host;

vgc_status vgc_step_host(const vgc_layer_host *layers, int n_layers, const float *g_host, float *g_dev,
                         float *s_dev, float *r, float *v, size_t n, const uint32_t *group_offsets, int K,
                         float alpha, float zeta, float scale, const vgc_message *out, uint32_t *words_host,
                         uint32_t *counters_host, void *ws_sqgrad, size_t ws_sqgrad_bytes, void *ws_compress,
                         size_t ws_compress_bytes, vgc_stream_t stream);

/* ---------------------------------------------------------------------------------------------
 * (4) Hybrid algorithm (Algorithm 2; Sec. 4.5): the variance criterion combined with the fixed
 * threshold tau of Strom's method.  Per parameter, every operation one rounded fp32 operation:
 *
 *   r1 = r + g;  v1 = v + s
 *   send = |r1| > tau  and  r1*r1 > alpha*v1          (both strict)
 *   if send:  emit Sign(r1);  r2 = r1 - Sign(r1)*tau
 *             v1 = max((v1 - (2*a)*tau) + tau*tau, 0)     a = |r1|, or |r2| when
 *                                                          correction_from_updated_r != 0
 *             r1 = r2
 *   r = r1;  v = v1 * zeta                             (v decays at every step, sent or not)
 *
 * a = |r1| is the reading under which the correction is the "(a - b)^2" of Sec. 4.5 for a single
 * sample (v - 2|r|tau + tau^2 = (|r| - tau)^2 when v = r^2); a = |r2| follows the order in which the
 * listing of Algorithm 2 states the two updates.  The message carries no magnitudes: each 32-bit word
 * is  index << 4 | sign << 3  (low three bits zero), ascending index -- the same container as the
 * basic algorithm's words, a choice of this library (the paper does not print the hybrid's format).
 *
 *   s       may be NULL, as for vgc_compress (the squared sums were accumulated into v already)
 *   out     DEVICE pointers: words [capacity], nnz [1], mask [n] or NULL (needs 4-byte alignment),
 *           dev_status [1] (sticky; VGC_DEV_CAPACITY when more than capacity elements were sent: nnz
 *           still counts them all, the first `capacity` words are valid, r and v are updated for all)
 *   ws      DEVICE scratch of vgc_compress_hybrid_workspace_bytes(n) bytes, 16-byte aligned
 * tau must be finite and >= 0; alpha, zeta as for vgc_compress.  Asynchronous on `stream`.
 *
 * vgc_decode_accumulate_hybrid:  u[idx] += scale * (-1)^sign * tau  for every word of every message
 * (views' group_exp is not read and may be NULL); otherwise as vgc_decode_accumulate.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    uint32_t *words;       /* [capacity] out */
    uint32_t capacity;
    uint32_t *nnz;         /* [1] out: elements sent */
    uint8_t *mask;         /* [n] out or NULL: 1 where the element was sent */
    uint32_t *dev_status;  /* [1] sticky VGC_DEV_* bits */
} vgc_hybrid_message;

size_t vgc_compress_hybrid_workspace_bytes(size_t n);
vgc_status vgc_compress_hybrid(const float *g, const float *s, float *r, float *v, size_t n, float alpha,
                               float zeta, float tau, int correction_from_updated_r,
                               const vgc_hybrid_message *out, void *ws, size_t ws_bytes, vgc_stream_t stream);
vgc_status vgc_decode_accumulate_hybrid(const vgc_message_view *msgs, int W, float tau, float scale, float *u,
                                        size_t n, uint32_t *dev_status, vgc_stream_t stream);
/* vgc_decode_sum for hybrid messages: u = scale * (sum of +-tau), every element written. */
vgc_status vgc_decode_sum_hybrid(const vgc_message_view *msgs, int W, float tau, float scale, float *u, size_t n,
                                 uint32_t *dev_status, vgc_stream_t stream);

/* ---------------------------------------------------------------------------------------------
 * (5) Index compression of a packed message (Sec. 4.2, last paragraph: the index field can be stored in
 * fewer bits).  The paper names the idea without a format; this one is the library's.  The words of a
 * message are in ascending index order, so the 28-bit index field is replaced by the difference to the
 * previous index:  v = (idx_i - idx_{i-1}) << 4 | (word_i & 15), written in the base-128 variable-length
 * code (seven bits per byte, least significant first, top bit = "another byte follows": 1 to 5 bytes).
 * Words are taken in runs of VGC_PACK_RUN; every run starts from idx_{-1} = 0, so runs are independent.
 *
 *   stream = [table: (runs + 1) x uint32 little endian][payload]     runs = ceil(nnz / VGC_PACK_RUN)
 *            table[j] = offset of run j's first byte inside the payload, table[runs] = payload length
 *
 * At send densities of 1e-2 .. 1e-3 a word takes 2 bytes instead of 4.  The 4-bit value field, the
 * per-tensor exponents and the word count travel unchanged.
 *
 * vgc_pack_indices     words [min(*nnz, max_words)] (device, as vgc_compress wrote them) -> packed (device,
 *                      at least vgc_pack_bound_bytes(max_words) bytes for a guaranteed fit); *packed_bytes
 *                      (device) receives the stream's length.  A too small buffer: the stream is cut,
 *                      VGC_DEV_CAPACITY is set and *packed_bytes still holds the length that was needed.
 *                      ws: vgc_pack_workspace_bytes(max_words) bytes of device scratch.
 * vgc_unpack_indices   the inverse: rebuilds min(*nnz, max_words) words from a stream.  A run whose bytes do not
 *                      parse (wrong length, a number longer than five bytes) sets VGC_DEV_RANGE and its words are
 *                      written as 0xFFFFFFFF, an index no buffer has, so that a decoder skips them.
 * Both only enqueue work on `stream`; nnz is read on the device.
 * ------------------------------------------------------------------------------------------- */
#define VGC_PACK_RUN 256
size_t vgc_pack_bound_bytes(uint32_t max_words);
size_t vgc_pack_workspace_bytes(uint32_t max_words);
vgc_status vgc_pack_indices(const uint32_t *words, const uint32_t *nnz, uint32_t max_words, uint8_t *packed,
                            size_t packed_capacity, uint32_t *packed_bytes, uint32_t *dev_status, void *ws,
                            size_t ws_bytes, vgc_stream_t stream);
vgc_status vgc_unpack_indices(const uint8_t *packed, const uint32_t *nnz, uint32_t max_words, uint32_t *words,
                              uint32_t *dev_status, vgc_stream_t stream);

#ifdef __cplusplus
}
#endif
#endif /* VGC_H_ */
