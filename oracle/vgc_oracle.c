/*
 * vgc_oracle.c -- TEST INFRASTRUCTURE, not product code.
 *
 * A plain, slow, single-threaded CPU statement of what the variance-based
 * gradient compression hot path computes (Tsuzuku, Imachi, Akiba: "Variance-based
 * Gradient Compression for Efficient Distributed Deep Learning").  Only the test
 * suite, the smoke check and the benchmark's cpu_baseline leg may call it; the
 * CUDA library shares no code, header, table or helper with this file.
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -shared -fPIC (no FMA contraction,
 * no flush-to-zero: the compressor's fp32 operations are one IEEE-754 binary32
 * round-to-nearest-even operation per statement, in the order written).
 *
 * Functions and the passage each follows:
 *   oracle_sqgrad_linear        Sec. 4.4 Eq. 2 right-hand side / Algorithm 1 "v_i +=" line:
 *                               sum over the mini-batch of squared per-example gradients
 *                               of a dense layer (definition written out, fp64).
 *   oracle_sqgrad_conv          same statistic for a conv weight with every
 *                               (example, output position) pair taken as one sample.
 *   oracle_sqgrad_conv_entries  the same definition evaluated on listed entries only.
 *   oracle_sqgrad_conv_exact    per-example conv gradients squared and summed (report only).
 *   oracle_compress             Algorithm 1 (Basic) loop body + Sec. 4.2 quantisation with
 *                               the Sec. 4.4 bit-level recipe + the 4+28-bit word of Sec. 4.2.
 *   oracle_decode_accumulate    decode half of CommunicateAndUpdate (Sec. 4.3, Fig. 1 caption).
 *   oracle_compress_hybrid      Algorithm 2 (Hybrid) loop body with the variance correction of Sec. 4.5.
 *   oracle_decode_hybrid        its receiver side: every word adds +-tau.
 *   oracle_pack_indices /       Sec. 4.2, last paragraph ("compressing parameter indexes"): the sorted 28-bit
 *   oracle_unpack_indices       index field stored as differences in a variable-length code.  The paper names
 *                               the idea without a format; the format is this build's (see the functions).
 *
 * Parity pins (tests/, run without a GPU): the Appendix B worked example; closed forms
 * of the Algorithm 1 state machine; equivalence of Eq. 2 with Eq. 1 via the last line of
 * Appendix A; residual accounting; brute-force per-example gradients for the squared sums;
 * for the hybrid: its reduction to the plain threshold method (alpha = 0), the "(a-b)^2" identity
 * of Sec. 4.5 on single samples, the never-send limits, agreement with Algorithm 1's test at tau = 0.
 * For the index code: byte strings written out by hand from the rule, the exact size in closed form, round trips, and
 * a second writing of the standard base-128 code in the tests.
 * Conventions the paper leaves open (scope of M_k, bit positions in the word, width of
 * the per-group exponent, the layout of the compressed index stream) are choices of this build:
 * "parity unpinned" for those.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_EXP_NONE INT32_MIN

static uint32_t bits_of(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }
static float float_of(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }

/* ------------------------------------------------------------------------- */
/* Squared per-example gradient sums                                          */
/* ------------------------------------------------------------------------- */

/* Dense layer y_z = W x_z with back-propagated error delta_z = df_z/dy_z.  The gradient
 * of example z for weight W[j][i] is delta[z][j] * x[z][i]; the statistic is the sum over
 * z of its square, times `scale` (1/B^2 when delta carries no 1/B; Algorithm 1 accumulates
 * (grad_z / B)^2).  x is [B][in], delta is [B][out], S is [out][in], all row-major fp32.
 * accumulate != 0 adds to the existing S (in fp64, one final rounding). */
void oracle_sqgrad_linear(const float *x, const float *delta, int B, int in, int out,
                          float scale, int accumulate, float *S)
{
    for (int j = 0; j < out; ++j) {
        for (int i = 0; i < in; ++i) {
            double acc = 0.0;
            for (int z = 0; z < B; ++z) {
                double grad = (double)delta[(size_t)z * out + j] * (double)x[(size_t)z * in + i];
                acc += grad * grad;
            }
            double res = (double)scale * acc;
            if (accumulate) res += (double)S[(size_t)j * in + i];
            S[(size_t)j * in + i] = (float)res;
        }
    }
}

static int conv_out_dim(int in, int k, int stride, int pad) { return (in + 2 * pad - k) / stride + 1; }

/* One entry S[o][c][kh][kw] of the conv statistic: cross-correlation, zero padding,
 * dilation 1, groups 1.  Each (example z, output position (ho,wo)) contributes
 * a = delta[z][o][ho][wo] * x[z][c][ho*sh+kh-ph][wo*sw+kw-pw] (0 outside the image);
 * the statistic is scale * sum a^2. */
static double conv_entry(const float *x, const float *delta, int B, int C, int H, int W, int Cout,
                         int Ho, int Wo, int sh, int sw, int ph, int pw,
                         int o, int c, int kh, int kw)
{
    double acc = 0.0;
    for (int z = 0; z < B; ++z) {
        for (int ho = 0; ho < Ho; ++ho) {
            int hi = ho * sh + kh - ph;
            if (hi < 0 || hi >= H) continue;
            for (int wo = 0; wo < Wo; ++wo) {
                int wi = wo * sw + kw - pw;
                if (wi < 0 || wi >= W) continue;
                double a = (double)delta[(((size_t)z * Cout + o) * Ho + ho) * Wo + wo] *
                           (double)x[(((size_t)z * C + c) * H + hi) * W + wi];
                acc += a * a;
            }
        }
    }
    return acc;
}

void oracle_sqgrad_conv(const float *x, const float *delta, int B, int C, int H, int W, int Cout,
                        int Kh, int Kw, int sh, int sw, int ph, int pw,
                        float scale, int accumulate, float *S)
{
    int Ho = conv_out_dim(H, Kh, sh, ph), Wo = conv_out_dim(W, Kw, sw, pw);
    for (int o = 0; o < Cout; ++o)
        for (int c = 0; c < C; ++c)
            for (int kh = 0; kh < Kh; ++kh)
                for (int kw = 0; kw < Kw; ++kw) {
                    size_t at = (((size_t)o * C + c) * Kh + kh) * Kw + kw;
                    double res = (double)scale *
                                 conv_entry(x, delta, B, C, H, W, Cout, Ho, Wo, sh, sw, ph, pw, o, c, kh, kw);
                    if (accumulate) res += (double)S[at];
                    S[at] = (float)res;
                }
}

/* The same definition on `n_idx` listed flat OIHW positions (no accumulate): lets a test
 * compare sampled entries of a layer whose full statistic is out of reach on a CPU. */
void oracle_sqgrad_conv_entries(const float *x, const float *delta, int B, int C, int H, int W, int Cout,
                                int Kh, int Kw, int sh, int sw, int ph, int pw, float scale,
                                const int64_t *flat_idx, int64_t n_idx, float *out)
{
    int Ho = conv_out_dim(H, Kh, sh, ph), Wo = conv_out_dim(W, Kw, sw, pw);
    for (int64_t q = 0; q < n_idx; ++q) {
        int64_t f = flat_idx[q];
        int kw = (int)(f % Kw); f /= Kw;
        int kh = (int)(f % Kh); f /= Kh;
        int c = (int)(f % C);   f /= C;
        int o = (int)f;
        out[q] = (float)((double)scale *
                         conv_entry(x, delta, B, C, H, W, Cout, Ho, Wo, sh, sw, ph, pw, o, c, kh, kw));
    }
}

/* Per-example reading: the gradient of example z is the sum over output positions, and
 * that sum is squared.  Differs from oracle_sqgrad_conv by the cross terms between
 * positions; equal when there is one output position. */
void oracle_sqgrad_conv_exact(const float *x, const float *delta, int B, int C, int H, int W, int Cout,
                              int Kh, int Kw, int sh, int sw, int ph, int pw, float scale, float *S)
{
    int Ho = conv_out_dim(H, Kh, sh, ph), Wo = conv_out_dim(W, Kw, sw, pw);
    for (int o = 0; o < Cout; ++o)
        for (int c = 0; c < C; ++c)
            for (int kh = 0; kh < Kh; ++kh)
                for (int kw = 0; kw < Kw; ++kw) {
                    double acc = 0.0;
                    for (int z = 0; z < B; ++z) {
                        double gz = 0.0;
                        for (int ho = 0; ho < Ho; ++ho) {
                            int hi = ho * sh + kh - ph;
                            if (hi < 0 || hi >= H) continue;
                            for (int wo = 0; wo < Wo; ++wo) {
                                int wi = wo * sw + kw - pw;
                                if (wi < 0 || wi >= W) continue;
                                gz += (double)delta[(((size_t)z * Cout + o) * Ho + ho) * Wo + wo] *
                                      (double)x[(((size_t)z * C + c) * H + hi) * W + wi];
                            }
                        }
                        acc += gz * gz;
                    }
                    S[(((size_t)o * C + c) * Kh + kh) * Kw + kw] = (float)((double)scale * acc);
                }
}

/* ------------------------------------------------------------------------- */
/* Compressor: Algorithm 1 loop body, then quantise and pack                   */
/* ------------------------------------------------------------------------- */

/* g, s: this step's sum of per-example gradients / B and sum of their squares.
 * r, v: residual and variance state, updated in place.  group_offsets[K+1] splits the
 * flat buffer into K weight tensors.  Outputs: words (ascending index), group_exp[K],
 * counters, optional mask (1 where the send test passed).  Returns 0, or 1 when the
 * message did not fit `capacity` (state is still updated, *nnz is the needed count). */
int oracle_compress(const float *g, const float *s, float *r, float *v, uint64_t n,
                    const uint32_t *group_offsets, int K, float alpha, float zeta,
                    uint32_t *words, uint64_t capacity, int32_t *group_exp,
                    uint32_t *nnz, uint32_t *n_criterion, uint32_t *n_dropped, uint8_t *mask)
{
    uint8_t *send = (uint8_t *)malloc(n ? n : 1);
    float *val = (float *)malloc((n ? n : 1) * sizeof(float));
    uint32_t criterion = 0, dropped = 0, emitted = 0;
    int overflow = 0;

    /* Algorithm 1, loop over parameters. */
    for (uint64_t i = 0; i < n; ++i) {
        float r1 = r[i] + g[i];            /* r_i += sum grad/B          */
        float v1 = v[i] + s[i];            /* v_i += sum (grad/B)^2      */
        float lhs = r1 * r1;
        float rhs = alpha * v1;
        send[i] = (lhs > rhs) ? 1 : 0;     /* strict test of Eq. 2       */
        if (send[i]) {
            val[i] = r1;                   /* Encode(r_i) works on this  */
            r[i] = 0.0f;
            v[i] = 0.0f;
            ++criterion;
        } else {
            val[i] = 0.0f;
            r[i] = r1;
            v[i] = v1 * zeta;              /* decay only when not sent   */
        }
        if (mask) mask[i] = send[i];
    }

    /* Sec. 4.2: per weight tensor, M_k = largest magnitude among the elements being
     * sent; floor(log2 M_k) is the biased exponent field minus 127 ("truncate the
     * mantissa", Sec. 4.4). */
    for (int k = 0; k < K; ++k) {
        float Mk = 0.0f;
        int any = 0;
        for (uint64_t i = group_offsets[k]; i < group_offsets[k + 1]; ++i) {
            if (!send[i]) continue;
            float a = float_of(bits_of(val[i]) & 0x7FFFFFFFu);
            if (!any || a > Mk) Mk = a;
            any = 1;
        }
        group_exp[k] = any ? (int32_t)((bits_of(Mk) >> 23) & 0xFFu) - 127 : ORACLE_EXP_NONE;
    }

    /* Quantise each sent value to a power of two relative to 2^E_k and pack. */
    for (int k = 0; k < K; ++k) {
        for (uint64_t i = group_offsets[k]; i < group_offsets[k + 1]; ++i) {
            if (!send[i]) continue;
            uint32_t b = bits_of(val[i]);
            uint32_t a = b & 0x7FFFFFFFu;
            /* add one at the top mantissa bit, then drop the mantissa: rounds |val| to
             * the nearer power of two, the midpoint 1.5*2^e going up (Sec. 4.4) */
            int32_t e1 = (int32_t)((a + 0x00400000u) >> 23) - 127;
            int32_t Ek = group_exp[k];
            int32_t e = e1 < Ek ? e1 : Ek;      /* values above 2^E_k are cut to 2^E_k */
            int32_t d = Ek - e;
            if (d > 7) { ++dropped; continue; }  /* not representable in 3 bits: not sent */
            uint32_t word = ((uint32_t)i << 4) | ((b >> 31) << 3) | (uint32_t)d;
            if (emitted < capacity) words[emitted] = word; else overflow = 1;
            ++emitted;
        }
    }
    *nnz = emitted;
    *n_criterion = criterion;
    *n_dropped = dropped;
    free(send);
    free(val);
    return overflow;
}

/* ------------------------------------------------------------------------- */
/* Decoder: sum W messages into the dense update                              */
/* ------------------------------------------------------------------------- */

/* words[w] / nnz[w] / group_exp[w] describe message w.  For every word, in message order
 * and then word order: u[idx] += scale * (-1)^sign * 2^(E_k - d), fp32.  Returns the
 * number of words whose index was >= n (skipped). */
uint64_t oracle_decode_accumulate(const uint32_t *const *words, const uint32_t *nnz,
                                  const int32_t *const *group_exp, int W,
                                  const uint32_t *group_offsets, int K, float scale,
                                  float *u, uint64_t n)
{
    uint64_t bad = 0;
    for (int w = 0; w < W; ++w) {
        for (uint32_t q = 0; q < nnz[w]; ++q) {
            uint32_t word = words[w][q];
            uint32_t idx = word >> 4;
            uint32_t sign = (word >> 3) & 1u;
            int32_t d = (int32_t)(word & 7u);
            if (idx >= n) { ++bad; continue; }
            int k = 0;
            while (k + 1 < K && idx >= group_offsets[k + 1]) ++k;   /* tensor holding idx */
            int32_t e = group_exp[w][k] - d;
            float value = float_of(((uint32_t)(e + 127) << 23) | (sign << 31));
            float term = scale * value;
            u[idx] = u[idx] + term;
        }
    }
    return bad;
}

/* ------------------------------------------------------------------------- */
/* Hybrid of the variance test with a fixed threshold (Algorithm 2, Sec. 4.5) */
/* ------------------------------------------------------------------------- */

/* One step over the flat buffer.  An element is sent when |r| > tau AND r^2 > alpha*v; what is
 * sent is Sign(r) (the receiver adds +-tau), r keeps the remainder r - Sign(r)*tau, and the
 * sum of squares is corrected as Sec. 4.5 derives it ("a^2 -> (a-b)^2"):
 *     v <- max(v - 2*|r|*tau + tau^2, 0)
 * with |r| the accumulated sum BEFORE the subtraction (pre_update_r != 0, the reading the
 * derivation fixes: for a single sample v = r^2 it gives exactly (|r| - tau)^2), or AFTER it
 * (pre_update_r == 0, the statement order of the Algorithm 2 listing).  v decays every step.
 * Words: index << 4 | sign << 3, ascending index.  Returns 1 if the message did not fit. */
int oracle_compress_hybrid(const float *g, const float *s, float *r, float *v, uint64_t n,
                           float alpha, float zeta, float tau, int pre_update_r,
                           uint32_t *words, uint64_t capacity, uint32_t *nnz, uint8_t *mask)
{
    uint32_t emitted = 0;
    int overflow = 0;
    for (uint64_t i = 0; i < n; ++i) {
        float r1 = r[i] + g[i];
        float v1 = v[i] + s[i];
        float absr = float_of(bits_of(r1) & 0x7FFFFFFFu);
        float lhs = r1 * r1;
        float rhs = alpha * v1;
        int send = (absr > tau) && (lhs > rhs);
        if (send) {
            uint32_t neg = bits_of(r1) >> 31;
            uint32_t word = ((uint32_t)i << 4) | (neg << 3);
            if (emitted < capacity) words[emitted] = word; else overflow = 1;
            ++emitted;
            float r2 = neg ? r1 + tau : r1 - tau;          /* r -= Sign(r) * tau */
            float a = pre_update_r ? absr : float_of(bits_of(r2) & 0x7FFFFFFFu);
            float twice = 2.0f * a;
            float cross = twice * tau;
            float diff = v1 - cross;
            float tsq = tau * tau;
            float corr = diff + tsq;
            v1 = corr > 0.0f ? corr : 0.0f;
            r1 = r2;
        }
        if (mask) mask[i] = (uint8_t)send;
        r[i] = r1;
        v[i] = v1 * zeta;                                   /* decay at every step */
    }
    *nnz = emitted;
    return overflow;
}

/* Receiver side of the hybrid: every word adds scale * (+-tau) to its element. */
uint64_t oracle_decode_hybrid(const uint32_t *const *words, const uint32_t *nnz, int W, float tau,
                              float scale, float *u, uint64_t n)
{
    uint64_t bad = 0;
    for (int w = 0; w < W; ++w)
        for (uint32_t q = 0; q < nnz[w]; ++q) {
            uint32_t word = words[w][q], idx = word >> 4;
            if (idx >= n) { ++bad; continue; }
            float value = ((word >> 3) & 1u) ? -tau : tau;
            float term = scale * value;
            u[idx] = u[idx] + term;
        }
    return bad;
}

/* ------------------------------------------------------------------------- */
/* Index compression of a packed message (Sec. 4.2, last paragraph)           */
/* ------------------------------------------------------------------------- */

/* The words of a message are in ascending index order, so an index is the previous one plus a
 * positive difference, and at send densities of 1e-2 .. 1e-3 the differences need 7 to 10 bits
 * instead of 28.  Format (a choice of this build):
 *   - the words are taken in runs of ORACLE_PACK_RUN = 256; a run starts afresh (its first
 *     "previous index" is 0), so runs can be decoded independently of one another;
 *   - word i of a run becomes the number  v = (idx_i - prev) << 4 | (word_i & 15)  -- the
 *     difference above the unchanged 4-bit value field (sign, d) -- written in the standard
 *     base-128 code: seven bits per byte, least significant group first, the top bit of a byte
 *     set when another byte follows (1 to 5 bytes, since v < 2^32);
 *   - the stream is  [table: (runs + 1) x uint32, little endian][payload], table[j] = offset of
 *     run j's first byte inside the payload, table[runs] = payload length; runs = ceil(nnz/256).
 * Returns the total size in bytes (table + payload); writes at most `capacity` bytes (a too
 * small buffer is detected by the caller comparing the two). */
#define ORACLE_PACK_RUN 256

uint64_t oracle_pack_indices(const uint32_t *words, uint32_t nnz, uint8_t *out, uint64_t capacity)
{
    const uint32_t runs = (nnz + ORACLE_PACK_RUN - 1) / ORACLE_PACK_RUN;
    const uint64_t table_bytes = 4ull * (runs + 1);
    uint64_t at = table_bytes;                       /* next payload byte, from the start of `out` */
    for (uint32_t j = 0; j <= runs; ++j) {
        const uint32_t first = j * ORACLE_PACK_RUN;
        const uint32_t offset = (uint32_t)(at - table_bytes);
        for (int b = 0; b < 4; ++b)                  /* table entry j, little endian */
            if (4ull * j + b < capacity) out[4ull * j + b] = (uint8_t)(offset >> (8 * b));
        if (j == runs) break;
        uint32_t prev = 0;
        for (uint32_t i = first; i < nnz && i < first + ORACLE_PACK_RUN; ++i) {
            const uint32_t idx = words[i] >> 4;
            uint32_t v = ((idx - prev) << 4) | (words[i] & 15u);
            prev = idx;
            for (;;) {
                const uint8_t low = (uint8_t)(v & 0x7Fu);
                v >>= 7;
                if (at < capacity) out[at] = (uint8_t)(low | (v ? 0x80u : 0u));
                ++at;
                if (!v) break;
            }
        }
    }
    return at;
}

/* The inverse: rebuilds the `nnz` 32-bit words from a stream written by the rule above.
 * Returns 0, or -1 when the stream is malformed (a number longer than five bytes, or a run
 * that does not end where the table says). */
int oracle_unpack_indices(const uint8_t *in, uint32_t nnz, uint32_t *words)
{
    const uint32_t runs = (nnz + ORACLE_PACK_RUN - 1) / ORACLE_PACK_RUN;
    const uint64_t table_bytes = 4ull * (runs + 1);
    for (uint32_t j = 0; j < runs; ++j) {
        uint32_t begin = 0, end = 0;
        for (int b = 0; b < 4; ++b) {
            begin |= (uint32_t)in[4ull * j + b] << (8 * b);
            end |= (uint32_t)in[4ull * (j + 1) + b] << (8 * b);
        }
        uint64_t at = table_bytes + begin;
        uint32_t prev = 0;
        const uint32_t first = j * ORACLE_PACK_RUN;
        for (uint32_t i = first; i < nnz && i < first + ORACLE_PACK_RUN; ++i) {
            uint32_t v = 0;
            int shift = 0;
            for (;;) {
                const uint8_t byte = in[at++];
                if (shift > 28) return -1;
                v |= (uint32_t)(byte & 0x7Fu) << shift;
                shift += 7;
                if (!(byte & 0x80u)) break;
            }
            const uint32_t idx = prev + (v >> 4);
            words[i] = (idx << 4) | (v & 15u);
            prev = idx;
        }
        if (at != table_bytes + end) return -1;
    }
    return 0;
}
