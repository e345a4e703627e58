/*
 * EOQ oracle -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, direct-loop CPU statement of what the EOQ 8-bit training
 * layer computes (arXiv 2105.13890): the quantizers Q / CQ / SQ of Sec. 3.2.2,
 * the per-datum strategies of Sec. 3.2.3 with every bit width k = 8 (Sec. 5.1),
 * the forward chain x0..x5, the error chain e0..e5 and the gradients of
 * Sec. 3.2.1, and the 8-bit update Q_u of Sec. 3.2.3.  Only the tests, the
 * smoke check and the CPU-baseline leg of the benchmark may call it.  It shares
 * no code with the CUDA path and never calls it.
 *
 * Representation.  A quantized tensor is (integer codes c, exponent p) with
 * real value c * 2^p.  Q(.,8) and CQ(.,8) live on the grid 2^-7, so forward
 * tensors have p = -7; SQ outputs carry the exponent log2(scale) - 7.
 *
 * Readings of the paper taken here (each is a convention of this build where
 * the paper is silent; "parity unpinned" marks those no published value fixes):
 *   - R(.) rounds to nearest, ties to even                (parity unpinned)
 *   - the formulas' grid 2^-(k-1) governs, not the prose "resolution 1/2^k"
 *   - x1 = x0 + b1 is kept exact (no int8 saturation); the zero padding of the
 *     convolution is applied to x1 (the halo is 0, not b1)
 *   - x2 = Q_a1(conv) is saturated to int16 codes         (parity unpinned)
 *   - gamma and the biases are layer-wise scalars with int16-range codes
 *   - d x5 / d x4 = [x4 > 0] (the clamp of Q_a2 is passed straight through)
 *                                                         (parity unpinned)
 *   - the shortcut joins at x4, before ReLU and Q_a2      (parity unpinned)
 *   - max|x| of SQ runs over the whole tensor; an all-zero tensor gives zero
 *     codes, keeps its exponent and raises a flag
 *   - weights are stored as int8 codes at p = -7; the update is plain SGD,
 *     w <- CQ(w - SQ(lr * g)), lr = lr_mant * 2^lr_exp     (parity unpinned)
 *   - stochastic rounding of the update is an extension, not in the paper
 *
 * Layouts: activations and errors NHWC, weights [c_out][kh][kw][c_in].
 * All accumulation is int64.  Build: gcc -O2 -fopenmp -ffp-contract=off -shared -fPIC.
 */
#include <fenv.h>
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <string.h>

typedef struct {
    int n, h, w, c_in, c_out, kh, kw, stride, pad;
} eoq_o_conv_t;

static int out_dim(int in, int k, int s, int p) { return (in + 2 * p - k) / s + 1; }

int eoq_o_out_h(const eoq_o_conv_t *d) { return out_dim(d->h, d->kh, d->stride, d->pad); }
int eoq_o_out_w(const eoq_o_conv_t *d) { return out_dim(d->w, d->kw, d->stride, d->pad); }

static int64_t sat64(int64_t v, int64_t lo, int64_t hi) { return v < lo ? lo : (v > hi ? hi : v); }

/* Floor division of a by 2^s together with the remainder in [0, 2^s). */
static int64_t floor_div_pow2(int64_t a, int s, int64_t *rem)
{
    int64_t d = (int64_t)1 << s;
    int64_t q = a / d;
    int64_t r = a % d;
    if (r < 0) { r += d; q -= 1; }
    *rem = r;
    return q;
}

/*
 * R(a / 2^s) for an integer a: nearest integer, ties to even (Sec. 3.2.2, the
 * rounding function R of the basic quantizer).  s = 0 returns a; s < 0 is the
 * exact product a * 2^-s.  s is capped at 62: a is below 2^62 in every caller,
 * so larger shifts round to 0 as well.
 */
int64_t eoq_o_rne_shr(int64_t a, int s)
{
    if (s == 0) return a;
    if (s < 0) return a * ((int64_t)1 << (-s));
    if (s > 62) s = 62;
    int64_t r, q = floor_div_pow2(a, s, &r);
    int64_t half = (int64_t)1 << (s - 1);
    if (r > half || (r == half && (q & 1))) q += 1;
    return q;
}

/* Q(x, 8) on a real: code = R(x * 2^7) (Sec. 3.2.2, basic quantization). */
int64_t eoq_o_q_code(double x)
{
    /* x * 128 is exact in double for every fp32 x; rint rounds ties to even
       under the default rounding mode. */
    return (int64_t)rint(x * 128.0);
}

/* CQ(x, 8): the Q code clamped to [-127, 127] (Sec. 3.2.2, clamp quantization). */
int64_t eoq_o_cq_code(double x) { return sat64(eoq_o_q_code(x), -127, 127); }

/*
 * R(log2 M) for a positive integer M (Sec. 3.2.2, scale(x) = 2^R(log2 max|x|)).
 * With f = floor(log2 M) the nearest integer is f + 1 exactly when
 * log2 M - f >= 1/2, i.e. M^2 >= 2^(2f+1).  A tie would need M = 2^(f+1/2),
 * which no integer is.
 */
int eoq_o_round_log2_u64(uint64_t M)
{
    int f = 0;
    while (f < 63 && (M >> (f + 1)) != 0) f++;
    unsigned __int128 sq = (unsigned __int128)M * M;
    unsigned __int128 th = (unsigned __int128)1 << (2 * f + 1);
    return f + (sq >= th ? 1 : 0);
}

/*
 * SQ(., 8) on integer codes a[i] at exponent p_a (Sec. 3.2.2, scale
 * quantization): scale = 2^(t + p_a), t = R(log2 max|a|); the normalised value
 * a * 2^p_a / scale is clamp-quantized, code = sat(R(a * 2^(7 - t)), -127, 127),
 * and the result carries exponent p_out = p_a + t - 7.
 * Returns 1 when the tensor is all zero (codes 0, exponent passed through).
 */
int eoq_o_sq_i64(const int64_t *a, size_t n, int p_a, int32_t *codes, int *p_out)
{
    uint64_t M = 0;
    for (size_t i = 0; i < n; i++) {
        uint64_t m = a[i] < 0 ? (uint64_t)(-a[i]) : (uint64_t)a[i];
        if (m > M) M = m;
    }
    if (M == 0) {
        for (size_t i = 0; i < n; i++) codes[i] = 0;
        *p_out = p_a;
        return 1;
    }
    int t = eoq_o_round_log2_u64(M);
    for (size_t i = 0; i < n; i++)
        codes[i] = (int32_t)sat64(eoq_o_rne_shr(a[i], t - 7), -127, 127);
    *p_out = p_a + t - 7;
    return 0;
}

/*
 * Q / CQ / SQ of an fp32 tensor (Sec. 3.2.2).  mode 0 = Q, 1 = CQ, 2 = SQ.
 * For SQ, t = R(log2 max|x|) is taken exactly from the binary form of the fp32
 * maximum: max = m * 2^e with m in [1/2, 1), and log2 m >= -1/2 iff m^2 >= 1/2.
 * Scaling by 2^(7 - t) is exact.  Returns 1 for an all-zero SQ input, -1 if a
 * value is not finite, else 0.  *p_out is -7 for Q and CQ.
 */
int eoq_o_quantize_f32(int mode, const float *x, size_t n, int32_t *codes, int *p_out)
{
    for (size_t i = 0; i < n; i++)
        if (!isfinite(x[i])) return -1;
    if (mode == 0 || mode == 1) {
        for (size_t i = 0; i < n; i++)
            codes[i] = (int32_t)(mode == 0 ? sat64(eoq_o_q_code(x[i]), INT32_MIN, INT32_MAX)
                                           : eoq_o_cq_code(x[i]));
        *p_out = -7;
        return 0;
    }
    float M = 0.0f;
    for (size_t i = 0; i < n; i++) {
        float m = fabsf(x[i]);
        if (m > M) M = m;
    }
    if (M == 0.0f) {
        for (size_t i = 0; i < n; i++) codes[i] = 0;
        *p_out = -7;
        return 1;
    }
    int e;
    double m = frexp((double)M, &e);
    int t = (m * m >= 0.5) ? e : e - 1;
    for (size_t i = 0; i < n; i++) {
        double v = rint(ldexp((double)x[i], 7 - t));
        codes[i] = (int32_t)sat64((int64_t)v, -127, 127);
    }
    *p_out = t - 7;
    return 0;
}

/* x1 = x0 + Q_b(b1) inside the image, 0 in the padding halo (Sec. 3.2.1, forward chain). */
static int64_t x1_at(const eoq_o_conv_t *d, const int8_t *x0, int b1_c, int n, int iy, int ix, int ic)
{
    if (iy < 0 || iy >= d->h || ix < 0 || ix >= d->w) return 0;
    size_t idx = (((size_t)n * d->h + iy) * d->w + ix) * d->c_in + ic;
    return (int64_t)x0[idx] + b1_c;
}

/*
 * conv(x1) of the forward chain (Sec. 3.2.1): A[n,y,x,oc] = sum over kh, kw, ic
 * of x1[n, y*s + kh - p, x*s + kw - p, ic] * w[oc, kh, kw, ic].  Exact integers.
 */
void eoq_o_conv_fwd_acc(const eoq_o_conv_t *d, const int8_t *x0, int b1_c, const int8_t *w, int64_t *A)
{
    int ho = eoq_o_out_h(d), wo = eoq_o_out_w(d);
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < d->n; n++)
        for (int y = 0; y < ho; y++)
            for (int x = 0; x < wo; x++)
                for (int oc = 0; oc < d->c_out; oc++) {
                    int64_t acc = 0;
                    for (int kh = 0; kh < d->kh; kh++)
                        for (int kw = 0; kw < d->kw; kw++)
                            for (int ic = 0; ic < d->c_in; ic++) {
                                int64_t a = x1_at(d, x0, b1_c, n, y * d->stride + kh - d->pad,
                                                  x * d->stride + kw - d->pad, ic);
                                int64_t b = w[(((size_t)oc * d->kh + kh) * d->kw + kw) * d->c_in + ic];
                                acc += a * b;
                            }
                    A[(((size_t)n * ho + y) * wo + x) * d->c_out + oc] = acc;
                }
}

/*
 * The rest of the forward chain on the accumulator (Sec. 3.2.1):
 *   x2 = Q_a1(conv)      code = sat16(R(A / 2^acc_shift))  (acc_shift = 7 when the input is at p = -7)
 *   x3 = Q_gamma(gamma) * x2                                (p = -14)
 *   x4 = x3 + Q_b(b2) [+ shortcut]                          (p = -14)
 *   x5 = Q_a2(relu(x4))  code = sat(R(max(x4, 0) / 2^7), -127, 127)
 * mask = [x4 > 0] is the ReLU derivative the error chain needs.  shortcut may
 * be NULL; relu = 0 leaves x4 as it is before Q_a2.  x2 and mask may be NULL.
 */
void eoq_o_fwd_epilogue(const int64_t *A, size_t n_el, int acc_shift, int gamma_c, int b2_c,
                        const int8_t *shortcut, int relu, int32_t *x2, int8_t *x5, uint8_t *mask)
{
    for (size_t i = 0; i < n_el; i++) {
        int64_t v2 = sat64(eoq_o_rne_shr(A[i], acc_shift), -32768, 32767);
        int64_t v3 = (int64_t)gamma_c * v2;
        int64_t v4 = v3 + (int64_t)b2_c * 128 + (shortcut ? (int64_t)shortcut[i] * 128 : 0);
        int64_t r = (relu && v4 < 0) ? 0 : v4;
        if (x2) x2[i] = (int32_t)v2;
        if (mask) mask[i] = v4 > 0;
        x5[i] = (int8_t)sat64(eoq_o_rne_shr(r, 7), -127, 127);
    }
}

/*
 * e3 * Q_w(w) of the error chain (Sec. 3.2.1), the adjoint of conv with respect
 * to its input: B[n,y,x,ic] = sum over oc, kh, kw of e3[n, yo, xo, oc] * w[oc,kh,kw,ic]
 * for those taps where yo = (y + p - kh) / s and xo = (x + p - kw) / s are
 * integers inside the output image.
 */
void eoq_o_conv_dgrad_acc(const eoq_o_conv_t *d, const int8_t *e3, const int8_t *w, int64_t *B)
{
    int ho = eoq_o_out_h(d), wo = eoq_o_out_w(d);
#pragma omp parallel for collapse(2) schedule(static)
    for (int n = 0; n < d->n; n++)
        for (int y = 0; y < d->h; y++)
            for (int x = 0; x < d->w; x++)
                for (int ic = 0; ic < d->c_in; ic++) {
                    int64_t acc = 0;
                    for (int kh = 0; kh < d->kh; kh++) {
                        int ty = y + d->pad - kh;
                        if (ty < 0 || ty % d->stride) continue;
                        int yo = ty / d->stride;
                        if (yo >= ho) continue;
                        for (int kw = 0; kw < d->kw; kw++) {
                            int tx = x + d->pad - kw;
                            if (tx < 0 || tx % d->stride) continue;
                            int xo = tx / d->stride;
                            if (xo >= wo) continue;
                            for (int oc = 0; oc < d->c_out; oc++) {
                                int64_t a = e3[(((size_t)n * ho + yo) * wo + xo) * d->c_out + oc];
                                int64_t b = w[(((size_t)oc * d->kh + kh) * d->kw + kw) * d->c_in + ic];
                                acc += a * b;
                            }
                        }
                    }
                    B[(((size_t)n * d->h + y) * d->w + x) * d->c_in + ic] = acc;
                }
}

/*
 * e3 * x1 of the weight gradient (Sec. 3.2.1), the adjoint of conv with respect
 * to the weights: G[oc,kh,kw,ic] = sum over n, y, x of
 * e3[n,y,x,oc] * x1[n, y*s + kh - p, x*s + kw - p, ic].
 */
void eoq_o_conv_wgrad_acc(const eoq_o_conv_t *d, const int8_t *e3, const int8_t *x0, int b1_c, int64_t *G)
{
    int ho = eoq_o_out_h(d), wo = eoq_o_out_w(d);
#pragma omp parallel for collapse(2) schedule(static)
    for (int oc = 0; oc < d->c_out; oc++)
        for (int kh = 0; kh < d->kh; kh++)
            for (int kw = 0; kw < d->kw; kw++)
                for (int ic = 0; ic < d->c_in; ic++) {
                    int64_t acc = 0;
                    for (int n = 0; n < d->n; n++)
                        for (int y = 0; y < ho; y++)
                            for (int x = 0; x < wo; x++) {
                                int64_t a = e3[(((size_t)n * ho + y) * wo + x) * d->c_out + oc];
                                int64_t b = x1_at(d, x0, b1_c, n, y * d->stride + kh - d->pad,
                                                  x * d->stride + kw - d->pad, ic);
                                acc += a * b;
                            }
                    G[(((size_t)oc * d->kh + kh) * d->kw + kw) * d->c_in + ic] = acc;
                }
}

/*
 * Head of the error chain (Sec. 3.2.1): e1 = e0 * [x4 > 0], e2 = e1,
 * e3 = Q_e(e2 * Q_gamma(gamma)), and the two scalar sums behind
 * g_b2 = Q_g(sum e1) and g_gamma = Q_g(sum e2 * x2).  e0 has exponent p0;
 * gamma * e1 has exponent p0 - 7.  mask holds one byte (0/1) per element; x2
 * may be NULL (sum_e1x2 is then 0).  Returns the SQ zero flag.
 */
int eoq_o_err_prescale(const int8_t *e0, int p0, const uint8_t *mask, const int32_t *x2, size_t n_el,
                       int gamma_c, int32_t *e3, int *p3, int64_t *sum_e1, int64_t *sum_e1x2)
{
    int64_t *t = (int64_t *)__builtin_malloc(sizeof(int64_t) * (n_el ? n_el : 1));
    int64_t s1 = 0, s2 = 0;
    for (size_t i = 0; i < n_el; i++) {
        int64_t e1 = mask[i] ? (int64_t)e0[i] : 0;
        s1 += e1;
        if (x2) s2 += e1 * (int64_t)x2[i];
        t[i] = (int64_t)gamma_c * e1;
    }
    int z = eoq_o_sq_i64(t, n_el, p0 - 7, e3, p3);
    __builtin_free(t);
    *sum_e1 = s1;
    *sum_e1x2 = s2;
    return z;
}

/* SplitMix64 output function (Steele, Lea, Flood 2014), used as a counter hash. */
static uint64_t mix64(uint64_t z)
{
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
    return z ^ (z >> 31);
}

/* The 64 random bits drawn for element idx of tensor tensor_id at a given step. */
uint64_t eoq_o_update_hash(uint64_t seed, uint64_t step, uint64_t tensor_id, uint64_t idx)
{
    uint64_t k = mix64(seed + 0x9E3779B97F4A7C15ULL * (step + 1));
    k = mix64(k + 0x9E3779B97F4A7C15ULL * (tensor_id + 1));
    return mix64(k + 0x9E3779B97F4A7C15ULL * (idx + 1));
}

/*
 * The 8-bit update (Sec. 3.2.3, update quantization): u = Q_u(lr * g) =
 * SQ(lr * g, 8) with lr = lr_mant * 2^lr_exp, then the parameter's own
 * quantizer is applied to theta - u: code = sat(R((theta - u) * 2^7), lo, hi)
 * with [lo, hi] = [-127, 127] for weights (Q_w = CQ) and the int16 range for
 * gamma and the biases (Q).  theta has exponent -7 and u has exponent p_u:
 * with d = p_u + 7 >= 0 the difference is already on the grid,
 * theta - u * 2^d; otherwise, in units of 2^p_u, it is v = theta * 2^s - u with
 * s = -d, and R(v / 2^s) rounds to nearest-even (stochastic = 0) or is
 * floor((v + r) / 2^s) with r the low s bits of the element's hash
 * (stochastic = 1; an extension, not in the paper).  For s > 40 the update is
 * below 2^-33 of a weight step and is dropped in both modes (exact for
 * nearest-even).  theta holds int32 codes.  Returns the SQ zero flag; *p_u_out
 * reports the exponent of u.
 */
int eoq_o_update(int32_t *theta, const int8_t *g, int p_g, size_t n, int lr_mant, int lr_exp, int lo, int hi,
                 int stochastic, uint64_t seed, uint64_t step, uint64_t tensor_id, int *p_u_out)
{
    int64_t *a = (int64_t *)__builtin_malloc(sizeof(int64_t) * (n ? n : 1));
    int32_t *u = (int32_t *)__builtin_malloc(sizeof(int32_t) * (n ? n : 1));
    for (size_t i = 0; i < n; i++) a[i] = (int64_t)lr_mant * g[i];
    int p_u;
    int z = eoq_o_sq_i64(a, n, p_g + lr_exp, u, &p_u);
    int d = p_u + 7;
    for (size_t i = 0; i < n; i++) {
        int64_t next;
        if (d >= 0) {
            /* |u| <= 127 and |theta| < 2^15: a shift of 40 or more saturates theta all the same */
            next = (int64_t)theta[i] - (int64_t)u[i] * ((int64_t)1 << (d > 40 ? 40 : d));
        } else if (-d > 40) {
            next = theta[i];
        } else {
            int s = -d;
            int64_t v = (int64_t)theta[i] * ((int64_t)1 << s) - u[i];
            if (!stochastic) {
                next = eoq_o_rne_shr(v, s);
            } else {
                uint64_t r = eoq_o_update_hash(seed, step, tensor_id, i) & (((uint64_t)1 << s) - 1);
                int64_t rem;
                next = floor_div_pow2(v + (int64_t)r, s, &rem);
            }
        }
        theta[i] = (int32_t)sat64(next, lo, hi);
    }
    *p_u_out = p_u;
    __builtin_free(a);
    __builtin_free(u);
    return z;
}

/* ------------------------------------------------------------------------------------------------
 * Network glue around the quantized convolution units (conventions of this build where the paper is
 * silent; every one of them is "parity unpinned" by the paper and pinned here only by exact integer
 * brute force, invariants and special cases).
 * ------------------------------------------------------------------------------------------------ */

/*
 * Max-pooling on int8 codes (the ImageNet networks of Sec. 5.1 pool after the first layer): window
 * k x k, stride s, padding p; padded positions never win.  idx receives the flat NHWC index of the
 * first maximum in (kh, kw) scan order, which is where the backward pass routes the error.
 */
void eoq_o_maxpool_fwd(const int8_t *x, int n, int h, int w, int c, int k, int s, int p, int8_t *y, int64_t *idx)
{
    int ho = out_dim(h, k, s, p), wo = out_dim(w, k, s, p);
    for (int b = 0; b < n; b++)
        for (int oy = 0; oy < ho; oy++)
            for (int ox = 0; ox < wo; ox++)
                for (int ch = 0; ch < c; ch++) {
                    int best = -1000;
                    int64_t arg = -1;
                    for (int kh = 0; kh < k; kh++)
                        for (int kw = 0; kw < k; kw++) {
                            int iy = oy * s + kh - p, ix = ox * s + kw - p;
                            if (iy < 0 || iy >= h || ix < 0 || ix >= w) continue;
                            int64_t i = (((int64_t)b * h + iy) * w + ix) * c + ch;
                            if ((int)x[i] > best) { best = x[i]; arg = i; }
                        }
                    int64_t o = (((int64_t)b * ho + oy) * wo + ox) * c + ch;
                    y[o] = (int8_t)best;
                    idx[o] = arg;
                }
}

/* Backward of max-pooling: every output error code is added at its argmax position (exact sums;
 * overlapping windows may hit one position several times).  S must hold n_in zeros on entry. */
void eoq_o_maxpool_bwd(const int8_t *e, const int64_t *idx, size_t n_out, int64_t *S)
{
    for (size_t o = 0; o < n_out; o++) S[idx[o]] += e[o];
}

/* Global average pooling hands the exact integer sum per (sample, channel) to the float head. */
void eoq_o_avgpool_sum(const int8_t *x, int n, int hw, int c, int64_t *sums)
{
    for (int b = 0; b < n; b++)
        for (int ch = 0; ch < c; ch++) {
            int64_t acc = 0;
            for (int i = 0; i < hw; i++) acc += x[((size_t)b * hw + i) * c + ch];
            sums[(size_t)b * c + ch] = acc;
        }
}

/*
 * Where two error streams meet (block input: branch error a at exponent pa, shortcut error b at pb):
 * both are brought to the smaller exponent p and added exactly, S = a * 2^(pa - p) + b * 2^(pb - p);
 * an operand more than 31 octaves below the other is dropped.  The caller applies Q_e = SQ to S.
 * mask_b (optional, one byte per element) gates operand b (the ReLU derivative at the join).
 */
int eoq_o_join(const int8_t *a, int pa, const int8_t *b, int pb, const uint8_t *mask_b, size_t n, int64_t *S)
{
    int p = pa < pb ? pa : pb;
    int sa = pa - p, sb = pb - p;
    for (size_t i = 0; i < n; i++) {
        int64_t va = a[i];
        int64_t vb = (mask_b && !mask_b[i]) ? 0 : b[i];
        if (sa > 31) S[i] = va;        /* b lies more than 31 octaves below a: dropped, the sum stays at pa */
        else if (sb > 31) S[i] = vb;   /* a dropped, the sum stays at pb */
        else S[i] = va * ((int64_t)1 << sa) + vb * ((int64_t)1 << sb);
    }
    if (sa > 31) return pa;
    if (sb > 31) return pb;
    return p;
}

/*
 * exp(x) in fp32 from fused multiply-adds and an exponent adjustment only, so that any IEEE-754
 * implementation reproduces it bit for bit: x = k ln2 + r with k = nearest integer of x log2(e),
 * r formed with a two-part ln2, e^r by a degree-7 Taylor polynomial in Horner form (|r| <= 0.35),
 * then scaled by 2^k.  Inputs below -87 return 0 (the softmax only sees x <= 0).
 */
float eoq_o_expf(float x)
{
    if (x < -87.0f) return 0.0f;
    if (x > 88.0f) x = 88.0f;
    float kf = rintf(x * 1.44269504088896341f);
    float r = fmaf(-kf, 0.693145751953125f, x);
    r = fmaf(-kf, 1.42860682030941723212e-6f, r);
    float p = 1.0f / 5040.0f;
    p = fmaf(p, r, 1.0f / 720.0f);
    p = fmaf(p, r, 1.0f / 120.0f);
    p = fmaf(p, r, 1.0f / 24.0f);
    p = fmaf(p, r, 1.0f / 6.0f);
    p = fmaf(p, r, 0.5f);
    p = fmaf(p, r, 1.0f);
    p = fmaf(p, r, 1.0f);
    return ldexpf(p, (int)kf);
}

/*
 * The unquantized last layer (Sec. 5.1 keeps it in floating point), written operation by operation
 * in fp32 so that the result does not depend on the machine:
 *   pooled[n,c] = (float)sum[n,c] * 2^-7 / hw
 *   logit[n,j]  = bias[j] + sum over c ascending of fma(W[j,c], pooled[n,c], .)   (one accumulator)
 *   softmax with the maximum subtracted, exp as above, denominator summed over j ascending
 *   dlogit[n,j] = (prob - [j == label]) * (1 / n)       (mean cross-entropy over the batch)
 *   dpooled[n,c] = sum over j ascending of fma(dlogit[n,j], W[j,c], .)          (W before its update)
 *   W[j,c]  <- fma(-lr, sum over n ascending of fma(dlogit[n,j], pooled[n,c], .), W[j,c]); bias alike
 * loss = mean over n of (log(denominator) - (logit[label] - max)), reported only.
 */
void eoq_o_head(const int64_t *sums, int n, int c, int hw, int classes, float *W, float *bias, const int32_t *labels,
                float lr, float *loss_out, float *dpooled, float *logits_out)
{
    float *pooled = (float *)__builtin_malloc(sizeof(float) * (size_t)n * c);
    float *dl = (float *)__builtin_malloc(sizeof(float) * (size_t)n * classes);
    for (size_t i = 0; i < (size_t)n * c; i++) pooled[i] = ((float)sums[i] * 0.0078125f) / (float)hw;
    float inv_n = 1.0f / (float)n;
    double loss = 0.0;
    for (int b = 0; b < n; b++) {
        float *l = dl + (size_t)b * classes;
        for (int j = 0; j < classes; j++) {
            float acc = bias[j];
            for (int k = 0; k < c; k++) acc = fmaf(W[(size_t)j * c + k], pooled[(size_t)b * c + k], acc);
            l[j] = acc;
            if (logits_out) logits_out[(size_t)b * classes + j] = acc;
        }
        float m = l[0];
        for (int j = 1; j < classes; j++) m = l[j] > m ? l[j] : m;
        float den = 0.0f;
        float ly = l[labels[b]] - m;
        for (int j = 0; j < classes; j++) {
            l[j] = eoq_o_expf(l[j] - m);
            den = den + l[j];
        }
        loss += (double)logf(den) - (double)ly;
        for (int j = 0; j < classes; j++) {
            float pr = l[j] / den;
            l[j] = (pr - (j == labels[b] ? 1.0f : 0.0f)) * inv_n;
        }
    }
    *loss_out = (float)(loss / n);
    for (int b = 0; b < n; b++)
        for (int k = 0; k < c; k++) {
            float acc = 0.0f;
            for (int j = 0; j < classes; j++) acc = fmaf(dl[(size_t)b * classes + j], W[(size_t)j * c + k], acc);
            dpooled[(size_t)b * c + k] = acc;
        }
    for (int j = 0; j < classes; j++) {
        for (int k = 0; k < c; k++) {
            float acc = 0.0f;
            for (int b = 0; b < n; b++) acc = fmaf(dl[(size_t)b * classes + j], pooled[(size_t)b * c + k], acc);
            W[(size_t)j * c + k] = fmaf(-lr, acc, W[(size_t)j * c + k]);
        }
        float db = 0.0f;
        for (int b = 0; b < n; b++) db = db + dl[(size_t)b * classes + j];
        bias[j] = fmaf(-lr, db, bias[j]);
    }
    __builtin_free(pooled);
    __builtin_free(dl);
}

/* ------------------------------------------------------------------------------------------------
 * Other bit widths (Sec. 3.2.2 defines Q, CQ and SQ for any k; Sec. 3.2.3 and Sec. 5 compare the 8-bit
 * update with the 24-bit update of earlier integer-training work).
 * ------------------------------------------------------------------------------------------------ */

/* SQ(., k) on integer codes at exponent p_a: code = sat(R(a * 2^(k-1-t)), +-(2^(k-1) - 1)), p_out = p_a + t - (k-1). */
int eoq_o_sq_i64_k(const int64_t *a, size_t n, int p_a, int k, int64_t *codes, int *p_out)
{
    uint64_t M = 0;
    for (size_t i = 0; i < n; i++) {
        uint64_t m = a[i] < 0 ? (uint64_t)(-a[i]) : (uint64_t)a[i];
        if (m > M) M = m;
    }
    if (M == 0) {
        for (size_t i = 0; i < n; i++) codes[i] = 0;
        *p_out = p_a;
        return 1;
    }
    int t = eoq_o_round_log2_u64(M);
    int64_t lim = ((int64_t)1 << (k - 1)) - 1;
    for (size_t i = 0; i < n; i++) codes[i] = sat64(eoq_o_rne_shr(a[i], t - (k - 1)), -lim, lim);
    *p_out = p_a + t - (k - 1);
    return 0;
}

/*
 * The update with an update quantizer of k_u bits and a master copy of the weights on the grid of Q(., k_m):
 *   u = Q_u(lr g) = SQ(lr g, k_u);   theta <- CQ(theta - u, k_m)   (theta: integer codes at exponent -(k_m - 1));
 * the layer then works on w = Q_w(theta) = CQ(theta, 8), i.e. code sat(R(theta / 2^(k_m - 8)), +-127).
 * k_u = k_m = 8 is the paper's 8-bit update (eoq_o_update); k_u = k_m = 24 the wide update it is compared with.
 * Alignment as in eoq_o_update; shifts beyond 38 bits drop the update (below 2^-38 of a master step).
 */
int eoq_o_update_k(int32_t *theta, int8_t *w8, const int8_t *g, int p_g, size_t n, int lr_mant, int lr_exp, int k_u, int k_m,
                   int stochastic, uint64_t seed, uint64_t step, uint64_t tensor_id, int *p_u_out)
{
    int64_t *a = (int64_t *)__builtin_malloc(sizeof(int64_t) * (n ? n : 1));
    int64_t *u = (int64_t *)__builtin_malloc(sizeof(int64_t) * (n ? n : 1));
    for (size_t i = 0; i < n; i++) a[i] = (int64_t)lr_mant * g[i];
    int p_u;
    int z = eoq_o_sq_i64_k(a, n, p_g + lr_exp, k_u, u, &p_u);
    int d = p_u + (k_m - 1);
    int64_t lim = ((int64_t)1 << (k_m - 1)) - 1;
    for (size_t i = 0; i < n; i++) {
        int64_t next;
        if (d >= 0) {
            next = (int64_t)theta[i] - u[i] * ((int64_t)1 << (d > 38 ? 38 : d));
        } else if (-d > 38) {
            next = theta[i];
        } else {
            int s = -d;
            int64_t v = (int64_t)theta[i] * ((int64_t)1 << s) - u[i];
            if (!stochastic) {
                next = eoq_o_rne_shr(v, s);
            } else {
                uint64_t r = eoq_o_update_hash(seed, step, tensor_id, i) & (((uint64_t)1 << s) - 1);
                int64_t rem;
                next = floor_div_pow2(v + (int64_t)r, s, &rem);
            }
        }
        theta[i] = (int32_t)sat64(next, -lim, lim);
        if (w8) w8[i] = (int8_t)sat64(eoq_o_rne_shr(theta[i], k_m - 8), -127, 127);
    }
    *p_u_out = p_u;
    __builtin_free(a);
    __builtin_free(u);
    return z;
}

/* ---------------------------------------------------------------------------------------------
 * Batch normalisation behind the same convolution: the comparison the paper draws in its efficiency
 * discussion (Sec. 5.3, "efficiency comparison of EOQ and traditional BN": the scale-and-bias of
 * the Fixup block against the mean / standard-deviation normalisation of a mini-batch).  Not part
 * of the EOQ method; it exists so that the cost of what EOQ removes can be measured beside it.
 *
 * Definition (training-mode batch normalisation per channel over all n*h*w positions of the batch):
 *   a      = A * 2^p                     the convolution output, exact integers A at exponent p
 *   mean   = sum(a) / P,  var = sum(a^2) / P - mean^2      (biased variance)
 *   y      = gamma * (a - mean) / sqrt(var + eps) + beta,  x5 = Q_a2(relu(y)),  mask = [y > 0]
 * Statistics are exact: S1 = sum A (64-bit), S2 = sum A^2 (128-bit), V = P * S2 - S1^2 (128-bit, >= 0).
 * From there double precision, every operation rounded once, in this order:
 *   mu = (double)S1 / P;  var_a = (hi(V) * 2^64 + lo(V)) / ((double)P * P)   (in units of A);
 *   inv = 1 / sqrt(var_a * 4^p + eps);  k = gamma * inv;  scale = (float)(k * 2^p);
 *   shift = (float)(beta - (k * 2^p) * mu);
 * then one fused multiply-add per element in single precision: y = fma((float)A, scale, shift), and
 * x5 = min(rint(y * 128), 127) for y > 0, else 0.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    double mu;      /* mean in units of A */
    double inv;     /* 1 / sqrt(var + eps), value units */
    float scale, shift;
} eoq_o_bn_channel_t;

static double u128_to_double(unsigned __int128 v)
{
    double hi = (double)(uint64_t)(v >> 64), lo = (double)(uint64_t)v;
    return hi * 18446744073709551616.0 + lo;
}

void eoq_o_bn_forward(const int64_t *A, int p, size_t P, int c, const float *gamma, const float *beta, float eps,
                      int8_t *x5, uint8_t *mask01, float *y_out, eoq_o_bn_channel_t *ch)
{
    for (int k = 0; k < c; k++) {
        int64_t s1 = 0;
        unsigned __int128 s2 = 0;
        for (size_t i = 0; i < P; i++) {
            int64_t a = A[i * c + k];
            s1 += a;
            s2 += (unsigned __int128)((__int128)a * a);
        }
        unsigned __int128 V = (unsigned __int128)P * s2 - (unsigned __int128)((__int128)s1 * s1);
        double Pd = (double)P;
        double mu = (double)s1 / Pd;
        double var_a = u128_to_double(V) / (Pd * Pd);
        double var_v = ldexp(var_a, 2 * p);
        double inv = 1.0 / sqrt(var_v + (double)eps);
        double kk = (double)gamma[k] * inv;
        double ks = ldexp(kk, p);
        ch[k].mu = mu;
        ch[k].inv = inv;
        ch[k].scale = (float)ks;
        ch[k].shift = (float)((double)beta[k] - ks * mu);
    }
    for (size_t i = 0; i < P; i++)
        for (int k = 0; k < c; k++) {
            float y = fmaf((float)A[i * c + k], ch[k].scale, ch[k].shift);
            if (y_out) y_out[i * c + k] = y;
            int pos = y > 0.0f;
            float r = rintf(y * 128.0f);
            x5[i * c + k] = (int8_t)(pos ? (r > 127.0f ? 127 : (int)r) : 0);
            if (mask01) mask01[i * c + k] = (uint8_t)pos;
        }
}

/*
 * Backward of the same normalisation (e: error codes at exponent p_e arriving at x5; the clamp of Q_a2 is
 * passed straight through as everywhere else, so dy = e * mask):
 *   dbeta = sum(dy),  dgamma = sum(dy * xhat),  xhat = (a - mean) * inv
 *   da    = gamma * inv * (dy - mean(dy) - xhat * mean(dy * xhat))
 * Exact sums D1 = sum(E * mask), D2 = sum(E * mask * A) (64-bit), then in double, in this order:
 *   cov = (double)D2 - mu * (double)D1;  g2 = (inv * 2^p) * cov * 2^pe   (= dgamma);  g1 = (double)D1 * 2^pe (= dbeta);
 *   k = gamma * inv;  ca = (float)(k * 2^pe);  m2 = g2 / P;  cb_d = -(k * m2) * (inv * 2^p);  cb = (float)cb_d;
 *   cc = (float)(-(k * (g1 / P)) - cb_d * mu);
 * and per element in single precision da = fma(ca, (float)(E * mask), fma(cb, (float)A, cc)).
 * The caller quantizes da with Q_e (SQ) like every other error tensor.
 */
void eoq_o_bn_backward(const int8_t *E, int p_e, const uint8_t *mask01, const int64_t *A, int p, size_t P, int c,
                       const float *gamma, const eoq_o_bn_channel_t *ch, float *da, float *dgamma, float *dbeta)
{
    float *ca = (float *)__builtin_malloc(sizeof(float) * 3 * (size_t)c), *cb = ca + c, *cc = cb + c;
    for (int k = 0; k < c; k++) {
        int64_t d1 = 0, d2 = 0;
        for (size_t i = 0; i < P; i++) {
            int64_t dy = mask01[i * c + k] ? (int64_t)E[i * c + k] : 0;
            d1 += dy;
            d2 += dy * A[i * c + k];
        }
        double Pd = (double)P;
        double cov = (double)d2 - ch[k].mu * (double)d1;
        double ip = ldexp(ch[k].inv, p);
        double g2 = ldexp(ip * cov, p_e);
        double g1 = ldexp((double)d1, p_e);
        double kk = (double)gamma[k] * ch[k].inv;
        double m2 = g2 / Pd;
        double cb_d = -(kk * m2) * ip;
        ca[k] = (float)ldexp(kk, p_e);
        cb[k] = (float)cb_d;
        cc[k] = (float)(-(kk * (g1 / Pd)) - cb_d * ch[k].mu);
        dgamma[k] = (float)g2;
        dbeta[k] = (float)g1;
    }
    for (size_t i = 0; i < P; i++)
        for (int k = 0; k < c; k++) {
            float dy = mask01[i * c + k] ? (float)E[i * c + k] : 0.0f;
            da[i * c + k] = fmaf(ca[k], dy, fmaf(cb[k], (float)A[i * c + k], cc[k]));
        }
    __builtin_free(ca);
}
