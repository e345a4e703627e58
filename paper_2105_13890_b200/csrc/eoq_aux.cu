// Glue between the quantized convolution units of a Fixup residual network (arXiv 2105.13890, Sec. 3.2.1 chains the
// units: x0 of a layer is x5 of the one before, e0 is the error handed back by its successor): max and average
// pooling on int8 codes, the exact join of two error streams followed by Q_e, the floating-point last layer
// (Sec. 5.1 leaves it unquantized) written operation by operation so that it is reproducible bit for bit, the
// quantized error it hands back, and the update of the scalar parameters (Sec. 3.2.3) on their 16-bit range.
// All of it is bandwidth- or latency-bound support work; none of it touches the tensor cores.
#include "eoq_device.cuh"
#include "eoq_internal.h"
#include "eoq_next_head.cuh"

namespace eoq {

namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ uint32_t pack4(int a, int b, int c, int d)
{
    return (uint32_t)(a & 0xff) | ((uint32_t)(b & 0xff) << 8) | ((uint32_t)(c & 0xff) << 16) | ((uint32_t)(d & 0xff) << 24);
}

inline int blocks_for(size_t items, int sm_count, int per_sm = 8)
{
    size_t b = (items + kThreads - 1) / kThreads, cap = (size_t)sm_count * per_sm;
    if (b > cap) b = cap;
    return b < 1 ? 1 : (int)b;
}

// same protocol as in the elementwise kernels: true in thread 0 of the block that arrives last
__device__ __forceinline__ bool last_block_done(DeviceState *dev)
{
    __shared__ unsigned last_s;
    __syncthreads();
    if (threadIdx.x == 0) {
        __threadfence();
        const unsigned t = atomicAdd(&dev->ticket, 1u);
        last_s = (t == gridDim.x - 1) ? 1u : 0u;
        if (last_s) {
            __threadfence();
            dev->ticket = 0;
        }
    }
    __syncthreads();
    return last_s != 0 && threadIdx.x == 0;
}

// ------------------------------------------------------------------ pooling

// One thread per 16 channels of an output pixel.  arg = kh * k + kw of the first maximum in scan order.
__global__ void maxpool_fwd_kernel(const int8_t *__restrict__ x, int n, int h, int w, int c, int k, int s, int p, int ho, int wo,
                                   int8_t *__restrict__ y, uint8_t *__restrict__ arg)
{
    const int groups = c / 16;
    const size_t items = (size_t)n * ho * wo * groups;
    // (the launcher keeps the item count below 2^32: 64-bit divisions would dominate the work of an item)
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < items; i += (size_t)gridDim.x * blockDim.x) {
        const uint32_t i32 = (uint32_t)i, pix = i32 / (uint32_t)groups, row = pix / (uint32_t)wo;
        const int g = (int)(i32 - pix * (uint32_t)groups), ox = (int)(pix - row * (uint32_t)wo);
        const int b = (int)(row / (uint32_t)ho), oy = (int)(row - (uint32_t)b * (uint32_t)ho);
        int best[16], at[16];
#pragma unroll
        for (int q = 0; q < 16; ++q) { best[q] = -1000; at[q] = 0; }
        for (int kh = 0; kh < k; ++kh) {
            const int iy = oy * s + kh - p;
            if (iy < 0 || iy >= h) continue;
            for (int kw = 0; kw < k; ++kw) {
                const int ix = ox * s + kw - p;
                if (ix < 0 || ix >= w) continue;
                const int4 v = __ldg(reinterpret_cast<const int4 *>(x + (((size_t)b * h + iy) * w + ix) * c + g * 16));
                const int8_t *e = reinterpret_cast<const int8_t *>(&v);
#pragma unroll
                for (int q = 0; q < 16; ++q)
                    if ((int)e[q] > best[q]) { best[q] = e[q]; at[q] = kh * k + kw; }
            }
        }
        reinterpret_cast<int4 *>(y)[i] = make_int4((int)pack4(best[0], best[1], best[2], best[3]), (int)pack4(best[4], best[5], best[6], best[7]),
                                                    (int)pack4(best[8], best[9], best[10], best[11]), (int)pack4(best[12], best[13], best[14], best[15]));
        reinterpret_cast<int4 *>(arg)[i] = make_int4((int)pack4(at[0], at[1], at[2], at[3]), (int)pack4(at[4], at[5], at[6], at[7]),
                                                      (int)pack4(at[8], at[9], at[10], at[11]), (int)pack4(at[12], at[13], at[14], at[15]));
    }
}

// Backward: every output error code is added at the input position its window elected; the exact sums are then
// coded with Q_e, which needs their maximum over the whole tensor first.  So the kernel runs twice: pass 0 reduces
// max |sum| into the handle's cell, pass 1 forms the sums again and codes them (no intermediate tensor is written).
// One thread per 16 channels of an input position gathers from the windows that cover it (at most
// ceil(k / stride)^2): a window's 16 codes count where its recorded position equals this one.  Four codes are
// handled per 32-bit word: bytes are compared at once, the chosen codes are kept with an offset of 128 (others as
// 128 itself) so that they add as unsigned halves of two words without carries between them.
//
// kNext: the consumer's error head rides along (the layer in front of the pool: e1 = e_in * [x4 > 0],
// e3 = Q_e(gamma * e1), sum of e1).  Coding is monotonic in |sum|, so max |e1| is the code of the largest masked
// |sum|: pass 0 reduces that second maximum as well (into the 64-bit cell), and pass 1 knows both scales, writes
// e_in (optional) and e3 and adds up e1 - the two kernels of a separate error head and their pass over e_in are gone.
template <int kPass, bool kNext>
__global__ void __launch_bounds__(kThreads)
maxpool_bwd_kernel(const int8_t *__restrict__ e, const int32_t *e_exp, const uint8_t *__restrict__ arg, int n, int h, int w, int c,
                   int k, int s, int p, int ho, int wo, int8_t *__restrict__ e_in, int32_t *e_in_exp,
                   const uint8_t *__restrict__ next_mask, const int32_t *next_gamma, int8_t *__restrict__ e3, int32_t *e3_exp,
                   long long *sum_e1, DeviceState *dev)
{
    const int groups = c / 16;
    const uint32_t items = (uint32_t)n * h * w * groups;   // below 2^31 (checked by the caller), so i + stride cannot wrap
    int t = 7;
    NextHead nh = {};
    if (kPass == 1) {
        const uint32_t M = dev->absmax_u32;
        t = M ? round_log2_u32(M) : 7;
        const int p_in = *e_exp;
        const int p0 = M ? p_in + t - 7 : p_in;
        if (kNext) nh = next_head_setup(next_gamma, (uint32_t)abs(sq_code32((int32_t)dev->absmax_u64, t)), dev);
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            if (e_in_exp) *e_in_exp = p0;
            if (!M) atomicOr(&dev->status, EOQ_DEV_SQ_ZERO);
            if (kNext) next_head_exponent(nh, p0, e3_exp, dev);
        }
    }
    uint32_t mx = 0, mx_masked = 0;
    int s1 = 0;
    long long s1_total = 0;
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < items; i += gridDim.x * blockDim.x) {
        const uint32_t pix = i / (uint32_t)groups, row = pix / (uint32_t)w;
        const int gi = (int)(i - pix * (uint32_t)groups), ix = (int)(pix - row * (uint32_t)w);
        const int b = (int)(row / (uint32_t)h), iy = (int)(row - (uint32_t)b * (uint32_t)h);
        // windows o with o * s - p <= i <= o * s - p + k - 1
        const int oy_lo = max(0, (iy + p - k + s) / s), oy_hi = min(ho - 1, (iy + p) / s);
        const int ox_lo = max(0, (ix + p - k + s) / s), ox_hi = min(wo - 1, (ix + p) / s);
        uint32_t even[4] = {0, 0, 0, 0}, odd[4] = {0, 0, 0, 0};
        int nwin = 0;
        auto take = [&](const int4 &ev, const int4 &av, int oy, int ox) {
            const uint32_t me = (uint32_t)((iy - (oy * s - p)) * k + (ix - (ox * s - p))) * 0x01010101u;
            const uint32_t ew[4] = {(uint32_t)ev.x, (uint32_t)ev.y, (uint32_t)ev.z, (uint32_t)ev.w};
            const uint32_t aw[4] = {(uint32_t)av.x, (uint32_t)av.y, (uint32_t)av.z, (uint32_t)av.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint32_t hit = __vcmpeq4(aw[q], me);           // 0xff in the bytes this position won
                const uint32_t v = (ew[q] & hit) ^ 0x80808080u;      // code + 128 there, 128 elsewhere
                even[q] += v & 0x00ff00ffu;
                odd[q] += (v >> 8) & 0x00ff00ffu;
            }
            ++nwin;
        };
        if (oy_hi - oy_lo <= 1 && ox_hi - ox_lo <= 1) {
            // the usual case (window at most twice the stride): at most 2 x 2 windows, all eight loads issued together
            int4 ev[4], av[4];
            bool in[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const int oy = oy_lo + (u >> 1), ox = ox_lo + (u & 1);
                in[u] = oy <= oy_hi && ox <= ox_hi;
                const size_t o = (((size_t)b * ho + oy) * wo + ox) * c + gi * 16;
                ev[u] = in[u] ? __ldg(reinterpret_cast<const int4 *>(e + o)) : make_int4(0, 0, 0, 0);
                av[u] = in[u] ? __ldg(reinterpret_cast<const int4 *>(arg + o)) : make_int4(0, 0, 0, 0);
            }
#pragma unroll
            for (int u = 0; u < 4; ++u)
                if (in[u]) take(ev[u], av[u], oy_lo + (u >> 1), ox_lo + (u & 1));
        } else {
            for (int oy = oy_lo; oy <= oy_hi; ++oy)
                for (int ox = ox_lo; ox <= ox_hi; ++ox) {
                    const size_t o = (((size_t)b * ho + oy) * wo + ox) * c + gi * 16;
                    take(__ldg(reinterpret_cast<const int4 *>(e + o)), __ldg(reinterpret_cast<const int4 *>(arg + o)), oy, ox);
                }
        }
        int sum[16];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            sum[4 * q + 0] = (int)(even[q] & 0xffffu) - 128 * nwin;
            sum[4 * q + 1] = (int)(odd[q] & 0xffffu) - 128 * nwin;
            sum[4 * q + 2] = (int)(even[q] >> 16) - 128 * nwin;
            sum[4 * q + 3] = (int)(odd[q] >> 16) - 128 * nwin;
        }
        const uint32_t mbits = kNext ? (uint32_t)__ldg(reinterpret_cast<const uint16_t *>(next_mask) + i) : 0u;
        if (kPass == 0) {
#pragma unroll
            for (int q = 0; q < 16; ++q) {
                const uint32_t v = (uint32_t)abs(sum[q]);
                mx = max(mx, v);
                if (kNext && ((mbits >> q) & 1u)) mx_masked = max(mx_masked, v);
            }
        } else {
            int cd[16];
            if (t >= 8) {   // a right shift by t - 7 >= 1 (sums are below 2^15, nothing can wrap)
                const int sh = t - 7, half_m1 = (1 << (sh - 1)) - 1;
#pragma unroll
                for (int q = 0; q < 16; ++q) cd[q] = sq_code32_shr(sum[q], sh, half_m1);
            } else {
#pragma unroll
                for (int q = 0; q < 16; ++q) cd[q] = sq_code32(sum[q], t);
            }
            if (e_in)
                reinterpret_cast<int4 *>(e_in)[i] =
                    make_int4((int)pack4(cd[0], cd[1], cd[2], cd[3]), (int)pack4(cd[4], cd[5], cd[6], cd[7]),
                              (int)pack4(cd[8], cd[9], cd[10], cd[11]), (int)pack4(cd[12], cd[13], cd[14], cd[15]));
            if (kNext) {
                int c3[16];
#pragma unroll
                for (int q = 0; q < 16; ++q) {
                    const int e1 = ((mbits >> q) & 1u) ? cd[q] : 0;
                    s1 += e1;
                    c3[q] = next_head_code(nh, e1);
                }
                reinterpret_cast<int4 *>(e3)[i] =
                    make_int4((int)pack4(c3[0], c3[1], c3[2], c3[3]), (int)pack4(c3[4], c3[5], c3[6], c3[7]),
                              (int)pack4(c3[8], c3[9], c3[10], c3[11]), (int)pack4(c3[12], c3[13], c3[14], c3[15]));
                s1_total += s1;
                s1 = 0;
            }
        }
    }
    if (kPass == 0) {
        mx = (uint32_t)block_max_u64(mx);
        if (kNext) mx_masked = (uint32_t)block_max_u64(mx_masked);
        if (threadIdx.x == 0) {
            if (mx) atomicMax(&dev->absmax_u32, mx);
            if (kNext && mx_masked) atomicMax(&dev->absmax_u64, (unsigned long long)mx_masked);
        }
    } else {
        if (kNext && sum_e1) {
            s1_total = block_sum_i64(s1_total);
            if (threadIdx.x == 0 && s1_total) atomicAdd(reinterpret_cast<unsigned long long *>(&dev->sum0), (unsigned long long)s1_total);
        }
        if (last_block_done(dev)) {
            dev->absmax_u32 = 0;
            if (kNext) {
                dev->absmax_u64 = 0;
                if (sum_e1) *sum_e1 = (long long)atomicExch(reinterpret_cast<unsigned long long *>(&dev->sum0), 0ull);
            }
        }
    }
}

// sums[b][ch] = sum over the hw positions of x[b][.][ch]; one block per (sample, 16-channel group)
__global__ void avgpool_sum_kernel(const int8_t *__restrict__ x, int hw, int c, int32_t *__restrict__ sums)
{
    __shared__ int part[kThreads][17];
    const int groups = c / 16, b = blockIdx.x / groups, g = blockIdx.x % groups;
    int acc[16];
#pragma unroll
    for (int q = 0; q < 16; ++q) acc[q] = 0;
    for (int i = threadIdx.x; i < hw; i += blockDim.x) {
        const int4 v = __ldg(reinterpret_cast<const int4 *>(x + ((size_t)b * hw + i) * c + g * 16));
        const int8_t *e = reinterpret_cast<const int8_t *>(&v);
#pragma unroll
        for (int q = 0; q < 16; ++q) acc[q] += e[q];
    }
#pragma unroll
    for (int q = 0; q < 16; ++q) part[threadIdx.x][q] = acc[q];
    __syncthreads();
    if (threadIdx.x < 16) {
        int t = 0;
        for (int i = 0; i < (int)blockDim.x; ++i) t += part[i][threadIdx.x];
        sums[(size_t)b * c + g * 16 + threadIdx.x] = t;
    }
}

// ------------------------------------------------------------------ join of two error streams + Q_e

__device__ __forceinline__ void unpack16(const int4 &v, int (&o)[16])
{
    const int8_t *b = reinterpret_cast<const int8_t *>(&v);
#pragma unroll
    for (int k = 0; k < 16; ++k) o[k] = b[k];
}

// pass = 0: max |S| into the handle's 64-bit cell; pass = 1: codes of SQ(S), their sum, exponent; cells back to zero.
// kNext: the error head of the layer that consumes the joined error rides along (see NextHead): pass 0 also reduces
// the maximum over the positions that layer's ReLU lets through, pass 1 also writes that layer's e3 and its two sums.
template <int kPass, bool kNext>
__global__ void join_kernel(const int8_t *__restrict__ a, const int32_t *a_exp, const int8_t *__restrict__ b, const int32_t *b_exp,
                            const uint8_t *__restrict__ mask_b, size_t n16, int8_t *out, int32_t *out_exp, long long *sum_out,
                            const uint8_t *__restrict__ next_mask, const int16_t *__restrict__ next_x2, const int32_t *next_gamma,
                            int8_t *__restrict__ e3, int32_t *e3_exp, long long *sum_e1, long long *sum_e1x2, DeviceState *dev)
{
    const JoinShift j = join_shift(__ldg(a_exp), __ldg(b_exp));
    unsigned long long mx = 0, mxm = 0;
    long long sum = 0, s1 = 0, s2 = 0;
    int t = 7;
    NextHead nh = {};
    if (kPass == 1) {
        const unsigned long long M = dev->absmax_u64;
        t = M ? round_log2_u64(M) : 7;
        const int p0 = M ? j.p + t - 7 : j.p;
        if (kNext) {
            const unsigned long long Mm = dev->absmax2_u64;
            nh = next_head_setup(next_gamma, (uint32_t)abs(sq_code64((long long)Mm, t)), dev);
        }
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            *out_exp = p0;
            if (!M) atomicOr(&dev->status, EOQ_DEV_SQ_ZERO);
            if (kNext) next_head_exponent(nh, p0, e3_exp, dev);
        }
    }
    // exponents a few octaves apart (the usual case) keep every sum inside 32 bits: 127 * 2^23 + 127 < 2^31
    const bool narrow = j.sa >= 0 && j.sb >= 0 && j.sa <= 23 && j.sb <= 23;
    const int ma = 1 << (j.sa < 0 ? 0 : min(j.sa, 23)), mb = 1 << (j.sb < 0 ? 0 : min(j.sb, 23));
    uint32_t mx32 = 0, mxm32 = 0;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (size_t)gridDim.x * blockDim.x) {
        int av[16], bv[16];
        unpack16(__ldg(reinterpret_cast<const int4 *>(a) + i), av);
        unpack16(__ldg(reinterpret_cast<const int4 *>(b) + i), bv);
        const uint32_t m = mask_b ? (uint32_t)__ldg(reinterpret_cast<const uint16_t *>(mask_b) + i) : 0xffffu;
        const uint32_t nm = kNext ? (uint32_t)__ldg(reinterpret_cast<const uint16_t *>(next_mask) + i) : 0u;
        int c[16];
        if (narrow) {
#pragma unroll
            for (int q = 0; q < 16; ++q) {
                const int s32 = av[q] * ma + (((m >> q) & 1u) ? bv[q] : 0) * mb;
                if (kPass == 0) {
                    const uint32_t v = (uint32_t)abs(s32);
                    mx32 = max(mx32, v);
                    if (kNext && ((nm >> q) & 1u)) mxm32 = max(mxm32, v);
                } else {
                    c[q] = sq_code32(s32, t);
                }
            }
        } else {
#pragma unroll
            for (int q = 0; q < 16; ++q) {
                const long long s = join_one(av[q], ((m >> q) & 1u) ? bv[q] : 0, j);
                if (kPass == 0) {
                    const unsigned long long u = (unsigned long long)(s < 0 ? -s : s);
                    mx = u > mx ? u : mx;
                    if (kNext && ((nm >> q) & 1u)) mxm = u > mxm ? u : mxm;
                } else {
                    c[q] = sq_code64(s, t);
                }
            }
        }
        if (kPass == 1) {
            int sum32 = 0;
#pragma unroll
            for (int q = 0; q < 16; ++q) sum32 += c[q];
            sum += sum32;
            reinterpret_cast<int4 *>(out)[i] = make_int4((int)pack4(c[0], c[1], c[2], c[3]), (int)pack4(c[4], c[5], c[6], c[7]),
                                                          (int)pack4(c[8], c[9], c[10], c[11]), (int)pack4(c[12], c[13], c[14], c[15]));
            if (kNext) {
                int e1[16], c3[16], a1 = 0;
#pragma unroll
                for (int q = 0; q < 16; ++q) {
                    e1[q] = ((nm >> q) & 1u) ? c[q] : 0;
                    a1 += e1[q];
                    c3[q] = next_head_code(nh, e1[q]);
                }
                s1 += a1;
                if (next_x2) {
                    const int4 lo = __ldg(reinterpret_cast<const int4 *>(next_x2) + 2 * i);
                    const int4 hi = __ldg(reinterpret_cast<const int4 *>(next_x2) + 2 * i + 1);
                    const int16_t *pl = reinterpret_cast<const int16_t *>(&lo), *ph = reinterpret_cast<const int16_t *>(&hi);
                    int a2 = 0;  // |e1 * x2| < 2^22, 16 terms
#pragma unroll
                    for (int q = 0; q < 8; ++q) a2 += e1[q] * pl[q] + e1[8 + q] * ph[q];
                    s2 += a2;
                }
                reinterpret_cast<int4 *>(e3)[i] =
                    make_int4((int)pack4(c3[0], c3[1], c3[2], c3[3]), (int)pack4(c3[4], c3[5], c3[6], c3[7]),
                              (int)pack4(c3[8], c3[9], c3[10], c3[11]), (int)pack4(c3[12], c3[13], c3[14], c3[15]));
            }
        }
    }
    if (kPass == 0) {
        mx = block_max_u64(mx > mx32 ? mx : (unsigned long long)mx32);
        if (kNext) mxm = block_max_u64(mxm > mxm32 ? mxm : (unsigned long long)mxm32);
        if (threadIdx.x == 0) {
            if (mx) atomicMax(&dev->absmax_u64, mx);
            if (kNext && mxm) atomicMax(&dev->absmax2_u64, mxm);
        }
    } else {
        if (sum_out) {
            sum = block_sum_i64(sum);
            if (threadIdx.x == 0 && sum) atomicAdd(reinterpret_cast<unsigned long long *>(&dev->sum0), (unsigned long long)sum);
        }
        if (kNext) {
            s1 = block_sum_i64(s1);
            s2 = block_sum_i64(s2);
            if (threadIdx.x == 0) {
                if (s1) atomicAdd(reinterpret_cast<unsigned long long *>(&dev->sum1), (unsigned long long)s1);
                if (s2) atomicAdd(reinterpret_cast<unsigned long long *>(&dev->sum2), (unsigned long long)s2);
            }
        }
        if (last_block_done(dev)) {
            if (sum_out) *sum_out = (long long)atomicExch(reinterpret_cast<unsigned long long *>(&dev->sum0), 0ull);
            dev->absmax_u64 = 0;
            if (kNext) {
                dev->absmax2_u64 = 0;
                const long long t1 = (long long)atomicExch(reinterpret_cast<unsigned long long *>(&dev->sum1), 0ull);
                const long long t2 = (long long)atomicExch(reinterpret_cast<unsigned long long *>(&dev->sum2), 0ull);
                if (sum_e1) *sum_e1 = t1;
                if (sum_e1x2) *sum_e1x2 = t2;
            }
        }
    }
}

// ------------------------------------------------------------------ the floating-point last layer

// exp(x) from fused multiply-adds and a power-of-two scaling only (x <= 88): x = k ln2 + r, degree-7 polynomial
__device__ __forceinline__ float exp_fma(float x)
{
    if (x < -87.0f) return 0.0f;
    if (x > 88.0f) x = 88.0f;
    const float kf = rintf(__fmul_rn(x, 1.44269504088896341f));
    float r = __fmaf_rn(-kf, 0.693145751953125f, x);
    r = __fmaf_rn(-kf, 1.42860682030941723212e-6f, r);
    float p = 1.0f / 5040.0f;
    p = __fmaf_rn(p, r, 1.0f / 720.0f);
    p = __fmaf_rn(p, r, 1.0f / 120.0f);
    p = __fmaf_rn(p, r, 1.0f / 24.0f);
    p = __fmaf_rn(p, r, 1.0f / 6.0f);
    p = __fmaf_rn(p, r, 0.5f);
    p = __fmaf_rn(p, r, 1.0f);
    p = __fmaf_rn(p, r, 1.0f);
    // 2^k with k in [-126, 127] is a normal number and the product is exact short of underflow, which x >= -87 excludes;
    // p < 2 and k = 127 only for x close to 88, where p * 2^127 stays finite
    return __fmul_rn(p, __int_as_float(((int)kf + 127) << 23));
}

// pooled[b][k] = (float)sum * 2^-7 / hw
__global__ void head_pooled_kernel(const int32_t *__restrict__ sums, int count, int hw, float *pooled)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < count) pooled[i] = __fdiv_rn(__fmul_rn(__int2float_rn(sums[i]), 0.0078125f), (float)hw);
}

// logits[b][j] = bias[j] + sum_k fma(W[j][k], pooled[b][k], .), k ascending into one accumulator per (b, j).
// A warp owns one class j and 32 samples (one per lane), so all lanes walk k together: 32 consecutive weights are
// loaded by the warp at once and handed round by shuffle, the pooled activations of the 32 samples sit in shared
// memory as [k][sample].  Every (b, j) still sees its own strictly sequential chain of fused multiply-adds.
constexpr int kHeadWarps = 8;
__global__ void head_logits_kernel(const float *__restrict__ pooled, int n, int c, int classes, const float *__restrict__ W,
                                   const float *__restrict__ bias, float *logits)
{
    extern __shared__ float ps[];  // [c][33]: row k holds the 32 samples' activations (padded: the fill walks k, the chains walk samples)
    const int b0 = blockIdx.y * 32, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < c * 32; i += blockDim.x) {
        const int sb = i / c, k = i - sb * c;   // consecutive threads read consecutive k of one sample
        ps[k * 33 + sb] = (b0 + sb < n) ? pooled[(size_t)(b0 + sb) * c + k] : 0.0f;
    }
    __syncthreads();
    const int j = blockIdx.x * kHeadWarps + warp;
    if (j >= classes) return;
    float acc = bias[j];
    const float *wj = W + (size_t)j * c;
    float wnext = lane < c ? __ldg(wj + lane) : 0.0f;
    for (int k0 = 0; k0 < c; k0 += 32) {
        const float wreg = wnext;
        if (k0 + 32 < c) wnext = (k0 + 32 + lane < c) ? __ldg(wj + k0 + 32 + lane) : 0.0f;   // the next 32 weights travel meanwhile
        const int kn = min(32, c - k0);
        if (kn == 32) {
#pragma unroll
            for (int kk = 0; kk < 32; ++kk) acc = __fmaf_rn(__shfl_sync(0xffffffffu, wreg, kk), ps[(k0 + kk) * 33 + lane], acc);
        } else {
            for (int kk = 0; kk < kn; ++kk) acc = __fmaf_rn(__shfl_sync(0xffffffffu, wreg, kk), ps[(k0 + kk) * 33 + lane], acc);
        }
    }
    if (b0 + lane < n) logits[(size_t)(b0 + lane) * classes + j] = acc;
}

// One block per sample: softmax with the maximum subtracted, the gradient of the mean cross-entropy with respect to
// the logits, the sample's loss.  The exponentials are formed in parallel; the denominator is then summed by one
// thread over j ascending into one accumulator, which is the order that makes the result reproducible.
__global__ void head_softmax_kernel(const float *__restrict__ logits, int n, int classes, const int32_t *__restrict__ labels, float *dl,
                                    double *loss_n)
{
    __shared__ float red[32];
    __shared__ float m_s, den_s;
    const int b = blockIdx.x;
    const float *l = logits + (size_t)b * classes;
    float *d = dl + (size_t)b * classes;
    float m = -3.4e38f;
    for (int j = threadIdx.x; j < classes; j += blockDim.x) m = l[j] > m ? l[j] : m;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float other = __shfl_xor_sync(0xffffffffu, m, o);
        m = other > m ? other : m;
    }
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        float mm = red[0];
        for (int i = 1; i < (int)(blockDim.x >> 5); ++i) mm = red[i] > mm ? red[i] : mm;
        m_s = mm;
    }
    __syncthreads();
    m = m_s;
    for (int j = threadIdx.x; j < classes; j += blockDim.x) d[j] = exp_fma(__fsub_rn(l[j], m));
    __syncthreads();
    const int y = labels[b];
    if (threadIdx.x == 0) {
        float den = 0.0f;
        for (int j = 0; j < classes; ++j) den = __fadd_rn(den, d[j]);
        den_s = den;
        loss_n[b] = (double)logf(den) - (double)__fsub_rn(l[y], m);
    }
    __syncthreads();
    const float den = den_s, inv_n = __fdiv_rn(1.0f, (float)n);
    for (int j = threadIdx.x; j < classes; j += blockDim.x) {
        const float pr = __fdiv_rn(d[j], den);
        d[j] = __fmul_rn(__fsub_rn(pr, j == y ? 1.0f : 0.0f), inv_n);
    }
}

// dpooled[b][k] = sum_j fma(dl[b][j], W[j][k], .), j ascending (W before its update); one thread also forms the mean loss.
// Every output is one chain of `classes` dependent multiply-adds, so the only parallelism is across outputs (n * c of
// them) and the only thing to hide is the memory traffic: a block owns kDpCh channels x kDpN samples, all its threads
// fetch the next kDpK rows of W (and of dl) together into registers while the chains run on the current rows in
// shared memory.
constexpr int kDpCh = 64, kDpN = 4, kDpK = 32;
__global__ void __launch_bounds__(kDpCh *kDpN)
head_dpooled_kernel(const float *__restrict__ dl, const float *__restrict__ W, int n, int c, int classes, float *dpooled,
                    const double *loss_n, float *loss_out)
{
    __shared__ float w_s[2][kDpK][kDpCh];
    __shared__ float d_s[2][kDpN][kDpK];
    if (blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0 && loss_out) {
        double s = 0.0;
        for (int b = 0; b < n; ++b) s += loss_n[b];
        *loss_out = (float)(s / n);
    }
    const int cl = threadIdx.x % kDpCh, nl = threadIdx.x / kDpCh;
    const int k = blockIdx.x * kDpCh + cl, b = blockIdx.y * kDpN + nl;
    const bool kin = k < c;
    constexpr int kRowsPerThread = kDpK / kDpN;   // rows of the W tile one thread fetches
    float wr[kRowsPerThread], dr = 0.0f;
    auto fetch = [&](int j0) {
#pragma unroll
        for (int r = 0; r < kRowsPerThread; ++r) {
            const int j = j0 + nl + r * kDpN;
            wr[r] = (kin && j < classes) ? __ldg(W + (size_t)j * c + k) : 0.0f;
        }
        if (threadIdx.x < kDpN * kDpK) {
            const int bb = blockIdx.y * kDpN + threadIdx.x / kDpK, j = j0 + threadIdx.x % kDpK;
            dr = (bb < n && j < classes) ? __ldg(dl + (size_t)bb * classes + j) : 0.0f;
        }
    };
    auto stash = [&](int buf) {
#pragma unroll
        for (int r = 0; r < kRowsPerThread; ++r) w_s[buf][nl + r * kDpN][cl] = wr[r];
        if (threadIdx.x < kDpN * kDpK) d_s[buf][threadIdx.x / kDpK][threadIdx.x % kDpK] = dr;
    };
    fetch(0);
    stash(0);
    __syncthreads();
    float acc = 0.0f;
    int buf = 0;
    for (int j0 = 0; j0 < classes; j0 += kDpK, buf ^= 1) {
        const bool more = j0 + kDpK < classes;
        if (more) fetch(j0 + kDpK);
        const int len = min(kDpK, classes - j0);
        if (len == kDpK) {
#pragma unroll
            for (int jj = 0; jj < kDpK; ++jj) acc = __fmaf_rn(d_s[buf][nl][jj], w_s[buf][jj][cl], acc);
        } else {
            for (int jj = 0; jj < len; ++jj) acc = __fmaf_rn(d_s[buf][nl][jj], w_s[buf][jj][cl], acc);
        }
        if (more) stash(buf ^ 1);
        __syncthreads();
    }
    if (kin && b < n) dpooled[(size_t)b * c + k] = acc;
}

// W[j][k] <- fma(-lr, sum_b fma(dl[b][j], pooled[b][k], .), W[j][k]), b ascending; bias[j] alike (thread k == 0)
__global__ void head_update_kernel(const float *__restrict__ dl, const float *__restrict__ pooled, int n, int c, int classes, float lr,
                                   float *W, float *bias)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= classes * c) return;
    const int j = i / c, k = i % c;
    float acc = 0.0f;
    int b = 0;
    for (; b + 8 <= n; b += 8) {
        float d8[8], p8[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            d8[u] = __ldg(dl + (size_t)(b + u) * classes + j);
            p8[u] = __ldg(pooled + (size_t)(b + u) * c + k);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) acc = __fmaf_rn(d8[u], p8[u], acc);
    }
    for (; b < n; ++b) acc = __fmaf_rn(__ldg(dl + (size_t)b * classes + j), __ldg(pooled + (size_t)b * c + k), acc);
    W[i] = __fmaf_rn(-lr, acc, W[i]);
    if (k == 0) {
        float db = 0.0f;
        for (int b = 0; b < n; ++b) db = __fadd_rn(db, dl[(size_t)b * classes + j]);
        bias[j] = __fmaf_rn(-lr, db, bias[j]);
    }
}

// ------------------------------------------------------------------ error handed back by the head

// ef[i] = dpooled[i] / hw and max |ef| (as float bit patterns) into the handle's cell
__global__ void head_error_scale_kernel(const float *__restrict__ dpooled, int count, int hw, float *ef, DeviceState *dev)
{
    uint32_t mx = 0;
    bool bad = false;
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < count; i += gridDim.x * blockDim.x) {
        const float v = __fdiv_rn(dpooled[i], (float)hw);
        ef[i] = v;
        const uint32_t a = __float_as_uint(v) & 0x7fffffffu;
        bad |= a >= 0x7f800000u;
        mx = max(mx, a);
    }
    mx = (uint32_t)block_max_u64(mx);
    bad = __syncthreads_or(bad);
    if (threadIdx.x == 0) {
        if (mx) atomicMax(&dev->absmax_u32, mx);
        if (bad) atomicOr(&dev->status, EOQ_DEV_NONFINITE);
    }
}

__device__ __forceinline__ int round_log2_f32bits_aux(uint32_t bits)
{
    const int eb = (int)((bits >> 23) & 0xffu);
    const uint32_t frac = bits & 0x7fffffu;
    if (eb == 0) return round_log2_u32(frac) - 149;
    const unsigned long long m = (1ull << 23) | frac;
    return (eb - 127) + ((m * m >= (1ull << 47)) ? 1 : 0);
}

// e[b][pos][ch] = SQ code of ef[b][ch] for every position; one thread per 16 channels of a pixel
__global__ void head_error_spread_kernel(const float *__restrict__ ef, int n, int hw, int c, int8_t *e, int32_t *e_exp, DeviceState *dev)
{
    const uint32_t mbits = dev->absmax_u32;
    const bool usable = mbits != 0 && mbits < 0x7f800000u;
    const int up = usable ? 7 - round_log2_f32bits_aux(mbits) : 7;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        *e_exp = usable ? -up : -7;
        if (mbits == 0) atomicOr(&dev->status, EOQ_DEV_SQ_ZERO);
    }
    const int groups = c / 16;
    const size_t items = (size_t)n * hw * groups;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < items; i += (size_t)gridDim.x * blockDim.x) {
        const int g = (int)(i % groups), b = (int)(i / ((size_t)groups * hw));
        const float *src = ef + (size_t)b * c + g * 16;
        int q[16];
#pragma unroll
        for (int k = 0; k < 16; ++k) {
            const float y = scalbnf(__ldg(src + k), up);
            q[k] = (fabsf(y) < 1.0e9f) ? clampi(__float2int_rn(y), -127, 127) : (y > 0.f ? 127 : (y < 0.f ? -127 : 0));
        }
        reinterpret_cast<int4 *>(e)[i] = make_int4((int)pack4(q[0], q[1], q[2], q[3]), (int)pack4(q[4], q[5], q[6], q[7]),
                                                    (int)pack4(q[8], q[9], q[10], q[11]), (int)pack4(q[12], q[13], q[14], q[15]));
    }
    if (last_block_done(dev)) dev->absmax_u32 = 0;
}

// ------------------------------------------------------------------ scalar parameters (Sec. 3.2.3 on a single value)

__device__ __forceinline__ unsigned long long mix64_aux(unsigned long long z)
{
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// One thread per scalar: g = Q_g({total}) (SQ of a single value), u = Q_u(lr g), theta <- Q(theta - u) saturated to 16 bits.
__global__ void scalar_update_kernel(const __grid_constant__ ScalarBatch b, int32_t lr_mant, int32_t lr_exp, int stochastic,
                                     unsigned long long seed, const unsigned long long *step_dev, unsigned long long step)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= b.num) return;
    const ScalarItem &it = b.item[i];
    if (step_dev) step = *step_dev;
    const long long total = *it.total;
    const int p_total = *it.exp + it.exp_bias;
    int g = 0, pg = p_total;
    if (total != 0) {
        const unsigned long long M = (unsigned long long)(total < 0 ? -total : total);
        const int t = round_log2_u64(M);
        g = sq_code64(total, t);
        pg = p_total + t - 7;
    }
    if (it.grad_out) { it.grad_out[0] = g; it.grad_out[1] = pg; }
    int theta = *it.theta;
    if (g != 0) {
        const int a = lr_mant * g;  // |a| < 2^15
        const int tu = round_log2_u32((uint32_t)abs(a));
        const int u = sq_code32(a, tu);
        const int d = (pg + lr_exp + tu - 7) + 7;  // exponent of u relative to the grid 2^-7
        long long next;
        if (d >= 0) {
            next = (long long)theta - (long long)u * (1ll << min(d, 40));
        } else if (-d > 40) {
            next = theta;
        } else {
            const int s = -d;
            const long long v = (long long)theta * (1ll << s) - u;
            if (!stochastic) {
                next = rne_shr64(v, s);
            } else {
                unsigned long long key = mix64_aux(seed + 0x9E3779B97F4A7C15ull * (step + 1));
                key = mix64_aux(key + 0x9E3779B97F4A7C15ull * ((unsigned long long)it.tensor_id + 1));
                const unsigned long long r = mix64_aux(key + 0x9E3779B97F4A7C15ull) & ((1ull << s) - 1ull);  // element index 0
                next = (v + (long long)r) >> s;
            }
        }
        theta = (int)(next < -32768 ? -32768 : (next > 32767 ? 32767 : next));
    }
    *it.theta = theta;
    if (it.mirror) *it.mirror = theta;
}

}  // namespace

// ------------------------------------------------------------------ launchers

cudaError_t launch_maxpool_fwd(const int8_t *x, int n, int h, int w, int c, int k, int s, int p, int8_t *y, uint8_t *arg,
                               int sm_count, cudaStream_t st)
{
    const int ho = (h + 2 * p - k) / s + 1, wo = (w + 2 * p - k) / s + 1;
    maxpool_fwd_kernel<<<blocks_for((size_t)n * ho * wo * (c / 16), sm_count), kThreads, 0, st>>>(x, n, h, w, c, k, s, p, ho, wo, y, arg);
    return cudaGetLastError();
}

cudaError_t launch_maxpool_bwd(const int8_t *e, const int32_t *e_exp, const uint8_t *arg, int n, int h, int w, int c, int k, int s,
                               int p, int8_t *e_in, int32_t *e_in_exp, const uint8_t *next_mask, const int32_t *next_gamma, int8_t *e3,
                               int32_t *e3_exp, long long *sum_e1, DeviceState *dev, int sm_count, cudaStream_t st,
                               const ReduceHook &hook)
{
    const int ho = (h + 2 * p - k) / s + 1, wo = (w + 2 * p - k) / s + 1;
    const int blocks = blocks_for((size_t)n * h * w * (c / 16), sm_count, 32);
    if (e3) {
        maxpool_bwd_kernel<0, true><<<blocks, kThreads, 0, st>>>(e, e_exp, arg, n, h, w, c, k, s, p, ho, wo, e_in, e_in_exp, next_mask,
                                                                 next_gamma, e3, e3_exp, sum_e1, dev);
        hook(&dev->absmax_u32, 1, EOQ_REDUCE_I32, EOQ_REDUCE_MAX, st);
        hook(&dev->absmax_u64, 1, EOQ_REDUCE_I64, EOQ_REDUCE_MAX, st);
        maxpool_bwd_kernel<1, true><<<blocks, kThreads, 0, st>>>(e, e_exp, arg, n, h, w, c, k, s, p, ho, wo, e_in, e_in_exp, next_mask,
                                                                 next_gamma, e3, e3_exp, sum_e1, dev);
        if (sum_e1) hook(sum_e1, 1, EOQ_REDUCE_I64, EOQ_REDUCE_SUM, st);
    } else {
        maxpool_bwd_kernel<0, false><<<blocks, kThreads, 0, st>>>(e, e_exp, arg, n, h, w, c, k, s, p, ho, wo, e_in, e_in_exp, nullptr,
                                                                  nullptr, nullptr, nullptr, nullptr, dev);
        hook(&dev->absmax_u32, 1, EOQ_REDUCE_I32, EOQ_REDUCE_MAX, st);
        maxpool_bwd_kernel<1, false><<<blocks, kThreads, 0, st>>>(e, e_exp, arg, n, h, w, c, k, s, p, ho, wo, e_in, e_in_exp, nullptr,
                                                                  nullptr, nullptr, nullptr, nullptr, dev);
    }
    return cudaGetLastError();
}

cudaError_t launch_avgpool_sum(const int8_t *x, int n, int hw, int c, int32_t *sums, cudaStream_t st)
{
    avgpool_sum_kernel<<<n * (c / 16), kThreads, 0, st>>>(x, hw, c, sums);
    return cudaGetLastError();
}

cudaError_t launch_join(const int8_t *a, const int32_t *a_exp, const int8_t *b, const int32_t *b_exp, const uint8_t *mask_b,
                        size_t n_el, int8_t *out, int32_t *out_exp, long long *sum_out, const uint8_t *next_mask,
                        const int16_t *next_x2, const int32_t *next_gamma, int8_t *e3, int32_t *e3_exp, long long *sum_e1,
                        long long *sum_e1x2, DeviceState *dev, int sm_count, cudaStream_t st, const ReduceHook &hook)
{
    const size_t n16 = n_el / 16;
    const int blocks = blocks_for(n16, sm_count, 8);
    if (e3) {
        join_kernel<0, true><<<blocks, kThreads, 0, st>>>(a, a_exp, b, b_exp, mask_b, n16, out, out_exp, sum_out, next_mask, next_x2,
                                                          next_gamma, e3, e3_exp, sum_e1, sum_e1x2, dev);
        hook(&dev->absmax_u64, 1, EOQ_REDUCE_I64, EOQ_REDUCE_MAX, st);
        hook(&dev->absmax2_u64, 1, EOQ_REDUCE_I64, EOQ_REDUCE_MAX, st);
        join_kernel<1, true><<<blocks, kThreads, 0, st>>>(a, a_exp, b, b_exp, mask_b, n16, out, out_exp, sum_out, next_mask, next_x2,
                                                          next_gamma, e3, e3_exp, sum_e1, sum_e1x2, dev);
        if (sum_out) hook(sum_out, 1, EOQ_REDUCE_I64, EOQ_REDUCE_SUM, st);
        if (sum_e1) hook(sum_e1, 1, EOQ_REDUCE_I64, EOQ_REDUCE_SUM, st);
        if (sum_e1x2) hook(sum_e1x2, 1, EOQ_REDUCE_I64, EOQ_REDUCE_SUM, st);
    } else {
        join_kernel<0, false><<<blocks, kThreads, 0, st>>>(a, a_exp, b, b_exp, mask_b, n16, out, out_exp, sum_out, nullptr, nullptr,
                                                           nullptr, nullptr, nullptr, nullptr, nullptr, dev);
        hook(&dev->absmax_u64, 1, EOQ_REDUCE_I64, EOQ_REDUCE_MAX, st);
        join_kernel<1, false><<<blocks, kThreads, 0, st>>>(a, a_exp, b, b_exp, mask_b, n16, out, out_exp, sum_out, nullptr, nullptr,
                                                           nullptr, nullptr, nullptr, nullptr, nullptr, dev);
        if (sum_out) hook(sum_out, 1, EOQ_REDUCE_I64, EOQ_REDUCE_SUM, st);
    }
    return cudaGetLastError();
}

cudaError_t launch_join_second(const int8_t *a, const int32_t *a_exp, const int8_t *b, const int32_t *b_exp, const uint8_t *mask_b,
                               size_t n_el, int8_t *out, int32_t *out_exp, long long *sum_out, const NextHeadArgs *next,
                               DeviceState *dev, int sm_count, cudaStream_t st)
{
    const size_t n16 = n_el / 16;
    const int blocks = blocks_for(n16, sm_count, 8);
    if (next)
        join_kernel<1, true><<<blocks, kThreads, 0, st>>>(a, a_exp, b, b_exp, mask_b, n16, out, out_exp, sum_out, next->mask, next->x2,
                                                          next->gamma, next->e3, next->e3_exp, next->sum_e1, next->sum_e1x2, dev);
    else
        join_kernel<1, false><<<blocks, kThreads, 0, st>>>(a, a_exp, b, b_exp, mask_b, n16, out, out_exp, sum_out, nullptr, nullptr,
                                                           nullptr, nullptr, nullptr, nullptr, nullptr, dev);
    return cudaGetLastError();
}

cudaError_t launch_head(const int32_t *sums, int n, int c, int hw, int classes, float *W, float *bias, const int32_t *labels,
                        float lr, float *loss_out, float *dpooled, float *logits, float *pooled, float *dl, double *loss_n,
                        cudaStream_t st)
{
    head_pooled_kernel<<<(n * c + 255) / 256, 256, 0, st>>>(sums, n * c, hw, pooled);
    {
        const size_t smem = (size_t)c * 33 * sizeof(float);
        cudaError_t e = cudaFuncSetAttribute(head_logits_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        dim3 grid((classes + kHeadWarps - 1) / kHeadWarps, (n + 31) / 32);
        head_logits_kernel<<<grid, 32 * kHeadWarps, smem, st>>>(pooled, n, c, classes, W, bias, logits);
    }
    head_softmax_kernel<<<n, 256, 0, st>>>(logits, n, classes, labels, dl, loss_n);
    head_dpooled_kernel<<<dim3((c + kDpCh - 1) / kDpCh, (n + kDpN - 1) / kDpN), kDpCh * kDpN, 0, st>>>(dl, W, n, c, classes, dpooled,
                                                                                                   loss_n, loss_out);
    if (lr != 0.0f) head_update_kernel<<<(classes * c + 127) / 128, 128, 0, st>>>(dl, pooled, n, c, classes, lr, W, bias);
    return cudaGetLastError();
}

cudaError_t launch_head_update(const float *dl, const float *pooled, int n, int c, int classes, float lr, float *W, float *bias,
                               cudaStream_t st)
{
    head_update_kernel<<<(classes * c + 127) / 128, 128, 0, st>>>(dl, pooled, n, c, classes, lr, W, bias);
    return cudaGetLastError();
}

cudaError_t launch_head_error(const float *dpooled, int n, int c, int hw, float *ef, int8_t *e, int32_t *e_exp, DeviceState *dev,
                              int sm_count, cudaStream_t st, const ReduceHook &hook)
{
    head_error_scale_kernel<<<blocks_for((size_t)n * c, sm_count, 1), kThreads, 0, st>>>(dpooled, n * c, hw, ef, dev);
    hook(&dev->absmax_u32, 1, EOQ_REDUCE_I32, EOQ_REDUCE_MAX, st);
    head_error_spread_kernel<<<blocks_for((size_t)n * hw * (c / 16), sm_count), kThreads, 0, st>>>(ef, n, hw, c, e, e_exp, dev);
    return cudaGetLastError();
}

cudaError_t launch_scalar_update(const ScalarBatch &b, int32_t lr_mant, int32_t lr_exp, int stochastic, uint64_t seed,
                                 const unsigned long long *step_dev, uint64_t step, cudaStream_t st)
{
    scalar_update_kernel<<<(b.num + 63) / 64, 64, 0, st>>>(b, lr_mant, lr_exp, stochastic, seed, step_dev, step);
    return cudaGetLastError();
}

}  // namespace eoq
