// Training-mode batch normalisation behind the int8 convolution, forward and backward: the operation the EOQ layer
// does without (arXiv 2105.13890, Sec. 5.3 compares the Fixup scale and bias against it).  It is here so that its
// cost can be measured on the same convolution output beside the fused scale-and-bias epilogue; it is not on the
// EOQ path.  What it needs and EOQ does not: per-channel reductions over the whole batch between the convolution
// and the activation (so the exact sums go through memory once more), a second pair of reductions in the backward
// pass, a square root and divisions per channel, and floating-point multiply-adds per element.
//
// Statistics are exact integers (sum and sum of squares of the int32 convolution sums; the squares in three 64-bit
// parts, a = h * 2^16 + l), the per-channel constants are formed in double precision with every operation rounded
// once in a fixed order, and each element takes one single-precision fused multiply-add: results do not depend on
// the order of the reductions and are reproducible bit for bit.
#include "eoq_device.cuh"
#include "eoq_internal.h"

namespace eoq {

namespace {

constexpr int kBnThreads = 256;
constexpr int kBnSplit = 16;       // threads of a finish kernel that share one channel
constexpr int kBnMaxParts = 296;   // blocks of a statistics kernel (rows of partial sums in the workspace)

__device__ __forceinline__ double u128_to_double(unsigned __int128 v)
{
    const double hi = __ull2double_rn((unsigned long long)(v >> 64)), lo = __ull2double_rn((unsigned long long)v);
    return __dadd_rn(__dmul_rn(hi, 18446744073709551616.0), lo);
}

// Every thread owns four consecutive channels (one 16-byte load of sums) and walks pixels with a fixed stride, so
// that its channels never change; the threads of a block meet in shared memory and the block writes its totals to
// its own row of `part` ([block][c][4]: s1, hh, hl, ll) - no global atomics; the finish kernel adds the rows.
constexpr int kBnUnroll = 4;
__global__ void __launch_bounds__(kBnThreads) bn_stats_kernel(const int32_t *__restrict__ acc, size_t pixels, int c,
                                                             unsigned long long *__restrict__ part)
{
    extern __shared__ unsigned long long cell[];   // [c][4]
    const int cg = c / 4;
    for (int i = threadIdx.x; i < c * 4; i += blockDim.x) cell[i] = 0ull;
    __syncthreads();
    const int g = threadIdx.x % cg, slot = threadIdx.x / cg, slots = blockDim.x / cg;
    long long s1[4] = {0, 0, 0, 0}, hh[4] = {0, 0, 0, 0}, hl[4] = {0, 0, 0, 0};
    unsigned long long ll[4] = {0, 0, 0, 0};
    const size_t stride = (size_t)gridDim.x * slots;
    for (size_t p0 = (size_t)blockIdx.x * slots + slot; p0 < pixels; p0 += kBnUnroll * stride) {
        int4 v[kBnUnroll];
#pragma unroll
        for (int u = 0; u < kBnUnroll; ++u) {
            const size_t p = p0 + u * stride;
            v[u] = p < pixels ? __ldg(reinterpret_cast<const int4 *>(acc + p * c) + g) : make_int4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < kBnUnroll; ++u) {
            const int a[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int h = a[q] >> 16;
                const unsigned l = (unsigned)a[q] & 0xffffu;
                s1[q] += a[q];
                hh[q] += h * h;                                   // < 2^30
                hl[q] += (long long)h * (long long)l;             // |.| < 2^31
                ll[q] += (unsigned long long)(l * l);             // < 2^32
            }
        }
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        unsigned long long *dst = cell + (size_t)(g * 4 + q) * 4;
        atomicAdd(dst + 0, (unsigned long long)s1[q]);
        atomicAdd(dst + 1, (unsigned long long)hh[q]);
        atomicAdd(dst + 2, (unsigned long long)hl[q]);
        atomicAdd(dst + 3, ll[q]);
    }
    __syncthreads();
    unsigned long long *row = part + (size_t)blockIdx.x * c * 4;
    for (int i = threadIdx.x; i < c * 4; i += blockDim.x) row[i] = cell[i];
}

__global__ void bn_finish_kernel(BnChannel *ch, const unsigned long long *__restrict__ part, int parts, size_t pixels, int c, int p,
                                 const float *__restrict__ gamma, const float *__restrict__ beta, float eps)
{
    // kBnSplit threads share a channel: each adds every kBnSplit-th row of partial sums, then the lanes meet by shuffle
    const int tid = blockIdx.x * blockDim.x + threadIdx.x, k = tid / kBnSplit, j = tid % kBnSplit;
    unsigned long long t[4] = {0, 0, 0, 0};
    if (k < c)
        for (int b = j; b < parts; b += kBnSplit) {
            const ulonglong2 *src = reinterpret_cast<const ulonglong2 *>(part + ((size_t)b * c + k) * 4);
            const ulonglong2 lo = src[0], hi = src[1];
            t[0] += lo.x;
            t[1] += lo.y;
            t[2] += hi.x;
            t[3] += hi.y;
        }
#pragma unroll
    for (int q = 0; q < 4; ++q)
#pragma unroll
        for (int d = kBnSplit / 2; d > 0; d >>= 1) t[q] += __shfl_down_sync(0xffffffffu, t[q], d, kBnSplit);
    if (k >= c || j != 0) return;
    const long long s1 = (long long)t[0];
    ch[k].s1 = s1;
    ch[k].shh = (long long)t[1];
    ch[k].shl = (long long)t[2];
    ch[k].sll = (long long)t[3];
    const __int128 s2 = ((__int128)(long long)t[1] << 32) + ((__int128)(long long)t[2] << 17) + (__int128)t[3];
    const unsigned __int128 V = (unsigned __int128)pixels * (unsigned __int128)s2 - (unsigned __int128)((__int128)s1 * s1);
    const double Pd = __ull2double_rn((unsigned long long)pixels);
    const double mu = __ddiv_rn(__ll2double_rn(s1), Pd);
    const double var_a = __ddiv_rn(u128_to_double(V), __dmul_rn(Pd, Pd));
    const double var_v = ldexp(var_a, 2 * p);
    const double inv = __ddiv_rn(1.0, __dsqrt_rn(__dadd_rn(var_v, (double)eps)));
    const double ks = ldexp(__dmul_rn((double)gamma[k], inv), p);
    ch[k].mu = mu;
    ch[k].inv = inv;
    ch[k].scale = __double2float_rn(ks);
    ch[k].shift = __double2float_rn(__dsub_rn((double)beta[k], __dmul_rn(ks, mu)));
}

// y = fma((float)a, scale, shift); x5 = Q_a2(relu(y)); mask bit = [y > 0].  One thread per 16 channels of a pixel.
__global__ void __launch_bounds__(kBnThreads) bn_apply_kernel(const int32_t *__restrict__ acc, size_t groups, int c,
                                                             const BnChannel *__restrict__ ch, int8_t *__restrict__ x5,
                                                             uint8_t *__restrict__ relu_mask)
{
    extern __shared__ float2 ss[];   // [c]: scale, shift
    for (int i = threadIdx.x; i < c; i += blockDim.x) ss[i] = make_float2(ch[i].scale, ch[i].shift);
    __syncthreads();
    const int gpp = c / 16;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < groups; i += (size_t)gridDim.x * blockDim.x) {
        const int k0 = (int)(i % gpp) * 16;
        const int4 *src = reinterpret_cast<const int4 *>(acc + i * 16);
        int code[16];
        unsigned bits = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int4 v = __ldg(src + q);
            const int a[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const float2 s = ss[k0 + 4 * q + r];
                const float y = __fmaf_rn(__int2float_rn(a[r]), s.x, s.y);
                const bool pos = y > 0.0f;
                code[4 * q + r] = pos ? min(__float2int_rn(y * 128.0f), 127) : 0;
                bits |= (pos ? 1u : 0u) << (4 * q + r);
            }
        }
        auto pack = [&](int j) {
            return (int)((uint32_t)(code[j] & 0xff) | ((uint32_t)(code[j + 1] & 0xff) << 8) | ((uint32_t)(code[j + 2] & 0xff) << 16) |
                         ((uint32_t)(code[j + 3] & 0xff) << 24));
        };
        reinterpret_cast<int4 *>(x5)[i] = make_int4(pack(0), pack(4), pack(8), pack(12));
        reinterpret_cast<uint16_t *>(relu_mask)[i] = (uint16_t)bits;
    }
}

// D1 = sum(E * mask), D2 = sum(E * mask * A) per channel; same thread layout as bn_stats_kernel, `part` [block][c][2].
__global__ void __launch_bounds__(kBnThreads) bn_bwd_stats_kernel(const int8_t *__restrict__ e, const uint8_t *__restrict__ relu_mask,
                                                                 const int32_t *__restrict__ acc, size_t pixels, int c,
                                                                 unsigned long long *__restrict__ part)
{
    extern __shared__ unsigned long long cell[];   // [c][2]
    const int cg = c / 4;
    for (int i = threadIdx.x; i < c * 2; i += blockDim.x) cell[i] = 0ull;
    __syncthreads();
    const int g = threadIdx.x % cg, slot = threadIdx.x / cg, slots = blockDim.x / cg;
    long long d1[4] = {0, 0, 0, 0}, d2[4] = {0, 0, 0, 0};
    const size_t stride = (size_t)gridDim.x * slots;
    for (size_t p0 = (size_t)blockIdx.x * slots + slot; p0 < pixels; p0 += kBnUnroll * stride) {
        int4 v[kBnUnroll];
        uint32_t ew[kBnUnroll], m[kBnUnroll];
#pragma unroll
        for (int u = 0; u < kBnUnroll; ++u) {
            const size_t p = p0 + u * stride;
            const size_t i0 = p * c + (size_t)g * 4;
            const bool in = p < pixels;
            v[u] = in ? __ldg(reinterpret_cast<const int4 *>(acc + i0)) : make_int4(0, 0, 0, 0);
            ew[u] = in ? __ldg(reinterpret_cast<const uint32_t *>(e + i0)) : 0u;
            m[u] = in ? (uint32_t)__ldg(relu_mask + (i0 >> 3)) >> (i0 & 7) : 0u;
        }
#pragma unroll
        for (int u = 0; u < kBnUnroll; ++u) {
            const int a[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const int dy = ((m[u] >> q) & 1u) ? (int)(int8_t)(ew[u] >> (8 * q)) : 0;
                d1[q] += dy;
                d2[q] += (long long)dy * a[q];
            }
        }
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        atomicAdd(cell + (size_t)(g * 4 + q) * 2 + 0, (unsigned long long)d1[q]);
        atomicAdd(cell + (size_t)(g * 4 + q) * 2 + 1, (unsigned long long)d2[q]);
    }
    __syncthreads();
    unsigned long long *row = part + (size_t)blockIdx.x * c * 2;
    for (int i = threadIdx.x; i < c * 2; i += blockDim.x) row[i] = cell[i];
}

__global__ void bn_bwd_finish_kernel(BnChannel *ch, const unsigned long long *__restrict__ part, int parts, size_t pixels, int c, int p,
                                     const int32_t *e_exp, const float *__restrict__ gamma, float *dgamma, float *dbeta)
{
    const int tid = blockIdx.x * blockDim.x + threadIdx.x, k = tid / kBnSplit, j = tid % kBnSplit;
    unsigned long long t0 = 0, t1 = 0;
    if (k < c)
        for (int b = j; b < parts; b += kBnSplit) {
            const ulonglong2 v = *reinterpret_cast<const ulonglong2 *>(part + ((size_t)b * c + k) * 2);
            t0 += v.x;
            t1 += v.y;
        }
#pragma unroll
    for (int d = kBnSplit / 2; d > 0; d >>= 1) {
        t0 += __shfl_down_sync(0xffffffffu, t0, d, kBnSplit);
        t1 += __shfl_down_sync(0xffffffffu, t1, d, kBnSplit);
    }
    if (k >= c || j != 0) return;
    ch[k].d1 = (long long)t0;
    ch[k].d2 = (long long)t1;
    const int p_e = *e_exp;
    const double Pd = __ull2double_rn((unsigned long long)pixels);
    const double mu = ch[k].mu, inv = ch[k].inv;
    const double d1 = __ll2double_rn((long long)t0), d2 = __ll2double_rn((long long)t1);
    const double cov = __dsub_rn(d2, __dmul_rn(mu, d1));
    const double ip = ldexp(inv, p);
    const double g2 = ldexp(__dmul_rn(ip, cov), p_e);
    const double g1 = ldexp(d1, p_e);
    const double kk = __dmul_rn((double)gamma[k], inv);
    const double m2 = __ddiv_rn(g2, Pd);
    const double cb_d = __dmul_rn(-__dmul_rn(kk, m2), ip);
    ch[k].ca = __double2float_rn(ldexp(kk, p_e));
    ch[k].cb = __double2float_rn(cb_d);
    ch[k].cc = __double2float_rn(__dsub_rn(-__dmul_rn(kk, __ddiv_rn(g1, Pd)), __dmul_rn(cb_d, mu)));
    dgamma[k] = __double2float_rn(g2);
    dbeta[k] = __double2float_rn(g1);
}

// da = fma(ca, E * mask, fma(cb, (float)A, cc)); one thread per 16 channels of a pixel
__global__ void __launch_bounds__(kBnThreads) bn_bwd_apply_kernel(const int8_t *__restrict__ e, const uint8_t *__restrict__ relu_mask,
                                                                 const int32_t *__restrict__ acc, size_t groups, int c,
                                                                 const BnChannel *__restrict__ ch, float *__restrict__ da)
{
    extern __shared__ float4 cs[];   // [c]: ca, cb, cc
    for (int i = threadIdx.x; i < c; i += blockDim.x) cs[i] = make_float4(ch[i].ca, ch[i].cb, ch[i].cc, 0.0f);
    __syncthreads();
    const int gpp = c / 16;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < groups; i += (size_t)gridDim.x * blockDim.x) {
        const int k0 = (int)(i % gpp) * 16;
        const int4 ev = __ldg(reinterpret_cast<const int4 *>(e) + i);
        const uint32_t m = __ldg(reinterpret_cast<const uint16_t *>(relu_mask) + i);
        const uint32_t ew[4] = {(uint32_t)ev.x, (uint32_t)ev.y, (uint32_t)ev.z, (uint32_t)ev.w};
        const int4 *src = reinterpret_cast<const int4 *>(acc + i * 16);
        float4 *dst = reinterpret_cast<float4 *>(da + i * 16);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const int4 v = __ldg(src + q);
            const int a[4] = {v.x, v.y, v.z, v.w};
            float o[4];
#pragma unroll
            for (int r = 0; r < 4; ++r) {
                const float4 k = cs[k0 + 4 * q + r];
                const float dy = ((m >> (4 * q + r)) & 1u) ? __int2float_rn((int)(int8_t)(ew[q] >> (8 * r))) : 0.0f;
                o[r] = __fmaf_rn(k.x, dy, __fmaf_rn(k.y, __int2float_rn(a[r]), k.z));
            }
            dst[q] = make_float4(o[0], o[1], o[2], o[3]);
        }
    }
}

inline int stats_threads(int c) { return (kBnThreads / (c / 4)) * (c / 4); }

inline int stats_grid(size_t pixels, int slots, int sm_count)
{
    size_t b = (pixels + (size_t)slots * kBnUnroll - 1) / ((size_t)slots * kBnUnroll), cap = (size_t)(2 * sm_count);
    if (cap > (size_t)kBnMaxParts) cap = kBnMaxParts;
    if (b > cap) b = cap;
    return b < 1 ? 1 : (int)b;
}

inline int grid_for(size_t items, int sm_count, int per_sm)
{
    size_t b = (items + kBnThreads - 1) / kBnThreads, cap = (size_t)sm_count * per_sm;
    if (b > cap) b = cap;
    return b < 1 ? 1 : (int)b;
}

}  // namespace

size_t bn_workspace_bytes(int c) { return sizeof(BnChannel) * (size_t)c + sizeof(unsigned long long) * 4 * (size_t)c * kBnMaxParts; }

cudaError_t launch_bn_fwd(const int32_t *acc, int p, size_t pixels, int c, const float *gamma, const float *beta, float eps,
                          int8_t *x5, uint8_t *relu_mask, BnChannel *ch, int sm_count, cudaStream_t st)
{
    unsigned long long *part = reinterpret_cast<unsigned long long *>(ch + c);
    const int threads = stats_threads(c), slots = threads / (c / 4), parts = stats_grid(pixels, slots, sm_count);
    bn_stats_kernel<<<parts, threads, sizeof(unsigned long long) * 4 * c, st>>>(acc, pixels, c, part);
    bn_finish_kernel<<<(c * kBnSplit + 127) / 128, 128, 0, st>>>(ch, part, parts, pixels, c, p, gamma, beta, eps);
    const size_t groups = pixels * (size_t)(c / 16);
    bn_apply_kernel<<<grid_for(groups, sm_count, 8), kBnThreads, sizeof(float2) * c, st>>>(acc, groups, c, ch, x5, relu_mask);
    return cudaGetLastError();
}

cudaError_t launch_bn_bwd(const int8_t *e, const int32_t *e_exp, const uint8_t *relu_mask, const int32_t *acc, int p, size_t pixels,
                          int c, const float *gamma, BnChannel *ch, float *da, float *dgamma, float *dbeta, int sm_count,
                          cudaStream_t st)
{
    unsigned long long *part = reinterpret_cast<unsigned long long *>(ch + c);
    const int threads = stats_threads(c), slots = threads / (c / 4), parts = stats_grid(pixels, slots, sm_count);
    bn_bwd_stats_kernel<<<parts, threads, sizeof(unsigned long long) * 2 * c, st>>>(e, relu_mask, acc, pixels, c, part);
    bn_bwd_finish_kernel<<<(c * kBnSplit + 127) / 128, 128, 0, st>>>(ch, part, parts, pixels, c, p, e_exp, gamma, dgamma, dbeta);
    const size_t groups = pixels * (size_t)(c / 16);
    bn_bwd_apply_kernel<<<grid_for(groups, sm_count, 8), kBnThreads, sizeof(float4) * c, st>>>(e, relu_mask, acc, groups, c, ch, da);
    return cudaGetLastError();
}

}  // namespace eoq
