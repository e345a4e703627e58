// Bandwidth-bound kernels of the EOQ layer (arXiv 2105.13890): the standalone quantizers Q / CQ / SQ
// (Sec. 3.2.2), the second phase of the scale quantizer after a convolution, the head of the error
// chain (Sec. 3.2.1), the 8-bit update (Sec. 3.2.3) and small layout helpers.
// Reductions run warp-shuffle -> one atomic per warp; 16 elements per thread with 128-bit accesses.
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

inline int grid_for(size_t work_items, int sm_count, int per_sm = 8)
{
    size_t blocks = (work_items + kThreads - 1) / kThreads;
    size_t cap = (size_t)sm_count * per_sm;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

// Every thread of every block calls this after the block's last use of the handle's reduction cells (no early
// returns before it).  True in thread 0 of the block that arrives last: by then every block has read what it
// needed and added what it had to add, so that thread may publish the sums and must put the cells back to zero.
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

// ------------------------------------------------------------------ fp32 -> Q / CQ / SQ

// R(log2 M) for a positive finite float given by its bit pattern.
__device__ __forceinline__ int round_log2_f32bits(uint32_t bits)
{
    const int eb = (int)((bits >> 23) & 0xffu);
    const uint32_t frac = bits & 0x7fffffu;
    if (eb == 0) return round_log2_u32(frac) - 149;  // subnormal: frac * 2^-149
    const unsigned long long m = (1ull << 23) | frac;  // M = m * 2^(eb - 150), m in [2^23, 2^24)
    return (eb - 127) + ((m * m >= (1ull << 47)) ? 1 : 0);
}

__global__ void absmax_f32_kernel(const float *__restrict__ src, size_t n, DeviceState *dev)
{
    uint32_t mx = 0;
    bool bad = false;
    const size_t n4 = n / 4;
    const float4 *s4 = reinterpret_cast<const float4 *>(src);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        float4 v = __ldg(s4 + i);
        uint32_t b[4] = {__float_as_uint(v.x), __float_as_uint(v.y), __float_as_uint(v.z), __float_as_uint(v.w)};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            uint32_t a = b[k] & 0x7fffffffu;
            bad |= a >= 0x7f800000u;
            mx = max(mx, a);
        }
    }
    for (size_t i = n4 * 4 + (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        uint32_t a = __float_as_uint(src[i]) & 0x7fffffffu;
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

// mode 0: Q -> int16, mode 1: CQ -> int8, mode 2: SQ -> int8 under the already reduced maximum.
__global__ void quantize_f32_kernel(int mode, const float *__restrict__ src, size_t n, void *dst, int32_t *dst_exp,
                                    DeviceState *dev)
{
    int up = 7;  // codes = R(x * 2^up)
    if (mode == 2) {
        const uint32_t mbits = dev->absmax_u32;
        if (mbits == 0 || mbits >= 0x7f800000u) {
            up = 7;
            if (blockIdx.x == 0 && threadIdx.x == 0) {
                if (mbits == 0) atomicOr(&dev->status, EOQ_DEV_SQ_ZERO);
                *dst_exp = -7;
            }
        } else {
            const int t = round_log2_f32bits(mbits);
            up = 7 - t;
            if (blockIdx.x == 0 && threadIdx.x == 0) *dst_exp = t - 7;
        }
    } else if (dst_exp && blockIdx.x == 0 && threadIdx.x == 0) {
        *dst_exp = -7;
    }
    const int lim = (mode == 0) ? 32767 : 127;
    const int lo = (mode == 0) ? -32768 : -127;
    auto code = [&](float x) -> int {
        float y = scalbnf(x, up);  // exact: a power-of-two scaling of a value that stays far from overflow
        if (!(fabsf(y) < 1.0e9f)) return (y > 0.f) ? lim : ((y < 0.f) ? lo : 0);
        return clampi(__float2int_rn(y), lo, lim);
    };
    const size_t n16 = n / 16;
    const float4 *s4 = reinterpret_cast<const float4 *>(src);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (size_t)gridDim.x * blockDim.x) {
        int c[16];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            float4 v = __ldg(s4 + i * 4 + k);
            c[4 * k + 0] = code(v.x);
            c[4 * k + 1] = code(v.y);
            c[4 * k + 2] = code(v.z);
            c[4 * k + 3] = code(v.w);
        }
        if (mode == 0) {
            int4 *d = reinterpret_cast<int4 *>(dst) + i * 2;
            d[0] = make_int4((c[0] & 0xffff) | (c[1] << 16), (c[2] & 0xffff) | (c[3] << 16),
                             (c[4] & 0xffff) | (c[5] << 16), (c[6] & 0xffff) | (c[7] << 16));
            d[1] = make_int4((c[8] & 0xffff) | (c[9] << 16), (c[10] & 0xffff) | (c[11] << 16),
                             (c[12] & 0xffff) | (c[13] << 16), (c[14] & 0xffff) | (c[15] << 16));
        } else {
            reinterpret_cast<int4 *>(dst)[i] =
                make_int4((int)pack4(c[0], c[1], c[2], c[3]), (int)pack4(c[4], c[5], c[6], c[7]),
                          (int)pack4(c[8], c[9], c[10], c[11]), (int)pack4(c[12], c[13], c[14], c[15]));
        }
    }
    for (size_t i = n16 * 16 + (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const int c = code(src[i]);
        if (mode == 0) reinterpret_cast<int16_t *>(dst)[i] = (int16_t)c;
        else reinterpret_cast<int8_t *>(dst)[i] = (int8_t)c;
    }
    if (mode == 2 && last_block_done(dev)) dev->absmax_u32 = 0;
}

// SQ of an fp32 image under the already reduced maximum: c_src channels in, c_dst (zero-padded) channels out,
// rows widened by `wmargin` zero pixels at both ends.  A thread writes kG = 16 or 8 channels of a pixel.
template <int kG>
__global__ void quantize_image_kernel(const float *__restrict__ src, int rows, int w, int c_src, int c_dst, int wmargin,
                                      int8_t *dst, int32_t *dst_exp, DeviceState *dev)
{
    const uint32_t mbits = dev->absmax_u32;
    int up = 7;
    const bool usable = mbits != 0 && mbits < 0x7f800000u;
    if (usable) up = 7 - round_log2_f32bits(mbits);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        *dst_exp = usable ? -up : -7;
        if (mbits == 0) atomicOr(&dev->status, EOQ_DEV_SQ_ZERO);
    }
    const int groups = c_dst / kG;
    const int w_mem = w + 2 * wmargin;
    const size_t items = (size_t)rows * w_mem * groups;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < items; i += (size_t)gridDim.x * blockDim.x) {
        int g, xm;
        size_t row;
        if (items <= 0xffffffffull) {  // 32-bit index arithmetic: three 64-bit divisions would dominate the item's work
            const uint32_t mp = (uint32_t)i / (uint32_t)groups, r = mp / (uint32_t)w_mem;
            g = (int)((uint32_t)i - mp * (uint32_t)groups);
            xm = (int)(mp - r * (uint32_t)w_mem) - wmargin;
            row = r;
        } else {
            g = (int)(i % groups);
            const size_t mp = i / groups;            // pixel index in the widened layout
            xm = (int)(mp % w_mem) - wmargin;
            row = mp / w_mem;
        }
        int c[kG];
#pragma unroll
        for (int k = 0; k < kG; ++k) {
            const int ch = g * kG + k;
            int v = 0;
            if (ch < c_src && xm >= 0 && xm < w) {
                const float y = scalbnf(__ldg(src + (row * w + xm) * c_src + ch), up);
                v = (fabsf(y) < 1.0e9f) ? clampi(__float2int_rn(y), -127, 127) : (y > 0.f ? 127 : (y < 0.f ? -127 : 0));
            }
            c[k] = v;
        }
        if (kG == 16)
            reinterpret_cast<int4 *>(dst)[i] =
                make_int4((int)pack4(c[0], c[1], c[2], c[3]), (int)pack4(c[4], c[5], c[6], c[7]),
                          (int)pack4(c[8 % kG], c[9 % kG], c[10 % kG], c[11 % kG]), (int)pack4(c[12 % kG], c[13 % kG], c[14 % kG], c[15 % kG]));
        else
            reinterpret_cast<int2 *>(dst)[i] = make_int2((int)pack4(c[0], c[1], c[2], c[3]), (int)pack4(c[4], c[5], c[6], c[7]));
    }
    if (last_block_done(dev)) dev->absmax_u32 = 0;
}

// w[oc][kh][kw][c] -> wp[oc][kh][8][c] with zeros in the unused taps; c = 16 (Pixel = int4) or 8 (int2)
template <typename Pixel>
__global__ void weight_pad_rows_kernel(const int8_t *__restrict__ w, int8_t *__restrict__ wp, int rows, int kw)
{
    const int i = blockIdx.x * blockDim.x + threadIdx.x;  // one pixel of the padded layout
    if (i >= rows * 8) return;
    const int r = i >> 3, t = i & 7;
    Pixel v = Pixel();
    if (t < kw) v = __ldg(reinterpret_cast<const Pixel *>(w) + (size_t)r * kw + t);
    reinterpret_cast<Pixel *>(wp)[i] = v;
}

// ------------------------------------------------------------------ int32 -> SQ (phase 2 of Q_e after dgrad)

__global__ void absmax_i32_kernel(const int32_t *__restrict__ src, size_t n, DeviceState *dev)
{
    uint32_t mx = 0;
    const size_t n4 = n / 4;
    const int4 *s4 = reinterpret_cast<const int4 *>(src);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n4; i += (size_t)gridDim.x * blockDim.x) {
        int4 v = __ldg(s4 + i);
        mx = max(max(mx, (uint32_t)abs(v.x)), max((uint32_t)abs(v.y), max((uint32_t)abs(v.z), (uint32_t)abs(v.w))));
    }
    for (size_t i = n4 * 4 + (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        mx = max(mx, (uint32_t)abs(src[i]));
    mx = (uint32_t)block_max_u64(mx);
    if (threadIdx.x == 0 && mx) atomicMax(&dev->absmax_u32, mx);
}

// One 256-bit streaming load (sm_100); ptr must be 32-byte aligned.
__device__ __forceinline__ void ld_global_256_stream(const int32_t *ptr, int *v)
{
    asm volatile("ld.global.cs.v8.b32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7])
                 : "l"(ptr));
}

// kNext: the error head of the layer that consumes dst rides along (see NextHead): the masked maximum sits in the
// handle's 64-bit cell (the GEMM epilogue reduced it beside the plain one), so the codes of e3 and the head's sums
// come out of the same pass.  n must then be a multiple of 16.
// kJoin: dst is the first operand of an error join; the join's first pass rides along: max |dst * 2^sa + b * 2^sb|
// over all positions (64-bit cell) and over those the consumer's ReLU lets through (second 64-bit cell).
template <bool kNext, bool kJoin>
__global__ void sq_i32_kernel(const int32_t *__restrict__ src, const int32_t *src_exp, int exp_bias, size_t n,
                              int8_t *dst, int32_t *dst_exp, long long *sum_codes, NextHeadArgs next, JoinStatArgs join,
                              DeviceState *dev)
{
    const uint32_t M = dev->absmax_u32;
    const int t = M ? round_log2_u32(M) : 7;
    const int p_in = (src_exp ? *src_exp : 0) + exp_bias;
    const int p0 = M ? p_in + t - 7 : p_in;
    NextHead nh = {};
    if (kNext) nh = next_head_setup(next.gamma, (uint32_t)abs(sq_code32((int32_t)dev->absmax_u64, t)), dev);
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        *dst_exp = p0;
        if (!M) atomicOr(&dev->status, EOQ_DEV_SQ_ZERO);
        if (kNext) next_head_exponent(nh, p0, next.e3_exp, dev);
    }
    long long sum = 0, s1 = 0, s2 = 0;
    const size_t n16 = n / 16;
    const int4 *s4 = reinterpret_cast<const int4 *>(src);
    const int sh = t - 7;
    JoinShift js = {0, 0, 0};
    bool j_narrow = true;
    int j_ma = 1, j_mb = 1;
    unsigned long long jmx = 0, jmxm = 0;
    if (kJoin) {
        js = join_shift(p0, __ldg(join.b_exp));
        j_narrow = js.sa >= 0 && js.sb >= 0 && js.sa <= 23 && js.sb <= 23;
        j_ma = 1 << (js.sa < 0 ? 0 : min(js.sa, 23));
        j_mb = 1 << (js.sb < 0 ? 0 : min(js.sb, 23));
    }
    // the maximum bounds every element, so |a| + 2^(sh-1) cannot wrap as long as M + M / 2^7 < 2^31
    const bool fast = sh >= 1 && M < 0x7e000000u;
    const int32_t half_m1 = fast ? (1 << (sh - 1)) - 1 : 0;
    const bool wide_in = (reinterpret_cast<uintptr_t>(src) & 31) == 0;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (size_t)gridDim.x * blockDim.x) {
        int c[16], a[16];
        if (wide_in) {   // two 256-bit loads: whole 32-byte sectors per lane
            ld_global_256_stream(src + i * 16, a);
            ld_global_256_stream(src + i * 16 + 8, a + 8);
        } else {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int4 v = __ldcs(s4 + i * 4 + k);
                a[4 * k + 0] = v.x;
                a[4 * k + 1] = v.y;
                a[4 * k + 2] = v.z;
                a[4 * k + 3] = v.w;
            }
        }
        if (fast) {
#pragma unroll
            for (int k = 0; k < 16; ++k) c[k] = sq_code32_shr(a[k], sh, half_m1);
        } else {
#pragma unroll
            for (int k = 0; k < 16; ++k) c[k] = sq_code32(a[k], t);
        }
        int s = 0;
#pragma unroll
        for (int k = 0; k < 16; ++k) s += c[k];
        sum += s;
        reinterpret_cast<int4 *>(dst)[i] =
            make_int4((int)pack4(c[0], c[1], c[2], c[3]), (int)pack4(c[4], c[5], c[6], c[7]),
                      (int)pack4(c[8], c[9], c[10], c[11]), (int)pack4(c[12], c[13], c[14], c[15]));
        if (kJoin) {
            const int4 bq = __ldg(reinterpret_cast<const int4 *>(join.b) + i);
            const int8_t *bb = reinterpret_cast<const int8_t *>(&bq);
            const uint32_t gate = join.mask_b ? (uint32_t)__ldg(reinterpret_cast<const uint16_t *>(join.mask_b) + i) : 0xffffu;
            const uint32_t nm = join.next_mask ? (uint32_t)__ldg(reinterpret_cast<const uint16_t *>(join.next_mask) + i) : 0u;
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                const int bv = ((gate >> k) & 1u) ? (int)bb[k] : 0;
                unsigned long long u;
                if (j_narrow) {
                    u = (unsigned long long)(uint32_t)abs(c[k] * j_ma + bv * j_mb);
                } else {
                    const long long v = join_one(c[k], bv, js);
                    u = (unsigned long long)(v < 0 ? -v : v);
                }
                jmx = u > jmx ? u : jmx;
                if ((nm >> k) & 1u) jmxm = u > jmxm ? u : jmxm;
            }
        }
        if (kNext) {
            const uint32_t bits = (uint32_t)__ldg(reinterpret_cast<const uint16_t *>(next.mask) + i);
            int e1[16], c3[16], a1 = 0;
#pragma unroll
            for (int k = 0; k < 16; ++k) {
                e1[k] = ((bits >> k) & 1u) ? c[k] : 0;
                a1 += e1[k];
                c3[k] = next_head_code(nh, e1[k]);
            }
            s1 += a1;
            if (next.x2) {
                const int4 lo = __ldg(reinterpret_cast<const int4 *>(next.x2) + 2 * i);
                const int4 hi = __ldg(reinterpret_cast<const int4 *>(next.x2) + 2 * i + 1);
                const int16_t *pl = reinterpret_cast<const int16_t *>(&lo), *ph = reinterpret_cast<const int16_t *>(&hi);
                int a2 = 0;  // |e1 * x2| < 2^22, 16 terms
#pragma unroll
                for (int k = 0; k < 8; ++k) a2 += e1[k] * pl[k] + e1[8 + k] * ph[k];
                s2 += a2;
            }
            reinterpret_cast<int4 *>(next.e3)[i] =
                make_int4((int)pack4(c3[0], c3[1], c3[2], c3[3]), (int)pack4(c3[4], c3[5], c3[6], c3[7]),
                          (int)pack4(c3[8], c3[9], c3[10], c3[11]), (int)pack4(c3[12], c3[13], c3[14], c3[15]));
        }
    }
    if (!kNext && !kJoin)
        for (size_t i = n16 * 16 + (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
            const int c = sq_code32(src[i], t);
            sum += c;
            dst[i] = (int8_t)c;
        }
    if (sum_codes) {
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
    if (kJoin) {
        // the join's second pass (the next kernel on the stream) reads these cells and puts them back to zero
        jmx = block_max_u64(jmx);
        jmxm = block_max_u64(jmxm);
        if (threadIdx.x == 0) {
            if (jmx) atomicMax(&dev->absmax_u64, jmx);
            if (jmxm) atomicMax(&dev->absmax2_u64, jmxm);
        }
    }
    if (last_block_done(dev)) {
        if (sum_codes) *sum_codes = (long long)atomicExch(reinterpret_cast<unsigned long long *>(&dev->sum0), 0ull);
        dev->absmax_u32 = 0;
        if (kNext) {
            dev->absmax_u64 = 0;
            const long long t1 = (long long)atomicExch(reinterpret_cast<unsigned long long *>(&dev->sum1), 0ull);
            const long long t2 = (long long)atomicExch(reinterpret_cast<unsigned long long *>(&dev->sum2), 0ull);
            if (next.sum_e1) *next.sum_e1 = t1;
            if (next.sum_e1x2) *next.sum_e1x2 = t2;
        }
    }
}

// Q_e for a strided 1x1 filter: only the pixels (y, x) with y and x multiples of the stride receive an error, the
// others are exactly zero.  The GEMM leaves its sums compact, [n][hq][wq][c]; this kernel writes the full tensor
// [n][h][w][c], codes on the grid and zeros elsewhere, so neither a cleared full-size int32 tensor nor a pass over
// it is needed.  A thread writes 16 channels of one pixel.
__global__ void sq_i32_scatter_kernel(const int32_t *__restrict__ src, const int32_t *src_exp, int exp_bias, int n_img, int hh,
                                      int ww, int c, int stride, int hq, int wq, int8_t *dst, int32_t *dst_exp,
                                      long long *sum_codes, DeviceState *dev)
{
    const uint32_t M = dev->absmax_u32;
    const int t = M ? round_log2_u32(M) : 7;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        const int p_in = (src_exp ? *src_exp : 0) + exp_bias;
        *dst_exp = M ? p_in + t - 7 : p_in;
        if (!M) atomicOr(&dev->status, EOQ_DEV_SQ_ZERO);
    }
    long long sum = 0;
    const uint32_t groups = (uint32_t)c / 16u;
    const size_t items = (size_t)n_img * hh * ww * groups;  // fits 32 bits (checked by the launcher)
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < items; i += (size_t)gridDim.x * blockDim.x) {
        const uint32_t pix = (uint32_t)i / groups, g = (uint32_t)i - pix * groups;
        const uint32_t row = pix / (uint32_t)ww, x = pix - row * (uint32_t)ww;
        const uint32_t img = row / (uint32_t)hh, y = row - img * (uint32_t)hh;
        int4 out = make_int4(0, 0, 0, 0);
        if (y % (uint32_t)stride == 0 && x % (uint32_t)stride == 0) {
            const size_t q = (((size_t)img * hq + y / (uint32_t)stride) * wq + x / (uint32_t)stride) * c + g * 16u;
            const int4 *s4 = reinterpret_cast<const int4 *>(src + q);
            int cdes[16];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int4 v = __ldcs(s4 + k);
                cdes[4 * k + 0] = sq_code32(v.x, t);
                cdes[4 * k + 1] = sq_code32(v.y, t);
                cdes[4 * k + 2] = sq_code32(v.z, t);
                cdes[4 * k + 3] = sq_code32(v.w, t);
            }
            int sc = 0;
#pragma unroll
            for (int k = 0; k < 16; ++k) sc += cdes[k];
            sum += sc;
            out = make_int4((int)pack4(cdes[0], cdes[1], cdes[2], cdes[3]), (int)pack4(cdes[4], cdes[5], cdes[6], cdes[7]),
                            (int)pack4(cdes[8], cdes[9], cdes[10], cdes[11]), (int)pack4(cdes[12], cdes[13], cdes[14], cdes[15]));
        }
        reinterpret_cast<int4 *>(dst)[i] = out;
    }
    if (sum_codes) {
        sum = block_sum_i64(sum);
        if (threadIdx.x == 0 && sum) atomicAdd(reinterpret_cast<unsigned long long *>(&dev->sum0), (unsigned long long)sum);
    }
    if (last_block_done(dev)) {
        if (sum_codes) *sum_codes = (long long)atomicExch(reinterpret_cast<unsigned long long *>(&dev->sum0), 0ull);
        dev->absmax_u32 = 0;
    }
}

// ------------------------------------------------------------------ int64 -> SQ (Q_g after the weight gradient)

// Last step before Q_g: sums the int32 split-K slices of the patch kernel into int64 (exact whatever the reduction
// length), or takes the int64 sums the other kernel left in `acc`; adds the b1 term of x1 = x0 + b1 (b1 times the
// sum of the error over the pixels whose tap falls inside the image); optionally copies the exact sums out; and
// reduces max |.|.  A block of 256 threads is (256 / groups) elements x `groups` slice groups: every thread adds
// its share of the slices with independent, coalesced loads and the groups meet in shared memory.
// (bx of nblocks): the block's place among the blocks of its tensor; max_cell: where max |.| is reduced (null: not at all)
__device__ __forceinline__ void wgrad_finalize_body(const int32_t *__restrict__ parts, int num_parts, int groups, size_t n, long long *acc,
                                                    const long long *__restrict__ tap_sums, size_t replica_stride, int32_t b1_c,
                                                    const int32_t *b1_dev, int c_in, long long *copy_out,
                                                    unsigned long long *max_cell, int bx, int nblocks)
{
    __shared__ long long part[256];
    if (b1_dev) b1_c = clampi(__ldg(b1_dev), -32768, 32767);
    const int bw = 256 / groups, tx = threadIdx.x % bw, ty = threadIdx.x / bw;
    unsigned long long mx = 0;
    for (size_t base = (size_t)bx * bw; base < n; base += (size_t)nblocks * bw) {
        const size_t i = base + tx;
        long long v = 0;
        if (parts) {
            if (i < n) {
                // four slices per round: their loads are independent and in flight together
                int s = ty;
                for (; s + 3 * groups < num_parts; s += 4 * groups) {
                    const int32_t a0 = __ldg(parts + (size_t)s * n + i), a1 = __ldg(parts + (size_t)(s + groups) * n + i);
                    const int32_t a2 = __ldg(parts + (size_t)(s + 2 * groups) * n + i), a3 = __ldg(parts + (size_t)(s + 3 * groups) * n + i);
                    v += ((long long)a0 + a1) + ((long long)a2 + a3);
                }
                for (; s < num_parts; s += groups) v += (long long)__ldg(parts + (size_t)s * n + i);
            }
            if (groups > 1) {
                part[threadIdx.x] = v;
                __syncthreads();
                if (ty == 0) {
                    v = 0;
                    for (int k = 0; k < groups; ++k) v += part[k * bw + tx];
                }
                __syncthreads();
            }
        } else if (i < n) {
            v = acc[i];
        }
        if (ty == 0 && i < n) {
            if (tap_sums) {  // index of (oc, tap); a 32-bit division whenever the tensor allows it
                const long long *t = tap_sums + (n <= 0xffffffffull ? (size_t)((uint32_t)i / (uint32_t)c_in) : i / (size_t)c_in);
                long long ts = 0;
#pragma unroll
                for (int r = 0; r < kTapReplicas; ++r) ts += __ldg(t + (size_t)r * replica_stride);
                v += (long long)b1_c * ts;
            }
            if (parts || tap_sums) acc[i] = v;
            if (copy_out) copy_out[i] = v;
            const unsigned long long a = (unsigned long long)(v < 0 ? -v : v);
            mx = a > mx ? a : mx;
        }
    }
    mx = block_max_u64(mx);
    if (threadIdx.x == 0 && mx && max_cell) atomicMax(max_cell, mx);
}

__global__ void wgrad_finalize_kernel(const int32_t *__restrict__ parts, int num_parts, int groups, size_t n, long long *acc,
                                      const long long *__restrict__ tap_sums, size_t replica_stride, int32_t b1_c,
                                      const int32_t *b1_dev, int c_in, long long *copy_out, DeviceState *dev, int sums_only)
{
    // sums_only: the sums are completed elsewhere (an all-reduce over replicas) before their maximum is taken
    wgrad_finalize_body(parts, num_parts, groups, n, acc, tap_sums, replica_stride, b1_c, b1_dev, c_in, copy_out,
                        sums_only ? nullptr : &dev->absmax_u64, (int)blockIdx.x, (int)gridDim.x);
}

// max |.| of int64 sums into the handle's 64-bit cell (used when the sums were completed by an all-reduce)
__global__ void absmax_i64_kernel(const long long *__restrict__ src, size_t n, DeviceState *dev)
{
    unsigned long long mx = 0;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x) {
        const long long v = src[i];
        const unsigned long long a = (unsigned long long)(v < 0 ? -v : v);
        mx = a > mx ? a : mx;
    }
    mx = block_max_u64(mx);
    if (threadIdx.x == 0 && mx) atomicMax(&dev->absmax_u64, mx);
}

// (bx of nblocks) as above; M: the tensor's max |.|; status: where a zero tensor is flagged
__device__ __forceinline__ void sq_i64_body(const long long *__restrict__ src, const int32_t *src_exp, int exp_bias, size_t n, int8_t *dst,
                                            int32_t *dst_exp, unsigned long long M, unsigned *status, int bx, int nblocks)
{
    const int t = M ? round_log2_u64(M) : 7;
    if (bx == 0 && threadIdx.x == 0) {
        const int p_in = (src_exp ? *src_exp : 0) + exp_bias;
        *dst_exp = M ? p_in + t - 7 : p_in;
        if (!M) atomicOr(status, EOQ_DEV_SQ_ZERO);
    }
    // four codes per thread and round (one 32-bit store); n is a multiple of 4 for every weight tensor with padded channels
    const size_t n4 = n / 4;
    for (size_t i = (size_t)bx * blockDim.x + threadIdx.x; i < n4; i += (size_t)nblocks * blockDim.x) {
        const longlong2 a = __ldg(reinterpret_cast<const longlong2 *>(src) + 2 * i);
        const longlong2 b = __ldg(reinterpret_cast<const longlong2 *>(src) + 2 * i + 1);
        reinterpret_cast<uint32_t *>(dst)[i] = pack4(sq_code64(a.x, t), sq_code64(a.y, t), sq_code64(b.x, t), sq_code64(b.y, t));
    }
    for (size_t i = n4 * 4 + (size_t)bx * blockDim.x + threadIdx.x; i < n; i += (size_t)nblocks * blockDim.x)
        dst[i] = (int8_t)sq_code64(src[i], t);
}

__global__ void sq_i64_kernel(const long long *__restrict__ src, const int32_t *src_exp, int exp_bias, size_t n,
                              int8_t *dst, int32_t *dst_exp, DeviceState *dev)
{
    sq_i64_body(src, src_exp, exp_bias, n, dst, dst_exp, dev->absmax_u64, &dev->status, (int)blockIdx.x, (int)gridDim.x);
    if (last_block_done(dev)) dev->absmax_u64 = 0;
}

// ------------------------------------------------------------------ head of the error chain

__device__ __forceinline__ void unpack16(const int4 &v, int (&o)[16])
{
    const int8_t *b = reinterpret_cast<const int8_t *>(&v);
#pragma unroll
    for (int k = 0; k < 16; ++k) o[k] = b[k];
}

// Pass 1: max |e1| and the sums behind g_b2 and g_gamma, with e1 = e0 * [x4 > 0].
// Expands 4 mask bits into 4 byte masks (0x00 / 0xff).
__device__ __forceinline__ uint32_t bits_to_bytes(uint32_t nibble)
{
    return (((nibble & 0xfu) * 0x00204081u) & 0x01010101u) * 0xffu;
}

__global__ void prescale_reduce_kernel(const int8_t *__restrict__ e0, const uint8_t *__restrict__ mask,
                                       const int16_t *__restrict__ x2, size_t n16, DeviceState *dev)
{
    uint32_t mx4 = 0;  // four running byte maxima of |e1|
    long long s1 = 0, s2 = 0;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    // four independent 16-element groups per iteration keep enough loads in flight to cover DRAM latency
    for (size_t i0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i0 < n16; i0 += 4 * stride) {
        int4 ev[4];
        uint32_t mv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const size_t i = i0 + u * stride;
            const bool in = i < n16;
            ev[u] = in ? __ldg(reinterpret_cast<const int4 *>(e0) + i) : make_int4(0, 0, 0, 0);
            mv[u] = (in && mask) ? (uint32_t)__ldg(reinterpret_cast<const uint16_t *>(mask) + i) : 0xffffu;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t w[4] = {(uint32_t)ev[u].x, (uint32_t)ev[u].y, (uint32_t)ev[u].z, (uint32_t)ev[u].w};
            int a1 = 0;
            uint32_t e1w[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                e1w[q] = w[q] & bits_to_bytes(mv[u] >> (4 * q));  // e1 = e0 * [x4 > 0], four codes per word
                mx4 = __vmaxu4(mx4, __vabsss4(e1w[q]));
                a1 = __dp4a((int)e1w[q], 0x01010101, a1);
            }
            s1 += a1;
            if (x2) {
                const size_t i = i0 + u * stride;
                if (i < n16) {
                    const int4 lo = __ldg(reinterpret_cast<const int4 *>(x2) + 2 * i);
                    const int4 hi = __ldg(reinterpret_cast<const int4 *>(x2) + 2 * i + 1);
                    const int16_t *pl = reinterpret_cast<const int16_t *>(&lo), *ph = reinterpret_cast<const int16_t *>(&hi);
                    const int8_t *eb = reinterpret_cast<const int8_t *>(e1w);
                    int a2 = 0;  // |e1 * x2| < 2^22, 16 terms
#pragma unroll
                    for (int k = 0; k < 8; ++k) a2 += (int)eb[k] * pl[k] + (int)eb[8 + k] * ph[k];
                    s2 += a2;
                }
            }
        }
    }
    uint32_t mx = max(max(mx4 & 0xffu, (mx4 >> 8) & 0xffu), max((mx4 >> 16) & 0xffu, mx4 >> 24));
    mx = (uint32_t)block_max_u64(mx);
    s1 = block_sum_i64(s1);
    s2 = block_sum_i64(s2);
    if (threadIdx.x == 0) {
        if (mx) atomicMax(&dev->absmax_u32, mx);
        if (s1) atomicAdd(reinterpret_cast<unsigned long long *>(&dev->sum0), (unsigned long long)s1);
        if (s2) atomicAdd(reinterpret_cast<unsigned long long *>(&dev->sum1), (unsigned long long)s2);
    }
}

// Pass 2: e3 = Q_e(gamma * e1) under the reduced maximum.
// gamma of a launch: the host value, or the code read from device memory (clamped to 16 bits, EOQ_DEV_RANGE raised)
__device__ __forceinline__ int32_t load_gamma(int32_t gamma_c, const int32_t *gamma_dev, DeviceState *dev)
{
    if (!gamma_dev) return gamma_c;
    int32_t g = __ldg(gamma_dev);
    if (g < -32768 || g > 32767) {
        if (blockIdx.x == 0 && threadIdx.x == 0) atomicOr(&dev->status, EOQ_DEV_RANGE);
        g = clampi(g, -32768, 32767);
    }
    return g;
}

__global__ void prescale_apply_kernel(const int8_t *__restrict__ e0, const int32_t *e0_exp,
                                      const uint8_t *__restrict__ mask, size_t n16, int32_t gamma_c,
                                      const int32_t *gamma_dev, int8_t *e3, int32_t *e3_exp, long long *sum_e1,
                                      long long *sum_e1x2, DeviceState *dev)
{
    gamma_c = load_gamma(gamma_c, gamma_dev, dev);
    const uint32_t M = dev->absmax_u32 * (uint32_t)abs(gamma_c);  // max |gamma * e1| < 2^7 * 2^15
    const int t = M ? round_log2_u32(M) : 7;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        const int p_in = *e0_exp - 7;
        *e3_exp = M ? p_in + t - 7 : p_in;
        if (!M) atomicOr(&dev->status, EOQ_DEV_SQ_ZERO);
        if (sum_e1) *sum_e1 = dev->sum0;
        if (sum_e1x2) *sum_e1x2 = dev->sum1;
    }
    // R(v * 2^(7-t)) for v = gamma * e1 (|v| < 2^22) on the floating-point pipe: kMagic + v read as a float is
    // 1.5 * 2^23 + v exactly; one fused multiply-add forms 1.5 * 2^23 + v * 2^(7-t) (the products are exact, the sum
    // is rounded once, to nearest even at unit spacing), so the low bits of the result are the rounded quotient.
    // For t < 7 the scaling is a left shift and nothing is rounded; either way |result| < 2^22 keeps the binade.
    constexpr uint32_t kMagic = 0x4B400000u;  // 1.5 * 2^23
    const float scale = __int_as_float((127 + 7 - t) << 23);  // 2^(7-t), t in [0, 22]
    const float rest = 12582912.0f - 12582912.0f * scale;  // exact: a multiple of a power of two below 2^31
    const uint32_t g = (uint32_t)gamma_c;
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i0 < n16; i0 += 4 * stride) {
        int4 ev[4];
        uint32_t mv[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const size_t i = i0 + u * stride;
            const bool in = i < n16;
            ev[u] = in ? __ldg(reinterpret_cast<const int4 *>(e0) + i) : make_int4(0, 0, 0, 0);
            mv[u] = (in && mask) ? (uint32_t)__ldg(reinterpret_cast<const uint16_t *>(mask) + i) : 0xffffu;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const size_t i = i0 + u * stride;
            if (i >= n16) continue;
            const uint32_t w[4] = {(uint32_t)ev[u].x, (uint32_t)ev[u].y, (uint32_t)ev[u].z, (uint32_t)ev[u].w};
            int c[16];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const uint32_t e1w = w[q] & bits_to_bytes(mv[u] >> (4 * q));  // e1 = e0 * [x4 > 0], four codes
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const int32_t e1 = (int32_t)(int8_t)(e1w >> (8 * k));
                    const uint32_t biased = g * (uint32_t)e1 + kMagic;
                    const uint32_t r = __float_as_uint(__fmaf_rn(__uint_as_float(biased), scale, rest));
                    c[4 * q + k] = clampi((int32_t)(r - kMagic), -127, 127);
                }
            }
            reinterpret_cast<int4 *>(e3)[i] =
                make_int4((int)pack4(c[0], c[1], c[2], c[3]), (int)pack4(c[4], c[5], c[6], c[7]),
                          (int)pack4(c[8], c[9], c[10], c[11]), (int)pack4(c[12], c[13], c[14], c[15]));
        }
    }
    if (last_block_done(dev)) {
        dev->absmax_u32 = 0;
        dev->sum0 = 0;
        dev->sum1 = 0;
    }
}

// Both passes of the error head in one kernel, for tensors small enough that every thread keeps its share of e1
// (up to kFusedGroups groups of 16 codes) in registers between the passes: e0 and the mask are read once and no
// second launch is needed.  Between the passes all blocks meet at a grid-wide barrier (a counter in the handle's
// device state), so the kernel is launched cooperatively: the launch guarantees that all its blocks are resident
// together.  The wait is bounded like every wait of the library; on timeout the kernel flags it and writes nothing.
constexpr int kFusedGroups = 6;
__global__ void __launch_bounds__(kThreads)
prescale_fused_kernel(const int8_t *__restrict__ e0, const int32_t *e0_exp, const uint8_t *__restrict__ mask,
                      const int16_t *__restrict__ x2, size_t n16, int32_t gamma_c, const int32_t *gamma_dev, int8_t *e3,
                      int32_t *e3_exp, long long *sum_e1, long long *sum_e1x2, DeviceState *dev, unsigned expected_blocks,
                      uint32_t spin_limit)
{
    __shared__ unsigned go_s;
    gamma_c = load_gamma(gamma_c, gamma_dev, dev);
    const size_t stride = (size_t)gridDim.x * blockDim.x;
    const size_t i0 = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    uint32_t e1w[kFusedGroups][4];
    uint32_t mx4 = 0;
    long long s1 = 0, s2 = 0;
    {
        int4 ev[kFusedGroups];
        uint32_t mv[kFusedGroups];
#pragma unroll
        for (int u = 0; u < kFusedGroups; ++u) {
            const size_t i = i0 + u * stride;
            const bool in = i < n16;
            ev[u] = in ? __ldg(reinterpret_cast<const int4 *>(e0) + i) : make_int4(0, 0, 0, 0);
            mv[u] = (in && mask) ? (uint32_t)__ldg(reinterpret_cast<const uint16_t *>(mask) + i) : 0xffffu;
        }
#pragma unroll
        for (int u = 0; u < kFusedGroups; ++u) {
            const uint32_t w[4] = {(uint32_t)ev[u].x, (uint32_t)ev[u].y, (uint32_t)ev[u].z, (uint32_t)ev[u].w};
            int a1 = 0;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                e1w[u][q] = w[q] & bits_to_bytes(mv[u] >> (4 * q));  // e1 = e0 * [x4 > 0], four codes per word
                mx4 = __vmaxu4(mx4, __vabsss4(e1w[u][q]));
                a1 = __dp4a((int)e1w[u][q], 0x01010101, a1);
            }
            s1 += a1;
            const size_t i = i0 + u * stride;
            if (x2 && i < n16) {
                const int4 lo = __ldg(reinterpret_cast<const int4 *>(x2) + 2 * i);
                const int4 hi = __ldg(reinterpret_cast<const int4 *>(x2) + 2 * i + 1);
                const int16_t *pl = reinterpret_cast<const int16_t *>(&lo), *ph = reinterpret_cast<const int16_t *>(&hi);
                const int8_t *eb = reinterpret_cast<const int8_t *>(e1w[u]);
                int a2 = 0;  // |e1 * x2| < 2^22, 16 terms
#pragma unroll
                for (int k = 0; k < 8; ++k) a2 += (int)eb[k] * pl[k] + (int)eb[8 + k] * ph[k];
                s2 += a2;
            }
        }
    }
    uint32_t mx = max(max(mx4 & 0xffu, (mx4 >> 8) & 0xffu), max((mx4 >> 16) & 0xffu, mx4 >> 24));
    mx = (uint32_t)block_max_u64(mx);
    s1 = block_sum_i64(s1);
    s2 = block_sum_i64(s2);
    if (threadIdx.x == 0) {
        if (mx) atomicMax(&dev->absmax_u32, mx);
        if (s1) atomicAdd(reinterpret_cast<unsigned long long *>(&dev->sum0), (unsigned long long)s1);
        if (s2) atomicAdd(reinterpret_cast<unsigned long long *>(&dev->sum1), (unsigned long long)s2);
        // grid-wide barrier: every block's contribution is in the cells once all have arrived
        __threadfence();
        atomicAdd(&dev->arrivals, 1u);
        unsigned ok = 0;
        // (expected_blocks is the grid size; a larger value, which only the library's self-test passes, makes this
        // wait run out)
        for (uint32_t it = 0; it < spin_limit; ++it) {
            if (*reinterpret_cast<volatile unsigned *>(&dev->arrivals) >= expected_blocks) { ok = 1; break; }
            __nanosleep(100);
        }
        if (!ok) atomicOr(&dev->status, EOQ_DEV_TIMEOUT);
        __threadfence();
        go_s = ok;
    }
    __syncthreads();
    if (!go_s) return;
    const uint32_t M = *reinterpret_cast<volatile unsigned *>(&dev->absmax_u32) * (uint32_t)abs(gamma_c);
    const int t = M ? round_log2_u32(M) : 7;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        const int p_in = *e0_exp - 7;
        *e3_exp = M ? p_in + t - 7 : p_in;
        if (!M) atomicOr(&dev->status, EOQ_DEV_SQ_ZERO);
        if (sum_e1) *sum_e1 = *reinterpret_cast<volatile long long *>(&dev->sum0);
        if (sum_e1x2) *sum_e1x2 = *reinterpret_cast<volatile long long *>(&dev->sum1);
    }
    // same rounding as prescale_apply_kernel: R(gamma * e1 * 2^(7-t)) with one FMA
    constexpr uint32_t kMagic = 0x4B400000u;
    const float scale = __int_as_float((127 + 7 - t) << 23);
    const float rest = 12582912.0f - 12582912.0f * scale;
    const uint32_t g = (uint32_t)gamma_c;
#pragma unroll
    for (int u = 0; u < kFusedGroups; ++u) {
        const size_t i = i0 + u * stride;
        if (i >= n16) continue;
        int c[16];
#pragma unroll
        for (int q = 0; q < 4; ++q)
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const int32_t e1 = (int32_t)(int8_t)(e1w[u][q] >> (8 * k));
                const uint32_t r = __float_as_uint(__fmaf_rn(__uint_as_float(g * (uint32_t)e1 + kMagic), scale, rest));
                c[4 * q + k] = clampi((int32_t)(r - kMagic), -127, 127);
            }
        reinterpret_cast<int4 *>(e3)[i] =
            make_int4((int)pack4(c[0], c[1], c[2], c[3]), (int)pack4(c[4], c[5], c[6], c[7]),
                      (int)pack4(c[8], c[9], c[10], c[11]), (int)pack4(c[12], c[13], c[14], c[15]));
    }
    if (last_block_done(dev)) {
        dev->absmax_u32 = 0;
        dev->sum0 = 0;
        dev->sum1 = 0;
        dev->arrivals = 0;
    }
}

// ------------------------------------------------------------------ 8-bit update

constexpr int kUpdChunk = 64;           // tensors per launch
constexpr int kUpdElemsPerBlock = 8192;  // elements one block covers

struct UpdateBatch {
    UpdateTensor t[kUpdChunk];
    int first_block[kUpdChunk + 1];
    int num;
    int tensor_base;  // index of t[0] in the whole call (cell of its maximum, counter of the hash)
};

__device__ __forceinline__ int find_tensor(const UpdateBatch &b, int block)
{
    int k = 0;
    while (k + 1 < b.num && block >= b.first_block[k + 1]) ++k;
    return k;
}

__global__ void update_absmax_kernel(const __grid_constant__ UpdateBatch b, DeviceState *dev)
{
    const int k = find_tensor(b, blockIdx.x);
    const UpdateTensor &T = b.t[k];
    const size_t begin = (size_t)(blockIdx.x - b.first_block[k]) * kUpdElemsPerBlock;
    const size_t end = min((size_t)T.n, begin + kUpdElemsPerBlock);
    uint32_t mx = 0;
    if (begin < end) {
        // 16-byte path when the tensor base allows it (it always does for 16-byte aligned tensors)
        const bool vec = (reinterpret_cast<uintptr_t>(T.g) & 15) == 0;
        size_t i = begin + (size_t)threadIdx.x * 16;
        if (vec) {
            for (; i + 16 <= end; i += (size_t)blockDim.x * 16) {
                int e[16];
                unpack16(__ldg(reinterpret_cast<const int4 *>(T.g + i)), e);
#pragma unroll
                for (int q = 0; q < 16; ++q) mx = max(mx, (uint32_t)abs(e[q]));
            }
        }
        // remaining elements of this block's range
        const size_t tail = vec ? begin + ((end - begin) / 16) * 16 : begin;
        for (size_t j = tail + threadIdx.x; j < end; j += blockDim.x) mx = max(mx, (uint32_t)abs((int)T.g[j]));
    }
    mx = (uint32_t)block_max_u64(mx);
    if (threadIdx.x == 0 && mx) atomicMax(&dev->tensor_absmax[b.tensor_base + k], mx);
}

// SplitMix64 output function (Steele, Lea, Flood 2014) as a counter hash.
__device__ __forceinline__ unsigned long long mix64(unsigned long long z)
{
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}

// w <- Q_w(w - Q_u(lr * g)) on int8 codes (Sec. 3.2.3).
__device__ __forceinline__ int update_one(int w, int g, int lr_mant, int t, int d, int stochastic,
                                          unsigned long long key, unsigned long long idx)
{
    const int u = sq_code32(lr_mant * g, t);
    long long next;
    if (d >= 0) {
        next = (long long)w - (long long)u * (1ll << min(d, 40));
    } else if (-d > 40) {
        next = w;
    } else {
        const int s = -d;
        const long long v = (long long)w * (1ll << s) - u;
        if (!stochastic) {
            next = rne_shr64(v, s);
        } else {
            const unsigned long long r = mix64(key + 0x9E3779B97F4A7C15ull * (idx + 1)) & ((1ull << s) - 1ull);
            next = (v + (long long)r) >> s;
        }
    }
    return (int)(next < -127 ? -127 : (next > 127 ? 127 : next));
}

__global__ void update_apply_kernel(const __grid_constant__ UpdateBatch b, int32_t lr_mant, int32_t lr_exp,
                                    int stochastic, unsigned long long seed, unsigned long long step,
                                    const unsigned long long *step_dev, DeviceState *dev)
{
    if (step_dev) step = *step_dev;  // device-resident step counter (bumped by step_bump_kernel behind the call)
    const int k = find_tensor(b, blockIdx.x);
    const UpdateTensor &T = b.t[k];
    const uint32_t M = dev->tensor_absmax[b.tensor_base + k] * (uint32_t)lr_mant;  // max |lr_mant * g| < 2^15
    if (M == 0) {
        if (threadIdx.x == 0 && blockIdx.x == b.first_block[k]) atomicOr(&dev->status, EOQ_DEV_SQ_ZERO);
        return;  // u = 0: the weights keep their codes
    }
    const int t = round_log2_u32(M);
    const int d = (__ldg(T.g_exp) + lr_exp + t - 7) + 7;  // exponent of u, relative to the weight grid 2^-7
    unsigned long long key = 0;
    if (stochastic) {
        key = mix64(seed + 0x9E3779B97F4A7C15ull * (step + 1));
        key = mix64(key + 0x9E3779B97F4A7C15ull * ((unsigned long long)(b.tensor_base + k) + 1));
    }
    const size_t begin = (size_t)(blockIdx.x - b.first_block[k]) * kUpdElemsPerBlock;
    const size_t end = min((size_t)T.n, begin + kUpdElemsPerBlock);
    if (begin >= end) return;
    const bool vec = ((reinterpret_cast<uintptr_t>(T.g) | reinterpret_cast<uintptr_t>(T.w)) & 15) == 0;
    if (vec) {
        for (size_t i = begin + (size_t)threadIdx.x * 16; i + 16 <= end; i += (size_t)blockDim.x * 16) {
            int gv[16], wv[16], c[16];
            unpack16(__ldg(reinterpret_cast<const int4 *>(T.g + i)), gv);
            unpack16(*reinterpret_cast<const int4 *>(T.w + i), wv);
#pragma unroll
            for (int q = 0; q < 16; ++q) c[q] = update_one(wv[q], gv[q], lr_mant, t, d, stochastic, key, i + q);
            *reinterpret_cast<int4 *>(T.w + i) =
                make_int4((int)pack4(c[0], c[1], c[2], c[3]), (int)pack4(c[4], c[5], c[6], c[7]),
                          (int)pack4(c[8], c[9], c[10], c[11]), (int)pack4(c[12], c[13], c[14], c[15]));
        }
    }
    const size_t tail = vec ? begin + ((end - begin) / 16) * 16 : begin;
    for (size_t j = tail + threadIdx.x; j < end; j += blockDim.x)
        T.w[j] = (int8_t)update_one(T.w[j], T.g[j], lr_mant, t, d, stochastic, key, j);
}

// The update with a k_u-bit update quantizer and k_m-bit master codes (Sec. 3.2.3 compares the 8-bit update with a
// 24-bit one): u = SQ(lr g, k_u), master <- CQ(master - u, k_m) on the grid 2^-(k_m - 1), w = Q_w(master).
__global__ void update_wide_apply_kernel(const __grid_constant__ UpdateBatch b, int32_t lr_mant, int32_t lr_exp, int k_u, int k_m,
                                         int stochastic, unsigned long long seed, unsigned long long step,
                                         const unsigned long long *step_dev, DeviceState *dev)
{
    if (step_dev) step = *step_dev;
    const int k = find_tensor(b, blockIdx.x);
    const UpdateTensor &T = b.t[k];
    const uint32_t M = dev->tensor_absmax[b.tensor_base + k] * (uint32_t)lr_mant;
    if (M == 0) {
        if (threadIdx.x == 0 && blockIdx.x == b.first_block[k]) atomicOr(&dev->status, EOQ_DEV_SQ_ZERO);
        return;
    }
    const int t = round_log2_u32(M);
    const int su = t - (k_u - 1);                                  // u code = R(lr_mant g / 2^su)
    const int d = (__ldg(T.g_exp) + lr_exp + su) + (k_m - 1);      // exponent of u relative to the master grid
    const long long lim_u = (1ll << (k_u - 1)) - 1, lim_m = (1ll << (k_m - 1)) - 1;
    unsigned long long key = 0;
    if (stochastic) {
        key = mix64(seed + 0x9E3779B97F4A7C15ull * (step + 1));
        key = mix64(key + 0x9E3779B97F4A7C15ull * ((unsigned long long)(b.tensor_base + k) + 1));
    }
    const size_t begin = (size_t)(blockIdx.x - b.first_block[k]) * kUpdElemsPerBlock;
    const size_t end = min((size_t)T.n, begin + kUpdElemsPerBlock);
    for (size_t j = begin + threadIdx.x; j < end; j += blockDim.x) {
        const long long a = (long long)lr_mant * T.g[j];
        long long u = su >= 0 ? rne_shr64(a, su) : a * (1ll << (-su));
        u = u < -lim_u ? -lim_u : (u > lim_u ? lim_u : u);
        const long long th = T.master[j];
        long long next;
        if (d >= 0) {
            next = th - u * (1ll << min(d, 38));
        } else if (-d > 38) {
            next = th;
        } else {
            const int s = -d;
            const long long v = th * (1ll << s) - u;
            if (!stochastic) {
                next = rne_shr64(v, s);
            } else {
                const unsigned long long r = mix64(key + 0x9E3779B97F4A7C15ull * (j + 1)) & ((1ull << s) - 1ull);
                next = (v + (long long)r) >> s;
            }
        }
        next = next < -lim_m ? -lim_m : (next > lim_m ? lim_m : next);
        T.master[j] = (int32_t)next;
        const long long w8 = rne_shr64(next, k_m - 8);
        T.w[j] = (int8_t)(w8 < -127 ? -127 : (w8 > 127 ? 127 : w8));
    }
}

__global__ void step_bump_kernel(unsigned long long *step_dev) { *step_dev += 1ull; }

// ------------------------------------------------------------------ layout helpers

// [n][rows][cols] -> [n][cols][rows] on bytes, 32 x 32 tiles through shared memory.
__global__ void transpose_bytes_kernel(const int8_t *__restrict__ src, int8_t *__restrict__ dst, int rows, int cols)
{
    __shared__ int8_t tile[32][33];
    const size_t img = (size_t)blockIdx.z * rows * cols;
    const int r0 = blockIdx.y * 32, c0 = blockIdx.x * 32;
    for (int r = threadIdx.y; r < 32; r += blockDim.y) {
        const int rr = r0 + r, cc = c0 + threadIdx.x;
        if (rr < rows && cc < cols) tile[r][threadIdx.x] = src[img + (size_t)rr * cols + cc];
    }
    __syncthreads();
    for (int c = threadIdx.y; c < 32; c += blockDim.y) {
        const int cc = c0 + c, rr = r0 + threadIdx.x;
        if (rr < rows && cc < cols) dst[img + (size_t)cc * rows + rr] = tile[threadIdx.x][c];
    }
}

// w[oc][tap][ic] -> wt[ic][tap][oc]
__global__ void weight_transpose_kernel(const int8_t *__restrict__ w, int8_t *__restrict__ wt, int c_out, int taps,
                                        int c_in)
{
    const size_t total = (size_t)c_out * taps * c_in;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
        const int oc = (int)(i % c_out);
        const int tap = (int)((i / c_out) % taps);
        const int ic = (int)(i / ((size_t)c_out * taps));
        wt[i] = w[((size_t)oc * taps + tap) * c_in + ic];
    }
}

// ------------------------------------------------------------------ b1 support

// table[class][oc] = sum over the taps valid for the class, and over ic, of w[oc][tap][ic]  (the forward
// pass adds b1 times this: conv(x0 + b1) = conv(x0) + b1 * conv(indicator of the image)).
// One block per output channel: warps reduce the taps' channel sums, then threads combine them per class.
__global__ void b1_weight_table_kernel(const int8_t *__restrict__ w, int32_t *table, eoq_conv_desc_t d, int ho, int wo,
                                       BorderClasses bc)
{
    __shared__ int32_t tap_sum[kMaxTaps];
    const int oc = blockIdx.x;
    const int taps = d.kh * d.kw;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    for (int t = warp; t < taps; t += nwarps) {
        const int4 *p = reinterpret_cast<const int4 *>(w + ((size_t)oc * taps + t) * d.c_in);
        int sum = 0;
        for (int i = lane; i < d.c_in / 16; i += 32) {
            const int4 v = __ldg(p + i);
            sum = __dp4a(v.x, 0x01010101, sum);
            sum = __dp4a(v.y, 0x01010101, sum);
            sum = __dp4a(v.z, 0x01010101, sum);
            sum = __dp4a(v.w, 0x01010101, sum);
        }
        if (d.c_in == 8 && lane == 0) {  // the 8-channel first layer: one 8-byte pixel per tap
            const int2 v = __ldg(reinterpret_cast<const int2 *>(p));
            sum = __dp4a(v.x, 0x01010101, sum);
            sum = __dp4a(v.y, 0x01010101, sum);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (lane == 0) tap_sum[t] = sum;
    }
    __syncthreads();
    for (int cls = threadIdx.x; cls < bc.nrc * bc.ncc; cls += blockDim.x) {
        const int rc = cls / bc.ncc, cc = cls % bc.ncc;
        int32_t sum = 0;
        for (int kh = 0; kh < d.kh; ++kh) {
            if (!tap_valid(rc, kh, ho, d.h, bc.nlo_h, bc.nhi_h, bc.nrc, d.stride, d.pad)) continue;
            for (int kw = 0; kw < d.kw; ++kw)
                if (tap_valid(cc, kw, wo, d.w, bc.nlo_w, bc.nhi_w, bc.ncc, d.stride, d.pad)) sum += tap_sum[kh * d.kw + kw];
        }
        table[(size_t)cls * d.c_out + oc] = sum;
    }
}

// What eoq_weight_prep derives from the weights of several layers in one launch: the b1 table of every layer
// (as b1_weight_table_kernel builds it) and, for a first layer on the filter-row path, the weights re-packed as
// [oc][kh][8][c_in] with zero taps.  One block per (layer, output channel).
__global__ void weight_prep_kernel(const __grid_constant__ PrepBatch b)
{
    __shared__ int32_t tap_sum[kMaxTaps];
    int k = 0;
    while (k + 1 < b.num && (int)blockIdx.x >= b.first_block[k + 1]) ++k;
    const PrepItem &it = b.item[k];
    const eoq_conv_desc_t &d = it.d;
    const BorderClasses &bc = it.bc;
    const int oc = blockIdx.x - b.first_block[k];
    const int taps = d.kh * d.kw;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    for (int t = warp; t < taps; t += nwarps) {
        const int8_t *p = it.w + ((size_t)oc * taps + t) * d.c_in;
        int sum = 0;
        for (int i = lane; i < d.c_in / 16; i += 32) {
            const int4 v = __ldg(reinterpret_cast<const int4 *>(p) + i);
            sum = __dp4a(v.x, 0x01010101, sum);
            sum = __dp4a(v.y, 0x01010101, sum);
            sum = __dp4a(v.z, 0x01010101, sum);
            sum = __dp4a(v.w, 0x01010101, sum);
        }
        if (d.c_in == 8 && lane == 0) {
            const int2 v = __ldg(reinterpret_cast<const int2 *>(p));
            sum = __dp4a(v.x, 0x01010101, sum);
            sum = __dp4a(v.y, 0x01010101, sum);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
        if (lane == 0) tap_sum[t] = sum;
    }
    __syncthreads();
    for (int cls = threadIdx.x; cls < bc.nrc * bc.ncc; cls += blockDim.x) {
        const int rc = cls / bc.ncc, cc = cls % bc.ncc;
        int32_t sum = 0;
        for (int kh = 0; kh < d.kh; ++kh) {
            if (!tap_valid(rc, kh, it.ho, d.h, bc.nlo_h, bc.nhi_h, bc.nrc, d.stride, d.pad)) continue;
            for (int kw = 0; kw < d.kw; ++kw)
                if (tap_valid(cc, kw, it.wo, d.w, bc.nlo_w, bc.nhi_w, bc.ncc, d.stride, d.pad)) sum += tap_sum[kh * d.kw + kw];
        }
        it.table[(size_t)cls * d.c_out + oc] = sum;
    }
    if (it.w_rows) {
        // this output channel's filter rows, each widened to 8 taps (c_in is 16 or 8: 4 or 2 words per tap)
        const int words = d.c_in / 4;
        const int32_t *src = reinterpret_cast<const int32_t *>(it.w) + (size_t)oc * taps * words;
        int32_t *dst = reinterpret_cast<int32_t *>(it.w_rows) + (size_t)oc * d.kh * 8 * words;
        for (int i = threadIdx.x; i < d.kh * 8 * words; i += blockDim.x) {
            const int r = i / (8 * words), t = (i / words) % 8, wd = i % words;
            dst[i] = t < d.kw ? __ldg(src + (r * d.kw + t) * words + wd) : 0;
        }
    }
}

// tap_sums[oc][tap] += sum of e3[n,y,x,oc] over the pixels for which the tap falls inside the image (the weight
// gradient adds b1 times this to every input channel).  Pixels are summed per border class first (the taps inside
// the image are the same for all pixels of a class).  A block owns a range of
// pixels and a slab of channels; a lane keeps 16 channels (one 128-bit load per pixel), so a warp covers
// 32 / (slab / 16) pixels per step.  Interior pixels (one class, almost all of a large image) accumulate in
// registers, border pixels in shared memory.
constexpr int kClassSlab = 128;
constexpr int kTapUnroll = 8;
// (bx, by): the block's place in the grid of its layer (pixel range, channel slab)
__device__ __forceinline__ void b1_tap_sums_body(const int8_t *__restrict__ e3, long long *tap_sums, size_t replica_stride, int c_out,
                                                 int ho, int wo, size_t pixels, int pixels_per_block, const BorderClasses &bc,
                                                 const eoq_conv_desc_t &d, int bx, int by)
{
    // the blocks spread their atomics over kTapReplicas copies of the sums (the consumer adds the copies): all
    // cells of one copy sit in a few kilobytes, i.e. behind one or two L2 slices, whose atomic rate bounds this kernel
    tap_sums += (size_t)(bx % kTapReplicas) * replica_stride;
    extern __shared__ int32_t cls_acc[];  // [classes][kClassSlab]
    const int classes = bc.nrc * bc.ncc;
    for (int i = threadIdx.x; i < classes * kClassSlab; i += blockDim.x) cls_acc[i] = 0;
    __syncthreads();
    const int slab_ch = min(kClassSlab, c_out - by * kClassSlab);  // channels of this slab (multiple of 16)
    const int lanes_per_pix = slab_ch / 16;
    const int pix_per_step = blockDim.x / lanes_per_pix;
    const int sub = threadIdx.x % lanes_per_pix, slot = threadIdx.x / lanes_per_pix;
    const int ch = by * kClassSlab + sub * 16;
    const int interior = (bc.nrc != ho && bc.ncc != wo) ? bc.nlo_h * bc.ncc + bc.nlo_w : -1;
    int acc[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) acc[k] = 0;
    const size_t begin = (size_t)bx * pixels_per_block;
    const size_t end = min(pixels, begin + (size_t)pixels_per_block);
    const bool small = pixels <= 0xffffffffull;
    if (slot < pix_per_step) {
        // kTapUnroll pixels per round: their loads are issued together and are in flight side by side
        for (size_t p0 = begin + slot; p0 < end; p0 += kTapUnroll * (size_t)pix_per_step) {
            int4 v[kTapUnroll];
            int cls[kTapUnroll];
#pragma unroll
            for (int u = 0; u < kTapUnroll; ++u) {
                const size_t p = p0 + (size_t)u * pix_per_step;
                cls[u] = -2;  // beyond the block's range
                v[u] = make_int4(0, 0, 0, 0);
                if (p < end) {
                    int x, y;
                    if (small) {  // 32-bit index arithmetic (a 64-bit division costs more than the rest of the pixel's work)
                        const uint32_t q = (uint32_t)p / (uint32_t)wo;
                        x = (int)((uint32_t)p - q * (uint32_t)wo);
                        y = (int)(q % (uint32_t)ho);
                    } else {
                        x = (int)(p % wo);
                        y = (int)((p / wo) % ho);
                    }
                    cls[u] = border_class(y, ho, bc.nlo_h, bc.nhi_h, bc.nrc) * bc.ncc + border_class(x, wo, bc.nlo_w, bc.nhi_w, bc.ncc);
                    v[u] = __ldg(reinterpret_cast<const int4 *>(e3 + p * c_out + ch));
                }
            }
#pragma unroll
            for (int u = 0; u < kTapUnroll; ++u) {
                if (cls[u] == -2) continue;
                const int8_t *b = reinterpret_cast<const int8_t *>(&v[u]);
                if (cls[u] == interior) {
#pragma unroll
                    for (int k = 0; k < 16; ++k) acc[k] += b[k];
                } else {
                    int32_t *dst = cls_acc + cls[u] * kClassSlab + sub * 16;
#pragma unroll
                    for (int k = 0; k < 16; ++k)
                        if (b[k]) atomicAdd(dst + k, (int)b[k]);
                }
            }
        }
        if (interior >= 0) {
            int32_t *dst = cls_acc + interior * kClassSlab + sub * 16;
#pragma unroll
            for (int k = 0; k < 16; ++k)
                if (acc[k]) atomicAdd(dst + k, acc[k]);
        }
    }
    __syncthreads();
    // a tap's sum is the sum over the classes for which the tap falls inside the image: formed here from the
    // block's class sums, one 64-bit atomic per (channel, tap) and block
    const int taps = d.kh * d.kw;
    __shared__ unsigned long long rows_in[32], cols_in[32];  // per filter row / column: the classes it is inside for
    if (threadIdx.x < d.kh) {
        unsigned long long m = 0;
        for (int rc = 0; rc < bc.nrc; ++rc)
            if (tap_valid(rc, threadIdx.x, ho, d.h, bc.nlo_h, bc.nhi_h, bc.nrc, d.stride, d.pad)) m |= 1ull << rc;
        rows_in[threadIdx.x] = m;
    } else if (threadIdx.x >= 32 && threadIdx.x < 32 + d.kw) {
        unsigned long long m = 0;
        for (int cc = 0; cc < bc.ncc; ++cc)
            if (tap_valid(cc, threadIdx.x - 32, wo, d.w, bc.nlo_w, bc.nhi_w, bc.ncc, d.stride, d.pad)) m |= 1ull << cc;
        cols_in[threadIdx.x - 32] = m;
    }
    __syncthreads();
    // consecutive threads take consecutive taps of a channel: neighbouring cells of tap_sums[oc][tap]
    for (int i = threadIdx.x; i < taps * slab_ch; i += blockDim.x) {
        const int c = i / taps, tap = i % taps;
        const unsigned long long cols = cols_in[tap % d.kw];
        long long sum = 0;
        for (unsigned long long rm = rows_in[tap / d.kw]; rm; rm &= rm - 1) {
            const int32_t *row = cls_acc + (__ffsll((long long)rm) - 1) * bc.ncc * kClassSlab + c;
            for (unsigned long long cm = cols; cm; cm &= cm - 1) sum += row[(__ffsll((long long)cm) - 1) * kClassSlab];
        }
        if (sum)
            atomicAdd(reinterpret_cast<unsigned long long *>(tap_sums + (size_t)(by * kClassSlab + c) * taps + tap),
                      (unsigned long long)sum);
    }
}


__global__ void b1_tap_sums_kernel(const int8_t *__restrict__ e3, long long *tap_sums, size_t replica_stride, int c_out, int ho,
                                   int wo, size_t pixels, int pixels_per_block, BorderClasses bc, eoq_conv_desc_t d)
{
    b1_tap_sums_body(e3, tap_sums, replica_stride, c_out, ho, wo, pixels, pixels_per_block, bc, d, (int)blockIdx.x, (int)blockIdx.y);
}

// ------------------------------------------------------------------ weight-gradient finish of many layers at once
// A block finds the layer it works for by its index (first[] holds the first block of every item).
__device__ __forceinline__ int finish_item_of(const int *first, int num, int block)
{
    int k = 0;
    while (k + 1 < num && block >= first[k + 1]) ++k;
    return k;
}

// zeroes what the finish accumulates into: the tap sums of every layer and its maximum cell (one block per layer)
__global__ void finish_zero_kernel(FinishBatch b)
{
    const FinishItem &it = b.item[blockIdx.x];
    int4 *dst = reinterpret_cast<int4 *>(it.tap_sums);
    const size_t n16 = it.zero_bytes / 16;
    for (size_t i = threadIdx.x; i < n16; i += blockDim.x) dst[i] = make_int4(0, 0, 0, 0);
}

__global__ void finish_taps_kernel(FinishBatch b)
{
    const int k = finish_item_of(b.tap_first, b.num, (int)blockIdx.x);
    const FinishItem &it = b.item[k];
    if (!it.b1_dev) return;
    const int local = (int)blockIdx.x - b.tap_first[k];
    b1_tap_sums_body(it.e3, it.tap_sums, (size_t)it.tap_stride, it.d.c_out, it.ho, it.wo, (size_t)it.pixels, it.pixels_per_block, it.bc,
                     it.d, local % it.tap_grid_x, local / it.tap_grid_x);
}

__global__ void finish_sums_kernel(FinishBatch b)
{
    const int k = finish_item_of(b.fin_first, b.num, (int)blockIdx.x);
    const FinishItem &it = b.item[k];
    wgrad_finalize_body(it.parts, it.num_parts, it.groups, (size_t)it.n, it.acc, it.b1_dev ? it.tap_sums : nullptr,
                        (size_t)it.tap_stride, 0, it.b1_dev, it.d.c_in, nullptr, it.max_cell, (int)blockIdx.x - b.fin_first[k],
                        it.fin_blocks);
}

__global__ void finish_code_kernel(FinishBatch b, unsigned *status)
{
    const int k = finish_item_of(b.sq_first, b.num, (int)blockIdx.x);
    const FinishItem &it = b.item[k];
    sq_i64_body(it.acc, it.e3_exp, -7, (size_t)it.n, it.g, it.g_exp, *it.max_cell, status, (int)blockIdx.x - b.sq_first[k],
                it.sq_blocks);
}

}  // namespace

// ------------------------------------------------------------------ launchers

cudaError_t launch_reset_cells(DeviceState *dev, cudaStream_t s)
{
    // every cell after the status word
    return cudaMemsetAsync(reinterpret_cast<char *>(dev) + offsetof(DeviceState, absmax_u32), 0,
                           offsetof(DeviceState, tensor_absmax) - offsetof(DeviceState, absmax_u32), s);
}

cudaError_t launch_quantize_f32(int mode, const float *src, size_t n, void *dst, int32_t *dst_exp, DeviceState *dev,
                                int sm_count, cudaStream_t s, const ReduceHook &hook)
{
    if (mode == 2) {
        absmax_f32_kernel<<<grid_for(n / 4 + 1, sm_count), kThreads, 0, s>>>(src, n, dev);
        hook(&dev->absmax_u32, 1, EOQ_REDUCE_I32, EOQ_REDUCE_MAX, s);  // float bit patterns of |x| order like integers
    }
    quantize_f32_kernel<<<grid_for(n / 16 + 1, sm_count), kThreads, 0, s>>>(mode, src, n, dst, dst_exp, dev);
    return cudaGetLastError();
}

cudaError_t launch_quantize_image(const float *src, int n, int h, int w, int c_src, int c_dst, int wmargin, int8_t *dst,
                                  int32_t *dst_exp, DeviceState *dev, int sm_count, cudaStream_t s, const ReduceHook &hook)
{
    const size_t count = (size_t)n * h * w * c_src;
    absmax_f32_kernel<<<grid_for(count / 4 + 1, sm_count), kThreads, 0, s>>>(src, count, dev);
    hook(&dev->absmax_u32, 1, EOQ_REDUCE_I32, EOQ_REDUCE_MAX, s);
    if (c_dst % 16 == 0) {
        const size_t items = (size_t)n * h * (w + 2 * wmargin) * (c_dst / 16);
        quantize_image_kernel<16><<<grid_for(items, sm_count), kThreads, 0, s>>>(src, n * h, w, c_src, c_dst, wmargin, dst, dst_exp, dev);
    } else {
        const size_t items = (size_t)n * h * (w + 2 * wmargin) * (c_dst / 8);
        quantize_image_kernel<8><<<grid_for(items, sm_count), kThreads, 0, s>>>(src, n * h, w, c_src, c_dst, wmargin, dst, dst_exp, dev);
    }
    return cudaGetLastError();
}

cudaError_t launch_weight_pad_rows(const int8_t *w, int8_t *wp, int c_out, int kh, int kw, int c_in, cudaStream_t s)
{
    const int rows = c_out * kh;
    if (c_in == 16) weight_pad_rows_kernel<int4><<<(rows * 8 + 255) / 256, 256, 0, s>>>(w, wp, rows, kw);
    else weight_pad_rows_kernel<int2><<<(rows * 8 + 255) / 256, 256, 0, s>>>(w, wp, rows, kw);
    return cudaGetLastError();
}

cudaError_t launch_sq_i32(const int32_t *src, const int32_t *src_exp, int exp_bias, size_t n, int8_t *dst,
                          int32_t *dst_exp, long long *sum_codes, bool max_already_reduced, DeviceState *dev,
                          int sm_count, cudaStream_t s, const ReduceHook &hook, const NextHeadArgs *next, const JoinStatArgs *join)
{
    if (!max_already_reduced) absmax_i32_kernel<<<grid_for(n / 4 + 1, sm_count), kThreads, 0, s>>>(src, n, dev);
    hook(&dev->absmax_u32, 1, EOQ_REDUCE_I32, EOQ_REDUCE_MAX, s);
    const int grid = grid_for(n / 16 + 1, sm_count);
    if (join) {
        // (no hook in this form: callers with replicas take the separate calls)
        sq_i32_kernel<false, true><<<grid, kThreads, 0, s>>>(src, src_exp, exp_bias, n, dst, dst_exp, sum_codes, NextHeadArgs{}, *join, dev);
    } else if (next) {
        // (only behind a GEMM whose epilogue reduced the masked maximum)
        hook(&dev->absmax_u64, 1, EOQ_REDUCE_I64, EOQ_REDUCE_MAX, s);
        sq_i32_kernel<true, false><<<grid, kThreads, 0, s>>>(src, src_exp, exp_bias, n, dst, dst_exp, sum_codes, *next, JoinStatArgs{}, dev);
        if (next->sum_e1) hook(next->sum_e1, 1, EOQ_REDUCE_I64, EOQ_REDUCE_SUM, s);
        if (next->sum_e1x2) hook(next->sum_e1x2, 1, EOQ_REDUCE_I64, EOQ_REDUCE_SUM, s);
    } else {
        sq_i32_kernel<false, false><<<grid, kThreads, 0, s>>>(src, src_exp, exp_bias, n, dst, dst_exp, sum_codes, NextHeadArgs{},
                                                              JoinStatArgs{}, dev);
    }
    if (sum_codes) hook(sum_codes, 1, EOQ_REDUCE_I64, EOQ_REDUCE_SUM, s);
    return cudaGetLastError();
}

cudaError_t launch_sq_i32_scatter(const int32_t *src, const int32_t *src_exp, int exp_bias, int n_img, int hh, int ww, int c,
                                  int stride, int hq, int wq, int8_t *dst, int32_t *dst_exp, long long *sum_codes,
                                  DeviceState *dev, int sm_count, cudaStream_t s, const ReduceHook &hook)
{
    const size_t items = (size_t)n_img * hh * ww * (c / 16);
    hook(&dev->absmax_u32, 1, EOQ_REDUCE_I32, EOQ_REDUCE_MAX, s);
    sq_i32_scatter_kernel<<<grid_for(items, sm_count), kThreads, 0, s>>>(src, src_exp, exp_bias, n_img, hh, ww, c, stride, hq, wq,
                                                                        dst, dst_exp, sum_codes, dev);
    if (sum_codes) hook(sum_codes, 1, EOQ_REDUCE_I64, EOQ_REDUCE_SUM, s);
    return cudaGetLastError();
}

cudaError_t launch_sq_i64(const long long *src, const int32_t *src_exp, int exp_bias, size_t n, int8_t *dst,
                          int32_t *dst_exp, long long *copy_out, const long long *tap_sums, size_t replica_stride,
                          int32_t b1_c, const int32_t *b1_dev, int c_in, const int32_t *parts, int num_parts,
                          DeviceState *dev, int sm_count, cudaStream_t s, const ReduceHook &hook)
{
    const int groups = !parts ? 1 : (num_parts >= 32 ? 8 : (num_parts >= 8 ? 4 : 1));
    const int bx = 256 / groups;
    size_t blocks = (n + bx - 1) / bx;
    if (blocks > (size_t)sm_count * 16) blocks = (size_t)sm_count * 16;
    if (hook.fn) {
        // replicas: local sums (b1 term included, it is linear in the error) -> all-reduce -> maximum of the global sums;
        // the copy for the caller is taken from the global sums as well
        wgrad_finalize_kernel<<<(unsigned)blocks, 256, 0, s>>>(parts, num_parts, groups, n, const_cast<long long *>(src), tap_sums,
                                                               replica_stride, b1_c, b1_dev, c_in, nullptr, dev, 1);
        hook(const_cast<long long *>(src), n, EOQ_REDUCE_I64, EOQ_REDUCE_SUM, s);
        absmax_i64_kernel<<<grid_for(n, sm_count, 4), kThreads, 0, s>>>(src, n, dev);
        if (copy_out) cudaMemcpyAsync(copy_out, src, n * sizeof(long long), cudaMemcpyDeviceToDevice, s);
    } else {
        wgrad_finalize_kernel<<<(unsigned)blocks, 256, 0, s>>>(parts, num_parts, groups, n, const_cast<long long *>(src), tap_sums,
                                                               replica_stride, b1_c, b1_dev, c_in, copy_out, dev, 0);
    }
    sq_i64_kernel<<<grid_for(n, sm_count, 4), kThreads, 0, s>>>(src, src_exp, exp_bias, n, dst, dst_exp, dev);
    return cudaGetLastError();
}

cudaError_t launch_err_prescale(const int8_t *e0, const int32_t *e0_exp, const uint8_t *mask, const int16_t *x2,
                                size_t n_el, int32_t gamma_c, const int32_t *gamma_dev, int8_t *e3, int32_t *e3_exp,
                                long long *sum_e1, long long *sum_e1x2, DeviceState *dev, int sm_count, cudaStream_t s,
                                int *kernels, bool force_timeout, const ReduceHook &hook)
{
    const size_t n16 = n_el / 16;
    *kernels = 2;
    // one cooperative kernel when every thread can hold its share of the tensor between the two passes
    static int blocks_per_sm = -1;
    static bool coop = false;
    if (blocks_per_sm < 0) {
        int dev_id = 0, can = 0, bps = 0;
        if (cudaGetDevice(&dev_id) == cudaSuccess &&
            cudaDeviceGetAttribute(&can, cudaDevAttrCooperativeLaunch, dev_id) == cudaSuccess && can &&
            cudaOccupancyMaxActiveBlocksPerMultiprocessor(&bps, prescale_fused_kernel, kThreads, 0) == cudaSuccess && bps > 0) {
            coop = true;
            blocks_per_sm = bps > 4 ? 4 : bps;  // leaves room on every SM for kernels of other streams
        } else {
            blocks_per_sm = 0;
        }
    }
    const size_t max_blocks = (size_t)blocks_per_sm * sm_count;
    const size_t need_blocks = (n16 + (size_t)kThreads * kFusedGroups - 1) / ((size_t)kThreads * kFusedGroups);
    if (coop && !hook.fn && n16 > 0 && need_blocks <= max_blocks) {
        // self-test of the bounded wait: one arrival more than there are blocks and a short limit
        unsigned expected = (unsigned)need_blocks + (force_timeout ? 1u : 0u);
        uint32_t spin_limit = force_timeout ? 2048u : kSpinLimit;
        void *args[] = {(void *)&e0, (void *)&e0_exp, (void *)&mask, (void *)&x2, (void *)&n16, (void *)&gamma_c,
                        (void *)&gamma_dev, (void *)&e3, (void *)&e3_exp, (void *)&sum_e1, (void *)&sum_e1x2, (void *)&dev,
                        (void *)&expected, (void *)&spin_limit};
        const cudaError_t e = cudaLaunchCooperativeKernel((const void *)prescale_fused_kernel, dim3((unsigned)need_blocks),
                                                          dim3(kThreads), args, 0, s);
        if (e != cudaErrorCooperativeLaunchTooLarge) {
            *kernels = 1;
            return e;
        }
        (void)cudaGetLastError();  // fewer SMs at hand than at start-up (e.g. a partitioned device): two kernels instead
    }
    prescale_reduce_kernel<<<grid_for(n16, sm_count), kThreads, 0, s>>>(e0, mask, x2, n16, dev);
    hook(&dev->absmax_u32, 1, EOQ_REDUCE_I32, EOQ_REDUCE_MAX, s);
    hook(&dev->sum0, 2, EOQ_REDUCE_I64, EOQ_REDUCE_SUM, s);  // sum0 and sum1 are adjacent
    prescale_apply_kernel<<<grid_for(n16, sm_count), kThreads, 0, s>>>(e0, e0_exp, mask, n16, gamma_c, gamma_dev, e3,
                                                                       e3_exp, sum_e1, sum_e1x2, dev);
    return cudaGetLastError();
}

cudaError_t launch_update(const UpdateTensor *t, int num, int32_t lr_mant, int32_t lr_exp, int stochastic,
                          uint64_t seed, uint64_t step, unsigned long long *step_dev, DeviceState *dev, int sm_count,
                          cudaStream_t s)
{
    (void)sm_count;
    cudaError_t e = cudaMemsetAsync(dev->tensor_absmax, 0, sizeof(unsigned) * 256, s);
    if (e != cudaSuccess) return e;
    for (int base = 0; base < num; base += kUpdChunk) {
        UpdateBatch b;
        b.num = num - base < kUpdChunk ? num - base : kUpdChunk;
        b.tensor_base = base;
        int blocks = 0;
        for (int k = 0; k < b.num; ++k) {
            b.t[k] = t[base + k];
            b.first_block[k] = blocks;
            blocks += (int)((t[base + k].n + kUpdElemsPerBlock - 1) / kUpdElemsPerBlock);
        }
        b.first_block[b.num] = blocks;
        if (blocks == 0) continue;
        update_absmax_kernel<<<blocks, kThreads, 0, s>>>(b, dev);
    }
    for (int base = 0; base < num; base += kUpdChunk) {
        UpdateBatch b;
        b.num = num - base < kUpdChunk ? num - base : kUpdChunk;
        b.tensor_base = base;
        int blocks = 0;
        for (int k = 0; k < b.num; ++k) {
            b.t[k] = t[base + k];
            b.first_block[k] = blocks;
            blocks += (int)((t[base + k].n + kUpdElemsPerBlock - 1) / kUpdElemsPerBlock);
        }
        b.first_block[b.num] = blocks;
        if (blocks == 0) continue;
        update_apply_kernel<<<blocks, kThreads, 0, s>>>(b, lr_mant, lr_exp, stochastic, seed, step, step_dev, dev);
    }
    if (step_dev) step_bump_kernel<<<1, 1, 0, s>>>(step_dev);
    return cudaGetLastError();
}

cudaError_t launch_update_wide(const UpdateTensor *t, int num, int32_t lr_mant, int32_t lr_exp, int k_u, int k_m, int stochastic,
                               uint64_t seed, uint64_t step, unsigned long long *step_dev, DeviceState *dev, cudaStream_t s)
{
    cudaError_t e = cudaMemsetAsync(dev->tensor_absmax, 0, sizeof(unsigned) * 256, s);
    if (e != cudaSuccess) return e;
    for (int pass = 0; pass < 2; ++pass)
        for (int base = 0; base < num; base += kUpdChunk) {
            UpdateBatch b;
            b.num = num - base < kUpdChunk ? num - base : kUpdChunk;
            b.tensor_base = base;
            int blocks = 0;
            for (int k = 0; k < b.num; ++k) {
                b.t[k] = t[base + k];
                b.first_block[k] = blocks;
                blocks += (int)((t[base + k].n + kUpdElemsPerBlock - 1) / kUpdElemsPerBlock);
            }
            b.first_block[b.num] = blocks;
            if (blocks == 0) continue;
            if (pass == 0) update_absmax_kernel<<<blocks, kThreads, 0, s>>>(b, dev);
            else update_wide_apply_kernel<<<blocks, kThreads, 0, s>>>(b, lr_mant, lr_exp, k_u, k_m, stochastic, seed, step, step_dev, dev);
        }
    if (step_dev) step_bump_kernel<<<1, 1, 0, s>>>(step_dev);
    return cudaGetLastError();
}

cudaError_t launch_layout_convert(const int8_t *src, int8_t *dst, int n, int c, int h, int w, int to_nhwc,
                                  cudaStream_t s)
{
    // NCHW is [n][c][hw]; NHWC is [n][hw][c]
    const int rows = to_nhwc ? c : h * w, cols = to_nhwc ? h * w : c;
    dim3 grid((cols + 31) / 32, (rows + 31) / 32, n), block(32, 8);
    transpose_bytes_kernel<<<grid, block, 0, s>>>(src, dst, rows, cols);
    return cudaGetLastError();
}

cudaError_t launch_weight_transpose(const int8_t *w, int8_t *wt, int c_out, int taps, int c_in, cudaStream_t s)
{
    const size_t total = (size_t)c_out * taps * c_in;
    int blocks = (int)((total + kThreads - 1) / kThreads);
    if (blocks > 148 * 16) blocks = 148 * 16;
    weight_transpose_kernel<<<blocks, kThreads, 0, s>>>(w, wt, c_out, taps, c_in);
    return cudaGetLastError();
}

cudaError_t launch_b1_weight_table(const int8_t *w, int32_t *table, const eoq_conv_desc_t &d, const BorderClasses &bc,
                                   cudaStream_t s)
{
    const int ho = (d.h + 2 * d.pad - d.kh) / d.stride + 1, wo = (d.w + 2 * d.pad - d.kw) / d.stride + 1;
    b1_weight_table_kernel<<<d.c_out, 128, 0, s>>>(w, table, d, ho, wo, bc);
    return cudaGetLastError();
}

cudaError_t launch_weight_prep(const PrepBatch &b, cudaStream_t s)
{
    weight_prep_kernel<<<b.first_block[b.num], 128, 0, s>>>(b);
    return cudaGetLastError();
}

cudaError_t launch_b1_error_sums(const int8_t *e3, long long *tap_sums, size_t replica_stride, const eoq_conv_desc_t &d, int ho,
                                 int wo, const BorderClasses &bc, int sm_count, cudaStream_t s)
{
    // tap_sums was zeroed by the caller
    const int classes = bc.nrc * bc.ncc;
    const size_t pixels = (size_t)d.n * ho * wo;
    const int slabs = (d.c_out + kClassSlab - 1) / kClassSlab;
    int blocks = (sm_count + slabs - 1) / slabs;  // more blocks only add atomics on the per-tap cells
    size_t ppb = (pixels + blocks - 1) / blocks;
    if (ppb < 64) ppb = 64;
    if (ppb > (1u << 23)) ppb = 1u << 23;  // keeps the int32 class sums exact
    blocks = (int)((pixels + ppb - 1) / ppb);
    dim3 grid(blocks, slabs);
    b1_tap_sums_kernel<<<grid, 256, sizeof(int32_t) * classes * kClassSlab, s>>>(e3, tap_sums, replica_stride, d.c_out, ho, wo,
                                                                               pixels, (int)ppb, bc, d);
    return cudaGetLastError();
}

void plan_finish_item(FinishItem &it, int sm_count)
{
    // the b1 error sums: as launch_b1_error_sums lays them out
    const int slabs = (it.d.c_out + kClassSlab - 1) / kClassSlab;
    int blocks = (sm_count + slabs - 1) / slabs;
    size_t ppb = ((size_t)it.pixels + blocks - 1) / blocks;
    if (ppb < 64) ppb = 64;
    if (ppb > (1u << 23)) ppb = 1u << 23;
    it.pixels_per_block = (int)ppb;
    it.tap_grid_x = (int)(((size_t)it.pixels + ppb - 1) / ppb);
    it.tap_grid_y = slabs;
    // slice sums and codes: as launch_sq_i64 sizes them, with a smaller cap (many tensors share the device)
    it.groups = !it.parts ? 1 : (it.num_parts >= 32 ? 8 : (it.num_parts >= 8 ? 4 : 1));
    const int bw = 256 / it.groups;
    size_t fb = ((size_t)it.n + bw - 1) / bw;
    if (fb > (size_t)sm_count * 4) fb = (size_t)sm_count * 4;
    it.fin_blocks = (int)(fb < 1 ? 1 : fb);
    size_t qb = ((size_t)it.n / 4 + kThreads - 1) / kThreads;
    if (qb > (size_t)sm_count * 2) qb = (size_t)sm_count * 2;
    it.sq_blocks = (int)(qb < 1 ? 1 : qb);
}

cudaError_t launch_wgrad_finish(const FinishBatch &b, unsigned *status, cudaStream_t s)
{
    int max_classes = 1;
    for (int k = 0; k < b.num; ++k) {
        const int c = b.item[k].bc.nrc * b.item[k].bc.ncc;
        if (b.item[k].b1_dev && c > max_classes) max_classes = c;
    }
    const size_t smem = sizeof(int32_t) * max_classes * kClassSlab;
    if (smem > 48 * 1024) {
        cudaError_t e = cudaFuncSetAttribute(finish_taps_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
    }
    finish_zero_kernel<<<b.num, 256, 0, s>>>(b);
    finish_taps_kernel<<<b.tap_first[b.num], 256, smem, s>>>(b);
    finish_sums_kernel<<<b.fin_first[b.num], 256, 0, s>>>(b);
    finish_code_kernel<<<b.sq_first[b.num], kThreads, 0, s>>>(b, status);
    return cudaGetLastError();
}

}  // namespace eoq
