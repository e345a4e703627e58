// Pieces shared by the two implicit-GEMM kernels: bounded barrier waits and the register epilogues of the
// forward chain and of error back-propagation (arXiv 2105.13890, Sec. 3.2.1).
#pragma once
#include "eoq_device.cuh"
#include "eoq_internal.h"

namespace eoq {

struct RoleCtx {
    volatile uint32_t *abort_flag;
    DeviceState *dev;
};

// Bounded wait on an mbarrier phase.  Every polling warp takes issue slots from the warp that feeds the tensor
// core (one thread, whose scalar work between two MMAs is on the critical path), so waiters that can afford a
// few dozen nanoseconds of extra latency (loaders, epilogue) back off between polls; the MMA issuer does not.
template <int kBackoffNs = 0>
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, const RoleCtx &c)
{
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (ptx::mbar_try_wait(bar, parity)) return true;
        if (*c.abort_flag) return false;
        if (kBackoffNs > 0) __nanosleep(kBackoffNs);
    }
    *c.abort_flag = 1u;
    atomicOr(&c.dev->status, EOQ_DEV_TIMEOUT);
    return false;
}

__device__ __forceinline__ uint32_t pack4(int a, int b, int c, int d)
{
    return (uint32_t)(a & 0xff) | ((uint32_t)(b & 0xff) << 8) | ((uint32_t)(c & 0xff) << 16) | ((uint32_t)(d & 0xff) << 24);
}

// R(a / 2^7) with ties to even in four integer operations: adding 63 plus the parity of the quotient carries
// into bit 7 exactly when the remainder exceeds one half, or equals it with an odd quotient.
__device__ __forceinline__ int32_t rne7(int32_t a) { return (a + 63 + ((a >> 7) & 1)) >> 7; }

// Forward chain on 16 consecutive output channels of one pixel (Sec. 3.2.1: x2 = Q_a1(conv), x3 = gamma x2,
// x4 = x3 + b2 [+ shortcut], x5 = Q_a2(relu(x4)); mask = [x4 > 0]).  kShift7: the input sits at exponent -7.
template <bool kShift7>
__device__ __forceinline__ void forward_16(const IgemmParams &p, const uint32_t *acc, size_t off, int col, int cls,
                                           int shift)
{
    int32_t a[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) a[i] = (int32_t)acc[i];
    if (p.b1_table) {
        const int4 *t = reinterpret_cast<const int4 *>(p.b1_table + (size_t)cls * p.N + col);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int4 v = __ldg(t + i);
            a[4 * i + 0] += p.b1_c * v.x;
            a[4 * i + 1] += p.b1_c * v.y;
            a[4 * i + 2] += p.b1_c * v.z;
            a[4 * i + 3] += p.b1_c * v.w;
        }
    }
    if (p.acc_out) {
        int4 *d = reinterpret_cast<int4 *>(p.acc_out + off);
#pragma unroll
        for (int i = 0; i < 4; ++i) d[i] = make_int4(a[4 * i], a[4 * i + 1], a[4 * i + 2], a[4 * i + 3]);
    }
    int32_t add[16];  // (b2 + shortcut) * 2^7, the part of x4 that does not depend on the accumulator
    const int32_t b2s = p.b2_c << 7;
    if (p.shortcut) {
        const int4 v = __ldg(reinterpret_cast<const int4 *>(p.shortcut + off));
        const int8_t *b = reinterpret_cast<const int8_t *>(&v);
#pragma unroll
        for (int i = 0; i < 16; ++i) add[i] = b2s + ((int32_t)b[i] << 7);
    } else {
#pragma unroll
        for (int i = 0; i < 16; ++i) add[i] = b2s;
    }
    uint32_t mbits = 0;
    const int32_t lo = p.relu ? 0 : -127 * 128 - 64;  // below this Q_a2 saturates at -127 anyway
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        int32_t v2;
        if (kShift7) {
            v2 = rne7(a[i]);
        } else if (shift >= 0) {
            v2 = rne_shr32(a[i], shift);
        } else {
            const long long w = (long long)a[i] << (-shift);
            v2 = (int32_t)(w < -32768 ? -32768 : (w > 32767 ? 32767 : w));
        }
        v2 = clampi(v2, -32768, 32767);
        a[i] = v2;
        const int32_t v4 = p.gamma_c * v2 + add[i];
        mbits |= (v4 > 0 ? 1u : 0u) << i;
        add[i] = min(rne7(max(v4, lo)), 127);
    }
    if (!p.relu) {
#pragma unroll
        for (int i = 0; i < 16; ++i) add[i] = max(add[i], -127);
    }
    int4 o;
    o.x = (int)pack4(add[0], add[1], add[2], add[3]);
    o.y = (int)pack4(add[4], add[5], add[6], add[7]);
    o.z = (int)pack4(add[8], add[9], add[10], add[11]);
    o.w = (int)pack4(add[12], add[13], add[14], add[15]);
    *reinterpret_cast<int4 *>(p.x5 + off) = o;
    if (p.relu_mask) *reinterpret_cast<uint16_t *>(p.relu_mask + (off >> 3)) = (uint16_t)mbits;
    if (p.x2) {
        int4 *d = reinterpret_cast<int4 *>(p.x2 + off);
        d[0] = make_int4((a[0] & 0xffff) | (a[1] << 16), (a[2] & 0xffff) | (a[3] << 16), (a[4] & 0xffff) | (a[5] << 16),
                         (a[6] & 0xffff) | (a[7] << 16));
        d[1] = make_int4((a[8] & 0xffff) | (a[9] << 16), (a[10] & 0xffff) | (a[11] << 16),
                         (a[12] & 0xffff) | (a[13] << 16), (a[14] & 0xffff) | (a[15] << 16));
    }
}

// Error back-propagation: keep the exact int32 sums (the scale quantizer needs the maximum over the whole
// tensor before any element can be coded) and track max |.|.
__device__ __forceinline__ uint32_t dgrad_16(const IgemmParams &p, const uint32_t *acc, size_t off)
{
    uint32_t mx = 0;
    int4 *d = reinterpret_cast<int4 *>(p.acc_out + off);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        int4 v = make_int4((int)acc[4 * i], (int)acc[4 * i + 1], (int)acc[4 * i + 2], (int)acc[4 * i + 3]);
        mx = max(mx, (uint32_t)abs(v.x));
        mx = max(mx, (uint32_t)abs(v.y));
        mx = max(mx, (uint32_t)abs(v.z));
        mx = max(mx, (uint32_t)abs(v.w));
        d[i] = v;
    }
    return mx;
}

}  // namespace eoq
