// A consumer's error head riding on the second pass of the kernel that produces its input error.
#pragma once
#include "eoq_device.cuh"
#include "eoq_internal.h"

namespace eoq {

// The error head of a layer (e1 = e * [x4 > 0], e3 = Q_e(gamma * e1), sum of e1, sum of e1 * x2) can ride on the second
// pass of the kernel that produces e: Q_e is monotonic in |.|, so max |e1| is the code of the largest masked |sum|, which
// the producer's first pass reduces beside its own maximum.  NextHead holds what the second pass needs.
struct NextHead {
    uint32_t g;         // gamma code
    float scale, rest;  // R(gamma * e1 * 2^(7 - t3)) = one fused multiply-add (see prescale_apply_kernel)
    uint32_t M3;        // max |gamma * e1|
    int t3;
};
constexpr uint32_t kHeadMagic = 0x4B400000u;  // 1.5 * 2^23

__device__ __forceinline__ NextHead next_head_setup(const int32_t *gamma_dev, uint32_t max_e1, DeviceState *dev)
{
    int gamma = __ldg(gamma_dev);
    if (gamma < -32768 || gamma > 32767) {
        if (blockIdx.x == 0 && threadIdx.x == 0) atomicOr(&dev->status, EOQ_DEV_RANGE);
        gamma = gamma < 0 ? -32768 : 32767;
    }
    NextHead nh;
    nh.g = (uint32_t)gamma;
    nh.M3 = max_e1 * (uint32_t)abs(gamma);
    nh.t3 = nh.M3 ? round_log2_u32(nh.M3) : 7;
    nh.scale = __int_as_float((127 + 7 - nh.t3) << 23);
    nh.rest = 12582912.0f - 12582912.0f * nh.scale;
    return nh;
}

__device__ __forceinline__ int next_head_code(const NextHead &nh, int e1)
{
    const uint32_t biased = nh.g * (uint32_t)e1 + kHeadMagic;
    const int v = (int)(__float_as_uint(__fmaf_rn(__uint_as_float(biased), nh.scale, nh.rest)) - kHeadMagic);
    return v < -127 ? -127 : (v > 127 ? 127 : v);
}

// exponent of e3 given the exponent p0 of e (the head sees e at p0 - 7 after the multiplication by gamma's grid)
__device__ __forceinline__ void next_head_exponent(const NextHead &nh, int p0, int32_t *e3_exp, DeviceState *dev)
{
    *e3_exp = nh.M3 ? p0 - 7 + nh.t3 - 7 : p0 - 7;
    if (!nh.M3) atomicOr(&dev->status, EOQ_DEV_SQ_ZERO);
}


// Join of two error streams: both at the smaller exponent, added exactly; an operand more than 31 octaves below the
// other is dropped.
struct JoinShift {
    int sa, sb, p;  // left shifts of the two operands (-1: operand dropped) and the exponent of the sums
};
__device__ __forceinline__ JoinShift join_shift(int pa, int pb)
{
    JoinShift j;
    const int p = min(pa, pb);
    j.sa = pa - p;
    j.sb = pb - p;
    j.p = p;
    if (j.sa > 31) { j.sb = -1; j.sa = 0; j.p = pa; }        // b lies more than 31 octaves below a
    else if (j.sb > 31) { j.sa = -1; j.sb = 0; j.p = pb; }
    return j;
}
__device__ __forceinline__ long long join_one(int a, int b, const JoinShift &j)
{
    const long long va = j.sa < 0 ? 0ll : (long long)a * (1ll << j.sa);
    const long long vb = j.sb < 0 ? 0ll : (long long)b * (1ll << j.sb);
    return va + vb;
}

}  // namespace eoq
